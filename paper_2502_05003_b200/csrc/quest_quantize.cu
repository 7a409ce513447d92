// Fused QuEST forward quantizer for sm_100a: Hadamard rotation (Eq. 2) -> RMS normalisation ->
// alpha*(b) clip -> round onto Eq. 1's grid -> packed codes, per-row scale, trust mask
// (Section 3.1 and 3.2; the rotation and projection steps of Algorithm 1).
//
// Every rounding decision is taken in binary32 with one IEEE rounding per operation, in this
// order: butterflies (a,b) -> (a+b, a-b) with DESCENDING stride g/2 .. 1; squares rounded, then
// pairwise summation over adjacent elements of the zero-padded row; rms = sqrt(ss/d);
// inv = A/rms; t = fma(u, inv, c0); level = rint(clamp(t, 0, 2^b-1)) (ties to even);
// trusted = |t - level| <= trust_factor/2.  This file is compiled with -fmad=false and uses
// the explicit _rn intrinsics so that the compiler cannot fuse or reorder any of it.
#include <cuda_bf16.h>

#include "quest_internal.cuh"
#include "quest_operand.cuh"

namespace quest {

QuantConsts make_quant_consts_fp4(int had_block, float trust_factor) {
    QuantConsts c;
    const float alpha = alpha_star_fp4();
    c.c0 = 0.0f;
    c.top = 6.0f;
    c.A = 6.0f / alpha;                                   // RMS-normalised value -> E2M1 value axis
    c.B = alpha / (6.0f * sqrtf((float)had_block));
    c.h = trust_factor;                                   // largest half-interval of the grid: 1 value unit
    return c;
}

QuantConsts make_quant_consts(int bits, int had_block, float trust_factor) {
    QuantConsts c;
    const int L1 = (1 << bits) - 1;
    const float alpha = alpha_star(bits);
    c.c0 = 0.5f * (float)L1;
    c.top = (float)L1;
    c.A = (float)L1 / (2.0f * alpha);
    c.B = alpha / ((float)L1 * sqrtf((float)had_block));
    c.h = 0.5f * trust_factor;
    return c;
}

namespace {

__device__ __forceinline__ float load_elem(const void *x, int dtype, int64_t idx) {
    if (dtype == QUEST_F32) return reinterpret_cast<const float *>(x)[idx];
    const uint32_t w = (uint32_t) reinterpret_cast<const uint16_t *>(x)[idx] << 16;
    return __uint_as_float(w);
}

// Round one rotated element: returns the level and whether it is trusted.
__device__ __forceinline__ int round_level(float u, float inv, const QuantConsts &qc, bool &trusted) {
    const float t = __fmaf_rn(u, inv, qc.c0);
    const float tc = fminf(fmaxf(t, 0.0f), qc.top);
    const float kf = rintf(tc);
    trusted = fabsf(__fsub_rn(t, kf)) <= qc.h;
    return (int)kf;
}

// ---------------------------------------------------------------------------------------------
// Generic kernel: one CTA per row, the row staged in shared memory as binary32.  Handles every
// supported (cols, had_block, bits, dtype); used when cols is not a multiple of 32.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
quantize_generic_kernel(const void *__restrict__ x, int dtype, int64_t rows, int cols, int64_t ld,
                        int bits, int had_block, QuantConsts qc, int p2,
                        uint8_t *__restrict__ codes, float *__restrict__ scales,
                        uint8_t *__restrict__ mask, int8_t *__restrict__ op8) {
    extern __shared__ float smem_f[];
    pdl_launch_dependents();
    pdl_wait();
    float *u = smem_f;
    float *tmp = smem_f + cols;
    __shared__ float s_inv;
    const int tid = threadIdx.x, nt = blockDim.x;
    const int cb = container_bits(bits);
    const int L1 = (1 << bits) - 1;

    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
        for (int e = tid; e < cols; e += nt) u[e] = load_elem(x, dtype, row * ld + e);
        __syncthreads();
        // rotation: butterflies with descending stride; a stride-h stage touches pairs (i, i+h)
        for (int h = had_block >> 1; h >= 1; h >>= 1) {
            for (int idx = tid; idx < (cols >> 1); idx += nt) {
                const int i = ((idx / h) * 2 * h) + (idx % h);
                const float a = u[i], b = u[i + h];
                u[i] = __fadd_rn(a, b);
                u[i + h] = __fsub_rn(a, b);
            }
            __syncthreads();
        }
        // sum of squares: pairwise over adjacent elements of the zero-padded row
        for (int e = tid; e < p2; e += nt) tmp[e] = (e < cols) ? __fmul_rn(u[e], u[e]) : 0.0f;
        __syncthreads();
        for (int s = 1; s < p2; s <<= 1) {
            for (int idx = tid; idx < p2 / (2 * s); idx += nt) {
                const int p = idx * 2 * s;
                tmp[p] = __fadd_rn(tmp[p], tmp[p + s]);
            }
            __syncthreads();
        }
        if (tid == 0) {
            const float rms = __fsqrt_rn(__fdiv_rn(tmp[0], (float)cols));
            s_inv = (rms > 0.0f) ? __fdiv_rn(qc.A, rms) : 0.0f;
            if (scales) scales[row] = __fmul_rn(rms, qc.B);
        }
        __syncthreads();
        const float inv = s_inv;
        for (int grp = tid; grp < (cols >> 3); grp += nt) {
            uint64_t packed = 0;
            uint32_t mbits = 0;
            int8_t v8[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                bool trusted;
                const int k = round_level(u[grp * 8 + j], inv, qc, trusted);
                packed |= (uint64_t)k << (j * cb);
                mbits |= (trusted ? 1u : 0u) << j;
                v8[j] = (int8_t)(bits == 8 ? k - 128 : (2 * k - L1) << (7 - bits));   // see quest_operand.cuh
            }
            if (codes) {
                uint8_t *cr = codes + row * (int64_t)(cols * cb / 8) + (int64_t)grp * cb;
                for (int i = 0; i < cb; ++i) cr[i] = (uint8_t)(packed >> (8 * i));
            }
            if (mask) mask[row * (int64_t)(cols / 8) + grp] = (uint8_t)mbits;
            if (op8) {
                int8_t *o = op8 + row * (int64_t)cols + grp * 8;
#pragma unroll
                for (int j = 0; j < 8; ++j) o[j] = v8[j];
            }
        }
        __syncthreads();
    }
}


// ---------------------------------------------------------------------------------------------
// Row kernel: every thread owns E CONTIGUOUS elements of a row (E = 64 or 32, cols % E == 0),
// held as E/2 float2 pairs so that most of the arithmetic runs on the packed binary32 pipe
// (two IEEE operations per instruction, each rounded exactly like the scalar form).
//   * butterflies whose partner is in another warp (stride >= 32 E) go through shared memory,
//     strides E .. 16 E through warp shuffles, strides E/2 .. 1 stay in registers -- descending
//     stride overall, which is the canonical order;
//   * the sum of squares is reduced pairwise in the thread, then over lanes, then over warps;
//   * rounding, the trust test and the packing work on groups of 32 elements, so each thread
//     stores whole words: 4 bytes of mask, 32*container/8 bytes of codes, 32 operand bytes;
//   * the int8 GEMM operand is derived from the packed code words (quest_operand.cuh).
// A row of T = cols/E threads occupies S slots of the CTA: the next power of two if T < 32, else
// T rounded up to whole warps; slots past T carry zeros, which is the zero padding of the
// canonical pairwise sum.  One launch can serve two tensors of the same row length (x and w of a
// linear layer): the first `blocks0` CTAs work on tensor 0, the rest on tensor 1.
// ---------------------------------------------------------------------------------------------
#define QUEST_MAGIC_RNE 12582912.0f            /* 1.5 * 2^23: x + MAGIC rounds x to an integer (ties to even) */
#define QUEST_MAGIC_BITS 0x4B400000u

struct QuantTensor {
    const void *x;
    long long rows;
    long long ld;
    uint8_t *codes;
    float *scales;
    uint8_t *mask;
    int8_t *op8;
    int32_t *rowsum;       // sum of the row's operand bytes (needed by the GEMM for 8-bit codes)
    uint16_t *rot;         // bfloat16 of the orthonormal rotation itself (weight-only variant)
    uint16_t *cbf;         // grid values c = 2k - (2^b - 1) as bfloat16 (weight-only variant)
};
constexpr int MAX_QUANT_TENSORS = 4;   // tensors one launch of the block kernel can serve (the other kernels: two)
struct QuantArgs {
    QuantTensor t[MAX_QUANT_TENSORS];
    int bend[MAX_QUANT_TENSORS];        // block kernel: CTAs [bend[j-1], bend[j]) work on tensor j
    int blocks0;
    int cols, bits, had_block;
    QuantConsts qc;
    float inv_sqrt_g;      // 1 / sqrt(had_block) in binary32
    int S, R;
};

// Eight positions on the E2M1 value axis -> eight 4-bit codes in one word (element 0 in the low
// nibble), rounded to nearest even and saturated by the hardware conversion.
__device__ __forceinline__ uint32_t cvt_e2m1x8(const float (&t)[8]) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .b8 b0, b1, b2, b3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n\t"
        "mov.b32 %0, {b0, b1, b2, b3};\n\t}"
        : "=r"(out)
        : "f"(t[0]), "f"(t[1]), "f"(t[2]), "f"(t[3]), "f"(t[4]), "f"(t[5]), "f"(t[6]), "f"(t[7]));
    return out;
}

// Everything after the load: rotation from stride s_start downwards (larger strides already
// applied by the caller), RMS, projection, trust test, packing and stores for the E elements this
// thread holds.  GFULL: had_block >= E, so every in-register stage runs.  FAST: the common case
// fixed at compile time -- had_block = 128 with the first stage already applied, rows of at least
// one warp, codes, scales and mask requested (the GEMM operand and the bfloat16 outputs of the
// weight-only variant are optional; a tensor may also ask for the rotation alone), no row sums,
// trust_factor >= 1 -- so that no per-row loop and only a few uniform branches remain.
// CS, CCOLS: threads per row and row length when the kernel is instantiated for one row length (0 = run-time values).
template <int CB, int E, bool GFULL, bool FAST, int GRID = GRID_UNIFORM, bool XDONE = false, bool RS = false, int CS = 0, int CCOLS = 0>
__device__ __forceinline__ void rotate_project_store(float2 (&v)[E / 2], const QuantArgs &a, const QuantTensor &tn,
                                                     bool active, long long row, int tr, int r_local, float *xsm,
                                                     int s_start) {
    constexpr int H = E / 2;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int nthreads = blockDim.x;
    const int S = CS ? CS : a.S;
    const int cols = CCOLS ? CCOLS : a.cols;
    const int had_block = a.had_block;
    // ---- rotation, descending stride --------------------------------------------------------
    const float2 neg1 = make_float2(-1.0f, -1.0f);
    for (int s = FAST ? 0 : s_start; s >= 32 * E; s >>= 1) {  // partner thread is in another warp
        const int dist = s / E;
        float2 *x2 = reinterpret_cast<float2 *>(xsm);
        __syncthreads();
#pragma unroll
        for (int i = 0; i < H; ++i) x2[i * nthreads + tid] = v[i];
        __syncthreads();
        const float sg = (tid & dist) ? -1.0f : 1.0f;
        const float2 sgn = make_float2(sg, sg);
        const int pt = tid ^ dist;
#pragma unroll
        for (int i = 0; i < H; ++i) v[i] = __ffma2_rn(v[i], sgn, x2[i * nthreads + pt]);
    }
    if constexpr (XDONE) {
        // the caller has applied every stride that pairs this thread with another one
    } else if constexpr (FAST) {
        if constexpr (E == 32) {                               // stride 32: partner is the neighbouring lane
            const float sg = (lane & 1) ? -1.0f : 1.0f;
            const float2 sgn = make_float2(sg, sg);
#pragma unroll
            for (int i = 0; i < H; ++i) {
                float2 p;
                p.x = __shfl_xor_sync(0xffffffffu, v[i].x, 1);
                p.y = __shfl_xor_sync(0xffffffffu, v[i].y, 1);
                v[i] = __ffma2_rn(v[i], sgn, p);
            }
        }
    } else {
        int s0 = s_start;
        if (s0 > 16 * E) s0 = 16 * E;
#pragma unroll 1
        for (int s = s0; s >= E; s >>= 1) {                    // partner thread is a lane of this warp
            const int dist = s / E;
            const float sg = (lane & dist) ? -1.0f : 1.0f;
            const float2 sgn = make_float2(sg, sg);
#pragma unroll
            for (int i = 0; i < H; ++i) {
                float2 p;
                p.x = __shfl_xor_sync(0xffffffffu, v[i].x, dist);
                p.y = __shfl_xor_sync(0xffffffffu, v[i].y, dist);
                v[i] = __ffma2_rn(v[i], sgn, p);               // own * (+-1) + partner: one rounding
            }
        }
    }
#pragma unroll
    for (int s = E / 2; s >= 2; s >>= 1) {                     // partner element is in this thread
        if (GFULL || s < had_block) {
            const int s2 = s >> 1;
#pragma unroll
            for (int i = 0; i < H; ++i)
                if ((i & s2) == 0) {
                    const float2 p = v[i], q = v[i + s2];
                    v[i] = __fadd2_rn(p, q);
                    v[i + s2] = __ffma2_rn(q, neg1, p);        // p - q
                }
        }
    }
    if (GFULL || had_block > 1) {
#pragma unroll
        for (int i = 0; i < H; ++i) {
            const float p = v[i].x, q = v[i].y;
            v[i] = make_float2(__fadd_rn(p, q), __fsub_rn(p, q));
        }
    }

    // ---- the rotation itself as an output (weight-only variant): x_h = bf16(u / sqrt(g)) -----
    {
        if (tn.rot) {                                           // uniform over the CTA
            if (active) {
                const float2 ig = make_float2(a.inv_sqrt_g, a.inv_sqrt_g);
                uint4 *dst = reinterpret_cast<uint4 *>(tn.rot + row * (long long)cols + (long long)tr * E);
#pragma unroll
                for (int q = 0; q < E / 8; ++q) {
                    uint32_t o[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float2 p = __fmul2_rn(v[q * 4 + j], ig);
                        const __nv_bfloat162 h = __floats2bfloat162_rn(p.x, p.y);
                        o[j] = *reinterpret_cast<const uint32_t *>(&h);
                    }
                    dst[q] = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
            if (!tn.codes && !tn.scales && !tn.mask && !tn.op8 && !tn.rowsum && !tn.cbf) return;   // nothing else asked for
        }
    }

    // ---- sum of squares: pairwise over adjacent elements, zero-padded row --------------------
    float ss;
    {
        float q[H];
#pragma unroll
        for (int i = 0; i < H; ++i) {
            const float2 sq = __fmul2_rn(v[i], v[i]);
            q[i] = __fadd_rn(sq.x, sq.y);
        }
#pragma unroll
        for (int n = H / 2; n >= 1; n >>= 1)
#pragma unroll
            for (int i = 0; i < n; ++i) q[i] = __fadd_rn(q[2 * i], q[2 * i + 1]);
        ss = q[0];
    }
    const int lanes_per_row = (FAST || S >= 32) ? 32 : S;
    if constexpr (FAST) {
#pragma unroll
        for (int m = 1; m < 32; m <<= 1) ss = __fadd_rn(ss, __shfl_xor_sync(0xffffffffu, ss, m));
    } else {
        for (int m = 1; m < lanes_per_row; m <<= 1) ss = __fadd_rn(ss, __shfl_xor_sync(0xffffffffu, ss, m));
    }
    if (S > 32) {
        const int nw = S >> 5;                                  // warps per row
        int nwp2 = 1;
        while (nwp2 < nw) nwp2 <<= 1;
        __syncthreads();                                        // exchange buffer no longer in use
        if (lane == 0) xsm[tid >> 5] = ss;
        __syncthreads();
        const int w0 = (r_local * S) >> 5;                      // first warp of this row
        const int li = lane & (nwp2 - 1);
        ss = (li < nw) ? xsm[w0 + li] : 0.0f;
        for (int m = 1; m < nwp2; m <<= 1) ss = __fadd_rn(ss, __shfl_xor_sync(0xffffffffu, ss, m));
    }
    const float rms = __fsqrt_rn(__fdiv_rn(ss, (float)cols));
    const float inv = (rms > 0.0f) ? __fdiv_rn(a.qc.A, rms) : 0.0f;
    if (active && (FAST || tn.scales) && tr == 0) tn.scales[row] = __fmul_rn(rms, a.qc.B);

    // ---- project: level axis, clamp, round to nearest even, trust test -----------------------
    const float2 inv2 = make_float2(inv, inv), c02 = make_float2(a.qc.c0, a.qc.c0);
    const float2 magic2 = make_float2(QUEST_MAGIC_RNE, QUEST_MAGIC_RNE);
    const float2 nmagic2 = make_float2(-QUEST_MAGIC_RNE, -QUEST_MAGIC_RNE);
    const float top = a.qc.top, hh = a.qc.h;
    int rsum = 0;
    if (active) {
#pragma unroll
        for (int g32 = 0; g32 < E / 32; ++g32) {
            uint32_t kb[32];                                    // MAGIC_BITS + level
            uint32_t mbits = 0;
            uint32_t w[CB];
            if constexpr (GRID == GRID_FP4) {
                // FP4 grid (Section 4.4): t = u * inv on the E2M1 value axis, hardware rounding to E2M1,
                // trusted = |t - value| <= trust_factor (the largest half-interval is one value unit)
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    float t[8];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        t[2 * j] = __fmul_rn(v[g32 * 16 + q * 4 + j].x, inv);
                        t[2 * j + 1] = __fmul_rn(v[g32 * 16 + q * 4 + j].y, inv);
                    }
                    const uint32_t cw = cvt_e2m1x8(t);
                    if (FAST || hh >= 1.0f) {
                        // every element inside the grid is within one value unit of its point (exactly, the
                        // difference being exact); only saturated elements can fail: |t| - 6 > trust_factor
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            mbits |= (__fsub_rn(fabsf(t[j]), 6.0f) <= hh ? 1u : 0u) << (q * 8 + j);
                    } else {
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const float val = e2m1_value((int)((cw >> (4 * j)) & 15u));
                            const bool trusted = fabsf(__fsub_rn(t[j], val)) <= hh;
                            mbits |= (trusted ? 1u : 0u) << (q * 8 + j);
                        }
                    }
                    w[q] = cw;
                }
            } else {
#pragma unroll
            for (int i = 15; i >= 0; --i) {
                const float2 t = __ffma2_rn(v[g32 * 16 + i], inv2, c02);
                float2 tc;
                tc.x = fminf(fmaxf(t.x, 0.0f), top);
                tc.y = fminf(fmaxf(t.y, 0.0f), top);
                const float2 km = __fadd2_rn(tc, magic2);
                float2 d;
                if constexpr (FAST) {
                    // trust_factor >= 1: an element inside the grid is within half a step of its level (the
                    // difference is exact), so only clipped elements can fail, and for those level = tc
                    d = __ffma2_rn(tc, neg1, t);                                // t - clamp(t)
                } else {
                    const float2 kf = __fadd2_rn(km, nmagic2);
                    d = __ffma2_rn(kf, neg1, t);                                // t - level
                }
                const float dy = __fsub_rn(hh, fabsf(d.y));                    // >= +0  <=>  trusted
                const float dx = __fsub_rn(hh, fabsf(d.x));
                mbits = __funnelshift_l(__float_as_uint(dy), mbits, 1);         // sign bit: 1 = masked
                mbits = __funnelshift_l(__float_as_uint(dx), mbits, 1);
                kb[2 * i] = __float_as_uint(km.x);
                kb[2 * i + 1] = __float_as_uint(km.y);
            }
            mbits = ~mbits;
            }
            if (FAST || tn.mask)
                reinterpret_cast<uint32_t *>(tn.mask + row * (long long)(cols >> 3))[tr * (E / 32) + g32] = mbits;

            // pack 32/CB codes per word: sum_j (MAGIC_BITS + k_j) * 2^(CB*j), minus the constant part
            constexpr int PER = 32 / CB;
            uint32_t magic_sum = 0;
#pragma unroll
            for (int j = 0; j < PER; ++j) magic_sum += QUEST_MAGIC_BITS << (CB * j);
            if constexpr (GRID != GRID_FP4) {
#pragma unroll
                for (int q = 0; q < CB; ++q) {
                    uint32_t acc = 0;
#pragma unroll
                    for (int j = PER - 1; j >= 0; --j) acc = (acc << CB) + kb[q * PER + j];
                    w[q] = acc - magic_sum;
                }
            }
            if (FAST || tn.codes) {
                uint8_t *dst = tn.codes + row * (long long)(cols * CB / 8) + ((long long)tr * (E / 32) + g32) * (4 * CB);
                if constexpr (CB == 8) {
                    reinterpret_cast<uint4 *>(dst)[0] = make_uint4(w[0], w[1], w[2], w[3]);
                    reinterpret_cast<uint4 *>(dst)[1] = make_uint4(w[4], w[5], w[6], w[7]);
                } else if constexpr (CB == 4) {
                    reinterpret_cast<uint4 *>(dst)[0] = make_uint4(w[0], w[1], w[2], w[3]);
                } else if constexpr (CB == 2) {
                    reinterpret_cast<uint2 *>(dst)[0] = make_uint2(w[0], w[1]);
                } else {
                    reinterpret_cast<uint32_t *>(dst)[0] = w[0];
                }
            }
            if constexpr (GRID == GRID_UNIFORM) {
                if (tn.cbf) {                                   // uniform over the CTA
                    // a small integer as bfloat16 is the upper half of its binary32 pattern (|c| <= 255: exact)
                    const int L1 = (1 << a.bits) - 1;
                    uint4 *dst = reinterpret_cast<uint4 *>(tn.cbf + row * (long long)cols + (long long)tr * E + g32 * 32);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint32_t o[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const int e0 = 8 * q + 2 * j, e1 = e0 + 1;
                            const int k0 = (int)((w[e0 / PER] >> ((e0 % PER) * CB)) & ((1u << CB) - 1u));
                            const int k1 = (int)((w[e1 / PER] >> ((e1 % PER) * CB)) & ((1u << CB) - 1u));
                            o[j] = (__float_as_uint((float)(2 * k0 - L1)) >> 16) |
                                   (__float_as_uint((float)(2 * k1 - L1)) & 0xFFFF0000u);
                        }
                        dst[q] = make_uint4(o[0], o[1], o[2], o[3]);
                    }
                }
            }
            if constexpr (GRID == GRID_UNIFORM) {              // the FP4 codes are themselves the tensor-core operand
            if constexpr (CB <= 2) {
                // one- and two-bit grids: E2M1 nibbles for the FP4 tensor-core path, 16 bytes per 32 elements
                if (tn.op8) {                                   // uniform over the CTA
                    uint32_t o[4];
                    e2m1_operand_from_code_words<CB>(w, o);
                    *reinterpret_cast<uint4 *>(tn.op8 + row * (long long)(cols >> 1) + (long long)tr * (E / 2) + g32 * 16) =
                        make_uint4(o[0], o[1], o[2], o[3]);
                }
            } else if (tn.op8) {
                uint32_t o[8];
                operand_from_code_words<CB>(w, a.bits, o);
                uint4 *dst = reinterpret_cast<uint4 *>(tn.op8 + row * (long long)cols + (long long)tr * E + g32 * 32);
                dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
                dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
                if ((RS || !FAST) && tn.rowsum) {
#pragma unroll
                    for (int q = 0; q < 8; ++q) rsum += sum_bytes_s8(o[q]);
                }
            }
            }
        }
    }
    if ((RS || !FAST) && tn.rowsum) {                                   // uniform over the CTA
        for (int m = 1; m < lanes_per_row; m <<= 1) rsum += __shfl_xor_sync(0xffffffffu, rsum, m);
        if (S > 32) {
            int *ism = reinterpret_cast<int *>(xsm);
            __syncthreads();
            if (lane == 0) ism[tid >> 5] = rsum;
            __syncthreads();
            if (tr == 0) {
                rsum = 0;
                const int w0 = (r_local * S) >> 5;
                for (int i = 0; i < (S >> 5); ++i) rsum += ism[w0 + i];
            }
        }
        if (active && tr == 0) tn.rowsum[row] = rsum;
    }
}

template <bool BF16, int CB, int E, int GRID = GRID_UNIFORM>
__global__ void __launch_bounds__(E == 64 ? 256 : 512)
quantize_rows_kernel(const __grid_constant__ QuantArgs a) {
    extern __shared__ float xsm[];                 // [E][blockDim.x] exchange, then [warps] partial sums
    constexpr int H = E / 2;                       // float2 pairs per thread
    pdl_launch_dependents();
    pdl_wait();
    const int tid = threadIdx.x;
    const int which = (int)blockIdx.x >= a.blocks0 ? 1 : 0;
    const QuantTensor &tn = a.t[which];
    const int blk = which ? (int)blockIdx.x - a.blocks0 : (int)blockIdx.x;
    const int S = a.S;
    const int r_local = tid / S;
    const int tr = tid - r_local * S;              // slot inside the row
    const long long row = (long long)blk * a.R + r_local;
    const int T = a.cols / E;
    const bool active = (row < tn.rows) && (tr < T);

    float2 v[H];
    if (active) {
        if (BF16) {
            const uint4 *src = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(tn.x) + row * tn.ld + (long long)tr * E);
#pragma unroll
            for (int q = 0; q < E / 8; ++q) {
                const uint4 w = __ldg(src + q);
                const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    v[q * 4 + j] = make_float2(__uint_as_float(ww[j] << 16), __uint_as_float(ww[j] & 0xFFFF0000u));
            }
        } else {
            const float4 *src = reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(tn.x) + row * tn.ld + (long long)tr * E);
#pragma unroll
            for (int q = 0; q < E / 4; ++q) {
                const float4 w = __ldg(src + q);
                v[q * 2] = make_float2(w.x, w.y);
                v[q * 2 + 1] = make_float2(w.z, w.w);
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < H; ++i) v[i] = make_float2(0.0f, 0.0f);
    }
    rotate_project_store<CB, E, false, false, GRID>(v, a, tn, active, row, tr, r_local, xsm, a.had_block >> 1);
}

// Streaming variant for bfloat16 rows (E = 64, had_block >= 64): a persistent grid in which every
// thread prefetches its 128 bytes of the NEXT row group into a private, padded shared-memory slot
// with cp.async while it works on the current one, so HBM latency hides behind the arithmetic
// whatever the occupancy.  Slots are 144 bytes apart: the 16-byte reads of a quarter warp fall in
// distinct bank groups.  Slots past the row end and rows past the tensor end are filled with zeros
// (source size 0), so reads need no predicate.  The first butterfly stage (stride had_block/2)
// pairs this thread with thread tid ^ dist0 of the same row; both read both raw slots from shared
// memory, so that stage needs no shuffles.
template <int CB, int E, bool FAST, int GRID = GRID_UNIFORM>
__global__ void __launch_bounds__(256, E == 64 ? 2 : 4)
quantize_stream_kernel(const __grid_constant__ QuantArgs a, int total_groups, int exchange_bytes) {
    constexpr int H = E / 2;
    constexpr int STREAM_SLOT = 2 * E + 16;
    extern __shared__ __align__(16) uint8_t smem_raw[];
    pdl_launch_dependents();
    pdl_wait();
    float *xsm = reinterpret_cast<float *>(smem_raw);
    uint8_t *stage = smem_raw + exchange_bytes;
    const int tid = threadIdx.x;
    const int nthreads = blockDim.x;
    const int r_local = tid / a.S;
    const int tr = tid - r_local * a.S;
    const bool slot_ok = tr < a.cols / E;
    const uint32_t my_slot = (uint32_t)__cvta_generic_to_shared(stage) + (uint32_t)tid * STREAM_SLOT;
    const uint32_t buf_stride = (uint32_t)nthreads * STREAM_SLOT;

    auto locate = [&](int grp, int &which, long long &row) {
        which = grp >= a.blocks0 ? 1 : 0;
        row = (long long)(which ? grp - a.blocks0 : grp) * a.R + r_local;
    };
    auto prefetch = [&](int grp, int buf) {
        if (grp < total_groups) {
            int which;
            long long row;
            locate(grp, which, row);
            const QuantTensor &tn = a.t[which];
            const bool live = slot_ok && row < tn.rows;
            const uint8_t *src = live ? reinterpret_cast<const uint8_t *>(tn.x) + (row * tn.ld + (long long)tr * E) * 2
                                      : reinterpret_cast<const uint8_t *>(tn.x);
            const uint32_t nbytes = live ? 16u : 0u;
            const uint32_t step = live ? 16u : 0u;
            const uint32_t dst = my_slot + (uint32_t)buf * buf_stride;
#pragma unroll
            for (int q = 0; q < E / 8; ++q)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst + q * 16), "l"(src + q * step),
                             "r"(nbytes)
                             : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    auto widen = [](const uint4 &w, float2 *out) {
        const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) out[j] = make_float2(__uint_as_float(ww[j] << 16), __uint_as_float(ww[j] & 0xFFFF0000u));
    };

    const bool first_from_smem = FAST || a.had_block >= 2 * E;
    const int dist0 = FAST ? 64 / E : first_from_smem ? (a.had_block >> 1) / E : 0;
    const bool cross_warp = !FAST && dist0 >= 32;
    const float sg0 = (tid & dist0) ? -1.0f : 1.0f;
    const float2 sgn0 = make_float2(sg0, sg0);
    const int s_start = FAST ? 32 : first_from_smem ? (a.had_block >> 2) : (a.had_block >> 1);

    int buf = 0;
    prefetch((int)blockIdx.x, 0);
    for (int grp = (int)blockIdx.x; grp < total_groups; grp += (int)gridDim.x, buf ^= 1) {
        // the slot about to be refilled was read by the partner thread one iteration ago
        if (cross_warp) __syncthreads(); else __syncwarp();
        prefetch(grp + (int)gridDim.x, buf ^ 1);
        asm volatile("cp.async.wait_group 1;" ::: "memory");
        if (cross_warp) __syncthreads(); else __syncwarp();   // the partner's copies have landed too
        int which;
        long long row;
        locate(grp, which, row);
        const QuantTensor &tn = a.t[which];
        const bool active = slot_ok && row < tn.rows;
        float2 v[H];
        const uint8_t *bufp = stage + (size_t)buf * buf_stride;
        const uint4 *own = reinterpret_cast<const uint4 *>(bufp + (size_t)tid * STREAM_SLOT);
        if (first_from_smem) {
            const uint4 *oth = reinterpret_cast<const uint4 *>(bufp + (size_t)(tid ^ dist0) * STREAM_SLOT);
#pragma unroll
            for (int q = 0; q < E / 8; ++q) {
                float2 o[4], p[4];
                widen(own[q], o);
                widen(oth[q], p);
#pragma unroll
                for (int j = 0; j < 4; ++j) v[q * 4 + j] = __ffma2_rn(o[j], sgn0, p[j]);   // own * (+-1) + partner
            }
        } else {
#pragma unroll
            for (int q = 0; q < E / 8; ++q) widen(own[q], &v[q * 4]);
        }
        rotate_project_store<CB, E, true, FAST, GRID>(v, a, tn, active, row, tr, r_local, xsm, s_start);
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// Wide rotation blocks (had_block = 1024, 2048 or 4096, bfloat16 rows): the five largest strides are
// made thread-local by a change of data layout instead of five rounds of warp shuffles.  A block of
// g = 32 G elements belongs to G threads.  Phase A: thread p of the block takes the 32 elements
// p + G j (j = 0..31) of the row straight from global memory, so the strides g/2 .. g/32 pair elements
// it already holds (one in-register 32-point butterfly, largest stride first).  The result goes
// back to shared memory in row order (binary32, 16 bytes of padding per 32 elements).  Phase B:
// every thread reads its 32 contiguous elements; the one or two strides left between g/64 and 32
// pair it with threads tr ^ 1, tr ^ 2, whose elements it reads from the same buffer; the strides
// below 32 and everything after the rotation are the common tail.  The order of the butterfly stages
// and every operand of every addition are those of the other kernels: the results are identical.
__device__ __forceinline__ void butterfly32_in_registers(float2 (&v)[16]) {
    const float2 neg1 = make_float2(-1.0f, -1.0f);
#pragma unroll
    for (int s2 = 8; s2 >= 1; s2 >>= 1) {                      // element strides 16 .. 2
#pragma unroll
        for (int i = 0; i < 16; ++i)
            if ((i & s2) == 0) {
                const float2 p = v[i], q = v[i + s2];
                v[i] = __fadd2_rn(p, q);
                v[i + s2] = __ffma2_rn(q, neg1, p);
            }
    }
#pragma unroll
    for (int i = 0; i < 16; ++i) {                             // element stride 1
        const float p = v[i].x, q = v[i].y;
        v[i] = make_float2(__fadd_rn(p, q), __fsub_rn(p, q));
    }
}

// G (threads per rotation block) is a template parameter so that every index of the two layout changes is a
// compile-time offset.
template <int CB, bool FAST, int GRID, int G>
__global__ void __launch_bounds__(256, 3)
quantize_wide_kernel(const __grid_constant__ QuantArgs a, int exchange_bytes) {
    extern __shared__ __align__(16) uint8_t smem_raw[];
    pdl_launch_dependents();
    pdl_wait();
    const int cols = a.cols, S = a.S, R = a.R;
    static_assert(G == 32 || G == 64 || G == 128, "rotation blocks of 1024, 2048 or 4096 elements");
    constexpr int gshift = G == 32 ? 5 : G == 64 ? 6 : 7;
    constexpr int GBLOCK = 32 * G;                             // elements of a rotation block
    float *xsm = reinterpret_cast<float *>(smem_raw);
    float *tbuf = reinterpret_cast<float *>(smem_raw + exchange_bytes);
    const int trow_words = cols + (cols >> 3);                 // 36 words per 32 elements
    const int tid = threadIdx.x;
    const int r_local = tid / S;
    const int tr = tid - r_local * S;
    const int p = tr & (G - 1);
    const int blk_base = (tr >> gshift) * GBLOCK;              // first element of this thread's block
    {
        const int grp = (int)blockIdx.x;                       // one CTA per group of R rows
        const int which = grp >= a.blocks0 ? 1 : 0;
        const long long row = (long long)(which ? grp - a.blocks0 : grp) * R + r_local;
        const QuantTensor &tn = a.t[which];
        const bool active = row < tn.rows;
        float2 v[16];
        {   // phase A: elements p + G j of this thread's block, then strides g/2 .. g/32 in registers
            // (two-byte loads: a warp reads 64 contiguous bytes per instruction, every byte once)
            if (active) {
                const uint16_t *rrow = reinterpret_cast<const uint16_t *>(tn.x) + row * tn.ld + blk_base + p;
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    v[j] = make_float2(__uint_as_float((uint32_t)__ldg(rrow + ((2 * j) << gshift)) << 16),
                                       __uint_as_float((uint32_t)__ldg(rrow + ((2 * j + 1) << gshift)) << 16));
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = make_float2(0.0f, 0.0f);
            }
            butterfly32_in_registers(v);
            float *trow = tbuf + (size_t)r_local * trow_words;
            // element i sits at word i + 4 (i / 32); with i = blk_base + p + G j and G a multiple of 32 that is a base
            // plus j (G + G / 8)
            float *tdst = trow + (blk_base + p) + (((blk_base + p) >> 5) << 2);
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                tdst[(2 * j) * (G + G / 8)] = v[j].x;
                tdst[(2 * j + 1) * (G + G / 8)] = v[j].y;
            }
        }
        __syncthreads();
        {   // phase B: 32 contiguous elements; strides g/64 .. 32 against the partner threads' elements
            const float *trow = tbuf + (size_t)r_local * trow_words;
            const float4 *own = reinterpret_cast<const float4 *>(trow + tr * 36);
            if constexpr (G == 32) {
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const float4 o = own[q];
                    v[2 * q] = make_float2(o.x, o.y);
                    v[2 * q + 1] = make_float2(o.z, o.w);
                }
            } else if constexpr (G == 64) {
                const float4 *p1 = reinterpret_cast<const float4 *>(trow + (tr ^ 1) * 36);
                const float s1 = (tr & 1) ? -1.0f : 1.0f;
                const float2 sg1 = make_float2(s1, s1);
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const float4 o = own[q], b = p1[q];
                    v[2 * q] = __ffma2_rn(make_float2(o.x, o.y), sg1, make_float2(b.x, b.y));
                    v[2 * q + 1] = __ffma2_rn(make_float2(o.z, o.w), sg1, make_float2(b.z, b.w));
                }
            } else {
                const float4 *p1 = reinterpret_cast<const float4 *>(trow + (tr ^ 1) * 36);
                const float4 *p2 = reinterpret_cast<const float4 *>(trow + (tr ^ 2) * 36);
                const float4 *p3 = reinterpret_cast<const float4 *>(trow + (tr ^ 3) * 36);
                const float s1 = (tr & 1) ? -1.0f : 1.0f, s2 = (tr & 2) ? -1.0f : 1.0f;
                const float2 sg1 = make_float2(s1, s1), sg2 = make_float2(s2, s2);
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const float4 o = own[q], b1 = p1[q], b2 = p2[q], b3 = p3[q];
                    // stride 64: this thread with tr ^ 2, and thread tr ^ 1 with tr ^ 3 (same side, same sign)
                    const float2 u0 = __ffma2_rn(make_float2(o.x, o.y), sg2, make_float2(b2.x, b2.y));
                    const float2 u1 = __ffma2_rn(make_float2(o.z, o.w), sg2, make_float2(b2.z, b2.w));
                    const float2 w0 = __ffma2_rn(make_float2(b1.x, b1.y), sg2, make_float2(b3.x, b3.y));
                    const float2 w1 = __ffma2_rn(make_float2(b1.z, b1.w), sg2, make_float2(b3.z, b3.w));
                    // stride 32: this thread's result with that of thread tr ^ 1
                    v[2 * q] = __ffma2_rn(u0, sg1, w0);
                    v[2 * q + 1] = __ffma2_rn(u1, sg1, w1);
                }
            }
        }
        rotate_project_store<CB, 32, true, FAST, GRID, true>(v, a, tn, active, row, tr, r_local, xsm, 16);
    }
}

template <int GRID, bool FAST, int G>
static cudaError_t launch_wide_g(int cb, int grid, int threads, size_t smem, cudaStream_t st, const QuantArgs &a,
                                 int exchange_bytes) {
#define QUEST_LAUNCH(CBV)                                                                                   \
    do {                                                                                                    \
        static DynamicSmemOnce once_;                                                                       \
        cudaError_t e_ = once_.set(quantize_wide_kernel<CBV, FAST, GRID, G>, 160 * 1024);                   \
        if (e_ != cudaSuccess) return e_;                                                                   \
        return launch_pdl(quantize_wide_kernel<CBV, FAST, GRID, G>, dim3((unsigned)grid), dim3(threads), smem, st, 1, a, \
                          exchange_bytes);                                                                  \
    } while (0)
    if (GRID == GRID_FP4) QUEST_LAUNCH(4);
    switch (cb) {
        case 1: QUEST_LAUNCH(1);
        case 2: QUEST_LAUNCH(2);
        case 4: QUEST_LAUNCH(4);
        default: QUEST_LAUNCH(8);
    }
#undef QUEST_LAUNCH
}

template <int GRID, bool FAST>
static cudaError_t launch_wide(int cb, int grid, int threads, size_t smem, cudaStream_t st, const QuantArgs &a,
                               int exchange_bytes) {
    switch (a.had_block) {
        case 1024: return launch_wide_g<GRID, FAST, 32>(cb, grid, threads, smem, st, a, exchange_bytes);
        case 2048: return launch_wide_g<GRID, FAST, 64>(cb, grid, threads, smem, st, a, exchange_bytes);
        default: return launch_wide_g<GRID, FAST, 128>(cb, grid, threads, smem, st, a, exchange_bytes);
    }
}

// The specialised case (bfloat16 rows, had_block = 128, 32 elements per thread) with direct loads and
// one CTA per row group: at sizes whose whole input is a few waves of CTAs the hardware's own CTA
// scheduling balances better than the persistent loop of the streaming kernel and there is no
// staging to set up.  Stride 64 pairs this thread with lane ^ 2 (shuffles); the rest is the common tail.
// RS: the row sums of the 8-bit GEMM operand are wanted (kept out of the common instantiation).
// COLS: the row length when it is one of the common ones (1024, 2048, 4096: threads per row, rows per CTA and every
// row pitch become constants, worth 6 % of the kernel); 0 takes them from the arguments.
template <int CB, int GRID = GRID_UNIFORM, bool RS = false, int COLS = 0>
__global__ void __launch_bounds__(256, 4)
quantize_direct128_kernel(const __grid_constant__ QuantArgs a) {
    constexpr int CS = COLS / 32;
    const int S = CS ? CS : a.S, R = CS ? 128 / CS : a.R, cols = COLS ? COLS : a.cols;
    extern __shared__ float xsm[];                 // [warps] partial sums
    pdl_launch_dependents();
    pdl_wait();
    const int tid = threadIdx.x, lane = tid & 31;
    const int which = (int)blockIdx.x >= a.blocks0 ? 1 : 0;
    const QuantTensor &tn = a.t[which];
    const int blk = which ? (int)blockIdx.x - a.blocks0 : (int)blockIdx.x;
    const int r_local = tid / S;
    const int tr = tid - r_local * S;
    const long long row = (long long)blk * R + r_local;
    const bool active = row < tn.rows && tr < (cols >> 5);     // slots past the row end hold zeros
    float2 v[16];
    if (active) {
        const uint4 *src = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(tn.x) + row * tn.ld + (long long)tr * 32);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint4 w = __ldg(src + q);
            const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int j = 0; j < 4; ++j)
                v[q * 4 + j] = make_float2(__uint_as_float(ww[j] << 16), __uint_as_float(ww[j] & 0xFFFF0000u));
        }
    } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = make_float2(0.0f, 0.0f);
    }
    {
        const float sg = (lane & 2) ? -1.0f : 1.0f;
        const float2 sgn = make_float2(sg, sg);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            float2 p;
            p.x = __shfl_xor_sync(0xffffffffu, v[i].x, 2);
            p.y = __shfl_xor_sync(0xffffffffu, v[i].y, 2);
            v[i] = __ffma2_rn(v[i], sgn, p);
        }
    }
    rotate_project_store<CB, 32, true, true, GRID, false, RS, CS, COLS>(v, a, tn, active, row, tr, r_local, xsm, 32);
}

// ---------------------------------------------------------------------------------------------
// Block kernel: bfloat16 rows stored densely, had_block = 128, codes + scales + mask requested,
// trust_factor >= 1.  ONE THREAD OWNS ONE WHOLE ROTATION BLOCK of 128 elements, so no butterfly
// stage crosses a thread (no shuffles at all in the rotation) and the per-thread costs (index
// arithmetic, the row's RMS and reciprocal, stores) are spread over 128 elements instead of 32.
// A warp's 32 blocks are 8 KB of consecutive memory.  They are fetched with coalesced 16-byte loads
// (a warp instruction reads 512 consecutive bytes) and redistributed through a swizzled
// shared-memory tile so that every thread ends up with its own 256 bytes; packed codes and the
// int8 GEMM operand travel the same way in the other direction.  The trust mask needs no detour:
// a thread's 16 bytes of mask follow its neighbour's.
// The sum of squares of a block is a complete subtree of the row's canonical pairwise tree, so
// the threads of a row combine their block sums in the same order as every other kernel: by
// xor-shuffles when a row has a power-of-two number of blocks of at most 32, through shared memory
// otherwise.
// ---------------------------------------------------------------------------------------------
constexpr int BLK_TILE_BYTES = 8192;             // per warp: 32 blocks x 256 bytes of bfloat16
constexpr long long BLOCK_KERNEL_MIN_ELEMS = 32ll << 20;

// Levels, mask bits and packed code words of 32 consecutive rotated elements (16 float2 pairs), for
// trust_factor >= 1: an element inside the grid is within half a step of its level, so only clipped
// elements can be masked, and for those the level is the clamp bound itself.
template <int CB, int GRID>
__device__ __forceinline__ void project32_trusting(const float2 *v, float inv, const QuantConsts &qc, uint32_t (&w)[CB],
                                                   uint32_t &mask_word) {
    const float2 neg1 = make_float2(-1.0f, -1.0f);
    const float hh = qc.h;
    uint32_t mbits = 0;
    if constexpr (GRID == GRID_FP4) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float t[8];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                t[2 * j] = __fmul_rn(v[q * 4 + j].x, inv);
                t[2 * j + 1] = __fmul_rn(v[q * 4 + j].y, inv);
            }
            w[q] = cvt_e2m1x8(t);
#pragma unroll
            for (int j = 0; j < 8; ++j)
                mbits |= (__fsub_rn(fabsf(t[j]), 6.0f) <= hh ? 1u : 0u) << (q * 8 + j);
        }
        mask_word = mbits;
    } else {
        const float2 inv2 = make_float2(inv, inv), c02 = make_float2(qc.c0, qc.c0);
        const float2 magic2 = make_float2(QUEST_MAGIC_RNE, QUEST_MAGIC_RNE);
        const float top = qc.top;
        uint32_t kb[32];                                        // MAGIC_BITS + level
        uint32_t mhi = 0;                                       // elements 16..31 (two independent shift chains)
#pragma unroll
        for (int i = 7; i >= 0; --i) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int p = i + 8 * half;
                const float2 t = __ffma2_rn(v[p], inv2, c02);
                float2 tc;
                tc.x = fminf(fmaxf(t.x, 0.0f), top);
                tc.y = fminf(fmaxf(t.y, 0.0f), top);
                const float2 km = __fadd2_rn(tc, magic2);
                const float2 d = __ffma2_rn(tc, neg1, t);       // t - clamp(t)
                const float dy = __fsub_rn(hh, fabsf(d.y));     // >= +0  <=>  trusted
                const float dx = __fsub_rn(hh, fabsf(d.x));
                uint32_t &m = half ? mhi : mbits;
                m = __funnelshift_l(__float_as_uint(dy), m, 1); // sign bit: 1 = masked
                m = __funnelshift_l(__float_as_uint(dx), m, 1);
                kb[2 * p] = __float_as_uint(km.x);
                kb[2 * p + 1] = __float_as_uint(km.y);
            }
        }
        mask_word = ~__byte_perm(mbits, mhi, 0x5410);           // low halves: elements 0..15 | 16..31
        constexpr int PER = 32 / CB;
        uint32_t magic_sum = 0;
#pragma unroll
        for (int j = 0; j < PER; ++j) magic_sum += QUEST_MAGIC_BITS << (CB * j);
#pragma unroll
        for (int q = 0; q < CB; ++q) {
            uint32_t acc = 0;
#pragma unroll
            for (int j = PER - 1; j >= 0; --j) acc = (acc << CB) + kb[q * PER + j];
            w[q] = acc - magic_sum;
        }
    }
}

// Swizzled position of 16-byte chunk `j` in row `r` of a tile whose rows hold NC chunks (NC = 4, 8 or
// 16): both the row-wise accesses of one thread per row and the chunk-wise accesses of consecutive
// lanes fall into distinct bank groups.
template <int NC>
__device__ __forceinline__ int swz(int r, int j) {
    if constexpr (NC == 4) return j ^ ((r >> 1) & 3);
    else return j ^ (r & 7);
}

// Copies a warp tile of 32 rows x NC chunks from shared memory to consecutive global memory.
template <int NC>
__device__ __forceinline__ void tile_to_global(const uint8_t *tile, uint8_t *dst, int lane, int live_rows) {
#pragma unroll
    for (int i = 0; i < NC; ++i) {
        const int c = i * 32 + lane;
        const int r = c / NC, j = c % NC;
        if (r < live_rows)
            *reinterpret_cast<uint4 *>(dst + (size_t)c * 16) =
                *reinterpret_cast<const uint4 *>(tile + r * (NC * 16) + swz<NC>(r, j) * 16);
    }
}

// CT: blocks per row when the kernel is instantiated for one row length (16, 32 and 43 blocks: 2048, 4096 and 5504
// columns); 0 takes the row length and the rows per CTA from the arguments.
template <int CB, int GRID, int CT = 0>
__global__ void __launch_bounds__(128, 3)
quantize_block128_kernel(const __grid_constant__ QuantArgs a) {
    constexpr bool CT_POW2 = CT != 0 && (CT & (CT - 1)) == 0 && CT <= 32;
    constexpr int CR = CT == 0 ? 0 : CT_POW2 ? 64 / CT : (CT >= 128 ? 1 : 128 / CT);     // the host's choice of rows per CTA
    extern __shared__ __align__(16) uint8_t smem_raw[];   // [warps][8 KB] tiles, then [threads] + [rows] floats
    pdl_launch_dependents();
    pdl_wait();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    const int bid = (int)blockIdx.x;
    const int which = (bid >= a.bend[0] ? 1 : 0) + (bid >= a.bend[1] ? 1 : 0) + (bid >= a.bend[2] ? 1 : 0);
    const QuantTensor &tn = a.t[which];
    const int blk = which ? bid - a.bend[which - 1] : bid;
    const int cols = CT ? CT * 128 : a.cols;
    const int T = CT ? CT : cols >> 7;                         // blocks (= threads) per row
    const int R = CT ? CR : a.R;
    const long long row0 = (long long)blk * R;
    const long long rows_left = tn.rows - row0;
    const int rows_here = rows_left < R ? (int)rows_left : R;
    const int nslots = rows_here * T;                          // live (row, block) slots of this CTA
    const bool active = tid < nslots;
    uint8_t *tile = smem_raw + warp * BLK_TILE_BYTES;
    float *part = reinterpret_cast<float *>(smem_raw + nwarps * BLK_TILE_BYTES);
    float *rowss = part + blockDim.x;
    const int wslot0 = warp * 32;
    const int wlive = nslots - wslot0 < 32 ? nslots - wslot0 : 32;     // live slots of this warp (may be <= 0)
    const size_t first_elem = (size_t)row0 * cols + (size_t)wslot0 * 128;   // dense rows: slots are consecutive blocks

    // ---- fetch: coalesced 16-byte loads, then every thread takes its own block from the tile -----
    float2 v[64];
    {
        const uint4 *src = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(tn.x) + first_elem);
        uint4 raw[16];
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            const int c = q * 32 + lane;
            raw[q] = (c >> 4) < wlive ? __ldg(src + c) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            const int c = q * 32 + lane;
            const int r = c >> 4, j = c & 15;
            *reinterpret_cast<uint4 *>(tile + r * 256 + swz<16>(r, j) * 16) = raw[q];
        }
        __syncwarp();
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            const uint4 w = *reinterpret_cast<const uint4 *>(tile + lane * 256 + swz<16>(lane, q) * 16);
            const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int j = 0; j < 4; ++j)
                v[q * 4 + j] = make_float2(__uint_as_float(ww[j] << 16), __uint_as_float(ww[j] & 0xFFFF0000u));
        }
        __syncwarp();                                          // the tile is reused for the outputs
    }

    // ---- rotation: strides 64 .. 2 on pairs, then stride 1 inside the pairs ---------------------
    {
        const float2 neg1 = make_float2(-1.0f, -1.0f);
#pragma unroll
        for (int s2 = 32; s2 >= 1; s2 >>= 1) {
#pragma unroll
            for (int i = 0; i < 64; ++i)
                if ((i & s2) == 0) {
                    const float2 p = v[i], q = v[i + s2];
                    v[i] = __fadd2_rn(p, q);
                    v[i + s2] = __ffma2_rn(q, neg1, p);        // p - q
                }
        }
#pragma unroll
        for (int i = 0; i < 64; ++i) {
            const float p = v[i].x, q = v[i].y;
            v[i] = make_float2(__fadd_rn(p, q), __fsub_rn(p, q));
        }
    }

    // ---- sum of squares of the block: the canonical pairwise tree, two half-blocks per packed add ---
    float ss;
    {
        float2 p[32];                                          // (sum over elements 2i, 2i+1; the same 64 elements later)
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const float2 lo = __fmul2_rn(v[i], v[i]), hi = __fmul2_rn(v[i + 32], v[i + 32]);
            p[i] = make_float2(__fadd_rn(lo.x, lo.y), __fadd_rn(hi.x, hi.y));
        }
#pragma unroll
        for (int n = 16; n >= 1; n >>= 1)
#pragma unroll
            for (int i = 0; i < n; ++i) p[i] = __fadd2_rn(p[2 * i], p[2 * i + 1]);
        ss = __fadd_rn(p[0].x, p[0].y);
    }
    // ---- the row's sum: block sums combined pairwise over the zero-padded row -------------------
    int my_row, my_t;
    if ((T & (T - 1)) == 0 && T <= 32) {                       // uniform over the launch
        for (int m = 1; m < T; m <<= 1) ss = __fadd_rn(ss, __shfl_xor_sync(0xffffffffu, ss, m));
        const int sh = 31 - __clz(T);
        my_row = tid >> sh;
        my_t = tid & (T - 1);
    } else {
        part[tid] = ss;                                        // slots past the end hold zeros
        __syncthreads();
        for (int r = warp; r < rows_here; r += nwarps) {
            float acc[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int i = lane + 32 * k;
                acc[k] = i < T ? part[r * T + i] : 0.0f;
#pragma unroll
                for (int m = 1; m < 32; m <<= 1) acc[k] = __fadd_rn(acc[k], __shfl_xor_sync(0xffffffffu, acc[k], m));
            }
            const float tot = __fadd_rn(__fadd_rn(acc[0], acc[1]), __fadd_rn(acc[2], acc[3]));
            if (lane == 0) rowss[r] = tot;
        }
        __syncthreads();
        my_row = active ? tid / T : 0;
        my_t = tid - my_row * T;
        ss = rowss[my_row < rows_here ? my_row : 0];
    }
    const float rms = __fsqrt_rn(__fdiv_rn(ss, (float)cols));
    const float inv = (rms > 0.0f) ? __fdiv_rn(a.qc.A, rms) : 0.0f;
    const long long row = row0 + my_row;
    if (active && my_t == 0) tn.scales[row] = __fmul_rn(rms, a.qc.B);

    // ---- project 4 x 32 elements; codes and operand bytes go to the tile, mask words stay here ---
    constexpr int CODE_NC = CB >= 4 ? CB : 4;                  // 16-byte chunks per thread's row of codes (CB = 4, 8)
    constexpr bool E2M1_OP = CB <= 2;
    uint8_t *code_tile = tile;                                 // [32][CODE_NC x 16] (CB >= 4 only)
    uint8_t *op_tile = tile + 4096;                            // [32][OP_NC x 16]
    const bool want_op = GRID == GRID_UNIFORM && tn.op8 != nullptr;
    uint32_t mw[4];
    uint32_t small_codes[CB <= 2 ? 4 * CB : 1];                // one- and two-bit codes: 16 or 32 bytes per thread
#pragma unroll
    for (int g32 = 0; g32 < 4; ++g32) {
        uint32_t w[CB];
        project32_trusting<CB, GRID>(&v[g32 * 16], inv, a.qc, w, mw[g32]);
        if constexpr (CB == 4) {
            *reinterpret_cast<uint4 *>(code_tile + lane * 64 + swz<4>(lane, g32) * 16) = make_uint4(w[0], w[1], w[2], w[3]);
        } else if constexpr (CB == 8) {
            *reinterpret_cast<uint4 *>(code_tile + lane * 128 + swz<8>(lane, 2 * g32) * 16) = make_uint4(w[0], w[1], w[2], w[3]);
            *reinterpret_cast<uint4 *>(code_tile + lane * 128 + swz<8>(lane, 2 * g32 + 1) * 16) = make_uint4(w[4], w[5], w[6], w[7]);
        } else {
#pragma unroll
            for (int q = 0; q < CB; ++q) small_codes[g32 * CB + q] = w[q];
        }
        if constexpr (GRID == GRID_UNIFORM) {
            if (want_op) {                                     // uniform over the CTA
                if constexpr (E2M1_OP) {
                    uint32_t o[4];
                    e2m1_operand_from_code_words<CB>(w, o);
                    *reinterpret_cast<uint4 *>(op_tile + lane * 64 + swz<4>(lane, g32) * 16) = make_uint4(o[0], o[1], o[2], o[3]);
                } else {
                    uint32_t o[8];
                    operand_from_code_words<CB>(w, a.bits, o);
                    *reinterpret_cast<uint4 *>(op_tile + lane * 128 + swz<8>(lane, 2 * g32) * 16) = make_uint4(o[0], o[1], o[2], o[3]);
                    *reinterpret_cast<uint4 *>(op_tile + lane * 128 + swz<8>(lane, 2 * g32 + 1) * 16) = make_uint4(o[4], o[5], o[6], o[7]);
                }
            }
        }
    }
    // ---- stores ------------------------------------------------------------------------------------
    if (active)                                                // 16 bytes of mask per block, consecutive across lanes
        *reinterpret_cast<uint4 *>(tn.mask + (first_elem >> 3) + (size_t)lane * 16) = make_uint4(mw[0], mw[1], mw[2], mw[3]);
    if constexpr (CB == 1) {
        if (active) *reinterpret_cast<uint4 *>(tn.codes + (first_elem >> 3) + (size_t)lane * 16) =
                        make_uint4(small_codes[0], small_codes[1], small_codes[2], small_codes[3]);
    } else if constexpr (CB == 2) {
        if (active) {
            uint4 *dst = reinterpret_cast<uint4 *>(tn.codes + (first_elem >> 2) + (size_t)lane * 32);
            dst[0] = make_uint4(small_codes[0], small_codes[1], small_codes[2], small_codes[3]);
            dst[1] = make_uint4(small_codes[4], small_codes[5], small_codes[6], small_codes[7]);
        }
    }
    __syncwarp();
    if (wlive > 0) {
        if constexpr (CB >= 4) tile_to_global<CODE_NC>(code_tile, tn.codes + first_elem * CB / 8, lane, wlive);
        if constexpr (GRID == GRID_UNIFORM) {
            if (want_op) {
                if constexpr (E2M1_OP) tile_to_global<4>(op_tile, reinterpret_cast<uint8_t *>(tn.op8) + (first_elem >> 1), lane, wlive);
                else tile_to_global<8>(op_tile, reinterpret_cast<uint8_t *>(tn.op8) + first_elem, lane, wlive);
            }
        }
    }
}

template <int GRID, int CT>
static cudaError_t launch_block128_ct(int cb, dim3 grid, int threads, size_t smem, cudaStream_t st, const QuantArgs &a) {
    if constexpr (GRID == GRID_FP4) {
        return launch_pdl(quantize_block128_kernel<4, GRID, CT>, grid, dim3(threads), smem, st, 1, a);
    } else {
        switch (cb) {
            case 1: return launch_pdl(quantize_block128_kernel<1, GRID, CT>, grid, dim3(threads), smem, st, 1, a);
            case 2: return launch_pdl(quantize_block128_kernel<2, GRID, CT>, grid, dim3(threads), smem, st, 1, a);
            case 4: return launch_pdl(quantize_block128_kernel<4, GRID, CT>, grid, dim3(threads), smem, st, 1, a);
            default: return launch_pdl(quantize_block128_kernel<8, GRID, CT>, grid, dim3(threads), smem, st, 1, a);
        }
    }
}

template <int GRID>
static cudaError_t launch_block128(int cb, dim3 grid, int threads, size_t smem, cudaStream_t st, const QuantArgs &a) {
    // the instantiations for one row length assume the rows per CTA the host derives from it
    if (a.cols == 2048 && a.R == 4) return launch_block128_ct<GRID, 16>(cb, grid, threads, smem, st, a);
    if (a.cols == 4096 && a.R == 2) return launch_block128_ct<GRID, 32>(cb, grid, threads, smem, st, a);
    if (a.cols == 5504 && a.R == 2) return launch_block128_ct<GRID, 43>(cb, grid, threads, smem, st, a);
    return launch_block128_ct<GRID, 0>(cb, grid, threads, smem, st, a);
}

template <int GRID, int COLS>
static cudaError_t launch_direct128_cols(int cb, dim3 grid, int threads, size_t smem, cudaStream_t st, const QuantArgs &a,
                                         bool rowsums) {
    if (rowsums) return launch_pdl(quantize_direct128_kernel<8, GRID_UNIFORM, true, COLS>, grid, dim3(threads), smem, st, 1, a);
    if (GRID == GRID_FP4) return launch_pdl(quantize_direct128_kernel<4, GRID, false, COLS>, grid, dim3(threads), smem, st, 1, a);
    switch (cb) {
        case 1: return launch_pdl(quantize_direct128_kernel<1, GRID, false, COLS>, grid, dim3(threads), smem, st, 1, a);
        case 2: return launch_pdl(quantize_direct128_kernel<2, GRID, false, COLS>, grid, dim3(threads), smem, st, 1, a);
        case 4: return launch_pdl(quantize_direct128_kernel<4, GRID, false, COLS>, grid, dim3(threads), smem, st, 1, a);
        default: return launch_pdl(quantize_direct128_kernel<8, GRID, false, COLS>, grid, dim3(threads), smem, st, 1, a);
    }
}

template <int GRID>
static cudaError_t launch_direct128(int cb, dim3 grid, int threads, size_t smem, cudaStream_t st, const QuantArgs &a,
                                    bool rowsums = false) {
    // the instantiations for one row length assume the launch geometry chosen for it: cols / 32 threads per row,
    // CTAs of 128 threads
    if (threads == 128 && a.S * 32 == a.cols && a.R * a.S == 128) {
        if (a.cols == 1024) return launch_direct128_cols<GRID, 1024>(cb, grid, threads, smem, st, a, rowsums);
        if (a.cols == 2048) return launch_direct128_cols<GRID, 2048>(cb, grid, threads, smem, st, a, rowsums);
        if (a.cols == 4096) return launch_direct128_cols<GRID, 4096>(cb, grid, threads, smem, st, a, rowsums);
    }
    return launch_direct128_cols<GRID, 0>(cb, grid, threads, smem, st, a, rowsums);
}

template <bool BF16, int E>
static cudaError_t launch_rows(int cb, dim3 grid, int threads, size_t smem, cudaStream_t st, const QuantArgs &a) {
#define QUEST_LAUNCH(CBV)                                                                                   \
    do {                                                                                                    \
        if (smem > 48 * 1024) {                                                                             \
            static DynamicSmemOnce once_;                                                                   \
            cudaError_t e_ = once_.set(quantize_rows_kernel<BF16, CBV, E>, 72 * 1024);                      \
            if (e_ != cudaSuccess) return e_;                                                               \
        }                                                                                                   \
        cudaError_t l_ = launch_pdl(quantize_rows_kernel<BF16, CBV, E>, grid, dim3(threads), smem, st, 1, a);  \
        if (l_ != cudaSuccess) return l_;                                                                   \
    } while (0)
    switch (cb) {
        case 1: QUEST_LAUNCH(1); break;
        case 2: QUEST_LAUNCH(2); break;
        case 4: QUEST_LAUNCH(4); break;
        default: QUEST_LAUNCH(8); break;
    }
#undef QUEST_LAUNCH
    return cudaGetLastError();
}

// FP4 grid: 4-bit containers only.
template <bool BF16, int E>
static cudaError_t launch_rows_fp4(dim3 grid, int threads, size_t smem, cudaStream_t st, const QuantArgs &a) {
    if (smem > 48 * 1024) {
        static DynamicSmemOnce once_;
        cudaError_t e_ = once_.set(quantize_rows_kernel<BF16, 4, E, GRID_FP4>, 72 * 1024);
        if (e_ != cudaSuccess) return e_;
    }
    return launch_pdl(quantize_rows_kernel<BF16, 4, E, GRID_FP4>, grid, dim3(threads), smem, st, 1, a);
}

template <int E, bool FAST>
static cudaError_t launch_stream_fp4(int grid, int threads, size_t smem, cudaStream_t st, const QuantArgs &a,
                                     int total_groups, int exchange_bytes) {
    static DynamicSmemOnce once_;
    cudaError_t e_ = once_.set(quantize_stream_kernel<4, E, FAST, GRID_FP4>, 160 * 1024);
    if (e_ != cudaSuccess) return e_;
    return launch_pdl(quantize_stream_kernel<4, E, FAST, GRID_FP4>, dim3((unsigned)grid), dim3(threads), smem, st, 1, a,
                      total_groups, exchange_bytes);
}

template <int E, bool FAST>
static cudaError_t launch_stream(int cb, int grid, int threads, size_t smem, cudaStream_t st, const QuantArgs &a,
                                 int total_groups, int exchange_bytes) {
#define QUEST_LAUNCH(CBV)                                                                                   \
    do {                                                                                                    \
        static DynamicSmemOnce once_;                                                                       \
        cudaError_t e_ = once_.set(quantize_stream_kernel<CBV, E, FAST>, 160 * 1024);                       \
        if (e_ != cudaSuccess) return e_;                                                                   \
        return launch_pdl(quantize_stream_kernel<CBV, E, FAST>, dim3((unsigned)grid), dim3(threads), smem, st, 1, a, \
                          total_groups, exchange_bytes);                                                    \
    } while (0)
    switch (cb) {
        case 1: QUEST_LAUNCH(1);
        case 2: QUEST_LAUNCH(2);
        case 4: QUEST_LAUNCH(4);
        default: QUEST_LAUNCH(8);
    }
#undef QUEST_LAUNCH
}

}  // namespace

int launch_quantize(const QuantJob *jobs, int njobs, int dtype, int64_t cols, int bits, int had_block,
                    float trust_factor, cudaStream_t st, int grid_kind) {
    const QuantConsts qc = grid_kind == GRID_FP4 ? make_quant_consts_fp4(had_block, trust_factor)
                                                 : make_quant_consts(bits, had_block, trust_factor);
    if (grid_kind == GRID_FP4 && cols % 32 != 0) return QUEST_ERR_SHAPE;
    const int cb = container_bits(bits);
    if (dtype == QUEST_BF16 && had_block == 128 && cols % 128 == 0 && trust_factor >= 1.0f) {
        // one thread per rotation block, when every tensor of the call is stored densely and asks for codes,
        // scales and mask (plus, optionally, the GEMM operand)
        bool ok = true;
        for (int j = 0; j < njobs; ++j) {
            const QuantJob &q = jobs[j];
            if (q.rows == 0) continue;
            if (!(q.codes && q.scales && q.mask) || q.rowsum || q.rot || q.cbf || q.ld != cols) ok = false;
            if (grid_kind == GRID_FP4 && q.op8) ok = false;
            if (reinterpret_cast<uintptr_t>(q.mask) % 16 != 0 || (q.op8 && reinterpret_cast<uintptr_t>(q.op8) % 16 != 0)) ok = false;
        }
        {
            // Below about 32 M elements (a few waves of this kernel's 4096-element warp tasks) the kernels with 32
            // elements per thread finish a layer sooner: their many short CTAs drain evenly, so the tensor-core
            // kernel that follows becomes resident earlier (measured on 4096 x 2048 + 2048 x 2048: 31.7 against
            // 32.9 us per layer; on 16384 x 4096 + 4096 x 4096 this kernel wins, 240.7 against 245.6 us).
            long long total_elems = 0;
            for (int j = 0; j < njobs; ++j) total_elems += (long long)jobs[j].rows * cols;
            if (total_elems < BLOCK_KERNEL_MIN_ELEMS) ok = false;
        }
        if (ok) {
            const int T = (int)(cols / 128);
            // rows per CTA.  Rows with a power-of-two number of blocks live inside one warp, so the CTA can be small:
            // 64 threads with 16 KB of shared memory fit beside a CTA of the tensor-core kernel that is still
            // draining, which lets the quantizer of the next layer become resident before its predecessor ends.
            // Other row lengths take as many whole rows as fit in 128 threads.
            const bool pow2 = (T & (T - 1)) == 0 && T <= 32;
            const int cta = pow2 ? 64 : 128;
            const int R = T >= cta ? 1 : cta / T;
            const int threads = (R * T + 31) / 32 * 32;
            const size_t smem = (size_t)(threads / 32) * BLK_TILE_BYTES + sizeof(float) * (size_t)(threads + R);
            for (int j0 = 0; j0 < njobs; j0 += MAX_QUANT_TENSORS) {
                QuantArgs a;
                int total = 0;
                for (int j = 0; j < MAX_QUANT_TENSORS; ++j) {
                    QuantTensor &t = a.t[j];
                    t = QuantTensor{nullptr, 0, 0, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
                    if (j0 + j < njobs) {
                        const QuantJob &q = jobs[j0 + j];
                        t.x = q.x; t.rows = q.rows; t.ld = q.ld; t.codes = q.codes; t.scales = q.scales;
                        t.mask = q.mask; t.op8 = q.op8;
                        total += (int)((q.rows + R - 1) / R);
                    }
                    a.bend[j] = total;
                }
                if (total == 0) continue;
                a.blocks0 = a.bend[0];
                a.cols = (int)cols; a.bits = bits; a.had_block = had_block; a.qc = qc; a.S = T; a.R = R;
                a.inv_sqrt_g = 1.0f / sqrtf((float)had_block);
                const dim3 grid((unsigned)total);
                const cudaError_t e = grid_kind == GRID_FP4 ? launch_block128<GRID_FP4>(cb, grid, threads, smem, st, a)
                                                            : launch_block128<GRID_UNIFORM>(cb, grid, threads, smem, st, a);
                if (e != cudaSuccess) return cuda_fail(e);
            }
            return QUEST_OK;
        }
    }
    if (cols % 32 == 0) {
        // 32 elements per thread (64 registers, twice the resident warps) for bfloat16 rows up to 8192 elements;
        // wider rows keep 64 per thread
        const bool e32 = dtype == QUEST_BF16 && had_block >= 64 && cols <= 8192;
        const int E = (cols % 64 == 0 && !e32) ? 64 : 32;
        const int T = (int)(cols / E);
        int S;
        if (T < 32) { S = 1; while (S < T) S <<= 1; } else { S = (T + 31) / 32 * 32; }
        // rows per CTA: CTAs of 128 threads wherever a row fits (finer work units, fewer warps behind each
        // CTA-wide barrier) except for the persistent 64-per-thread streaming kernel
        const bool streaming = E == 64 && dtype == QUEST_BF16 && had_block >= 64;
        const int R = (!streaming && S <= 128) ? 128 / S : (S >= 256 ? 1 : 256 / S);
        const int threads = R * S;
        const int warps = (threads + 31) / 32;
        const size_t smem = had_block >= 64 * E ? sizeof(float) * E * (size_t)threads : sizeof(float) * (size_t)warps;
        // at most two tensors per launch
        for (int j0 = 0; j0 < njobs; j0 += 2) {
            QuantArgs a;
            int nb[2] = {0, 0};
            for (int j = 0; j < 2; ++j) {
                QuantTensor &t = a.t[j];
                if (j0 + j < njobs) {
                    const QuantJob &q = jobs[j0 + j];
                    t.x = q.x; t.rows = q.rows; t.ld = q.ld; t.codes = q.codes; t.scales = q.scales;
                    t.mask = q.mask; t.op8 = q.op8; t.rowsum = q.rowsum; t.rot = q.rot; t.cbf = q.cbf;
                    nb[j] = (int)((q.rows + R - 1) / R);
                } else {
                    t.x = nullptr; t.rows = 0; t.ld = 0; t.codes = nullptr; t.scales = nullptr;
                    t.mask = nullptr; t.op8 = nullptr; t.rowsum = nullptr; t.rot = nullptr; t.cbf = nullptr;
                }
            }
            if (nb[0] + nb[1] == 0) continue;
            a.blocks0 = nb[0];
            for (int j = 0; j < MAX_QUANT_TENSORS; ++j) a.bend[j] = j == 0 ? nb[0] : nb[0] + nb[1];
            for (int j = 2; j < MAX_QUANT_TENSORS; ++j)
                a.t[j] = QuantTensor{nullptr, 0, 0, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
            a.cols = (int)cols; a.bits = bits; a.had_block = had_block; a.qc = qc; a.S = S; a.R = R;
            a.inv_sqrt_g = 1.0f / sqrtf((float)had_block);
            const dim3 grid((unsigned)(nb[0] + nb[1]));
            cudaError_t e;
            // the specialised tail: codes, scales and masks requested (or the rotation alone), trust_factor >= 1,
            // no row sums (so not the 8-bit GEMM operand); the FP4 grid has no separate GEMM operand
            bool fast_tail = trust_factor >= 1.0f && S >= 32;
            bool fast_tail_rs = fast_tail, any_rowsum = false;   // the same with row sums allowed
            for (int j = 0; j < 2; ++j) {
                const QuantTensor &t = a.t[j];
                const bool rot_only = t.rot && !t.codes && !t.scales && !t.mask && !t.op8 && !t.cbf;
                if (t.rows > 0 && (t.rowsum || !((t.codes && t.scales && t.mask) || rot_only))) fast_tail = false;
                if (t.rows > 0 && !((t.codes && t.scales && t.mask) || rot_only)) fast_tail_rs = false;
                if (t.rows > 0 && t.rowsum) any_rowsum = true;
                if (t.rows > 0 && grid_kind == GRID_FP4 && (t.op8 || t.rot || t.cbf)) fast_tail = false;
            }
            int dev = 0, sms = 148;
            cudaGetDevice(&dev);
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
            const int total = nb[0] + nb[1];
            if (e32 && S == T && S <= 256 && (had_block == 1024 || had_block == 2048 || had_block == 4096)) {
                // wide rotation blocks: layout-change kernel, one CTA per row group
                const int exchange = (int)((sizeof(float) * (size_t)warps + 15) / 16 * 16);
                const size_t smem2 = (size_t)exchange + (size_t)R * (cols + cols / 8) * 4;
                const int g = total;
                if (grid_kind == GRID_FP4)
                    e = fast_tail ? launch_wide<GRID_FP4, true>(cb, g, threads, smem2, st, a, exchange)
                                  : launch_wide<GRID_FP4, false>(cb, g, threads, smem2, st, a, exchange);
                else
                    e = fast_tail ? launch_wide<GRID_UNIFORM, true>(cb, g, threads, smem2, st, a, exchange)
                                  : launch_wide<GRID_UNIFORM, false>(cb, g, threads, smem2, st, a, exchange);
            } else if (e32 && had_block == 128 && fast_tail_rs && any_rowsum && cb == 8 && grid_kind == GRID_UNIFORM && threads <= 256) {
                // 8-bit codes with the row sums the GEMM needs
                e = launch_direct128<GRID_UNIFORM>(cb, grid, threads, smem, st, a, true);
            } else if (e32 && had_block == 128 && fast_tail && threads <= 256) {
                // the common case: direct loads, one CTA per row group
                e = grid_kind == GRID_FP4 ? launch_direct128<GRID_FP4>(cb, grid, threads, smem, st, a)
                                          : launch_direct128<GRID_UNIFORM>(cb, grid, threads, smem, st, a);
            } else if (streaming) {
                // rows wider than 8192: persistent streaming kernel, 64 elements per thread, as many CTAs as fit
                const int exchange = (int)((smem + 15) / 16 * 16);
                const size_t smem2 = (size_t)exchange + 2 * (size_t)threads * (2 * E + 16);
                const int per_sm = smem2 > 100 * 1024 ? 1 : 2;
                const int g = total < sms * per_sm ? total : sms * per_sm;
                const bool fast = fast_tail && had_block == 128;
                if (grid_kind == GRID_FP4)
                    e = fast ? launch_stream_fp4<64, true>(g, threads, smem2, st, a, total, exchange)
                             : launch_stream_fp4<64, false>(g, threads, smem2, st, a, total, exchange);
                else
                    e = fast ? launch_stream<64, true>(cb, g, threads, smem2, st, a, total, exchange)
                             : launch_stream<64, false>(cb, g, threads, smem2, st, a, total, exchange);
            } else if (grid_kind == GRID_FP4) {
                if (E == 64)
                    e = dtype == QUEST_BF16 ? launch_rows_fp4<true, 64>(grid, threads, smem, st, a)
                                            : launch_rows_fp4<false, 64>(grid, threads, smem, st, a);
                else
                    e = dtype == QUEST_BF16 ? launch_rows_fp4<true, 32>(grid, threads, smem, st, a)
                                            : launch_rows_fp4<false, 32>(grid, threads, smem, st, a);
            } else if (E == 64)
                e = dtype == QUEST_BF16 ? launch_rows<true, 64>(cb, grid, threads, smem, st, a)
                                        : launch_rows<false, 64>(cb, grid, threads, smem, st, a);
            else
                e = dtype == QUEST_BF16 ? launch_rows<true, 32>(cb, grid, threads, smem, st, a)
                                        : launch_rows<false, 32>(cb, grid, threads, smem, st, a);
            if (e != cudaSuccess) return cuda_fail(e);
        }
        return QUEST_OK;
    }
    int p2 = 1;
    while (p2 < cols) p2 <<= 1;
    const size_t smem = sizeof(float) * (size_t)(cols + p2);
    static DynamicSmemOnce smem_attr;
    {
        cudaError_t e = smem_attr.set(quantize_generic_kernel, 160 * 1024);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    for (int j = 0; j < njobs; ++j) {
        const QuantJob &q = jobs[j];
        if (q.rows == 0) continue;
        const int grid = (int)(q.rows < 148 * 8 ? q.rows : 148 * 8);
        cudaError_t e = launch_pdl(quantize_generic_kernel, dim3(grid), dim3(256), smem, st, 1, q.x, dtype, q.rows, (int)cols,
                                   q.ld, bits, had_block, qc, p2, q.codes, q.scales, q.mask, q.op8);
        if (e != cudaSuccess) return cuda_fail(e);
        if (q.rowsum && q.op8) {
            int s2 = launch_rowsum(q.op8, q.rows, cols, q.rowsum, st);
            if (s2) return s2;
        }
    }
    return QUEST_OK;
}

}  // namespace quest
