// Fused QuEST forward quantizer for sm_100a: Hadamard rotation (Eq. 2) -> RMS normalisation ->
// alpha*(b) clip -> round onto Eq. 1's grid -> packed codes, per-row scale, trust mask
// (Section 3.1 and 3.2; lines 2-5 of Algorithm 1).
//
// Every rounding decision is taken in binary32 with one IEEE rounding per operation, in this
// order: butterflies (a,b) -> (a+b, a-b) with DESCENDING stride g/2 .. 1; squares rounded, then
// pairwise summation over adjacent elements of the zero-padded row; rms = sqrt(ss/d);
// inv = A/rms; t = fma(u, inv, c0); level = rint(clamp(t, 0, 2^b-1)) (ties to even);
// trusted = |t - level| <= trust_factor/2.  This file is compiled with -fmad=false and uses
// the explicit _rn intrinsics so that the compiler cannot fuse or reorder any of it.
#include "quest_internal.cuh"

namespace quest {

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
                v8[j] = (int8_t)(bits == 8 ? k - 128 : 2 * k - L1);
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
// Row kernel: every thread owns 32 CONTIGUOUS elements of a row (cols % 32 == 0).
//   * butterflies of stride >= 1024 go through shared memory (rows wider than a warp's span),
//     strides 32..512 through warp shuffles, strides 16..1 stay in registers -- descending
//     stride overall, which is the canonical order;
//   * the sum of squares is reduced pairwise in the thread, then over lanes, then over warps;
//   * rounding, the trust test and the packing work on the thread's 32 elements, so each
//     thread stores whole words: 32*container/8 bytes of codes, 4 bytes of mask, 32 operand bytes.
// A row of T = cols/32 threads occupies S slots of the CTA: the next power of two if T < 32,
// else T rounded up to whole warps; slots past T carry zeros, which is the zero padding of the
// canonical pairwise sum.
// ---------------------------------------------------------------------------------------------
#define QUEST_MAGIC_RNE 12582912.0f            /* 1.5 * 2^23: x + MAGIC rounds x to an integer (ties to even) */
#define QUEST_MAGIC_BITS 0x4B400000u

__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// (a, b) -> (a + b, a - b) on two independent lanes with the packed binary32 instructions
__device__ __forceinline__ void butterfly2(float &a0, float &a1, float &b0, float &b1) {
    const uint64_t A = pack2(a0, a1), B = pack2(b0, b1);
    uint64_t S, D;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(S) : "l"(A), "l"(B));
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(D) : "l"(A), "l"(B));
    unpack2(S, a0, a1);
    unpack2(D, b0, b1);
}
// own * sgn + partner on two lanes (sgn = +-1: an exact add or subtract, one rounding)
__device__ __forceinline__ void fma2(float &x0, float &x1, float s, float p0, float p1) {
    const uint64_t X = pack2(x0, x1), Sg = pack2(s, s), P = pack2(p0, p1);
    uint64_t R;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(R) : "l"(X), "l"(Sg), "l"(P));
    unpack2(R, x0, x1);
}

template <bool BF16, int CB>
__global__ void __launch_bounds__(512)
quantize_row32_kernel(const void *__restrict__ x, int64_t rows, int cols, int64_t ld, int bits, int had_block,
                      QuantConsts qc, int S, int R,
                      uint8_t *__restrict__ codes, float *__restrict__ scales, uint8_t *__restrict__ mask,
                      int8_t *__restrict__ op8) {
    extern __shared__ float xsm[];                 // [32][blockDim.x] exchange, then [warps] partial sums
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int nthreads = blockDim.x;
    const int r_local = tid / S;
    const int tr = tid - r_local * S;              // slot inside the row
    const int64_t row = (int64_t)blockIdx.x * R + r_local;
    const int T = cols >> 5;
    const bool active = (row < rows) && (tr < T);

    float v[32];
    if (active) {
        if (BF16) {
            const uint4 *src = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(x) + row * ld + tr * 32);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint4 w = __ldg(src + q);
                const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    v[q * 8 + 2 * j] = __uint_as_float(ww[j] << 16);
                    v[q * 8 + 2 * j + 1] = __uint_as_float(ww[j] & 0xFFFF0000u);
                }
            }
        } else {
            const float4 *src = reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(x) + row * ld + tr * 32);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const float4 w = __ldg(src + q);
                v[q * 4] = w.x; v[q * 4 + 1] = w.y; v[q * 4 + 2] = w.z; v[q * 4 + 3] = w.w;
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = 0.0f;
    }

    // ---- rotation, descending stride --------------------------------------------------------
    for (int s = had_block >> 1; s >= 1024; s >>= 1) {        // partner thread is in another warp
        const int dist = s >> 5;
        __syncthreads();
#pragma unroll
        for (int i = 0; i < 32; ++i) xsm[i * nthreads + tid] = v[i];
        __syncthreads();
        const float sgn = (tid & dist) ? -1.0f : 1.0f;
        const int pt = tid ^ dist;
#pragma unroll
        for (int i = 0; i < 32; i += 2)
            fma2(v[i], v[i + 1], sgn, xsm[i * nthreads + pt], xsm[(i + 1) * nthreads + pt]);
    }
    {
        int s0 = had_block >> 1;
        if (s0 > 512) s0 = 512;
#pragma unroll 1
        for (int s = s0; s >= 32; s >>= 1) {                   // partner thread is a lane of this warp
            const int dist = s >> 5;
            const float sgn = (lane & dist) ? -1.0f : 1.0f;
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                const float p0 = __shfl_xor_sync(0xffffffffu, v[i], dist);
                const float p1 = __shfl_xor_sync(0xffffffffu, v[i + 1], dist);
                fma2(v[i], v[i + 1], sgn, p0, p1);
            }
        }
    }
#pragma unroll
    for (int s = 16; s >= 2; s >>= 1) {                        // partner element is in this thread
        if (s < had_block) {
#pragma unroll
            for (int i = 0; i < 32; i += 2)
                if ((i & s) == 0) butterfly2(v[i], v[i + 1], v[i + s], v[i + s + 1]);
        }
    }
    if (had_block > 1) {
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
            const float a = v[i], b = v[i + 1];
            v[i] = __fadd_rn(a, b);
            v[i + 1] = __fsub_rn(a, b);
        }
    }

    // ---- sum of squares: pairwise over adjacent elements, zero-padded row --------------------
    float ss;
    {
        float q[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) q[i] = __fadd_rn(__fmul_rn(v[2 * i], v[2 * i]), __fmul_rn(v[2 * i + 1], v[2 * i + 1]));
#pragma unroll
        for (int n = 8; n >= 1; n >>= 1)
#pragma unroll
            for (int i = 0; i < n; ++i) q[i] = __fadd_rn(q[2 * i], q[2 * i + 1]);
        ss = q[0];
    }
    const int lanes_per_row = S < 32 ? S : 32;
    for (int m = 1; m < lanes_per_row; m <<= 1) ss = __fadd_rn(ss, __shfl_xor_sync(0xffffffffu, ss, m));
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
    const float inv = (rms > 0.0f) ? __fdiv_rn(qc.A, rms) : 0.0f;
    if (!active) return;
    if (scales && tr == 0) scales[row] = __fmul_rn(rms, qc.B);

    // ---- project: level axis, clamp, round to nearest even, trust test -----------------------
    uint32_t kb[32];                                            // MAGIC_BITS + level
    uint32_t mbits = 0;
#pragma unroll
    for (int i = 31; i >= 0; --i) {
        const float t = __fmaf_rn(v[i], inv, qc.c0);
        const float tc = fminf(fmaxf(t, 0.0f), qc.top);
        const float km = __fadd_rn(tc, QUEST_MAGIC_RNE);
        const float kf = __fsub_rn(km, QUEST_MAGIC_RNE);
        const float dlt = __fsub_rn(qc.h, fabsf(__fsub_rn(t, kf)));   // >= +0  <=>  trusted
        mbits = __funnelshift_l(__float_as_uint(dlt), mbits, 1);         // sign bit: 1 = masked
        kb[i] = __float_as_uint(km);
    }
    mbits = ~mbits;
    if (mask) reinterpret_cast<uint32_t *>(mask + row * (int64_t)(cols >> 3))[tr] = mbits;

    if (codes) {
        // pack 32/CB codes per word: sum_j (MAGIC_BITS + k_j) * 2^(CB*j), minus the constant part
        constexpr int PER = 32 / CB;
        constexpr int WORDS = CB;
        uint32_t magic_sum = 0;
#pragma unroll
        for (int j = 0; j < PER; ++j) magic_sum += QUEST_MAGIC_BITS << (CB * j);
        uint32_t w[WORDS];
#pragma unroll
        for (int q = 0; q < WORDS; ++q) {
            uint32_t acc = 0;
#pragma unroll
            for (int j = PER - 1; j >= 0; --j) acc = (acc << CB) + kb[q * PER + j];
            w[q] = acc - magic_sum;
        }
        uint8_t *dst = codes + row * (int64_t)(cols * CB / 8) + (int64_t)tr * (4 * CB);
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
    if (op8) {
        // int8 operand of the tensor-core contraction: c = 2k - (2^b - 1), or k - 128 at b = 8
        const int L1 = (1 << bits) - 1;
        uint32_t o[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            uint32_t acc = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int k = (int)(kb[q * 4 + j] - QUEST_MAGIC_BITS);
                const int val = (bits == 8) ? (k - 128) : (2 * k - L1);
                acc |= (uint32_t)(val & 0xFF) << (8 * j);
            }
            o[q] = acc;
        }
        uint4 *dst = reinterpret_cast<uint4 *>(op8 + row * (int64_t)cols + (int64_t)tr * 32);
        dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
        dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
}

template <bool BF16>
static cudaError_t launch_row32(int cb, dim3 grid, int threads, size_t smem, cudaStream_t st,
                                const void *x, int64_t rows, int cols, int64_t ld, int bits, int had_block,
                                QuantConsts qc, int S, int R, uint8_t *codes, float *scales, uint8_t *mask,
                                int8_t *op8) {
#define QUEST_LAUNCH(CBV)                                                                                   \
    do {                                                                                                    \
        if (smem > 48 * 1024) {                                                                             \
            cudaError_t e_ = cudaFuncSetAttribute(quantize_row32_kernel<BF16, CBV>,                         \
                                                  cudaFuncAttributeMaxDynamicSharedMemorySize, 72 * 1024);  \
            if (e_ != cudaSuccess) return e_;                                                               \
        }                                                                                                   \
        quantize_row32_kernel<BF16, CBV><<<grid, threads, smem, st>>>(x, rows, cols, ld, bits, had_block,   \
                                                                      qc, S, R, codes, scales, mask, op8);  \
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

}  // namespace

int launch_quantize(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                    int bits, int had_block, float trust_factor,
                    uint8_t *codes, float *scales, uint8_t *mask, int8_t *op8, cudaStream_t st) {
    if (rows == 0) return QUEST_OK;
    const QuantConsts qc = make_quant_consts(bits, had_block, trust_factor);
    if (cols % 32 == 0) {
        const int T = (int)(cols / 32);
        int S;
        if (T < 32) { S = 1; while (S < T) S <<= 1; } else { S = (T + 31) / 32 * 32; }
        const int R = S >= 256 ? 1 : 256 / S;
        const int threads = R * S;
        const int warps = threads / 32;
        const size_t smem = had_block >= 2048 ? sizeof(float) * 32 * (size_t)threads : sizeof(float) * (size_t)warps;
        const dim3 grid((unsigned)((rows + R - 1) / R));
        const int cb = container_bits(bits);
        cudaError_t e = dtype == QUEST_BF16
            ? launch_row32<true>(cb, grid, threads, smem, st, x, rows, (int)cols, ld, bits, had_block, qc, S, R,
                                 codes, scales, mask, op8)
            : launch_row32<false>(cb, grid, threads, smem, st, x, rows, (int)cols, ld, bits, had_block, qc, S, R,
                                  codes, scales, mask, op8);
        return e == cudaSuccess ? QUEST_OK : cuda_fail(e);
    }
    int p2 = 1;
    while (p2 < cols) p2 <<= 1;
    const size_t smem = sizeof(float) * (size_t)(cols + p2);
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(quantize_generic_kernel,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
        if (e != cudaSuccess) return cuda_fail(e);
        attr_done = true;
    }
    const int grid = (int)(rows < 148 * 8 ? rows : 148 * 8);
    quantize_generic_kernel<<<grid, 256, smem, st>>>(x, dtype, rows, (int)cols, ld, bits, had_block, qc, p2,
                                                     codes, scales, mask, op8);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? QUEST_OK : cuda_fail(e);
}

}  // namespace quest
