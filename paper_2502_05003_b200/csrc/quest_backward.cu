// QuEST training backward for one linear layer (Algorithm 2) on sm_100a:
//
//   dL/dxq_h = dL/dy wq_h                      dL/dx = IHT(M(x_h; xq_h) * dL/dxq_h)
//   dL/dwq_h = dL/dy^T xq_h                    dL/dw = IHT(M(w_h; wq_h) * dL/dwq_h)
//
// The products run in 16-bit precision on the tensor cores (Section 3.3, "Implementation").  dL/dy is
// used as it is (bfloat16); the quantized operand is dequantised to bfloat16, xq_h = bf16(sx[m] c_x),
// wq_h = bf16(sw[n] c_w) with c = 2k - (2^b - 1): one rounding per product.  Nothing is transposed: the
// tensor cores read an operand whose memory rows run along the contraction index as an MN-major
// operand (quest_gemm.cu).  Stages:
//   1. dequant_codes_kernel   wq_h [N x K], xq_h [M x K] from the packed codes and scales
//   2. gemm (bfloat16 mode)   d1[m][k] = M_x[m][k] sum_n dy[m][n] wq_h[n][k]   (dy K-major, wq_h MN-major)
//                             d2[n][k] = M_w[n][k] sum_m dy[m][n] xq_h[m][k]   (dy and xq_h MN-major)
//   3. iht_rows_kernel        block Hadamard transform, 1/sqrt(g), store in the output type
//      (for blocks of 128 stages 2 and 3 are one kernel: the transform runs in the GEMM epilogue,
//      where a thread holds exactly one block of its output row)
#include <cuda_bf16.h>
#include <math.h>

#include "quest_internal.cuh"

namespace quest {
namespace {

__device__ __forceinline__ uint16_t bf16_bits(float v) {
    __nv_bfloat16 h = __float2bfloat16_rn(v);
    return *reinterpret_cast<uint16_t *>(&h);
}

// Packed level indices and per-row scales -> dequantised values bf16(scale[r] * c) [rows x K], dense.
// One thread converts 8 consecutive elements (one 16-byte store; K % 32 == 0 keeps them in one row).
template <int CB>
__global__ void __launch_bounds__(256)
dequant_codes_kernel(const uint8_t *__restrict__ codes0, const float *__restrict__ scales0, uint16_t *__restrict__ out0,
                     long long n_oct0, const uint8_t *__restrict__ codes1, const float *__restrict__ scales1,
                     uint16_t *__restrict__ out1, long long n_oct1, int bits, int K) {
    pdl_launch_dependents();
    pdl_wait();
    long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n_oct0 + n_oct1) return;
    const bool second = t >= n_oct0;                         // up to two tensors per launch
    if (second) t -= n_oct0;
    const uint8_t *codes = second ? codes1 : codes0;
    const float *scales = second ? scales1 : scales0;
    uint16_t *out = second ? out1 : out0;
    const int L1 = (1 << bits) - 1;
    const float sc = __ldg(scales + t / (K / 8));
    const uint32_t *c32 = reinterpret_cast<const uint32_t *>(codes);
    uint32_t lo, hi = 0;                                     // the 8 * CB bits of this thread's levels
    if constexpr (CB == 8) { lo = __ldg(c32 + 2 * t); hi = __ldg(c32 + 2 * t + 1); }
    else if constexpr (CB == 4) lo = __ldg(c32 + t);
    else if constexpr (CB == 2) lo = (__ldg(c32 + (t >> 1)) >> (16 * (int)(t & 1))) & 0xFFFFu;
    else lo = (__ldg(c32 + (t >> 2)) >> (8 * (int)(t & 3))) & 0xFFu;
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        int k0, k1;
        if constexpr (CB == 8) {
            const uint32_t w = j < 2 ? lo : hi;
            k0 = (int)((w >> (16 * (j & 1))) & 0xFFu);
            k1 = (int)((w >> (16 * (j & 1) + 8)) & 0xFFu);
        } else {
            k0 = (int)((lo >> (2 * j * CB)) & ((1u << CB) - 1u));
            k1 = (int)((lo >> ((2 * j + 1) * CB)) & ((1u << CB) - 1u));
        }
        o[j] = (uint32_t)bf16_bits(sc * (float)(2 * k0 - L1)) | ((uint32_t)bf16_bits(sc * (float)(2 * k1 - L1)) << 16);
    }
    *reinterpret_cast<uint4 *>(out + t * 8) = make_uint4(o[0], o[1], o[2], o[3]);
}

// Inverse orthonormal block Hadamard transform of every row of d [rows x cols] (binary32, dense),
// stored as out_dtype with row stride ld.  Every thread owns 32 contiguous elements; descending
// stride: partners in other warps through shared memory, partners in this warp through shuffles,
// the rest in registers.  A row of T = cols/32 threads occupies S slots as in the quantizer.
__global__ void __launch_bounds__(512)
iht_rows_kernel(const void *__restrict__ d, int in_dtype, long long ld_in, long long rows, int cols, int had_block,
                float inv_sqrt_g, void *__restrict__ out, int out_dtype, long long ld, int S, int R) {
    extern __shared__ float xsm[];                 // [32][blockDim.x] exchange
    pdl_launch_dependents();
    pdl_wait();
    const int tid = threadIdx.x, lane = tid & 31, nthreads = blockDim.x;
    const int r_local = tid / S;
    const int tr = tid - r_local * S;
    const long long row = (long long)blockIdx.x * R + r_local;
    const bool active = row < rows && tr < cols / 32;
    float v[32];
    if (active && in_dtype == QUEST_F32) {
        const float4 *src = reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(d) + row * ld_in + (long long)tr * 32);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float4 w = __ldg(src + q);
            v[4 * q] = w.x; v[4 * q + 1] = w.y; v[4 * q + 2] = w.z; v[4 * q + 3] = w.w;
        }
    } else if (active) {
        const uint4 *src = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(d) + row * ld_in + (long long)tr * 32);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint4 w = __ldg(src + q);
            const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                v[8 * q + 2 * j] = __uint_as_float(ww[j] << 16);
                v[8 * q + 2 * j + 1] = __uint_as_float(ww[j] & 0xFFFF0000u);
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = 0.0f;
    }
    for (int s = had_block >> 1; s >= 1024; s >>= 1) {        // partner thread is in another warp
        const int dist = s >> 5;
        __syncthreads();
#pragma unroll
        for (int i = 0; i < 32; ++i) xsm[i * nthreads + tid] = v[i];
        __syncthreads();
        const float sg = (tid & dist) ? -1.0f : 1.0f;
        const int pt = tid ^ dist;
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = fmaf(v[i], sg, xsm[i * nthreads + pt]);
    }
    {
        int s0 = had_block >> 1;
        if (s0 > 512) s0 = 512;
#pragma unroll 1
        for (int s = s0; s >= 32; s >>= 1) {                   // partner thread is a lane of this warp
            const int dist = s >> 5;
            const float sg = (lane & dist) ? -1.0f : 1.0f;
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = fmaf(v[i], sg, __shfl_xor_sync(0xffffffffu, v[i], dist));
        }
    }
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) {
        if (s < had_block) {
#pragma unroll
            for (int i = 0; i < 32; ++i)
                if ((i & s) == 0) {
                    const float a = v[i], b = v[i + s];
                    v[i] = a + b;
                    v[i + s] = a - b;
                }
        }
    }
    if (!active) return;
    if (out_dtype == QUEST_F32) {
        float4 *dst = reinterpret_cast<float4 *>(reinterpret_cast<float *>(out) + row * ld + (long long)tr * 32);
#pragma unroll
        for (int q = 0; q < 8; ++q)
            dst[q] = make_float4(v[4 * q] * inv_sqrt_g, v[4 * q + 1] * inv_sqrt_g, v[4 * q + 2] * inv_sqrt_g,
                                 v[4 * q + 3] * inv_sqrt_g);
    } else {
        uint4 *dst = reinterpret_cast<uint4 *>(reinterpret_cast<uint16_t *>(out) + row * ld + (long long)tr * 32);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            uint32_t w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
                w[j] = (uint32_t)bf16_bits(v[8 * q + 2 * j] * inv_sqrt_g) |
                       ((uint32_t)bf16_bits(v[8 * q + 2 * j + 1] * inv_sqrt_g) << 16);
            dst[q] = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
}

struct BwdWorkspace {
    uint16_t *wh, *xh;      // dequantised operands [N x K], [M x K]
    float *d1, *d2;         // masked products when the inverse transform is a separate kernel
    size_t bytes;
};
BwdWorkspace carve_bwd(void *base, int64_t M, int64_t N, int64_t K) {
    BwdWorkspace w;
    uint8_t *b = reinterpret_cast<uint8_t *>(base);
    size_t off = 0;
    auto take = [&](size_t n) { uint8_t *p = b + off; off += align_up(n, 256); return p; };
    w.wh = reinterpret_cast<uint16_t *>(take((size_t)N * K * 2));
    w.xh = reinterpret_cast<uint16_t *>(take((size_t)M * K * 2));
    w.d1 = reinterpret_cast<float *>(take((size_t)M * K * 4));
    w.d2 = reinterpret_cast<float *>(take((size_t)N * K * 4));
    w.bytes = off;
    return w;
}

int launch_iht(const float *d, int64_t rows, int64_t cols, int had_block, void *out, int out_dtype, int64_t ld,
               cudaStream_t st) {
    return launch_hadamard_rows(d, QUEST_F32, cols, rows, cols, had_block, out, out_dtype, ld, st);
}

}  // namespace

// Orthonormal block Hadamard transform (its own inverse) of every row: in [rows x cols] with row
// stride ld_in (16-byte aligned rows), out with row stride ld; cols % 32 == 0.
int launch_hadamard_rows(const void *in, int in_dtype, int64_t ld_in, int64_t rows, int64_t cols, int had_block,
                         void *out, int out_dtype, int64_t ld, cudaStream_t st) {
    if (rows == 0) return QUEST_OK;
    const int T = (int)(cols / 32);
    int S;
    if (T < 32) { S = 1; while (S < T) S <<= 1; } else { S = (T + 31) / 32 * 32; }
    const int R = S <= 128 ? 128 / S : 1;      // CTAs of 128 threads where a row fits
    const int threads = R * S;
    const size_t smem = had_block >= 2048 ? sizeof(float) * 32 * (size_t)threads : 0;
    if (smem > 48 * 1024) {
        static DynamicSmemOnce smem_attr;
        cudaError_t e = smem_attr.set(iht_rows_kernel, 72 * 1024);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    const long long grid = (rows + R - 1) / R;
    cudaError_t e = launch_pdl(iht_rows_kernel, dim3((unsigned)grid), dim3(threads), smem, st, 1, in, in_dtype, (long long)ld_in,
                               (long long)rows, (int)cols, had_block, 1.0f / sqrtf((float)had_block), out, out_dtype,
                               (long long)ld, S, R);
    return e == cudaSuccess ? QUEST_OK : cuda_fail(e);
}

namespace {

bool bwd_shape_ok(int64_t M, int64_t N, int64_t K) {
    return M > 0 && N > 0 && K >= 32 && K % 32 == 0 && K <= 16384 && M % 8 == 0 && N % 8 == 0 &&
           M <= ((int64_t)1 << 24) && N <= ((int64_t)1 << 24);
}

}  // namespace
}  // namespace quest

using namespace quest;

extern "C" size_t quest_bwd_workspace_bytes(int64_t M, int64_t N, int64_t K) {
    if (!bwd_shape_ok(M, N, K)) return 0;
    return carve_bwd(nullptr, M, N, K).bytes;
}

extern "C" int quest_linear_bwd(const void *dy, int64_t M, int64_t N, int64_t K, int bits, int had_block,
                                const uint8_t *xq, const float *sx, const uint8_t *mx,
                                const uint8_t *wq, const float *sw, const uint8_t *mw,
                                void *dx, void *dw, int out_dtype,
                                void *workspace, size_t workspace_bytes, void *stream) {
    if (!dy || !xq || !sx || !mx || !wq || !sw || !mw) return QUEST_ERR_NULL;
    if (!dx && !dw) return QUEST_ERR_NULL;
    if (bits < 1 || bits > 8) return QUEST_ERR_BITS;
    if (!bwd_shape_ok(M, N, K)) return QUEST_ERR_SHAPE;
    if (had_block < 1 || (had_block & (had_block - 1)) != 0 || had_block > K || K % had_block != 0)
        return QUEST_ERR_HAD_BLOCK;
    if (out_dtype != QUEST_F32 && out_dtype != QUEST_BF16) return QUEST_ERR_DTYPE;
    auto al = [](const void *p, size_t a) { return reinterpret_cast<uintptr_t>(p) % a == 0; };
    if (!al(dy, 16) || !al(mx, 16) || !al(mw, 16) || !al(sw, 4) || !al(sx, 4) || !al(xq, 4) || !al(wq, 4) || (dx && !al(dx, 16)) ||
        (dw && !al(dw, 16)))
        return QUEST_ERR_ALIGN;
    if (!workspace || !al(workspace, 256) || workspace_bytes < quest_bwd_workspace_bytes(M, N, K))
        return QUEST_ERR_WORKSPACE;
    int s = check_device();
    if (s) return s;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    BwdWorkspace ws = carve_bwd(workspace, M, N, K);
    struct Stage {                                   // RAII bracket for quest_stage_timing
        void *h;
        Stage(int id, cudaStream_t s_) : h(stage_begin(id, s_)) {}
        ~Stage() { stage_end(h); }
    };
    {
        // both dequantised operands in one launch, then the two products back to back
        Stage prep(QUEST_STAGE_UNPACK, st);
        const long long n0 = dx ? (long long)N * (K / 8) : 0, n1 = dw ? (long long)M * (K / 8) : 0;
        const dim3 grid((unsigned)((n0 + n1 + 255) / 256));
        cudaError_t e;
        switch (container_bits(bits)) {
            case 1: e = launch_pdl(dequant_codes_kernel<1>, grid, dim3(256), 0, st, 1, wq, sw, ws.wh, n0, xq, sx, ws.xh, n1, bits, (int)K); break;
            case 2: e = launch_pdl(dequant_codes_kernel<2>, grid, dim3(256), 0, st, 1, wq, sw, ws.wh, n0, xq, sx, ws.xh, n1, bits, (int)K); break;
            case 4: e = launch_pdl(dequant_codes_kernel<4>, grid, dim3(256), 0, st, 1, wq, sw, ws.wh, n0, xq, sx, ws.xh, n1, bits, (int)K); break;
            default: e = launch_pdl(dequant_codes_kernel<8>, grid, dim3(256), 0, st, 1, wq, sw, ws.wh, n0, xq, sx, ws.xh, n1, bits, (int)K); break;
        }
        if (e != cudaSuccess) return cuda_fail(e);
    }
    if (dx) {
        Stage gemm_stage(QUEST_STAGE_GEMM, st);
        // activation gradient of Algorithm 2 with its trust mask: d1[m][k] = M_x[m][k] * sum_n dy[m][n] wq_h[n][k]
        // (blocks of 128: the inverse transform is fused into the contraction's epilogue)
        if (had_block == 128 && M > 128 && K > 128) {
            if ((s = launch_gemm_bf16_masked(dy, ws.wh, M, K, N, mx, dx, out_dtype, true, 1, st))) return s;
        } else {
            if ((s = launch_gemm_bf16_masked(dy, ws.wh, M, K, N, mx, ws.d1, QUEST_F32, false, 1, st))) return s;
            if ((s = launch_iht(ws.d1, M, K, had_block, dx, out_dtype, K, st))) return s;
        }
    }
    if (dw) {
        Stage gemm_stage(QUEST_STAGE_GEMM, st);
        // weight gradient of Algorithm 2 with its trust mask: d2[n][k] = M_w[n][k] * sum_m dy[m][n] xq_h[m][k]
        if (had_block == 128 && N > 128 && K > 128) {
            if ((s = launch_gemm_bf16_masked(dy, ws.xh, N, K, M, mw, dw, out_dtype, true, 2, st))) return s;
        } else {
            if ((s = launch_gemm_bf16_masked(dy, ws.xh, N, K, M, mw, ws.d2, QUEST_F32, false, 2, st))) return s;
            if ((s = launch_iht(ws.d2, N, K, had_block, dw, out_dtype, K, st))) return s;
        }
    }
    return QUEST_OK;
}
