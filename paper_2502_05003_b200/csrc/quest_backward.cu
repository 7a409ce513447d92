// QuEST training backward for one linear layer (Algorithm 2) on sm_100a:
//
//   dL/dxq_h = dL/dy wq_h                      dL/dx = IHT(M(x_h; xq_h) * dL/dxq_h)
//   dL/dwq_h = dL/dy^T xq_h                    dL/dw = IHT(M(w_h; wq_h) * dL/dwq_h)
//
// The products run in 16-bit precision on the tensor cores (Section 3.3, "Implementation"): the
// integer grid values c = 2k - (2^b - 1) are exact in bfloat16, and the per-row scale of the
// quantized operand is folded into dL/dy before it is rounded to bfloat16 (the scale multiplies
// the contraction index, so it cannot be pulled out of the sum).  Stages:
//   1. scale_dy_kernel        a1[m][n] = bf16(dy[m][n] sw[n])         (operand of line 2)
//                             a2[n][m] = bf16(dy[m][n] sx[m])         (operand of line 4, transposed)
//   2. codes_to_bf16_t_kernel ct[k][r] = bf16(c[r][k])  for w and x   (K-major operands)
//   3. gemm (quest_gemm.cu, bfloat16 mode): masked binary32 products  d1 [M x K], d2 [N x K]
//   4. iht_rows_kernel        block Hadamard transform, 1/sqrt(g), store in the output type
//      (for blocks of 128 stages 3 and 4 are one kernel: the transform runs in the GEMM epilogue,
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

// dy [M x N] bfloat16 -> a1 [M x N] = dy * sw[n], a2 [N x M] = (dy * sx[m])^T, both rounded to bfloat16.
// 64 x 64 tiles, 256 threads, 16-byte accesses on both sides (M and N are multiples of 8, so an
// 8-element chunk is inside or outside the matrix as a whole).
__global__ void __launch_bounds__(256)
scale_dy_kernel(const uint16_t *__restrict__ dy, const float *__restrict__ sx, const float *__restrict__ sw,
                int M, int N, uint16_t *__restrict__ a1, uint16_t *__restrict__ a2) {
    __shared__ uint32_t tile[64][33];                          // [m][n pairs]; odd pitch keeps the transposed reads apart
    pdl_launch_dependents();
    pdl_wait();
    const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
    const int t = threadIdx.x;
    const int chunk = t & 7;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int ml = (t >> 3) + 32 * i;
        const int m = m0 + ml, n = n0 + chunk * 8;
        uint32_t q[4] = {0u, 0u, 0u, 0u};
        if (m < M && n < N) {
            const uint4 w = __ldg(reinterpret_cast<const uint4 *>(dy + (long long)m * N + n));
            const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
            const float sxm = __ldg(sx + m);
            const float4 s0 = __ldg(reinterpret_cast<const float4 *>(sw + n));
            const float4 s1 = __ldg(reinterpret_cast<const float4 *>(sw + n + 4));
            const float swn[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
            uint32_t o[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float lo = __uint_as_float(ww[j] << 16), hi = __uint_as_float(ww[j] & 0xFFFF0000u);
                o[j] = (uint32_t)bf16_bits(lo * swn[2 * j]) | ((uint32_t)bf16_bits(hi * swn[2 * j + 1]) << 16);
                q[j] = (uint32_t)bf16_bits(lo * sxm) | ((uint32_t)bf16_bits(hi * sxm) << 16);
            }
            *reinterpret_cast<uint4 *>(a1 + (long long)m * N + n) = make_uint4(o[0], o[1], o[2], o[3]);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) tile[ml][chunk * 4 + j] = q[j];
    }
    __syncthreads();
    const uint16_t *t16 = reinterpret_cast<const uint16_t *>(&tile[0][0]);
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int nl = (t >> 3) + 32 * i;
        const int n = n0 + nl, m = m0 + chunk * 8;
        if (n < N && m < M) {
            uint32_t o[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
                o[j] = (uint32_t)t16[(chunk * 8 + 2 * j) * 66 + nl] | ((uint32_t)t16[(chunk * 8 + 2 * j + 1) * 66 + nl] << 16);
            *reinterpret_cast<uint4 *>(a2 + (long long)n * M + m) = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
}

// packed codes [rows x K] -> ct [K x rows] bfloat16 grid values c = 2k - (2^b - 1).
// Tiles of 64 rows x 128 columns, 256 threads: a thread expands whole 32-bit code words into
// shared memory, then the tile leaves transposed in 16-byte pieces (rows is a multiple of 8).
template <int CB>
__global__ void __launch_bounds__(256)
codes_to_bf16_t_kernel(const uint8_t *__restrict__ codes, int bits, int rows, int K, uint16_t *__restrict__ ct) {
    __shared__ __align__(16) uint16_t tile[128][72];           // [k][row], pitch 144 bytes
    pdl_launch_dependents();
    pdl_wait();
    constexpr int PER = 32 / CB;                               // codes per word
    constexpr int WPR = 128 / PER;                             // words per tile row
    const int L1 = (1 << bits) - 1;
    const int r0 = blockIdx.y * 64, k0 = blockIdx.x * 128;
    const int t = threadIdx.x;
    const long long row_words = (long long)K * CB / 32;
#pragma unroll
    for (int i = 0; i < (64 * WPR) / 256; ++i) {
        const int w = t + 256 * i;
        const int rl = w & 63, wl = w >> 6;                    // consecutive lanes: consecutive rows (conflict-free tile writes)
        const int r = r0 + rl, k = k0 + wl * PER;
        uint32_t word = 0;
        const bool ok = r < rows && k < K;
        if (ok) word = __ldg(reinterpret_cast<const uint32_t *>(codes) + r * row_words + (k0 / PER) + wl);
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const int lev = (word >> (j * CB)) & ((1 << CB) - 1);
            tile[wl * PER + j][rl] = ok ? bf16_bits((float)(2 * lev - L1)) : (uint16_t)0;    // |c| <= 255: exact
        }
    }
    __syncthreads();
    const int chunk = t & 7;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int kl = (t >> 3) + 32 * i;
        const int k = k0 + kl, r = r0 + chunk * 8;
        if (k < K && r < rows)
            *reinterpret_cast<uint4 *>(ct + (long long)k * rows + r) = *reinterpret_cast<const uint4 *>(&tile[kl][chunk * 8]);
    }
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
    uint16_t *a1, *a2, *cwt, *cxt;
    float *d1, *d2;
    size_t bytes;
};
BwdWorkspace carve_bwd(void *base, int64_t M, int64_t N, int64_t K) {
    BwdWorkspace w;
    uint8_t *b = reinterpret_cast<uint8_t *>(base);
    size_t off = 0;
    auto take = [&](size_t n) { uint8_t *p = b + off; off += align_up(n, 256); return p; };
    w.a1 = reinterpret_cast<uint16_t *>(take((size_t)M * N * 2));
    w.a2 = reinterpret_cast<uint16_t *>(take((size_t)M * N * 2));
    w.cwt = reinterpret_cast<uint16_t *>(take((size_t)K * N * 2));
    w.cxt = reinterpret_cast<uint16_t *>(take((size_t)K * M * 2));
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
    const int R = S >= 256 ? 1 : 256 / S;
    const int threads = R * S;
    const size_t smem = had_block >= 2048 ? sizeof(float) * 32 * (size_t)threads : 0;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(iht_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 72 * 1024);
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
    if (!al(dy, 16) || !al(mx, 16) || !al(mw, 16) || !al(sw, 16) || !al(xq, 4) || !al(wq, 4) || (dx && !al(dx, 16)) ||
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
    Stage *prep = new Stage(QUEST_STAGE_UNPACK, st);   // operand preparation of the whole call up to the first product
    cudaError_t e = launch_pdl(scale_dy_kernel, dim3((unsigned)((N + 63) / 64), (unsigned)((M + 63) / 64)), dim3(256), 0, st, 1,
                               reinterpret_cast<const uint16_t *>(dy), sx, sw, (int)M, (int)N, ws.a1, ws.a2);
    if (e != cudaSuccess) { delete prep; return cuda_fail(e); }
    auto codes_t = [&](const uint8_t *codes, int64_t rows, uint16_t *ct) -> cudaError_t {
        const dim3 grid((unsigned)((K + 127) / 128), (unsigned)((rows + 63) / 64));
        switch (container_bits(bits)) {
            case 1: return launch_pdl(codes_to_bf16_t_kernel<1>, grid, dim3(256), 0, st, 1, codes, bits, (int)rows, (int)K, ct);
            case 2: return launch_pdl(codes_to_bf16_t_kernel<2>, grid, dim3(256), 0, st, 1, codes, bits, (int)rows, (int)K, ct);
            case 4: return launch_pdl(codes_to_bf16_t_kernel<4>, grid, dim3(256), 0, st, 1, codes, bits, (int)rows, (int)K, ct);
            default: return launch_pdl(codes_to_bf16_t_kernel<8>, grid, dim3(256), 0, st, 1, codes, bits, (int)rows, (int)K, ct);
        }
    };
    if (dx) {
        e = codes_t(wq, N, ws.cwt);
        if (prep) { delete prep; prep = nullptr; }
        if (e != cudaSuccess) return cuda_fail(e);
        Stage gemm_stage(QUEST_STAGE_GEMM, st);
        // line 2 and the mask of line 3: d1[m][k] = M_x[m][k] * sum_n a1[m][n] cwt[k][n]
        // (blocks of 128: the inverse transform is fused into the contraction's epilogue)
        if (had_block == 128 && M > 128 && K > 128) {
            if ((s = launch_gemm_bf16_masked(ws.a1, ws.cwt, M, K, N, mx, dx, out_dtype, true, st))) return s;
        } else {
            if ((s = launch_gemm_bf16_masked(ws.a1, ws.cwt, M, K, N, mx, ws.d1, QUEST_F32, false, st))) return s;
            if ((s = launch_iht(ws.d1, M, K, had_block, dx, out_dtype, K, st))) return s;
        }
    }
    if (dw) {
        e = codes_t(xq, M, ws.cxt);
        if (prep) { delete prep; prep = nullptr; }
        if (e != cudaSuccess) return cuda_fail(e);
        Stage gemm_stage(QUEST_STAGE_GEMM, st);
        // line 4 and the mask of line 5: d2[n][k] = M_w[n][k] * sum_m a2[n][m] cxt[k][m]
        if (had_block == 128 && N > 128 && K > 128) {
            if ((s = launch_gemm_bf16_masked(ws.a2, ws.cxt, N, K, M, mw, dw, out_dtype, true, st))) return s;
        } else {
            if ((s = launch_gemm_bf16_masked(ws.a2, ws.cxt, N, K, M, mw, ws.d2, QUEST_F32, false, st))) return s;
            if ((s = launch_iht(ws.d2, N, K, had_block, dw, out_dtype, K, st))) return s;
        }
    }
    return QUEST_OK;
}
