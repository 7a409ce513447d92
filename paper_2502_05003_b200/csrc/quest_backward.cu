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

// dy [M x N] bfloat16 -> a1 [M x N], a2 [N x M]; 32 x 32 tiles, block (32, 8).
__global__ void __launch_bounds__(256)
scale_dy_kernel(const uint16_t *__restrict__ dy, const float *__restrict__ sx, const float *__restrict__ sw,
                int M, int N, uint16_t *__restrict__ a1, uint16_t *__restrict__ a2) {
    __shared__ uint16_t tile[32][34];
    pdl_launch_dependents();
    pdl_wait();
    const int m0 = blockIdx.y * 32, n0 = blockIdx.x * 32;
    const int tx = threadIdx.x, ty = threadIdx.y;
    const int n = n0 + tx;
    const float swn = n < N ? __ldg(sw + n) : 0.0f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty + 8 * i;
        float v = 0.0f;
        if (m < M && n < N) v = __uint_as_float((uint32_t)__ldg(dy + (long long)m * N + n) << 16);
        if (m < M && n < N) a1[(long long)m * N + n] = bf16_bits(v * swn);
        const float sxm = m < M ? __ldg(sx + m) : 0.0f;
        tile[ty + 8 * i][tx] = bf16_bits(v * sxm);
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int nn = n0 + ty + 8 * i, mm = m0 + tx;
        if (nn < N && mm < M) a2[(long long)nn * M + mm] = tile[tx][ty + 8 * i];
    }
}

// packed codes [rows x K] -> ct [K x rows] bfloat16 grid values; 32 x 32 tiles, block (32, 8).
__global__ void __launch_bounds__(256)
codes_to_bf16_t_kernel(const uint8_t *__restrict__ codes, int bits, int rows, int K, uint16_t *__restrict__ ct) {
    __shared__ uint16_t tile[32][34];
    pdl_launch_dependents();
    pdl_wait();
    const int cb = container_bits(bits);
    const int per = 8 / cb;
    const int L1 = (1 << bits) - 1;
    const int r0 = blockIdx.y * 32, k0 = blockIdx.x * 32;
    const int tx = threadIdx.x, ty = threadIdx.y;
    const long long row_bytes = (long long)K * cb / 8;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = r0 + ty + 8 * i, k = k0 + tx;
        float c = 0.0f;
        if (r < rows && k < K) {
            const int byte = __ldg(codes + r * row_bytes + k / per);
            const int lev = (byte >> ((k % per) * cb)) & ((1 << cb) - 1);
            c = (float)(2 * lev - L1);
        }
        tile[ty + 8 * i][tx] = bf16_bits(c);               // |c| <= 255: exact
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int kk = k0 + ty + 8 * i, rr = r0 + tx;
        if (kk < K && rr < rows) ct[(long long)kk * rows + rr] = tile[tx][ty + 8 * i];
    }
}

// Inverse orthonormal block Hadamard transform of every row of d [rows x cols] (binary32, dense),
// stored as out_dtype with row stride ld.  Every thread owns 32 contiguous elements; descending
// stride: partners in other warps through shared memory, partners in this warp through shuffles,
// the rest in registers.  A row of T = cols/32 threads occupies S slots as in the quantizer.
__global__ void __launch_bounds__(512)
iht_rows_kernel(const float *__restrict__ d, long long rows, int cols, int had_block, float inv_sqrt_g,
                void *__restrict__ out, int out_dtype, long long ld, int S, int R) {
    extern __shared__ float xsm[];                 // [32][blockDim.x] exchange
    pdl_launch_dependents();
    pdl_wait();
    const int tid = threadIdx.x, lane = tid & 31, nthreads = blockDim.x;
    const int r_local = tid / S;
    const int tr = tid - r_local * S;
    const long long row = (long long)blockIdx.x * R + r_local;
    const bool active = row < rows && tr < cols / 32;
    float v[32];
    if (active) {
        const float4 *src = reinterpret_cast<const float4 *>(d + row * cols + (long long)tr * 32);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float4 w = __ldg(src + q);
            v[4 * q] = w.x; v[4 * q + 1] = w.y; v[4 * q + 2] = w.z; v[4 * q + 3] = w.w;
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
    cudaError_t e = launch_pdl(iht_rows_kernel, dim3((unsigned)grid), dim3(threads), smem, st, 1, d, (long long)rows, (int)cols,
                               had_block, 1.0f / sqrtf((float)had_block), out, out_dtype, (long long)ld, S, R);
    return e == cudaSuccess ? QUEST_OK : cuda_fail(e);
}

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
    if (!al(dy, 16) || !al(mx, 4) || !al(mw, 4) || (dx && !al(dx, 16)) || (dw && !al(dw, 16))) return QUEST_ERR_ALIGN;
    if (!workspace || !al(workspace, 256) || workspace_bytes < quest_bwd_workspace_bytes(M, N, K))
        return QUEST_ERR_WORKSPACE;
    int s = check_device();
    if (s) return s;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    BwdWorkspace ws = carve_bwd(workspace, M, N, K);
    const dim3 blk(32, 8);
    cudaError_t e = launch_pdl(scale_dy_kernel, dim3((unsigned)((N + 31) / 32), (unsigned)((M + 31) / 32)), blk, 0, st, 1,
                               reinterpret_cast<const uint16_t *>(dy), sx, sw, (int)M, (int)N, ws.a1, ws.a2);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dx) {
        e = launch_pdl(codes_to_bf16_t_kernel, dim3((unsigned)((K + 31) / 32), (unsigned)((N + 31) / 32)), blk, 0, st, 1, wq, bits,
                       (int)N, (int)K, ws.cwt);
        if (e != cudaSuccess) return cuda_fail(e);
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
        e = launch_pdl(codes_to_bf16_t_kernel, dim3((unsigned)((K + 31) / 32), (unsigned)((M + 31) / 32)), blk, 0, st, 1, xq, bits,
                       (int)M, (int)K, ws.cxt);
        if (e != cudaSuccess) return cuda_fail(e);
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
