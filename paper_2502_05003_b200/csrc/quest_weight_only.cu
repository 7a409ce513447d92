// Weight-only variant of the forward pass (Section 4.5, "Weight-only quantization"): Algorithm 1 with the
// rounding of the activations left out.  The weights go through the full quantizer; the
// activations are rotated by the same block Hadamard transform and stay in bfloat16:
//
//   x_h = bf16(HT(x))                     launch_hadamard_rows  (binary32 butterflies, one rounding)
//   w -> codes, sw, trust mask            launch_quantize
//   c_w = bf16(2k - (2^b - 1))            codes_to_bf16_kernel  (exact: |c| <= 255)
//   y[m][n] = sw[n] sum_k x_h[m][k] c_w[n][k]    tcgen05 kind::f16 contraction, binary32 accumulators
#include <cuda_bf16.h>

#include "quest_internal.cuh"

namespace quest {
namespace {

// One thread converts 32 consecutive elements of a row (rows are dense, K % 32 == 0).
template <int CB>
__global__ void __launch_bounds__(256)
codes_to_bf16_kernel(const uint8_t *__restrict__ codes, int bits, long long n_groups, uint16_t *__restrict__ out) {
    pdl_launch_dependents();
    pdl_wait();
    const long long gidx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (gidx >= n_groups) return;
    constexpr int PER = 32 / CB;
    const int L1 = (1 << bits) - 1;
    uint32_t w[CB];
    const uint32_t *src = reinterpret_cast<const uint32_t *>(codes) + gidx * CB;
#pragma unroll
    for (int q = 0; q < CB; ++q) w[q] = __ldg(src + q);
    uint4 *dst = reinterpret_cast<uint4 *>(out + gidx * 32);
#pragma unroll
    for (int q = 0; q < 4; ++q) {                       // 8 elements per 16-byte store
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int e0 = 8 * q + 2 * j, e1 = e0 + 1;
            const int k0 = (w[e0 / PER] >> ((e0 % PER) * CB)) & ((1 << CB) - 1);
            const int k1 = (w[e1 / PER] >> ((e1 % PER) * CB)) & ((1 << CB) - 1);
            // a small integer as bfloat16: the upper half of its binary32 pattern (no rounding: |c| <= 255)
            o[j] = (__float_as_uint((float)(2 * k0 - L1)) >> 16) | (__float_as_uint((float)(2 * k1 - L1)) & 0xFFFF0000u);
        }
        dst[q] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

struct WoWorkspace {
    uint16_t *xh;      // [M x K] rotated activations
    uint16_t *cw;      // [N x K] grid values of w
    uint8_t *wq;       // packed codes of w when the caller does not keep them
    float *sw;         // [N] scales when the caller does not keep them
    size_t bytes;
};
WoWorkspace carve_wo(void *base, int64_t M, int64_t N, int64_t K) {
    WoWorkspace w;
    uint8_t *b = reinterpret_cast<uint8_t *>(base);
    size_t off = 0;
    auto take = [&](size_t n) { uint8_t *p = b + off; off += align_up(n, 256); return p; };
    w.xh = reinterpret_cast<uint16_t *>(take((size_t)M * K * 2));
    w.cw = reinterpret_cast<uint16_t *>(take((size_t)N * K * 2));
    w.wq = take((size_t)N * K);
    w.sw = reinterpret_cast<float *>(take((size_t)N * 4));
    w.bytes = off;
    return w;
}

bool wo_shape_ok(int64_t M, int64_t N, int64_t K) {
    return M >= 0 && N >= 0 && K >= 32 && K % 32 == 0 && K <= 16384 && M <= ((int64_t)1 << 24) && N <= ((int64_t)1 << 24);
}

}  // namespace

int launch_codes_to_bf16(const uint8_t *codes, int bits, int64_t rows, int64_t K, void *out, cudaStream_t st) {
    const long long n_groups = (long long)rows * (K / 32);
    if (n_groups == 0) return QUEST_OK;
    const dim3 grid((unsigned)((n_groups + 255) / 256));
    uint16_t *o = reinterpret_cast<uint16_t *>(out);
    cudaError_t e;
    switch (container_bits(bits)) {
        case 1: e = launch_pdl(codes_to_bf16_kernel<1>, grid, dim3(256), 0, st, 1, codes, bits, n_groups, o); break;
        case 2: e = launch_pdl(codes_to_bf16_kernel<2>, grid, dim3(256), 0, st, 1, codes, bits, n_groups, o); break;
        case 4: e = launch_pdl(codes_to_bf16_kernel<4>, grid, dim3(256), 0, st, 1, codes, bits, n_groups, o); break;
        default: e = launch_pdl(codes_to_bf16_kernel<8>, grid, dim3(256), 0, st, 1, codes, bits, n_groups, o); break;
    }
    return e == cudaSuccess ? QUEST_OK : cuda_fail(e);
}

}  // namespace quest

using namespace quest;

extern "C" size_t quest_weight_only_workspace_bytes(int64_t M, int64_t N, int64_t K) {
    if (!wo_shape_ok(M, N, K)) return 0;
    return carve_wo(nullptr, M, N, K).bytes;
}

extern "C" int quest_linear_fwd_weight_only(const void *x, int x_dtype, int64_t ldx, const void *w, int w_dtype, int64_t ldw,
                                            int64_t M, int64_t N, int64_t K, int bits_w, int had_block, float trust_factor,
                                            void *y, int y_dtype, int64_t ldy, void *xh, uint8_t *wq, float *sw, uint8_t *mw,
                                            void *workspace, size_t workspace_bytes, void *stream) {
    if (M > 0 && N > 0 && (!x || !w || !y)) return QUEST_ERR_NULL;
    if ((x_dtype != QUEST_F32 && x_dtype != QUEST_BF16) || (w_dtype != QUEST_F32 && w_dtype != QUEST_BF16) ||
        (y_dtype != QUEST_F32 && y_dtype != QUEST_BF16))
        return QUEST_ERR_DTYPE;
    if (bits_w < 1 || bits_w > 8) return QUEST_ERR_BITS;
    if (!wo_shape_ok(M, N, K) || ldx < K || ldw < K || ldy < N) return QUEST_ERR_SHAPE;
    if (had_block < 1 || (had_block & (had_block - 1)) != 0 || had_block > K || K % had_block != 0)
        return QUEST_ERR_HAD_BLOCK;
    if (!(trust_factor >= 0.0f)) return QUEST_ERR_TRUST;
    auto al = [](const void *p, size_t a) { return reinterpret_cast<uintptr_t>(p) % a == 0; };
    const size_t xes = x_dtype == QUEST_F32 ? 4 : 2, wes = w_dtype == QUEST_F32 ? 4 : 2, yes = y_dtype == QUEST_F32 ? 4 : 2;
    if (!al(x, 16) || (size_t)ldx * xes % 16 != 0 || !al(w, 16) || (size_t)ldw * wes % 16 != 0 || !al(y, yes) ||
        (xh && !al(xh, 16)) || (wq && !al(wq, 4)) || (sw && !al(sw, 4)))
        return QUEST_ERR_ALIGN;
    if (!workspace || !al(workspace, 256) || workspace_bytes < quest_weight_only_workspace_bytes(M, N, K))
        return QUEST_ERR_WORKSPACE;
    if (M == 0 || N == 0) return QUEST_OK;
    int s = check_device();
    if (s) return s;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    WoWorkspace ws = carve_wo(workspace, M, N, K);
    uint16_t *xh_buf = xh ? reinterpret_cast<uint16_t *>(xh) : ws.xh;
    uint8_t *wq_buf = wq ? wq : ws.wq;
    float *sw_buf = sw ? sw : ws.sw;
    {
        void *h = stage_begin(QUEST_STAGE_QUANT_W, st);
        QuantJob job = {w, N, ldw, wq_buf, sw_buf, mw, nullptr, nullptr};
        s = launch_quantize(&job, 1, w_dtype, K, bits_w, had_block, trust_factor, st);
        stage_end(h);
        if (s) return s;
    }
    {
        void *h = stage_begin(QUEST_STAGE_UNPACK, st);
        s = launch_hadamard_rows(x, x_dtype, ldx, M, K, had_block, xh_buf, QUEST_BF16, K, st);
        if (!s) s = launch_codes_to_bf16(wq_buf, bits_w, N, K, ws.cw, st);
        stage_end(h);
        if (s) return s;
    }
    void *h = stage_begin(QUEST_STAGE_GEMM, st);
    s = launch_gemm_bf16_scaled(xh_buf, ws.cw, sw_buf, M, N, K, y, y_dtype, ldy, st);
    stage_end(h);
    return s;
}
