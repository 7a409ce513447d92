// Weight-only variant of the forward pass (Section 4.5, "Weight-only quantization"): Algorithm 1 with the
// rounding of the activations left out.  The weights go through the full quantizer; the
// activations are rotated by the same block Hadamard transform and stay in bfloat16:
//
//   x_h = bf16(HT(x))                     quantizer launch, rotation output (binary32 butterflies, one rounding)
//   w -> codes, sw, trust mask,           same launch
//        c_w = bf16(2k - (2^b - 1))       (exact: |c| <= 255)
//   y[m][n] = sw[n] sum_k x_h[m][k] c_w[n][k]    tcgen05 kind::f16 contraction, binary32 accumulators
#include <cuda_bf16.h>

#include "quest_internal.cuh"

namespace quest {
namespace {

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
        // one launch when x and w share a type: rows of x leave as x_h, rows of w as codes, scale, mask and
        // bfloat16 grid values
        void *h = stage_begin(QUEST_STAGE_QUANT_W, st);
        QuantJob jobs[2];
        jobs[0] = QuantJob{x, M, ldx, nullptr, nullptr, nullptr, nullptr, nullptr, xh_buf, nullptr};
        jobs[1] = QuantJob{w, N, ldw, wq_buf, sw_buf, mw, nullptr, nullptr, nullptr, ws.cw};
        if (x_dtype == w_dtype) {
            s = launch_quantize(jobs, 2, x_dtype, K, bits_w, had_block, trust_factor, st);
        } else {
            s = launch_quantize(&jobs[0], 1, x_dtype, K, bits_w, had_block, trust_factor, st);
            if (!s) s = launch_quantize(&jobs[1], 1, w_dtype, K, bits_w, had_block, trust_factor, st);
        }
        stage_end(h);
        if (s) return s;
    }
    void *h = stage_begin(QUEST_STAGE_GEMM, st);
    s = launch_gemm_bf16_scaled(xh_buf, ws.cw, sw_buf, M, N, K, y, y_dtype, ldy, st);
    stage_end(h);
    return s;
}
