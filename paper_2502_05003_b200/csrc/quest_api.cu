// extern "C" entry points of the library: host-side argument validation, workspace carving and
// the launch sequence of each call.  Declarations and argument documentation: include/quest.h.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include "quest_internal.cuh"
#include "quest_operand.cuh"

namespace quest {

// Written by a kernel whose bounded wait expired; read and cleared by quest_device_status.
__device__ int g_timeout_word = 0;

static thread_local char t_cuda_msg[256] = "";

int cuda_fail(cudaError_t e) {
    snprintf(t_cuda_msg, sizeof(t_cuda_msg), "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
    return QUEST_ERR_CUDA;
}
int cuda_fail_msg(const char *msg) {
    snprintf(t_cuda_msg, sizeof(t_cuda_msg), "%s", msg);
    return QUEST_ERR_CUDA;
}

int *device_status_word() {
    static int *cached[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!cached[dev]) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_timeout_word);
        if (e != cudaSuccess) {
            cuda_fail(e);
            return nullptr;
        }
        cached[dev] = reinterpret_cast<int *>(p);
    }
    return cached[dev];
}

int check_device() {
    static int cached[64] = {0};   // 0 unknown, 1 ok, 2 wrong architecture
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= 64) return QUEST_ERR_DEVICE;
    if (!cached[dev]) {
        int major = 0;
        e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) return cuda_fail(e);
        cached[dev] = (major == 10) ? 1 : 2;
    }
    return cached[dev] == 1 ? QUEST_OK : QUEST_ERR_DEVICE;
}

// Optional per-stage timing: CUDA events recorded on the caller's stream around each stage.
struct StageTimer {
    bool enabled = false;
    cudaEvent_t ev[QUEST_NUM_STAGES][2] = {};
    bool created = false;
    bool pending[QUEST_NUM_STAGES] = {};
    bool captured[QUEST_NUM_STAGES] = {};      // recorded inside a stream capture: re-recorded at every graph replay
    double total_ms[QUEST_NUM_STAGES] = {};
    long long count[QUEST_NUM_STAGES] = {};
};
static StageTimer g_timer;

struct StageScope {
    int id;
    cudaStream_t st;
    bool on;
    bool capturing = false;
    StageScope(int id_, cudaStream_t st_) : id(id_), st(st_), on(g_timer.enabled && g_timer.created) {
        if (on) {
            cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
            capturing = cudaStreamIsCapturing(st, &cs) == cudaSuccess && cs == cudaStreamCaptureStatusActive;
            record(g_timer.ev[id][0]);
        }
    }
    void record(cudaEvent_t ev) {
        // inside a capture the record becomes a graph node that times every replay
        if (capturing) cudaEventRecordWithFlags(ev, st, cudaEventRecordExternal);
        else cudaEventRecord(ev, st);
    }
    ~StageScope() {
        if (on) {
            record(g_timer.ev[id][1]);
            if (capturing) g_timer.captured[id] = true;
            else g_timer.pending[id] = true;
        }
    }
};

// Stage brackets for translation units other than this one.
void *stage_begin(int id, cudaStream_t st) { return new StageScope(id, st); }
void stage_end(void *scope) { delete static_cast<StageScope *>(scope); }

static bool is_pow2(int64_t v) { return v > 0 && (v & (v - 1)) == 0; }
static bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

static int validate_quantize(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld, int bits,
                             int had_block, float trust_factor, const uint8_t *codes, const uint8_t *mask) {
    if (!x && rows != 0) return QUEST_ERR_NULL;
    if (dtype != QUEST_F32 && dtype != QUEST_BF16) return QUEST_ERR_DTYPE;
    if (bits < 1 || bits > 8) return QUEST_ERR_BITS;
    if (rows < 0 || rows > (int64_t)1 << 31 || cols < 8 || cols > 16384 || cols % 8 != 0 || ld < cols)
        return QUEST_ERR_SHAPE;
    if (!is_pow2(had_block) || had_block > cols || cols % had_block != 0) return QUEST_ERR_HAD_BLOCK;
    if (!(trust_factor >= 0.0f) || isinf(trust_factor)) return QUEST_ERR_TRUST;
    const size_t esz = dtype == QUEST_F32 ? 4 : 2;
    if (!aligned(x, 16) || (ld * esz) % 16 != 0) return QUEST_ERR_ALIGN;
    if (codes && !aligned(codes, 16)) return QUEST_ERR_ALIGN;
    if (mask && !aligned(mask, 4)) return QUEST_ERR_ALIGN;
    return QUEST_OK;
}

static int validate_gemm_shape(int64_t M, int64_t N, int64_t K, int bits_x, int bits_w) {
    if (bits_x < 1 || bits_x > 8 || bits_w < 1 || bits_w > 8) return QUEST_ERR_BITS;
    if (M < 0 || N < 0 || M > (int64_t)1 << 30 || N > (int64_t)1 << 30 || K < 32 || K % 32 != 0 ||
        K > 65504)
        return QUEST_ERR_SHAPE;
    const int64_t worst = K * (((int64_t)1 << bits_x) - 1) * (((int64_t)1 << bits_w) - 1);
    if (worst >= ((int64_t)1 << 31)) return QUEST_ERR_OVERFLOW;
    return QUEST_OK;
}

}  // namespace quest

using namespace quest;

extern "C" {

float quest_alpha_star(int bits) { return alpha_star(bits); }

size_t quest_codes_bytes(int64_t rows, int64_t cols, int bits) {
    if (rows < 0 || cols < 0 || bits < 1 || bits > 8) return 0;
    return (size_t)rows * (size_t)cols * (size_t)container_bits(bits) / 8;
}

size_t quest_workspace_bytes(int64_t M, int64_t N, int64_t K, int bits_x, int bits_w) {
    if (validate_gemm_shape(M, N, K, bits_x, bits_w) != QUEST_OK) return 0;
    size_t b = carve_workspace(nullptr, M, N, K).bytes;
    return b ? b : 256;
}

const char *quest_status_string(int status) {
    switch (status) {
        case QUEST_OK: return "ok";
        case QUEST_ERR_NULL: return "a required pointer is NULL";
        case QUEST_ERR_SHAPE: return "unsupported shape or leading dimension";
        case QUEST_ERR_BITS: return "bits must be in 1..8";
        case QUEST_ERR_HAD_BLOCK: return "had_block must be a power of two that divides cols";
        case QUEST_ERR_DTYPE: return "unknown dtype code";
        case QUEST_ERR_ALIGN: return "pointer or leading dimension not aligned as required";
        case QUEST_ERR_TRUST: return "trust_factor must be finite and >= 0";
        case QUEST_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case QUEST_ERR_OVERFLOW: return "K*(2^bx-1)*(2^bw-1) does not fit in int32";
        case QUEST_ERR_DEVICE: return "current device is not compute capability 10.x";
        case QUEST_ERR_CUDA: return "CUDA call failed";
        case QUEST_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel expired";
        case QUEST_ERR_STATIC_LIMIT: return "problem too large for the library's static scratch (QUEST_STATIC_SCRATCH_BYTES)";
        default: return "unknown status";
    }
}

const char *quest_last_cuda_error(void) { return t_cuda_msg; }

int quest_device_status(void *stream) {
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    int *word = device_status_word();
    if (!word) return QUEST_ERR_CUDA;
    int v = 0;
    cudaError_t e = cudaMemcpyAsync(&v, word, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e);
    if (v != 0) {
        e = cudaMemsetAsync(word, 0, sizeof(int), st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) return cuda_fail(e);
        return QUEST_ERR_DEVICE_TIMEOUT;
    }
    return QUEST_OK;
}

int quest_last_device_status(void *stream) { return quest_device_status(stream); }

int quest_selftest_bounded_wait(int64_t limit_cycles, int *report, void *stream) {
    if (limit_cycles < 1000 || limit_cycles > 4000000000ll) return QUEST_ERR_SHAPE;
    int s = check_device();
    if (s) return s;
    return launch_bounded_wait_probe(limit_cycles, report, reinterpret_cast<cudaStream_t>(stream));
}

int quest_stage_timing(int enable) {
    if (enable && !g_timer.created) {
        for (int i = 0; i < QUEST_NUM_STAGES; ++i)
            for (int j = 0; j < 2; ++j) {
                cudaError_t e = cudaEventCreate(&g_timer.ev[i][j]);
                if (e != cudaSuccess) return cuda_fail(e);
            }
        g_timer.created = true;
    }
    g_timer.enabled = enable != 0;
    return QUEST_OK;
}

int quest_stage_times(double *total_ms, long long *counts, int reset) {
    for (int i = 0; i < QUEST_NUM_STAGES; ++i) {
        if (g_timer.pending[i] || g_timer.captured[i]) {
            cudaError_t e = cudaEventSynchronize(g_timer.ev[i][1]);
            float ms = 0.0f;
            if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, g_timer.ev[i][0], g_timer.ev[i][1]);
            if (e != cudaSuccess) return cuda_fail(e);
            g_timer.total_ms[i] += ms;
            g_timer.count[i] += 1;
            g_timer.pending[i] = false;
        }
        if (total_ms) total_ms[i] = g_timer.total_ms[i];
        if (counts) counts[i] = g_timer.count[i];
        if (reset) {
            g_timer.total_ms[i] = 0.0;
            g_timer.count[i] = 0;
        }
        if (reset > 1) g_timer.captured[i] = false;
    }
    return QUEST_OK;
}

int quest_quantize(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld_elems,
                   int bits, int had_block, float trust_factor,
                   uint8_t *codes, float *scales, uint8_t *mask, void *stream) {
    int s = validate_quantize(x, dtype, rows, cols, ld_elems, bits, had_block, trust_factor, codes, mask);
    if (s) return s;
    if ((s = check_device())) return s;
    if (rows == 0) return QUEST_OK;
    StageScope scope(QUEST_STAGE_QUANT_X, reinterpret_cast<cudaStream_t>(stream));
    const QuantJob job = {x, rows, ld_elems, codes, scales, mask, nullptr, nullptr};
    return launch_quantize(&job, 1, dtype, cols, bits, had_block, trust_factor, reinterpret_cast<cudaStream_t>(stream));
}

int quest_trust_mask(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld_elems,
                     int bits, int had_block, float trust_factor, uint8_t *mask, void *stream) {
    if (!mask) return QUEST_ERR_NULL;
    int s = validate_quantize(x, dtype, rows, cols, ld_elems, bits, had_block, trust_factor, nullptr, mask);
    if (s) return s;
    if ((s = check_device())) return s;
    if (rows == 0) return QUEST_OK;
    const QuantJob job = {x, rows, ld_elems, nullptr, nullptr, mask, nullptr, nullptr};
    return launch_quantize(&job, 1, dtype, cols, bits, had_block, trust_factor, reinterpret_cast<cudaStream_t>(stream));
}

int quest_lowbit_gemm(const uint8_t *xq, const float *sx, int bits_x,
                      const uint8_t *wq, const float *sw, int bits_w,
                      int64_t M, int64_t N, int64_t K,
                      void *y, int y_dtype, int64_t ldy_elems, int32_t *acc,
                      void *workspace, size_t workspace_bytes, void *stream) {
    int s = validate_gemm_shape(M, N, K, bits_x, bits_w);
    if (s) return s;
    if (M == 0 || N == 0) return QUEST_OK;            /* empty product: nothing to write */
    if (!xq || !wq) return QUEST_ERR_NULL;
    if (!y && !acc) return QUEST_ERR_NULL;
    if (y && (!sx || !sw)) return QUEST_ERR_NULL;
    if (y) {
        if (y_dtype != QUEST_F32 && y_dtype != QUEST_BF16) return QUEST_ERR_DTYPE;
        if (ldy_elems < N) return QUEST_ERR_SHAPE;
        if (!aligned(y, y_dtype == QUEST_F32 ? 4 : 2)) return QUEST_ERR_ALIGN;
    }
    if (!aligned(xq, 16) || !aligned(wq, 16) || (acc && !aligned(acc, 4))) return QUEST_ERR_ALIGN;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < quest_workspace_bytes(M, N, K, bits_x, bits_w))
        return QUEST_ERR_WORKSPACE;
    if ((s = check_device())) return s;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    Workspace ws = carve_workspace(workspace, M, N, K);
    const bool need_rs_a = bits_w == 8;    // sum of x operand values multiplies the offset of the w codes
    const bool need_rs_b = bits_x == 8;
    {
        StageScope scope(QUEST_STAGE_UNPACK, st);
        const bool e4 = e2m1_operands(bits_x, bits_w);
        if ((s = launch_unpack_pair(xq, bits_x, M, ws.a8, need_rs_a ? ws.rs_a : nullptr, wq, bits_w, N, ws.b8,
                                    need_rs_b ? ws.rs_b : nullptr, K, e4, st)))
            return s;
    }
    StageScope scope(QUEST_STAGE_GEMM, st);
    return launch_gemm(ws.a8, ws.b8, ws.rs_a, ws.rs_b, bits_x, bits_w, sx, sw, M, N, K, y, y_dtype, ldy_elems, acc,
                       st);
}

int quest_linear_fwd_quantize(const void *x, const void *w, int dtype, int64_t M, int64_t N, int64_t K,
                              int bits, int had_block, float trust_factor,
                              uint8_t *xq, float *sx, uint8_t *mx,
                              uint8_t *wq, float *sw, uint8_t *mw, int w_is_cached,
                              void *workspace, size_t workspace_bytes, void *stream) {
    if (!xq || !sx || !wq || !sw) return QUEST_ERR_NULL;
    if (!w_is_cached && !w) return QUEST_ERR_NULL;
    if (w_is_cached < 0 || w_is_cached > 2) return QUEST_ERR_SHAPE;
    int s = validate_gemm_shape(M, N, K, bits, bits);
    if (s) return s;
    if ((s = validate_quantize(x, dtype, M, K, K, bits, had_block, trust_factor, xq, mx))) return s;
    if (!w_is_cached && (s = validate_quantize(w, dtype, N, K, K, bits, had_block, trust_factor, wq, mw))) return s;
    if (!aligned(wq, 16)) return QUEST_ERR_ALIGN;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < quest_workspace_bytes(M, N, K, bits, bits))
        return QUEST_ERR_WORKSPACE;
    if ((s = check_device())) return s;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    Workspace ws = carve_workspace(workspace, M, N, K);
    const bool need_rs = bits == 8;
    // codes, scale, mask, the int8 operand (and its row sums for 8-bit codes) in one pass; x and w
    // share one launch when both are quantized
    const QuantJob jx = {x, M, K, xq, sx, mx, ws.a8, need_rs ? ws.rs_a : nullptr};
    if (w_is_cached) {
        {
            StageScope scope(QUEST_STAGE_QUANT_X, st);
            if ((s = launch_quantize(&jx, 1, dtype, K, bits, had_block, trust_factor, st))) return s;
        }
        if (w_is_cached != 2) {      // 2: the workspace still holds w's operand from an earlier call
            StageScope scope(QUEST_STAGE_UNPACK, st);
            if ((s = launch_unpack(wq, bits, N, K, ws.b8, need_rs ? ws.rs_b : nullptr, st, e2m1_operands(bits, bits)))) return s;
        }
    } else {
        StageScope scope(QUEST_STAGE_QUANT_X, st);
        const QuantJob jobs[2] = {jx, {w, N, K, wq, sw, mw, ws.b8, need_rs ? ws.rs_b : nullptr}};
        if ((s = launch_quantize(jobs, 2, dtype, K, bits, had_block, trust_factor, st))) return s;
    }
    return QUEST_OK;
}

int quest_linear_fwd_contract(const float *sx, const float *sw, int64_t M, int64_t N, int64_t K, int bits,
                              void *y, int y_dtype, void *workspace, size_t workspace_bytes, void *stream) {
    if (!y || !sx || !sw) return QUEST_ERR_NULL;
    if (y_dtype != QUEST_F32 && y_dtype != QUEST_BF16) return QUEST_ERR_DTYPE;
    int s = validate_gemm_shape(M, N, K, bits, bits);
    if (s) return s;
    if (!aligned(y, y_dtype == QUEST_F32 ? 4 : 2)) return QUEST_ERR_ALIGN;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < quest_workspace_bytes(M, N, K, bits, bits))
        return QUEST_ERR_WORKSPACE;
    if ((s = check_device())) return s;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    Workspace ws = carve_workspace(workspace, M, N, K);
    StageScope scope(QUEST_STAGE_GEMM, st);
    return launch_gemm(ws.a8, ws.b8, ws.rs_a, ws.rs_b, bits, bits, sx, sw, M, N, K, y, y_dtype, N, nullptr, st);
}

int quest_linear_fwd(const void *x, const void *w, int dtype, int64_t M, int64_t N, int64_t K,
                     int bits, int had_block, float trust_factor,
                     void *y, int y_dtype,
                     uint8_t *xq, float *sx, uint8_t *mx,
                     uint8_t *wq, float *sw, uint8_t *mw, int w_is_cached,
                     void *workspace, size_t workspace_bytes, void *stream) {
    // every argument check of both halves comes before the first launch
    if (!y) return QUEST_ERR_NULL;
    if (y_dtype != QUEST_F32 && y_dtype != QUEST_BF16) return QUEST_ERR_DTYPE;
    if (!aligned(y, y_dtype == QUEST_F32 ? 4 : 2)) return QUEST_ERR_ALIGN;
    int s = quest_linear_fwd_quantize(x, w, dtype, M, N, K, bits, had_block, trust_factor, xq, sx, mx, wq, sw, mw,
                                      w_is_cached, workspace, workspace_bytes, stream);
    if (s) return s;
    return quest_linear_fwd_contract(sx, sw, M, N, K, bits, y, y_dtype, workspace, workspace_bytes, stream);
}

// ---- MLP block: three Algorithm-1 layers with the SwiGLU fused into the first contraction -------

namespace {
struct MlpWorkspace {
    int8_t *b_gu; int32_t *rs_gu;     // operands of w_gate rows [0, I) and w_up rows [I, 2I), K = H
    int8_t *a_x;  int32_t *rs_x;      // operand of x [T x H]
    int8_t *b_d;  int32_t *rs_d;      // operand of w_down [H x I]
    int8_t *a_h;  int32_t *rs_h;      // operand of h [T x I]
    size_t bytes;
};
MlpWorkspace carve_mlp(void *base, int64_t T, int64_t H, int64_t I) {
    MlpWorkspace w;
    uint8_t *b = reinterpret_cast<uint8_t *>(base);
    size_t off = 0;
    auto take = [&](size_t n) { uint8_t *p = b + off; off += align_up(n, 256); return p; };
    w.b_gu = reinterpret_cast<int8_t *>(take((size_t)(2 * I * H)));
    w.rs_gu = reinterpret_cast<int32_t *>(take((size_t)(2 * I) * 4));
    w.a_x = reinterpret_cast<int8_t *>(take((size_t)(T * H)));
    w.rs_x = reinterpret_cast<int32_t *>(take((size_t)T * 4));
    w.b_d = reinterpret_cast<int8_t *>(take((size_t)(H * I)));
    w.rs_d = reinterpret_cast<int32_t *>(take((size_t)H * 4));
    w.a_h = reinterpret_cast<int8_t *>(take((size_t)(T * I)));
    w.rs_h = reinterpret_cast<int32_t *>(take((size_t)T * 4));
    w.bytes = off;
    return w;
}
}  // namespace

size_t quest_mlp_workspace_bytes(int64_t T, int64_t H, int64_t I) {
    if (validate_gemm_shape(T, I, H, 1, 1) != QUEST_OK || validate_gemm_shape(T, H, I, 1, 1) != QUEST_OK) return 0;
    if (H > 16384 || I > 16384) return 0;
    return carve_mlp(nullptr, T, H, I).bytes;
}

int quest_mlp_fwd(const void *x, const void *w_gate, const void *w_up, const void *w_down, int dtype,
                  int64_t T, int64_t H, int64_t I, int bits, int had_block, float trust_factor,
                  void *h, void *y, int y_dtype, const quest_mlp_saved *sv,
                  void *workspace, size_t workspace_bytes, void *stream) {
    if (!x || !w_gate || !w_up || !w_down || !h || !y || !sv) return QUEST_ERR_NULL;
    if (!sv->xq || !sv->sx || !sv->wgq || !sv->swg || !sv->wuq || !sv->swu || !sv->hq || !sv->sh || !sv->wdq || !sv->swd)
        return QUEST_ERR_NULL;
    if (y_dtype != QUEST_F32 && y_dtype != QUEST_BF16) return QUEST_ERR_DTYPE;
    int s = validate_gemm_shape(T, I, H, bits, bits);
    if (s) return s;
    if ((s = validate_gemm_shape(T, H, I, bits, bits))) return s;
    if ((s = validate_quantize(x, dtype, T, H, H, bits, had_block, trust_factor, sv->xq, sv->mx))) return s;
    if ((s = validate_quantize(w_gate, dtype, I, H, H, bits, had_block, trust_factor, sv->wgq, sv->mwg))) return s;
    if ((s = validate_quantize(w_up, dtype, I, H, H, bits, had_block, trust_factor, sv->wuq, sv->mwu))) return s;
    if ((s = validate_quantize(h, QUEST_BF16, T, I, I, bits, had_block, trust_factor, sv->hq, sv->mh))) return s;
    if ((s = validate_quantize(w_down, dtype, H, I, I, bits, had_block, trust_factor, sv->wdq, sv->mwd))) return s;
    if (!aligned(y, y_dtype == QUEST_F32 ? 4 : 2)) return QUEST_ERR_ALIGN;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < quest_mlp_workspace_bytes(T, H, I))
        return QUEST_ERR_WORKSPACE;
    if (T == 0) return QUEST_OK;
    if ((s = check_device())) return s;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    MlpWorkspace ws = carve_mlp(workspace, T, H, I);
    const bool rs = bits == 8;
    const size_t up_off = (size_t)I * (size_t)(e2m1_operands(bits, bits) ? H / 2 : H);   // operand bytes of the gate rows
    {
        StageScope scope(QUEST_STAGE_QUANT_X, st);
        const QuantJob jobs[3] = {{x, T, H, sv->xq, sv->sx, sv->mx, ws.a_x, rs ? ws.rs_x : nullptr},
                                  {w_gate, I, H, sv->wgq, sv->swg, sv->mwg, ws.b_gu, rs ? ws.rs_gu : nullptr},
                                  {w_up, I, H, sv->wuq, sv->swu, sv->mwu, ws.b_gu + up_off, rs ? ws.rs_gu + I : nullptr}};
        if ((s = launch_quantize(jobs, 3, dtype, H, bits, had_block, trust_factor, st))) return s;
    }
    {
        StageScope scope(QUEST_STAGE_GEMM, st);
        if ((s = launch_gemm_swiglu(ws.a_x, ws.b_gu, ws.rs_x, ws.rs_gu, bits, sv->sx, sv->swg, sv->swu, T, I, H, h, st))) return s;
    }
    {
        StageScope scope(QUEST_STAGE_QUANT_W, st);
        const QuantJob jh = {h, T, I, sv->hq, sv->sh, sv->mh, ws.a_h, rs ? ws.rs_h : nullptr};
        const QuantJob jd = {w_down, H, I, sv->wdq, sv->swd, sv->mwd, ws.b_d, rs ? ws.rs_d : nullptr};
        if (dtype == QUEST_BF16) {
            const QuantJob jobs[2] = {jh, jd};
            if ((s = launch_quantize(jobs, 2, QUEST_BF16, I, bits, had_block, trust_factor, st))) return s;
        } else {
            if ((s = launch_quantize(&jh, 1, QUEST_BF16, I, bits, had_block, trust_factor, st))) return s;
            if ((s = launch_quantize(&jd, 1, dtype, I, bits, had_block, trust_factor, st))) return s;
        }
    }
    StageScope scope(QUEST_STAGE_GEMM, st);
    return launch_gemm(ws.a_h, ws.b_d, ws.rs_h, ws.rs_d, bits, bits, sv->sh, sv->swd, T, H, I, y, y_dtype, H, nullptr, st);
}

// ---- FP4 (E2M1) grid variant (Section 4.4, "The FP4 Format") -----------------------------------

float quest_alpha_star_fp4(void) { return alpha_star_fp4(); }

int quest_quantize_fp4(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld_elems,
                       int had_block, float trust_factor,
                       uint8_t *codes, float *scales, uint8_t *mask, void *stream) {
    int s = validate_quantize(x, dtype, rows, cols, ld_elems, 4, had_block, trust_factor, codes, mask);
    if (s) return s;
    if (cols % 32 != 0) return QUEST_ERR_SHAPE;
    if ((s = check_device())) return s;
    if (rows == 0) return QUEST_OK;
    const QuantJob job = {x, rows, ld_elems, codes, scales, mask, nullptr, nullptr};
    return launch_quantize(&job, 1, dtype, cols, 4, had_block, trust_factor, reinterpret_cast<cudaStream_t>(stream),
                           GRID_FP4);
}

int quest_lowbit_gemm_fp4(const uint8_t *xq, const float *sx, const uint8_t *wq, const float *sw,
                          int64_t M, int64_t N, int64_t K,
                          void *y, int y_dtype, int64_t ldy_elems, int32_t *acc4,
                          void *workspace, size_t workspace_bytes, void *stream) {
    int s = validate_gemm_shape(M, N, K, 4, 4);
    if (s) return s;
    if (M == 0 || N == 0) return QUEST_OK;
    if (!xq || !wq) return QUEST_ERR_NULL;
    if (!y && !acc4) return QUEST_ERR_NULL;
    if (y && (!sx || !sw)) return QUEST_ERR_NULL;
    if (y) {
        if (y_dtype != QUEST_F32 && y_dtype != QUEST_BF16) return QUEST_ERR_DTYPE;
        if (ldy_elems < N) return QUEST_ERR_SHAPE;
        if (!aligned(y, y_dtype == QUEST_F32 ? 4 : 2)) return QUEST_ERR_ALIGN;
    }
    if (!aligned(xq, 16) || !aligned(wq, 16) || (acc4 && !aligned(acc4, 4))) return QUEST_ERR_ALIGN;
    if ((s = check_device())) return s;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    (void)workspace;
    (void)workspace_bytes;
    StageScope scope(QUEST_STAGE_GEMM, st);
    return launch_gemm_e2m1(xq, wq, sx, sw, M, N, K, y, y_dtype, ldy_elems, acc4, 4, st);
}

int quest_linear_fwd_fp4(const void *x, const void *w, int dtype, int64_t M, int64_t N, int64_t K,
                         int had_block, float trust_factor,
                         void *y, int y_dtype,
                         uint8_t *xq, float *sx, uint8_t *mx,
                         uint8_t *wq, float *sw, uint8_t *mw, int w_is_cached,
                         void *workspace, size_t workspace_bytes, void *stream) {
    if (!y || !xq || !sx || !wq || !sw) return QUEST_ERR_NULL;
    if (!w_is_cached && !w) return QUEST_ERR_NULL;
    if (y_dtype != QUEST_F32 && y_dtype != QUEST_BF16) return QUEST_ERR_DTYPE;
    int s = validate_gemm_shape(M, N, K, 4, 4);
    if (s) return s;
    if ((s = validate_quantize(x, dtype, M, K, K, 4, had_block, trust_factor, xq, mx))) return s;
    if (!w_is_cached && (s = validate_quantize(w, dtype, N, K, K, 4, had_block, trust_factor, wq, mw))) return s;
    if (!aligned(xq, 16) || !aligned(wq, 16) || !aligned(y, y_dtype == QUEST_F32 ? 4 : 2)) return QUEST_ERR_ALIGN;
    if ((s = check_device())) return s;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    (void)workspace;
    (void)workspace_bytes;
    // the packed codes are the tensor-core operands: nothing is unpacked
    const QuantJob jx = {x, M, K, xq, sx, mx, nullptr, nullptr};
    {
        StageScope scope(QUEST_STAGE_QUANT_X, st);
        if (w_is_cached) {
            if ((s = launch_quantize(&jx, 1, dtype, K, 4, had_block, trust_factor, st, GRID_FP4))) return s;
        } else {
            const QuantJob jobs[2] = {jx, {w, N, K, wq, sw, mw, nullptr, nullptr}};
            if ((s = launch_quantize(jobs, 2, dtype, K, 4, had_block, trust_factor, st, GRID_FP4))) return s;
        }
    }
    StageScope scope(QUEST_STAGE_GEMM, st);
    return launch_gemm_e2m1(xq, wq, sx, sw, M, N, K, y, y_dtype, N, nullptr, 4, st);
}

}  // extern "C"
