// Internal declarations shared by the translation units of the library (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "quest.h"

namespace quest {

// alpha*(b), b = 1..8 (Section 3.1): minimiser of the Gaussian quantisation MSE on the
// 2^b-point grid, rounded to binary32.
__host__ __device__ inline float alpha_star(int bits) {
    switch (bits) {
        case 1: return 0.7978846f;
        case 2: return 1.4935300f;
        case 3: return 2.0510680f;
        case 4: return 2.5140045f;
        case 5: return 2.9161513f;
        case 6: return 3.2779846f;
        case 7: return 3.6110970f;
        case 8: return 3.9222038f;
        default: return 0.0f;
    }
}

__host__ __device__ inline int container_bits(int bits) {
    return bits == 1 ? 1 : bits == 2 ? 2 : bits <= 4 ? 4 : 8;
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Per-row constants of the projection, computed once on the host in binary32.
struct QuantConsts {
    float c0;      // (2^b-1)/2: centre of the level axis
    float top;     // 2^b-1: highest level
    float A;       // (2^b-1)/(2 alpha*): RMS-normalised value -> level-axis slope
    float B;       // alpha*/((2^b-1) sqrt(g)): RMS of the un-normalised rotation -> scale
    float h;       // trust_factor/2: trust bound in level steps (FP4 grid: trust_factor, in E2M1 value units)
};
QuantConsts make_quant_consts(int bits, int had_block, float trust_factor);

// Rounding grids: the uniform zero-free grid of Eq. 1, or the FP4 (E2M1) grid of Section 4.4.
enum { GRID_UNIFORM = 0, GRID_FP4 = 1 };
// alpha*_FP4: minimiser of the Gaussian quantisation MSE on the E2M1 grid scaled to [-1, 1].
__host__ __device__ inline float alpha_star_fp4() { return 2.9224751f; }

// Operand layout of the int8 tensor-core contraction inside the workspace.
struct Workspace {
    int8_t *a8;        // [M x K] int8 operand values of x
    int8_t *b8;        // [N x K] int8 operand values of w
    int32_t *rs_a;     // [M] row sums of a8 (used only with 8-bit codes)
    int32_t *rs_b;     // [N]
    size_t bytes;
};
Workspace carve_workspace(void *base, int64_t M, int64_t N, int64_t K);

// Programmatic dependent launch.  Every kernel of the library is launched with the
// programmatic-stream-serialization attribute and (1) lets the next kernel in the stream begin
// its launch and set-up early, (2) waits for the previous kernel's grid to complete and flush
// before it touches global memory.  The wait is what keeps stream order; launched without the
// attribute both instructions are no-ops.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              int cluster_x, Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    int n = 0;
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
    if (cluster_x > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = (unsigned)cluster_x;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = n;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
    return e == cudaSuccess ? cudaGetLastError() : e;
}
#endif

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) applies to the current device only.  One static
// instance per kernel (per template instantiation of a launcher) remembers on which devices of this
// process the attribute has been set; setting it twice is harmless, so the race between two host
// threads that both see "not yet" is benign.
struct DynamicSmemOnce {
    bool done[64] = {};
    template <typename Kernel>
    cudaError_t set(Kernel kernel, int bytes) {
        int dev = -1;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64 && done[dev]) return cudaSuccess;
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e == cudaSuccess && dev >= 0 && dev < 64) done[dev] = true;
        return e;
    }
};

// Status / error plumbing.
int cuda_fail(cudaError_t e);             // records the message, returns QUEST_ERR_CUDA
int cuda_fail_msg(const char *msg);
int *device_status_word();                // device address of the timeout word (current device)
int check_device();                       // QUEST_OK iff current device is sm_10x

// Launchers (each returns a quest_status; arguments already validated).
// One tensor of a quantizer launch: rows of `x` -> any of codes / scales / mask / int8 GEMM
// operand / per-row sum of the operand bytes (each nullable).
struct QuantJob {
    const void *x;
    int64_t rows;
    int64_t ld;
    uint8_t *codes;
    float *scales;
    uint8_t *mask;
    int8_t *op8;
    int32_t *rowsum;
    uint16_t *rot = nullptr;   // [rows x cols] bfloat16 of the orthonormal rotation (no quantization needed for it)
    uint16_t *cbf = nullptr;   // [rows x cols] grid values as bfloat16
};
// Up to two tensors with the same row length, dtype and parameters share one launch.
int launch_quantize(const QuantJob *jobs, int njobs, int dtype, int64_t cols, int bits, int had_block,
                    float trust_factor, cudaStream_t st, int grid = GRID_UNIFORM);
int launch_unpack(const uint8_t *codes, int bits, int64_t rows, int64_t K, int8_t *out,
                  int32_t *rowsum, cudaStream_t st, bool e2m1 = false);
// Both operands of one contraction in a single launch (row sums follow where asked for).
int launch_unpack_pair(const uint8_t *xq, int bits_x, int64_t M, int8_t *a8, int32_t *rs_a,
                       const uint8_t *wq, int bits_w, int64_t N, int8_t *b8, int32_t *rs_b, int64_t K, bool e2m1,
                       cudaStream_t st);
int launch_rowsum(const int8_t *a8, int64_t rows, int64_t K, int32_t *rowsum, cudaStream_t st);
int launch_gemm(const int8_t *a8, const int8_t *b8, const int32_t *rs_a, const int32_t *rs_b,
                int bits_x, int bits_w, const float *sx, const float *sw,
                int64_t M, int64_t N, int64_t K, void *y, int y_dtype, int64_t ldy,
                int32_t *acc, cudaStream_t st);

int launch_gemm_swiglu(const int8_t *a8, const int8_t *b8, const int32_t *rs_a, const int32_t *rs_b, int bits,
                       const float *sx, const float *sw_gate, const float *sw_up, int64_t M, int64_t I, int64_t K,
                       void *h, cudaStream_t st);

int launch_bounded_wait_probe(long long limit_cycles, int *report, cudaStream_t st);

// Per-stage event timing (quest_stage_timing): bracket a stage of another translation unit.
void *stage_begin(int id, cudaStream_t st);
void stage_end(void *scope);

// opl: 0 both operands K-major ([rows x Kc]); 1 b MN-major ([Kc x J]); 2 a and b MN-major ([Kc x I], [Kc x J]).
int launch_gemm_bf16_masked(const void *a, const void *b, int64_t I, int64_t J, int64_t Kc,
                            const uint8_t *mask, void *out, int out_dtype, bool fuse_iht128, int opl, cudaStream_t st);

// Contraction of E2M1 nibble operands (tcgen05 kind::mxf4, unit block scales): acc = acc_mul * sum v_x v_w
// (int32, exact), y = sx sw sum v_x v_w.  xq, wq 16-byte aligned, K % 32 == 0.  Serves the FP4 grid
// (acc_mul = 4) and, inside launch_gemm, the one- and two-bit uniform grids (acc_mul = 1).
int launch_gemm_e2m1(const uint8_t *xq, const uint8_t *wq, const float *sx, const float *sw, int64_t M, int64_t N,
                     int64_t K, void *y, int y_dtype, int64_t ldy, int32_t *acc, int acc_mul, cudaStream_t st);
// Orthonormal block Hadamard transform of every row (binary32 or bfloat16 in, binary32 or bfloat16 out).
int launch_hadamard_rows(const void *in, int in_dtype, int64_t ld_in, int64_t rows, int64_t cols, int had_block,
                         void *out, int out_dtype, int64_t ld, cudaStream_t st);
// Weight-only contraction: y[m][n] = sw[n] * sum_k a[m][k] b[n][k], bfloat16 operands (dense, K contiguous),
// binary32 accumulation.
int launch_gemm_bf16_scaled(const void *a, const void *b, const float *sw, int64_t M, int64_t N, int64_t K,
                            void *y, int y_dtype, int64_t ldy, cudaStream_t st);

}  // namespace quest
