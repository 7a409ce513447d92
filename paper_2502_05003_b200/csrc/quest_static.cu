// quest_lowbit_gemm_static: the low-bit GEMM for callers that cannot provide scratch memory.
//
// quest_lowbit_gemm needs a workspace for the int8 operands the tensor cores read, and the
// caller has to allocate it.  Some callers cannot: a plug-in that is handed input and output
// pointers by a host application and has no allocator of its own; a serving process that
// reserved all of device memory for its own pools at start-up, so that a later cudaMalloc fails;
// a latency-critical loop that must not take the device-wide synchronisation cudaMalloc and
// cudaFree imply.  For them the scratch lives in this file, in a fixed array that is part of the
// library image: every GPU that loads the library holds QUEST_STATIC_SCRATCH_BYTES of it until
// the process exits, whether or not this entry point is ever called.
//
// The array's name is only meaningful to device code.  On the host it names a stand-in object,
// not device memory, so the address the kernels receive is looked up once per device with
// cudaGetSymbolAddress while that device is current.
#include "quest_internal.cuh"

namespace quest {
namespace {

static __device__ __align__(256) unsigned char g_static_scratch[QUEST_STATIC_SCRATCH_BYTES];

// Device address of the array on the current device (nullptr and a recorded CUDA error on failure).
void *static_scratch_address() {
    static void *cached[64] = {nullptr};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) {
        cuda_fail(e);
        return nullptr;
    }
    if (dev < 0 || dev >= 64) {
        cuda_fail_msg("device ordinal out of range for the static scratch table");
        return nullptr;
    }
    if (!cached[dev]) {
        void *ptr = nullptr;
        e = cudaGetSymbolAddress((void **)&ptr, g_static_scratch);
        if (e != cudaSuccess) {
            cuda_fail(e);
            return nullptr;
        }
        cached[dev] = ptr;
    }
    return cached[dev];
}

}  // namespace
}  // namespace quest

using namespace quest;

extern "C" int quest_lowbit_gemm_static(const uint8_t *xq, const float *sx, int bits_x,
                                        const uint8_t *wq, const float *sw, int bits_w,
                                        int64_t M, int64_t N, int64_t K,
                                        void *y, int y_dtype, int64_t ldy_elems, int32_t *acc,
                                        void *stream) {
    // Size first: quest_workspace_bytes is 0 for shapes and bit-widths the GEMM does not accept.
    if (bits_x < 1 || bits_x > 8 || bits_w < 1 || bits_w > 8) return QUEST_ERR_BITS;
    const size_t need = quest_workspace_bytes(M, N, K, bits_x, bits_w);
    if (need == 0) {
        const int64_t worst = K * (((int64_t)1 << bits_x) - 1) * (((int64_t)1 << bits_w) - 1);
        return (K >= 32 && K % 32 == 0 && K <= 65504 && worst >= ((int64_t)1 << 31))
                   ? QUEST_ERR_OVERFLOW : QUEST_ERR_SHAPE;
    }
    if (need > (size_t)QUEST_STATIC_SCRATCH_BYTES) return QUEST_ERR_STATIC_LIMIT;
    if (M == 0 || N == 0) return QUEST_OK;
    int s = check_device();
    if (s) return s;
    void *scratch = static_scratch_address();
    if (!scratch) return QUEST_ERR_CUDA;
    // Same validation, unpack launches and tensor-core kernel as the workspace variant; every
    // byte of the scratch that the kernels read is written by this call first.
    return quest_lowbit_gemm(xq, sx, bits_x, wq, sw, bits_w, M, N, K, y, y_dtype, ldy_elems, acc,
                             scratch, (size_t)QUEST_STATIC_SCRATCH_BYTES, stream);
}
