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
// supported (cols, had_block, bits, dtype).  Correctness reference for the specialised kernels.
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

}  // namespace

int launch_quantize(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                    int bits, int had_block, float trust_factor,
                    uint8_t *codes, float *scales, uint8_t *mask, int8_t *op8, cudaStream_t st) {
    if (rows == 0) return QUEST_OK;
    const QuantConsts qc = make_quant_consts(bits, had_block, trust_factor);
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
