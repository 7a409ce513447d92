// int8 tensor-core operand values from packed level indices (device code shared by the quantizer
// and the unpack kernel of the low-bit GEMM).
//
// For b < 8 the operand byte of level k is the top-aligned offset-binary code with half an LSB
// set,  v = ((k << (8-b)) | (1 << (7-b))) ^ 0x80  =  2^(7-b) * c   with c = 2k - (2^b - 1)
// the grid value of Eq. 1: an exact power-of-two multiple of c that fits int8 (|v| <= 127) and
// costs one shift and one three-input logic operation per four elements.  The contraction of two
// such operands is 2^(14-bx-bw) * sum_k cx cw; the GEMM epilogue shifts it back (exact).
// For b = 8 (|c| up to 255) the operand is v = k - 128 = k ^ 0x80 and the epilogue restores the
// grid-value product from per-row sums of v.  (When both operands have at most two bits the operand is
// an E2M1 nibble instead: see e2m1_operands below.)
#pragma once
#include <stdint.h>

namespace quest {

__host__ __device__ inline int operand_shift(int bits) { return bits == 8 ? 0 : 7 - bits; }

__device__ __forceinline__ uint32_t lop3_mask_xor_set(uint32_t x, uint32_t m, uint32_t c) {
    // per bit: m ? x ^ c : c
    return ((x ^ c) & m) | (c & ~m);
}
__device__ __forceinline__ uint32_t byte_perm(uint32_t a, uint32_t b, uint32_t sel) { return __byte_perm(a, b, sel); }

// 4x4 byte transpose: in[j] holds bytes (e_j, e_{4+j}, e_{8+j}, e_{12+j}); out[m] = (e_{4m}, .., e_{4m+3}).
__device__ __forceinline__ void transpose4x4(const uint32_t (&in)[4], uint32_t (&out)[4]) {
    const uint32_t a = byte_perm(in[0], in[1], 0x5140);   // (e0, e1, e4, e5)
    const uint32_t b = byte_perm(in[2], in[3], 0x5140);   // (e2, e3, e6, e7)
    const uint32_t c = byte_perm(in[0], in[1], 0x7362);   // (e8, e9, e12, e13)
    const uint32_t d = byte_perm(in[2], in[3], 0x7362);   // (e10, e11, e14, e15)
    out[0] = byte_perm(a, b, 0x5410);
    out[1] = byte_perm(a, b, 0x7632);
    out[2] = byte_perm(c, d, 0x5410);
    out[3] = byte_perm(c, d, 0x7632);
}

// 32 consecutive codes (CB words of CB-bit containers, element 0 lowest) -> 32 operand bytes in
// element order (8 words).
template <int CB>
__device__ __forceinline__ void operand_from_code_words(const uint32_t (&w)[CB], int bits, uint32_t (&o)[8]) {
    if constexpr (CB == 8) {
        if (bits == 8) {
#pragma unroll
            for (int q = 0; q < 8; ++q) o[q] = w[q] ^ 0x80808080u;
        } else {
            const uint32_t m = (0xFFu << (8 - bits)) & 0xFFu;
            const uint32_t M = m * 0x01010101u, C = (0x80u | (1u << (7 - bits))) * 0x01010101u;
#pragma unroll
            for (int q = 0; q < 8; ++q) o[q] = lop3_mask_xor_set(w[q] << (8 - bits), M, C);
        }
    } else if constexpr (CB == 4) {
        const int up = 4 - bits;                               // 0 at b = 4, 1 at b = 3
        const uint32_t m = (0xFFu << (8 - bits)) & 0xFFu;
        const uint32_t M = m * 0x01010101u, C = (0x80u | (1u << (7 - bits))) * 0x01010101u;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint32_t lo = lop3_mask_xor_set(w[q] << (4 + up), M, C);   // elements 0, 2, 4, 6 of the word
            const uint32_t hi = lop3_mask_xor_set(w[q] << up, M, C);         // elements 1, 3, 5, 7
            o[2 * q] = byte_perm(lo, hi, 0x5140);
            o[2 * q + 1] = byte_perm(lo, hi, 0x7362);
        }
    } else if constexpr (CB == 2) {
        const uint32_t M = 0xC0C0C0C0u, C = 0xA0A0A0A0u;       // b = 2: (k << 6 | 32) ^ 128
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            uint32_t x[4], t[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) x[j] = lop3_mask_xor_set(w[q] << (6 - 2 * j), M, C);
            transpose4x4(x, t);
#pragma unroll
            for (int j = 0; j < 4; ++j) o[4 * q + j] = t[j];
        }
    } else {
        const uint32_t M = 0x80808080u, C = 0xC0C0C0C0u;       // b = 1: (k << 7 | 64) ^ 128
        uint32_t x[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) x[j] = lop3_mask_xor_set(w[0] << (7 - j), M, C);   // bytes (e_j, e_{8+j}, e_{16+j}, e_{24+j})
        // two 4x4 transposes give, for m = 0..3, elements 8m..8m+3 and 8m+4..8m+7
        uint32_t a[4] = {x[0], x[1], x[2], x[3]}, b[4] = {x[4], x[5], x[6], x[7]}, ta[4], tb[4];
        transpose4x4(a, ta);
        transpose4x4(b, tb);
#pragma unroll
        for (int m2 = 0; m2 < 4; ++m2) {
            o[2 * m2] = ta[m2];
            o[2 * m2 + 1] = tb[m2];
        }
    }
}

// FP4 (E2M1) codes: sign << 3 | magnitude index m, values +-{0, .5, 1, 1.5, 2, 3, 4, 6}.
__device__ __forceinline__ float e2m1_value(int code) {
    const int m = code & 7, e = m >> 1;
    const float mag = e ? __uint_as_float(((uint32_t)(126 + e) << 23) | ((uint32_t)(m & 1) << 22)) : 0.5f * (float)m;
    return (code & 8) ? -mag : mag;
}

// The uniform grids of one and two bits are subsets of the E2M1 values (+-1; +-1, +-3), so when both
// operands of a contraction have at most two bits their operand is the E2M1 nibble of the grid value
// (two elements per byte, element 0 in the low nibble) and the contraction runs on the FP4 tensor-core
// path at twice the int8 rate:  b = 1: k = 0, 1 -> 0xA (-1), 0x2 (+1);  b = 2: k = 0..3 -> 0xD (-3),
// 0xA (-1), 0x2 (+1), 0x5 (+3).
__host__ __device__ inline bool e2m1_operands(int bits_x, int bits_w) { return bits_x <= 2 && bits_w <= 2; }

// 32 consecutive codes (CB = 1 or 2 words) -> 32 E2M1 nibbles in element order (4 words).
template <int CB>
__device__ __forceinline__ void e2m1_operand_from_code_words(const uint32_t (&w)[CB], uint32_t (&o)[4]) {
    static_assert(CB == 1 || CB == 2, "only the one- and two-bit grids are E2M1 subsets");
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        if constexpr (CB == 1) {
            const uint32_t b = (w[0] >> (8 * q)) & 0xFFu;          // eight levels, one bit each
            uint32_t t = (b | (b << 12)) & 0x000F000Fu;            // spread: bit j -> bit 0 of nibble j
            t = (t | (t << 6)) & 0x03030303u;
            t = (t | (t << 3)) & 0x11111111u;
            o[q] = 0xAAAAAAAAu ^ (t << 3);                         // k = 1 clears the sign bit
        } else {
            const uint32_t h = (w[q >> 1] >> (16 * (q & 1))) & 0xFFFFu;   // eight levels, two bits each
            uint32_t t = (h | (h << 8)) & 0x00FF00FFu;             // spread: level j -> low bits of nibble j
            t = (t | (t << 4)) & 0x0F0F0F0Fu;
            t = (t | (t << 2)) & 0x33333333u;
            const uint32_t x = (t ^ (t >> 1)) & 0x11111111u;       // k1 ^ k0: set for the inner levels (+-1)
            const uint32_t k1 = (t >> 1) & 0x11111111u;
            // sign = !k1; +-3 = 0b101 (bits 0 and 2) when the level bits agree, +-1 = 0b010 otherwise
            o[q] = ((k1 ^ 0x11111111u) << 3) | ((x ^ 0x11111111u) * 5u) | (x << 1);
        }
    }
}

// Sum of the four signed bytes of a word.
__device__ __forceinline__ int sum_bytes_s8(uint32_t w) { return __dp4a((int)w, 0x01010101, 0); }

}  // namespace quest
