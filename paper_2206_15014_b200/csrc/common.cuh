// Shared host-side helpers of the nmsparse library (error bookkeeping, pattern validation).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>
#include "../../include/nmsparse.h"

namespace nm {

// Records the text of a failed CUDA call for nm_last_cuda_error(); returns NM_ERR_CUDA.
int record_cuda_error(cudaError_t e, const char* where);
int record_text_error(const char* text);

#define NM_CUDA_TRY(expr)                                                 \
    do {                                                                  \
        cudaError_t e__ = (expr);                                         \
        if (e__ != cudaSuccess) return nm::record_cuda_error(e__, #expr); \
    } while (0)

// Field width of one metadata entry.
__host__ __device__ inline int meta_field_bits(int m) { return m == 4 ? 2 : 4; }

// NM_OK when (out, in, n, m, bits) is a pattern the library packs.
int check_pattern(int out, int in, int n, int m, int bits);

// Bytes of one row of packed values / u32 words of one row of metadata.
inline size_t values_row_bytes(int in, int n, int m, int bits) { return (size_t)(in / m) * n * bits / 8; }
inline size_t meta_row_words(int in, int n, int m) {
    if (n == m) return 0;
    return ((size_t)(in / m) * n * meta_field_bits(m) + 31) / 32;
}

inline bool aligned(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }

#ifdef __CUDACC__
// Signed integer code of v / s: clamp(rne(fl32(v / s))) to BITS bits, Eq. 5 with offset 0.  The scale is
// shared by many values, so the quotient is formed from the correctly rounded reciprocal r = RN(1 / s)
// with one FMA correction step (q = v * r; q += r * (v - s * q)), which lands within an ulp or two of the
// IEEE quotient.  That can only change the rounded integer when the quotient sits next to a
// half-integer: those cases (and anything non-finite, e.g. a subnormal scale whose reciprocal
// overflows) take the true IEEE division, so the result is the same bit for bit.
// Rounding to the nearest-even integer is done by adding 1.5 * 2^23 (the sum's own rounding does it; the
// quotient is first clamped one code beyond the range so that it stays where that works): ordinary
// adds instead of the quarter-rate float -> int conversions, which otherwise bound the epilogue.
template <int BITS>
__device__ __forceinline__ int quantise_rn(float v, float s, float r) {
    constexpr int hi = (1 << (BITS - 1)) - 1, lo = -(1 << (BITS - 1));
    constexpr float kMagic = 12582912.0f;  // 1.5 * 2^23 = 0x4B400000
    float q = __fmul_rn(v, r);
    q = __fmaf_rn(__fmaf_rn(-s, q, v), r, q);
    float qc = fminf(fmaxf(q, (float)(lo - 1)), (float)(hi + 1));
    float t = __fadd_rn(qc, kMagic);
    const float f = __fsub_rn(qc, __fsub_rn(t, kMagic));     // clamped quotient minus its rounded value, in [-0.5, 0.5]
    if (!(fabsf(f) <= 0.49996948f) || !(fabsf(q) <= 3.0e38f)) {  // within 2^-15 of a tie, or not finite
        q = __fdiv_rn(v, s);
        qc = fminf(fmaxf(q, (float)(lo - 1)), (float)(hi + 1));
        t = __fadd_rn(qc, kMagic);
    }
    const int c = __float_as_int(t) - 0x4B400000;
    return max(lo, min(hi, c));
}

// The same 8-bit code for a NORMAL scale s (>= FLT_MIN, so that r = RN(1 / s) is finite and v * r cannot be
// NaN for finite v), split so that the common case has no branch.  quantise8_fast uses the plain product
// v * r, which is within 2^-23 relative, i.e. 2^-16 absolute for |quotient| <= 129, of the IEEE
// quotient; it sets `near_tie` when the result sits within 2^-15 of a half-integer, where that error
// could change the rounded integer, and the caller then takes quantise8_exact (true IEEE division) for
// those values.  Clamping the quotient to [-128.49, 127.49] before the add of 1.5 * 2^23 (whose own
// rounding rounds to the nearest-even integer) leaves nothing to clamp afterwards: a quotient beyond
// the range, infinite included, rounds to the end code either way.
__device__ __forceinline__ int quantise8_fast(float v, float r, bool& near_tie) {
    constexpr float kMagic = 12582912.0f;  // 1.5 * 2^23 = 0x4B400000
    const float qc = fminf(fmaxf(__fmul_rn(v, r), -128.49f), 127.49f);
    const float t = __fadd_rn(qc, kMagic);
    const float f = __fsub_rn(qc, __fsub_rn(t, kMagic));
    near_tie |= !(fabsf(f) <= 0.49996948f);
    return __float_as_int(t) - 0x4B400000;
}
__device__ __forceinline__ int quantise8_exact(float v, float s) {
    constexpr float kMagic = 12582912.0f;
    const float qc = fminf(fmaxf(__fdiv_rn(v, s), -128.49f), 127.49f);
    return __float_as_int(__fadd_rn(qc, kMagic)) - 0x4B400000;
}
#endif

}  // namespace nm
