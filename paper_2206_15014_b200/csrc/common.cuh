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

// Form of the projection kernel forced by nm_debug_set_option("pack_form") (0 = automatic).
extern int g_pack_form;

#ifdef NM_TEST_HOOKS
// Timeout test only: the unit (per block) whose copies warp 0 of block 0 of the staged projection kernel leaves unissued.
int pack_set_skip_unit(int unit);
#endif

// Multiprocessors of the current device (cached per device; 148 when the query fails).
int sm_count();

inline bool aligned(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }

#ifdef __CUDACC__
// Signed integer code of v / s: clamp(rne(fl32(v / s))) to BITS bits, Eq. 5 with offset 0, for a scale that
// many values share: the quotient comes from the correctly rounded reciprocal r = RN(1 / s).  `fast_ok` (once
// per scale) says that s lies in [2^-126, 2^125], where r = RN(1 / s) is a normal number: then the plain product v * r is
// within |q| * 1.5 * 2^-23 <= 2^-15.4 of the IEEE quotient over the clamped range, so it rounds to the same
// integer unless it sits within 2^-15 of a half-integer; those values (6 in 100000), NaNs and scales outside
// the range take the true division.  Clamping the quotient to [lo - 0.49, hi + 0.49] before the add of
// 1.5 * 2^23 leaves nothing to clamp afterwards (a quotient beyond the range rounds to the end code either way).
// The add's own rounding rounds to the nearest-even integer: ordinary adds instead of quarter-rate float -> int
// conversions.
template <int BITS>
__device__ __forceinline__ int quantise_shared_scale(float v, float s, float r, bool fast_ok) {
    constexpr float kLo = -(float)(1 << (BITS - 1)) - 0.49f, kHi = (float)((1 << (BITS - 1)) - 1) + 0.49f;
    constexpr float kMagic = 12582912.0f;  // 1.5 * 2^23 = 0x4B400000
    float qc = fminf(fmaxf(__fmul_rn(v, r), kLo), kHi);
    float t = __fadd_rn(qc, kMagic);
    const float f = __fsub_rn(qc, __fsub_rn(t, kMagic));
    if (!(fabsf(f) <= 0.49996948f) || !fast_ok) {
        qc = fminf(fmaxf(__fdiv_rn(v, s), kLo), kHi);
        t = __fadd_rn(qc, kMagic);
    }
    return __float_as_int(t) - 0x4B400000;
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
