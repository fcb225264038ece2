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

}  // namespace nm
