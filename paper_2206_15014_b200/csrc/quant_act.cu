// Dynamic per-tensor symmetric 8-bit activation quantiser: |max| reduction and the quantise pass.
#include "common.cuh"
#include <cuda_runtime.h>

namespace nm {

// Non-negative floats order like their bit patterns, so an unsigned atomicMax folds the maximum.
__global__ void __launch_bounds__(256) absmax_kernel(const float* __restrict__ Y, size_t count,
                                                     float* __restrict__ absmax) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // a dependent kernel may begin its set-up early
    const size_t n4 = count >> 2;
    const float4* Y4 = reinterpret_cast<const float4*>(Y);
    float a = 0.0f;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        float4 v = __ldcs(Y4 + i);
        a = fmaxf(a, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
    }
    if (blockIdx.x == 0 && threadIdx.x < (count & 3)) a = fmaxf(a, fabsf(Y[(n4 << 2) + threadIdx.x]));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
    __shared__ float red[8];
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = a;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < 8; ++i) a = fmaxf(a, red[i]);
        atomicMax(reinterpret_cast<unsigned*>(absmax), __float_as_uint(a));
    }
}

__device__ __forceinline__ int quantise8(float y, float s) {
    int q = __float2int_rn(__fdiv_rn(y, s));  // IEEE division, round half to even
    return max(-128, min(127, q));
}

__device__ __forceinline__ unsigned pack4(float4 v, float s) {
    return (unsigned)(quantise8(v.x, s) & 0xff) | ((unsigned)(quantise8(v.y, s) & 0xff) << 8) |
           ((unsigned)(quantise8(v.z, s) & 0xff) << 16) | ((unsigned)(quantise8(v.w, s) & 0xff) << 24);
}

// Each thread turns 16 floats into one 16-byte store.
__global__ void __launch_bounds__(256) quantize_act_kernel(const float* __restrict__ Y, size_t count,
                                                           const float* __restrict__ absmax,
                                                           int8_t* __restrict__ Xq,
                                                           float* __restrict__ sx_out) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // a dependent kernel may begin its set-up early
    const float a = *absmax;
    const float s = (a == 0.0f) ? 1.0f : __fdiv_rn(a, 127.0f);
    if (sx_out && blockIdx.x == 0 && threadIdx.x == 0) *sx_out = s;
    const size_t n16 = count >> 4;
    const float4* Y4 = reinterpret_cast<const float4*>(Y);
    uint4* X16 = reinterpret_cast<uint4*>(Xq);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (size_t)gridDim.x * blockDim.x) {
        float4 v0 = __ldcs(Y4 + 4 * i), v1 = __ldcs(Y4 + 4 * i + 1), v2 = __ldcs(Y4 + 4 * i + 2),
               v3 = __ldcs(Y4 + 4 * i + 3);
        X16[i] = make_uint4(pack4(v0, s), pack4(v1, s), pack4(v2, s), pack4(v3, s));
    }
    if (blockIdx.x == 0 && threadIdx.x < (count & 15)) {
        size_t i = (n16 << 4) + threadIdx.x;
        Xq[i] = (int8_t)quantise8(Y[i], s);
    }
}

static int grid_for(size_t units) {
    size_t blocks = (units + 255) / 256;
    size_t cap = (size_t)sm_count() * 8;
    return (int)(blocks < 1 ? 1 : (blocks > cap ? cap : blocks));
}

}  // namespace nm

extern "C" {

int nm_absmax(const float* Y, size_t count, float* absmax, void* stream) {
    if (!absmax || (!Y && count)) return NM_ERR_NULL;
    if (count == 0) return NM_OK;
    if (!nm::aligned(Y, 16) || !nm::aligned(absmax, 4)) return NM_ERR_ALIGN;
    nm::absmax_kernel<<<nm::grid_for(count >> 2), 256, 0, (cudaStream_t)stream>>>(Y, count, absmax);
    NM_CUDA_TRY(cudaGetLastError());
    return NM_OK;
}

int nm_quantize_act(const float* Y, size_t count, const float* absmax, int8_t* Xq, float* sx_out,
                    void* stream) {
    if (!absmax || ((!Y || !Xq) && count)) return NM_ERR_NULL;
    if (count && (!nm::aligned(Y, 16) || !nm::aligned(Xq, 16))) return NM_ERR_ALIGN;
    if (sx_out == absmax) return NM_ERR_SHAPE;  // one thread writes the scale while the others still read the maximum
    nm::quantize_act_kernel<<<nm::grid_for(count >> 4), 256, 0, (cudaStream_t)stream>>>(Y, count, absmax, Xq, sx_out);
    NM_CUDA_TRY(cudaGetLastError());
    return NM_OK;
}

}  // extern "C"
