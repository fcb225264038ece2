// Host-only entry points of the nmsparse C ABI: sizes, validation, status polling, error text.
#include "common.cuh"
#include <stdio.h>
#include <string.h>

namespace nm {

static thread_local char g_last_error[256] = "";

int record_cuda_error(cudaError_t e, const char* where) {
    snprintf(g_last_error, sizeof(g_last_error), "%s: %s", where, cudaGetErrorString(e));
    (void)cudaGetLastError();  // reset the last-error slot so later calls start clean
    return NM_ERR_CUDA;
}

int record_text_error(const char* text) {
    snprintf(g_last_error, sizeof(g_last_error), "%s", text);
    return NM_ERR_CUDA;
}

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (!cached[dev]) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
        cached[dev] = v;
    }
    return cached[dev];
}

int check_pattern(int out, int in, int n, int m, int bits) {
    if (out < 0 || in < 0 || n < 1 || m < 1 || n > m) return NM_ERR_SHAPE;
    if (bits != 4 && bits != 8) return NM_ERR_UNSUPPORTED;
    if (n != m) {
        if (m != 4 && m != 8) return NM_ERR_UNSUPPORTED;
        if (!((m == 4 && (n == 1 || n == 2)) || (m == 8 && (n == 1 || n == 2 || n == 4))))
            return NM_ERR_UNSUPPORTED;
    }
    if (in % m) return NM_ERR_SHAPE;
    if (((long long)(in / m) * n * bits) % 8) return NM_ERR_SHAPE;
    return NM_OK;
}

}  // namespace nm

extern "C" {

int nm_packed_sizes(int out, int in, int n, int m, int bits, size_t* values_bytes,
                    size_t* meta_bytes) {
    if (!values_bytes || !meta_bytes) return NM_ERR_NULL;
    int rc = nm::check_pattern(out, in, n, m, bits);
    if (rc != NM_OK) return rc;
    *values_bytes = (size_t)out * nm::values_row_bytes(in, n, m, bits);
    *meta_bytes = (size_t)out * nm::meta_row_words(in, n, m) * 4;
    return NM_OK;
}

int nm_poll_status(const uint32_t* status, void* stream) {
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return nm::record_cuda_error(e, "cudaStreamSynchronize");
    if (!status) return NM_OK;
    uint32_t h = 0;
    e = cudaMemcpy(&h, status, sizeof(h), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return nm::record_cuda_error(e, "cudaMemcpy(status)");
    if (h & NM_STATUS_TIMEOUT) return NM_ERR_TIMEOUT;
    if (h & NM_STATUS_NONFINITE) return NM_ERR_NONFINITE;
    return NM_OK;
}

const char* nm_strerror(int code) {
    switch (code) {
        case NM_OK: return "ok";
        case NM_ERR_NULL: return "a required pointer is NULL";
        case NM_ERR_SHAPE: return "invalid shape or N:M pattern";
        case NM_ERR_UNSUPPORTED: return "pattern, bit width or size not supported";
        case NM_ERR_ALIGN: return "pointer or row pitch not aligned as required";
        case NM_ERR_WORKSPACE: return "workspace missing or too small";
        case NM_ERR_CUDA: return "a CUDA call failed (see nm_last_cuda_error)";
        case NM_ERR_NONFINITE: return "NaN or Inf met in W + U";
        case NM_ERR_TIMEOUT: return "a bounded device-side wait expired";
        default: return "unknown nmsparse code";
    }
}

const char* nm_last_cuda_error(void) { return nm::g_last_error; }

double nm_bits_per_param(int n, int m, int bits, int index_bits) {
    if (n < 1 || m < 1 || n > m || bits < 1) return -1.0;
    if (n == m) return (double)bits;  // dense: no index metadata
    const int ib = index_bits < 0 ? nm::meta_field_bits(m) : index_bits;
    return (double)n * (double)(bits + ib) / (double)m;
}

int nm_encoder_cost(const nm_component_cfg_t* cfg, int index_bits, double* compression, double* mac_reduction) {
    if (!cfg) return NM_ERR_NULL;
    // Q, K, V and the attention output are hidden x hidden, the two feed-forward matrices 4 x that
    static const int units[6] = {1, 1, 1, 1, 4, 4};
    double bits = 0.0, saved = 0.0;
    for (int i = 0; i < 6; ++i) {
        const double b = nm_bits_per_param(cfg[i].n, cfg[i].m, cfg[i].bits, index_bits);
        if (b < 0.0) return NM_ERR_SHAPE;
        bits += units[i] * b;
        // a pattern that always fits the 2-of-4 hardware form (at most two kept values in any aligned chunk of
        // four: 1:4, 2:4, 1:8, 2:8) executes half of the dense multiply-accumulates
        const bool sparse_path = cfg[i].n != cfg[i].m && cfg[i].n <= 2 && (cfg[i].m == 4 || cfg[i].m == 8);
        if (sparse_path) saved += 0.5 * units[i];
    }
    if (compression) *compression = 1.0 - bits / (12.0 * 32.0);
    if (mac_reduction) *mac_reduction = saved / 12.0;
    return NM_OK;
}

int nm_version(void) { return 101; }

}  // extern "C"
