// Version, status strings, argument validation and the host-only bit allocation.
#include "slim_common.cuh"

#include <algorithm>
#include <atomic>
#include <vector>

namespace slim {

static std::atomic<int> g_last_cuda_error{0};

void set_cuda_error(cudaError_t e) {
    g_last_cuda_error.store(static_cast<int>(e));
    (void)cudaGetLastError();  // clear the sticky-free error state of the runtime
}

int make_group_table(int N, int K, int g, const uint8_t* bits_host, GroupTable* out) {
    if (bits_host == nullptr || N < 0 || K < 0) return SLIM_ERR_INVALID_ARG;
    if (g != 128 && g != 256 && g != 512) return SLIM_ERR_UNSUPPORTED;
    if (K % g != 0 || N % 16 != 0) return SLIM_ERR_UNSUPPORTED;
    const int G = K / SLIM_GROUP;                      // K-tiles
    if (G > SLIM_MAX_GROUPS) return SLIM_ERR_UNSUPPORTED;
    out->G = G;
    out->gshift = g == 128 ? 0 : (g == 256 ? 1 : 2);
    int acc = 0;
    for (int j = 0; j < G; ++j) {
        const int b = bits_host[j >> out->gshift];
        if (b < 1 || b > 4) return SLIM_ERR_INVALID_ARG;
        out->bits[j] = static_cast<uint8_t>(b);
        out->prefix[j] = static_cast<uint16_t>(acc);
        acc += b;
    }
    out->prefix[G] = static_cast<uint16_t>(acc);
    for (int j = G; j < SLIM_MAX_GROUPS; ++j) { out->bits[j] = 0; out->prefix[j + 1] = static_cast<uint16_t>(acc); }
    return SLIM_OK;
}

}  // namespace slim

extern "C" {

int slim_version(void) { return (SLIM_FORMAT_VERSION << 16) | 1; }

const char* slim_status_string(int status) {
    switch (status) {
        case SLIM_OK: return "ok";
        case SLIM_ERR_INVALID_ARG: return "invalid argument";
        case SLIM_ERR_UNSUPPORTED: return "unsupported shape or group size";
        case SLIM_ERR_ALIGNMENT: return "device pointer not 16-byte aligned";
        case SLIM_ERR_WORKSPACE: return "workspace missing or too small";
        case SLIM_ERR_CUDA: return "CUDA runtime error";
        case SLIM_ERR_TIMEOUT: return "device-side wait timed out";
        case SLIM_ERR_STATIC_SCRATCH: return "shape needs more scratch than the library's built-in array holds";
        default: return "unknown status";
    }
}

int slim_last_cuda_error(void) { return slim::g_last_cuda_error.load(); }

int slim_packed_bytes(int N, int K, int g, const uint8_t* bits_host, size_t* out_bytes) {
    if (out_bytes == nullptr) return SLIM_ERR_INVALID_ARG;
    if (slim::is_small_group(g)) return slim::small_packed_bytes(N, K, g, bits_host, out_bytes);
    slim::GroupTable gt;
    const int st = slim::make_group_table(N, K, g, bits_host, &gt);
    if (st != SLIM_OK) return st;
    *out_bytes = static_cast<size_t>(16) * static_cast<size_t>(N) * gt.prefix[gt.G];
    return SLIM_OK;
}

int slim_allocate_bits(const double* salience_host, int G, int avg_bits, int p, uint8_t* bits_host_out) {
    if (salience_host == nullptr || bits_host_out == nullptr || G < 0) return SLIM_ERR_INVALID_ARG;
    if (avg_bits < 2 || avg_bits > 3) return SLIM_ERR_INVALID_ARG;
    if (p < 0) p = G / 4;
    if (2 * p > G) return SLIM_ERR_INVALID_ARG;
    std::vector<int> order(G);
    for (int j = 0; j < G; ++j) order[j] = j;
    std::stable_sort(order.begin(), order.end(),
                     [&](int a, int b) { return salience_host[a] > salience_host[b]; });
    for (int j = 0; j < G; ++j) bits_host_out[j] = static_cast<uint8_t>(avg_bits);
    for (int i = 0; i < p; ++i) {
        bits_host_out[order[i]] = static_cast<uint8_t>(avg_bits + 1);
        bits_host_out[order[G - 1 - i]] = static_cast<uint8_t>(avg_bits - 1);
    }
    return SLIM_OK;
}

}  // extern "C"
