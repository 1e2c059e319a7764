// Host-side helpers of the C ABI: status word, kept-length / FLOPs arithmetic,
// workspace sizes.
#include <math.h>

#include "common.cuh"

namespace dash {

__device__ int g_status_word = 0;

int* status_word_ptr() {
    // one address per device; looked up on first use with that device current
    static std::atomic<int*> ptrs[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    int* p = ptrs[dev].load(std::memory_order_acquire);
    if (!p) {
        if (cudaGetSymbolAddress((void**)&p, g_status_word) != cudaSuccess) return nullptr;
        ptrs[dev].store(p, std::memory_order_release);      // two threads that race here store the same address
    }
    return p;
}

size_t compact_ws_bytes_pub(int64_t n);
size_t attention_ws_bytes(int64_t n, int S, int Hq, int Hkv, int D, dash_dtype dt);
size_t decode_ws_bytes(int64_t n, int S, int Hq, int Hkv, int D);

}  // namespace dash

extern "C" const char* dash_status_string(int status) {
    switch (status) {
        case DASH_OK: return "ok";
        case DASH_ERR_INVALID_ARG: return "invalid argument";
        case DASH_ERR_UNSUPPORTED: return "unsupported configuration";
        case DASH_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case DASH_ERR_CUDA: return "CUDA runtime error";
        case DASH_ERR_TIMEOUT: return "a device-side wait gave up";
        case DASH_ERR_TOO_LARGE: return "input exceeds the fixed scratch of this entry point (use the variant that takes a workspace)";
        default: return "unknown status";
    }
}

extern "C" int dash_check_status(void* stream) {
    int* p = dash::status_word_ptr();
    if (!p) return DASH_ERR_CUDA;
    int h = 0;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemcpyAsync(&h, p, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return DASH_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return DASH_ERR_CUDA;
    if (h != 0) {
        if (cudaMemsetAsync(p, 0, sizeof(int), st) != cudaSuccess) return DASH_ERR_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return DASH_ERR_CUDA;
    }
    return h;
}

extern "C" int64_t dash_keep_count(int64_t n, double rho, int keep_first, int keep_last, int mode) {
    if (n < 0 || !(rho >= 0.0) || !(rho < 1.0) || keep_first < 0 || keep_last < 0) return -1;
    if (mode == 0) return (int64_t)floor((1.0 - rho) * (double)n);
    if (mode == 1) {
        int64_t n_fix = (int64_t)keep_first + keep_last;
        if (n_fix > n) n_fix = n;
        int64_t drop = (int64_t)floor(nearbyint(rho * (double)(n - n_fix)));   // ties to even
        return n - drop;
    }
    return -1;
}

extern "C" double dash_flops_per_layer(double n, double d, double m) {
    return 4.0 * n * d * d + 2.0 * n * n * d + 2.0 * n * d * m;
}

extern "C" double dash_flops_speedup(double n, double n_hat, int L, int l_s, double d, double m) {
    double c_full = L * dash_flops_per_layer(n, d, m);
    double c_ours = l_s * dash_flops_per_layer(n, d, m) + (L - l_s) * dash_flops_per_layer(n_hat, d, m);
    return c_full / c_ours;
}

extern "C" size_t dash_workspace_bytes(dash_ws_op op, int64_t n, int S, int Hq, int Hkv, int D, dash_dtype dt) {
    if (n < 0) return 0;
    switch (op) {
        case DASH_WS_COMPACT: return dash::compact_ws_bytes_pub(n);
        case DASH_WS_ATTENTION: return dash::attention_ws_bytes(n, S, Hq, Hkv, D, dt);
        case DASH_WS_DECODE: return dash::decode_ws_bytes(n, S, Hq, Hkv, D);
        default: return 0;
    }
}
