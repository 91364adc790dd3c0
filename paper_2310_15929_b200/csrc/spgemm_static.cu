// esp_spgemm_static: esp_spgemm for token-major X without any caller-supplied or allocated scratch.
//
// Some hosts of this library cannot allocate device memory at the point where they run a layer: an
// inference engine that has handed all of HBM to its own pool and calls operators through a hook that
// carries only input and output pointers, or a latency-critical serving thread for which cudaMalloc is
// off limits because it may synchronise the whole device.  For them the transposed copy of X that the fast
// kernels read lives in a fixed array inside the library's device image instead of a workspace.
#include "esp_common.cuh"

#include <mutex>

namespace esp {
namespace {

// The scratch itself.  Every GPU that loads the library holds these bytes until the process exits.
// In host code this name is only a handle for the runtime, not a device address: the address kernels may
// use is obtained with cudaGetSymbolAddress (below), once per device.
static __device__ __align__(256) unsigned char g_static_scratch[ESP_STATIC_SCRATCH_BYTES];

std::mutex g_static_mu;
void *g_static_addr[64] = {};

// Device address of g_static_scratch on the current device (looked up on the first call per device).
esp_status_t static_scratch_address(void **out) {
    int dev = -1;
    ESP_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return ESP_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return ESP_ERR_CUDA;
        g_static_addr[dev] = p;
    }
    *out = g_static_addr[dev];
    return ESP_OK;
}

}  // namespace
}  // namespace esp

extern "C" esp_status_t esp_spgemm_static(const void *X, int M, int K, long ldx, const void *packed,
                                          const int32_t *perm, int N, void *Y, long ldy, int out_dtype,
                                          void *cuda_stream) {
    using namespace esp;
    if (!X || !packed || !Y) return ESP_ERR_INVALID_ARG;
    if (out_dtype != ESP_OUT_F16 && out_dtype != ESP_OUT_F32) return ESP_ERR_INVALID_ARG;
    if (M <= 0 || N <= 0 || K <= 0 || K % 8 != 0 || ldy < N || ldx < K) return ESP_ERR_SHAPE;
    if (ldx % 8 != 0) return ESP_ERR_ALIGNMENT;
    auto misaligned = [](const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
    if (misaligned(X) || misaligned(packed) || misaligned(Y) || misaligned(perm)) return ESP_ERR_ALIGNMENT;
    esp_gemm_opts o;
    esp_gemm_opts_default(&o);
    o.x_layout = ESP_X_TOKEN_MAJOR;
    o.out_dtype = out_dtype;
    const size_t need = gemm_workspace_min_bytes(M, K, o);   // the transposed copy; X images only if they fit too
    if (need > (size_t)ESP_STATIC_SCRATCH_BYTES) return ESP_ERR_STATIC_LIMIT;
    DeviceInfo di;
    esp_status_t st = device_info(&di);
    if (st != ESP_OK) return st;
    if (di.cc_major != 10) return ESP_ERR_UNSUPPORTED;
    void *scratch = nullptr;
    st = static_scratch_address(&scratch);
    if (st != ESP_OK) return st;
    GemmPlan plan;
    st = plan_gemm(M, N, K, o, (size_t)ESP_STATIC_SCRATCH_BYTES, &plan);
    if (st != ESP_OK) return st;
    // The transposing pre-pass writes every element of the K x ceil16(M) region the GEMM reads (zeros in the
    // padding columns), and the tiling pass every byte of the images, so nothing has to be cleared although the
    // array keeps the previous call's contents.
    return launch_spgemm((const __half *)X, M, K, ldx, packed, perm, N, Y, ldy, o, plan, scratch,
                         (size_t)ESP_STATIC_SCRATCH_BYTES, (cudaStream_t)cuda_stream);
}
