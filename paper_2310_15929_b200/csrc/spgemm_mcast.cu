// Companion library (libesparse_mc.so) of libesparse.so: the four-CTA form of the tiled pair kernel in which one tiled load
// delivers a weight tile to both pairs of the cluster at once (cluster multicast of the tensor memory unit).  It lives in a
// translation unit and a shared object of its own so that the main library contains no multicast load at all; the main
// library looks for this one beside itself and reports ESP_ERR_UNSUPPORTED for ESP_KERNEL_QUAD_MULTICAST when it is absent.
// Only memory of the GPU the kernel runs on is ever loaded this way (the packed weight passed to esp_spgemm).
//
// The kernel itself is spgemm_pair_kernel<2, TN, true, kShareReplicate> of spgemm_pair.cuh; this file supplies its load.
#define g_device_status g_device_status_mc   // this object's own status word (read through esp_mc_device_status)
#include "spgemm_device.cuh"

namespace esp {
namespace {

#include "spgemm_pair.cuh"

// Tiled load of a [rows x 1024-byte] box, written to shared-memory offset `dst` of every CTA in `cta_mask`; the bytes each
// destination received are reported to the barrier at `bar`'s offset in the even-ranked CTA of that destination's pair
// (`bar` itself lies in an even-ranked CTA: .cta_group::2 picks the pair member by that parity).
template <>
struct SharedTileLoad<kShareReplicate> {
    static __device__ __forceinline__ void rows(uint32_t dst, const CUtensorMap *map, int row, uint32_t bar, uint16_t cta_mask) {
        asm volatile(
            "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.multicast::cluster"
            " [%0], [%1, {%2, %3}], [%4], %5;" ::"r"(dst),
            "l"(map), "r"(0), "r"(row), "r"(bar), "h"(cta_mask)
            : "memory");
    }
};

template <int TN>
esp_status_t launch_quad_multicast(const GemmParams &p, bool dependent, cudaStream_t stream) {
    using L = PairCfg<2, TN>;
    auto kern = spgemm_pair_kernel<2, TN, true, kShareReplicate>;
    ESP_CUDA_OK(ensure_dynamic_smem((const void *)kern, L::kTotal));
    const int f_tiles = (p.N + 127) / 128, t_tiles = (p.M + TN - 1) / TN;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(4 * ((f_tiles + 3) / 4), (t_tiles + 1) / 2, 1);
    cfg.blockDim = dim3(kPairThreads);
    cfg.dynamicSmemBytes = L::kTotal;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 4;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 2 : 1;
    CUtensorMap wmap, xmap;
    memset(&wmap, 0, sizeof(wmap));
    memset(&xmap, 0, sizeof(xmap));
    esp_status_t st = make_rows_tensor_map(p.packed, (size_t)f_tiles * p.k_tiles * kTileBytes, kTileBytes / 1024, &wmap);
    if (st == ESP_OK) st = make_rows_tensor_map(p.ximg, xtile_image_bytes<TN>(p.M, p.K), L::kXStage / 1024, &xmap);
    if (st != ESP_OK) return st;
    ESP_CUDA_OK(cudaLaunchKernelEx(&cfg, kern, p, wmap, xmap));
    return ESP_OK;
}

}  // namespace
}  // namespace esp

#define ESP_MC_EXPORT extern "C" __attribute__((visibility("default")))

// The main library's GemmParams (same header, checked by size), the token tile (192, 224 or 240), whether the launch is a
// programmatic dependent of the tiling pass before it, the stream.  Returns an esp_status_t.
ESP_MC_EXPORT int esp_mc_launch_pair(const void *gemm_params, size_t params_size, int token_tile, int dependent, void *stream) {
    if (!gemm_params || params_size != sizeof(esp::GemmParams)) return ESP_ERR_INVALID_ARG;
    const esp::GemmParams &p = *reinterpret_cast<const esp::GemmParams *>(gemm_params);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    switch (token_tile) {
        case 192: return esp::launch_quad_multicast<192>(p, dependent != 0, s);
        case 224: return esp::launch_quad_multicast<224>(p, dependent != 0, s);
        case 240: return esp::launch_quad_multicast<240>(p, dependent != 0, s);
        default: return ESP_ERR_INVALID_ARG;
    }
}

// Reads (and clears, if set) this object's device status word after the caller has synchronised.
ESP_MC_EXPORT int esp_mc_device_status(int *out) {
    int h = 0;
    const int zero = 0;
    if (cudaMemcpyFromSymbol(&h, esp::g_device_status, sizeof(int)) != cudaSuccess) return ESP_ERR_CUDA;
    if (h != 0 && cudaMemcpyToSymbol(esp::g_device_status, &zero, sizeof(int)) != cudaSuccess) return ESP_ERR_CUDA;
    if (out) *out = h;
    return ESP_OK;
}
