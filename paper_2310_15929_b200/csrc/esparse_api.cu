// C ABI of the esparse library: argument validation on the host, then stream-ordered launches.
#include "esp_common.cuh"

#include <mutex>
#include <vector>

namespace esp {

esp_status_t device_info(DeviceInfo *out) {
    static std::mutex mu;
    static DeviceInfo cache[64];
    int dev = -1;
    ESP_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return ESP_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (cache[dev].device != dev) {
        DeviceInfo d;
        d.device = dev;
        ESP_CUDA_OK(cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev));
        ESP_CUDA_OK(cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev));
        ESP_CUDA_OK(cudaDeviceGetAttribute(&d.cc_minor, cudaDevAttrComputeCapabilityMinor, dev));
        ESP_CUDA_OK(cudaDeviceGetAttribute(&d.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
        cache[dev] = d;
    }
    *out = cache[dev];
    return ESP_OK;
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static esp_status_t check_prune_opts(const esp_prune_opts *o) {
    if (!o || o->struct_size != sizeof(esp_prune_opts)) return ESP_ERR_INVALID_ARG;
    const bool is24 = (o->n_keep == 2 && o->m_group == 4), is48 = (o->n_keep == 4 && o->m_group == 8);
    if (!is24 && !is48) return ESP_ERR_UNSUPPORTED;
    if (is48 && o->use_lbs) return ESP_ERR_UNSUPPORTED;      // 4:8: metric, global shuffle, selection, compression only
    if (o->bins < 2 || o->bins > 512) return ESP_ERR_UNSUPPORTED;
    if (o->lbs_block < 4 || o->lbs_block > 256 || o->lbs_block % 4 != 0) return ESP_ERR_INVALID_ARG;
    if (o->lbs_max_swaps < 0) return ESP_ERR_INVALID_ARG;
    if (o->global_bin_range != 0 && o->global_bin_range != 1) return ESP_ERR_INVALID_ARG;
    return ESP_OK;
}

static esp_status_t check_gemm_opts(const esp_gemm_opts *o) {
    if (!o || o->struct_size != sizeof(esp_gemm_opts)) return ESP_ERR_INVALID_ARG;
    if (o->x_layout != ESP_X_TOKEN_MAJOR && o->x_layout != ESP_X_CHANNEL_MAJOR) return ESP_ERR_INVALID_ARG;
    if (o->out_dtype != ESP_OUT_F16 && o->out_dtype != ESP_OUT_F32) return ESP_ERR_INVALID_ARG;
    if (o->split_k < 0 || o->split_k > 8) return ESP_ERR_INVALID_ARG;
    if (o->force_kernel != ESP_KERNEL_AUTO && o->force_kernel != ESP_KERNEL_GATHER && o->force_kernel != ESP_KERNEL_TMA &&
        o->force_kernel != ESP_KERNEL_STREAM && o->force_kernel != ESP_KERNEL_PAIR && o->force_kernel != ESP_KERNEL_PAIR_TILED &&
        o->force_kernel != ESP_KERNEL_QUAD_TILED && o->force_kernel != ESP_KERNEL_PAIR_PERSIST &&
        o->force_kernel != ESP_KERNEL_QUAD_MULTICAST && o->force_kernel != ESP_KERNEL_STREAM_IMAGES)
        return ESP_ERR_INVALID_ARG;
    if (o->static_weights != 0 && o->static_weights != 1) return ESP_ERR_INVALID_ARG;
    if (o->activation != ESP_ACT_NONE && o->activation != ESP_ACT_RELU) return ESP_ERR_INVALID_ARG;
    if (o->pipeline_stages != 0 && (o->pipeline_stages < 2 || o->pipeline_stages > 12)) return ESP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(o->bias) & 1u) != 0) return ESP_ERR_ALIGNMENT;
    if (o->token_tile < 0 || o->token_tile > 256 || o->token_tile % 16 != 0) return ESP_ERR_INVALID_ARG;
    return ESP_OK;
}

}  // namespace esp

using namespace esp;

extern "C" {

const char *esp_status_string(esp_status_t status) {
    switch (status) {
        case ESP_OK: return "ok";
        case ESP_ERR_INVALID_ARG: return "invalid argument";
        case ESP_ERR_SHAPE: return "bad shape or leading dimension";
        case ESP_ERR_ALIGNMENT: return "pointer or leading dimension not 16-byte aligned";
        case ESP_ERR_WORKSPACE: return "workspace missing or too small";
        case ESP_ERR_UNSUPPORTED: return "unsupported configuration or device";
        case ESP_ERR_CUDA: return "CUDA runtime error";
        case ESP_ERR_TIMEOUT: return "a bounded in-kernel wait gave up";
        case ESP_ERR_STATIC_LIMIT: return "sizes exceed the built-in scratch of esp_spgemm_static";
        default: return "unknown status";
    }
}

int esp_version(void) { return 100; }

void esp_prune_opts_default(esp_prune_opts *o) {
    if (!o) return;
    o->struct_size = sizeof(esp_prune_opts);
    o->alpha = 1.0;
    o->bins = 100;
    o->n_keep = 2;
    o->m_group = 4;
    o->lbs_block = 256;
    o->lbs_max_swaps = 0;
    o->use_entropy = 1;
    o->use_norm = 1;
    o->use_gns = 1;
    o->use_lbs = 1;
    o->score_override = nullptr;
    o->global_bin_range = 0;
    o->perm_override = nullptr;
}

void esp_gemm_opts_default(esp_gemm_opts *o) {
    if (!o) return;
    o->struct_size = sizeof(esp_gemm_opts);
    o->x_layout = ESP_X_TOKEN_MAJOR;
    o->out_dtype = ESP_OUT_F16;
    o->split_k = 0;
    o->force_kernel = ESP_KERNEL_AUTO;
    o->token_tile = 0;
    o->static_weights = 0;
    o->pipeline_stages = 0;
    o->activation = ESP_ACT_NONE;
    o->bias = nullptr;
}

size_t esp_metric_prune_workspace_bytes(int No, int C, int T, const esp_prune_opts *opts) {
    if (No <= 0 || C <= 0 || T < 0 || C % 8 != 0 || check_prune_opts(opts) != ESP_OK) return 0;
    return carve_prune_workspace(nullptr, No, C, T, *opts).total_bytes;
}

size_t esp_packed_bytes(int No, int C) {
    if (No <= 0 || C <= 0) return 0;
    return (size_t)ceil_div(No, kTileFeat) * (size_t)ceil_div(C, kTileK) * (size_t)kTileBytes;
}

esp_status_t esp_metric_prune(const void *W, int No, int C, long ldw, const void *Xcal, int T, long ldx,
                              const esp_prune_opts *opts, void *vals, void *meta, int32_t *perm, void *packed,
                              double *chan_norm, double *chan_entropy, double *chan_score, esp_prune_stats *stats,
                              void *workspace, size_t workspace_bytes, void *cuda_stream) {
    esp_status_t st = check_prune_opts(opts);
    if (st != ESP_OK) return st;
    if (!W || !vals || !meta || !perm) return ESP_ERR_INVALID_ARG;
    if (opts->m_group == 8 && packed) return ESP_ERR_UNSUPPORTED;    // no tensor-core form of 4:8: nothing to pack
    if (!Xcal && !opts->score_override) return ESP_ERR_INVALID_ARG;
    if (stats && stats->struct_size != sizeof(esp_prune_stats)) return ESP_ERR_INVALID_ARG;
    if (No <= 0 || C <= 0 || C % 8 != 0 || ldw < C) return ESP_ERR_SHAPE;
    if (Xcal && (T <= 0 || ldx < C)) return ESP_ERR_SHAPE;
    if (ldw % 8 != 0 || (Xcal && ldx % 8 != 0)) return ESP_ERR_ALIGNMENT;
    if (!aligned16(W) || !aligned16(Xcal) || !aligned16(vals) || !aligned16(meta) || !aligned16(perm) ||
        !aligned16(packed) || !aligned16(workspace))
        return ESP_ERR_ALIGNMENT;
    PruneWorkspace w = carve_prune_workspace(workspace, No, C, Xcal ? T : 0, *opts);
    if (!workspace || workspace_bytes < w.total_bytes) return ESP_ERR_WORKSPACE;
    DeviceInfo di;
    st = device_info(&di);
    if (st != ESP_OK) return st;
    if (di.cc_major != 10) return ESP_ERR_UNSUPPORTED;
    return launch_prune((const __half *)W, No, C, ldw, (const __half *)Xcal, Xcal ? T : 0, ldx, *opts, (__half *)vals,
                        (uint8_t *)meta, perm, packed, chan_norm, chan_entropy, chan_score, stats, w,
                        (cudaStream_t)cuda_stream);
}

size_t esp_calib_state_bytes(int C, int bins) {
    if (C <= 0 || C % 8 != 0 || bins < 2 || bins > 512) return 0;
    return carve_calib_state(nullptr, C, bins).total_bytes;
}

static esp_status_t check_calib(const void *state, int C, int bins) {
    if (!state) return ESP_ERR_INVALID_ARG;
    if (C <= 0 || C % 8 != 0) return ESP_ERR_SHAPE;
    if (bins < 2 || bins > 512) return ESP_ERR_UNSUPPORTED;
    if (!aligned16(state)) return ESP_ERR_ALIGNMENT;
    return ESP_OK;
}

esp_status_t esp_calib_reset(void *state, int C, int bins, void *cuda_stream) {
    esp_status_t st = check_calib(state, C, bins);
    if (st != ESP_OK) return st;
    return launch_calib_reset(carve_calib_state(state, C, bins), C, bins, (cudaStream_t)cuda_stream);
}

static esp_status_t check_chunk(const void *X, int T, int C, long ldx) {
    if (!X) return ESP_ERR_INVALID_ARG;
    if (T <= 0 || ldx < C) return ESP_ERR_SHAPE;
    if (ldx % 8 != 0 || !aligned16(X)) return ESP_ERR_ALIGNMENT;
    return ESP_OK;
}

esp_status_t esp_calib_range(void *state, const void *X, int T, int C, long ldx, int bins, void *cuda_stream) {
    esp_status_t st = check_calib(state, C, bins);
    if (st == ESP_OK) st = check_chunk(X, T, C, ldx);
    if (st != ESP_OK) return st;
    return launch_calib_range(carve_calib_state(state, C, bins), (const __half *)X, T, C, ldx, (cudaStream_t)cuda_stream);
}

esp_status_t esp_calib_histogram(void *state, const void *X, int T, int C, long ldx, int bins, void *cuda_stream) {
    esp_status_t st = check_calib(state, C, bins);
    if (st == ESP_OK) st = check_chunk(X, T, C, ldx);
    if (st != ESP_OK) return st;
    return launch_calib_histogram(carve_calib_state(state, C, bins), (const __half *)X, T, C, ldx, bins, (cudaStream_t)cuda_stream);
}

esp_status_t esp_calib_finish(void *state, int C, long long T_total, const esp_prune_opts *opts, double *chan_norm,
                              double *chan_entropy, double *chan_score, void *cuda_stream) {
    if (!opts || opts->struct_size != sizeof(esp_prune_opts) || !chan_score) return ESP_ERR_INVALID_ARG;
    esp_status_t st = check_calib(state, C, opts->bins);
    if (st != ESP_OK) return st;
    if (T_total <= 0 || T_total > 0x7FFFFFFFLL) return ESP_ERR_SHAPE;
    return launch_calib_finish(carve_calib_state(state, C, opts->bins), C, opts->bins, T_total, *opts, chan_norm, chan_entropy,
                               chan_score, (cudaStream_t)cuda_stream);
}

esp_status_t esp_pack(const void *vals, const void *meta, int No, int C, void *packed, void *cuda_stream) {
    if (!vals || !meta || !packed) return ESP_ERR_INVALID_ARG;
    if (No <= 0 || C <= 0 || C % 8 != 0) return ESP_ERR_SHAPE;
    if (!aligned16(vals) || !aligned16(meta) || !aligned16(packed)) return ESP_ERR_ALIGNMENT;
    return launch_pack((const __half *)vals, (const uint8_t *)meta, No, C, packed, (cudaStream_t)cuda_stream);
}

esp_status_t esp_decompress(const void *vals, const void *meta, const int32_t *perm, int No, int C, void *W_out,
                            long ldw, void *cuda_stream) {
    if (!vals || !meta || !W_out) return ESP_ERR_INVALID_ARG;
    if (No <= 0 || C <= 0 || C % 8 != 0 || ldw < C) return ESP_ERR_SHAPE;
    return launch_decompress((const __half *)vals, (const uint8_t *)meta, perm, No, C, (__half *)W_out, ldw,
                             (cudaStream_t)cuda_stream);
}

size_t esp_spgemm_workspace_bytes(int M, int N, int K, const esp_gemm_opts *opts) {
    (void)N;
    if (M <= 0 || K <= 0 || check_gemm_opts(opts) != ESP_OK) return 0;
    // K-slices are reduced through distributed shared memory inside a cluster: no global scratch for that.
    // Token-major X is first transposed (not permuted) into the workspace so channels become rows.
    return gemm_workspace_bytes(M, K, *opts);
}

esp_status_t esp_spgemm_plan(int M, int N, int K, const esp_gemm_opts *opts, int have_workspace, int *kernel,
                             int *token_tile, int *split_k, int *stages) {
    esp_status_t st = check_gemm_opts(opts);
    if (st != ESP_OK) return st;
    if (M <= 0 || N <= 0 || K <= 0 || K % 8 != 0) return ESP_ERR_SHAPE;
    DeviceInfo di;
    st = device_info(&di);
    if (st != ESP_OK) return st;
    if (di.cc_major != 10) return ESP_ERR_UNSUPPORTED;
    GemmPlan plan;
    st = plan_gemm(M, N, K, *opts, have_workspace != 0 ? gemm_workspace_bytes(M, K, *opts) : 0, &plan);
    if (st != ESP_OK) return st;
    if (kernel) *kernel = plan.kernel;
    if (token_tile) *token_tile = plan.token_tile;
    if (split_k) *split_k = plan.split_k;
    if (stages) *stages = plan.stages;
    return ESP_OK;
}

esp_status_t esp_spgemm(const void *X, int M, int K, long ldx, const void *packed, const int32_t *perm, int N,
                        void *Y, long ldy, const esp_gemm_opts *opts, void *workspace, size_t workspace_bytes,
                        void *cuda_stream) {
    esp_status_t st = check_gemm_opts(opts);
    if (st != ESP_OK) return st;
    if (!X || !packed || !Y) return ESP_ERR_INVALID_ARG;
    if (M <= 0 || N <= 0 || K <= 0 || K % 8 != 0 || ldy < N) return ESP_ERR_SHAPE;
    if (opts->x_layout == ESP_X_TOKEN_MAJOR ? (ldx < K) : (ldx < M)) return ESP_ERR_SHAPE;
    if (ldx % 8 != 0) return ESP_ERR_ALIGNMENT;
    if (!aligned16(X) || !aligned16(packed) || !aligned16(Y) || !aligned16(perm)) return ESP_ERR_ALIGNMENT;
    DeviceInfo di;
    st = device_info(&di);
    if (st != ESP_OK) return st;
    if (di.cc_major != 10) return ESP_ERR_UNSUPPORTED;
    GemmPlan plan;
    const bool have_ws = workspace && aligned16(workspace);
    st = plan_gemm(M, N, K, *opts, have_ws ? workspace_bytes : 0, &plan);
    if (st != ESP_OK) return st;
    return launch_spgemm((const __half *)X, M, K, ldx, packed, perm, N, Y, ldy, *opts, plan, workspace,
                         workspace_bytes, (cudaStream_t)cuda_stream);
}

esp_status_t esp_spgemm_grouped(int count, const void *const *X, int M, int K, long ldx, const void *const *packed,
                                const int32_t *const *perm, const int *N, void *const *Y, const long *ldy,
                                const esp_gemm_opts *opts, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    esp_status_t st = check_gemm_opts(opts);
    if (st != ESP_OK) return st;
    if (count < 1 || count > ESP_MAX_GROUP || !X || !packed || !N || !Y || !ldy || opts->bias) return ESP_ERR_INVALID_ARG;
    if (M <= 0 || K <= 0 || K % 8 != 0) return ESP_ERR_SHAPE;
    if (opts->x_layout == ESP_X_TOKEN_MAJOR ? (ldx < K) : (ldx < M)) return ESP_ERR_SHAPE;
    if (ldx % 8 != 0) return ESP_ERR_ALIGNMENT;
    for (int i = 0; i < count; ++i) {
        if (!X[i] || !packed[i] || !Y[i]) return ESP_ERR_INVALID_ARG;
        if (N[i] <= 0 || ldy[i] < N[i]) return ESP_ERR_SHAPE;
        if (!aligned16(X[i]) || !aligned16(packed[i]) || !aligned16(Y[i]) || (perm && !aligned16(perm[i]))) return ESP_ERR_ALIGNMENT;
    }
    DeviceInfo di;
    st = device_info(&di);
    if (st != ESP_OK) return st;
    if (di.cc_major != 10) return ESP_ERR_UNSUPPORTED;
    const bool have_ws = workspace && aligned16(workspace);
    st = launch_spgemm_group(count, X, M, K, ldx, packed, perm, N, Y, ldy, *opts, have_ws ? workspace : nullptr,
                             have_ws ? workspace_bytes : 0, (cudaStream_t)cuda_stream);
    if (st != ESP_ERR_UNSUPPORTED) return st;
    // sizes that do not plan onto one streaming launch: the problems one after the other, each with its share of the workspace
    const size_t share = have_ws ? (workspace_bytes / (size_t)count) & ~(size_t)255 : 0;
    for (int i = 0; i < count; ++i) {
        st = esp_spgemm(X[i], M, K, ldx, packed[i], perm ? perm[i] : nullptr, N[i], Y[i], ldy[i], opts,
                        share ? (uint8_t *)workspace + (size_t)i * share : nullptr, share, cuda_stream);
        if (st != ESP_OK) return st;
    }
    return ESP_OK;
}

esp_status_t esp_spgemm_tune(const void *X, int M, int K, long ldx, const void *packed, const int32_t *perm, int N,
                             void *Y, long ldy, esp_gemm_opts *opts, void *workspace, size_t workspace_bytes, int reps,
                             float *best_us, float *planned_us, void *cuda_stream) {
    esp_status_t st = check_gemm_opts(opts);
    if (st != ESP_OK) return st;
    if (reps < 1 || reps > 1000) return ESP_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) {
        if (e0) cudaEventDestroy(e0);
        return ESP_ERR_CUDA;
    }
    // candidates: the planner's own choice first, then every (kernel, token tile, K-slices) the sizes admit
    struct Cand { int kernel, tile, split, stages; };
    std::vector<Cand> cands;
    cands.push_back({opts->force_kernel, opts->token_tile, opts->split_k, opts->pipeline_stages});
    if (M > 64) {
        for (int tile : {240, 224, 192, 128}) {
            if (tile > 128 && M <= 128) continue;
            for (int split = 1; split <= (tile == 128 ? 4 : 1); ++split) {      // K-slices: 128-token tiles only
                cands.push_back({ESP_KERNEL_PAIR_TILED, tile, split, 0});
                cands.push_back({ESP_KERNEL_PAIR, tile, split, 0});
            }
        }
        cands.push_back({ESP_KERNEL_PAIR, 256, 1, 0});
        if (M > 256)
            for (int tile : {240, 224, 192}) cands.push_back({ESP_KERNEL_PAIR_PERSIST, tile, 1, 0});      // never planned, sometimes ahead
    }
    if (M <= 1024) {
        for (int tile : {64, 128})
            for (int split = 1; split <= 8; ++split) {
                if (tile >= 2 * M && tile > 64) continue;
                cands.push_back({ESP_KERNEL_STREAM_IMAGES, tile, split, 0});
            }
        for (int tile : {16, 32, 64, 128, 256}) {
            if (tile < M && tile < 256 && (M + tile - 1) / tile > 8) continue;      // many narrow token tiles: never the best
            if (tile >= 2 * M && tile > 16) continue;
            for (int split = 1; split <= 8; ++split)
                for (int stages : {0, 2, 3, 4, 6, 8}) cands.push_back({ESP_KERNEL_STREAM, tile, split, stages});
        }
    }
    esp_gemm_opts best = *opts;
    float best_t = -1.f, first_t = -1.f;
    esp_status_t result = ESP_OK;
    for (size_t i = 0; i < cands.size(); ++i) {
        esp_gemm_opts o = *opts;
        o.force_kernel = cands[i].kernel;
        o.token_tile = cands[i].tile;
        o.split_k = cands[i].split;
        o.pipeline_stages = cands[i].stages;
        GemmPlan plan;
        const bool have_ws = workspace && aligned16(workspace);
        if (check_gemm_opts(&o) != ESP_OK || plan_gemm(M, N, K, o, have_ws ? workspace_bytes : 0, &plan) != ESP_OK) continue;
        if (i > 0 && cands[i].kernel == ESP_KERNEL_STREAM &&
            (plan.split_k != cands[i].split || (cands[i].stages != 0 && plan.stages != cands[i].stages)))
            continue;                                                          // stepped down or clamped: a duplicate
        if (i > 0 && cands[i].kernel != ESP_KERNEL_STREAM && plan.split_k != cands[i].split) continue;
        // one untimed call (first-use set-up, caches), then `reps` timed ones
        st = esp_spgemm(X, M, K, ldx, packed, perm, N, Y, ldy, &o, workspace, workspace_bytes, cuda_stream);
        if (st != ESP_OK) {
            if (i == 0) { result = st; break; }        // the caller's own configuration must work
            continue;
        }
        cudaEventRecord(e0, stream);
        for (int r = 0; r < reps && st == ESP_OK; ++r)
            st = esp_spgemm(X, M, K, ldx, packed, perm, N, Y, ldy, &o, workspace, workspace_bytes, cuda_stream);
        cudaEventRecord(e1, stream);
        if (cudaEventSynchronize(e1) != cudaSuccess) { result = ESP_ERR_CUDA; break; }
        if (st != ESP_OK) continue;
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        const float us = ms * 1000.f / (float)reps;
        if (i == 0) first_t = us;
        if (best_t < 0.f || us < best_t) { best_t = us; best = o; }
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (result != ESP_OK) return result;
    if (best_t < 0.f) return ESP_ERR_UNSUPPORTED;
    if (esp_last_device_status() != ESP_OK) return ESP_ERR_TIMEOUT;
    *opts = best;
    if (best_us) *best_us = best_t;
    if (planned_us) *planned_us = first_t;
    return ESP_OK;
}

esp_status_t esp_selftest_wait_timeout(void *cuda_stream) {
    DeviceInfo di;
    esp_status_t st = device_info(&di);
    if (st != ESP_OK) return st;
    return launch_wait_timeout_selftest((cudaStream_t)cuda_stream);
}

esp_status_t esp_last_device_status(void) {
    int h = 0, zero = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return ESP_ERR_CUDA;
    if (cudaMemcpyFromSymbol(&h, g_device_status, sizeof(int)) != cudaSuccess) return ESP_ERR_CUDA;
    if (h != 0 && cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int)) != cudaSuccess) return ESP_ERR_CUDA;
    int hc = 0;                               // the companion library's kernels have a status word of their own
    if (companion_device_status(&hc) != ESP_OK) return ESP_ERR_CUDA;
    return (esp_status_t)(h != 0 ? h : hc);
}

int esp_multicast_available(void) { return companion_available() ? 1 : 0; }

}  // extern "C"
