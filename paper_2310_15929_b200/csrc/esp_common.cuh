// Shared declarations of the esparse CUDA library (device status word, launch helpers).
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "../../include/esparse.h"

namespace esp {

// Device-side status word: a kernel whose bounded wait gives up stores ESP_ERR_TIMEOUT here and exits.
// (The library is one translation unit, so the definition lives here.)
__device__ int g_device_status = 0;

constexpr int kTileFeat = 128;              // features per packed tile (MMA M)
constexpr int kTileK = 128;                 // permuted channels per packed tile
constexpr int kTileValBytes = kTileFeat * (kTileK / 2) * 2;   // 16384: kept fp16 values
constexpr int kTileMetaBytes = kTileFeat * kTileK / 8;        // 2048: 4 bits per group of 4
constexpr int kTileBytes = kTileValBytes + kTileMetaBytes;    // 18432

inline int ceil_div(long a, long b) { return (int)((a + b - 1) / b); }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct DeviceInfo {
    int device = -1;
    int sm_count = 0;
    int cc_major = 0, cc_minor = 0;
    int max_smem_optin = 0;
};
// Cached properties of the current device (ESP_ERR_CUDA on failure).
esp_status_t device_info(DeviceInfo *out);

#define ESP_CUDA_OK(expr)                                  \
    do {                                                   \
        cudaError_t e_ = (expr);                           \
        if (e_ != cudaSuccess) return ESP_ERR_CUDA;        \
    } while (0)

// ---- pruning launchers (prune_kernels.cu) ----------------------------------------------------------
struct PruneWorkspace {
    // all pointers into the caller's workspace
    double *part_sumsq; float *part_min; float *part_max;   // [splits][C]
    double *lo, *hi, *norm, *entropy, *score, *mean;         // [C]
    unsigned int *counts;                                    // [C][bins]
    unsigned long long *colsum;                              // [C]
    int32_t *theta0;                                         // [C]
    unsigned long long *counters;                            // [8]: 0 near-tie groups, 1 lbs swaps, 2 near-ties of the sort, 3 of the swaps
    double *objective;                                       // [4]: after gns, after lbs, identity order
    double *sorted_mean;                                     // [C] channel means in rank order
    uint16_t *wt;                                            // [C][ldt] |W| bits, channel-major
    double *table;                                           // [nblocks][64][4][256]
    double *base;                                            // [C/4]
    long ldt;
    int splits;
    size_t total_bytes;
};
PruneWorkspace carve_prune_workspace(void *ws, int No, int C, int T, const esp_prune_opts &o);

esp_status_t launch_prune(const __half *W, int No, int C, long ldw, const __half *Xcal, int T, long ldx,
                          const esp_prune_opts &o, __half *vals, uint8_t *meta, int32_t *perm, void *packed,
                          double *chan_norm, double *chan_entropy, double *chan_score,
                          esp_prune_stats *stats, PruneWorkspace &w, cudaStream_t stream);
esp_status_t launch_pack(const __half *vals, const uint8_t *meta, int No, int C, void *packed, cudaStream_t stream);
esp_status_t launch_decompress(const __half *vals, const uint8_t *meta, const int32_t *perm, int No, int C,
                               __half *out, long ldw, cudaStream_t stream);

// ---- streaming calibration (prune_kernels.cu)
struct CalibState {
    double *sumsq, *lo, *hi, *norm;
    unsigned int *counts;
    double *part_sumsq; float *part_min; float *part_max;
    size_t total_bytes;
};
CalibState carve_calib_state(void *state, int C, int bins);
esp_status_t launch_calib_reset(const CalibState &c, int C, int bins, cudaStream_t stream);
esp_status_t launch_calib_range(const CalibState &c, const __half *X, int T, int C, long ldx, cudaStream_t stream);
esp_status_t launch_calib_histogram(const CalibState &c, const __half *X, int T, int C, long ldx, int bins, cudaStream_t stream);
esp_status_t launch_calib_finish(const CalibState &c, int C, int bins, long long T_total, const esp_prune_opts &o, double *chan_norm,
                                 double *chan_entropy, double *chan_score, cudaStream_t stream);

// ---- GEMM launchers (spgemm_kernels.cu) ------------------------------------------------------------
struct GemmPlan {
    int kernel;        // ESP_KERNEL_* (never AUTO)
    int token_tile;    // MMA N
    int split_k;       // cluster size along K
    int stages;
};
esp_status_t plan_gemm(int M, int N, int K, const esp_gemm_opts &o, size_t workspace_bytes, GemmPlan *plan);
size_t gemm_workspace_bytes(int M, int K, const esp_gemm_opts &o);        // everything any plan could use
size_t gemm_workspace_min_bytes(int M, int K, const esp_gemm_opts &o);    // below this only the gather kernel runs
// One streaming-kernel launch for `count` problems; ESP_ERR_UNSUPPORTED if these sizes do not plan onto that kernel.
esp_status_t launch_spgemm_group(int count, const void *const *X, int M, int K, long ldx, const void *const *packed,
                                 const int32_t *const *perm, const int *N, void *const *Y, const long *ldy,
                                 const esp_gemm_opts &o, void *workspace, size_t workspace_bytes, cudaStream_t stream);
esp_status_t launch_wait_timeout_selftest(cudaStream_t stream);
// The optional companion library (ESP_KERNEL_QUAD_MULTICAST): found and loaded?  Its device status word (0 if absent).
bool companion_available();
esp_status_t companion_device_status(int *out);
esp_status_t launch_spgemm(const __half *X, int M, int K, long ldx, const void *packed, const int32_t *perm,
                           int N, void *Y, long ldy, const esp_gemm_opts &o, const GemmPlan &plan,
                           void *workspace, size_t workspace_bytes, cudaStream_t stream);

}  // namespace esp
