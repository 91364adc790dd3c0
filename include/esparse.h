/*
 * esparse.h -- C ABI of the E-Sparse hot path for NVIDIA B200 (sm_100a).
 *
 * Two operations, as the paper states the problem:
 *
 *   esp_metric_prune   calibration activations + a layer's weight  ->  channel permutation,
 *                      2:4-pruned weight in compressed form (kept values + 2-bit positions).
 *                      Sections "Information Richness - Entropy" (Eq. 1-3), "Information Reorder -
 *                      Channel Shuffle" (Eq. 5, Algorithm 1) and step (1) of "Efficient Sparse-GEMM
 *                      Implementation".
 *   esp_spgemm         the pruned layer's forward product  Y = X . P . W_s^T  on the sparse tensor
 *                      cores ("Efficient Sparse-GEMM Implementation", Table 5).
 *
 * Conventions
 *   - All tensor pointers are DEVICE pointers unless the comment says "host".  The caller owns every
 *     buffer, including workspaces; the library allocates no device memory and keeps no state besides a
 *     per-process cache of device properties.
 *   - Everything is stream-ordered on `cuda_stream` (a cudaStream_t passed as void*; NULL = default
 *     stream).  Nothing synchronises unless stated.
 *   - Inputs are never written.  Errors are return codes; argument errors are detected on the host
 *     before anything is launched.  No call traps, aborts or throws.
 *   - Notation: W is [No, C] row-major fp16 (No output features, C input channels); Xcal is [T, C]
 *     fp16 calibration activations; perm[p] = original channel placed at permuted position p.
 */
#ifndef ESPARSE_H_
#define ESPARSE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ESP_OK = 0,
    ESP_ERR_INVALID_ARG = 1,   /* NULL where a pointer is required, bad enum, bad struct_size        */
    ESP_ERR_SHAPE = 2,         /* non-positive sizes, C % 8 != 0, leading dimension too small         */
    ESP_ERR_ALIGNMENT = 3,     /* a base pointer or leading dimension is not 16-byte aligned          */
    ESP_ERR_WORKSPACE = 4,     /* workspace NULL or smaller than the *_workspace_bytes() answer       */
    ESP_ERR_UNSUPPORTED = 5,   /* pattern other than 2:4 / 4:8, bins > 512, device is not sm_100      */
    ESP_ERR_CUDA = 6,          /* a CUDA runtime call or a launch failed                              */
    ESP_ERR_TIMEOUT = 7,       /* a bounded in-kernel wait gave up (reported by esp_last_device_status) */
    ESP_ERR_STATIC_LIMIT = 8   /* esp_spgemm_static: the sizes need more than ESP_STATIC_SCRATCH_BYTES   */
} esp_status_t;

/* Static string for a status code (never NULL). */
const char *esp_status_string(esp_status_t status);

/* Library version: major * 10000 + minor * 100 + patch. */
int esp_version(void);

/* ------------------------------------------------------------------------------------------------
 * Pruning: metric, shuffle, 2:4 selection, compression.
 * ---------------------------------------------------------------------------------------------- */

typedef struct {
    size_t struct_size;          /* = sizeof(esp_prune_opts)                                         */
    double alpha;                /* weight of the norm in Eq. 3; the paper gives no value             */
    int bins;                    /* K of Eq. 1 (paper: 100); 2..512                                   */
    int n_keep, m_group;         /* N:M pattern: 2:4, or 4:8 (Table 1's second pattern: metric, global shuffle,
                                    selection and compression only -- use_lbs must be 0 and packed NULL,
                                    no tensor-core form exists; meta then holds one byte per group of 8,
                                    bit p = position p kept, vals the 4 kept weights in position order)   */
    int lbs_block;               /* m of the local block shuffle (paper: 256); multiple of 4, <= 256  */
    int lbs_max_swaps;           /* cap on swaps per block; 0 = until no swap improves (Algorithm 1)  */
    int use_entropy;             /* 0 drops IR_c from the score (norm-only baseline of Table 4)       */
    int use_norm;                /* 0 drops alpha * AM_c                                              */
    int use_gns;                 /* 0 skips the global naive shuffle (identity start order)           */
    int use_lbs;                 /* 0 skips the local block shuffle                                   */
    const double *score_override;/* optional device f64[C]: use these s_c instead of computing them   */
    int global_bin_range;        /* Eq. 1 does not say what is divided into K bins.  0 (default): each channel's
                                    own [min, max]; 1: the layer's [min, max] over all channels, so that a
                                    narrow channel falls into few bins and gets a low entropy             */
    const int32_t *perm_override;/* optional device i32[C]: start from this channel order instead of the
                                    global shuffle's (a stored permutation, e.g. to re-compress updated
                                    weights); the block shuffle still runs on it if use_lbs is set.
                                    Must be a permutation of 0..C-1 (not checked).                     */
} esp_prune_opts;

typedef struct {
    size_t struct_size;          /* = sizeof(esp_prune_stats)                                         */
    long long near_tie_groups;   /* groups whose 2nd and 3rd metric differ by < 1e-6 relative         */
    long long near_tie_sort;     /* global shuffle: neighbours in rank whose mean metrics differ by < 1e-6
                                    relative (0 when the shuffle is off or the order is given)        */
    long long near_tie_swaps;    /* block shuffle: applied swaps whose gain beats the runner-up's by < 1e-6
                                    relative                                                           */
    long long lbs_swaps_total;   /* swaps applied by the local block shuffle                          */
    double obj_identity;         /* Eq. 5 objective (2 of every 4 kept) under the original channel order */
    double obj_after_gns;        /* Eq. 5 objective under the order after the global shuffle          */
    double obj_after_lbs;        /* Eq. 5 objective under the final order                             */
} esp_prune_stats;

/* Fills *opts with the paper's settings (bins 100, 2:4, block 256, everything on, alpha = 1). */
void esp_prune_opts_default(esp_prune_opts *opts);

/* Bytes of device workspace esp_metric_prune needs for these sizes (0 on bad arguments). */
size_t esp_metric_prune_workspace_bytes(int No, int C, int T, const esp_prune_opts *opts);

/*
 * Bytes of the tensor-core-ready copy of a compressed [No, C] weight.  Layout (opaque to callers):
 * tiles of 128 features x 128 permuted channels, each 18432 bytes = 16384 bytes of kept fp16 values in
 * the 128-byte-swizzled shared-memory image the MMA reads + 2048 bytes of position metadata in the
 * order the tensor-memory copy expects.  No and C are padded up to multiples of 128 with zeros.
 */
size_t esp_packed_bytes(int No, int C);

/*
 * The whole producer (Eq. 1-3, global + local shuffle, 2-of-4 selection, compression).
 *
 *   W      [No, C] fp16, leading dimension ldw (elements, >= C, multiple of 8)
 *   Xcal   [T, C]  fp16, leading dimension ldx (elements, >= C, multiple of 8); may be NULL when
 *          opts->score_override is given
 *   vals   out, fp16 [No, C/2]: kept weights, bit copies of W, two per group in position order
 *   meta   out, u8 [No, C/8]: per group a nibble idx0 | idx1 << 2 (idx0 < idx1 = kept positions 0..3);
 *          byte g/2 holds group g in its low (g even) or high (g odd) nibble
 *   perm   out, int32 [C]
 *   packed out, optional (NULL to skip): esp_packed_bytes(No, C) bytes, what esp_spgemm consumes
 *   chan_norm / chan_entropy / chan_score  out, optional device f64[C]: AM_c, IR_c, s_c
 *   stats  out, optional HOST struct; when non-NULL the call synchronises the stream once
 *
 * C must be a multiple of 8.  Returns ESP_OK or an error code; on error nothing was launched unless
 * the code is ESP_ERR_CUDA.
 */
esp_status_t esp_metric_prune(const void *W, int No, int C, long ldw,
                              const void *Xcal, int T, long ldx,
                              const esp_prune_opts *opts,
                              void *vals, void *meta, int32_t *perm, void *packed,
                              double *chan_norm, double *chan_entropy, double *chan_score,
                              esp_prune_stats *stats,
                              void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Streaming calibration: the channel statistics of Eq. 1-3 accumulated over many chunks of activations (the paper
 * calibrates on 128 sequences) without holding them all at once.  Per-channel bins need the channel's range first,
 * so the chunks are passed twice:
 *
 *   esp_calib_reset(state)                          once
 *   esp_calib_range(state, chunk)                   every chunk: sum of squares, minimum, maximum
 *   esp_calib_histogram(state, chunk)               every chunk again: bin counts on the final [min, max]
 *   esp_calib_finish(state, T_total, opts, ...)     AM_c, IR_c, s_c  ->  pass s_c as opts->score_override to
 *                                                   esp_metric_prune (Xcal = NULL)
 *
 * The result equals esp_metric_prune's on the concatenated chunks: counts and ranges exactly, the norm up to the order
 * of its fp64 additions.  `state` is esp_calib_state_bytes(C, bins) bytes of caller-owned device memory; chunks are
 * [T, C] fp16 with leading dimension ldx; bins is opts->bins (100 in the paper) in every call.
 */
size_t esp_calib_state_bytes(int C, int bins);
esp_status_t esp_calib_reset(void *state, int C, int bins, void *cuda_stream);
esp_status_t esp_calib_range(void *state, const void *X, int T, int C, long ldx, int bins, void *cuda_stream);
esp_status_t esp_calib_histogram(void *state, const void *X, int T, int C, long ldx, int bins, void *cuda_stream);
esp_status_t esp_calib_finish(void *state, int C, long long T_total, const esp_prune_opts *opts, double *chan_norm,
                              double *chan_entropy, double *chan_score, void *cuda_stream);

/*
 * Re-tiles (vals, meta) as written by esp_metric_prune into the packed form (step (1) of "Efficient
 * Sparse-GEMM Implementation": the compressed format the GEMM reads).  Same shapes as above.
 */
esp_status_t esp_pack(const void *vals, const void *meta, int No, int C, void *packed, void *cuda_stream);

/*
 * Inverse of the compression, for checking: dense fp16 [No, C] (leading dimension ldw) in ORIGINAL
 * channel order with zeros where pruned.  perm NULL = identity.
 */
esp_status_t esp_decompress(const void *vals, const void *meta, const int32_t *perm, int No, int C,
                            void *W_out, long ldw, void *cuda_stream);

/* ------------------------------------------------------------------------------------------------
 * Sparse GEMM.
 * ---------------------------------------------------------------------------------------------- */

enum { ESP_X_TOKEN_MAJOR = 0,    /* X[t, c] at X + t * ldx + c  (tokens are rows)                      */
       ESP_X_CHANNEL_MAJOR = 1 };/* X[t, c] at X + c * ldx + t  (channels are rows: the activation
                                    handed over transposed)                                           */
enum { ESP_OUT_F16 = 0, ESP_OUT_F32 = 1 };
enum { ESP_ACT_NONE = 0, ESP_ACT_RELU = 1 };
enum { ESP_KERNEL_AUTO = 0,
       ESP_KERNEL_GATHER = 1,    /* element gather of X, any layout, no workspace (slow for large M)    */
       ESP_KERNEL_TMA = 2,       /* channel-major X rows fetched four at a time by the tensor memory
                                    unit's row gather (correct, but that unit retires such gathers too
                                    slowly to feed the MMA; kept for comparison)                        */
       ESP_KERNEL_STREAM = 4,    /* channel-major X rows streamed by asynchronous 16-byte copies, weight
                                    tiles by bulk copies; every token count (default up to 256 tokens,
                                    except where the pair kernel below is faster)                       */
       ESP_KERNEL_PAIR = 5,      /* large M: two SMs share one 512-feature x token_tile MMA tile
                                    (token_tile 240 by default; 128, 192, 224 or 256 on request); X rows
                                    are gathered through the permutation by 16-byte copies              */
       ESP_KERNEL_PAIR_TILED = 6,/* the same tile, fed by bulk copies: a pass over X first writes the
                                    permuted, swizzled operand images into the workspace (default for
                                    more than 256 tokens when the workspace has room; token_tile 128..240) */
       ESP_KERNEL_QUAD_TILED = 7,/* ESP_KERNEL_PAIR_TILED with two such tiles (same features, neighbouring
                                    token tiles) per cluster of four SMs: every weight tile is fetched once per
                                    cluster and handed to the other pair through distributed shared memory
                                    (token_tile 192, 224 or 240; slower than ESP_KERNEL_PAIR_TILED on every
                                    shape measured: kept for comparison)                                */
       ESP_KERNEL_PAIR_PERSIST = 8,/* ESP_KERNEL_PAIR_TILED as a persistent kernel: one CTA pair per two SMs walks
                                    the tiles, the operand ring never drains between tiles and the epilogue (warps of
                                    its own, accumulators straight from registers to Y) runs under the next tile's
                                    first steps (token_tile 192, 224 or 240; same results bit for bit; within a few
                                    per cent of ESP_KERNEL_PAIR_TILED either way, so only esp_spgemm_tune picks it) */
       ESP_KERNEL_STREAM_IMAGES = 10,/* ESP_KERNEL_STREAM for token_tile 32, 64, 128 or 256, fed like
                                    ESP_KERNEL_PAIR_TILED: a pass over X writes the permuted, swizzled operand images of every
                                    (token block, channel step) into the workspace and a stage's X is one bulk copy per
                                    block instead of 16-byte row copies; same results bit for bit; needs the workspace
                                    (default for 17..256 tokens on large weights)                        */
       ESP_KERNEL_QUAD_MULTICAST = 9 };/* the cluster of ESP_KERNEL_QUAD_TILED with every weight tile delivered to
                                    both pairs by ONE tiled load (cluster multicast of the tensor memory unit) instead
                                    of a hand-over: token_tile 192, 224 or 240, same results bit for bit.  Its kernel
                                    is in the optional companion library libesparse_mc.so, looked for beside this
                                    library; without it the call returns ESP_ERR_UNSUPPORTED
                                    (esp_multicast_available() tells).  Single-GPU use only: the packed weight must
                                    lie in the memory of the GPU the call runs on.                      */

typedef struct {
    size_t struct_size;          /* = sizeof(esp_gemm_opts)                                           */
    int x_layout;                /* ESP_X_*                                                           */
    int out_dtype;               /* ESP_OUT_*: type of Y                                              */
    int split_k;                 /* K-slices reduced inside a thread-block cluster; 0 = choose, 1..8  */
    int force_kernel;            /* ESP_KERNEL_*                                                      */
    int token_tile;              /* tokens per tile (16, 32, 64, 128 or 256; pair kernel: see above);
                                    0 = choose                                                        */
    int static_weights;          /* 1 = `packed` and `perm` are not written by work still pending on the
                                    stream (the usual case at inference).  The kernel is then launched as
                                    a programmatic dependent of the preceding kernel: its weight prefetch
                                    overlaps that kernel's tail, and only the reads of X and the writes
                                    of Y wait for it.  0 (default) = plain stream order.                 */
    int pipeline_stages;         /* depth of the streaming kernel's shared-memory ring (2..12 tiles in flight
                                    per CTA; clamped to what shared memory holds and to the channel steps of
                                    a K-slice); 0 = choose.  Ignored by the other kernels.              */
    int activation;              /* ESP_ACT_*: applied to the fp32 sum (+ bias) before it is rounded to
                                    the output type.  The paper times the bare product (Table 5); OPT's
                                    linears carry a bias and fc1 a ReLU, which this folds into the same
                                    launch                                                               */
    const void *bias;            /* device fp16 [N], added to every token row; NULL = none            */
} esp_gemm_opts;

void esp_gemm_opts_default(esp_gemm_opts *opts);

/*
 * Bytes of device workspace esp_spgemm can use: for token-major X a transposed (channels-as-rows, not
 * permuted) copy of X, which lets the fast kernels run, and for more than 256 tokens the permuted X operand
 * images of ESP_KERNEL_PAIR_TILED (about 2.2 * M * K bytes).  With a smaller workspace the call still works:
 * without room for the images through ESP_KERNEL_PAIR, without room for the transposed copy (or with
 * NULL) through the element-gather kernel.  The workspace is scratch: nothing in it outlives the call's work
 * on the stream, and calls on different streams need different workspaces.
 */
size_t esp_spgemm_workspace_bytes(int M, int N, int K, const esp_gemm_opts *opts);

/*
 * The search of step (2) of "Efficient Sparse-GEMM Implementation" (the paper tries the library's algorithms per weight
 * shape and keeps the fastest): times esp_spgemm on the caller's buffers for every (kernel, token tile, K-slices) the
 * sizes admit (and every ring depth of the streaming kernel), `reps` calls each after one untimed call, the configuration
 * in *opts first, and writes the fastest into opts->force_kernel / token_tile / split_k / pipeline_stages (the other
 * fields are kept).  best_us / planned_us (optional, host) receive the time per call of the winner and of the
 * configuration *opts came in with.  The calls repeat on the same buffers, so small weights are timed from L2.  Y and the
 * workspace are written; the stream is synchronised.  Persisting the four integers per (M, N, K, layout) is the
 * caller's: binding.py has save_plan_table / load_plan_table.
 */
esp_status_t esp_spgemm_tune(const void *X, int M, int K, long ldx, const void *packed, const int32_t *perm, int N,
                             void *Y, long ldy, esp_gemm_opts *opts, void *workspace, size_t workspace_bytes, int reps,
                             float *best_us, float *planned_us, void *cuda_stream);

/*
 * Reports the launch configuration esp_spgemm would use for these sizes on the current device (the
 * counterpart of step (2) of "Efficient Sparse-GEMM Implementation", where the paper searches the library's
 * algorithms per weight shape): kernel (ESP_KERNEL_*), tokens per CTA tile, K-slices per cluster, pipeline
 * stages.  have_workspace says whether a workspace of esp_spgemm_workspace_bytes() will be passed.
 * Output pointers may be NULL.  Launches nothing.
 */
esp_status_t esp_spgemm_plan(int M, int N, int K, const esp_gemm_opts *opts, int have_workspace,
                             int *kernel, int *token_tile, int *split_k, int *stages);

/*
 * Y[t, j] = sum over kept weights of row j:  w * X[t, perm[position of w]]   (fp32 accumulation)
 *
 *   X       fp16, M tokens x K channels in the layout opts->x_layout names, leading dimension ldx
 *           (elements; multiple of 8)
 *   packed  esp_packed_bytes(N, K) bytes from esp_metric_prune / esp_pack
 *   perm    int32 [K] or NULL for the identity; applied while the X tile is loaded (up to 256 tokens, or without
 *           a workspace) or by the pass that writes the X operand images into the workspace (more tokens)
 *   opts    layout, output type, optional bias and activation: Y = act(product + bias), bias and activation applied
 *           to the finished fp32 sum
 *   Y       out, [M, N] row-major (Y[t, j] at Y + t * ldy + j), fp16 or fp32 per opts->out_dtype
 *
 * The result does not depend on scheduling: K-slices are summed in slice order.
 */
esp_status_t esp_spgemm(const void *X, int M, int K, long ldx,
                        const void *packed, const int32_t *perm, int N,
                        void *Y, long ldy, const esp_gemm_opts *opts,
                        void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Several independent products in one launch: Y[i] = X[i] . P[i] . W_s[i]^T for i < count <= ESP_MAX_GROUP, each with its
 * own weight, permutation, input and output.  (The paper times a layer's Q/K/V as one GEMM, Table 5; this keeps the three
 * weights, and their three channel permutations, separate.)  M, K, ldx and the options are common, N[i] and ldy[i] are
 * per problem; X, packed, perm, N, Y, ldy are HOST arrays of `count` entries (perm[i] may be NULL; opts->bias is not
 * supported here and must be NULL).  Up to 256 tokens the problems share one launch of the streaming kernel -- what a
 * short launch loses to start-up and drain is paid once; for more tokens the call is the same as `count` calls of
 * esp_spgemm.  workspace: count * esp_spgemm_workspace_bytes(M, max N, K, opts) bytes.
 */
#define ESP_MAX_GROUP 4
esp_status_t esp_spgemm_grouped(int count, const void *const *X, int M, int K, long ldx, const void *const *packed,
                                const int32_t *const *perm, const int *N, void *const *Y, const long *ldy,
                                const esp_gemm_opts *opts, void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * The product for hosts that cannot allocate device memory.  (The paper has no counterpart: this is a
 * deployment convenience of this library, not a step of the method.)
 *
 * Same result as esp_spgemm with token-major X (X[t, c] at X + t * ldx + c), default options and a
 * workspace -- but the transposed copy of X that the fast kernels read goes into a fixed array of
 * ESP_STATIC_SCRATCH_BYTES inside the library's device image, so the caller passes only inputs and outputs
 * and the call performs no cudaMalloc, cudaFree or other allocation.  It is meant for callers that run
 * layers from a hook which carries no workspace pointer while all device memory belongs to their host
 * engine's pool, and for threads that must not call cudaMalloc because it can synchronise the device.
 *
 *   - Limit: K * round_up(M, 16) * 2 bytes must not exceed ESP_STATIC_SCRATCH_BYTES (8 MiB: M <= 1024 at
 *     K = 4096, M <= 112 at K = 36864); larger sizes return ESP_ERR_STATIC_LIMIT and launch nothing.
 *     Every GPU on which the library is loaded holds the array until the process exits.
 *   - The first call on each device looks up the array's device address (with that device current).
 *     Make that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps the previous call's contents.  Nothing in it
 *     has to start at zero (the region a call reads is rewritten in full first), but two calls whose
 *     kernels overlap on the GPU -- different streams, or the same call from two threads -- race on it:
 *     keep calls to this entry point stream-ordered with respect to each other.
 *   - out_dtype is ESP_OUT_F16 or ESP_OUT_F32; perm NULL = identity; other arguments as in esp_spgemm.
 */
#define ESP_STATIC_SCRATCH_BYTES (8u << 20)
esp_status_t esp_spgemm_static(const void *X, int M, int K, long ldx,
                               const void *packed, const int32_t *perm, int N,
                               void *Y, long ldy, int out_dtype, void *cuda_stream);

/*
 * Exercises the failure path of the kernels' bounded waits without faulting anything (no counterpart in the paper;
 * every barrier wait of the GEMM kernels is bounded so that a lost signal ends in a status code, not a hang): launches one
 * tiny kernel whose wait can never be satisfied; after about a millisecond it gives up, records ESP_ERR_TIMEOUT in the
 * device status word and returns normally.  The next esp_last_device_status() returns ESP_ERR_TIMEOUT, and the
 * context stays usable.
 */
esp_status_t esp_selftest_wait_timeout(void *cuda_stream);

/*
 * Reads and clears the device-side status word of the current device (synchronises the device).
 * Kernels bound every wait on a barrier; a wait that gives up records ESP_ERR_TIMEOUT here and the
 * kernel exits cleanly.  Returns ESP_OK if no kernel reported anything.
 */
esp_status_t esp_last_device_status(void);

/*
 * 1 if the companion library with ESP_KERNEL_QUAD_MULTICAST was found beside this one and loaded, else 0 (no counterpart
 * in the paper).  Host-only; the first call does the look-up.
 */
int esp_multicast_available(void);

#ifdef __cplusplus
}
#endif
#endif /* ESPARSE_H_ */
