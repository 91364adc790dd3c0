// Pair kernel: large token counts (prefill), channel-major X.  Included by spgemm_kernels.cu inside
// namespace esp { namespace { ... } } after the helpers it uses.
//
// At the sparse tensor-core rate a CTA consumes a 128-channel step of a 128-feature x 256-token tile in 512
// clocks; filling shared memory for it (18 KB of weights + 64 KB of gathered X rows) would need 164 B/clk
// per SM, several times what an SM can pull in.  So the tile is made as large as tensor memory allows and is
// shared by two SMs:
//
//   * a cluster of two CTAs issues one MMA of 256 features x TN tokens (tcgen05.mma.sp.cta_group::2): each CTA
//     supplies its own 128 feature rows of the compressed weight and HALF of the tokens of the X tile;
//   * each CTA carries NA = 2 such accumulators (2 x TN fp32 columns of tensor memory + metadata columns use
//     all 512), so the pair covers 512 features x TN tokens and an X row is gathered once for 512 features.
//
// With TN = 240 a 128-channel step moves 36 KB of weight tiles (bulk asynchronous copies) and 30 KB of X rows
// (16-byte asynchronous copies) per CTA for 960 clocks of MMA: 70 B/clk per SM instead of 164.
//
// Two measured properties of the SM's copy paths shape the producers (B200, data resident in L2):
//   * bulk copies issued by ONE thread complete one after the other, about 0.45 us each whatever their size
//     (18 KB copies: 41 GB/s per SM from one thread, 81 from two, 134 from four), so the weight tiles of a
//     stage are issued by different lanes;
//   * 16-byte asynchronous row copies deliver about 25 GB/s per SM from 128 threads, 44 from 256 and 60 from
//     512, independent of how many stages are in flight, so sixteen warps gather X.
//
// grid (2 x feature-pair tiles, token tiles, K-slices), cluster (2, 1, K-slices), block 576 (one K-slice unless the planner
// splits a 128-token grid that is far below one wave; the four-CTA form at the end of this comment uses cluster (4,1,1)).
// In both CTAs of a pair:
//   warp 0             idle
//   warp 1             tensor-memory allocation; lane 0 of the leader CTA (rank 0): tcgen05.cp + MMAs for the pair;
//                      lane 0 of rank 1: forwards "my stage is full" to the leader's barrier
//   warps 2..17        X row producers (lane 0 of six of them also issues the weight-tile copies), then epilogue
//                      (four warps per quarter of the accumulator lanes)
// A stage's `empty` barrier and the final `accum` barrier are signalled in both CTAs at once by
// tcgen05.commit with a CTA mask.  No load uses cluster multicast.
//
// TILED = true is the same kernel fed differently: a pass over X (xtile_kernel) applies the permutation and writes,
// for every (token tile, CTA rank, 128-channel step), the exact shared-memory image of the X operand (kXStage bytes,
// swizzled) into the caller's workspace.  A stage is then three bulk copies (two weight tiles, one X image), each from
// lane 0 of a warp of its own; the sixteen warps no longer gather, they only run the epilogue.  The 16-byte gather
// path delivers 32 B/clk per SM, bulk copies about 70: the price is one more pass over X.  That pass and the GEMM run
// concurrently: the GEMM is launched as the pass's programmatic dependent and takes each image when its flag is up.
//
// K-slices (128-token tiles): the pairs of one cluster take consecutive ranges of channel steps; after a cluster barrier
// every CTA pushes its fp32 partial rows to the CTA of the same pair rank in the owning slice (16-byte asynchronous remote
// stores), which adds the slices in slice order.
//
// SHARE != 0 (tiled form only) puts two pairs on the same 512 features and neighbouring token tiles into one cluster of
// four, so that a weight tile leaves L2 once per two token tiles.  kShareHandOver: each CTA fetches one of its two weight
// tiles and hands a copy to the other pair through distributed shared memory.  kShareReplicate: each CTA fetches one weight
// tile with a load that the memory system delivers to both pairs (that load is supplied by another translation unit, see
// SharedTileLoad below).  Both are bit-identical to the plain form and both are slower on every shape measured: the
// hand-over chain does not fit a three-slot ring, a cluster of four leaves 16 of 148 SMs idle (33 clusters fit), and in
// either form every SM still takes in the same 68 KB per step -- what limits the kernel is that intake, not the bytes
// leaving L2.  Kept for comparison, never planned.

__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// arrives on the barrier at this shared-memory offset in every CTA of the mask once the MMAs issued so far are done
__device__ __forceinline__ void tc_commit_pair(uint32_t bar, uint16_t cta_mask) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
                 "h"(cta_mask)
                 : "memory");
}
__device__ __forceinline__ void tc_copy_128x128b_pair(uint32_t taddr, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::2.128x128b [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void tc_mma_sparse_f16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t e_tmem,
                                                       uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.sp.cta_group::2.kind::f16 [%0], %1, %2, [%3], %4, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(e_tmem), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Waits of the two single-thread roles (forwarder, MMA issuer), each alone in its warp: poll without sleeping first --
// a sleeping poll adds its sleep to every hand-over of the ring -- then fall back to the bounded, abort-aware wait.
__device__ __forceinline__ bool mbar_wait_1t(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    for (uint32_t i = 0; i < (1u << 15); ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait(bar, parity, abort_flag);
}
// Tiled load of a [rows x 1024-byte] box of a tensor seen as rows of 256 32-bit words, for a CTA pair: the bytes land in
// this CTA's shared memory, their count is reported to `bar`, a shared::cluster address that may lie in the peer CTA
// (.cta_group::2).  No cluster multicast.  The first coordinate is 0: always 16-byte aligned.
__device__ __forceinline__ void tma_rows_pair(uint32_t dst, const CUtensorMap *map, int row, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(map), "r"(0), "r"(row), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx_cluster(uint32_t cluster_bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.release.cluster.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_bar), "r"(bytes) : "memory");
}
// One non-blocking look at a barrier.  The result is a register the caller reads much later: the instruction's round
// trip (a few hundred clocks even when the phase is complete) then overlaps whatever is issued in between.
__device__ __forceinline__ uint32_t mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
__device__ __forceinline__ bool mbar_wait_cluster_1t(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    for (uint32_t i = 0; i < (1u << 15); ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
    }
    return mbar_wait_cluster(bar, parity, abort_flag);
}

// Tiled load of a [rows x 1024-byte] box into this CTA's shared memory, completing on one of this CTA's barriers.
__device__ __forceinline__ void tma_rows_local(uint32_t dst, const CUtensorMap *map, int row, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
                 "l"(map), "r"(0), "r"(row), "r"(bar)
                 : "memory");
}
// Bulk copy from this CTA's shared memory into another CTA's of the cluster (plain peer copy, one source, one destination:
// no multicast); the bytes complete on a barrier that lies in the destination CTA.
__device__ __forceinline__ void dsmem_copy(uint32_t dst_cluster, uint32_t src_cta, uint32_t bytes, uint32_t bar_cluster) {
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_cluster),
                 "r"(src_cta), "r"(bytes), "r"(bar_cluster)
                 : "memory");
}

constexpr int kPairProducers = 512;                  // X producer threads (warps 2..17)
constexpr int kPairThreads = 64 + kPairProducers;

template <int NA, int TN>
struct PairCfg {
    static constexpr int kHalf = TN / 2;                              // tokens of X each CTA stages
    static constexpr int kTokBlocks = (kHalf + 63) / 64;              // 64-token blocks of 128 rows x 128 bytes
    static constexpr int kXStage = kTokBlocks * 16384;
    static constexpr int kWStage = NA * kTileBytes;
    static constexpr int kStage = kWStage + kXStage;                  // a multiple of 1024
    static constexpr int kStagesFit = (227 * 1024 - 512 - 1024) / kStage;
    static constexpr int kStages = kStagesFit > 8 ? 8 : kStagesFit;
    static constexpr int kBarOff = kStages * kStage;
    static constexpr int kTotal = kBarOff + 512 + 1024;
    static constexpr uint32_t kTmemCols = 512;
    static_assert(NA * 256 <= 512 && TN + 8 <= 256 + (NA == 1 ? 8 : 0) && TN % 16 == 0, "tensor memory layout");
    __host__ __device__ static constexpr uint32_t acc_col(int a) { return (uint32_t)a * 256u; }
    __host__ __device__ static constexpr uint32_t meta_col(int a, int buf) { return (uint32_t)a * 256u + TN + 4u * buf; }
};

// X [K, ldx] channel-major -> images of the pair kernel's X stages: image (h, kt) with h = 2 * token tile + CTA rank holds
// channels perm[kt*128 .. +127] of tokens h's half tile, as [64-token block][128 rows][128 bytes] with the 16-byte chunk c
// of row r stored at chunk c ^ (r & 7).  Rows beyond K and tokens beyond M are zero.  grid (2 * token tiles, k_tiles):
// early channel steps of every token tile first, the order the GEMM consumes them in.
//
// flags[h * k_tiles + kt] goes 0 -> 1 when image (h, kt) is complete.  The dependent GEMM may start once every CTA
// here has passed griddepcontrol.launch_dependents, which each CTA issues only after it has lowered its own flag (left
// up by the previous call, or garbage in a fresh workspace): the GEMM never sees a stale 1.
template <int TN>
__global__ void __launch_bounds__(256) xtile_kernel(const uint16_t *__restrict__ X, long ldx, int M, int K,
                                                    const int32_t *__restrict__ perm, uint8_t *__restrict__ img,
                                                    uint32_t *__restrict__ flags, int k_tiles) {
    using L = PairCfg<2, TN>;
    const int h = blockIdx.x, kt = blockIdx.y;
    const int tok_cta = (h >> 1) * TN + (h & 1) * L::kHalf;
    uint8_t *dst = img + ((size_t)h * k_tiles + kt) * L::kXStage;
    uint32_t *flag = flags + (size_t)h * k_tiles + kt;
    // thread -> chunk cc = tid & 7 of rows (tid >> 3) + 32 * i; its permutation entries do not depend on the preceding
    // kernel, and all of its row loads are in flight together
    const int cc = threadIdx.x & 7, r0 = threadIdx.x >> 3;
    int ch[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int kpos = kt * kTileK + r0 + 32 * i;
        ch[i] = kpos < K ? (perm ? __ldg(perm + kpos) : kpos) : -1;
    }
    grid_dependency_wait();                  // X may be the preceding kernel's output; the images may still be read by it
    if (threadIdx.x == 0) {
        asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(flag), "r"(0u) : "memory");
        __threadfence();
    }
    __syncthreads();
    grid_launch_dependents();
    uint4 v[4][L::kTokBlocks];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
        for (int tb = 0; tb < L::kTokBlocks; ++tb) {
            const int local = tb * 64 + cc * 8, t = tok_cta + local;
            v[i][tb] = make_uint4(0u, 0u, 0u, 0u);
            if (ch[i] >= 0 && local < L::kHalf && t < M) {
                const uint16_t *src = X + (long)ch[i] * ldx + t;
                if (t + 8 <= M) {
                    v[i][tb] = __ldg(reinterpret_cast<const uint4 *>(src));
                } else {
                    uint16_t e[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) e[j] = (t + j < M) ? __ldg(src + j) : (uint16_t)0;
                    v[i][tb] = make_uint4(e[0] | ((uint32_t)e[1] << 16), e[2] | ((uint32_t)e[3] << 16),
                                          e[4] | ((uint32_t)e[5] << 16), e[6] | ((uint32_t)e[7] << 16));
                }
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = r0 + 32 * i;
#pragma unroll
        for (int tb = 0; tb < L::kTokBlocks; ++tb)
            *reinterpret_cast<uint4 *>(dst + tb * 16384 + r * 128 + ((cc ^ (r & 7)) << 4)) = v[i][tb];
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(flag), "r"(1u) : "memory");
}

// ---- token-major X: the same images straight from X [M, ldx], one pass instead of a transposed copy plus the pass above.
// A CTA reads 64 tokens x 64 consecutive channels (128 contiguous bytes per token), transposes them in shared memory and
// writes, for each of its channels c, the 128-byte image row of position inv[c] in the permuted order (a whole swizzled
// row: 64 tokens).  An image gets rows from every channel group, so completion is counted per half tile h: the CTA that
// finishes h raises all of h's flags.  xtile_prep_kernel inverts the permutation and clears flags and counters first.
__global__ void xtile_prep_kernel(const int32_t *__restrict__ perm, int K, int32_t *__restrict__ inv, uint32_t *__restrict__ flags,
                                  int n_flags, uint32_t *__restrict__ counts, int n_counts) {
    grid_dependency_wait();                  // a preceding GEMM on this workspace may still be reading its flags
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < K) inv[perm ? __ldg(perm + i) : i] = i;
    if (i < n_flags) flags[i] = 0u;
    if (i < n_counts) counts[i] = 0u;
}

template <int TN>
__global__ void __launch_bounds__(256) xtile_tm_kernel(const uint16_t *__restrict__ X, long ldx, int M, int K,
                                                       const int32_t *__restrict__ inv, uint8_t *__restrict__ img,
                                                       uint32_t *__restrict__ flags, uint32_t *__restrict__ counts, int k_tiles) {
    using L = PairCfg<2, TN>;
    __shared__ uint32_t s[64][33];           // [channel][token pair], one word of padding per row
    __shared__ int s_last;
    const int h = blockIdx.x, tb = blockIdx.y, c0 = blockIdx.z * 64;
    const int tok_cta = (h >> 1) * TN + (h & 1) * L::kHalf;
    grid_dependency_wait();                  // inv, the cleared flags and X itself come from preceding kernels
    grid_launch_dependents();                // the GEMM may start: every flag it can see now is 0 or freshly raised
    uint16_t *s16 = reinterpret_cast<uint16_t *>(&s[0][0]);
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const int idx = threadIdx.x + 256 * j;
        const int chunk = idx & 7, tok = idx >> 3;
        const int local = tb * 64 + tok, t = tok_cta + local, c = c0 + chunk * 8;
        uint16_t e[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) e[i] = 0;
        if (local < L::kHalf && t < M && c < K) {
            const uint16_t *src = X + (long)t * ldx + c;
            if (c + 8 <= K) {
                const uint4 v = __ldg(reinterpret_cast<const uint4 *>(src));
                e[0] = (uint16_t)v.x; e[1] = (uint16_t)(v.x >> 16); e[2] = (uint16_t)v.y; e[3] = (uint16_t)(v.y >> 16);
                e[4] = (uint16_t)v.z; e[5] = (uint16_t)(v.z >> 16); e[6] = (uint16_t)v.w; e[7] = (uint16_t)(v.w >> 16);
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) if (c + i < K) e[i] = __ldg(src + i);
            }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) s16[(chunk * 8 + i) * 66 + tok] = e[i];
    }
    __syncthreads();
    uint8_t *base = img + (size_t)h * k_tiles * L::kXStage + tb * 16384;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const int idx = threadIdx.x + 256 * j;
        const int cc = idx & 7, ch = idx >> 3;
        const int c = c0 + ch;
        if (c < K) {
            const int q = __ldg(inv + c), kt = q >> 7, r = q & 127;
            const uint4 v = make_uint4(s[ch][cc * 4], s[ch][cc * 4 + 1], s[ch][cc * 4 + 2], s[ch][cc * 4 + 3]);
            *reinterpret_cast<uint4 *>(base + (size_t)kt * L::kXStage + r * 128 + ((cc ^ (r & 7)) << 4)) = v;
        }
    }
    if (blockIdx.z == gridDim.z - 1) {       // rows of the last channel step beyond K
        for (int idx = threadIdx.x; idx < (k_tiles * kTileK - K) * 8; idx += 256) {
            const int cc = idx & 7, q = K + (idx >> 3), r = q & 127;
            *reinterpret_cast<uint4 *>(base + (size_t)(q >> 7) * L::kXStage + r * 128 + ((cc ^ (r & 7)) << 4)) = make_uint4(0u, 0u, 0u, 0u);
        }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t done = atomicAdd(counts + h, 1u) + 1u;
        s_last = done == gridDim.y * gridDim.z;
        if (s_last) __threadfence();
    }
    __syncthreads();
    if (s_last)
        for (int kt = threadIdx.x; kt < k_tiles; kt += 256)
            asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(flags + (size_t)h * k_tiles + kt), "r"(1u) : "memory");
}

// How the two pairs of a four-CTA cluster share weight tiles (SHARE below): not at all (clusters of two), by a hand-over
// through distributed shared memory, or by a load that the memory system delivers to both pairs at once.  The last form's
// load instruction is not in this file: the translation unit that builds that form specialises this struct with
//   static __device__ void rows(uint32_t dst, const CUtensorMap *map, int row, uint32_t bar, uint16_t cta_mask)
// (box of whole 1024-byte rows to offset `dst` of every CTA of the mask, bytes reported to the barrier at `bar`'s offset in the
// even CTA of each destination's pair).
constexpr int kShareNone = 0, kShareHandOver = 1, kShareReplicate = 2;
template <int SHARE>
struct SharedTileLoad;

template <int NA, int TN, bool TILED, int SHARE = kShareNone>
__global__ void __launch_bounds__(kPairThreads, 1) spgemm_pair_kernel(const GemmParams p, const __grid_constant__ CUtensorMap wmap,
                                                                      const __grid_constant__ CUtensorMap xmap) {
    using L = PairCfg<NA, TN>;
    constexpr int STAGES = L::kStages;
    constexpr bool QUAD = SHARE != kShareNone;                            // clusters of four: two pairs on the same features
    constexpr bool REPL = SHARE == kShareReplicate;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar_base = sbase + L::kBarOff;
    auto full = [&](int s) { return bar_base + 8u * s; };
    auto empty = [&](int s) { return bar_base + 8u * (8 + s); };
    const uint32_t accum_bar = bar_base + 8u * 24;
    const uint32_t recv_bar = bar_base + 8u * 26;
    auto wland = [&](int s) { return bar_base + 8u * (16 + s); };     // QUAD: this CTA's own weight tile of the stage has landed
    auto wrecv = [&](int s) { return bar_base + 8u * (32 + s); };     // QUAD: the partner's weight tile has arrived here
    static_assert(SHARE == kShareNone || (TILED && NA == 2), "the four-CTA forms exist for the tiled two-accumulator kernel");
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + L::kBarOff + 8 * 25);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + L::kBarOff + 8 * 25 + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // cluster (2, 1, split): ranks 2z and 2z + 1 are the CTA pair of K-slice z.
    // QUAD, cluster (4, 1, 1): ranks 0, 1 and ranks 2, 3 are two pairs on the SAME 512 features and on neighbouring token
    // tiles.  Each CTA fetches only one of its two weight tiles from L2 / HBM (the pair on the first token tile fetches
    // accumulator 0's, the other pair accumulator 1's) and hands a copy to the CTA of the same pair rank in the other pair
    // through distributed shared memory: a weight tile crosses the L2 -> SM path once per two token tiles.
    const uint32_t crank = cluster_ctarank();
    const uint32_t rank = crank & 1u;                                     // 0 = leader of its pair
    const uint32_t lead = crank & ~1u;                                    // cluster rank of the pair's leader
    const int split = QUAD ? 1 : (int)gridDim.z, slice = QUAD ? 0 : (int)(crank >> 1);
    const int qpair = QUAD ? (int)(crank >> 1) : 0;                       // which of the cluster's two token tiles
    // Cluster -> tile.  Clusters start in the order of their linear index (x fastest).  Taken row by row, one wave of
    // clusters would span every feature pair on one or two token tiles, i.e. stream the whole weight from HBM once per
    // wave.  With p.raster_panel = P > 1 the index runs down panels of P token tiles instead (P tiles of one feature pair,
    // then the next pair): a wave then covers about 74 / P feature pairs x P token tiles, whose weight tiles and X images
    // together stay in L2 while the wave runs.
    int pair_idx = (int)blockIdx.x >> (QUAD ? 2 : 1);
    int ttile = (int)blockIdx.y;                                          // (QUAD: index of the pair of token tiles)
    if (p.raster_panel > 1) {
        const int f_pairs = (int)gridDim.x >> (QUAD ? 2 : 1), t_tiles = (int)gridDim.y;
        const int c = ttile * f_pairs + pair_idx;
        const int per_panel = p.raster_panel * f_pairs;
        const int panel = c / per_panel, r = c - panel * per_panel;
        const int height = min(p.raster_panel, t_tiles - panel * p.raster_panel);
        pair_idx = r / height;
        ttile = panel * p.raster_panel + (r - pair_idx * height);
    }
    if (QUAD) ttile = 2 * ttile + qpair;
    const bool has_tokens = ttile * TN < p.M;                             // (QUAD with an odd number of token tiles: the last cluster's second pair only hands on weights)
    const int tok0 = ttile * TN;                                          // first token of the pair's tile
    const int tok_cta = tok0 + (int)rank * L::kHalf;                      // first token this CTA stages
    const int kt_begin = slice * p.k_tiles_per_split;
    const int nk = max(0, min(p.k_tiles, kt_begin + p.k_tiles_per_split) - kt_begin);
    const int f_tiles = (p.N + 127) / 128;
    const int cnt4 = (((TN + split - 1) / split) + 3) & ~3;               // K-slice reduction: token rows per owner
    const int owned = max(0, min(cnt4, TN - slice * cnt4));
    int ftile[NA];
    bool present[NA];
    int n_present = 0, n_present_peer = 0;
#pragma unroll
    for (int a = 0; a < NA; ++a) {
        ftile[a] = pair_idx * (2 * NA) + 2 * a + (int)rank;               // MMA a: rows 0..127 from rank 0, 128..255 from rank 1
        present[a] = ftile[a] < f_tiles;
        n_present += present[a] ? 1 : 0;
        n_present_peer += (pair_idx * (2 * NA) + 2 * a + 1 - (int)rank) < f_tiles ? 1 : 0;
    }

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            // The MMA thread waits on one barrier per step, the leader's.  Gather form: one arrival per weight-tile copy +
            // the X threads, + rank 1's relayed "my stage has landed".  Tiled form: every copy of BOTH CTAs arrives on it
            // and reports its bytes to it directly (rank 1's own `full` barriers stay unused).
            // QUAD: the X copies of both CTAs (if the pair has tokens) + from each CTA of the pair one "my own weight tile
            // has landed" and one "the partner's tile has arrived"; a slot is free once BOTH pairs' MMAs are done with it.
            // REPL: the X copies of both CTAs (if the pair has tokens) + the four weight-tile copies of the cluster, each of
            // which reports to both pairs' leaders.
            mbar_init(full(s), QUAD ? (has_tokens ? 6u : 4u)
                               : TILED ? 2u + (uint32_t)n_present + (uint32_t)n_present_peer
                                       : (uint32_t)kPairProducers + (uint32_t)n_present + (rank == 0 ? 1u : 0u));
            mbar_init(empty(s), QUAD ? 2 : 1);
            if (QUAD && !REPL) { mbar_init(wland(s), 1); mbar_init(wrecv(s), 1); }
        }
        mbar_init(accum_bar, 1);
        mbar_init(recv_bar, 1);
        *abort_flag = 0;
        fence_barrier_init();
        // K-slices: every slice sends this CTA its owned rows of all NA accumulators (128 features x `owned` rows of fp32 each)
        if (split > 1) mbar_arrive_expect_tx(recv_bar, (uint32_t)(NA * split * owned * 512));
    }
    if (warp == 1) tmem_alloc_pair(smem_u32(tmem_slot), L::kTmemCols);
    // a feature tile beyond N: zero values and legal metadata once, never loaded
#pragma unroll
    for (int a = 0; a < NA; ++a) {
        if (!present[a]) {
            for (int s = 0; s < STAGES; ++s) {
                uint32_t *dst = reinterpret_cast<uint32_t *>(smem + s * L::kStage + a * kTileBytes);
                for (int i = threadIdx.x; i < kTileBytes / 4; i += kPairThreads) dst[i] = (i < kTileValBytes / 4) ? 0u : 0x44444444u;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                      // both CTAs have their barriers and tensor memory before any cross-CTA signal
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    grid_launch_dependents();                // (static_weights) the next launch may be set up while this one runs

    if (warp == 0) {
        // idle: keeps the producer warps at indices 2..17 (tensor-memory lane quarter = warp index % 4)
        if (split > 1) cluster_sync_all();   // K-slices: "every pair's MMAs are done with the ring" (see the epilogue)
    } else if (warp == 1) {
        if (lane == 0 && rank != 0) {
            // gather form: forward "my operands of this stage have landed" to the leader
            for (int it = 0; it < (TILED ? 0 : nk); ++it) {
                const int s = it % STAGES;
                const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
                if (!mbar_wait_1t(full(s), ph, abort_flag)) break;
                if (!TILED) fence_async_smem();   // rows written by cp.async (generic proxy) -> read by the MMA (async proxy)
                mbar_arrive_remote(map_to_rank(full(s), lead));
            }
        } else if (lane == 0) {
            // One thread issues every MMA of the pair, so its own instruction stream must stay far shorter than the
            // MMAs' execution time: all descriptors are built once (stage 0) and a stage only adds its byte offset
            // (>> 4) to their low words; the loop is unrolled over the ring and the metadata double buffer so that
            // every column index and offset is a compile-time constant.
            constexpr uint32_t idesc = instr_desc_sparse_f16(256, TN, 1);
            const uint16_t pair_mask = (uint16_t)(3u << lead);            // both CTAs of this pair
            uint64_t ad0[NA][4], bd0[4], md0[NA];
#pragma unroll
            for (int a = 0; a < NA; ++a) {
                md0[a] = smem_desc(sbase + a * kTileBytes + kTileValBytes, 0, 128, kLayoutNone);
#pragma unroll
                for (int j = 0; j < 4; ++j) ad0[a][j] = smem_desc(sbase + a * kTileBytes + j * 32, 16, 1024, kLayoutSw128);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) bd0[j] = smem_desc(sbase + L::kWStage + j * 4096, 16384, 1024, kLayoutSw128);
            constexpr int kUnroll = STAGES * 2;                           // ring slot and metadata buffer both periodic
            bool alive = true;
            uint32_t seen = 0;                                            // the next step's barrier was seen complete
            for (int it0 = 0; it0 < nk && alive; it0 += kUnroll) {
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    const int it = it0 + u;
                    if (it >= nk) break;
                    // it0 is a multiple of 2 * STAGES: slot and barrier phase of step it0 + u are compile-time constants
                    const int s = u % STAGES;
                    const uint32_t ph = (uint32_t)(u / STAGES) & 1u;
                    uint32_t seen_a = 0, seen_b = 0;
                    const uint32_t nbar = full((u + 1) % STAGES), nph = (uint32_t)(((u + 1) % kUnroll) / STAGES) & 1u;
                    // Rank 1's arrival only relays that its stage is complete: one barrier for both CTAs, no cluster-scope
                    // acquire; a proxy fence only where the rows were written by cp.async.  A wait costs this thread ~300 clocks even
                    // when the phase is complete -- with the ~700 it needs to issue a step's MMAs that is more than the 960
                    // they run -- so the next step's barrier is looked at without blocking while this step is being issued,
                    // and waited on only if not seen yet.
                    if (!seen && !mbar_wait_1t(full(s), ph, abort_flag)) { alive = false; break; }
                    if (!TILED) fence_async_smem();
                    if (it + 1 < nk) seen_a = mbar_test(nbar, nph);
                    tc_fence_after();
                    const uint64_t soff = (uint64_t)((uint32_t)(s * L::kStage) >> 4);   // added to the address field
#pragma unroll
                    for (int a = 0; a < NA; ++a) {
                        const uint32_t e_col = L::meta_col(a, u & 1);     // == meta_col(a, it & 1) (kUnroll is even)
                        tc_copy_128x128b_pair(tmem + e_col, md0[a] + soff);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint32_t col = e_col + j;
                            tc_mma_sparse_f16_pair(tmem + L::acc_col(a), ad0[a][j] + soff, bd0[j] + soff, tmem + (col & ~1u),
                                                   idesc | (col & 1u), (it > 0 || j > 0) ? 1u : 0u);
                        }
                        if (it + 1 < nk) seen_b |= mbar_test(nbar, nph);
                    }
                    tc_commit_pair(empty(s), QUAD ? (uint16_t)0xF : pair_mask);
                    seen = seen_a | seen_b;
                }
            }
            tc_commit_pair(accum_bar, pair_mask);
        }
        __syncwarp();
        if (split > 1) cluster_sync_all();
    } else {
        const int g = threadIdx.x - 64;
        bool alive = true;
        if constexpr (TILED) {
            // ---- copy issuers: lane 0 of warp 2 + s * (NA + 1) + kind feeds ring slot s with weight tile `kind` (< NA) or
            // with the X image (kind == NA); it meets every phase of its slot's `empty` barrier.  The other lanes wait at
            // the vote below without polling.
            constexpr int kCopies = REPL ? 2 : QUAD ? 4 : NA + 1;
            static_assert(kCopies * STAGES <= 15, "one issuing warp per copy of the ring; warp 17 polls the accumulator barrier");
            const int iw = warp - 2;
            if constexpr (REPL) if (lane == 0 && iw < kCopies * STAGES) {
                // ---- two lanes per ring slot: 0 fetches ONE weight tile (accumulator `qpair`'s, for this CTA's pair rank)
                // into this CTA and into the CTA of the same pair rank in the other pair with a single load; 1 fetches the X
                // image.  Both of this CTA's weight tiles of a stage therefore arrive from two loads, one of its own and one
                // of the other pair's, and a tile crosses the L2 -> SM path once per two token tiles.  A slot may be refilled
                // once BOTH pairs' MMAs are done with it (`empty` takes both commits), since the load writes into both.
                const int s = iw / kCopies, role = iw % kCopies;
                const int a_own = qpair;
                const uint32_t full_own = map_to_rank(full(s), lead), full_other = map_to_rank(full(s), lead ^ 2u);
                constexpr int kRowBytes = 1024;
                if (role == 0) {
                    const int row_step = kTileBytes / kRowBytes;
                    const int row0 = ftile[a_own] * p.k_tiles * row_step;
                    const uint32_t dst = sbase + s * L::kStage + a_own * kTileBytes;
                    const uint16_t both = (uint16_t)((1u << rank) | (1u << (rank + 2u)));
                    for (int it = s; it < nk; it += STAGES) {
                        const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
                        if (!mbar_wait_1t(empty(s), ph ^ 1u, abort_flag)) { alive = false; break; }
                        if (present[a_own]) {
                            mbar_arrive_expect_tx_cluster(full_own, kTileBytes);
                            mbar_arrive_expect_tx_cluster(full_other, kTileBytes);
                            SharedTileLoad<SHARE>::rows(dst, &wmap, row0 + it * row_step, full_own, both);
                        } else {
                            mbar_arrive_remote(full_own);
                            mbar_arrive_remote(full_other);
                        }
                    }
                } else if (has_tokens) {
                    const uint32_t *xflag = p.xflags + (size_t)(ttile * 2 + rank) * p.k_tiles;
                    const int row_step = L::kXStage / kRowBytes;
                    const int row0 = (int)((ttile * 2 + rank) * p.k_tiles) * row_step;
                    const uint32_t dst = sbase + s * L::kStage + L::kWStage;
                    for (int it = s; it < nk; it += STAGES) {
                        const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
                        if (!xflag_wait(xflag + it, abort_flag)) { alive = false; break; }
                        asm volatile("fence.proxy.async;" ::: "memory");
                        if (!mbar_wait_1t(empty(s), ph ^ 1u, abort_flag)) { alive = false; break; }
                        mbar_arrive_expect_tx_cluster(full_own, (uint32_t)L::kXStage);
                        tma_rows_pair(dst, &xmap, row0 + it * row_step, full_own);
                    }
                }
            }
            if (QUAD && !REPL && lane == 0 && iw < kCopies * STAGES) {
                // ---- four lanes per ring slot: 0 fetches this CTA's share of the weight tiles, 1 the X image, 2 hands the
                // fetched tile on to the partner CTA once it has landed, 3 reports the tile received from the partner
                const int s = iw / kCopies, role = iw % kCopies;
                const int a_own = qpair, a_got = 1 - qpair;
                const uint32_t partner = crank ^ 2u;
                const uint32_t lead_full = map_to_rank(full(s), lead);
                constexpr int kRowBytes = 1024;
                if (role == 0) {
                    const int row_step = kTileBytes / kRowBytes;
                    const int row0 = ftile[a_own] * p.k_tiles * row_step;
                    const uint32_t dst = sbase + s * L::kStage + a_own * kTileBytes;
                    for (int it = s; it < nk; it += STAGES) {
                        const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
                        if (!mbar_wait_1t(empty(s), ph ^ 1u, abort_flag)) { alive = false; break; }
                        if (present[a_own]) {
                            mbar_arrive_expect_tx(wland(s), kTileBytes);
                            tma_rows_local(dst, &wmap, row0 + it * row_step, wland(s));
                        } else {
                            mbar_arrive(wland(s));
                        }
                    }
                } else if (role == 1) {
                    if (has_tokens) {
                        const uint32_t *xflag = p.xflags + (size_t)(ttile * 2 + rank) * p.k_tiles;
                        const int row_step = L::kXStage / kRowBytes;
                        const int row0 = (int)((ttile * 2 + rank) * p.k_tiles) * row_step;
                        const uint32_t dst = sbase + s * L::kStage + L::kWStage;
                        for (int it = s; it < nk; it += STAGES) {
                            const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
                            if (!xflag_wait(xflag + it, abort_flag)) { alive = false; break; }
                            asm volatile("fence.proxy.async;" ::: "memory");
                            if (!mbar_wait_1t(empty(s), ph ^ 1u, abort_flag)) { alive = false; break; }
                            mbar_arrive_expect_tx_cluster(lead_full, (uint32_t)L::kXStage);
                            tma_rows_pair(dst, &xmap, row0 + it * row_step, lead_full);
                        }
                    }
                } else if (role == 2) {
                    // (the partner's slot is free: this CTA's `empty` barrier of the round took both pairs' commits before
                    // the tile was fetched)
                    const uint32_t src = sbase + s * L::kStage + a_own * kTileBytes;
                    const uint32_t dst = map_to_rank(src, partner), rbar = map_to_rank(wrecv(s), partner);
                    for (int it = s; it < nk; it += STAGES) {
                        const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
                        if (!mbar_wait_1t(wland(s), ph, abort_flag)) { alive = false; break; }
                        if (present[a_own]) {
                            mbar_arrive_expect_tx_cluster(rbar, kTileBytes);
                            dsmem_copy(dst, src, kTileBytes, rbar);
                        } else {
                            mbar_arrive_remote(rbar);
                        }
                        mbar_arrive_remote(lead_full);
                    }
                } else {
                    (void)a_got;
                    for (int it = s; it < nk; it += STAGES) {
                        const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
                        if (!mbar_wait_cluster_1t(wrecv(s), ph, abort_flag)) { alive = false; break; }
                        mbar_arrive_remote(lead_full);
                    }
                }
            }
            if (!QUAD && lane == 0 && iw < kCopies * STAGES) {
                const int s = iw / kCopies, kind = iw % kCopies;
                const bool is_x = kind == NA;
                const uint32_t *xflag = p.xflags + (size_t)(ttile * 2 + rank) * p.k_tiles + kt_begin;
                if (is_x || present[kind]) {
                    const uint32_t bytes = is_x ? (uint32_t)L::kXStage : (uint32_t)kTileBytes;
                    constexpr int kRowBytes = 1024;                       // the tensor maps see both buffers as 1024-byte rows
                    const CUtensorMap *map = is_x ? &xmap : &wmap;
                    const int row0 = is_x ? (int)((ttile * 2 + rank) * p.k_tiles + kt_begin) * (L::kXStage / kRowBytes)
                                          : (ftile[kind] * p.k_tiles + kt_begin) * (kTileBytes / kRowBytes);
                    const int row_step = (int)bytes / kRowBytes;
                    const uint32_t dst = sbase + s * L::kStage + (is_x ? L::kWStage : kind * kTileBytes);
                    const uint32_t lead_full = map_to_rank(full(s), lead);
                    for (int it = s; it < nk; it += STAGES) {
                        const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
                        if (is_x) {
                            // the image is written by the tiling pass while this kernel runs: wait for its flag (long up,
                            // except in the first steps) before the slot's own wait, then order the generic-proxy writes
                            // just acquired before this thread's asynchronous-proxy read
                            if (!xflag_wait(xflag + it, abort_flag)) { alive = false; break; }
                            asm volatile("fence.proxy.async;" ::: "memory");
                        }
                        if (!mbar_wait_1t(empty(s), ph ^ 1u, abort_flag)) { alive = false; break; }
                        mbar_arrive_expect_tx_cluster(lead_full, bytes);
                        tma_rows_pair(dst, map, row0 + it * row_step, lead_full);
                    }
                }
            }
        } else {
        // ---- X producers: thread g copies 16-byte chunk (g & 7) of rows (g >> 3) and (g >> 3) + 64 of every 64-token
        // block.  Its two permutation entries are loaded kAhead steps early into registers (the loop is unrolled by
        // kAhead so the register ring has constant indices): the load's latency never sits between two steps.
        const int cc = g & 7, rg = g >> 3;
        const uint16_t *xb = reinterpret_cast<const uint16_t *>(p.X);
        constexpr int kAhead = 4;
        auto channel_of = [&](int it, int row) -> int {
            const int kpos = (kt_begin + it) * kTileK + row;
            return (it < nk && kpos < p.K) ? (p.perm ? __ldg(p.perm + kpos) : kpos) : -1;
        };
        int nxt[kAhead][2];
#pragma unroll
        for (int u = 0; u < kAhead; ++u) { nxt[u][0] = channel_of(u, rg); nxt[u][1] = channel_of(u, rg + 64); }
        grid_dependency_wait();              // (static_weights) X and Y may belong to the preceding kernel until it is done
        for (int it0 = 0; it0 < nk; it0 += kAhead) {
#pragma unroll
            for (int u = 0; u < kAhead; ++u) {
                const int it = it0 + u;
                if (it >= nk) break;
                const int ch[2] = {nxt[u][0], nxt[u][1]};
                nxt[u][0] = channel_of(it + kAhead, rg);
                nxt[u][1] = channel_of(it + kAhead, rg + 64);
                const int s = it % STAGES;
                const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
                if (alive && !mbar_wait(empty(s), ph ^ 1u, abort_flag)) alive = false;
                if (!alive) continue;
                const uint32_t xs = sbase + s * L::kStage + L::kWStage;
#pragma unroll
                for (int tb = 0; tb < L::kTokBlocks; ++tb) {
                    const int local = tb * 64 + cc * 8;                   // token index inside this CTA's half
                    if (local < L::kHalf) {
                        const int t = tok_cta + local;
                        const int valid = min(8, max(0, p.M - t));
#pragma unroll
                        for (int i = 0; i < 2; ++i) {
                            const int r = rg + 64 * i;
                            const bool in = ch[i] >= 0 && valid > 0;
                            const uint16_t *src = in ? xb + (long)ch[i] * p.ldx + t : xb;
                            cp_async_16(xs + tb * 16384 + r * 128 + ((cc ^ (r & 7)) << 4), src, in ? valid * 2 : 0);
                        }
                    }
                }
                cp_async_arrive_noinc(full(s));
                // Weight tile a of this stage is issued by lane 0 of producer warp s * NA + a: copies issued by one thread
                // do not overlap, and spinning lanes of one warp would hold each other up, so every copy of the ring
                // has a warp of its own, which has just seen the stage's `empty` barrier anyway.
                if (lane == 0 && (warp - 2) / NA == s && (warp - 2) < NA * STAGES) {
                    const int a = (warp - 2) % NA;
                    if (present[a]) {
                        mbar_arrive_expect_tx(full(s), kTileBytes);
                        bulk_load(sbase + s * L::kStage + a * kTileBytes,
                                  p.packed + ((long)ftile[a] * p.k_tiles + kt_begin + it) * kTileBytes, kTileBytes, full(s));
                    }
                }
            }
        }
        }
        // ---- epilogue: this CTA's 128 feature rows of every accumulator, all TN token columns; warp w reads lane
        // quarter w % 4 and the 16-column pieces (w - 2) / 4, + 4, + 8, ...
        const int quarter = warp & 3;
        const int cgrp = (warp - 2) >> 2;
        const int f_local = quarter * 32 + lane;
        // One thread polls the accumulator barrier; the other 511 sleep on a named barrier meanwhile (in the tiled form
        // most of them are idle for the whole main loop, and hundreds of polling lanes slow every other barrier down).
        if (!alive) *abort_flag = 1;
        __syncwarp();
        if (warp == 17 && lane == 0 && nk > 0) (void)mbar_wait_cluster(accum_bar, 0, abort_flag);
        __syncwarp();
        asm volatile("bar.sync 1, %0;" ::"n"(kPairProducers) : "memory");
        const bool ok = *abort_flag == 0;
        tc_fence_after();
        const bool y_vec = (reinterpret_cast<uintptr_t>(p.Y) & 15) == 0;
        // accumulator a -> shared memory [token][128 features] in the output type -> 16-byte stores along the features.
        // fp16 output: both accumulators are staged side by side (2 x TN x 256 bytes) and stored in one sweep.
        auto stage_acc = [&](int a, uint8_t *area, auto out_tag) {
            using OutT = decltype(out_tag);
            const float bias_f = epilogue_bias(p, (long)ftile[a] * 128 + f_local);
#pragma unroll 1
            for (int c0 = cgrp * 16; c0 < TN; c0 += 64) {
                uint32_t v[16];
                if (nk > 0 && ok) {
                    tmem_load_16(tmem + ((uint32_t)(quarter * 32) << 16) + L::acc_col(a) + c0, v);
                } else {
#pragma unroll
                    for (int e = 0; e < 16; ++e) v[e] = 0;
                }
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const float y = epilogue_apply(__uint_as_float(v[e]), bias_f, p.act);
                    if (sizeof(OutT) == 4) reinterpret_cast<float *>(area)[(c0 + e) * 128 + f_local] = y;
                    else reinterpret_cast<__half *>(area)[(c0 + e) * 128 + f_local] = __float2half_rn(y);
                }
            }
        };
        auto store_acc = [&](int a, const uint8_t *area, auto out_tag) {
            using OutT = decltype(out_tag);
            constexpr int kPer = 16 / (int)sizeof(OutT);                  // features per 16-byte piece
            constexpr int kPieces = 128 / kPer;                           // pieces per token row
            if (!present[a]) return;
            const int f_valid = min(128, p.N - ftile[a] * 128);
            const bool vec_ok = y_vec && (((long)p.ldy * (long)sizeof(OutT)) % 16 == 0);
            OutT *yo = reinterpret_cast<OutT *>(p.Y) + (long)ftile[a] * 128;
            for (int idx = g; idx < TN * kPieces; idx += kPairProducers) {
                const int row = idx / kPieces, c = idx % kPieces;
                const int t = tok0 + row;
                if (!ok || t >= p.M) continue;
                const int f0 = c * kPer;
                OutT *dst = yo + (long)t * p.ldy + f0;
                const OutT *srcp = reinterpret_cast<const OutT *>(area) + row * 128 + f0;
                if (vec_ok && f0 + kPer <= f_valid) {
                    *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(srcp);
                } else {
                    for (int e = 0; e < kPer; ++e)
                        if (f0 + e < f_valid) dst[e] = srcp[e];
                }
            }
        };
        if (split > 1) {
            // ---- K-slices: the pairs of the cluster hold partial sums of the same tile.  Its token rows are dealt to the
            // slices in runs of cnt4 rows; every CTA sends, for each accumulator, the rows of each run to the CTA of the
            // same pair rank in the owning slice (16-byte asynchronous remote stores: four token columns of one feature,
            // completing on the owner's barrier), into the ring, which a cluster barrier has just declared free everywhere.
            // The owner adds the slices in slice order and stores its rows.
            cluster_sync_all();
            const int groups = cnt4 >> 2;
#pragma unroll 1
            for (int a = 0; a < NA; ++a) {
#pragma unroll 1
                for (int c0 = cgrp * 16; c0 < TN; c0 += 64) {
                    uint32_t v[16];
                    if (nk > 0 && ok) {
                        tmem_load_16(tmem + ((uint32_t)(quarter * 32) << 16) + L::acc_col(a) + c0, v);
                    } else {
#pragma unroll
                        for (int e = 0; e < 16; ++e) v[e] = 0;
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int row = c0 + 4 * j;
                        const int owner = row / cnt4, rg = (row - owner * cnt4) >> 2;
                        const uint32_t local = sbase + (uint32_t)((((a * split + slice) * groups + rg) * 128 + f_local) * 16);
                        const uint32_t dst_rank = (uint32_t)(2 * owner) + rank;
                        st_async_v4(map_to_rank(local, dst_rank), v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3],
                                    map_to_rank(recv_bar, dst_rank));
                    }
                }
            }
            tc_fence_before();
            const bool got = mbar_wait_cluster(recv_bar, 0, abort_flag);
            const bool fine = got && ok && (*abort_flag == 0);
            const float4 *recv = reinterpret_cast<const float4 *>(smem);
            for (int q = g; q < NA * groups * 128; q += kPairProducers) {
                const int a = q / (groups * 128), rg = (q / 128) % groups, f = q & 127;
                if (rg * 4 >= owned || !present[a]) continue;
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
                for (int z = 0; z < split; ++z) {                     // slice order: deterministic
                    const float4 part = recv[((a * split + z) * groups + rg) * 128 + f];
                    acc[0] += part.x; acc[1] += part.y; acc[2] += part.z; acc[3] += part.w;
                }
                const long feature = (long)ftile[a] * 128 + f;
                if (!fine || feature >= p.N) continue;
                const float bias_f = epilogue_bias(p, feature);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int t = tok0 + slice * cnt4 + rg * 4 + e;
                    if (t >= p.M) continue;
                    const float y = epilogue_apply(acc[e], bias_f, p.act);
                    if (p.out_f32) reinterpret_cast<float *>(p.Y)[(long)t * p.ldy + feature] = y;
                    else reinterpret_cast<__half *>(p.Y)[(long)t * p.ldy + feature] = __float2half_rn(y);
                }
            }
        } else if (!p.out_f32) {
#pragma unroll 1
            for (int a = 0; a < NA; ++a) stage_acc(a, smem + (size_t)a * TN * 256, __half());
            tc_fence_before();
            asm volatile("bar.sync 1, %0;" ::"n"(kPairProducers) : "memory");
#pragma unroll 1
            for (int a = 0; a < NA; ++a) store_acc(a, smem + (size_t)a * TN * 256, __half());
        } else {
#pragma unroll 1
            for (int a = 0; a < NA; ++a) {
                if (a > 0) asm volatile("bar.sync 1, %0;" ::"n"(kPairProducers) : "memory");   // the staging area is free again
                stage_acc(a, smem, float());
                tc_fence_before();
                asm volatile("bar.sync 1, %0;" ::"n"(kPairProducers) : "memory");
                store_acc(a, smem, float());
            }
        }
        tc_fence_before();
    }
    __syncthreads();
    cluster_sync_all();                      // both CTAs are done with tensor memory and with each other's barriers
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem, L::kTmemCols);
    }
}

template <int TN>
size_t xtile_image_bytes(int M, int K) {
    return (size_t)2 * ((M + TN - 1) / TN) * ((K + kTileK - 1) / kTileK) * PairCfg<2, TN>::kXStage;
}
template <int TN>
size_t xtile_flag_bytes(int M, int K) {
    return align_up((size_t)2 * ((M + TN - 1) / TN) * ((K + kTileK - 1) / kTileK) * 4, 256);
}
template <int TN>
size_t xtile_bytes(int M, int K) {           // images | one flag word per image | inverse permutation | one counter per half tile
    return xtile_image_bytes<TN>(M, K) + xtile_flag_bytes<TN>(M, K) + align_up((size_t)K * 4, 256) +
           align_up((size_t)2 * ((M + TN - 1) / TN) * 4, 256);
}

// Token-major X: inverse permutation and cleared flags, then the transposing tiling pass.
template <int TN>
esp_status_t launch_xtile_tm(const GemmParams &p, const uint16_t *X_tm, long ldx_tm, uint8_t *img, uint32_t *flags,
                             bool dependent, cudaStream_t stream) {
    using L = PairCfg<2, TN>;
    const int n_h = 2 * ((p.M + TN - 1) / TN), n_flags = n_h * p.k_tiles;
    int32_t *inv = reinterpret_cast<int32_t *>(reinterpret_cast<uint8_t *>(flags) + xtile_flag_bytes<TN>(p.M, p.K));
    uint32_t *counts = reinterpret_cast<uint32_t *>(reinterpret_cast<uint8_t *>(inv) + align_up((size_t)p.K * 4, 256));
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    const int n = std::max(p.K, std::max(n_flags, n_h));
    cfg.gridDim = dim3((n + 255) / 256, 1, 1);
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    ESP_CUDA_OK(cudaLaunchKernelEx(&cfg, xtile_prep_kernel, p.perm, p.K, inv, flags, n_flags, counts, n_h));
    cfg.gridDim = dim3(n_h, L::kTokBlocks, (p.K + 63) / 64);
    cfg.numAttrs = 1;                        // always a programmatic dependent of the preparation kernel
    ESP_CUDA_OK(cudaLaunchKernelEx(&cfg, xtile_tm_kernel<TN>, X_tm, ldx_tm, p.M, p.K, (const int32_t *)inv, img, flags, counts,
                                   p.k_tiles));
    return ESP_OK;
}

template <int TN>
esp_status_t launch_xtile(const GemmParams &p, uint8_t *img, uint32_t *flags, bool dependent, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * ((p.M + TN - 1) / TN), p.k_tiles, 1);
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    ESP_CUDA_OK(cudaLaunchKernelEx(&cfg, xtile_kernel<TN>, reinterpret_cast<const uint16_t *>(p.X), p.ldx, p.M, p.K, p.perm, img,
                                   flags, p.k_tiles));
    return ESP_OK;
}

// Tensor map over a linear buffer seen as rows of 1024 bytes (256 32-bit words); box = box_rows whole rows, no swizzle.
inline esp_status_t make_rows_tensor_map(const void *base, size_t bytes, int box_rows, CUtensorMap *map) {
    // (a layer calls with the same buffers again and again: the last few maps are kept per thread)
    struct Entry { const void *base; size_t bytes; int box_rows; CUtensorMap map; };
    thread_local Entry cache[16];
    thread_local int n = 0, next = 0;
    for (int i = 0; i < n; ++i)
        if (cache[i].base == base && cache[i].bytes == bytes && cache[i].box_rows == box_rows) {
            *map = cache[i].map;
            return ESP_OK;
        }
    Entry *slot = &cache[next];
    EncodeTiledFn encode = nullptr;
    esp_status_t st = tensor_map_encoder(&encode);
    if (st != ESP_OK) return st;
    cuuint64_t dims[2] = {256, (cuuint64_t)(bytes / 1024)};
    cuuint64_t strides[1] = {1024};
    cuuint32_t box[2] = {256, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void *>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return ESP_ERR_CUDA;
    *slot = Entry{base, bytes, box_rows, *map};
    next = (next + 1) % 16;
    if (n < 16) ++n;
    return ESP_OK;
}

template <int NA, int TN, bool TILED = false>
esp_status_t launch_pair(const GemmParams &p, bool dependent, cudaStream_t stream, int split = 1) {
    using L = PairCfg<NA, TN>;
    auto kern = spgemm_pair_kernel<NA, TN, TILED>;
    ESP_CUDA_OK(ensure_dynamic_smem((const void *)kern, L::kTotal));
    const int f_tiles = (p.N + 127) / 128;
    cudaLaunchConfig_t cfg = {};
    // K-slices: the ring must hold the pushed partial rows of every slice (NA x split x cnt4 x 512 bytes)
    const int cnt4 = (((TN + split - 1) / split) + 3) & ~3;
    if (split < 1 || split > 4 || (split > 1 && (size_t)NA * split * cnt4 * 512 > (size_t)L::kStages * L::kStage)) return ESP_ERR_INVALID_ARG;
    cfg.gridDim = dim3(2 * ((f_tiles + 2 * NA - 1) / (2 * NA)), (p.M + TN - 1) / TN, split);
    cfg.blockDim = dim3(kPairThreads);
    cfg.dynamicSmemBytes = L::kTotal;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = split;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 2 : 1;
    CUtensorMap wmap, xmap;
    memset(&wmap, 0, sizeof(wmap));
    memset(&xmap, 0, sizeof(xmap));
    if constexpr (TILED) {
        esp_status_t st = make_rows_tensor_map(p.packed, (size_t)f_tiles * p.k_tiles * kTileBytes, kTileBytes / 1024, &wmap);
        if (st == ESP_OK) st = make_rows_tensor_map(p.ximg, xtile_image_bytes<TN>(p.M, p.K), L::kXStage / 1024, &xmap);
        if (st != ESP_OK) return st;
    }
    ESP_CUDA_OK(cudaLaunchKernelEx(&cfg, kern, p, wmap, xmap));
    return ESP_OK;
}

// The four-CTA form of the tiled pair kernel: two pairs per cluster on the same 512 features and two neighbouring token
// tiles; each weight tile is fetched once per cluster and handed to the other pair through distributed shared memory.
template <int TN>
esp_status_t launch_quad(const GemmParams &p, bool dependent, cudaStream_t stream) {
    using L = PairCfg<2, TN>;
    auto kern = spgemm_pair_kernel<2, TN, true, kShareHandOver>;
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
