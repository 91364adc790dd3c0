// esp_spgemm: Y = X . P . W_s^T on the 5th-generation tensor cores with the sparse-operand MMA
// ("Efficient Sparse-GEMM Implementation": the product every pruned linear layer runs).
//
// Orientation.  The sparse operand must be the MMA's A operand, so each CTA computes a tile of Y^T:
//   D[feature (128 TMEM lanes), token (TMEM columns)] += Wc[feature, k/2] (sparse, metadata in TMEM) * Xp[k, token]
// The compressed weight arrives as pre-swizzled 18 KB tiles (16 KB values + 2 KB metadata), one bulk
// async copy per pipeline stage; the metadata is copied shared -> tensor memory with tcgen05.cp right
// before the four K=32 MMAs of a 128-channel tile.  The permutation P is applied while the X tile is
// brought into shared memory (element gather in this file), never as a separate pass over X.
// K is split across the CTAs of a thread-block cluster; partial tiles are summed in slice order through
// distributed shared memory, so no global scratch is used and the result is deterministic.
#include "esp_common.cuh"

#include <cuda.h>

#include <cstdio>
#include <cstdlib>
#include <map>
#include <mutex>
#include <string>

#include <dlfcn.h>

#include "spgemm_device.cuh"

namespace esp {
namespace {

template <int BN, int STAGES>
struct GatherSmem {
    static constexpr int kWBytes = STAGES * kTileBytes;
    static constexpr int kXStage = BN * 256;                   // BN tokens x 128 channels fp16
    static constexpr int kXBytes = STAGES * kXStage;
    static constexpr int kStageArea = kWBytes + kXBytes;
    static constexpr int kReduceBytes = BN * 128 * 4;          // fp32 partial tile, aliases the stage area
    static constexpr int kMain = kStageArea > kReduceBytes ? kStageArea : kReduceBytes;
    static constexpr int kBarOff = kMain;                      // barriers, TMEM slot, abort flag
    static constexpr int kTotal = kBarOff + 256 + 1024;        // + slack for 1024-byte alignment of the base
};

// --------------------------------------------------------------------------------------------------
// Gather kernel: any M, either X layout; the X tile is gathered element-wise through the permutation by
// four warps.  Used for decode shapes (X is tiny and cache resident, the weight stream is the cost).
// grid (feature tiles, token tiles, split_k), cluster (1, 1, split_k), block 192:
//   warp 0 lane 0  weight-tile producer (bulk async copies)      warp 1 lane 0  MMA issuer
//   warps 2..5     X gather producers, then epilogue (one TMEM lane quarter each)
// --------------------------------------------------------------------------------------------------
template <int BN, int STAGES>
__global__ void __launch_bounds__(192) spgemm_gather_kernel(const GemmParams p) {
    using L = GatherSmem<BN, STAGES>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t w_base = sbase, x_base = sbase + L::kWBytes;
    const uint32_t bar_base = sbase + L::kBarOff;
    auto full_w = [&](int s) { return bar_base + 8u * s; };
    auto full_x = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto empty = [&](int s) { return bar_base + 8u * (2 * STAGES + s); };
    const uint32_t accum_bar = bar_base + 8u * (3 * STAGES);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + L::kBarOff + 8 * (3 * STAGES + 1));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + L::kBarOff + 8 * (3 * STAGES + 1) + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ft = blockIdx.x, tok0 = blockIdx.y * BN;
    const int split = (int)gridDim.z, slice = (int)blockIdx.z;
    const int kt_begin = slice * p.k_tiles_per_split;
    const int kt_end = min(p.k_tiles, kt_begin + p.k_tiles_per_split);
    const int nk = max(0, kt_end - kt_begin);
    constexpr uint32_t kTmemCols = tmem_cols_for(BN);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_w(s), 1);
            mbar_init(full_x(s), 4);
            mbar_init(empty(s), 1);
        }
        mbar_init(accum_bar, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 0) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            const uint8_t *src = p.packed + ((long)ft * p.k_tiles + kt_begin) * kTileBytes;
            for (int it = 0; it < nk; ++it) {
                const int s = it % STAGES;
                const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
                if (!mbar_wait(empty(s), ph ^ 1u, abort_flag)) break;
                mbar_arrive_expect_tx(full_w(s), kTileBytes);
                bulk_load(w_base + s * kTileBytes, src + (long)it * kTileBytes, kTileBytes, full_w(s));
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc_sparse_f16(128, BN, 0);
            for (int it = 0; it < nk; ++it) {
                const int s = it % STAGES;
                const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
                if (!mbar_wait(full_w(s), ph, abort_flag)) break;
                if (!mbar_wait(full_x(s), ph, abort_flag)) break;
                tc_fence_after();
                const uint32_t wa = w_base + s * kTileBytes;
                const uint32_t xa = x_base + s * L::kXStage;
                const uint32_t e_col = BN + (it & 1) * 4;
                tc_copy_128x128b(tmem + e_col, smem_desc(wa + kTileValBytes, 0, 128, kLayoutNone));
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t col = e_col + j;
                    const uint64_t ad = smem_desc(wa + j * 32, 16, 1024, kLayoutSw128);
                    const uint64_t bd = smem_desc(xa + (j >> 1) * (BN * 128) + (j & 1) * 64, 16, 1024, kLayoutSw128);
                    tc_mma_sparse_f16(tmem, ad, bd, tmem + (col & ~1u), idesc | (col & 1u), (it > 0 || j > 0) ? 1u : 0u);
                }
                tc_commit(empty(s));
            }
            tc_commit(accum_bar);
        }
    } else {
        // ---- X gather: thread g owns channel chunk (g & 15) of tokens (g >> 4) + 8 i
        const int g = threadIdx.x - 64;
        const int chunk = g & 15;
        bool alive = true;
        for (int it = 0; it < nk && alive; ++it) {
            const int s = it % STAGES;
            const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
            if (!mbar_wait(empty(s), ph ^ 1u, abort_flag)) { alive = false; break; }
            const int kc = (kt_begin + it) * kTileK + chunk * 8;
            int th[8];
            if (kc + 8 <= p.K && p.perm) {
                const int4 a = __ldg(reinterpret_cast<const int4 *>(p.perm + kc));
                const int4 b = __ldg(reinterpret_cast<const int4 *>(p.perm + kc + 4));
                th[0] = a.x; th[1] = a.y; th[2] = a.z; th[3] = a.w;
                th[4] = b.x; th[5] = b.y; th[6] = b.z; th[7] = b.w;
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) th[e] = (kc + e < p.K) ? (p.perm ? p.perm[kc + e] : kc + e) : -1;
            }
            uint8_t *xs = smem + L::kWBytes + s * L::kXStage + (chunk >> 3) * (BN * 128);
            const int q = chunk & 7;
            for (int row = g >> 4; row < BN; row += 8) {
                const int t = tok0 + row;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (t < p.M) {
                    uint16_t h[8];
                    const uint16_t *xb = reinterpret_cast<const uint16_t *>(p.X);
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        long off = p.x_channel_major ? ((long)th[e] * p.ldx + t) : ((long)t * p.ldx + th[e]);
                        h[e] = th[e] >= 0 ? __ldg(xb + off) : (uint16_t)0;
                    }
                    v.x = h[0] | ((uint32_t)h[1] << 16);
                    v.y = h[2] | ((uint32_t)h[3] << 16);
                    v.z = h[4] | ((uint32_t)h[5] << 16);
                    v.w = h[6] | ((uint32_t)h[7] << 16);
                }
                *reinterpret_cast<uint4 *>(xs + row * 128 + ((q ^ (row & 7)) << 4)) = v;
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(full_x(s));
        }
        // ---- epilogue: TMEM lane quarter (warp & 3)
        const int quarter = warp & 3;
        const int f_local = quarter * 32 + lane;
        const long feature = (long)ft * 128 + f_local;
        bool ok = alive && (nk == 0 || mbar_wait(accum_bar, 0, abort_flag));
        tc_fence_after();
        float *stage_f32 = reinterpret_cast<float *>(smem);
        const float bias_f = epilogue_bias(p, feature);
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 16) {
            uint32_t v[16];
            if (nk > 0) {
                tmem_load_16(tmem + ((uint32_t)(quarter * 32) << 16) + c0, v);
            } else {
#pragma unroll
                for (int e = 0; e < 16; ++e) v[e] = 0;
            }
            if (split == 1) {
                if (ok && feature < p.N) {
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        const int t = tok0 + c0 + e;
                        if (t < p.M) {
                            const float y = epilogue_apply(__uint_as_float(v[e]), bias_f, p.act);
                            if (p.out_f32) reinterpret_cast<float *>(p.Y)[(long)t * p.ldy + feature] = y;
                            else reinterpret_cast<__half *>(p.Y)[(long)t * p.ldy + feature] = __float2half_rn(y);
                        }
                    }
                }
            } else {
#pragma unroll
                for (int e = 0; e < 16; ++e) stage_f32[(c0 + e) * 128 + f_local] = __uint_as_float(v[e]);
            }
        }
        tc_fence_before();
    }

    if (split > 1) {
        // all partial tiles are in shared memory: sum them in slice order, each CTA finishing 1/split of the tokens
        cluster_sync_all();
        const uint32_t rank = cluster_ctarank();
        const bool ok = (*abort_flag == 0);
        for (int idx = threadIdx.x; idx < BN * 128; idx += 192) {
            const int row = idx >> 7, f_local = idx & 127;
            if ((row % split) != (int)rank) continue;
            const int t = tok0 + row;
            const long feature = (long)ft * 128 + f_local;
            if (t >= p.M || feature >= p.N) continue;
            float acc = 0.f;
            for (int r = 0; r < split; ++r) acc += ld_dsmem_f32(sbase + (uint32_t)idx * 4u, (uint32_t)r);
            if (ok) {
                acc = epilogue_value(p, acc, feature);
                if (p.out_f32) reinterpret_cast<float *>(p.Y)[(long)t * p.ldy + feature] = acc;
                else reinterpret_cast<__half *>(p.Y)[(long)t * p.ldy + feature] = __float2half_rn(acc);
            }
        }
        cluster_sync_all();
    }
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

template <int BN, int STAGES>
esp_status_t launch_gather(const GemmParams &p, int f_tiles, int t_tiles, int split, cudaStream_t stream) {
    using L = GatherSmem<BN, STAGES>;
    auto kern = spgemm_gather_kernel<BN, STAGES>;
    ESP_CUDA_OK(ensure_dynamic_smem((const void *)kern, L::kTotal));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(f_tiles, t_tiles, split);
    cfg.blockDim = dim3(192);
    cfg.dynamicSmemBytes = L::kTotal;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = split;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    ESP_CUDA_OK(cudaLaunchKernelEx(&cfg, kern, p));
    return ESP_OK;
}


// --------------------------------------------------------------------------------------------------
// TMA kernel: large token counts (prefill), channel-major X.
// The X tile of a stage is 128 permuted channels x BN tokens.  Channel rows are fetched by the tensor
// memory unit four arbitrary rows at a time (tile::gather4, row indices = 4 consecutive entries of the
// permutation), 64 tokens (128 bytes) per row, landing 128-byte swizzled as an MN-major B operand: the
// permutation costs nothing beyond the loads themselves and no permuted copy of X exists anywhere.
// grid (feature tiles, token tiles, split_k), cluster (1,1,split_k), block 192:
//   warp 0  producer: lane 0 issues the weight-tile bulk copy, all lanes issue gather4 row loads
//   warp 1  lane 0 issues tcgen05.cp (metadata) + 4 sparse MMAs per stage
//   warps 2..5  epilogue
// --------------------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap *map, int x, int r0, int r1, int r2, int r3,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cta.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];" ::"r"(dst),
        "l"(map), "r"(x), "r"(r0), "r"(r1), "r"(r2), "r"(r3), "r"(bar)
        : "memory");
}

template <int BN>
struct TmaCfg {
    static constexpr int kXStage = 128 * BN * 2;
    static constexpr int kStage = kTileBytes + kXStage;
    static constexpr int kStages = (BN == 256) ? 2 : (BN == 128) ? 4 : 6;
    static constexpr int kBarOff = kStages * kStage;
    static constexpr int kTotal = kBarOff + 256 + 1024;
};

template <int BN>
__global__ void __launch_bounds__(192) spgemm_tma_kernel(const GemmParams p, const __grid_constant__ CUtensorMap xmap) {
    using L = TmaCfg<BN>;
    constexpr int STAGES = L::kStages;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar_base = sbase + L::kBarOff;
    auto full = [&](int s) { return bar_base + 8u * s; };
    auto empty = [&](int s) { return bar_base + 8u * (8 + s); };
    const uint32_t accum_bar = bar_base + 8u * 16;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + L::kBarOff + 8 * 17);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + L::kBarOff + 8 * 17 + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ft = blockIdx.x, tok0 = blockIdx.y * BN;
    const int split = (int)gridDim.z, slice = (int)blockIdx.z;
    const int kt_begin = slice * p.k_tiles_per_split;
    const int kt_end = min(p.k_tiles, kt_begin + p.k_tiles_per_split);
    const int nk = max(0, kt_end - kt_begin);
    constexpr uint32_t kTmemCols = tmem_cols_for(BN);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
        mbar_init(accum_bar, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 0) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        const uint8_t *w_src = p.packed + ((long)ft * p.k_tiles + kt_begin) * kTileBytes;
        bool alive = true;
        for (int it = 0; it < nk && alive; ++it) {
            const int s = it % STAGES;
            const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
            // this lane's permutation entries: rows 4*lane .. 4*lane+3 of the stage
            const int kpos = (kt_begin + it) * kTileK + lane * 4;
            int4 rows;
            if (kpos + 4 <= p.K && p.perm) {
                rows = __ldg(reinterpret_cast<const int4 *>(p.perm + kpos));
            } else {
                int r[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) r[e] = (kpos + e < p.K) ? (p.perm ? __ldg(p.perm + kpos + e) : kpos + e) : p.K;   // K = out of range: zero fill
                rows = make_int4(r[0], r[1], r[2], r[3]);
            }
            if (!mbar_wait(empty(s), ph ^ 1u, abort_flag)) { alive = false; }
            alive = __all_sync(0xFFFFFFFFu, alive);
            if (!alive) break;
            const uint32_t stage = sbase + s * L::kStage;
            if (lane == 0) {
                mbar_arrive_expect_tx(full(s), L::kStage);
                bulk_load(stage, w_src + (long)it * kTileBytes, kTileBytes, full(s));
            }
            __syncwarp();
#pragma unroll
            for (int tb = 0; tb < BN / 64; ++tb)
                tma_gather4(stage + kTileBytes + tb * 16384 + lane * 512, &xmap, tok0 + tb * 64, rows.x, rows.y, rows.z, rows.w, full(s));
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc_sparse_f16(128, BN, 1);
            for (int it = 0; it < nk; ++it) {
                const int s = it % STAGES;
                const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
                if (!mbar_wait(full(s), ph, abort_flag)) break;
                tc_fence_after();
                const uint32_t wa = sbase + s * L::kStage;
                const uint32_t xa = wa + kTileBytes;
                const uint32_t e_col = BN + (it & 1) * 4;
                tc_copy_128x128b(tmem + e_col, smem_desc(wa + kTileValBytes, 0, 128, kLayoutNone));
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t col = e_col + j;
                    const uint64_t ad = smem_desc(wa + j * 32, 16, 1024, kLayoutSw128);
                    const uint64_t bd = smem_desc(xa + j * 4096, 16384, 1024, kLayoutSw128);
                    tc_mma_sparse_f16(tmem, ad, bd, tmem + (col & ~1u), idesc | (col & 1u), (it > 0 || j > 0) ? 1u : 0u);
                }
                tc_commit(empty(s));
            }
            tc_commit(accum_bar);
        }
    } else {
        const int quarter = warp & 3;
        const int f_local = quarter * 32 + lane;
        const long feature = (long)ft * 128 + f_local;
        const bool ok = (nk == 0 || mbar_wait(accum_bar, 0, abort_flag));
        tc_fence_after();
        float *stage_f32 = reinterpret_cast<float *>(smem);
        const float bias_f = epilogue_bias(p, feature);
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 16) {
            uint32_t v[16];
            if (nk > 0) {
                tmem_load_16(tmem + ((uint32_t)(quarter * 32) << 16) + c0, v);
            } else {
#pragma unroll
                for (int e = 0; e < 16; ++e) v[e] = 0;
            }
            if (split == 1) {
                if (ok && feature < p.N) {
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        const int t = tok0 + c0 + e;
                        if (t < p.M) {
                            const float y = epilogue_apply(__uint_as_float(v[e]), bias_f, p.act);
                            if (p.out_f32) reinterpret_cast<float *>(p.Y)[(long)t * p.ldy + feature] = y;
                            else reinterpret_cast<__half *>(p.Y)[(long)t * p.ldy + feature] = __float2half_rn(y);
                        }
                    }
                }
            } else {
#pragma unroll
                for (int e = 0; e < 16; ++e) stage_f32[(c0 + e) * 128 + f_local] = __uint_as_float(v[e]);
            }
        }
        tc_fence_before();
    }

    if (split > 1) {
        cluster_sync_all();
        const uint32_t rank = cluster_ctarank();
        const bool ok = (*abort_flag == 0);
        for (int idx = threadIdx.x; idx < BN * 128; idx += 192) {
            const int row = idx >> 7, f_local = idx & 127;
            if ((row % split) != (int)rank) continue;
            const int t = tok0 + row;
            const long feature = (long)ft * 128 + f_local;
            if (t >= p.M || feature >= p.N) continue;
            float acc = 0.f;
            for (int r = 0; r < split; ++r) acc += ld_dsmem_f32(sbase + (uint32_t)idx * 4u, (uint32_t)r);
            if (ok) {
                acc = epilogue_value(p, acc, feature);
                if (p.out_f32) reinterpret_cast<float *>(p.Y)[(long)t * p.ldy + feature] = acc;
                else reinterpret_cast<__half *>(p.Y)[(long)t * p.ldy + feature] = __float2half_rn(acc);
            }
        }
        cluster_sync_all();
    }
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}


// --------------------------------------------------------------------------------------------------
// Streaming kernel: every token count, channel-major X.  A stage holds one compressed weight tile
// (18 KB, one bulk asynchronous copy) and the matching X tile: 128 permuted channel rows x BN tokens,
// fetched by four producer warps with 16-byte asynchronous copies (cp.async) that complete on the stage's
// mbarrier, landing swizzled as an MN-major B operand.  (Measured on B200: the tensor memory unit retires one
// four-row gather per ~60 clocks, 8.5 B/clk per SM, far below what the MMA consumes; plain asynchronous row
// copies are not bound by that.)
//
// Decode shapes (BN = 16 / 32 / 64) are bound by the HBM stream of weight tiles, so everything is arranged
// to get those copies in flight at once: the first weight tiles are issued by thread 0 right after it has
// initialised the barriers, before tensor memory is allocated and before the CTA's first barrier; the grid is
// sized so that all CTAs are resident together (no second wave); and with `static_weights` the kernel is
// launched as a programmatic dependent of the preceding kernel on the stream, so this prologue -- which
// touches only the weights and the permutation -- overlaps the predecessor's tail, and only the X rows
// wait for it (griddepcontrol.wait).
//
// K is split across the CTAs of a cluster.  Partial tiles are reduced by pushing: the tile's tokens are dealt to the
// cluster ranks in contiguous runs of `cnt4` rows (a multiple of 4, so that four accumulator columns always go to one
// owner as one 16-byte store); every CTA sends its fp32 partial rows straight into the owner's shared memory with
// asynchronous remote stores (slot = sender's rank) that complete on the owner's mbarrier; the owner adds the slots in
// rank order -- deterministic, no global scratch.  Token tiles up to 32 keep a receive area of their own and push as
// soon as their accumulator is complete; wider tiles, whose partials would crowd out the ring, receive into the ring
// itself once a cluster barrier has told every CTA that all MMAs of the cluster are done reading it.  (Measured on
// 4096 x 4096 at 128 tokens: owners pulling the rows from their peers with remote loads took 8.4 us for 64 KB per CTA;
// element-wise pushes for slice counts that are not a power of two took 10 us at 32 tokens.  The 16-byte pushes take
// about 1.5 us.)
// grid (feature tiles, token tiles, split_k), cluster (1,1,split_k), block 192:
//   warp 0 lane 0  weight-tile producer        warp 1  tensor-memory allocation; lane 0: tcgen05.cp + sparse MMAs
//   warps 2..5     X row producers, then epilogue (one quarter of the accumulator lanes each)
// --------------------------------------------------------------------------------------------------
template <int BN>
struct StreamCfg {
    static constexpr int kRowBytes = BN >= 64 ? 128 : BN * 2;        // one channel row inside a block of <= 64 tokens
    static constexpr int kTokBlocks = BN >= 64 ? BN / 64 : 1;
    static constexpr int kChunks = kRowBytes / 16;                   // 16-byte pieces per row and block
    static constexpr int kBlockBytes = 128 * kRowBytes;              // 128 channel rows of one token block
    static constexpr int kXStage = 128 * BN * 2;
    static constexpr int kStage = kTileBytes + kXStage;              // a multiple of 1024
    static constexpr uint32_t kLayout = BN >= 64 ? 2u : BN == 32 ? 4u : 6u;   // 128 / 64 / 32-byte swizzle
    static constexpr int kSwzShift = BN >= 64 ? 0 : BN == 32 ? 1 : 2;         // row bits that feed the XOR
    static constexpr bool kEarlyPush = BN <= 32;                     // partial rows pushed into a receive area of their own
    // 16-byte asynchronous row copies deliver 25 / 44 / 60 GB/s per SM from 128 / 256 / 512 threads: wide X tiles get
    // sixteen producer warps, narrow ones (little X per weight tile) four
    static constexpr int kProd = BN >= 64 ? 512 : 128;
    static constexpr int kThreads = 64 + kProd;
};
// Rows of a token tile that one cluster rank owns in the K-slice reduction (a multiple of 4; rank o owns rows
// [o * cnt4, (o + 1) * cnt4) of the tile, clipped to the tile).
__host__ __device__ inline int stream_cnt4(int bn, int split) { return (((bn + split - 1) / split) + 3) & ~3; }
// Pushed partials at one owner: [sender][group of 4 rows][128 features][4 rows] fp32.
inline size_t stream_push_bytes(int bn, int split) { return split > 1 ? (size_t)split * stream_cnt4(bn, split) * 512 : 0; }
inline size_t stream_recv_bytes(int bn, int split) { return bn <= 32 ? stream_push_bytes(bn, split) : 0; }   // beside the ring
inline size_t stream_smem_bytes(int bn, int stages, int split) {
    size_t ring = (size_t)stages * (kTileBytes + 256 * bn);
    if (bn > 32 && ring < stream_push_bytes(bn, split)) ring = stream_push_bytes(bn, split);   // wide tiles receive into the ring
    return ring + stream_recv_bytes(bn, split) + kPermRing * 512 + 512 + 1024;
}

template <int BN>
__global__ void __launch_bounds__(StreamCfg<BN>::kThreads) spgemm_stream_kernel(const GemmGroup grp, const int stages) {
    using L = StreamCfg<BN>;
    // this CTA's problem: selected with constant indices so that the parameters stay in registers
    GemmParams p = grp.p[0];
    int ft_first = 0;
#pragma unroll
    for (int i = 1; i < ESP_MAX_GROUP; ++i)
        if (i < grp.count && (int)blockIdx.x >= grp.ft_start[i]) { p = grp.p[i]; ft_first = grp.ft_start[i]; }
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const int split = (int)gridDim.z, slice = (int)blockIdx.z;
    // layout (matches stream_smem_bytes): ring of stages | pushed partials (narrow tiles) | permutation ring | barriers;
    // wide tiles receive the pushed partials at the start of the ring
    const int cnt4 = stream_cnt4(BN, split);
    const uint32_t push_bytes = split > 1 ? (uint32_t)(split * cnt4 * 512) : 0u;
    uint32_t ring_bytes = (uint32_t)stages * L::kStage;
    if (!L::kEarlyPush && ring_bytes < push_bytes) ring_bytes = push_bytes;
    const uint32_t recv_off = L::kEarlyPush ? ring_bytes : 0u;
    const uint32_t perm_off = ring_bytes + (L::kEarlyPush ? push_bytes : 0u);
    const uint32_t bar_off = perm_off + kPermRing * 512;
    const uint32_t bar_base = sbase + bar_off;
    auto full = [&](int s) { return bar_base + 8u * s; };
    auto empty = [&](int s) { return bar_base + 8u * (kMaxStages + s); };
    const uint32_t accum_bar = bar_base + 8u * (2 * kMaxStages);
    const uint32_t recv_bar = bar_base + 8u * (2 * kMaxStages + 1);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + bar_off + 8 * (2 * kMaxStages + 2));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + bar_off + 8 * (2 * kMaxStages + 2) + 4);
    int *perm_s = reinterpret_cast<int *>(smem + perm_off);          // [kPermRing][128]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ft = (int)blockIdx.x - ft_first, tok0 = blockIdx.y * BN;
    const int kt_begin = slice * p.k_tiles_per_split;
    const int kt_end = min(p.k_tiles, kt_begin + p.k_tiles_per_split);
    const int nk = max(0, kt_end - kt_begin);
    constexpr uint32_t kTmemCols = tmem_cols_for(BN);
    const uint8_t *w_src = p.packed + ((long)ft * p.k_tiles + kt_begin) * kTileBytes;
    const int prefetch = min(stages, nk);
    // Image form (a workspace): a tiling pass has written the permuted, swizzled X operand of every (64-token
    // block -- BN < 64: token tile --, channel step) into the workspace; a stage's X is then one bulk copy per token
    // block instead of 16-byte row copies from every producer thread (which are limited to one 32-byte sector per clock
    // per SM).
    const bool imaged = p.ximg != nullptr;
    const uint32_t rank = (split > 1) ? cluster_ctarank() : 0u;
    const int owned = max(0, min(cnt4, BN - (int)rank * cnt4));      // rows of this tile that this CTA finishes

    if (threadIdx.x == 0) {
        // gather form: every X producer thread + the weight-tile copy; image form: the weight-tile copy + the X image copies
        for (int s = 0; s < stages; ++s) { mbar_init(full(s), imaged ? 2u : (uint32_t)L::kProd + 1u); mbar_init(empty(s), 1); }
        mbar_init(accum_bar, 1);
        mbar_init(recv_bar, 1);
        *abort_flag = 0;
        fence_barrier_init();
        // every sender delivers 128 features x (rows of this tile that this CTA owns) floats
        if (split > 1) mbar_arrive_expect_tx(recv_bar, (uint32_t)(split * owned * 512));
    }
    if (warp == 0) {
        // The weight stream starts now: nothing below is needed for these copies.  Lane s owns stage s (bulk copies
        // issued by one thread complete one after the other, copies of different threads overlap).
        __syncwarp();
        if (lane < prefetch) {
            mbar_arrive_expect_tx(full(lane), kTileBytes);
            bulk_load(sbase + lane * L::kStage, w_src + (long)lane * kTileBytes, kTileBytes, full(lane));
        }
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    if (warp >= 2 && warp < 6 && !imaged) {
        // permutation entries of the first stages, all loads in flight together (the X addresses depend on them)
        const int g = threadIdx.x - 64;
        int pre[kPermRing];
#pragma unroll
        for (int it = 0; it < kPermRing; ++it) {
            const int kpos = (kt_begin + it) * kTileK + g;
            pre[it] = (it < nk && kpos < p.K) ? (p.perm ? __ldg(p.perm + kpos) : kpos) : -1;
        }
#pragma unroll
        for (int it = 0; it < kPermRing; ++it) perm_s[it * 128 + g] = pre[it];
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (split > 1) cluster_arrive();       // every CTA of the cluster is running and has its barriers set up
    grid_launch_dependents();

    // Cluster barrier protocol (split > 1): phase A = "every CTA has its barriers set up" (arrived above); wide tiles add
    // phase B = "every CTA's MMAs are done with the ring".  Every thread takes part in every phase, whatever happened to it.
    if (warp == 0) {
        // (later weight tiles are issued by the X producer warps below, right after they have seen the stage's `empty`)
        if (split > 1) {
            cluster_wait();
            if (!L::kEarlyPush) { cluster_arrive(); cluster_wait(); }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc_sparse_f16(128, BN, 1);
            for (int it = 0; it < nk; ++it) {
                const int s = it % stages;
                const uint32_t ph = (uint32_t)(it / stages) & 1u;
                if (!mbar_wait(full(s), ph, abort_flag)) break;
                fence_async_smem();          // rows written by cp.async (generic proxy) -> read by the MMA (async proxy)
                tc_fence_after();
                const uint32_t wa = sbase + s * L::kStage;
                const uint32_t xa = wa + kTileBytes;
                const uint32_t e_col = BN + (it & 1) * 4;
                tc_copy_128x128b(tmem + e_col, smem_desc(wa + kTileValBytes, 0, 128, kLayoutNone));
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t col = e_col + j;
                    const uint64_t ad = smem_desc(wa + j * 32, 16, 1024, kLayoutSw128);
                    const uint64_t bd = (BN >= 64) ? smem_desc(xa + j * 4096, L::kBlockBytes, 1024, kLayoutSw128)
                                                   : smem_desc(xa + j * 32 * L::kRowBytes, 8 * L::kRowBytes, 8 * L::kRowBytes, L::kLayout);
                    tc_mma_sparse_f16(tmem, ad, bd, tmem + (col & ~1u), idesc | (col & 1u), (it > 0 || j > 0) ? 1u : 0u);
                }
                tc_commit(empty(s));
            }
            tc_commit(accum_bar);
        }
        __syncwarp();
        if (split > 1) {
            cluster_wait();
            if (!L::kEarlyPush) { cluster_arrive(); cluster_wait(); }
        }
    } else {
        // ---- X producers: thread g copies the 16-byte pieces e = g, g + 128, ... of the stage's 128 rows
        const int g = threadIdx.x - 64;
        constexpr int kPieces = 128 * L::kChunks;                     // per token block
        constexpr int kPerThread = (kPieces + L::kProd - 1) / L::kProd;
        const uint16_t *xb = reinterpret_cast<const uint16_t *>(p.X);
        const bool ring_refill = nk > kPermRing;                      // long K-slices: keep the ring kPermRing stages ahead
        bool alive = true;
        int refill = -1;
        if (imaged) {
            // ---- image form: lane 0 of producer warp q feeds the ring slots s = q, q + 4, ...: the weight tile (beyond the
            // start-up ones) and the X images of the tile's 64-token blocks, each a bulk copy.  A slot always has the same
            // feeder, which therefore waits for the slot's `empty` phases one after the other (a thread that ran two phases
            // ahead of a barrier would see the older phase of the same parity as complete).  The images are written by
            // the tiling pass this kernel is a programmatic dependent of; a raised flag also says that everything before
            // that pass is complete (its CTAs waited for it), so Y may be written once any flag has been seen.
            const int q = warp - 2;
            const int h0 = (int)blockIdx.y * L::kTokBlocks;                              // first 64-token block of this tile
            const int n_blocks = BN < 64 ? 1 : min(L::kTokBlocks, 2 * ((p.M + 127) / 128) - h0);   // (64-token blocks: the pass writes whole 128-token pairs)
            if (q < 4 && lane == 0) {
                for (int it = 0; it < nk; ++it) {
                    const int s = it % stages;
                    if ((s & 3) != q) continue;
                    const uint32_t ph = (uint32_t)(it / stages) & 1u;
                    const int kt = kt_begin + it;
                    bool seen = true;
                    for (int tb = 0; tb < n_blocks; ++tb) seen = seen && xflag_wait(p.xflags + (size_t)(h0 + tb) * p.k_tiles + kt, abort_flag);
                    if (!seen) { alive = false; break; }
                    asm volatile("fence.proxy.async;" ::: "memory");   // the pass's generic-proxy writes, just acquired -> this thread's bulk read
                    if (!mbar_wait(empty(s), ph ^ 1u, abort_flag)) { alive = false; break; }
                    if (it >= prefetch) {
                        mbar_arrive_expect_tx(full(s), kTileBytes);
                        bulk_load(sbase + s * L::kStage, w_src + (long)it * kTileBytes, kTileBytes, full(s));
                    }
                    mbar_arrive_expect_tx(full(s), (uint32_t)(n_blocks * L::kBlockBytes));
                    for (int tb = 0; tb < n_blocks; ++tb)
                        bulk_load(sbase + s * L::kStage + kTileBytes + tb * L::kBlockBytes,
                                  p.ximg + ((size_t)(h0 + tb) * p.k_tiles + kt) * L::kBlockBytes, L::kBlockBytes, full(s));
                }
            }
            if (nk == 0) grid_dependency_wait();                      // (no flag to see: wait for the stream order itself)
        } else {
        grid_dependency_wait();                                       // X may come from the preceding kernel
        for (int it = 0; it < nk; ++it) {
            const int s = it % stages;
            const uint32_t ph = (uint32_t)(it / stages) & 1u;
            const int *pr = perm_s + (it % kPermRing) * 128;
            if (ring_refill && it > 0 && g < 128) perm_s[((it - 1) % kPermRing) * 128 + g] = refill;   // entries of stage it-1+kPermRing
            int ch[kPerThread];
#pragma unroll
            for (int i = 0; i < kPerThread; ++i) {
                const int e = g + L::kProd * i;
                ch[i] = (e < kPieces) ? pr[e / L::kChunks] : -1;
            }
            if (ring_refill) {
                asm volatile("bar.sync 1, %0;" ::"n"(L::kProd) : "memory");   // everyone has read this stage's entries
                const int kpos = (kt_begin + it + kPermRing) * kTileK + g;
                refill = (g < 128 && it + kPermRing < nk && kpos < p.K) ? (p.perm ? __ldg(p.perm + kpos) : kpos) : -1;
            }
            // (a thread whose wait gave up keeps looping without copying: the named barrier above needs every producer)
            if (alive && !mbar_wait(empty(s), ph ^ 1u, abort_flag)) alive = false;
            if (!alive) continue;
            const uint32_t xs = sbase + s * L::kStage + kTileBytes;
#pragma unroll
            for (int tb = 0; tb < L::kTokBlocks; ++tb) {
#pragma unroll
                for (int i = 0; i < kPerThread; ++i) {
                    const int e = g + L::kProd * i;
                    if (e < kPieces) {
                        const int r = e / L::kChunks, cc = e % L::kChunks;
                        const int t = tok0 + tb * 64 + cc * 8;
                        const int valid = min(8, max(0, p.M - t));
                        const bool in = ch[i] >= 0 && valid > 0;
                        const uint16_t *src = in ? xb + (long)ch[i] * p.ldx + t : xb;
                        const int cs = cc ^ ((r >> L::kSwzShift) & (L::kChunks - 1));
                        cp_async_16(xs + tb * L::kBlockBytes + r * L::kRowBytes + (cs << 4), src, in ? valid * 2 : 0);
                    }
                }
            }
            cp_async_arrive_noinc(full(s));
            // Weight tile of this stage (beyond the first `stages`, which were issued at start-up): lane 0 of producer warp
            // s % 4.  Copies issued by one thread do not overlap and lanes spinning in one warp hold each other up, so
            // the issuing duty rotates over the four producer warps, which have just seen `empty` anyway.
            if (it >= prefetch && lane == 0 && (warp - 2) == (s & 3)) {   // (one of the first four producer warps)
                mbar_arrive_expect_tx(full(s), kTileBytes);
                bulk_load(sbase + s * L::kStage, w_src + (long)it * kTileBytes, kTileBytes, full(s));
            }
        }
        }
        // ---- epilogue.  One K-slice: the first four producer warps (one quarter of the accumulator lanes each) stage
        // the tile in shared memory and store it.  Several: every producer warp pushes partial rows to their owners
        // (warp w reads lane quarter w % 4 and the 16-column pieces (w - 2) / 4, + kProd / 128, ...), then finishes the rows
        // this CTA owns.
        const int quarter = warp & 3;
        const int f_local = quarter * 32 + lane;
        if (imaged) {
            // Almost every producer thread has been idle since the start: one of them polls the accumulator barrier, the
            // others sleep on a named barrier (hundreds of lanes polling through the main loop slow the CTA's other
            // barrier operations down).
            if (warp == (L::kProd > 128 ? 6 : 5) && lane == 31 && nk > 0) (void)mbar_wait(accum_bar, 0, abort_flag);
            __syncwarp();
            asm volatile("bar.sync 1, %0;" ::"n"(L::kProd) : "memory");
        }
        if (split == 1) {
            if (warp < 6) {
            const bool ok = __all_sync(0xFFFFFFFFu, alive && (nk == 0 || mbar_wait(accum_bar, 0, abort_flag)));   // warp-uniform
            tc_fence_after();
            // accumulators -> shared memory [token][128 features] in the output type -> 16-byte stores
            const int esize = p.out_f32 ? 4 : 2;
            const float bias_f = epilogue_bias(p, (long)ft * 128 + f_local);
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 16) {
                uint32_t v[16];
                if (nk > 0 && ok) {
                    tmem_load_16(tmem + ((uint32_t)(quarter * 32) << 16) + c0, v);
                } else {
#pragma unroll
                    for (int e = 0; e < 16; ++e) v[e] = 0;
                }
                if (p.out_f32) {
#pragma unroll
                    for (int e = 0; e < 16; ++e)
                        reinterpret_cast<float *>(smem)[(c0 + e) * 128 + f_local] = epilogue_apply(__uint_as_float(v[e]), bias_f, p.act);
                } else {
#pragma unroll
                    for (int e = 0; e < 16; ++e)
                        reinterpret_cast<__half *>(smem)[(c0 + e) * 128 + f_local] =
                            __float2half_rn(epilogue_apply(__uint_as_float(v[e]), bias_f, p.act));
                }
            }
            tc_fence_before();
            asm volatile("bar.sync 2, 128;" ::: "memory");
            const int row_bytes = 128 * esize;
            const int chunks_per_row = row_bytes / 16;
            const int f_valid = min(128, p.N - ft * 128);
            const bool vec_ok = (((long)p.ldy * esize) % 16 == 0) && ((reinterpret_cast<uintptr_t>(p.Y) & 15) == 0);
            uint8_t *yb = reinterpret_cast<uint8_t *>(p.Y);
            for (int idx = g; idx < BN * chunks_per_row; idx += 128) {
                const int row = idx / chunks_per_row, c = idx % chunks_per_row;
                const int t = tok0 + row;
                if (!ok || t >= p.M) continue;
                const int f0 = c * (16 / esize);
                uint8_t *dst = yb + ((long)t * p.ldy + (long)ft * 128 + f0) * esize;
                const uint8_t *srcp = smem + (size_t)row * row_bytes + c * 16;
                if (vec_ok && f0 + 16 / esize <= f_valid) {
                    *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(srcp);
                } else {
                    for (int e = 0; e < 16 / esize; ++e)
                        if (f0 + e < f_valid) {
                            if (p.out_f32) reinterpret_cast<float *>(dst)[e] = reinterpret_cast<const float *>(srcp)[e];
                            else reinterpret_cast<uint16_t *>(dst)[e] = reinterpret_cast<const uint16_t *>(srcp)[e];
                        }
                }
            }
            }
        } else {
            constexpr int kPushGroups = L::kProd / 128;                  // 16-column pieces pushed side by side
            const int cgrp = (warp - 2) >> 2;
            const bool ok = __all_sync(0xFFFFFFFFu, alive && (nk == 0 || mbar_wait(accum_bar, 0, abort_flag)));   // warp-uniform
            tc_fence_after();
            cluster_wait();                                          // phase A: every CTA of the cluster has its barriers
            if (!L::kEarlyPush) { cluster_arrive(); cluster_wait(); }   // phase B: every CTA's MMAs are done with the ring
            const int groups = cnt4 >> 2;                            // 4-row groups per owner
#pragma unroll 1
            for (int c0 = cgrp * 16; c0 < BN; c0 += 16 * kPushGroups) {
                uint32_t v[16];
                if (nk > 0 && ok) {
                    tmem_load_16(tmem + ((uint32_t)(quarter * 32) << 16) + c0, v);
                } else {
#pragma unroll
                    for (int e = 0; e < 16; ++e) v[e] = 0;
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int row = c0 + 4 * j;
                    const int owner = row / cnt4, rg = (row - owner * cnt4) >> 2;
                    const uint32_t local = sbase + recv_off + (uint32_t)((((int)rank * groups + rg) * 128 + f_local) * 16);
                    st_async_v4(map_to_rank(local, (uint32_t)owner), v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3],
                                map_to_rank(recv_bar, (uint32_t)owner));
                }
            }
            tc_fence_before();
            const bool got = mbar_wait_cluster(recv_bar, 0, abort_flag);
            const bool fine = got && (*abort_flag == 0);
            const float4 *recv = reinterpret_cast<const float4 *>(smem + recv_off);
            const int f_valid = min(128, p.N - ft * 128);
            for (int q = g; q < (owned >> 2) * 128; q += L::kProd) {
                const int rg = q >> 7, f = q & 127;
                float a[4] = {0.f, 0.f, 0.f, 0.f};
                for (int r = 0; r < split; ++r) {                    // slice order: deterministic
                    const float4 part = recv[(r * groups + rg) * 128 + f];
                    a[0] += part.x; a[1] += part.y; a[2] += part.z; a[3] += part.w;
                }
                if (!fine || f >= f_valid) continue;
                const float bias_f = epilogue_bias(p, (long)ft * 128 + f);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int t = tok0 + (int)rank * cnt4 + rg * 4 + e;
                    if (t >= p.M) continue;
                    const long o = (long)t * p.ldy + (long)ft * 128 + f;
                    const float y = epilogue_apply(a[e], bias_f, p.act);
                    if (p.out_f32) reinterpret_cast<float *>(p.Y)[o] = y;
                    else reinterpret_cast<__half *>(p.Y)[o] = __float2half_rn(y);
                }
            }
        }
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

// X [K, ldx] channel-major -> the streaming kernel's X stages for 16- and 32-token tiles: image (t, kt) holds channels
// perm[kt*128 .. +127] of tokens BN t .. BN t + BN - 1 as [128 rows][2 BN bytes] with the 16-byte chunk c of row r stored
// at the chunk the kernel's B descriptor expects (64-byte swizzle for 32 tokens: c ^ ((r >> 1) & 3); 32-byte swizzle for 16:
// c ^ ((r >> 2) & 1)).  Rows beyond K and tokens beyond M are zero.  grid (token tiles, k_tiles), block 256: thread -> row
// and chunk(s).  Flags as in xtile_kernel: lowered before the dependent launch may start, raised when the image is complete.
template <int BN>
__global__ void __launch_bounds__(256) xtile_narrow_kernel(const uint16_t *__restrict__ X, long ldx, int M, int K,
                                                           const int32_t *__restrict__ perm, uint8_t *__restrict__ img,
                                                           uint32_t *__restrict__ flags, int k_tiles) {
    using L = StreamCfg<BN>;
    static_assert(BN == 16 || BN == 32, "narrow tiles");
    constexpr int kPer = L::kChunks / 2;                                  // chunks per thread: 2 threads per row
    const int t = blockIdx.x, kt = blockIdx.y;
    uint8_t *dst = img + ((size_t)t * k_tiles + kt) * L::kBlockBytes;
    uint32_t *flag = flags + (size_t)t * k_tiles + kt;
    const int r = threadIdx.x >> 1, c0 = (threadIdx.x & 1) * kPer;
    const int kpos = kt * kTileK + r;
    const int ch = kpos < K ? (perm ? __ldg(perm + kpos) : kpos) : -1;
    grid_dependency_wait();                  // X may be the preceding kernel's output; the images may still be read by it
    if (threadIdx.x == 0) {
        asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(flag), "r"(0u) : "memory");
        __threadfence();
    }
    __syncthreads();
    grid_launch_dependents();
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        const int cc = c0 + i, tok = t * BN + cc * 8;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (ch >= 0 && tok < M) {
            const uint16_t *src = X + (long)ch * ldx + tok;
            if (tok + 8 <= M) {
                v = __ldg(reinterpret_cast<const uint4 *>(src));
            } else {
                uint16_t e[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) e[j] = (tok + j < M) ? __ldg(src + j) : (uint16_t)0;
                v = make_uint4(e[0] | ((uint32_t)e[1] << 16), e[2] | ((uint32_t)e[3] << 16), e[4] | ((uint32_t)e[5] << 16),
                               e[6] | ((uint32_t)e[7] << 16));
            }
        }
        const int cs = cc ^ ((r >> L::kSwzShift) & (L::kChunks - 1));
        *reinterpret_cast<uint4 *>(dst + r * L::kRowBytes + (cs << 4)) = v;
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(flag), "r"(1u) : "memory");
}
inline size_t xtile_narrow_image_bytes(int M, int K, int bn) { return (size_t)((M + bn - 1) / bn) * ((K + kTileK - 1) / kTileK) * 256 * bn; }
inline size_t xtile_narrow_bytes(int M, int K, int bn) {    // images | one flag word per image
    return xtile_narrow_image_bytes(M, K, bn) + align_up((size_t)((M + bn - 1) / bn) * ((K + kTileK - 1) / kTileK) * 4, 256);
}
template <int BN>
esp_status_t launch_xtile_narrow(const GemmParams &p, uint8_t *img, uint32_t *flags, bool dependent, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((p.M + BN - 1) / BN, p.k_tiles, 1);
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    ESP_CUDA_OK(cudaLaunchKernelEx(&cfg, xtile_narrow_kernel<BN>, reinterpret_cast<const uint16_t *>(p.X), p.ldx, p.M, p.K, p.perm, img,
                                   flags, p.k_tiles));
    return ESP_OK;
}

template <int BN>
esp_status_t launch_stream(const GemmParams &p, int f_tiles, int t_tiles, int split, int stages, bool dependent,
                           cudaStream_t stream) {
    auto kern = spgemm_stream_kernel<BN>;
    const size_t smem = stream_smem_bytes(BN, stages, split);
    ESP_CUDA_OK(ensure_dynamic_smem((const void *)kern, (int)smem));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(f_tiles, t_tiles, split);
    cfg.blockDim = dim3(StreamCfg<BN>::kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = split;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 2 : 1;
    GemmGroup grp;
    grp.count = 1;
    for (int i = 0; i <= ESP_MAX_GROUP; ++i) grp.ft_start[i] = i == 0 ? 0 : f_tiles;
    for (int i = 0; i < ESP_MAX_GROUP; ++i) grp.p[i] = p;
    ESP_CUDA_OK(cudaLaunchKernelEx(&cfg, kern, grp, stages));
    return ESP_OK;
}

// The same launch for a group of problems (feature tiles concatenated along grid.x).
template <int BN>
esp_status_t launch_stream_group(const GemmGroup &grp, int t_tiles, int split, int stages, bool dependent, cudaStream_t stream) {
    auto kern = spgemm_stream_kernel<BN>;
    const size_t smem = stream_smem_bytes(BN, stages, split);
    ESP_CUDA_OK(ensure_dynamic_smem((const void *)kern, (int)smem));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grp.ft_start[grp.count], t_tiles, split);
    cfg.blockDim = dim3(StreamCfg<BN>::kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = split;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 2 : 1;
    ESP_CUDA_OK(cudaLaunchKernelEx(&cfg, kern, grp, stages));
    return ESP_OK;
}

// Clusters of `split` CTAs of the streaming kernel that can be resident at once on this device.
template <int BN>
int stream_cluster_capacity(int split, int stages) {
    auto kern = spgemm_stream_kernel<BN>;
    const size_t smem = stream_smem_bytes(BN, stages, split);
    if (ensure_dynamic_smem((const void *)kern, (int)smem) != cudaSuccess) return 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(1, 1, split);
    cfg.blockDim = dim3(StreamCfg<BN>::kThreads);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = split;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
    // The occupancy calculator answers with one CTA per SM for these kernels whatever their size (it cannot know how much
    // tensor memory a CTA will allocate); CTAs do share an SM when shared memory, threads and tensor-memory columns
    // allow.  So its answer is taken as the packing of clusters onto GPCs at the calculator's CTAs per SM and scaled.
    int api_per_sm = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&api_per_sm, kern, StreamCfg<BN>::kThreads, smem) != cudaSuccess || api_per_sm < 1) {
        cudaGetLastError();
        api_per_sm = 1;
    }
    int dev = 0, smem_per_sm = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev);
    int per_sm = (int)((size_t)smem_per_sm / (smem + 1024));
    per_sm = per_sm < 2048 / StreamCfg<BN>::kThreads ? per_sm : 2048 / StreamCfg<BN>::kThreads;
    per_sm = per_sm < 512 / (int)tmem_cols_for(BN) ? per_sm : 512 / (int)tmem_cols_for(BN);
    if (per_sm < api_per_sm) per_sm = api_per_sm;
    const int clusters = (int)((long)n * per_sm / api_per_sm);
    if (log_plans())
        fprintf(stderr, "esparse occupancy tile=%d split=%d stages=%d smem=%zu: calculator clusters=%d at %d CTAs/SM, taken %d at %d CTAs/SM\n", BN,
                split, stages, smem, n, api_per_sm, clusters, per_sm);
    return clusters;
}

#include "spgemm_pair.cuh"
#include "spgemm_persist.cuh"

// Tensor map over channel-major X: dim 0 = tokens (contiguous), dim 1 = channels (ldx apart); box = 64 tokens
// x 1 row (the row-gather form loads four such rows per instruction), 128-byte swizzle, zero fill outside.
inline esp_status_t make_x_tensor_map(const __half *X, int M, int K, long ldx, CUtensorMap *map) {
    EncodeTiledFn encode = nullptr;
    esp_status_t est = tensor_map_encoder(&encode);
    if (est != ESP_OK) return est;
    cuuint64_t dims[2] = {(cuuint64_t)M, (cuuint64_t)K};
    cuuint64_t strides[1] = {(cuuint64_t)ldx * 2};
    cuuint32_t box[2] = {64, 1};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<__half *>(X), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? ESP_OK : ESP_ERR_CUDA;
}

template <int BN>
esp_status_t launch_tma(const GemmParams &p, int f_tiles, int t_tiles, int split, cudaStream_t stream) {
    using L = TmaCfg<BN>;
    CUtensorMap map;
    esp_status_t st = make_x_tensor_map(p.X, p.M, p.K, p.ldx, &map);
    if (st != ESP_OK) return st;
    auto kern = spgemm_tma_kernel<BN>;
    ESP_CUDA_OK(ensure_dynamic_smem((const void *)kern, L::kTotal));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(f_tiles, t_tiles, split);
    cfg.blockDim = dim3(192);
    cfg.dynamicSmemBytes = L::kTotal;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = split;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    ESP_CUDA_OK(cudaLaunchKernelEx(&cfg, kern, p, map));
    return ESP_OK;
}

// [M, K] token-major -> [K, ldt] channel-major (a transposed, not permuted, copy; ldt >= M).
__global__ void __launch_bounds__(256) transpose_x_kernel(const uint16_t *__restrict__ X, int M, int K, long ldx,
                                                          uint16_t *__restrict__ Xt, long ldt) {
    __shared__ uint16_t tile[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int k0 = blockIdx.x * 32, m0 = blockIdx.y * 32;
    // As a programmatic dependent (static_weights): the GEMM behind this copy may start at once and prefetch its weights;
    // X, and the workspace the preceding GEMM may still read, are touched only after that kernel is done.
    grid_launch_dependents();
    grid_dependency_wait();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty + 8 * i, k = k0 + tx;
        tile[ty + 8 * i][tx] = (m < M && k < K) ? X[(long)m * ldx + k] : (uint16_t)0;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int k = k0 + ty + 8 * i, m = m0 + tx;
        if (k < K && m < ldt) Xt[(long)k * ldt + m] = tile[tx][ty + 8 * i];
    }
}

static cudaError_t launch_transpose(const uint16_t *X, int M, int K, long ldx, uint16_t *Xt, long ldt, bool dependent,
                                    cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ceil_div(K, 32), ceil_div(ldt, 32), 1);
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, transpose_x_kernel, X, M, K, ldx, Xt, ldt);
}

// A wait nobody ends: one thread polls a barrier that receives no arrival, gives up after a short limit, records
// ESP_ERR_TIMEOUT and returns -- the same path every bounded wait of the GEMM kernels takes when it runs out.
__global__ void wait_timeout_selftest_kernel() {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        fence_barrier_init();
        bool done = false;
        for (uint32_t i = 0; i < (1u << 12) && !done; ++i) {
            done = mbar_try_wait(smem_u32(&bar), 0);
            if (!done) __nanosleep(64);
        }
        if (!done) {
            abort_flag = 1;
            atomicExch(&g_device_status, (int)ESP_ERR_TIMEOUT);
        }
    }
}

}  // namespace

esp_status_t launch_wait_timeout_selftest(cudaStream_t stream) {
    wait_timeout_selftest_kernel<<<1, 32, 0, stream>>>();
    ESP_CUDA_OK(cudaGetLastError());
    return ESP_OK;
}

static long transposed_ld(int M) { return (long)((M + 15) / 16 * 16); }

// Workspace = [transposed copy of token-major X] [X images of the tiled pair kernel].  The first part is required for
// every kernel but the gather kernel when X is token-major; the second lets large M use the tiled pair kernel.
static size_t transpose_bytes(int M, int K, const esp_gemm_opts &o) {
    if (o.x_layout == ESP_X_CHANNEL_MAJOR || o.force_kernel == ESP_KERNEL_GATHER) return 0;
    return align_up((size_t)K * (size_t)transposed_ld(M) * 2, 256);
}
static size_t ximg_bytes(int M, int K, int tn) {
    switch (tn) {
        case 128: return xtile_bytes<128>(M, K);
        case 192: return xtile_bytes<192>(M, K);
        case 224: return xtile_bytes<224>(M, K);
        default: return xtile_bytes<240>(M, K);
    }
}
size_t gemm_workspace_min_bytes(int M, int K, const esp_gemm_opts &o) { return transpose_bytes(M, K, o); }
size_t gemm_workspace_bytes(int M, int K, const esp_gemm_opts &o) {
    size_t n = transpose_bytes(M, K, o);
    const bool pair_possible = o.force_kernel == ESP_KERNEL_PAIR_TILED || o.force_kernel == ESP_KERNEL_STREAM_IMAGES || (o.force_kernel == ESP_KERNEL_AUTO && M > 16) || o.force_kernel == ESP_KERNEL_QUAD_TILED ||
                               o.force_kernel == ESP_KERNEL_PAIR_PERSIST || o.force_kernel == ESP_KERNEL_QUAD_MULTICAST;
    if (pair_possible) {
        size_t img = 0;
        for (int tn : {128, 192, 224, 240}) img = std::max(img, ximg_bytes(M, K, tn));
        n += img;
    }
    return n;
}

// Resident capacity (in CTAs) of the streaming kernel for one configuration, cached per process.
static int stream_capacity_ctas(int bn, int split, int stages) {
    static std::mutex mu;
    static std::map<long, int> cache;
    int dev = 0;
    cudaGetDevice(&dev);
    const long key = (((long)dev * 512 + bn) * 16 + split) * 16 + stages;
    std::lock_guard<std::mutex> lock(mu);
    auto it = cache.find(key);
    if (it != cache.end()) return it->second;
    int clusters = 0;
    switch (bn) {
        case 16: clusters = stream_cluster_capacity<16>(split, stages); break;
        case 32: clusters = stream_cluster_capacity<32>(split, stages); break;
        case 64: clusters = stream_cluster_capacity<64>(split, stages); break;
        case 128: clusters = stream_cluster_capacity<128>(split, stages); break;
        case 256: clusters = stream_cluster_capacity<256>(split, stages); break;
        default: break;
    }
    cache[key] = clusters * split;
    return clusters * split;
}

static esp_status_t plan_gemm_uncached(int M, int N, int K, const esp_gemm_opts &o, size_t workspace_bytes, GemmPlan *plan) {
    const bool have_workspace = workspace_bytes >= transpose_bytes(M, K, o) && (workspace_bytes > 0 || o.x_layout == ESP_X_CHANNEL_MAJOR);
    DeviceInfo di;
    esp_status_t st = device_info(&di);
    if (st != ESP_OK) return st;
    GemmPlan g;
    const int k_tiles = ceil_div(K, kTileK);
    const int f_tiles = ceil_div(N, kTileFeat);
    const bool channel_major_available = (o.x_layout == ESP_X_CHANNEL_MAJOR) || have_workspace;
    int bn = o.token_tile;
    g.kernel = ESP_KERNEL_GATHER;
    if (o.force_kernel != ESP_KERNEL_GATHER && channel_major_available) {
        if (o.force_kernel == ESP_KERNEL_TMA) g.kernel = ESP_KERNEL_TMA;
        else if (o.force_kernel == ESP_KERNEL_PAIR) g.kernel = ESP_KERNEL_PAIR;
        else if (o.force_kernel == ESP_KERNEL_PAIR_TILED) g.kernel = ESP_KERNEL_PAIR_TILED;
        else if (o.force_kernel == ESP_KERNEL_QUAD_TILED) g.kernel = ESP_KERNEL_QUAD_TILED;
        else if (o.force_kernel == ESP_KERNEL_PAIR_PERSIST) g.kernel = ESP_KERNEL_PAIR_PERSIST;
        else if (o.force_kernel == ESP_KERNEL_QUAD_MULTICAST) g.kernel = ESP_KERNEL_QUAD_MULTICAST;
        else if (o.force_kernel == ESP_KERNEL_STREAM) g.kernel = ESP_KERNEL_STREAM;
        else if (o.force_kernel == ESP_KERNEL_STREAM_IMAGES) g.kernel = ESP_KERNEL_STREAM_IMAGES;
        else {
            // The pair kernel takes every M > 64; a requested token tile or slice count that only the streaming kernel has
            // (tiles below 128 tokens, more than four slices, slices of a 256-token tile) goes there.
            const bool stream_only = (bn != 0 && bn < 128) || o.split_k > 4 || (bn == 256 && o.split_k > 1);
            // Up to 256 tokens the pair kernel pays only where the weight gives it twenty pairs or more per K-slice (its
            // set-up and drain cost about 10 us; measured at 128 tokens: 11008 x 4096 26.5 against the streaming kernel's
            // 28.5 us, but 4096 x 4096 20.3 against 14.6).
            const long pairs128 = (long)ceil_div(f_tiles, 4) * ceil_div(M, 128);
            const bool pair = !stream_only && (M > 256 || (M > 64 && pairs128 >= 20));
            g.kernel = pair ? ESP_KERNEL_PAIR : ESP_KERNEL_STREAM;
            // 17..256 tokens on a large weight: the streaming kernel fed from X images.  Its row gather limits the
            // streaming kernel once the X tile is a good part of a stage; the images cost one more (small) launch, which pays
            // from about 40 M weight elements (measured, gather form -> image form: 36864 x 9216 at 32 / 64 tokens
            // 78 -> 67 / 118 -> 68 us; 9216 x 9216 at 64 / 128 tokens 41 -> 28 / 47 -> 37 us; but 9216 x 9216 at 32 tokens
            // 22.5 -> 28.4, 4096 x 4096 at 128 tokens 15.0 -> 17.1).  It also replaces the pair kernel's gather form where that
            // would run K-slices at 129..256 tokens (9216 x 9216 at 256 tokens: 95 -> 55 us).
            const long weight = (long)N * K;
            const bool images_room = workspace_bytes >= transpose_bytes(M, K, o) + ximg_bytes(M, K, 128);
            if (images_room && bn == 0 && o.split_k <= 8 && M > 16 && M <= 256) {
                const long per_wave = di.sm_count / 2 > 0 ? di.sm_count / 2 : 1;
                if (!pair) {
                    const bool pays = M <= 32 ? weight >= 200000000L : M <= 64 ? (f_tiles >= 64 || weight >= 64000000L) : M <= 128 ? weight >= 40000000L : weight >= 16000000L;
                    // (up to 32 tokens: 32-token images -- 36864 x 9216 at 32 tokens 67.5 -> 64.3 us, 9216 x 36864 76 -> 70)
                    if (pays) { g.kernel = ESP_KERNEL_STREAM_IMAGES; bn = M <= 32 ? 32 : (M > 128 && weight >= 64000000L) ? 128 : 64; }
                } else if (M > 128 && o.split_k == 0 && weight >= 80000000L && per_wave / pairs128 >= 2) {
                    g.kernel = ESP_KERNEL_STREAM_IMAGES;
                    bn = 128;
                }
            }
        }
    }
    const bool wide_only = g.kernel == ESP_KERNEL_QUAD_TILED || g.kernel == ESP_KERNEL_PAIR_PERSIST ||
                           g.kernel == ESP_KERNEL_QUAD_MULTICAST;                                      // no 128-token form
    if (g.kernel == ESP_KERNEL_PAIR || g.kernel == ESP_KERNEL_PAIR_TILED || wide_only) {
        const long f_pairs = ceil_div(f_tiles, 4), per_wave = di.sm_count / 2 > 0 ? di.sm_count / 2 : 1;
        if (bn == 0) {
            // cost ~ waves of clusters x time of one wave, in clocks: a channel step costs its MMAs (8 x TN/2 clocks) and its
            // 36 KB of weights + X tile (64-token blocks: 16 KB for TN = 128, else 32 KB) at the ~70 B/clk an SM pulls from
            // L2.  Wide tiles win once the grid fills the machine; a grid of less than one wave runs faster on narrow ones.
            double best = -1.0;
            for (int tn : {240, 224, 192, 128}) {
                if (tn == 128 && wide_only) continue;
                const long clusters = f_pairs * ceil_div(M, tn);
                const double mma = 4.0 * tn, copy = (36864.0 + (tn > 128 ? 32768.0 : 16384.0)) / 70.0;
                // per wave: the channel steps (both terms show in the measured step time), an epilogue that grows with the
                // tile (about ten steps' worth at 240 tokens) and a fixed set-up.  Waves: a grid of up to two waves runs as
                // whole waves (equal tiles end together); over many waves the clusters drift apart and the last, partial wave
                // costs less and less of a whole one (measured at 4.4 waves: already closer to the fractional count).
                const double w = (double)clusters / (double)per_wave, whole = (double)ceil_div(clusters, per_wave);
                const double waves = w <= 2.0 ? whole : w + (whole - w) * (2.0 / w);
                const double cost = waves * (0.5 * (mma + copy) * k_tiles + 40.0 * tn + 2000.0);
                if (best < 0.0 || cost < best) { best = cost; bn = tn; }
            }
        }
        if (bn != 128 && bn != 192 && bn != 224 && bn != 240 && bn != 256) return ESP_ERR_INVALID_ARG;
        // K-slices (128-token tiles only: the pushed partial rows of all slices must fit the ring): as many as fill one
        // wave of pairs, each slice keeping at least four channel steps
        int split = 1;
        if (bn == 128) {
            const long pairs = f_pairs * ceil_div(M, 128);
            // (beyond 256 tokens two slices at most: three ran far slower than two -- 4096 x 4096 at 384 tokens 46 against
            // 30 us, 4096 x 11008 at 384 tokens 70 against 50 -- and four no faster)
            split = o.split_k > 0 ? o.split_k : (int)std::min<long>(M > 256 ? 2 : 4, std::max<long>(1, per_wave / pairs));
            while (split > 1 && (k_tiles / split < 4 || (long)ceil_div(k_tiles, split) * (split - 1) >= k_tiles)) --split;
        } else if (o.split_k > 1) {
            return ESP_ERR_INVALID_ARG;
        }
        // the tiled form needs room for the X images behind the transposed copy; without it the gather form runs.  Up to
        // 128 tokens the gather form is taken anyway: one launch instead of two, and X is small.
        const bool room = bn != 256 && workspace_bytes >= transpose_bytes(M, K, o) + ximg_bytes(M, K, bn);
        if ((g.kernel == ESP_KERNEL_PAIR_TILED || wide_only) && !room) return ESP_ERR_WORKSPACE;
        if (wide_only && (bn == 128 || bn == 256)) return ESP_ERR_INVALID_ARG;
        // (129..256 tokens in one K-slice: the tiled form too -- 11008 x 4096 at 256 tokens 37.4 -> 33.4 us, 13824 x 5120
        // 47.2 -> 41.6; with K-slices the gather form stays ahead there)
        if (g.kernel == ESP_KERNEL_PAIR && o.force_kernel == ESP_KERNEL_AUTO && room && (M > 256 || (M > 128 && split == 1)))
            g.kernel = ESP_KERNEL_PAIR_TILED;
        g.token_tile = bn;
        g.split_k = split;
        g.stages = 0;
        *plan = g;
        return ESP_OK;
    }
    // (33..64 tokens: two 32-token tiles beat one of 64 unless the weight has many feature tiles -- the second pass over the
    // weight comes from L2, and the narrow tile keeps more CTAs per SM; 5120 x 5120: 13.1 against 15.7 us)
    if (bn == 0) bn = M <= 16 ? 16 : M <= 32 ? 32 : M <= 64 ? (f_tiles <= 64 && g.kernel == ESP_KERNEL_STREAM ? 32 : 64) : M <= 128 ? 128 : 256;
    // (a weight of a few tiles: narrow token tiles, so that the tiles x K-slices come to about one CTA per SM; re-reading
    // so small a weight per token tile costs nothing.  512 x 512 at 128 tokens: 3.1 us with 16-token tiles against 8.4)
    if (o.token_tile == 0 && g.kernel == ESP_KERNEL_STREAM && M > 16 && (long)f_tiles * k_tiles <= 64) {
        for (int narrow : {16, 32, 64}) {
            if (narrow >= bn) break;
            if ((long)f_tiles * ceil_div(M, narrow) * std::min(k_tiles, 8) <= 2L * di.sm_count) { bn = narrow; break; }
        }
    }
    if (g.kernel == ESP_KERNEL_TMA && bn < 64) bn = 64;
    if (g.kernel == ESP_KERNEL_STREAM_IMAGES && workspace_bytes < transpose_bytes(M, K, o) + ximg_bytes(M, K, 128)) return ESP_ERR_WORKSPACE;
    if (bn != 16 && bn != 32 && bn != 64 && bn != 128 && bn != 256) return ESP_ERR_INVALID_ARG;
    g.token_tile = bn;
    g.stages = 4;
    const int t_tiles = ceil_div(M, bn);
    const long tiles = (long)f_tiles * t_tiles;
    auto no_empty_slice = [&](int split) { return (long)ceil_div(k_tiles, split) * (split - 1) < k_tiles; };
    if (g.kernel == ESP_KERNEL_STREAM || g.kernel == ESP_KERNEL_STREAM_IMAGES) {
        // Pick K-slices and CTAs per SM so that, if possible, the whole grid is resident at once and each CTA
        // has a short chain of tiles: cost ~ waves x (tiles per CTA + fixed start-up and reduction time).
        const size_t per_stage = (size_t)kTileBytes + 256 * (size_t)bn;
        double best_cost = 1e30;
        int best_split = 0, best_stages = 0;
        int wanted = o.split_k > k_tiles ? k_tiles : o.split_k;      // a requested split steps down to one without empty slices
        while (wanted > 1 && !no_empty_slice(wanted)) --wanted;
        for (int split = 1; split <= 8 && split <= k_tiles; ++split) {
            if (wanted != 0 && split != wanted) continue;
            if (!no_empty_slice(split)) continue;
            const int kts = ceil_div(k_tiles, split);
            const size_t fixed = stream_recv_bytes(bn, split) + kPermRing * 512 + 512 + 1024;
            int last_stages = -1;
            for (int r = 1; r <= 4; ++r) {
                const size_t budget = (size_t)di.max_smem_optin / r - (r > 1 ? 1024 : 0);
                if (budget < fixed + 2 * per_stage) break;
                int stages = (int)((budget - fixed) / per_stage);
                if (o.pipeline_stages > 0) {                              // a requested ring depth: this one only, or what fits
                    if (r > 1) break;
                    if (stages > o.pipeline_stages) stages = o.pipeline_stages;
                }
                if (stages > kMaxStages) stages = kMaxStages;
                if (stages > kts) stages = kts < 2 ? 2 : kts;
                if (stages == last_stages) continue;
                last_stages = stages;
                const int cap = stream_capacity_ctas(bn, split, stages);
                if (cap <= 0) continue;
                const long ctas = tiles * split;
                const long waves = (ctas + cap - 1) / cap;
                // per CTA: kts steps + set-up, reduction and epilogue, which grow with the token tile (measured: a 256-token
                // tile in one wave of 32 steps beats three waves of 8)
                // wide token tiles are bound by their X gather, which CTAs sharing an SM share: a step costs as many
                // times more as CTAs of one wave sit on an SM
                const long in_wave = ctas < cap ? ctas : cap;
                const double share = (bn >= 64 && g.kernel == ESP_KERNEL_STREAM) ? (double)((in_wave + di.sm_count - 1) / di.sm_count) : 1.0;
                double cost = (double)waves * (kts * share + 2.0 + bn / 32.0) + (split > 1 ? 0.25 + 0.05 * split : 0.0) + 0.01 * r;
                // with static_weights consecutive launches overlap on an SM: prefer leaving room for a CTA of the next one
                // (not when every CTA has an SM of its own anyway: a deeper ring is then free, measured 16.0 -> 12.6 us on
                // 4096 x 4096 at 64 tokens)
                if (o.static_weights && o.pipeline_stages == 0 && ctas > di.sm_count &&
                    2 * (stream_smem_bytes(bn, stages, split) + 1024) > (size_t)di.max_smem_optin)
                    cost += 3.0;
                if (log_plans())
                    fprintf(stderr, "esparse plan M=%d N=%d K=%d tile=%d: split=%d stages=%d capacity=%d ctas=%ld waves=%ld cost=%.2f\n", M, N, K,
                            bn, split, stages, cap, ctas, waves, cost);
                if (cost < best_cost) { best_cost = cost; best_split = split; best_stages = stages; }
            }
        }
        if (best_split == 0) return ESP_ERR_UNSUPPORTED;
        g.split_k = best_split;
        g.stages = best_stages;
        *plan = g;
        return ESP_OK;
    }
    int split = o.split_k;
    if (split == 0) {
        split = 1;
        while (split < 8 && tiles * split < di.sm_count && k_tiles / (split * 2) >= 4) split *= 2;
    }
    if (split > k_tiles) split = k_tiles;
    if (split < 1) split = 1;
    while (split > 1 && !no_empty_slice(split)) --split;
    g.split_k = split;
    *plan = g;
    return ESP_OK;
}


// The plan of a call is a pure function of its sizes, its options, the workspace size and the device: the last few are
// remembered per thread, so that a layer's repeated calls do not walk the candidates again.
esp_status_t plan_gemm(int M, int N, int K, const esp_gemm_opts &o, size_t workspace_bytes, GemmPlan *plan) {
    struct Key { int dev, M, N, K, x_layout, split_k, force_kernel, token_tile, static_weights, pipeline_stages; size_t ws; };
    struct Entry { Key key; GemmPlan plan; };
    thread_local Entry cache[32];
    thread_local int n = 0, next = 0;
    int dev = 0;
    cudaGetDevice(&dev);
    const Key key{dev, M, N, K, o.x_layout, o.split_k, o.force_kernel, o.token_tile, o.static_weights, o.pipeline_stages, workspace_bytes};
    if (!log_plans())
        for (int i = 0; i < n; ++i) {
            const Key &k = cache[i].key;
            if (k.dev == key.dev && k.M == key.M && k.N == key.N && k.K == key.K && k.x_layout == key.x_layout && k.split_k == key.split_k &&
                k.force_kernel == key.force_kernel && k.token_tile == key.token_tile && k.static_weights == key.static_weights &&
                k.pipeline_stages == key.pipeline_stages && k.ws == key.ws) {
                *plan = cache[i].plan;
                return ESP_OK;
            }
        }
    const esp_status_t st = plan_gemm_uncached(M, N, K, o, workspace_bytes, plan);
    if (st == ESP_OK) {
        cache[next] = Entry{key, *plan};
        next = (next + 1) % 32;
        if (n < 32) ++n;
    }
    return st;
}

// ---- the optional companion library: the one kernel form whose weight loads use cluster multicast is built into a shared
// object of its own (libesparse_mc.so, from spgemm_mcast.cu), looked for once beside this library.
namespace {
struct Companion {
    int (*launch)(const void *, size_t, int, int, void *) = nullptr;
    int (*status)(int *) = nullptr;
};
const Companion *companion() {
    static Companion c;
    static std::once_flag once;
    static bool ok = false;
    std::call_once(once, [] {
        Dl_info info;
        if (!dladdr(reinterpret_cast<const void *>(&plan_gemm), &info) || !info.dli_fname) return;
        std::string path(info.dli_fname);
        const size_t slash = path.rfind('/');
        path = (slash == std::string::npos ? std::string() : path.substr(0, slash + 1)) + "libesparse_mc.so";
        void *h = dlopen(path.c_str(), RTLD_NOW | RTLD_LOCAL);
        if (!h) return;
        c.launch = reinterpret_cast<int (*)(const void *, size_t, int, int, void *)>(dlsym(h, "esp_mc_launch_pair"));
        c.status = reinterpret_cast<int (*)(int *)>(dlsym(h, "esp_mc_device_status"));
        ok = c.launch != nullptr && c.status != nullptr;
    });
    return ok ? &c : nullptr;
}

// The tiling pass over X (channel-major, or token-major when x_tm is given) and then the planned form of the tiled pair
// kernel as its programmatic dependent (it waits on the image flags, not on the grid).
template <int TN>
esp_status_t launch_tiled_form(GemmParams &p, const GemmPlan &plan, const uint16_t *x_tm, long ldx_tm, uint8_t *img, bool dependent,
                               cudaStream_t stream, int sm_count) {
    uint32_t *flags = reinterpret_cast<uint32_t *>(img + xtile_image_bytes<TN>(p.M, p.K));
    p.ximg = img;
    p.xflags = flags;
    esp_status_t st = x_tm ? launch_xtile_tm<TN>(p, x_tm, ldx_tm, img, flags, dependent, stream) : launch_xtile<TN>(p, img, flags, dependent, stream);
    if (st != ESP_OK) return st;
    if constexpr (TN == 128) {
        if (plan.kernel != ESP_KERNEL_PAIR_TILED) return ESP_ERR_INVALID_ARG;
        return launch_pair<2, 128, true>(p, true, stream, plan.split_k);
    } else {
        switch (plan.kernel) {
            case ESP_KERNEL_QUAD_TILED: return launch_quad<TN>(p, true, stream);
            case ESP_KERNEL_PAIR_PERSIST: return launch_pair_persist<TN>(p, true, stream, sm_count);
            case ESP_KERNEL_QUAD_MULTICAST: {
                const Companion *c = companion();
                return c ? (esp_status_t)c->launch(&p, sizeof(p), TN, 1, stream) : ESP_ERR_UNSUPPORTED;
            }
            default: return launch_pair<2, TN, true>(p, true, stream);
        }
    }
}
}  // namespace

bool companion_available() { return companion() != nullptr; }
esp_status_t companion_device_status(int *out) {
    *out = 0;
    const Companion *c = companion();
    return c ? (esp_status_t)c->status(out) : ESP_OK;
}

esp_status_t launch_spgemm(const __half *X, int M, int K, long ldx, const void *packed, const int32_t *perm, int N,
                           void *Y, long ldy, const esp_gemm_opts &o, const GemmPlan &plan, void *workspace,
                           size_t workspace_bytes, cudaStream_t stream) {
    GemmParams p;
    p.X = X; p.ldx = ldx; p.M = M; p.K = K; p.N = N;
    p.x_channel_major = (o.x_layout == ESP_X_CHANNEL_MAJOR) ? 1 : 0;
    p.packed = (const uint8_t *)packed;
    p.perm = perm;
    p.Y = Y; p.ldy = ldy;
    p.out_f32 = (o.out_dtype == ESP_OUT_F32) ? 1 : 0;
    p.bias = reinterpret_cast<const __half *>(o.bias);
    p.act = o.activation;
    p.k_tiles = ceil_div(K, kTileK);
    p.k_tiles_per_split = ceil_div(p.k_tiles, plan.split_k);
    p.ximg = nullptr;
    p.xflags = nullptr;
    p.raster_panel = 0;
    const int f_tiles = ceil_div(N, kTileFeat), t_tiles = ceil_div(M, plan.token_tile);
    const bool quad_form = plan.kernel == ESP_KERNEL_QUAD_TILED || plan.kernel == ESP_KERNEL_QUAD_MULTICAST;
    if (plan.kernel == ESP_KERNEL_PAIR || plan.kernel == ESP_KERNEL_PAIR_TILED || quad_form || plan.kernel == ESP_KERNEL_PAIR_PERSIST) {
        // Panels pay once a row of clusters (every feature pair on one token tile) is a good part of a wave: about eight
        // token tiles per panel (six where the weight has few feature pairs), the panels evened out over the token tiles.
        // Measured (M = 8192 unless noted): 22016 x 8192 1.79 -> 1.96 PFLOP/s; 36864 x 9216 at 4096 tokens 1.56 -> 1.94;
        // 8192 x 22016 1.76 -> 1.83; 8192 x 8192 (its 75 MB of weights stay in L2 anyway) unchanged.
        const int f_pairs = ceil_div(f_tiles, 4);
        if (f_pairs >= 12 && t_tiles >= 4) {
            const int want = f_pairs >= 20 ? 8 : 6;
            const int panels = std::max(1, (t_tiles + want / 2) / want);
            p.raster_panel = ceil_div(t_tiles, panels);
            if (quad_form) p.raster_panel = (p.raster_panel + 1) / 2;   // counted in pairs of token tiles there
        }
    }
    if (plan.kernel != ESP_KERNEL_GATHER) {
        if (!p.x_channel_major && plan.kernel != ESP_KERNEL_PAIR_TILED &&
            !(plan.kernel == ESP_KERNEL_STREAM_IMAGES && plan.token_tile >= 64)) {
            // token-major input: transposed (not permuted) copy into the caller's workspace
            const long ldt = transposed_ld(M);
            if (!workspace || workspace_bytes < (size_t)K * ldt * 2) return ESP_ERR_WORKSPACE;
            ESP_CUDA_OK(launch_transpose(reinterpret_cast<const uint16_t *>(X), M, K, ldx, reinterpret_cast<uint16_t *>(workspace),
                                         ldt, o.static_weights != 0, stream));
            p.X = reinterpret_cast<const __half *>(workspace);
            p.ldx = ldt;
            p.x_channel_major = 1;
        }
        const bool dependent = o.static_weights != 0;
        if (plan.kernel == ESP_KERNEL_PAIR_TILED || quad_form || plan.kernel == ESP_KERNEL_PAIR_PERSIST) {
            if (plan.kernel == ESP_KERNEL_QUAD_MULTICAST && !companion_available()) return ESP_ERR_UNSUPPORTED;
            DeviceInfo di;
            if (device_info(&di) != ESP_OK) return ESP_ERR_CUDA;
            const size_t off = transpose_bytes(M, K, o);
            if (!workspace || workspace_bytes < off + ximg_bytes(M, K, plan.token_tile)) return ESP_ERR_WORKSPACE;
            uint8_t *img = reinterpret_cast<uint8_t *>(workspace) + off;
            const uint16_t *x_tm = p.x_channel_major ? nullptr : reinterpret_cast<const uint16_t *>(X);   // token-major: one transposing pass
            switch (plan.token_tile) {
                case 128: return launch_tiled_form<128>(p, plan, x_tm, ldx, img, dependent, stream, di.sm_count);
                case 192: return launch_tiled_form<192>(p, plan, x_tm, ldx, img, dependent, stream, di.sm_count);
                case 224: return launch_tiled_form<224>(p, plan, x_tm, ldx, img, dependent, stream, di.sm_count);
                case 240: return launch_tiled_form<240>(p, plan, x_tm, ldx, img, dependent, stream, di.sm_count);
                default: return ESP_ERR_INVALID_ARG;
            }
        }
        if (plan.kernel == ESP_KERNEL_PAIR) {
            switch (plan.token_tile) {
                case 128: return launch_pair<2, 128>(p, dependent, stream, plan.split_k);
                case 192: return launch_pair<2, 192>(p, dependent, stream);
                case 224: return launch_pair<2, 224>(p, dependent, stream);
                case 240: return launch_pair<2, 240>(p, dependent, stream);
                case 256: return launch_pair<1, 256>(p, dependent, stream);
                default: return ESP_ERR_INVALID_ARG;
            }
        }
        if (plan.kernel == ESP_KERNEL_STREAM_IMAGES) {
            // the tiling pass writes the images of 64-token blocks (the 128-token pair kernel's format); the streaming kernel
            // follows as its programmatic dependent and takes each image when its flag is up
            const size_t off = transpose_bytes(M, K, o);
            uint8_t *img = reinterpret_cast<uint8_t *>(workspace) + off;
            if (plan.token_tile < 64) {      // narrow tiles: images of their own format, from channel-major X (transposed above if need be)
                const int bn = plan.token_tile;
                if (!workspace || workspace_bytes < off + xtile_narrow_bytes(M, K, bn)) return ESP_ERR_WORKSPACE;
                uint32_t *flags_n = reinterpret_cast<uint32_t *>(img + xtile_narrow_image_bytes(M, K, bn));
                p.ximg = img;
                p.xflags = flags_n;
                if (bn == 32) {
                    const esp_status_t st_n = launch_xtile_narrow<32>(p, img, flags_n, dependent, stream);
                    return st_n != ESP_OK ? st_n : launch_stream<32>(p, f_tiles, t_tiles, plan.split_k, plan.stages, true, stream);
                }
                const esp_status_t st_n = launch_xtile_narrow<16>(p, img, flags_n, dependent, stream);
                return st_n != ESP_OK ? st_n : launch_stream<16>(p, f_tiles, t_tiles, plan.split_k, plan.stages, true, stream);
            }
            if (!workspace || workspace_bytes < off + ximg_bytes(M, K, 128)) return ESP_ERR_WORKSPACE;
            uint32_t *flags = reinterpret_cast<uint32_t *>(img + xtile_image_bytes<128>(M, K));
            p.ximg = img;
            p.xflags = flags;
            const esp_status_t st = p.x_channel_major ? launch_xtile<128>(p, img, flags, dependent, stream)
                                                      : launch_xtile_tm<128>(p, reinterpret_cast<const uint16_t *>(X), ldx, img, flags, dependent, stream);
            if (st != ESP_OK) return st;
            switch (plan.token_tile) {
                case 64: return launch_stream<64>(p, f_tiles, t_tiles, plan.split_k, plan.stages, true, stream);
                case 128: return launch_stream<128>(p, f_tiles, t_tiles, plan.split_k, plan.stages, true, stream);
                case 256: return launch_stream<256>(p, f_tiles, t_tiles, plan.split_k, plan.stages, true, stream);
                default: return ESP_ERR_INVALID_ARG;
            }
        }
        if (plan.kernel == ESP_KERNEL_STREAM) {
            switch (plan.token_tile) {
                case 16: return launch_stream<16>(p, f_tiles, t_tiles, plan.split_k, plan.stages, dependent, stream);
                case 32: return launch_stream<32>(p, f_tiles, t_tiles, plan.split_k, plan.stages, dependent, stream);
                case 64: return launch_stream<64>(p, f_tiles, t_tiles, plan.split_k, plan.stages, dependent, stream);
                case 128: return launch_stream<128>(p, f_tiles, t_tiles, plan.split_k, plan.stages, dependent, stream);
                case 256: return launch_stream<256>(p, f_tiles, t_tiles, plan.split_k, plan.stages, dependent, stream);
                default: return ESP_ERR_INVALID_ARG;
            }
        }
        switch (plan.token_tile) {
            case 64: return launch_tma<64>(p, f_tiles, t_tiles, plan.split_k, stream);
            case 128: return launch_tma<128>(p, f_tiles, t_tiles, plan.split_k, stream);
            case 256: return launch_tma<256>(p, f_tiles, t_tiles, plan.split_k, stream);
            default: return ESP_ERR_INVALID_ARG;
        }
    }
    switch (plan.token_tile) {
        case 16: return launch_gather<16, 6>(p, f_tiles, t_tiles, plan.split_k, stream);
        case 32: return launch_gather<32, 6>(p, f_tiles, t_tiles, plan.split_k, stream);
        case 64: return launch_gather<64, 5>(p, f_tiles, t_tiles, plan.split_k, stream);
        case 128: return launch_gather<128, 4>(p, f_tiles, t_tiles, plan.split_k, stream);
        case 256: return launch_gather<256, 2>(p, f_tiles, t_tiles, plan.split_k, stream);
        default: return ESP_ERR_INVALID_ARG;
    }
}

esp_status_t launch_spgemm_group(int count, const void *const *X, int M, int K, long ldx, const void *const *packed,
                                 const int32_t *const *perm, const int *N, void *const *Y, const long *ldy,
                                 const esp_gemm_opts &o, void *workspace, size_t workspace_bytes, cudaStream_t stream) {
    if (M > 256) return ESP_ERR_UNSUPPORTED;
    int f_total = 0;
    for (int i = 0; i < count; ++i) f_total += ceil_div(N[i], kTileFeat);
    const size_t tbytes = transpose_bytes(M, K, o);
    if (tbytes > 0 && (!workspace || workspace_bytes < tbytes * (size_t)count)) return ESP_ERR_UNSUPPORTED;
    GemmPlan plan;
    esp_gemm_opts og = o;                    // (a group shares one launch of the streaming kernel's gather form)
    if (og.force_kernel == ESP_KERNEL_AUTO && M <= 64) og.force_kernel = ESP_KERNEL_STREAM;
    esp_status_t st = plan_gemm(M, f_total * kTileFeat, K, og, workspace ? workspace_bytes : 0, &plan);
    if (st != ESP_OK) return st;
    if (plan.kernel != ESP_KERNEL_STREAM) return ESP_ERR_UNSUPPORTED;
    GemmGroup grp;
    grp.count = count;
    int ft = 0;
    for (int i = 0; i < ESP_MAX_GROUP; ++i) {
        const int j = i < count ? i : 0;
        GemmParams &p = grp.p[i];
        p.X = (const __half *)X[j]; p.ldx = ldx; p.M = M; p.K = K; p.N = N[j];
        p.x_channel_major = 1;
        p.packed = (const uint8_t *)packed[j];
        p.perm = perm ? perm[j] : nullptr;
        p.Y = Y[j]; p.ldy = ldy[j];
        p.out_f32 = (o.out_dtype == ESP_OUT_F32) ? 1 : 0;
        p.bias = nullptr;
        p.act = o.activation;
        p.k_tiles = ceil_div(K, kTileK);
        p.k_tiles_per_split = ceil_div(p.k_tiles, plan.split_k);
        p.ximg = nullptr;
        p.xflags = nullptr;
        p.raster_panel = 0;
        grp.ft_start[i] = ft;
        if (i < count) {
            if (o.x_layout != ESP_X_CHANNEL_MAJOR) {      // token-major: a transposed copy per distinct input, one after the other
                const long ldt = transposed_ld(M);
                int first = i;
                for (int e = 0; e < i; ++e)
                    if (X[e] == X[i]) { first = e; break; }                 // same-input linears (q, k, v) share the copy
                uint16_t *xt = reinterpret_cast<uint16_t *>(reinterpret_cast<uint8_t *>(workspace) + (size_t)first * tbytes);
                if (first == i)
                    ESP_CUDA_OK(launch_transpose(reinterpret_cast<const uint16_t *>(X[i]), M, K, ldx, xt, ldt, o.static_weights != 0, stream));
                p.X = reinterpret_cast<const __half *>(xt);
                p.ldx = ldt;
            }
            ft += ceil_div(N[i], kTileFeat);
        }
    }
    for (int i = count; i <= ESP_MAX_GROUP; ++i) grp.ft_start[i] = ft;
    const int t_tiles = ceil_div(M, plan.token_tile);
    const bool dependent = o.static_weights != 0;
    switch (plan.token_tile) {
        case 16: return launch_stream_group<16>(grp, t_tiles, plan.split_k, plan.stages, dependent, stream);
        case 32: return launch_stream_group<32>(grp, t_tiles, plan.split_k, plan.stages, dependent, stream);
        case 64: return launch_stream_group<64>(grp, t_tiles, plan.split_k, plan.stages, dependent, stream);
        case 128: return launch_stream_group<128>(grp, t_tiles, plan.split_k, plan.stages, dependent, stream);
        case 256: return launch_stream_group<256>(grp, t_tiles, plan.split_k, plan.stages, dependent, stream);
        default: return ESP_ERR_INVALID_ARG;
    }
}

}  // namespace esp
