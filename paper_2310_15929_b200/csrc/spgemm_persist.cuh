// Persistent form of the tiled pair kernel (included by spgemm_kernels.cu after spgemm_pair.cuh).
//
// The plain pair kernel runs one 512-feature x TN-token tile per CTA pair: every tile pays tensor-memory allocation and
// barrier set-up (1.5 us), the fill of an empty ring (2.6 us) and an epilogue (about 5 us) during which nothing is
// loaded, about 15 % of a tile's time at K = 8192.  Here one pair per two SMs stays resident and walks the tiles
// c = cluster, cluster + clusters, ... (same cluster -> tile map, so the pairs active at any moment cover the same
// neighbourhood of tiles as a wave of the plain kernel):
//   * the ring never drains: the copy issuers run ahead into the next tile while the epilogue of the current one
//     is still storing;
//   * the epilogue has warps of its own and writes the accumulators straight from registers to Y (a warp stores the 32
//     consecutive features of one token per instruction), so it needs no staging area in the ring;
//   * the MMA thread starts the next tile as soon as the epilogue warps of both CTAs have read the accumulators out
//     (barrier `acc_free`), not when their stores are done.
// Same MMAs in the same order as the plain kernel: results are identical bit for bit.
//
// grid (2 x resident pairs), cluster (2,1,1), block 864:
//   warp 0        idle
//   warp 1        tensor-memory allocation; lane 0 of the leader CTA issues every tcgen05.cp / MMA of the pair
//   warps 2..10   lane 0: copy issuer of ring slot (w - 2) / 3 for weight tile 0 / weight tile 1 / the X image
//   warps 11..26  epilogue: warp w reads lane quarter w % 4 (a hardware rule); the 2 x TN/16 column pieces of a tile go
//                 round the four warps of a quarter.  (Eight warps needed 7.7 us to read a tile's accumulators out, during
//                 which the MMA thread waits: two warps per scheduler do not hide the load -> convert -> store chain.)
constexpr int kPersistEpiWarps = 16;
constexpr int kPersistFirstEpi = 11;
constexpr int kPersistThreads = (kPersistFirstEpi + kPersistEpiWarps) * 32;

template <int TN>
__global__ void __launch_bounds__(kPersistThreads, 1) spgemm_pair_persist_kernel(const GemmParams p, const __grid_constant__ CUtensorMap wmap,
                                                                                 const __grid_constant__ CUtensorMap xmap, const int f_pairs,
                                                                                 const int t_tiles) {
    using L = PairCfg<2, TN>;
    constexpr int NA = 2;
    constexpr int STAGES = L::kStages;
    static_assert(STAGES == 3, "nine issuing warps: three copies for each of three ring slots");
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar_base = sbase + L::kBarOff;
    auto full = [&](int s) { return bar_base + 8u * s; };
    auto empty = [&](int s) { return bar_base + 8u * (8 + s); };
    const uint32_t accum_bar = bar_base + 8u * 24;
    const uint32_t accfree_bar = bar_base + 8u * 26;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + L::kBarOff + 8 * 25);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + L::kBarOff + 8 * 25 + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                              // 0 = leader of the pair
    const int cid = (int)blockIdx.x >> 1, n_clusters = (int)gridDim.x >> 1;
    const int n_tiles = f_pairs * t_tiles;
    const int nk = p.k_tiles;
    const int f_tiles = (p.N + 127) / 128;
    // linear tile index -> (feature pair, token tile): down panels of p.raster_panel token tiles, as in the plain kernel
    auto tile_of = [&](int c, int &pair_idx, int &ttile) {
        if (p.raster_panel > 1) {
            const int per_panel = p.raster_panel * f_pairs;
            const int panel = c / per_panel, r = c - panel * per_panel;
            const int height = min(p.raster_panel, t_tiles - panel * p.raster_panel);
            pair_idx = r / height;
            ttile = panel * p.raster_panel + (r - pair_idx * height);
        } else {
            ttile = c / f_pairs;
            pair_idx = c - ttile * f_pairs;
        }
    };
    const int my_tiles = cid < n_tiles ? (n_tiles - cid + n_clusters - 1) / n_clusters : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full(s), 6);           // the two X images + the four weight copies of the pair (absent tiles arrive without bytes)
            mbar_init(empty(s), 1);
        }
        mbar_init(accum_bar, 1);
        mbar_init(accfree_bar, 2 * kPersistEpiWarps);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc_pair(smem_u32(tmem_slot), L::kTmemCols);
    // Weight-tile areas start as zero values with legal metadata: a feature tile beyond N is never loaded, the MMA then
    // reads what the area holds (this, or an earlier tile's weights: either way legal operands for rows nobody stores).
    for (int s = 0; s < STAGES; ++s) {
        uint32_t *dst = reinterpret_cast<uint32_t *>(smem + s * L::kStage);
        for (int i = threadIdx.x; i < NA * kTileBytes / 4; i += kPersistThreads)
            dst[i] = ((i % (kTileBytes / 4)) < kTileValBytes / 4) ? 0u : 0x44444444u;
    }
    fence_async_smem();                      // generic-proxy writes above -> later bulk copies into, and MMA reads of, the same bytes
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    grid_launch_dependents();

    if (warp == 1) {
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = instr_desc_sparse_f16(256, TN, 1);
            uint64_t ad0[NA][4], bd0[4], md0[NA];
#pragma unroll
            for (int a = 0; a < NA; ++a) {
                md0[a] = smem_desc(sbase + a * kTileBytes + kTileValBytes, 0, 128, kLayoutNone);
#pragma unroll
                for (int j = 0; j < 4; ++j) ad0[a][j] = smem_desc(sbase + a * kTileBytes + j * 32, 16, 1024, kLayoutSw128);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) bd0[j] = smem_desc(sbase + L::kWStage + j * 4096, 16384, 1024, kLayoutSw128);
            constexpr int kUnroll = STAGES * 2;                           // ring slot and metadata buffer both periodic in the global step
            const int total = my_tiles * nk;
            bool alive = true;
            uint32_t seen = 0;
            int it = 0, tile_i = 0;
            for (int gs0 = 0; gs0 < total && alive; gs0 += kUnroll) {
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    const int gs = gs0 + u;
                    if (gs >= total) break;
                    // gs0 is a multiple of 2 * STAGES, so slot and barrier phase of step gs0 + u are compile-time constants
                    // (this thread's instruction stream is the kernel's critical path: no division per step)
                    const int s = u % STAGES;
                    const uint32_t ph = (uint32_t)(u / STAGES) & 1u;
                    uint32_t seen_a = 0, seen_b = 0;
                    const uint32_t nbar = full((u + 1) % STAGES), nph = (uint32_t)(((u + 1) % kUnroll) / STAGES) & 1u;
                    // a new tile overwrites the accumulators: the epilogue warps of both CTAs must have read the last one out
                    if (it == 0 && tile_i > 0 && !mbar_wait_cluster_1t(accfree_bar, (uint32_t)(tile_i - 1) & 1u, abort_flag)) { alive = false; break; }
                    if (!seen && !mbar_wait_1t(full(s), ph, abort_flag)) { alive = false; break; }
                    if (gs + 1 < total) seen_a = mbar_test(nbar, nph);
                    tc_fence_after();
                    const uint64_t soff = (uint64_t)((uint32_t)(s * L::kStage) >> 4);
#pragma unroll
                    for (int a = 0; a < NA; ++a) {
                        const uint32_t e_col = L::meta_col(a, u & 1);
                        tc_copy_128x128b_pair(tmem + e_col, md0[a] + soff);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint32_t col = e_col + j;
                            tc_mma_sparse_f16_pair(tmem + L::acc_col(a), ad0[a][j] + soff, bd0[j] + soff, tmem + (col & ~1u),
                                                   idesc | (col & 1u), (it > 0 || j > 0) ? 1u : 0u);
                        }
                        if (gs + 1 < total) seen_b |= mbar_test(nbar, nph);
                    }
                    tc_commit_pair(empty(s), (uint16_t)3);
                    seen = seen_a | seen_b;
                    if (++it == nk) {
                        tc_commit_pair(accum_bar, (uint16_t)3);           // this tile's accumulators are complete (both CTAs)
                        it = 0;
                        ++tile_i;
                    }
                }
            }
        }
    } else if (warp >= 2 && warp < 11) {
        // ---- copy issuers: ring slot s = (w - 2) / 3, copy kind = (w - 2) % 3 (weight tile 0, weight tile 1, X image); the
        // lane meets every phase of its slot's `empty` barrier: global steps gs = s, s + 3, ... across all of this pair's tiles
        if (lane == 0) {
            const int iw = warp - 2, s = iw / 3, kind = iw % 3;
            const bool is_x = kind == NA;
            const uint32_t bytes = is_x ? (uint32_t)L::kXStage : (uint32_t)kTileBytes;
            constexpr int kRowBytes = 1024;
            const CUtensorMap *map = is_x ? &xmap : &wmap;
            const int row_step = (int)bytes / kRowBytes;
            const uint32_t dst = sbase + s * L::kStage + (is_x ? L::kWStage : kind * kTileBytes);
            const uint32_t lead_full = map_to_rank(full(s), 0);
            int base = 0;                                                // global step of the tile's first channel step
            bool alive = true;
            for (int c = cid; c < n_tiles && alive; c += n_clusters, base += nk) {
                int pair_idx, ttile;
                tile_of(c, pair_idx, ttile);
                const int ft = pair_idx * (2 * NA) + 2 * kind + (int)rank;
                const bool have = is_x || ft < f_tiles;
                const uint32_t *xflag = p.xflags + (size_t)(ttile * 2 + rank) * nk;
                const int row0 = is_x ? (int)((ttile * 2 + rank) * nk) * row_step : ft * nk * row_step;
                for (int it = ((s - base) % STAGES + STAGES) % STAGES; it < nk; it += STAGES) {
                    const uint32_t ph = (uint32_t)((base + it) / STAGES) & 1u;
                    if (is_x) {
                        if (!xflag_wait(xflag + it, abort_flag)) { alive = false; break; }
                        asm volatile("fence.proxy.async;" ::: "memory");
                    }
                    if (!mbar_wait_1t(empty(s), ph ^ 1u, abort_flag)) { alive = false; break; }
                    if (have) {
                        mbar_arrive_expect_tx_cluster(lead_full, bytes);
                        tma_rows_pair(dst, map, row0 + it * row_step, lead_full);
                    } else {
                        mbar_arrive_remote(lead_full);
                    }
                }
            }
            if (!alive) *abort_flag = 1;
        }
    } else if (warp >= kPersistFirstEpi) {
        // ---- epilogue warps
        const int quarter = warp & 3;
        const int sub = (warp - kPersistFirstEpi) >> 2;                   // which of the quarter's four warps
        constexpr int kPieces = TN / 16;                                  // 16-column pieces per accumulator
        const uint32_t lead_free = map_to_rank(accfree_bar, 0);
        uint8_t *wbuf = smem + L::kBarOff + 512 + (size_t)(warp - kPersistFirstEpi) * 1024;   // this warp's transposition buffer (behind the barriers)
        const bool y_vec = (reinterpret_cast<uintptr_t>(p.Y) & 15) == 0;
        int tile_i = 0;
        bool ok = true;
        for (int c = cid; c < n_tiles; c += n_clusters, ++tile_i) {
            int pair_idx, ttile;
            tile_of(c, pair_idx, ttile);
            const int tok0 = ttile * TN;
            // one lane polls the accumulator barrier for all eight epilogue warps, which sleep on a named barrier meanwhile
            // (lanes that poll through a whole main loop slow the CTA's other barrier operations down)
            if (ok && nk > 0 && warp == kPersistFirstEpi && lane == 0 && !mbar_wait_cluster(accum_bar, (uint32_t)tile_i & 1u, abort_flag)) *abort_flag = 1;
            __syncwarp();
            asm volatile("bar.sync 1, %0;" ::"n"(kPersistEpiWarps * 32) : "memory");
            ok = ok && *abort_flag == 0;
            tc_fence_after();
            int last_k = -1;
            for (int k = sub; k < NA * kPieces; k += 4) last_k = k;
#pragma unroll 1
            for (int k = sub; k < NA * kPieces; k += 4) {
                const int a = k / kPieces, c0 = (k - a * kPieces) * 16;
                uint32_t v[16];
                if (nk > 0 && ok) {
                    tmem_load_16(tmem + ((uint32_t)(quarter * 32) << 16) + L::acc_col(a) + c0, v);
                } else {
#pragma unroll
                    for (int e = 0; e < 16; ++e) v[e] = 0;
                }
                if (k == last_k) {
                    // this warp has read its share of the tile's accumulators: one arrival per warp on the leader's barrier
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_remote(lead_free);
                }
                // 16 tokens x this warp's 32 features: transposed through the warp's own 2 KB of shared memory, so that a lane
                // stores 16 bytes of consecutive features of one token (sixteen 2-byte stores per lane, one feature each, made
                // the epilogue several microseconds longer per tile)
                const int ft = pair_idx * (2 * NA) + 2 * a + (int)rank;
                const long feat0 = (long)ft * 128 + quarter * 32;            // first feature of this warp's 32
                const bool any = ok && ft < f_tiles && feat0 < p.N;
                const float bias_f = any ? epilogue_bias(p, feat0 + lane) : 0.f;
                const int esize = p.out_f32 ? 4 : 2;
                const int per = 16 / esize;                                  // features per 16-byte piece
                const int pieces_per_row = 32 / per;                         // 4 (fp16) or 8 (fp32)
                const bool vec_ok = y_vec && (((long)p.ldy * esize) % 16 == 0);
                // the buffer holds 1 KB: sixteen tokens of fp16, or eight of fp32 (two rounds)
                const int rounds = p.out_f32 ? 2 : 1, tok_per_round = 16 / rounds;
                for (int rd = 0; rd < rounds; ++rd) {
                    __syncwarp();                                            // the previous piece has been read out of the buffer
                    if (p.out_f32) {
                        float *buf = reinterpret_cast<float *>(wbuf);
#pragma unroll
                        for (int e = 0; e < 16; ++e)
                            if ((e >> 3) == rd) buf[(e & 7) * 32 + lane] = epilogue_apply(__uint_as_float(v[e]), bias_f, p.act);
                    } else {
                        __half *buf = reinterpret_cast<__half *>(wbuf);
#pragma unroll
                        for (int e = 0; e < 16; ++e) buf[e * 32 + lane] = __float2half_rn(epilogue_apply(__uint_as_float(v[e]), bias_f, p.act));
                    }
                    __syncwarp();
                    if (!any) continue;
                    for (int q = lane; q < tok_per_round * pieces_per_row; q += 32) {
                        const int e = q / pieces_per_row, part = q % pieces_per_row;
                        const int t = tok0 + c0 + rd * tok_per_round + e;
                        if (t >= p.M) continue;
                        const long f0 = feat0 + part * per;
                        const uint8_t *src = wbuf + (size_t)(e * 32 + part * per) * esize;
                        uint8_t *dstp = reinterpret_cast<uint8_t *>(p.Y) + ((long)t * p.ldy + f0) * esize;
                        if (vec_ok && f0 + per <= p.N) {
                            *reinterpret_cast<uint4 *>(dstp) = *reinterpret_cast<const uint4 *>(src);
                        } else {
                            for (int i = 0; i < per; ++i)
                                if (f0 + i < p.N) {
                                    if (p.out_f32) reinterpret_cast<float *>(dstp)[i] = reinterpret_cast<const float *>(src)[i];
                                    else reinterpret_cast<uint16_t *>(dstp)[i] = reinterpret_cast<const uint16_t *>(src)[i];
                                }
                        }
                    }
                }
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
esp_status_t launch_pair_persist(const GemmParams &p, bool dependent, cudaStream_t stream, int sm_count) {
    using L = PairCfg<2, TN>;
    constexpr int kSmem = L::kTotal + kPersistEpiWarps * 1024;           // + the epilogue warps' transposition buffers
    static_assert(kSmem <= 227 * 1024, "shared memory");
    auto kern = spgemm_pair_persist_kernel<TN>;
    ESP_CUDA_OK(ensure_dynamic_smem((const void *)kern, kSmem));
    const int f_tiles = (p.N + 127) / 128, f_pairs = (f_tiles + 3) / 4, t_tiles = (p.M + TN - 1) / TN;
    const long n_tiles = (long)f_pairs * t_tiles;
    const int resident = sm_count / 2 > 0 ? sm_count / 2 : 1;            // one CTA per SM (tensor memory and shared memory are full)
    const int clusters = (int)(n_tiles < resident ? n_tiles : resident);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * clusters, 1, 1);
    cfg.blockDim = dim3(kPersistThreads);
    cfg.dynamicSmemBytes = kSmem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
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
    ESP_CUDA_OK(cudaLaunchKernelEx(&cfg, kern, p, wmap, xmap, f_pairs, t_tiles));
    return ESP_OK;
}
