// Kernel body of the CTA-pair SpMM (included by spmm_tc_pair.cu inside its anonymous namespace).
//
// Shared memory per CTA (identical layout in both CTAs, 1024-byte aligned):
//   num_stages x [weight tile | metadata (sparse) | 2 boxes of X (this CTA's 128 columns)]
//   | 4 warps x 2 staging tiles | barriers | TMEM base | abort flag
// The leader's MMA issuer loop with the number of MMAs per kept block fixed at compile time (the loop is
// bound by this one thread's instruction latency: descriptors of stage 0 are built once, a later stage or
// K step only moves the start-address field, and the MMAs of a block are a straight line).
struct PairMmaArgs {
    uint32_t ring, bar_full, bar_empty, bar_tfull, bar_tempty, tmem_base;
    int first_pair_tile, pair_tile_stride;
    volatile int *abort_flag;
};
template <bool kSparse, int NM>
__device__ __forceinline__ void pair_mma_role(const PairParams &p, const PairMmaArgs &a) {
    constexpr uint32_t kIdesc = make_idesc_pair(kSparse);
    constexpr int kMetaCol = kPairTileN;          // two 4-column metadata buffers after the accumulator
    const uint64_t a_desc0 = make_smem_desc(a.ring, 2048, 128, kLayoutNone);
    const uint64_t b_desc0 = make_smem_desc(a.ring + p.entry_bytes, p.box_bytes, 1024, kLayoutSw128);
    const uint64_t m_desc0 = make_smem_desc(a.ring + p.a_bytes, 128, 128, kLayoutNone);
    const uint32_t stage_step = p.stage_bytes >> 4, ring_span = p.num_stages * stage_step;
    uint32_t off = 0, full = a.bar_full, empty = a.bar_empty, ph = 0, acc_ph = 0, meta_buf = 0;
    for (int t = a.first_pair_tile; t < p.num_tiles && !*a.abort_flag; t += a.pair_tile_stride) {
        const int len = p.pair_len[t % p.npairs];
        if (!mbar_wait(a.bar_tempty, acc_ph ^ 1u, a.abort_flag)) break;
        tc_fence_after();
        uint32_t accum = 0;
        bool ok = true;
        for (int e = 0; e < len; ++e) {
            if (!mbar_wait(full, ph, a.abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint64_t ad = a_desc0 + off, bd = b_desc0 + off;
            if constexpr (kSparse) {
                const uint32_t meta_tmem = a.tmem_base + kMetaCol + 4 * meta_buf;
                tmem_copy_128x128b_pair(meta_tmem, m_desc0 + off);
#pragma unroll
                for (int j = 0; j < NM; ++j)
                    mma_sparse_pair(a.tmem_base, ad + j * 256, bd + j * 256, kIdesc | (uint32_t)(j & 1), accum | (uint32_t)j,
                                    meta_tmem + (j & ~1));
                meta_buf ^= 1u;
            } else {
#pragma unroll
                for (int j = 0; j < NM; ++j) mma_dense_pair(a.tmem_base, ad + j * 256, bd + j * 128, kIdesc, accum | (uint32_t)j);
            }
            accum = 1u;
            mma_commit_pair(empty);                 // both CTAs may refill this stage
            off += stage_step; full += 8; empty += 8;
            if (off == ring_span) { off = 0; full = a.bar_full; empty = a.bar_empty; ph ^= 1u; }
        }
        if (!ok) break;
        mma_commit_pair(a.bar_tfull);               // both CTAs' accumulators are complete
        acc_ph ^= 1u;
    }
}

template <bool kSparse, typename OutT>
__global__ void __launch_bounds__(kThreads, 1)
spmm_tc_pair_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_y,
                    const __grid_constant__ CUtensorMap map_a, PairParams p) {
    constexpr int kTmemCols = 512;
    constexpr int kOutCols = 128 / (int)sizeof(OutT);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t ring = smem_base;
    const uint32_t staging = ring + p.num_stages * p.stage_bytes;
    const uint32_t ctrl = staging + kEpiWarps * 2 * kStageTileBytes;
    uint8_t *ctrl_gen = smem_gen + (ctrl - smem_base);
    const uint32_t bar_full = ctrl, bar_empty = ctrl + 8 * kPairMaxStages, bar_tfull = ctrl + 16 * kPairMaxStages,
                   bar_tempty = bar_tfull + 8;
    volatile uint32_t *tmem_base_slot = reinterpret_cast<volatile uint32_t *>(ctrl_gen + 16 * kPairMaxStages + 16);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(ctrl_gen + 16 * kPairMaxStages + 20);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();
    const bool leader = rank == 0;
    if (threadIdx.x == 0) {
        for (uint32_t s = 0; s < p.num_stages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        mbar_init(bar_tfull, 1);
        mbar_init(bar_tempty, 2 * kEpiWarps);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(const_cast<uint32_t *>(tmem_base_slot)), kTmemCols);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                      // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_base_slot;
    const uint32_t stage_tx = p.entry_bytes + kPairBoxes * p.box_bytes;
    const int first_pair_tile = blockIdx.x >> 1, pair_tile_stride = gridDim.x >> 1;

    if (warp == 0) {
        // ------------------------------------------------ producer (both CTAs): step 1
        // (running stage/barrier addresses and image rows: this thread's own instruction latency bounds the loop)
        if (lane == 0) {
            constexpr int kAhead = 8;            // union-list entries held in registers ahead of their use
            const uint32_t leader_full0 = map_to_cta(bar_full, 0);
            const uint32_t ring_end = ring + p.num_stages * p.stage_bytes;
            const int entry_rows = (int)(p.entry_bytes >> 8);
            uint32_t dst = ring, full_own = bar_full, full_leader = leader_full0, empty = bar_empty, ph = 0;
            for (int t = first_pair_tile; t < p.num_tiles && !*abort_flag; t += pair_tile_stride) {
                const int pr = t % p.npairs, ct = t / p.npairs;
                const int st = 2 * pr + (int)rank;
                const int len = p.pair_len[pr];
                const int32_t *cols = p.pair_col + (int64_t)pr * p.pwcap;
                const int32_t *src = p.pair_src + (int64_t)pr * p.pwcap * 2 + rank;
                const int base_row = (int)(((int64_t)st * p.wcap * p.entry_bytes) >> 8);
                const int xz = ct * 4 + kPairBoxes * (int)rank;
                int col_q[kAhead], src_q[kAhead];
#pragma unroll
                for (int u = 0; u < kAhead; ++u) {
                    col_q[u] = u < len ? __ldg(cols + u) : 0;
                    src_q[u] = u < len ? __ldg(src + 2 * u) : -1;
                }
                bool ok = true;
                for (int e0 = 0; e0 < len && ok; e0 += kAhead) {
#pragma unroll
                    for (int u = 0; u < kAhead; ++u) {
                        const int e = e0 + u;
                        if (e >= len) break;
                        const int krow = col_q[u] * p.bk;
                        const int idx = src_q[u];
                        if (e + kAhead < len) { col_q[u] = __ldg(cols + e + kAhead); src_q[u] = __ldg(src + 2 * (e + kAhead)); }
                        if (!mbar_wait(empty, ph ^ 1u, abort_flag)) { ok = false; break; }
                        if (leader) mbar_expect_tx(full_own, 2 * stage_tx);
                        // a side that does not keep this block of the union loads a zero tile (row past the image)
                        const int arow = idx >= 0 ? base_row + idx * entry_rows : p.image_rows;
                        tma_load_2d_pair(dst, &map_a, 0, arow, full_leader);
                        tma_load_3d_pair(dst + p.entry_bytes, &map_x, 0, krow, xz, full_leader);
                        dst += p.stage_bytes; full_own += 8; full_leader += 8; empty += 8;
                        if (dst == ring_end) { dst = ring; full_own = bar_full; full_leader = leader_full0; empty = bar_empty; ph ^= 1u; }
                    }
                }
                if (!ok) break;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer (leader CTA only): steps 2 + 3
        if (leader && lane == 0) {
            const PairMmaArgs a{ring, bar_full, bar_empty, bar_tfull, bar_tempty, tmem_base, first_pair_tile,
                                pair_tile_stride, abort_flag};
            const int nmma = kSparse ? p.bk / 32 : p.bk / 16;
            if constexpr (kSparse) {
                switch (nmma) {
                    case 1: pair_mma_role<true, 1>(p, a); break;
                    case 2: pair_mma_role<true, 2>(p, a); break;
                    case 3: pair_mma_role<true, 3>(p, a); break;
                    default: pair_mma_role<true, 4>(p, a); break;
                }
            } else {
                switch (nmma) {
                    case 2: pair_mma_role<false, 2>(p, a); break;
                    case 4: pair_mma_role<false, 4>(p, a); break;
                    case 6: pair_mma_role<false, 6>(p, a); break;
                    default: pair_mma_role<false, 8>(p, a); break;
                }
            }
        }
    } else {
        // ------------------------------------------------ epilogue (both CTAs)
        const int q = warp & 3;
        const uint32_t stg = staging + (uint32_t)(warp - 2) * 2 * kStageTileBytes;
        uint8_t *stg_gen = smem_gen + (stg - smem_base);
        const uint32_t leader_tempty = map_to_cta(bar_tempty, 0);
        uint32_t acc_ph = 0, buf = 0;
        for (int t = first_pair_tile; t < p.num_tiles; t += pair_tile_stride) {
            const int pr = t % p.npairs, ct = t / p.npairs;
            const int st = 2 * pr + (int)rank;
            int go = 0;
            if (lane == 0) go = !*abort_flag && mbar_wait(bar_tfull, acc_ph, abort_flag);
            go = __shfl_sync(0xFFFFFFFFu, go, 0);
            if (!go) break;
            tc_fence_after();
            const uint32_t t_addr = tmem_base + ((uint32_t)(32 * q) << 16);
#pragma unroll 1
            for (int c = 0; c < kPairTileN / kOutCols; ++c) {
                uint32_t out[32];
                if constexpr (sizeof(OutT) == 2) {
                    uint32_t r0[32], r1[32];
                    tmem_ld32(t_addr + c * 64, r0);
                    tmem_ld32(t_addr + c * 64 + 32, r1);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        out[i] = pack_bf16(__uint_as_float(r0[2 * i]), __uint_as_float(r0[2 * i + 1]));
                        out[16 + i] = pack_bf16(__uint_as_float(r1[2 * i]), __uint_as_float(r1[2 * i + 1]));
                    }
                } else {
                    tmem_ld32(t_addr + c * 32, out);
                    tmem_ld_wait();
                }
                const int x0 = ct * kPairTileN + c * kOutCols, y0 = st * kTileM + 32 * q;
                if (lane == 0) bulk_wait_read<1>();
                __syncwarp();
                uint8_t *tile = stg_gen + buf * kStageTileBytes + lane * 128;
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    *reinterpret_cast<uint4 *>(tile + ((j ^ (lane & 7)) << 4)) =
                        make_uint4(out[4 * j], out[4 * j + 1], out[4 * j + 2], out[4 * j + 3]);
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    if (x0 < p.ncols && y0 < p.rows) tma_store_2d(&map_y, stg + buf * kStageTileBytes, x0, y0);
                    bulk_commit();
                }
                buf ^= 1u;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) remote_arrive(leader_tempty);
            acc_ph ^= 1u;
        }
        if (lane == 0) bulk_wait_read<0>();
    }

    // ------------------------------------------------ teardown (every wait above is bounded)
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0) atomicCAS(p.status, 0, (int)CRISP_TIMEOUT);
        const unsigned long long t0 = clock64();
        while ((unsigned long long)(clock64() - t0) < 2000000ull) __nanosleep(1000);
    }
    cluster_sync_all();                      // neither CTA frees tensor memory while the other still uses the pair
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}
