// Prefill GEMM on CTA pairs (included by tl_gemm.cu after GemmParams and the helpers).
//
// A tcgen05.mma occupies the tensor pipe for N/2 clocks per 16-deep K step whether it is issued for one CTA
// (cta_group::1, M = 64 or 128) or for a pair (cta_group::2, M = 256: measured 128 clocks for 256 x 256 x 16).  The
// pair form therefore does twice the work per instruction and per operand byte staged in shared memory: each CTA
// holds only its own half of the tile's weights and tokens, and the one thread that issues MMAs has half as many
// instructions to get out per flop.
// So for large M two CTAs share one 256-token x 256-column output tile:
//   - each CTA loads ITS 128 weight columns (the same one-box-per-stage tile-major view as the single-CTA
//     kernel) and HALF of the 256 token rows; 32 KB per CTA per 64-row K step instead of 48 KB, six stages;
//   - the even ("leader") CTA issues every MMA; the instruction reads the M-side operand (weights, 128 rows
//     from each CTA) and the N-side operand (tokens, 128 rows from each CTA) out of both shared memories
//     and writes 128 accumulator lanes x 256 columns into each CTA's tensor memory;
//   - TMA completions of both CTAs count on the leader's "full" barrier, which the leader arms for the bytes
//     of both (a cluster-scope arrive per stage from the peer measured ~600 clocks and starved the MMAs);
//     tcgen05.commit is multicast so the
//     "stage free" and "accumulator ready" barriers of both CTAs fire together; "accumulator drained"
//     arrivals of both CTAs' epilogue warps go to the leader;
//   - each CTA's epilogue writes its own 128 columns of C: every warp moves 32 tokens x 32 columns at a time from
//     tensor memory through a 4 KB block of shared memory (behind the pipeline stages) to C with a tiled bulk
//     store, which clips the ragged edges (plain stores from the registers when the switch is off).
// With 256 x 256 tiles the kernel is held back by operand traffic out of L2 (32 KB per CTA per 64-row K step).  A
// tile may therefore cover two 256-token blocks (kHalves = 2): one weight slab per stage serves both (48 KB per CTA
// for twice the work, four stages), two MMAs per K step into the two halves of tensor memory, and eight epilogue
// warps because the epilogue is no longer hidden behind the next tile's MMAs.  Whole waves of clusters take such
// tiles; what is left of the tile grid runs as 256-token tiles.
// No TMA multicast is used.  Every wait is on a barrier in the waiter's own shared memory and is bounded.
#pragma once

namespace tl {

__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx_cluster(uint32_t cluster_addr, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.release.cluster.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_addr),
                 "r"(bytes)
                 : "memory");
}
// TMA loads of a CTA pair: the bytes land in the issuing CTA's shared memory, the completion is counted on
// the barrier at `bar_cluster_addr` (the leader's).
__device__ __forceinline__ void tma_pair_load_2d(void* dst, const void* tmap, uint32_t bar_cluster_addr, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], "
        "[%2];" ::"r"(smem_u32(dst)),
        "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar_cluster_addr), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tma_pair_load_5d(void* dst, const void* tmap, uint32_t bar_cluster_addr, int c0, int c1,
                                                 int c2, int c3, int c4) {
    asm volatile(
        "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, "
        "%5, %6, %7}], [%2];" ::"r"(smem_u32(dst)),
        "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
        : "memory");
}
__device__ __forceinline__ void umma_pair_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_pair_f8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The same with the descriptors given as 32-bit halves (constant upper words, offsets added to the lower word).
template <bool kFp8>
__device__ __forceinline__ void umma_pair_split(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                                uint32_t idesc, uint32_t accumulate) {
    if (kFp8)
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b64 a, b;\n\t"
            "mov.b64 a, {%1, %2};\n\tmov.b64 b, {%3, %4};\n\t"
            "setp.ne.b32 p, %6, 0;\n\t"
            "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], a, b, %5, p;\n\t}"
            ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
            : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b64 a, b;\n\t"
            "mov.b64 a, {%1, %2};\n\tmov.b64 b, {%3, %4};\n\t"
            "setp.ne.b32 p, %6, 0;\n\t"
            "tcgen05.mma.cta_group::2.kind::f16 [%0], a, b, %5, p;\n\t}"
            ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
            : "memory");
}
// Arrives on the barrier at the same shared-memory offset in both CTAs once the MMAs issued so far are done.
__device__ __forceinline__ void umma_pair_commit_both(uint64_t* bar) {
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(smem_u32(bar)), "h"(uint16_t(3))
        : "memory");
}

constexpr int kPairBand = 8;      // m-tiles per band of the tile order

// Tile order: bands of kPairBand m-tiles, inside a band the n-tile index moves slowest.  The clusters that run
// together then cover about 8 x 9 tiles instead of 16 x 4.6: fewer operand bytes per wave (every cluster of a
// wave re-reads the A rows of its m-tile and the B columns of its n-tile; what they share is fetched from HBM
// once), and the band's A rows stay warm in L2 while the wave front moves along N.
__device__ __forceinline__ void pair_tile_coords(int tile, int m_tiles, int n_tiles, int* m_tile, int* n_tile) {
    const int band_tiles = kPairBand * n_tiles;
    const int band = tile / band_tiles, r = tile - band * band_tiles;
    const int band_rows = m_tiles - band * kPairBand < kPairBand ? m_tiles - band * kPairBand : kPairBand;
    *m_tile = band * kPairBand + r % band_rows;
    *n_tile = r / band_rows;
}

// One output tile of the pair kernel: rows [row0, row0 + 256 * halves) x weight columns of pair tile n_tile.
struct PairTile {
    int row0, n_tile, halves;
};

// kHalves = 1: every tile is 256 tokens x 256 columns.  kHalves = 2: the first p.pair_big_tiles tiles are
// 512 tokens x 256 columns (numbered like the 256-token tiles, over 512-row m-tiles); what is left of the grid
// of big tiles follows as 256-token tiles, two per big tile, so that the last wave is not half empty.
template <int kHalves>
__device__ __forceinline__ PairTile pair_decode(const GemmParams& p, int tile, int m_tiles, int n_tiles) {
    PairTile t;
    int m_tile;
    if (kHalves == 1) {
        pair_tile_coords(tile, m_tiles, n_tiles, &m_tile, &t.n_tile);
        t.row0 = m_tile * 256;
        t.halves = 1;
    } else if (tile < p.pair_big_tiles) {
        pair_tile_coords(tile, m_tiles, n_tiles, &m_tile, &t.n_tile);
        t.row0 = m_tile * 512;
        t.halves = p.M - t.row0 > 256 ? 2 : 1;
    } else {
        const int s = tile - p.pair_big_tiles;
        pair_tile_coords(p.pair_big_tiles + (s >> 1), m_tiles, n_tiles, &m_tile, &t.n_tile);
        t.row0 = m_tile * 512 + (s & 1) * 256;
        t.halves = t.row0 < p.M ? 1 : 0;                  // 0: nothing there (a ragged last m-tile)
    }
    return t;
}

// One cluster = one output tile at a time (256 or 512 tokens x 256 columns); CTA rank r owns columns
// n0 + 128 r .. + 127 and loads half of every 256-token block.  With 512-token tiles a stage carries one weight
// slab for two token blocks (48 KB per CTA instead of 2 x 32 KB for the same work: a quarter less traffic from
// L2, which is what limits the 256-token form), both accumulators belong to one tile and the epilogue is no
// longer hidden behind the next tile's MMAs.
// Dense problems only (no experts, no stream-K, TMA-readable weights); p.BM == 256, per-CTA tile 128 columns.
// kHalves = 2 runs with four more epilogue warps (one set per token block): its epilogue is exposed.
template <bool kFp8, int kHalves>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kHalves == 2 ? kPairBigThreads : kGemmThreads, 1)
gemm_pair_kernel(const __grid_constant__ GemmParams p) {
    constexpr int kBK = 64, kKSteps = 4;
    constexpr uint32_t kWBytes = kBK * 128 * 2;           // this CTA's weight slab per stage
    constexpr uint32_t kTokBytes = 128 * kAtomBytes;      // this CTA's half of one 256-token block per stage
    constexpr uint32_t kStageBytes = kWBytes + kHalves * kTokBytes;

    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kPairStagesMax];     // used in the leader only
    __shared__ __align__(8) uint64_t empty_bar[kPairStagesMax];    // one copy per CTA
    __shared__ __align__(8) uint64_t acc_full_bar[2];              // one copy per CTA
    __shared__ __align__(8) uint64_t acc_empty_bar[2];             // used in the leader only
    __shared__ uint32_t tmem_slot;
    __shared__ uint32_t abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_cta_rank();
    uint8_t* stages = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.num_stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full_bar[b], 1); mbar_init(&acc_empty_bar[b], 8 * kHalves); }
        abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&p.tmap_b);
        tma_prefetch_desc(&p.tmap_a[3]);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                     "r"(512)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync();                 // both CTAs' barriers are initialised before anyone touches the peer's
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_slot;
    volatile uint32_t* abort_ptr = &abort_flag;

    const int m_tiles = (p.M + 256 * kHalves - 1) / (256 * kHalves);
    const int n_pair_tiles = (p.N + 255) / 256;
    const int tiles_total = kHalves == 1 ? m_tiles * n_pair_tiles
                                         : p.pair_big_tiles + 2 * (m_tiles * n_pair_tiles - p.pair_big_tiles);
    const int first_tile = int(cluster_id_x()), tile_step = int(num_clusters_x());

    if (warp == 0) {
        // ============================================================ TMA producer (one per CTA)
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, issued = 0;
            bool ok = true;
            int ks[4], km[4];                                       // K part of the coordinate maps, in registers
#pragma unroll
            for (int i = 0; i < 4; ++i) { ks[i] = p.ck_shift[i]; km[i] = p.ck_mask[i]; }
            for (int tile = first_tile; ok && tile < tiles_total; tile += tile_step) {
                const PairTile pt = pair_decode<kHalves>(p, tile, m_tiles, n_pair_tiles);
                if (pt.halves == 0) continue;
                const int n0 = pt.n_tile * 256 + int(rank) * 128;   // this CTA's weight columns
                const int row0 = pt.row0 + int(rank) * 128;         // this CTA's half of the (first) token block
                int cn[4];                                          // column part of the weight box's coordinates
#pragma unroll
                for (int i = 0; i < 4; ++i) cn[i] = (n0 >> p.cn_shift[i]) & p.cn_mask[i];
                for (int kit = 0; kit < p.k_iters; ++kit) {
                    if (!mbar_wait_bounded(&empty_bar[stage], phase ^ 1, abort_ptr, p.status, kWaitProducerEmpty, p.wait_limit_ns)) {
                        ok = false;
                        break;
                    }
                    uint8_t* sw = stages + size_t(stage) * kStageBytes;
                    // The leader's producer alone arms the barrier, for the bytes of BOTH CTAs; the peer only
                    // issues its copies.  Their completions may be counted before the leader has armed the
                    // phase (the byte count then goes negative for a moment); the phase cannot complete before
                    // the arrival, and the peer cannot run a whole ring ahead because its "stage free" barrier
                    // is only signalled after the leader's MMAs have consumed the stage.
                    const uint32_t full_leader = map_to_cta(smem_u32(&full_bar[stage]), 0);
                    if (rank == 0) mbar_arrive_expect_tx(&full_bar[stage], 2 * (kWBytes + uint32_t(pt.halves) * kTokBytes));
                    const int k = (kit * kBK) << p.k_shift;         // K element (8-bit types: twice as many per stage)
                    tma_pair_load_2d(sw + kWBytes, &p.tmap_a[3], full_leader, k, row0);
                    if (kHalves == 2 && pt.halves == 2)
                        tma_pair_load_2d(sw + kWBytes + kTokBytes, &p.tmap_a[3], full_leader, k, row0 + 256);
                    tma_pair_load_5d(sw, &p.tmap_b, full_leader, 0, ((k >> ks[0]) & km[0]) + cn[0], ((k >> ks[1]) & km[1]) + cn[1],
                                     ((k >> ks[2]) & km[2]) + cn[2], ((k >> ks[3]) & km[3]) + cn[3]);
                    ++issued;
                    if (++stage == uint32_t(p.num_stages)) { stage = 0; phase ^= 1; }
                }
            }
            (void)issued;
        }
    } else if (warp == 1) {
        // ============================================================= MMA issuer (leader CTA only)
        if (rank == 0 && lane == 0) {
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            // fp32 accumulate, bf16 x bf16, A (weights) MN-major, B (tokens) K-major, M = 256 over the pair, N = 256
            // (weights K-major when they are stored [N][K])
            // (8-bit operands: format codes 0 = E4M3 in place of 1 = bf16)
            const uint32_t idesc = (1u << 4) | (kFp8 ? 0u : (1u << 7) | (1u << 10)) | (p.w_kmajor ? 0u : (1u << 15)) |
                                   ((256u >> 3) << 17) | ((256u >> 4) << 24);
            bool ok = true;
            // constant descriptor words and per-K-step offsets, in registers for the issue loop
            const uint64_t tok_hi64 = smem_desc_hi(16u, 1024u, 2u);
            const uint32_t tok_hi = uint32_t(tok_hi64 >> 32), tok_lo_const = uint32_t(tok_hi64);
            const uint32_t w_hi = uint32_t(p.w_desc_hi >> 32), w_lo_const = uint32_t(p.w_desc_hi);
            uint32_t w_off[kKSteps];
#pragma unroll
            for (int j = 0; j < kKSteps; ++j) w_off[j] = p.kstep_off[j] >> 4;
            for (int tile = first_tile; ok && tile < tiles_total; tile += tile_step) {
                const PairTile pt = pair_decode<kHalves>(p, tile, m_tiles, n_pair_tiles);
                if (pt.halves == 0) continue;
                if (!mbar_wait_bounded(&acc_empty_bar[acc], acc_phase ^ 1, abort_ptr, p.status, kWaitMmaAccEmpty, p.wait_limit_ns)) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * 256u;
                for (int kit = 0; kit < p.k_iters; ++kit) {
                    if (!mbar_wait_bounded(&full_bar[stage], phase, abort_ptr, p.status, kWaitMmaFull, p.wait_limit_ns)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint32_t sw = smem_u32(stages + size_t(stage) * kStageBytes);
                    const uint32_t w_lo0 = w_lo_const | ((sw & 0x3FFFFu) >> 4);
                    const uint32_t tok_lo0 = tok_lo_const | (((sw + kWBytes) & 0x3FFFFu) >> 4);
                    const uint32_t first = kit > 0 ? 1u : 0u;
                    const bool two = kHalves == 2 && pt.halves == 2;
#pragma unroll
                    for (int j = 0; j < kKSteps; ++j) {
                        const uint32_t accum = j > 0 ? 1u : first;
                        umma_pair_split<kFp8>(d_tmem, w_lo0 + w_off[j], w_hi, tok_lo0 + uint32_t(j) * 2u, tok_hi, idesc, accum);
                        if (two)                                    // the same weights on the second token block
                            umma_pair_split<kFp8>(d_tmem + 256u, w_lo0 + w_off[j], w_hi,
                                                  tok_lo0 + (kTokBytes >> 4) + uint32_t(j) * 2u, tok_hi, idesc, accum);
                    }
                    umma_pair_commit_both(&empty_bar[stage]);       // frees the stage in both CTAs
                    if (++stage == uint32_t(p.num_stages)) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                umma_pair_commit_both(&acc_full_bar[acc]);          // accumulator complete, both CTAs
                if (kHalves == 1) acc ^= 1;                         // (512-token tiles own both accumulators)
                if (acc == 0) acc_phase ^= 1;
            }
        }
    } else {
        // =============================================================== epilogue (both CTAs)
        const int quarter = warp & 3;
        const int my_half = kHalves == 2 ? (warp - 2) >> 2 : 0;     // warps 2..5 drain token block 0, 6..9 block 1
        uint8_t* out_stage = stages + size_t(p.num_stages) * kStageBytes + size_t(warp - 2) * p.out_bufs * kPairStageOutBytes;
        uint32_t out_buf = 0;
        uint32_t acc = 0, acc_phase = 0;
        for (int tile = first_tile; tile < tiles_total; tile += tile_step) {
            const PairTile pt = pair_decode<kHalves>(p, tile, m_tiles, n_pair_tiles);
            if (pt.halves == 0) continue;
            const int n0 = pt.n_tile * 256 + int(rank) * 128;
            const bool ok = mbar_wait_bounded(&acc_full_bar[acc], acc_phase, abort_ptr, p.status, kWaitEpilogueAccFull, p.wait_limit_ns);
            tc_fence_after_sync();
            if (ok) {
                const int n_local = quarter * 32 + lane;
                const bool n_ok = n0 + n_local < p.N;
                for (int h = my_half; h < pt.halves; h += kHalves) {
                    const int row0 = pt.row0 + h * 256;
                    const int rows = p.M - row0 < 256 ? p.M - row0 : 256;
                    float* out = p.C + int64_t(row0) * p.ldc + n0;
                    const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + acc * 256u + uint32_t(h) * 256u;
                    if (p.c_tma) {
                        // The 32 tokens x 32 columns this warp holds after one tcgen05.ld go to shared memory as a
                        // row-major block (lane = column: conflict-free) and from there to C as one tiled bulk store,
                        // which clips rows beyond M and columns beyond N.  The next block's tcgen05.ld is in flight
                        // meanwhile.  The block is reused once the previous store has read it.
                        const int cx = n0 + quarter * 32, chunks = (rows + 31) >> 5;
                        uint32_t va[32], vb[32];
                        auto emit = [&](const uint32_t (&v)[32], int c) {
                            uint8_t* blk = out_stage + out_buf * kPairStageOutBytes;
                            if (lane == 0) {
                                if (p.out_bufs == 2) bulk_wait_group_read<1>(); else bulk_wait_group_read<0>();
                            }
                            __syncwarp();
                            if (p.Cb == nullptr) {
                                float* st = reinterpret_cast<float*>(blk);
#pragma unroll
                                for (int i = 0; i < 32; ++i) st[i * 32 + lane] = __uint_as_float(v[i]);
                            } else {
                                __nv_bfloat16* st = reinterpret_cast<__nv_bfloat16*>(blk);
#pragma unroll
                                for (int i = 0; i < 32; ++i) st[i * 32 + lane] = __float2bfloat16_rn(__uint_as_float(v[i]));
                            }
                            fence_proxy_async_smem();
                            __syncwarp();
                            if (lane == 0) {
                                tma_store_2d(&p.tmap_c, blk, cx, row0 + c * 32);
                                bulk_commit_group();
                            }
                            if (p.out_bufs == 2) out_buf ^= 1;
                        };
                        tmem_ld_32x32b_x32(taddr, va);
                        for (int c = 0; c < chunks; c += 2) {
                            tmem_ld_wait();
                            if (c + 1 < chunks) tmem_ld_32x32b_x32(taddr + (c + 1) * 32, vb);
                            emit(va, c);
                            if (c + 1 >= chunks) break;
                            tmem_ld_wait();
                            if (c + 2 < chunks) tmem_ld_32x32b_x32(taddr + (c + 2) * 32, va);
                            emit(vb, c + 1);
                        }
                    } else if (p.Cb == nullptr) {
                        for (int c0 = 0; c0 < 256; c0 += 32) {
                            if (c0 >= rows) break;
                            uint32_t v[32];
                            tmem_ld_32x32b_x32(taddr + c0, v);
                            tmem_ld_wait();
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if (n_ok && c0 + i < rows) out[int64_t(c0 + i) * p.ldc + n_local] = __uint_as_float(v[i]);
                        }
                    } else {                                        // bf16 C
                        __nv_bfloat16* outb = p.Cb + int64_t(row0) * p.ldc + n0 + n_local;
                        for (int c0 = 0; c0 < 256; c0 += 32) {
                            if (c0 >= rows) break;
                            uint32_t v[32];
                            tmem_ld_32x32b_x32(taddr + c0, v);
                            tmem_ld_wait();
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if (n_ok && c0 + i < rows) outb[int64_t(c0 + i) * p.ldc] = __float2bfloat16_rn(__uint_as_float(v[i]));
                        }
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&acc_empty_bar[acc]), 0));
            if (kHalves == 1) acc ^= 1;
            if (acc == 0) acc_phase ^= 1;
            if (*abort_ptr) break;
        }
        if (p.c_tma && lane == 0) bulk_wait_group<0>();             // this warp's stores are done before the CTA leaves
    }

    // Neither CTA may leave while its peer can still signal its barriers or read its shared memory.
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync();
    if (warp == 1) {
        tc_fence_after_sync();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
    }
}

}  // namespace tl
