// Device side of the tiled GEMM (included by the translation units that instantiate or launch it): parameters,
// scheduler, helpers and the single-CTA kernel.  See tl_gemm.cu for the overview.
#pragma once

#include "tl_common.cuh"

#include <cuda_bf16.h>

namespace tl {

constexpr int kGemmThreads = 192;          // TMA path: producer, MMA issuer, four epilogue warps
constexpr int kGenericThreads = 352;       // tile rows under 16 bytes: four more warps that transpose the stage in place or build
                                           // the weight operand by hand, and one that streams raw memory tiles into shared memory
constexpr int kMaxStages = 16;
constexpr int kMaxExperts = 1024;
constexpr int kNumBoxChoices = 5;          // token boxes of 16, 32, 64, 128, 256 rows
constexpr int kAtomBytes = 128;            // one swizzle row: 64 bf16
constexpr int kMaxDynamicSmem = 227 * 1024 - 10 * 1024;   // 227 KB per CTA minus the kernel's static shared memory

struct alignas(64) GemmParams {
    CUtensorMap tmap_a[kNumBoxChoices];
    CUtensorMap tmap_b;
    CUtensorMap tmap_c;         // pair kernel, c_tma: C (fp32 or bf16) as [M][N] with boxes of 32 rows x 32 columns
    int out_bufs;               // pair kernel: 32 x 32 blocks of C each epilogue warp may have on their way (1 or 2)
    int c_tma;                  // 1: the pair kernel's epilogue stages C in shared memory and writes it with tiled bulk stores
    float* C;
    float* partials;            // stream-K partial tiles: slot = BM x BN floats
    const int32_t* offsets;     // grouped: device E+1 row offsets; dense: nullptr
    uint32_t* status;
    uint64_t wait_limit_ns;     // bound of every barrier wait in the kernel
    uint32_t stall_extra_tx;    // test hook: bytes added to what the first stage's barrier expects (0 in normal use)
    // Two grouped products in one launch, the second one's tokens being the first one's output (expert FFN): one
    // counter per m-tile.  tile_flags_mode 1: every epilogue warp adds one to tile_flags[m-tile] once its share of a
    // whole output tile is stored; 2: the producer loads an m-tile's tokens only after tile_flags[m-tile] has reached
    // tile_flags_target (bounded wait).  0: not used.
    uint32_t* tile_flags;
    int tile_flags_mode;
    uint32_t tile_flags_target;
    int tile_flags_skip_cta0;   // test hook: CTA 0 does not add to the counters, so that the waits on its m-tiles run out
    int provisional_skew;       // test hook: rows added to the expert offsets read before the wait (0 in normal use)
    int reduce_split;           // stream-K reduction: 1 = every boundary inside a split tile sums a share of it
    int64_t ldc;                // N
    int M;                      // dense rows (grouped: total rows)
    int N, K, E;
    int BM;                     // token rows per CTA tile: 16, 32, 64, 128 or 256
    int umma_m;                 // weights-on-N kernels: rows of the MMA's token side, 64 when BM <= 64, else 128
    int a_rows;                 // token rows a stage holds per 64-wide K slice: max(BM, umma_m) there, else BM; rows
                                // beyond BM are zeroed once and never written again
    int BN;                     // weight columns per CTA tile: 128 or 256
    int n_tiles, k_iters;
    int stream_k;               // 0: whole tiles round-robin, 1: contiguous K-iteration ranges
    int cluster_k;              // S > 1: launched in clusters of S CTAs; cluster c owns output tile c, CTA rank r of it the
                                // r-th of S equal parts of the K loop; the partial tiles are added through distributed
                                // shared memory (no workspace, no reduction kernel).  Dense, weights-on-N kernels only.
    int num_stages;
    int prefetch_stages;        // stages of weights each CTA asks into L2 before it waits for its predecessor
    int pair_big_tiles;         // pair kernel with 512-token tiles: how many tiles are of that size (the rest 256)
    // Gated epilogue (expert FFN): weight columns 2j / 2j+1 hold gate_j / up_j; H[row][j] = bf16(silu(g) * u)
    // replaces C.  Weights-on-N kernels only.
    int epi_swiglu;
    __nv_bfloat16* H;
    int64_t ldh;
    __nv_bfloat16* Cb;          // non-null: C is written as bf16 (one rounding to nearest even) instead of fp32
    // weight-operand geometry
    int row_major;              // 1: the weight is not tiled ([K][N] row-major, or [N][K] when w_kmajor)
    int w_kmajor;               // 1: weights stored [N][K], K contiguous (Eq. 2 as printed): K-major MMA operand
    int k_inner;                // 1: tensor-map dimensions ordered (64, row in tile, tile along K, atom, tile along N)
    // Tensor-map coordinates 1..4 of a weight box as shifts and masks of its first K element k and weight column n:
    // c[i] = ((k >> ck_shift[i]) & ck_mask[i]) + ((n >> cn_shift[i]) & cn_mask[i]) + c_expert[i] * (expert offset).
    // (Set by the host for the layout at hand: the producer's loop has no layout branches.)
    int ck_shift[4], ck_mask[4], cn_shift[4], cn_mask[4], c_expert[4];
    int fp8;                    // 1: both operands are 8-bit floating point (E4M3); needs w_kmajor
    int k_shift;                // log2(K elements per 2 bytes): a stage holds (BK << k_shift) K-elements
    int w_atom_log2;            // K-major weights: log2(elements in one swizzle row of 128, 64 or 32 bytes)
    uint64_t w_desc_hi;         // weight operand's shared-memory descriptor without its start address
    int br_log2, bc_log2;       // memory tile: rows x contiguous columns of the stored matrix (tiled layouts only)
    int k_coord_per_expert;     // added per expert to the coordinate of the stacked dimension (blocks or rows)
    int box_rows, box_atoms;    // rows and 128-byte atoms of one box
    int kbx, nbx;               // boxes per stage along K and along N
    uint32_t box_bytes;
    uint32_t lbo, sbo;          // descriptor strides of the weight operand, bytes
    uint32_t ugroup_off;        // bytes between the 128-column groups of a 256-column tile
    uint32_t kstep_off[8];      // byte offset of each 16-row K step inside a stage
    // generic-address path (Section 4.4: memory tiles that TMA cannot box)
    int generic_b;              // 1: warps 6..9 build the weight operand with Eq. 1-2 address arithmetic
                                // 2: memory tiles with 8- or 4-byte rows: the copy engine lands the stage's tiles as stored,
                                //    warps 6..9 transpose 8- or 4-byte pieces in place (see fixup_stage_in_place)
    int raw_slots;              // generic path: ring of raw stage images (memory order) behind the pipeline stages
    uint32_t smem_limit;        // dynamic shared memory of the launch, bytes (the bulk copies check their destination against it)
    int64_t b_bytes;            // size of the weight buffer, bytes (... and their source against this)
    const uint8_t* B;           // raw weight pointer (generic path only)
    int64_t expert_bytes;       // K*N*2
    int blocks_per_row;         // N / bc
};

struct tl_true { static constexpr bool value = true; };
struct tl_false { static constexpr bool value = false; };

struct TileInfo {
    int n0;          // first weight column
    int row0;        // first row of A / C
    int rows;        // valid rows (<= BM)
    int expert;
    int flip;        // odd m-tile of its (expert, n-tile): walks K backwards (see decode_tile)
    int mtile;       // index of the m-tile among all m-tiles of the problem (experts in order)
};

// ------------------------------------------------------------------ scheduler
struct Work {
    int tile, kbeg, kend;
};

constexpr int kRangeTabMax = 256;      // CTAs whose range starts are tabulated in shared memory

// Work of one CTA.  Three schedules:
//   stream_k == 0   whole tiles, round-robin over the grid;
//   stream_k == 1   whole rounds of tiles round-robin (dp_tiles = the largest multiple of the grid below the tile
//                   count, or all tiles, see whole_rounds_tiles:
//                   tiles next to each other in the order run at the same time on different SMs and share
//                   what they read through L2), then the flattened (tile, K iteration) space of the tiles that
//                   are left cut into one contiguous range per CTA ("stream-K": all SMs stay busy to the end; a
//                   CTA that owns only part of a tile's K loop leaves a partial tile for the reduction kernel);
//   stream_k == 2   cluster split-K: tile = cluster index, K loop cut over the cluster's CTAs.
// All arithmetic of the cut part works on the tiles after dp_tiles ("cut space": iteration x = (tile - dp_tiles) *
// k_iters + k iteration).
constexpr int kNoCutStages = 32;      // see Sched::no_cut

struct Sched {
    int stream_k, k_iters, tiles_total, grid_eff, cta, grid;
    int dp_tiles;       // tiles handed out whole before the cut part starts (0 unless stream_k == 1)
    int next_tile;
    long long it, it_end, it_begin;
    const int* tab;     // tab[c] = first iteration (cut space) of CTA c (grid_eff + 1 entries), or nullptr

    // Even split of the cut space; a fixed function of the CTA index.
    __device__ static long long split(long long total, int grid_eff, int c) { return (total * c) / grid_eff; }
    // Tiles handed out whole.  The cut of what is left after the whole rounds costs a fixed 5 to 10 us (partial tiles
    // through the workspace, the reduction kernel's work and wake-up), more than a last, partly filled round of short
    // tiles does (its few CTAs stream at a higher rate each).  With tiles of at most 32 stages and enough of them to
    // occupy three quarters of the CTAs nothing is cut: measured on grouped products of 0.8 to 17 rounds with 12 and 32
    // stages per tile, handing every tile out whole was faster in 36 of 38 cases (by up to 30 %; the two others lost 1 %),
    // whether the last round held 4 tiles or 138.
    __device__ static bool no_cut(long long tiles_total, int grid, int k_iters) {
        return tiles_total * 4 >= 3ll * grid && k_iters <= kNoCutStages;
    }
    __device__ static int whole_rounds_tiles(int tiles_total, int grid, int k_iters) {
        if (grid <= 0) return 0;
        if (no_cut(tiles_total, grid, k_iters)) return tiles_total;
        return (tiles_total / grid) * grid;
    }
    __device__ long long cut_total() const { return static_cast<long long>(tiles_total - dp_tiles) * k_iters; }
    __device__ long long range_begin(int c) const { return tab ? tab[c] : split(cut_total(), grid_eff, c); }
    __device__ static int effective_grid(long long total, int grid) { return total < grid ? static_cast<int>(total) : grid; }
    // Cluster split-K: the one work item of this CTA (tile = cluster index, the rank's share of the K loop).
    __device__ void init_cluster(int k_iters_, int tiles_total_, int cluster, int rank, int size) {
        stream_k = 2; k_iters = k_iters_; tiles_total = tiles_total_; cta = cluster; tab = nullptr; grid_eff = 0;
        grid = 0; dp_tiles = 0;
        next_tile = cluster;
        it_begin = it = static_cast<long long>(k_iters_) * rank / size;
        it_end = static_cast<long long>(k_iters_) * (rank + 1) / size;
        if (cluster >= tiles_total_) it_end = it;
    }
    __device__ void init(int stream_k_, int k_iters_, int tiles_total_, int grid_, int cta_, const int* tab_) {
        stream_k = stream_k_; k_iters = k_iters_; tiles_total = tiles_total_; cta = cta_; tab = tab_; grid = grid_;
        dp_tiles = stream_k ? whole_rounds_tiles(tiles_total, grid, k_iters) : 0;
        grid_eff = effective_grid(cut_total(), grid);
        next_tile = cta;
        if (grid_eff == 0 || cta >= grid_eff) { it = it_end = it_begin = 0; return; }
        it_begin = it = range_begin(cta);
        it_end = range_begin(cta + 1);
    }
    __device__ bool next(Work& w) {
        if (stream_k != 2 && next_tile < (stream_k ? dp_tiles : tiles_total)) {
            w.tile = next_tile; w.kbeg = 0; w.kend = k_iters;
            next_tile += grid;
            return true;
        }
        if (!stream_k || it >= it_end) return false;
        if (stream_k == 2) {
            w.tile = next_tile; w.kbeg = static_cast<int>(it); w.kend = static_cast<int>(it_end);
            it = it_end;
            return true;
        }
        int t = static_cast<int>(it / k_iters);
        int kb = static_cast<int>(it - static_cast<long long>(t) * k_iters);
        long long left = it_end - it;
        int ke = (k_iters - kb) < left ? k_iters : kb + static_cast<int>(left);
        w.tile = dp_tiles + t; w.kbeg = kb; w.kend = ke;
        it += ke - kb;
        return true;
    }
    // CTA whose range holds iteration x of the cut space.
    __device__ int owner(long long x) const {
        if (tab) {                                   // largest c with tab[c] <= x
            int lo = 0, hi = grid_eff;
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (tab[mid] <= x) lo = mid; else hi = mid;
            }
            return lo;
        }
        long long total = cut_total();
        int c = static_cast<int>(((x + 1) * grid_eff + total - 1) / total) - 1;
        if (c < 0) c = 0;
        if (c >= grid_eff) c = grid_eff - 1;
        while (c > 0 && range_begin(c) > x) --c;
        while (c + 1 < grid_eff && range_begin(c + 1) <= x) ++c;
        return c;
    }
    // Partial-tile slot of CTA c for tile t (of the cut part): 2c when the tile is the first thing c works on there, else 2c+1.
    __device__ int slot(int c, int t) const {
        return 2 * c + (range_begin(c) < static_cast<long long>(t - dp_tiles) * k_iters ? 1 : 0);
    }
};

__device__ __forceinline__ TileInfo decode_tile(const GemmParams& p, const int* prefix, const int* row_start, int tile,
                                                bool flip_odd = false) {
    // prefix[e] = tiles of experts before e; tiles of one expert: n-tile major, m-tile minor.
    int lo = 0, hi = p.E;                  // find e with prefix[e] <= tile < prefix[e+1]
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (prefix[mid] <= tile) lo = mid; else hi = mid;
    }
    const int e = lo;
    const int local = tile - prefix[e];
    const int mt = (prefix[e + 1] - prefix[e]) / p.n_tiles;
    const int row_begin = row_start[e];
    const int row_end = row_start[e + 1];
    TileInfo t;
    t.expert = e;
    t.n0 = (local / mt) * p.BN;
    t.row0 = row_begin + (local % mt) * p.BM;
    // The m-tiles of one (expert, n-tile) follow each other in the tile order and read the same weight slab.  Odd
    // ones walk K from the far end, so that what the even one before them read last is read again first, while it
    // is still in L2.
    // (flip_odd: only where one CTA meets these tiles one after another, i.e. in the cut part of the schedule.  Tiles
    // handed out round-robin run at the same time on different SMs and share the slab while both walk it forwards.)
    t.flip = flip_odd ? (local % mt) & 1 : 0;
    t.rows = row_end - t.row0 < p.BM ? row_end - t.row0 : p.BM;
    t.mtile = p.tile_flags_mode ? prefix[e] / p.n_tiles + local % mt : 0;
    return t;
}

// Expert row offsets into shared memory (dense problems: one "expert" holding rows 0..M).
// (Offsets are clamped to 0..M and read past L1: the GEMM kernel reads them once before and once after it has
// waited for its predecessor in the stream, see there.)
__device__ __forceinline__ int clamp_row(int r, int M) { return r < 0 ? 0 : (r > M ? M : r); }
__device__ __forceinline__ void load_row_starts(const GemmParams& p, int* row_start, int skew = 0) {
    for (int e = threadIdx.x; e <= p.E; e += blockDim.x)
        row_start[e] = p.offsets ? clamp_row(__ldcg(p.offsets + e) + skew, p.M) : (e == 0 ? 0 : p.M);
}

// prefix[e] = output tiles of the experts before e (n_tiles x m-tiles each); one warp, shuffle scan.
__device__ __forceinline__ void tile_prefix(const GemmParams& p, const int* row_start, int* prefix) {
    const int lane = threadIdx.x & 31;
    int carry = 0;
    for (int base = 0; base < p.E; base += 32) {
        const int e = base + lane;
        int v = 0;
        if (e < p.E) {
            const int rows = row_start[e + 1] - row_start[e];
            v = rows > 0 ? ((rows + p.BM - 1) / p.BM) * p.n_tiles : 0;
        }
        int incl = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += up;
        }
        if (e < p.E) prefix[e] = carry + incl - v;
        carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) prefix[p.E] = carry;
}

// Shared-memory matrix descriptor: start address, leading and stride byte offsets in 16-byte units; descriptor
// version 1 (bit 46); swizzle mode in bits 61..63: 2 = 128-byte, 4 = 64-byte, 6 = 32-byte.
__host__ __device__ __forceinline__ uint64_t smem_desc_hi(uint32_t lbo, uint32_t sbo, uint32_t layout) {
    return (uint64_t(lbo >> 4) << 16) | (uint64_t(sbo >> 4) << 32) | (uint64_t(1) << 46) | (uint64_t(layout) << 61);
}
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return uint64_t((addr & 0x3FFFFu) >> 4) | smem_desc_hi(lbo, sbo, 2u);
}
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, uint64_t hi) {
    return uint64_t((addr & 0x3FFFFu) >> 4) | hi;
}

__device__ __forceinline__ void epilogue_bar_sync() {
    asm volatile("bar.sync 1, 128;" ::: "memory");
}

// One warp builds one stage of weights on the generic-address path.  The stage is kBK/br runs of kBN/bc whole
// memory tiles; `raw` holds them in memory order, run r at r * kBN*br*2 (bulk copies put them there).  Chunks of 16
// bytes are read in that order; kPieces = rows held by one chunk (1 when a block row is at least 16 bytes).  Rows >=
// k_rows_left and columns >= n_cols_left (tile overhang: nothing was copied there) are filled with zeros.
template <int kBK, int kBN, int kPieces>
__device__ __forceinline__ void generic_fill_stage(uint8_t* sw, const uint8_t* raw, int br_log2,
                                                   int bc_log2, int k_rows_left, int n_cols_left, int lane) {
    // (lane: 0..127 over the four warps that share the stage)
    constexpr int kChunks = kBK * kBN * 2 / 16;
    const int run_log2 = bc_log2 + 1;                       // log2(bytes of one block row)
    const int g_log2 = br_log2 + run_log2;                  // log2(G)
    const int seg_log2 = br_log2 + 1 + (kBN == 64 ? 6 : kBN == 128 ? 7 : 8);   // log2(kBN * br * 2): bytes of one run of tiles
#pragma unroll 1
    for (int base = 0; base < kChunks; base += 128 * 4) {
        uint4 v[4];
        int kl[4], nl[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int byte = (base + i * 128 + lane) << 4;  // byte offset inside the stage's memory image
            const int seg = byte >> seg_log2, o = byte & ((1 << seg_log2) - 1);
            const int ib = o & ((1 << g_log2) - 1);         // byte inside the memory tile
            kl[i] = (seg << br_log2) + (ib >> run_log2);    // Eq. 1 inverted: row and column inside the stage
            nl[i] = ((o >> g_log2) << bc_log2) + ((ib & ((1 << run_log2) - 1)) >> 1);
            v[i] = make_uint4(0, 0, 0, 0);
            if (kl[i] < k_rows_left && nl[i] < n_cols_left)
                v[i] = *reinterpret_cast<const uint4*>(raw + byte);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t word[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
#pragma unroll
            for (int pc = 0; pc < kPieces; ++pc) {
                const int k = kl[i] + pc, n = nl[i];
                uint8_t* dst = sw + (n >> 6) * (kBK * kAtomBytes) + k * kAtomBytes + ((((n & 63) >> 3) ^ (k & 7)) << 4) +
                               (n & 7) * 2;
                if (kPieces == 1) *reinterpret_cast<uint4*>(dst) = v[i];
                else if (kPieces == 2) *reinterpret_cast<uint2*>(dst) = make_uint2(word[2 * pc], word[2 * pc + 1]);
                else if (kPieces == 4) *reinterpret_cast<uint32_t*>(dst) = word[pc];
                else *reinterpret_cast<uint16_t*>(dst) = uint16_t(word[pc >> 1] >> ((pc & 1) * 16));
            }
        }
    }
}

// Where chunk c of a raw stage image (its c-th 16 bytes in memory order) goes in the swizzled operand image: byte
// offset of the chunk, or of its first row piece.  The same for every stage of a launch, so it is tabulated once.
template <int kBK, int kBN>
__device__ __forceinline__ uint32_t generic_chunk_dst(int c, int br_log2, int bc_log2) {
    const int run_log2 = bc_log2 + 1, g_log2 = br_log2 + run_log2;
    const int seg_log2 = br_log2 + 1 + (kBN == 64 ? 6 : kBN == 128 ? 7 : 8);
    const int byte = c << 4;
    const int seg = byte >> seg_log2, o = byte & ((1 << seg_log2) - 1);
    const int ib = o & ((1 << g_log2) - 1);
    const int k = (seg << br_log2) + (ib >> run_log2);      // Eq. 1 inverted
    const int n = ((o >> g_log2) << bc_log2) + ((ib & ((1 << run_log2) - 1)) >> 1);
    return uint32_t((n >> 6) * (kBK * kAtomBytes) + k * kAtomBytes + ((((n & 63) >> 3) ^ (k & 7)) << 4) + (n & 7) * 2);
}

// The same stage build for a stage that lies wholly inside the matrix (no overhang, so no zero fill): per chunk one
// table entry, one 16-byte read and kPieces stores.  A chunk's row pieces sit in consecutive rows kl .. kl + kPieces - 1
// (kl a multiple of kPieces), i.e. 128 bytes apart with the 16-byte column group XOR-ed by the row's low three bits.
template <int kBK, int kBN, int kPieces>
__device__ __forceinline__ void generic_fill_stage_interior(uint8_t* sw, const uint8_t* raw, const uint16_t* tab, int lane) {
    constexpr int kPerLane = kBK * kBN * 2 / 16 / 128;       // lane: 0..127 over the four warps that share the stage
#pragma unroll 4
    for (int i = 0; i < kPerLane; ++i) {
        const int c = i * 128 + lane;
        const uint32_t d0 = tab[c];
        const uint4 v = *reinterpret_cast<const uint4*>(raw + (c << 4));
        if (kPieces == 1) {
            *reinterpret_cast<uint4*>(sw + d0) = v;
        } else {
            const uint32_t word[4] = {v.x, v.y, v.z, v.w};
            const uint32_t k7 = (d0 >> 7) & 7u, nchunk = ((d0 >> 4) & 7u) ^ k7;
#pragma unroll
            for (int pc = 0; pc < kPieces; ++pc) {
                uint8_t* dst = sw + (((d0 + uint32_t(pc) * kAtomBytes) & ~0x70u) | ((nchunk ^ (k7 + uint32_t(pc))) << 4));
                if (kPieces == 2) *reinterpret_cast<uint2*>(dst) = make_uint2(word[2 * pc], word[2 * pc + 1]);
                else if (kPieces == 4) *reinterpret_cast<uint32_t*>(dst) = word[pc];
                else *reinterpret_cast<uint16_t*>(dst) = uint16_t(word[pc >> 1] >> ((pc & 1) * 16));
            }
        }
    }
}

// silu(g) * u in fp32, rounded once to bf16 (nearest even).
__device__ __forceinline__ __nv_bfloat16 swiglu_bf16(float g, float u) {
    return __float2bfloat16_rn(g / (1.0f + expf(-g)) * u);
}

// Tensor-map coordinates of the weight box that starts at K element k and weight column n (kc_expert: the
// expert's offset along the stacked dimension).
__device__ __forceinline__ void weight_box_coords(const GemmParams& p, int k, int n, int kc_expert, int (&c)[5]) {
    c[0] = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i)
        c[i + 1] = ((k >> p.ck_shift[i]) & p.ck_mask[i]) + ((n >> p.cn_shift[i]) & p.cn_mask[i]) + p.c_expert[i] * kc_expert;
}

// Memory tiles of br rows x 4 columns (8-byte rows) or br x 2 columns (4-byte rows), as the copy engine landed them:
// the stage is an array of groups of 2 (or 4) tiles next to each other along N, 16 br bytes each, and a group covers br
// rows x 8 columns.  A 16-byte chunk of a tile holds 2 (or 4) rows of its 4 (or 2) columns; the chunks at the same
// place in the group's tiles hold the same rows.  Writing every row's 2 (or 4) pieces side by side at row * 16 inside
// the same group turns it into a br x 8 memory tile with 16-byte rows, i.e. br/8 core matrices of the no-swizzle
// MN-major operand, which the MMA reads as it is.  In place: a group is handled by one warp, which reads all of it
// before it writes any of it.  8-byte rows: a thread takes the 2 chunks that hold the same row pair and writes 2 rows;
// 4-byte rows: see below.  128 threads (tid 0..127) share the stage; every access lies inside the stage's
// kBK * kBN * 2 bytes of weights.
template <int kBK, int kBN>
__device__ __forceinline__ void fixup_stage_in_place(uint8_t* sw, int br_log2, int bc_log2, int tid) {
    const uint32_t group_bytes = 16u << br_log2;
    // (kBatch work items have their loads in flight together: all reads, then all writes)
    if (bc_log2 == 2) {
        constexpr int kItems = kBK * kBN / 16;
        constexpr int kBatch = kItems >= 1024 ? 8 : (kItems >= 512 ? 4 : kItems / 128);
        static_assert(kItems % (128 * kBatch) == 0, "whole batches");
        const int tpg_log2 = br_log2 - 1;                          // threads per group: one per pair of rows
        const uint32_t tile_bytes = 8u << br_log2;
        // Item i writes rows 2i and 2i+1 of the finished image, 32 bytes at i * 32.  Of every eight lanes four write their
        // second row first, so that the eight 16-byte stores of a quarter warp fall into eight different bank groups
        // (stores 32 bytes apart would pair up).  Those lanes fetch the two 8-byte halves of each chunk in the other
        // order, so the rows come out of the loads in the order they are stored and no register has to be picked;
        // which lanes: such that lanes l and l + 8 differ, which keeps the sixteen 8-byte loads of a half warp apart too.
        const uint32_t hi_first = ((uint32_t(tid) >> 2) ^ (uint32_t(tid) >> 3)) & 1u;
        const uint32_t src0 = (uint32_t(tid) >> tpg_log2) * group_bytes + (uint32_t(tid) & ((1u << tpg_log2) - 1)) * 16u;
        const uint32_t h0 = hi_first * 8u, h1 = 8u - h0;
        // (128 items further = 4096 bytes further: a group of br / 2 items is 16 br bytes)
        for (int it = 0; it < kItems / (128 * kBatch); ++it) {
            uint2 a0[kBatch], a1[kBatch], b0[kBatch], b1[kBatch];
#pragma unroll
            for (int j = 0; j < kBatch; ++j) {
                const uint8_t* src = sw + src0 + uint32_t(it * kBatch + j) * 4096u;
                a0[j] = *reinterpret_cast<const uint2*>(src + h0);                // one row x columns 0..3
                a1[j] = *reinterpret_cast<const uint2*>(src + h1);                // the other row
                b0[j] = *reinterpret_cast<const uint2*>(src + tile_bytes + h0);   // x columns 4..7
                b1[j] = *reinterpret_cast<const uint2*>(src + tile_bytes + h1);
            }
            __syncwarp();
#pragma unroll
            for (int j = 0; j < kBatch; ++j) {
                uint8_t* dst = sw + size_t(tid + (it * kBatch + j) * 128) * 32;
                *reinterpret_cast<uint4*>(dst + 2 * h0) = make_uint4(a0[j].x, a0[j].y, b0[j].x, b0[j].y);
                *reinterpret_cast<uint4*>(dst + 2 * h1) = make_uint4(a1[j].x, a1[j].y, b1[j].x, b1[j].y);
            }
        }
    } else {
        // 4-byte rows: word by word.  A warp takes 512 bytes = 32 rows of the finished image at a time; lane l owns one
        // row and fetches its 4-byte piece from each of the group's four tiles with four 32-bit loads, then stores the four
        // pieces side by side.  Lanes take the tiles in different orders (tile (j + lane / 8) % 4 in
        // step j), which spreads every load and store over all banks; all offsets are per-lane constants, the loop adds
        // only the block's base.  (A 4 x 4 word transpose between lanes with shuffles took three times the instructions
        // and ran at 1.3-1.4 x the row-major time where this form runs at 1.15-1.25 x; 16-byte loads of whole chunks as
        // above would hit each bank four times for 8-row tiles.)  A warp works through batches of four consecutive
        // blocks, all loads first, then all stores: a group (at most 128 rows = four blocks) is read completely before
        // any of it is overwritten, and no other warp touches it.
        constexpr int kBlocks = kBK * kBN * 2 / 512;               // 512-byte blocks per stage
        constexpr int kBatch = kBlocks >= 16 ? 4 : kBlocks / 4;
        static_assert(kBlocks % (4 * kBatch) == 0, "whole batches");
        const int lane = tid & 31, wrp = tid >> 5;
        const bool small = br_log2 < 5;                             // several whole groups per block
        const int k = small ? lane & ((1 << br_log2) - 1) : lane;   // row inside the group (small) or inside the block
        const int gl = small ? lane >> br_log2 : 0;
        const uint32_t grp = uint32_t(gl) << (br_log2 + 4);
        const int spg_log2 = small ? 0 : br_log2 - 5;               // blocks per group
        uint32_t src_off[4], dst_off[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t pj = uint32_t(j + (lane >> 3)) & 3u;
            src_off[j] = grp + (pj << (br_log2 + 2)) + uint32_t(k) * 4u;
            dst_off[j] = grp + uint32_t(k) * 16u + pj * 4u;
        }
        for (int b0 = wrp * kBatch; b0 < kBlocks; b0 += 4 * kBatch) {
            uint32_t v[kBatch][4];
#pragma unroll
            for (int i = 0; i < kBatch; ++i) {
                const int b = b0 + i;
                // (tiles of 32 rows and more: the block's rows come from its group's tiles, 128 bytes further per block
                // inside each tile)
                const uint8_t* src = small ? sw + size_t(b) * 512
                                           : sw + (size_t(b >> spg_log2) << (br_log2 + 4)) + size_t(b & ((1 << spg_log2) - 1)) * 128;
#pragma unroll
                for (int j = 0; j < 4; ++j) v[i][j] = *reinterpret_cast<const uint32_t*>(src + src_off[j]);
            }
            __syncwarp();
#pragma unroll
            for (int i = 0; i < kBatch; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) *reinterpret_cast<uint32_t*>(sw + size_t(b0 + i) * 512 + dst_off[j]) = v[i][j];
        }
    }
}

// kBK: weight rows per stage (64 or 128).  kBN: weight columns per CTA tile (64, 128 or 256).
// kWN selects which side of the MMA the weights are on.  The tensor pipe takes N/2 clocks per MMA whatever M is,
// and the thread that issues the MMAs runs alone in its warp (every scalar instruction between two MMAs costs it
// several clocks), so for small token tiles what matters is how many weight bytes one instruction consumes:
//   kWN = false  weights on the M side: kBN/128 MMAs per K step, each 128 (or 64) weight columns x up to 256
//                tokens.  For prefill (256-token tiles): the accumulator is C transposed, TMEM lane = weight
//                column, and the epilogue writes 128-byte row segments.
//   kWN = true   weights on the N side: one MMA per K step covers all kBN (up to 256) weight columns, tokens
//                (at most 128 per tile) on the M side.  For decode and MoE: 8 KB of weights per instruction
//                instead of 4 KB, half as many instructions per byte streamed.  TMEM lane =
//                token, and every thread writes its token's row of C in 16-byte pieces.
// (The body is a device function so that one kernel can run two products one after the other, see gemm_chain_kernel:
// alloc_tmem / free_tmem say whether this call allocates tensor memory at its start and frees it at its end.)
template <int kBK, int kBN, bool kWN, bool kFp8>
__device__ __forceinline__ void gemm_body(const GemmParams& p, bool alloc_tmem, bool free_tmem) {
    constexpr int kNumN = kWN ? 1 : (kBN >= 128 ? kBN / 128 : 1);     // MMAs per K step
    constexpr int kUmmaM = kWN ? 128 : (kBN >= 128 ? 128 : 64);       // rows of the MMA's M side
    constexpr int kKSteps = kBK / 16;
    constexpr int kSubK = kBK / 64;                        // token boxes per stage
    constexpr uint32_t kWBytes = kBK * kBN * 2;            // weight bytes per stage
    constexpr int kStagePitch = kBN + 4;                   // floats between rows of a partial tile kept in shared memory

    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
    __shared__ __align__(8) uint64_t raw_full_bar[kMaxStages];      // generic path: raw image landed / raw image consumed
    __shared__ __align__(8) uint64_t raw_empty_bar[kMaxStages];
    __shared__ __align__(8) uint64_t acc_full_bar[2];
    __shared__ __align__(8) uint64_t acc_empty_bar[2];
    __shared__ uint32_t tmem_slot;
    __shared__ uint32_t abort_flag;
    __shared__ int prefix[kMaxExperts + 1];
    __shared__ int row_start[kMaxExperts + 1];      // copy of the expert row offsets (dense: 0, M)
    __shared__ int range_tab[kRangeTabMax + 1];     // stream-K: first flattened iteration of every CTA

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t stage_bytes = kWBytes + uint32_t(kSubK) * p.a_rows * kAtomBytes;
    uint8_t* stages = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

    const int acc_cols = kWN ? kBN : p.BM;                   // TMEM columns of one MMA's accumulator
    uint32_t tmem_cols = 32;
    while (tmem_cols < uint32_t(2 * kNumN * acc_cols)) tmem_cols <<= 1;

    // ---------------------------------------------------------------- set-up
    if (threadIdx.x == 0) {
        // (generic_b == 1: the producer and the four permuting warps arrive on a stage's "full" barrier; generic_b == 2:
        // the copies land on raw_full_bar[stage] and the four warps that fix the stage up arrive on "full")
        for (int s = 0; s < p.num_stages; ++s) {
            mbar_init(&full_bar[s], p.generic_b == 1 ? 5 : p.generic_b == 2 ? 4 : 1);
            mbar_init(&empty_bar[s], 1);
            if (p.generic_b == 2) mbar_init(&raw_full_bar[s], 1);
        }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full_bar[b], 1); mbar_init(&acc_empty_bar[b], 4); }
        if (p.generic_b == 1)
            for (int r = 0; r < p.raw_slots; ++r) { mbar_init(&raw_full_bar[r], 1); mbar_init(&raw_empty_bar[r], 4); }
        abort_flag = 0;
        fence_mbar_init();
        if (p.generic_b != 1) tma_prefetch_desc(&p.tmap_b);
        for (int i = 0; i < kNumBoxChoices; ++i) tma_prefetch_desc(&p.tmap_a[i]);
    }
    if (warp == 1 && alloc_tmem) {
        tmem_alloc(&tmem_slot, tmem_cols);
        tmem_relinquish();
    }
    // Token rows between BM and the rows the MMA reads are zeroed once; no copy ever writes them.  (The MMA's token
    // side has at least 64 rows.  Whatever lies there is multiplied with the weights at full rate, and with stale
    // data instead of zeros the tensor pipe draws enough power to pull the SM clock down under the board's cap.)
    if (p.a_rows > p.BM && warp >= 2) {
        const int per = (p.a_rows - p.BM) * (kAtomBytes / 16);          // 16-byte pieces per 64-wide K slice
        const int total = p.num_stages * kSubK * per;
        for (int i = int(threadIdx.x) - 64; i < total; i += int(blockDim.x) - 64) {
            const int s = i / (kSubK * per), r = i % (kSubK * per);
            uint8_t* slice = stages + size_t(s) * stage_bytes + kWBytes + size_t(r / per) * p.a_rows * kAtomBytes;
            *reinterpret_cast<uint4*>(slice + size_t(p.BM) * kAtomBytes + size_t(r % per) * 16) = make_uint4(0, 0, 0, 0);
        }
        fence_proxy_async_smem();
    }
    // Launched with programmatic stream serialisation: everything up to the wait below (barriers, tensor memory,
    // descriptor prefetch, the schedule's tables, a prefetch of the first weights into L2) may run while the kernel
    // before this one in the stream is still finishing.  Nothing that kernel may have written (tokens, the
    // partial-tile workspace, C) is used before the wait, which returns once it has completed and its writes are
    // visible.  Dense problems build their tables from the launch parameters alone.  Grouped problems read the
    // expert offsets, which that kernel may still be writing: the tables built before the wait are provisional
    // (offsets clamped to 0..M, so that whatever was read gives bounded arithmetic), the offsets are read again
    // after the wait, and the tables are rebuilt if a single one differs.
    // generic-address path: the chunk table (see generic_chunk_dst), after the raw ring
    if (p.generic_b == 1 && warp >= 6 && warp < 10) {
        uint16_t* tab = reinterpret_cast<uint16_t*>(stages + size_t(p.num_stages) * stage_bytes + size_t(p.raw_slots) * kWBytes);
        for (int c = int(threadIdx.x) - 192; c < int(kWBytes / 16); c += 128)
            tab[c] = uint16_t(generic_chunk_dst<kBK, kBN>(c, p.br_log2, p.bc_log2));
    }
    int tiles_total = 0;
    Sched sched;
    auto build_tables = [&](int skew) {
        // tiles before each expert (dense: one "expert" holding all M rows)
        load_row_starts(p, row_start, skew);
        __syncthreads();
        if (warp == 2) tile_prefix(p, row_start, prefix);
        __syncthreads();
        tiles_total = prefix[p.E];
        // Range starts of all CTAs, once, so that nothing on the critical path divides 64-bit numbers.
        // (of the part of the schedule that is cut along K: the tiles left after the whole rounds)
        const long long total_iters =
            static_cast<long long>(tiles_total - Sched::whole_rounds_tiles(tiles_total, gridDim.x, p.k_iters)) * p.k_iters;
        const int grid_eff0 = Sched::effective_grid(total_iters, gridDim.x);
        const bool use_tab = p.stream_k && grid_eff0 > 0 && grid_eff0 <= kRangeTabMax && total_iters < (1ll << 31);
        if (use_tab) {
            for (int c = threadIdx.x; c <= grid_eff0; c += blockDim.x)
                range_tab[c] = static_cast<int>(Sched::split(total_iters, grid_eff0, c));
        }
        __syncthreads();
        if (p.cluster_k > 1) sched.init_cluster(p.k_iters, tiles_total, int(cluster_id_x()), int(cluster_cta_rank()), p.cluster_k);
        else sched.init(p.stream_k, p.k_iters, tiles_total, gridDim.x, blockIdx.x, use_tab ? range_tab : nullptr);
    };
    build_tables(p.provisional_skew);          // (test hook: wrong on purpose, so that the check below fails)
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_slot;
    // While the kernel before this one in the stream is still finishing, ask for the first stages of this CTA's
    // weights to be brought into L2.  A prefetch delivers nothing to the SM and L2 is the point of coherence, so
    // this is safe whatever that kernel is still writing (and whatever the provisional tables of a grouped problem
    // point at: coordinates outside the tensor are skipped by the copy engine); it takes the cold start (page walks,
    // first DRAM accesses) off this kernel's critical path.
    // (issued by an epilogue thread, which has nothing else to do yet, so that the producer is not held up)
    if (threadIdx.x == 64 && p.generic_b != 1 && p.prefetch_stages > 0) {
        Sched first = sched;
        Work w;
        if (first.next(w)) {
            const TileInfo t = decode_tile(p, prefix, row_start, w.tile, first.stream_k == 1 && w.tile >= first.dp_tiles);
            const int kc_expert = t.expert * p.k_coord_per_expert;
            for (int s = 0, kit = w.kbeg; s < p.prefetch_stages && kit < w.kend; ++s, ++kit) {
                const int kq = t.flip ? p.k_iters - 1 - kit : kit;
                const int k0 = (kq * kBK) << p.k_shift;
                for (int kb = 0; kb < p.kbx; ++kb)
                    for (int nb = 0; nb < p.nbx; ++nb) {
                        int c[5];
                        weight_box_coords(p, k0 + kb * p.box_rows, t.n0 + nb * p.box_atoms * 64, kc_expert, c);
                        tma_prefetch_5d(&p.tmap_b, c[0], c[1], c[2], c[3], c[4]);
                    }
            }
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (p.offsets != nullptr) {
        int differs = 0;
        for (int e = threadIdx.x; e <= p.E; e += blockDim.x) differs |= row_start[e] != clamp_row(__ldcg(p.offsets + e), p.M);
        if (__syncthreads_or(differs)) build_tables(0);
    }
    // Let the kernel that follows in the stream (the stream-K reduction, or the next product) be scheduled already:
    // it does its own set-up and then blocks until this whole grid has finished.
    if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    volatile uint32_t* abort_ptr = &abort_flag;

    if (warp == 0) {
        // ============================================================ TMA producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            uint32_t issued = 0;
            Work w;
            bool ok = true;
            // the K part of the coordinate maps, in registers for the whole loop
            const bool one_box = p.kbx == 1 && p.nbx == 1;
            uint64_t* land_bar = p.generic_b == 2 ? raw_full_bar : full_bar;      // where a stage's copies are counted
            int ks[4], km[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { ks[i] = p.ck_shift[i]; km[i] = p.ck_mask[i]; }
            while (ok && sched.next(w)) {
                const TileInfo t = decode_tile(p, prefix, row_start, w.tile, sched.stream_k == 1 && w.tile >= sched.dp_tiles);
                int bi = 0;
                while ((16 << bi) < t.rows) ++bi;
                const uint32_t a_bytes = uint32_t(16 << bi) * kAtomBytes;
                const uint32_t tx = uint32_t(kSubK) * a_bytes + uint32_t(p.kbx * p.nbx) * p.box_bytes;
                const int kc_expert = t.expert * p.k_coord_per_expert;
                int cn[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) cn[i] = ((t.n0 >> p.cn_shift[i]) & p.cn_mask[i]) + p.c_expert[i] * kc_expert;
                if (p.tile_flags_mode == 2) {
                    // The tile's token rows are another product's output, written by other CTAs of this launch: wait
                    // (bounded) until every warp that stores a part of this m-tile has said so (each of them has ordered
                    // its stores before the copy engine's reads by a proxy fence of its own).
                    const uint32_t* flag = p.tile_flags + t.mtile;
                    uint64_t t0 = 0;
                    uint32_t polls = 0;
                    while (true) {
                        uint32_t seen;
                        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(flag) : "memory");
                        if (seen >= p.tile_flags_target) break;
                        __nanosleep(64);
                        if ((++polls & 63u) == 0) {
                            const uint64_t now = global_timer_ns();
                            if (t0 == 0) t0 = now;
                            if (*abort_ptr || now - t0 > p.wait_limit_ns) {
                                atomicCAS(p.status, 0u, kWaitTileFlag);
                                *abort_ptr = 1;
                                ok = false;
                                break;
                            }
                        }
                    }
                    if (!ok) break;
                    asm volatile("fence.proxy.async.global;" ::: "memory");     // (and on the reading side as well)
                }
                for (int kit = w.kbeg; kit < w.kend; ++kit) {
                    if (!mbar_wait_bounded(&empty_bar[stage], phase ^ 1, abort_ptr, p.status, kWaitProducerEmpty, p.wait_limit_ns)) {
                        ok = false;
                        break;
                    }
                    uint8_t* sw = stages + size_t(stage) * stage_bytes;
                    uint8_t* sa = sw + kWBytes;
                    // (test hook: the first stage of every CTA may be armed for more bytes than its copies deliver, so
                    // that the wait on it runs out and the give-up path below is exercised)
                    mbar_arrive_expect_tx(&land_bar[stage], issued == 0 ? tx + p.stall_extra_tx : tx);
                    const int kq = t.flip ? p.k_iters - 1 - kit : kit;
                    const int k0 = (kq * kBK) << p.k_shift;         // first K element of the stage
#pragma unroll
                    for (int sub = 0; sub < kSubK; ++sub)
                        tma_load_2d(sa + size_t(sub) * p.a_rows * kAtomBytes, &p.tmap_a[bi], &land_bar[stage],
                                    k0 + ((sub * 64) << p.k_shift), t.row0);
                    if (one_box) {
                        // the usual case, one box per stage: the column part of the coordinates was worked out once
                        // for the tile, only the K part changes from stage to stage
                        tma_load_5d(sw, &p.tmap_b, &land_bar[stage], 0, ((k0 >> ks[0]) & km[0]) + cn[0],
                                    ((k0 >> ks[1]) & km[1]) + cn[1], ((k0 >> ks[2]) & km[2]) + cn[2],
                                    ((k0 >> ks[3]) & km[3]) + cn[3]);
                    } else {
                        for (int kb = 0; kb < p.kbx; ++kb) {
                            const int k = k0 + kb * p.box_rows;
                            for (int nb = 0; nb < p.nbx; ++nb) {
                                const int n = t.n0 + nb * p.box_atoms * 64;
                                uint8_t* dst = sw + size_t(kb * p.nbx + nb) * p.box_bytes;
                                int c[5];
                                weight_box_coords(p, k, n, kc_expert, c);
                                tma_load_5d(dst, &p.tmap_b, &land_bar[stage], c[0], c[1], c[2], c[3], c[4]);
                            }
                        }
                    }
                    ++issued;
                    if (++stage == uint32_t(p.num_stages)) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok || *abort_ptr) {
                // Giving up: let the copies already issued land before the CTA's shared memory goes away.
                uint32_t s = stage, ph = phase;
                const uint32_t back = issued < uint32_t(p.num_stages) ? issued : uint32_t(p.num_stages);
                for (uint32_t i = 0; i < back; ++i) {
                    if (s == 0) { s = p.num_stages; ph ^= 1; }
                    --s;
                    const uint64_t t0 = global_timer_ns();
                    const uint64_t drain_ns = p.wait_limit_ns < 20000000ull ? p.wait_limit_ns : 20000000ull;
                    while (!mbar_try_wait(&land_bar[s], ph) && global_timer_ns() - t0 < drain_ns) {}
                }
            }
        }
    } else if (warp == 1) {
        // ============================================================= MMA issuer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            Work w;
            bool ok = true;
            // Descriptor words that do not change: the upper halves, the constant bits of the lower halves, and
            // the (address >> 4) offsets of every K step (kept in registers: the loop below adds one per MMA).
            const uint64_t tok_hi64 = smem_desc_hi(16u, 1024u, 2u);
            const uint32_t tok_hi = uint32_t(tok_hi64 >> 32), tok_lo_const = uint32_t(tok_hi64);
            const uint32_t w_hi = uint32_t(p.w_desc_hi >> 32), w_lo_const = uint32_t(p.w_desc_hi);
            uint32_t w_off[kKSteps], tok_off[kKSteps];
#pragma unroll
            for (int j = 0; j < kKSteps; ++j) {
                w_off[j] = p.kstep_off[j] >> 4;
                tok_off[j] = (uint32_t(j >> 2) * uint32_t(p.a_rows) * kAtomBytes + uint32_t(j & 3) * 32u) >> 4;
            }
            const uint32_t ugroup16 = p.ugroup_off >> 4;
            // Tiles of two 128-row token blocks (weights on N, BM = 256): every K step is issued twice, on the same
            // weight slab, into the two accumulators, which then both belong to the tile.
            const bool two_blocks = kWN && p.BM > 128;
            while (ok && sched.next(w)) {
                const TileInfo t = decode_tile(p, prefix, row_start, w.tile);
                const uint32_t n_mma = kWN ? uint32_t(kBN) : uint32_t((t.rows + 15) & ~15);
                // fp32 accumulate, bf16 x bf16; the weights operand is MN-major (bit 15: A, bit 16: B), the token
                // operand K-major; M = kUmmaM, N = n_mma
                const uint32_t w_major = p.w_kmajor ? 0u : (kWN ? (1u << 16) : (1u << 15));
                // (8-bit operands: format codes 0 = E4M3 in place of 1 = bf16)
                // (weights on N: 64-row instructions for tiles of up to 64 tokens unless the launch asks for 128 rows always)
                const uint32_t m_mma = kWN ? (p.umma_m == 64 && t.rows <= 64 ? 64u : 128u) : uint32_t(kUmmaM);
                const uint32_t idesc = (1u << 4) | (kFp8 ? 0u : (1u << 7) | (1u << 10)) | w_major |
                                       ((n_mma >> 3) << 17) | ((m_mma >> 4) << 24);
                if (!mbar_wait_bounded(&acc_empty_bar[acc], acc_phase ^ 1, abort_ptr, p.status, kWaitMmaAccEmpty, p.wait_limit_ns)) {
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * uint32_t(kNumN * acc_cols);
                // (the loop exists twice so that the usual one carries nothing for the second token block: the issuing
                // thread has no slack)
                auto k_loop = [&](auto second_block) {
                    for (int kit = w.kbeg; kit < w.kend; ++kit) {
                        if (!mbar_wait_bounded(&full_bar[stage], phase, abort_ptr, p.status, kWaitMmaFull, p.wait_limit_ns)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after_sync();
                        const uint32_t sw = smem_u32(stages + size_t(stage) * stage_bytes);
                        const uint32_t w_lo0 = w_lo_const | ((sw & 0x3FFFFu) >> 4);
                        const uint32_t tok_lo0 = tok_lo_const | (((sw + kWBytes) & 0x3FFFFu) >> 4);
                        const uint32_t first = kit > w.kbeg ? 1u : 0u;
#pragma unroll
                        for (int j = 0; j < kKSteps; ++j) {
#pragma unroll
                            for (int u = 0; u < kNumN; ++u) {
                                const uint32_t accum = j > 0 ? 1u : first;
                                const uint32_t w_lo = w_lo0 + w_off[j] + uint32_t(u) * ugroup16;
                                if (kWN) {
                                    umma_split<kFp8>(d_tmem, tok_lo0 + tok_off[j], tok_hi, w_lo, w_hi, idesc, accum);
                                    if (decltype(second_block)::value)   // rows 128.. of the token slab: 128 swizzle rows further
                                        umma_split<kFp8>(d_tmem + uint32_t(kBN), tok_lo0 + tok_off[j] + ((128u * kAtomBytes) >> 4),
                                                         tok_hi, w_lo, w_hi, idesc, accum);
                                } else {
                                    umma_split<kFp8>(d_tmem + uint32_t(u * acc_cols), w_lo, w_hi, tok_lo0 + tok_off[j], tok_hi, idesc,
                                                     accum);
                                }
                            }
                        }
                        umma_commit(&empty_bar[stage]);      // frees the stage once these MMAs have read it
                        if (++stage == uint32_t(p.num_stages)) { stage = 0; phase ^= 1; }
                    }
                };
                if (kWN && two_blocks && t.rows > 128) k_loop(tl_true{});
                else k_loop(tl_false{});
                if (!ok) break;
                umma_commit(&acc_full_bar[acc]);         // accumulator complete
                if (!two_blocks) acc ^= 1;               // (two blocks: the tile owned both accumulators)
                if (acc == 0) acc_phase ^= 1;
            }
        }
    } else if (warp == 10 && p.generic_b == 1) {
        // ================================ generic-address path: raw memory tiles -> shared memory
        // A stage's weights are kBK/br runs of whole memory tiles, each run contiguous in the tile-major buffer
        // (Eq. 1-2: tiles follow each other along a row of the tile grid).  One untiled bulk copy per run brings them
        // into a ring of raw stage images, several stages ahead of the warps that permute them: the copy engine
        // keeps the bytes in flight, no thread holds them in registers.  Lane l issues runs l, l + 32, ...
        const int br = 1 << p.br_log2;
        const int G = br << (p.bc_log2 + 1);
        const uint32_t run_full = uint32_t(kBN) * br * 2;                 // one run of tiles that spans the CTA tile
        uint8_t* raw_ring = stages + size_t(p.num_stages) * stage_bytes;
        uint32_t slot = 0, phase = 0, issued = 0;
        Work w;
        bool ok = true;
        while (ok && sched.next(w)) {
            const TileInfo t = decode_tile(p, prefix, row_start, w.tile, sched.stream_k == 1 && w.tile >= sched.dp_tiles);
            const uint8_t* Bexp = p.B + int64_t(t.expert) * p.expert_bytes;
            const int nblk0 = t.n0 >> p.bc_log2;
            const int n_cols = p.N - t.n0 < kBN ? p.N - t.n0 : kBN;
            const uint32_t run_bytes = uint32_t(n_cols >> p.bc_log2) * uint32_t(G);      // whole memory tiles inside the matrix
            for (int kit = w.kbeg; kit < w.kend; ++kit) {
                int got = 1;
                if (lane == 0)
                    got = mbar_wait_bounded(&raw_empty_bar[slot], phase ^ 1, abort_ptr, p.status, kWaitProducerEmpty, p.wait_limit_ns);
                if (!__shfl_sync(0xffffffffu, got, 0)) { ok = false; break; }
                const int kq = t.flip ? p.k_iters - 1 - kit : kit;
                const int k_rows = p.K - kq * kBK < kBK ? p.K - kq * kBK : kBK;
                const int runs = k_rows >> p.br_log2;
                if (lane == 0) mbar_arrive_expect_tx(&raw_full_bar[slot], uint32_t(runs) * run_bytes);
                __syncwarp();
                const uint8_t* src0 = Bexp + (int64_t((kq * kBK) >> p.br_log2) * p.blocks_per_row + nblk0) * G;
                uint8_t* dst0 = raw_ring + size_t(slot) * kWBytes;
                for (int r = lane; r < runs; r += 32) {
                    uint8_t* dst = dst0 + size_t(r) * run_full;
                    const uint8_t* src = src0 + int64_t(r) * p.blocks_per_row * G;
                    // A copy that would leave the weight buffer or this CTA's shared memory, or is not 16-byte
                    // granular, is not issued: the status word says so and the kernel gives up in the bounded way.
                    const bool fine = src >= p.B && src + run_bytes <= p.B + p.b_bytes && dst >= smem_raw &&
                                      dst + run_bytes <= smem_raw + p.smem_limit && run_bytes > 0 && (run_bytes & 15u) == 0 &&
                                      (reinterpret_cast<uintptr_t>(src) & 15u) == 0 && (smem_u32(dst) & 15u) == 0;
                    if (fine) {
                        bulk_load_1d(dst, src, run_bytes, &raw_full_bar[slot]);
                    } else {
                        atomicCAS(p.status, 0u, kBadCopy);
                        *abort_ptr = 1;
                    }
                }
                ++issued;
                if (++slot == uint32_t(p.raw_slots)) { slot = 0; phase ^= 1; }
            }
        }
        if (lane == 0 && (!ok || *abort_ptr)) {
            // Giving up: let the copies already issued land before the CTA's shared memory goes away.
            uint32_t s = slot, ph = phase;
            const uint32_t back = issued < uint32_t(p.raw_slots) ? issued : uint32_t(p.raw_slots);
            for (uint32_t i = 0; i < back; ++i) {
                if (s == 0) { s = p.raw_slots; ph ^= 1; }
                --s;
                const uint64_t t0 = global_timer_ns();
                const uint64_t drain_ns = p.wait_limit_ns < 20000000ull ? p.wait_limit_ns : 20000000ull;
                while (!mbar_try_wait(&raw_full_bar[s], ph) && global_timer_ns() - t0 < drain_ns) {}
            }
        }
    } else if (warp >= 6 && p.generic_b == 2) {
        // ================================ memory tiles with 8- or 4-byte rows: fixed up where the copy engine put them
        // Every warp takes part in every stage, in order (a parity wait cannot tell two phases apart).
        if (warp < 10) {
            const int tid = (warp - 6) * 32 + lane;
            uint32_t it_global = 0;
            Work w;
            bool ok = true;
            while (ok && sched.next(w)) {
                for (int kit = w.kbeg; kit < w.kend; ++kit, ++it_global) {
                    const uint32_t stage = it_global % uint32_t(p.num_stages);
                    const uint32_t phase = (it_global / uint32_t(p.num_stages)) & 1u;
                    if (!mbar_wait_bounded(&raw_full_bar[stage], phase, abort_ptr, p.status, kWaitMmaFull, p.wait_limit_ns)) {
                        ok = false;
                        break;
                    }
                    fixup_stage_in_place<kBK, kBN>(stages + size_t(stage) * stage_bytes, p.br_log2, p.bc_log2, tid);
                    fence_proxy_async_smem();            // generic-proxy stores -> visible to the tensor-core (async) proxy
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&full_bar[stage]);
                }
                if (*abort_ptr) break;
            }
        }
    } else if (warp >= 6) {
        // ================================ generic-address weight operand (Section 4.4 of the paper)
        // Memory tiles whose rows are shorter than a TMA box allows.  The raw image of a stage (its memory tiles in
        // memory order) is read in 16-byte chunks; Eq. 1 inverted gives every chunk's (row, column), and the chunk
        // (or its 16/(2 bc) row pieces) is stored where the 128-byte-swizzled MN-major operand layout wants it.
        // The four warps share every stage (a quarter of its chunks each) and each arrives on the stage's barriers.
        // Every warp takes part in every iteration, in order, so the barrier it polls is never more than one phase
        // behind the one it asks for (a parity wait cannot tell two phases apart).
        const int lane4 = (warp - 6) * 32 + lane;
        const int run_bytes = 2 << p.bc_log2;                      // one block row
        const int pieces = run_bytes >= 16 ? 1 : 16 / run_bytes;  // rows held by one 16-byte chunk
        const uint8_t* raw_ring = stages + size_t(p.num_stages) * stage_bytes;
        const uint16_t* tab = reinterpret_cast<const uint16_t*>(raw_ring + size_t(p.raw_slots) * kWBytes);
        uint32_t it_global = 0;
        Work w;
        bool ok = true;
        while (ok && sched.next(w)) {
            const TileInfo t = decode_tile(p, prefix, row_start, w.tile, sched.stream_k == 1 && w.tile >= sched.dp_tiles);
            for (int kit = w.kbeg; kit < w.kend; ++kit, ++it_global) {
                const uint32_t stage = it_global % uint32_t(p.num_stages);
                const uint32_t phase = (it_global / uint32_t(p.num_stages)) & 1u;
                const uint32_t slot = it_global % uint32_t(p.raw_slots);
                const uint32_t raw_phase = (it_global / uint32_t(p.raw_slots)) & 1u;
                if (!mbar_wait_bounded(&empty_bar[stage], phase ^ 1, abort_ptr, p.status, kWaitProducerEmpty, p.wait_limit_ns) ||
                    !mbar_wait_bounded(&raw_full_bar[slot], raw_phase, abort_ptr, p.status, kWaitMmaFull, p.wait_limit_ns)) {
                    ok = false;
                    break;
                }
                uint8_t* sw = stages + size_t(stage) * stage_bytes;
                const uint8_t* raw = raw_ring + size_t(slot) * kWBytes;
                const int kq = t.flip ? p.k_iters - 1 - kit : kit;
                const int k_rows_left = p.K - kq * kBK, n_cols_left = p.N - t.n0;
                if (k_rows_left >= kBK && n_cols_left >= kBN) {
                    switch (pieces) {
                        case 1: generic_fill_stage_interior<kBK, kBN, 1>(sw, raw, tab, lane4); break;
                        case 2: generic_fill_stage_interior<kBK, kBN, 2>(sw, raw, tab, lane4); break;
                        case 4: generic_fill_stage_interior<kBK, kBN, 4>(sw, raw, tab, lane4); break;
                        default: generic_fill_stage_interior<kBK, kBN, 8>(sw, raw, tab, lane4); break;
                    }
                } else {
                    switch (pieces) {
                        case 1: generic_fill_stage<kBK, kBN, 1>(sw, raw, p.br_log2, p.bc_log2, k_rows_left, n_cols_left, lane4); break;
                        case 2: generic_fill_stage<kBK, kBN, 2>(sw, raw, p.br_log2, p.bc_log2, k_rows_left, n_cols_left, lane4); break;
                        case 4: generic_fill_stage<kBK, kBN, 4>(sw, raw, p.br_log2, p.bc_log2, k_rows_left, n_cols_left, lane4); break;
                        default: generic_fill_stage<kBK, kBN, 8>(sw, raw, p.br_log2, p.bc_log2, k_rows_left, n_cols_left, lane4); break;
                    }
                }
                fence_proxy_async_smem();            // generic-proxy stores -> visible to the tensor-core (async) proxy
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(&full_bar[stage]);
                    mbar_arrive(&raw_empty_bar[slot]);   // the raw image has been read: its slot may be overwritten
                }
            }
        }
    } else {
        // =============================================================== epilogue
        const int quarter = warp & 3;                    // TMEM lanes 32*quarter .. +31
        uint32_t acc = 0, acc_phase = 0;
        Work w;
        while (sched.next(w)) {
            const TileInfo t = decode_tile(p, prefix, row_start, w.tile);
            const bool full = (w.kbeg == 0 && w.kend == p.k_iters);
            const int n_mma = (t.rows + 15) & ~15;
            bool ok = mbar_wait_bounded(&acc_full_bar[acc], acc_phase, abort_ptr, p.status, kWaitEpilogueAccFull, p.wait_limit_ns);
            tc_fence_after_sync();
            float* out;
            int64_t ld;
            if (full) {
                out = p.C + int64_t(t.row0) * p.ldc + t.n0;
                ld = p.ldc;
            } else if (p.cluster_k > 1) {
                // cluster split-K: the partial tile stays in this CTA's shared memory (the pipeline's stages are
                // free: this CTA has one work item and its last MMA has completed), rows kStagePitch floats apart
                out = reinterpret_cast<float*>(stages);
                ld = kStagePitch;
            } else {
                out = p.partials + size_t(sched.slot(sched.cta, w.tile)) * p.BM * kBN;
                ld = kBN;
            }
            if (ok && kWN) {
                // TMEM lane = token row, columns = the tile's kBN weight columns: each thread owns one row of C.
                // (MMA of 64 rows: rows 16q..16q+15 sit in the lower half of lane quarter q, the upper 16 lanes of
                // each quarter hold nothing.)
                const bool m64 = p.umma_m == 64 && t.rows <= 64;
                // (tiles of two 128-row token blocks, BM = 256: the second block's rows sit in the second accumulator)
                const int blocks = p.BM > 128 && t.rows > 128 ? 2 : 1;
                for (int blk = 0; blk < blocks; ++blk) {
                const int row = m64 ? (lane < 16 ? quarter * 16 + lane : p.BM) : blk * 128 + quarter * 32 + lane;
                const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + (acc + uint32_t(blk)) * uint32_t(acc_cols);
                if ((m64 ? quarter * 16 : blk * 128 + quarter * 32) < t.rows) {      // this lane quarter holds at least one real row
                    float* dst = out + int64_t(row) * ld;
                    const bool gated = full && p.epi_swiglu;
                    __nv_bfloat16* hdst = p.H + int64_t(t.row0 + row) * p.ldh + (t.n0 >> 1);
#pragma unroll 1
                    for (int c0 = 0; c0 < kBN; c0 += 32) {
                        uint32_t v[32];
                        tmem_ld_32x32b_x32(taddr + c0, v);
                        tmem_ld_wait();
                        if (gated) {
                            // 32 columns = 16 (gate, up) pairs -> 16 bf16 = two 16-byte stores
                            if (row < t.rows && t.n0 + c0 < p.N) {
                                uint32_t h2[8];
#pragma unroll
                                for (int i = 0; i < 8; ++i) {
                                    const __nv_bfloat16 lo = swiglu_bf16(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]));
                                    const __nv_bfloat16 hi = swiglu_bf16(__uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3]));
                                    h2[i] = uint32_t(__bfloat16_as_ushort(lo)) | (uint32_t(__bfloat16_as_ushort(hi)) << 16);
                                }
                                uint4* q = reinterpret_cast<uint4*>(hdst + (c0 >> 1));
                                q[0] = make_uint4(h2[0], h2[1], h2[2], h2[3]);
                                q[1] = make_uint4(h2[4], h2[5], h2[6], h2[7]);
                            }
                        } else if (full && p.Cb) {
                            // 32 columns -> 32 bf16 = four 16-byte stores
                            if (row < t.rows) {
                                __nv_bfloat16* cdst = p.Cb + int64_t(t.row0 + row) * p.ldc + t.n0 + c0;
#pragma unroll
                                for (int i = 0; i < 32; i += 8)
                                    if (t.n0 + c0 + i < p.N) {
                                        uint32_t h[4];
#pragma unroll
                                        for (int j = 0; j < 4; ++j)
                                            h[j] = uint32_t(__bfloat16_as_ushort(__float2bfloat16_rn(__uint_as_float(v[i + 2 * j])))) |
                                                   (uint32_t(__bfloat16_as_ushort(__float2bfloat16_rn(__uint_as_float(v[i + 2 * j + 1])))) << 16);
                                        *reinterpret_cast<uint4*>(cdst + i) = make_uint4(h[0], h[1], h[2], h[3]);
                                    }
                            }
                        } else if (row < t.rows) {
#pragma unroll
                            for (int i = 0; i < 32; i += 4)
                                if (!full || t.n0 + c0 + i < p.N)
                                    *reinterpret_cast<float4*>(dst + c0 + i) =
                                        make_float4(__uint_as_float(v[i]), __uint_as_float(v[i + 1]),
                                                    __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
                        }
                    }
                }
                }
            }
            if (ok && !kWN) {
#pragma unroll
                for (int u = 0; u < kNumN; ++u) {
                    // M = 128: accumulator row r sits in TMEM lane r.  M = 64: rows 16q..16q+15 sit in the
                    // lower half of lane quarter q, the upper 16 lanes of each quarter hold nothing.
                    const int n_local = kUmmaM == 128 ? u * 128 + quarter * 32 + lane : quarter * 16 + lane;
                    const bool lane_ok = kUmmaM == 128 || lane < 16;
                    const bool n_ok = lane_ok && (full ? (t.n0 + n_local < p.N) : true);
                    const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) +
                                           acc * uint32_t(kNumN * acc_cols) + uint32_t(u * acc_cols);
                    const bool to_bf16 = full && p.Cb != nullptr;
                    __nv_bfloat16* outb = p.Cb + int64_t(t.row0) * p.ldc + t.n0 + n_local;
                    for (int c0 = 0; c0 < n_mma; c0 += 32) {
                        if (n_mma - c0 >= 32) {
                            uint32_t v[32];
                            tmem_ld_32x32b_x32(taddr + c0, v);
                            tmem_ld_wait();
                            if (to_bf16) {
#pragma unroll
                                for (int i = 0; i < 32; ++i)
                                    if (n_ok && c0 + i < t.rows) outb[int64_t(c0 + i) * p.ldc] = __float2bfloat16_rn(__uint_as_float(v[i]));
                            } else {
#pragma unroll
                                for (int i = 0; i < 32; ++i)
                                    if (n_ok && c0 + i < t.rows) out[int64_t(c0 + i) * ld + n_local] = __uint_as_float(v[i]);
                            }
                        } else {
                            uint32_t v[16];
                            tmem_ld_32x32b_x16(taddr + c0, v);
                            tmem_ld_wait();
                            if (to_bf16) {
#pragma unroll
                                for (int i = 0; i < 16; ++i)
                                    if (n_ok && c0 + i < t.rows) outb[int64_t(c0 + i) * p.ldc] = __float2bfloat16_rn(__uint_as_float(v[i]));
                            } else {
#pragma unroll
                                for (int i = 0; i < 16; ++i)
                                    if (n_ok && c0 + i < t.rows) out[int64_t(c0 + i) * ld + n_local] = __uint_as_float(v[i]);
                            }
                        }
                    }
                }
            }
            // accumulator drained: hand it back to the MMA warp
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty_bar[acc]);
            if (p.tile_flags_mode == 1 && ok && full && !(p.tile_flags_skip_cta0 && blockIdx.x == 0)) {
                // this warp's part of the tile is stored: visible device-wide, also to the copy engines that will read
                // it as another product's tokens, before the m-tile's counter moves
                asm volatile("fence.proxy.async.global;" ::: "memory");
                __threadfence();
                __syncwarp();
                if (lane == 0) atomicAdd(p.tile_flags + t.mtile, 1u);
            }
            if (!(kWN && p.BM > 128)) acc ^= 1;          // (two token blocks: the tile owned both accumulators)
            if (acc == 0) acc_phase ^= 1;

            if (*abort_ptr) break;
        }
    }

    // --------------------------------------------------------------- teardown
    tc_fence_before_sync();
    __syncthreads();
    if (kWN && p.cluster_k > 1) {
        // Cluster split-K: every CTA of the cluster holds its share of the K sum of the same tile in its shared
        // memory.  CTA rank r adds the r-th share of the tile's 16-byte vectors over all ranks, in rank (= K) order,
        // reading the peers' copies through distributed shared memory, and writes C.  The first barrier makes the
        // partial tiles visible cluster-wide; after the second nobody reads a peer's memory any more.  All threads
        // of all CTAs reach both (every wait before this point is bounded).
        cluster_sync();
        if (warp >= 2 && warp < 6 && !*abort_ptr) {
            const int S = p.cluster_k, rank = int(cluster_cta_rank());
            const int tile = int(cluster_id_x());
            if (tile < tiles_total) {
                const TileInfo t = decode_tile(p, prefix, row_start, tile);
                constexpr int kVecPerRow = kBN / 4;
                const int total_vec = t.rows * kVecPerRow;
                const int v_begin = int(static_cast<long long>(total_vec) * rank / S);
                const int v_end = int(static_cast<long long>(total_vec) * (rank + 1) / S);
                const uint32_t base = smem_u32(stages);
                for (int v = v_begin + (int(threadIdx.x) - 64); v < v_end; v += 128) {
                    const int r = v / kVecPerRow, c4 = (v % kVecPerRow) * 4;
                    const uint32_t local = base + uint32_t(r * kStagePitch + c4) * 4u;
                    float4 x[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (j < S) x[j] = ld_cluster_f4(map_to_cta(local, uint32_t(j)));
                    float4 sum = x[0];
#pragma unroll
                    for (int j = 1; j < 8; ++j)
                        if (j < S) { sum.x += x[j].x; sum.y += x[j].y; sum.z += x[j].z; sum.w += x[j].w; }
                    if (t.n0 + c4 < p.N) {
                        if (p.Cb) {
                            const uint32_t lo = uint32_t(__bfloat16_as_ushort(__float2bfloat16_rn(sum.x))) |
                                                (uint32_t(__bfloat16_as_ushort(__float2bfloat16_rn(sum.y))) << 16);
                            const uint32_t hi = uint32_t(__bfloat16_as_ushort(__float2bfloat16_rn(sum.z))) |
                                                (uint32_t(__bfloat16_as_ushort(__float2bfloat16_rn(sum.w))) << 16);
                            *reinterpret_cast<uint2*>(p.Cb + int64_t(t.row0 + r) * p.ldc + t.n0 + c4) = make_uint2(lo, hi);
                        } else {
                            *reinterpret_cast<float4*>(p.C + int64_t(t.row0 + r) * p.ldc + t.n0 + c4) = sum;
                        }
                    }
                }
            }
        }
        cluster_sync();
    }
    if (warp == 1 && free_tmem) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, tmem_cols);
    }
    // The barriers are dead from here on; a later call of this body in the same kernel initialises them afresh.
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.num_stages; ++s) { mbar_inval(&full_bar[s]); mbar_inval(&empty_bar[s]); }
        for (int b = 0; b < 2; ++b) { mbar_inval(&acc_full_bar[b]); mbar_inval(&acc_empty_bar[b]); }
        if (p.generic_b == 1)
            for (int r = 0; r < p.raw_slots; ++r) { mbar_inval(&raw_full_bar[r]); mbar_inval(&raw_empty_bar[r]); }
        if (p.generic_b == 2)
            for (int s = 0; s < p.num_stages; ++s) mbar_inval(&raw_full_bar[s]);
    }
    __syncthreads();
}

template <int kBK, int kBN, bool kWN, bool kFp8>
__global__ void __launch_bounds__(kGenericThreads, 1) gemm_kernel(const __grid_constant__ GemmParams p) {
    gemm_body<kBK, kBN, kWN, kFp8>(p, true, true);
}


// Stream-K reduction.  The GEMM kernel leaves the partial sum of every (CTA, split tile) in its workspace slot
// and does no synchronisation of its own; this kernel, ordered after it by the stream, adds the partials of
// each split tile in K order (lowest CTA first) and writes C.  One CTA per boundary between two ranges of
// the GEMM grid.  A tile cut by several boundaries is shared between their CTAs: each sums a contiguous share of
// the tile's 16-byte vectors over ALL contributors, so every element is still one sum in K order and the bits do
// not depend on how the tile was shared (p.reduce_split == 0: the first boundary inside the tile sums all of it).
// (A device function, so that a kernel that runs two products can sum the first one's split tiles itself: `boundary`
// is the index of the boundary this CTA owns, `first` / `nthreads` the threads of the CTA that take part -- they
// must be whole warps starting at a multiple of 32 -- and `pdl` says whether this is the stand-alone kernel, which
// waits for the GEMM grid through griddepcontrol.)
template <bool kStandalone>
__device__ __forceinline__ void streamk_reduce_body(const GemmParams& p, int gemm_grid, int boundary, int* prefix,
                                                    int* row_start, int* slot_of) {
    // Launched with programmatic stream serialisation, and the GEMM kernel lets its dependents launch as soon
    // as it has started: this grid is resident and has done all of its index arithmetic (which reads only
    // the call's inputs) while the GEMM grid is still running.  Nothing the GEMM kernel wrote is read before
    // griddepcontrol.wait, which returns once that grid has completed and its writes are visible.
    // The kernel after this one in the stream may start its own set-up now; it waits for this grid to complete
    // before it reads or writes anything.
    if (kStandalone && threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    load_row_starts(p, row_start);
    __syncthreads();
    if (threadIdx.x < 32) tile_prefix(p, row_start, prefix);
    __syncthreads();
    Sched sched;
    sched.init(1, p.k_iters, prefix[p.E], gemm_grid, 0, nullptr);
    const int c = boundary + 1;                            // boundary between CTA c-1 and CTA c
    // Does this boundary cut a tile, and which share of the tile is this CTA's?
    bool active = c < sched.grid_eff;
    int tile = 0, c_lo = 0, c_hi = 0, share = 0, shares = 1;
    if (active) {
        // (iterations count from the first tile of the part of the schedule that is cut along K)
        const long long b = sched.range_begin(c);
        const int cut_tile = int(b / p.k_iters);
        tile = sched.dp_tiles + cut_tile;
        const long long tile_begin = static_cast<long long>(cut_tile) * p.k_iters;
        active = b != tile_begin;                          // else the boundary coincides with a tile boundary
        if (active) {
            c_lo = sched.owner(tile_begin);
            c_hi = sched.owner(tile_begin + p.k_iters - 1);
            if (p.reduce_split) {
                share = c - c_lo - 1;                      // boundaries c_lo+1 .. c_hi lie inside the tile
                shares = c_hi - c_lo;
            } else {
                active = c == c_lo + 1;                    // the first boundary inside the tile sums all of it
            }
        }
    }
    TileInfo t = {0, 0, 0, 0, 0, 0};
    if (active) {
        t = decode_tile(p, prefix, row_start, tile);
        // slots of the contributors, computed before the wait (the load loop below must not divide)
        for (int j = threadIdx.x; j <= c_hi - c_lo && j < kRangeTabMax; j += blockDim.x) slot_of[j] = sched.slot(c_lo + j, tile);
    }
    __syncthreads();
    // EVERY CTA waits, also those with nothing to add: a grid whose CTAs all left before the GEMM grid finished
    // would count as complete, and the kernel after it in the stream would stop waiting for the GEMM.
    if (kStandalone) asm volatile("griddepcontrol.wait;" ::: "memory");
    if (!active) return;
    float* dst = p.C + int64_t(t.row0) * p.ldc + t.n0;
    const int vec_per_row = p.BN / 4;
    const int total_vec = t.rows * vec_per_row;
    const int v_begin = int(static_cast<long long>(total_vec) * share / shares);
    const int v_end = int(static_cast<long long>(total_vec) * (share + 1) / shares);
    const size_t slot_floats = size_t(p.BM) * p.BN;
    const int nthr = int(blockDim.x);
    for (int v0 = v_begin; v0 < v_end; v0 += 4 * nthr) {
        float4 sum[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) sum[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int c0 = c_lo; c0 <= c_hi; c0 += 4) {         // four contributors' loads in flight together
            float4 x[4][4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const bool c_ok = c0 + j <= c_hi;
                const int jj = c_ok ? c0 + j - c_lo : 0;
                const int slot = jj < kRangeTabMax ? slot_of[jj] : sched.slot(c_lo + jj, tile);
                const float4* src = reinterpret_cast<const float4*>(p.partials + size_t(slot) * slot_floats);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int v = v0 + q * nthr + int(threadIdx.x);
                    x[j][q] = (c_ok && v < v_end) ? __ldcg(src + v) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (c0 + j > c_hi) break;                  // absent contributors add nothing (not even +0)
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    sum[q].x += x[j][q].x; sum[q].y += x[j][q].y; sum[q].z += x[j][q].z; sum[q].w += x[j][q].w;
                }
            }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int v = v0 + q * nthr + int(threadIdx.x);
            if (v < v_end) {
                const int r = v / vec_per_row, c4 = (v % vec_per_row) * 4;
                if (t.n0 + c4 < p.N) {
                    if (p.epi_swiglu) {
                        const __nv_bfloat16 lo = swiglu_bf16(sum[q].x, sum[q].y), hi = swiglu_bf16(sum[q].z, sum[q].w);
                        *reinterpret_cast<uint32_t*>(p.H + int64_t(t.row0 + r) * p.ldh + ((t.n0 + c4) >> 1)) =
                            uint32_t(__bfloat16_as_ushort(lo)) | (uint32_t(__bfloat16_as_ushort(hi)) << 16);
                    } else if (p.Cb) {
                        const uint32_t lo = uint32_t(__bfloat16_as_ushort(__float2bfloat16_rn(sum[q].x))) |
                                            (uint32_t(__bfloat16_as_ushort(__float2bfloat16_rn(sum[q].y))) << 16);
                        const uint32_t hi = uint32_t(__bfloat16_as_ushort(__float2bfloat16_rn(sum[q].z))) |
                                            (uint32_t(__bfloat16_as_ushort(__float2bfloat16_rn(sum[q].w))) << 16);
                        *reinterpret_cast<uint2*>(p.Cb + int64_t(t.row0 + r) * p.ldc + t.n0 + c4) = make_uint2(lo, hi);
                    } else {
                        *reinterpret_cast<float4*>(dst + int64_t(r) * p.ldc + c4) = sum[q];
                    }
                }
            }
        }
    }
}

// The kernel's instantiations are compiled in translation units of their own, one per (orientation, element type):
// weights on the N or on the M side of the MMA, bf16 or FP8.  Each raises the kernel's shared-memory limit on first
// use per device and launches with the given configuration; TL_ERR_UNSUPPORTED for a (cta_k, cta_n) outside
// {64, 128} x {64, 128, 256}.
int launch_gemm_wn_bf16(int bk, int bn, const cudaLaunchConfig_t* cfg, const GemmParams& p);
int launch_gemm_wn_fp8(int bk, int bn, const cudaLaunchConfig_t* cfg, const GemmParams& p);
int launch_gemm_wm_bf16(int bk, int bn, const cudaLaunchConfig_t* cfg, const GemmParams& p);
int launch_gemm_wm_fp8(int bk, int bn, const cudaLaunchConfig_t* cfg, const GemmParams& p);
// Two grouped products in one cooperative launch (tl_gemm_chain.cu); weights-on-N, bf16, tile 64 x 256 only.
int launch_gemm_chain(int bk, int bn, int grid, size_t smem, cudaStream_t stream, const GemmParams& p1,
                      const GemmParams& p2, unsigned long long* counter, unsigned long long target1,
                      unsigned long long target2, bool skip_cta0);
// Clusters of `size` CTAs of the single-CTA GEMM kernel (one CTA per SM) that can be resident at the same time on the
// current device: clusters live inside one GPC, so 148 SMs hold 45 clusters of 3 but only 15 of 8.
int gemm_max_active_clusters(int size, int* out);
// CTA-pair kernel (tl_gemm_pair.cu): halves = 2 for 512-token tiles.
int launch_gemm_pair(bool fp8, int halves, int clusters, size_t smem, cudaStream_t stream, const GemmParams& p);
// Clusters of the pair kernel that can be resident together on the current device.
int pair_max_active_clusters(int* out);
constexpr int kPairStagesMax = 8;
constexpr int kPairStageOutBytes = 4096;   // per epilogue warp: 32 tokens x 32 columns of fp32 C on their way to a bulk store
constexpr int kPairDynamicSmem = 226 * 1024;   // the pair kernels' static shared memory is a few barriers only
constexpr int kPairBigThreads = 320;       // pair kernel with 512-token tiles: producer, MMA issuer, eight epilogue warps

}  // namespace tl
