// Tiled GEMM reading a tile-major (or row-major) weight operand, for sm_100a.
//
//   C[M x N] (fp32) = A[M x K] (bf16 or FP8, K contiguous) x B[K x N]                      (Section 2.3)
//
// B is read through a 5-D tensor-map view of the tile-major buffer (the 4-D view of Eq. 3 with the contiguous
// extent of a memory tile split into swizzle rows of 128, 64 or 32 bytes).  One TMA instruction fills a pipeline
// stage: its box is a whole number of memory tiles, or the part of a tile that lies inside the CTA tile, and it
// lands in shared memory in exactly the canonical swizzled operand form that tcgen05.mma reads -- MN-major for
// weights stored with N contiguous, K-major for weights stored [N][K] (Eq. 2 as printed).  The weights can sit on
// either side of the instruction:
//   weights on N (tiles of up to 128 token rows: decode, MoE)  tokens are the M-side operand (64-row MMAs for
//                tiles of up to 64 tokens, else 128 rows; spare rows are zeroed once), one MMA covers all cta_n
//                weight columns; TMEM lane = token row;
//   weights on M (256-token tiles)  TMEM lane = weight column, the accumulator holds C transposed.
// Memory tiles whose rows are shorter than 32 bytes cannot be boxed: four more warps load them with Eq. 1-2
// address arithmetic and build the operand image by hand (Section 4.4).
//
// One persistent CTA per SM:
//   warp 0      TMA producer   (one lane)   ring of shared-memory stages, mbarrier expect-tx
//   warp 1      MMA issuer     (one lane)   tcgen05.mma into one of two TMEM accumulators
//   warps 2..5  epilogue                    tcgen05.ld -> fp32 -> C, or silu(gate) * up -> bf16 (expert FFN)
//   warps 6..9  hand-addressed weight loads (only when the memory tile cannot be boxed)
// Work is a list of (output tile, K range).  Data-parallel mode hands whole tiles round-robin; stream-K mode cuts
// the flattened (tile, K iteration) space into one contiguous range per CTA (decode: all SMs stream weights even
// when there are fewer tiles than SMs).  Partial tiles go to a workspace and a second small kernel
// (streamk_reduce_kernel, launched with programmatic stream serialisation so that it is resident before this one
// ends) adds them in K order and writes C.  Nothing ever spins on another CTA; every mbarrier wait is bounded
// (see mbar_wait_bounded).  Large dense problems run on CTA pairs instead (tl_gemm_pair.cuh).
#include "tl_common.cuh"

#include <cuda_bf16.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>

namespace tl {

constexpr int kGemmThreads = 192;          // TMA path: producer, MMA issuer, four epilogue warps
constexpr int kGenericThreads = 320;       // generic-address path: four more warps that load the weights by hand
constexpr int kMaxStages = 16;
constexpr int kMaxExperts = 1024;
constexpr int kNumBoxChoices = 5;          // token boxes of 16, 32, 64, 128, 256 rows
constexpr int kAtomBytes = 128;            // one swizzle row: 64 bf16
constexpr int kMaxDynamicSmem = 227 * 1024 - 10 * 1024;   // 227 KB per CTA minus the kernel's static shared memory

struct alignas(64) GemmParams {
    CUtensorMap tmap_a[kNumBoxChoices];
    CUtensorMap tmap_b;
    float* C;
    float* partials;            // stream-K partial tiles: slot = BM x BN floats
    const int32_t* offsets;     // grouped: device E+1 row offsets; dense: nullptr
    uint32_t* status;
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
    int generic_b;              // 1: warps 6..9 load the weights with Eq. 1-2 address arithmetic
    const uint8_t* B;           // raw weight pointer (generic path only)
    int64_t expert_bytes;       // K*N*2
    int blocks_per_row;         // N / bc
};

struct TileInfo {
    int n0;          // first weight column
    int row0;        // first row of A / C
    int rows;        // valid rows (<= BM)
    int expert;
    int flip;        // odd m-tile of its (expert, n-tile): walks K backwards (see decode_tile)
};

// ------------------------------------------------------------------ scheduler
struct Work {
    int tile, kbeg, kend;
};

constexpr int kRangeTabMax = 256;      // CTAs whose range starts are tabulated in shared memory

struct Sched {
    int stream_k, k_iters, tiles_total, grid_eff, cta;
    int next_tile;
    long long it, it_end, it_begin;
    const int* tab;     // tab[c] = first flattened iteration of CTA c (grid_eff + 1 entries), or nullptr

    // Even split of the flattened (tile, K iteration) space; a fixed function of the CTA index.
    __device__ static long long split(long long total, int grid_eff, int c) { return (total * c) / grid_eff; }
    __device__ long long range_begin(int c) const {
        return tab ? tab[c] : split(static_cast<long long>(tiles_total) * k_iters, grid_eff, c);
    }
    __device__ static int effective_grid(long long total, int grid) { return total < grid ? static_cast<int>(total) : grid; }
    __device__ void init(int stream_k_, int k_iters_, int tiles_total_, int grid, int cta_, const int* tab_) {
        stream_k = stream_k_; k_iters = k_iters_; tiles_total = tiles_total_; cta = cta_; tab = tab_;
        grid_eff = effective_grid(static_cast<long long>(tiles_total) * k_iters, grid);
        next_tile = cta;
        if (grid_eff == 0 || cta >= grid_eff) { it = it_end = it_begin = 0; next_tile = tiles_total; return; }
        it_begin = it = range_begin(cta);
        it_end = range_begin(cta + 1);
    }
    __device__ bool next(Work& w) {
        if (!stream_k) {
            if (next_tile >= tiles_total) return false;
            w.tile = next_tile; w.kbeg = 0; w.kend = k_iters;
            next_tile += gridDim.x;
            return true;
        }
        if (it >= it_end) return false;
        int t = static_cast<int>(it / k_iters);
        int kb = static_cast<int>(it - static_cast<long long>(t) * k_iters);
        long long left = it_end - it;
        int ke = (k_iters - kb) < left ? k_iters : kb + static_cast<int>(left);
        w.tile = t; w.kbeg = kb; w.kend = ke;
        it += ke - kb;
        return true;
    }
    // CTA whose range holds flattened iteration x.
    __device__ int owner(long long x) const {
        if (tab) {                                   // largest c with tab[c] <= x
            int lo = 0, hi = grid_eff;
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (tab[mid] <= x) lo = mid; else hi = mid;
            }
            return lo;
        }
        long long total = static_cast<long long>(tiles_total) * k_iters;
        int c = static_cast<int>(((x + 1) * grid_eff + total - 1) / total) - 1;
        if (c < 0) c = 0;
        if (c >= grid_eff) c = grid_eff - 1;
        while (c > 0 && range_begin(c) > x) --c;
        while (c + 1 < grid_eff && range_begin(c + 1) <= x) ++c;
        return c;
    }
    // Partial-tile slot of CTA c for tile t: 2c when the tile is the first thing c works on, else 2c+1.
    __device__ int slot(int c, int t) const {
        return 2 * c + (range_begin(c) < static_cast<long long>(t) * k_iters ? 1 : 0);
    }
};

__device__ __forceinline__ TileInfo decode_tile(const GemmParams& p, const int* prefix, const int* row_start, int tile) {
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
    t.flip = (local % mt) & 1;
    t.rows = row_end - t.row0 < p.BM ? row_end - t.row0 : p.BM;
    return t;
}

// Expert row offsets into shared memory (dense problems: one "expert" holding rows 0..M).
__device__ __forceinline__ void load_row_starts(const GemmParams& p, int* row_start) {
    for (int e = threadIdx.x; e <= p.E; e += blockDim.x) row_start[e] = p.offsets ? p.offsets[e] : (e == 0 ? 0 : p.M);
}

// prefix[e] = output tiles of the experts before e (n_tiles x m-tiles each); one warp, shuffle scan.
__device__ __forceinline__ void tile_prefix(const GemmParams& p, const int* row_start, int* prefix) {
    const int lane = threadIdx.x & 31;
    int carry = 0;
    for (int base = 0; base < p.E; base += 32) {
        const int e = base + lane;
        int v = 0;
        if (e < p.E) v = ((row_start[e + 1] - row_start[e] + p.BM - 1) / p.BM) * p.n_tiles;
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

// Optional per-CTA timestamps (nanoseconds of %globaltimer), compiled in only with -DTL_TIMELINE:
// slot 0 kernel entry, 1 set-up done, 2 first stage landed, 3 last MMA committed, 4 first epilogue
// started, 5 last epilogue (and fix-up) done, 6 producer done.
#ifdef TL_TIMELINE
__device__ uint64_t* g_timeline = nullptr;
__device__ int g_reverse = 0;
#define TL_TIMELINE_INIT() uint64_t* const tl_tl = g_timeline ? g_timeline + blockIdx.x * 8 : nullptr; bool tl_once = true; (void)tl_once
#define TL_STAMP(slot) do { if (tl_tl) tl_tl[(slot)] = global_timer_ns(); } while (0)
#define TL_STAMP_ONCE(slot) do { if (tl_once) { tl_once = false; if (tl_tl) tl_tl[(slot)] = global_timer_ns(); } } while (0)
// cycle counters per CTA (16 per CTA): 0 producer wait-empty, 1 producer issue, 2 stages issued, 3 MMA wait-full,
// 4 MMA wait-accumulator, 5 MMA issue, 6 epilogue wait, 7 epilogue drain, 8 epilogue fix-up, 9 work items
__device__ unsigned long long* g_counters = nullptr;
#define TL_CLOCK() clock64()
#define TL_COUNT(slot, v) do { if (g_counters) atomicAdd(&g_counters[blockIdx.x * 16 + (slot)], (unsigned long long)(v)); } while (0)
#else
#define TL_CLOCK() 0ll
#define TL_COUNT(slot, v) do { } while (0)
#define TL_TIMELINE_INIT() do { } while (0)
#define TL_STAMP(slot) do { } while (0)
#define TL_STAMP_ONCE(slot) do { } while (0)
#endif

__device__ __forceinline__ void epilogue_bar_sync() {
    asm volatile("bar.sync 1, 128;" ::: "memory");
}

// One warp fills one stage of weights on the generic-address path.  The stage is kBK/br runs of
// kBN/bc whole memory tiles; run r starts at src0 + r*krow_stride and is kBN*br*2 contiguous bytes.
// Chunks of 16 bytes are read in memory order, 16 loads in flight per lane; kPieces = rows held by one
// chunk (1 when a block row is at least 16 bytes).  Rows >= k_rows_left and columns >= n_cols_left
// (tile overhang) are filled with zeros.
template <int kBK, int kBN, int kPieces>
__device__ __forceinline__ void generic_fill_stage(uint8_t* sw, const uint8_t* src0, int64_t krow_stride, int br_log2,
                                                   int bc_log2, int k_rows_left, int n_cols_left, int lane) {
    constexpr int kChunks = kBK * kBN * 2 / 16;
    const int run_log2 = bc_log2 + 1;                       // log2(bytes of one block row)
    const int g_log2 = br_log2 + run_log2;                  // log2(G)
    const int seg_log2 = br_log2 + 1 + (kBN == 64 ? 6 : kBN == 128 ? 7 : 8);   // log2(kBN * br * 2): bytes of one run of tiles
#pragma unroll 1
    for (int base = 0; base < kChunks; base += 32 * 16) {
        uint4 v[16];
        int kl[16], nl[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int byte = (base + i * 32 + lane) << 4;   // byte offset inside the stage's memory image
            const int seg = byte >> seg_log2, o = byte & ((1 << seg_log2) - 1);
            const int ib = o & ((1 << g_log2) - 1);         // byte inside the memory tile
            kl[i] = (seg << br_log2) + (ib >> run_log2);    // Eq. 1 inverted: row and column inside the stage
            nl[i] = ((o >> g_log2) << bc_log2) + ((ib & ((1 << run_log2) - 1)) >> 1);
            v[i] = make_uint4(0, 0, 0, 0);
            if (kl[i] < k_rows_left && nl[i] < n_cols_left)
                v[i] = __ldg(reinterpret_cast<const uint4*>(src0 + int64_t(seg) * krow_stride + o));
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) {
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
template <int kBK, int kBN, bool kWN, bool kFp8>
__global__ void __launch_bounds__(kGenericThreads, 1) gemm_kernel(const __grid_constant__ GemmParams p) {
    constexpr int kNumN = kWN ? 1 : (kBN >= 128 ? kBN / 128 : 1);     // MMAs per K step
    constexpr int kUmmaM = kWN ? 128 : (kBN >= 128 ? 128 : 64);       // rows of the MMA's M side
    constexpr int kKSteps = kBK / 16;
    constexpr int kSubK = kBK / 64;                        // token boxes per stage
    constexpr uint32_t kWBytes = kBK * kBN * 2;            // weight bytes per stage

    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
    __shared__ __align__(8) uint64_t acc_full_bar[2];
    __shared__ __align__(8) uint64_t acc_empty_bar[2];
    __shared__ uint32_t tmem_slot;
    __shared__ uint32_t abort_flag;
    __shared__ int prefix[kMaxExperts + 1];
    __shared__ int row_start[kMaxExperts + 1];      // copy of the expert row offsets (dense: 0, M)
    __shared__ int range_tab[kRangeTabMax + 1];     // stream-K: first flattened iteration of every CTA

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    TL_TIMELINE_INIT();
    if (threadIdx.x == 0) { TL_STAMP(0); TL_COUNT(10, TL_CLOCK()); TL_COUNT(12, global_timer_ns()); }
    const uint32_t stage_bytes = kWBytes + uint32_t(kSubK) * p.a_rows * kAtomBytes;
    uint8_t* stages = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

    const int acc_cols = kWN ? kBN : p.BM;                   // TMEM columns of one MMA's accumulator
    uint32_t tmem_cols = 32;
    while (tmem_cols < uint32_t(2 * kNumN * acc_cols)) tmem_cols <<= 1;

    // ---------------------------------------------------------------- set-up
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.num_stages; ++s) { mbar_init(&full_bar[s], p.generic_b ? 2 : 1); mbar_init(&empty_bar[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full_bar[b], 1); mbar_init(&acc_empty_bar[b], 4); }
        abort_flag = 0;
        fence_mbar_init();
        if (!p.generic_b) tma_prefetch_desc(&p.tmap_b);
        for (int i = 0; i < kNumBoxChoices; ++i) tma_prefetch_desc(&p.tmap_a[i]);
    }
    if (warp == 1) {
        tmem_alloc(&tmem_slot, tmem_cols);
        tmem_relinquish();
    }
    // Dense stream-K problems: while the kernel before this one in the stream is still finishing, ask for the
    // first stages of this CTA's weights to be brought into L2.  A prefetch delivers nothing to the SM and L2 is
    // the point of coherence, so this is safe whatever that kernel is still writing; it takes the cold start
    // (page walks, first DRAM accesses) off this kernel's critical path.
    // (issued by an epilogue thread, which has nothing else to do yet, so that the producer is not held up)
    if (threadIdx.x == 64 && p.stream_k && !p.generic_b && p.offsets == nullptr && p.prefetch_stages > 0) {
        const int mt = (p.M + p.BM - 1) / p.BM;
        const long long total = static_cast<long long>(mt) * p.n_tiles * p.k_iters;
        const int geff = Sched::effective_grid(total, gridDim.x);
        if (int(blockIdx.x) < geff) {
            long long it = Sched::split(total, geff, blockIdx.x);
            const long long it_end = Sched::split(total, geff, blockIdx.x + 1);
            for (int s = 0; s < p.prefetch_stages && it < it_end; ++s, ++it) {
                const int tile = int(it / p.k_iters), kit = int(it - static_cast<long long>(tile) * p.k_iters);
                const int n0 = (tile / mt) * p.BN;
                const int k0 = (kit * kBK) << p.k_shift;
                for (int kb = 0; kb < p.kbx; ++kb)
                    for (int nb = 0; nb < p.nbx; ++nb) {
                        int c[5];
                        weight_box_coords(p, k0 + kb * p.box_rows, n0 + nb * p.box_atoms * 64, 0, c);
                        tma_prefetch_5d(&p.tmap_b, c[0], c[1], c[2], c[3], c[4]);
                    }
            }
        }
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
    // Launched with programmatic stream serialisation: everything above (barriers, tensor memory, descriptor
    // prefetch) may run while the kernel before this one in the stream is still finishing.  Nothing that kernel
    // may have written (tokens, expert offsets, the partial-tile workspace, C) is touched before this wait, which
    // returns once it has completed and its writes are visible.
    // Grouped problems read the expert offsets, which that kernel may have produced, for the tables below; dense
    // problems build their tables from the launch parameters alone and wait afterwards.
    const bool tables_first = p.offsets == nullptr;
    if (!tables_first) asm volatile("griddepcontrol.wait;" ::: "memory");
    // tiles before each expert (dense: one "expert" holding all M rows)
    load_row_starts(p, row_start);
    __syncthreads();
    if (warp == 2) tile_prefix(p, row_start, prefix);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_slot;
    const int tiles_total = prefix[p.E];
    // Range starts of all CTAs, once, so that nothing on the critical path divides 64-bit numbers.
    const long long total_iters = static_cast<long long>(tiles_total) * p.k_iters;
    const int grid_eff0 = Sched::effective_grid(total_iters, gridDim.x);
    const bool use_tab = p.stream_k && grid_eff0 > 0 && grid_eff0 <= kRangeTabMax && total_iters < (1ll << 31);
    if (use_tab) {
        for (int c = threadIdx.x; c <= grid_eff0; c += blockDim.x)
            range_tab[c] = static_cast<int>(Sched::split(total_iters, grid_eff0, c));
        __syncthreads();
    }
    Sched sched;
#ifdef TL_TIMELINE
    // measurement builds: optionally hand the ranges out in reverse CTA order; record the SM id
    sched.init(p.stream_k, p.k_iters, tiles_total, gridDim.x, g_reverse ? gridDim.x - 1 - blockIdx.x : blockIdx.x,
               use_tab ? range_tab : nullptr);
    if (threadIdx.x == 0 && tl_tl) { uint32_t smid; asm volatile("mov.u32 %0, %smid;" : "=r"(smid)); tl_tl[7] = smid; }
#else
    sched.init(p.stream_k, p.k_iters, tiles_total, gridDim.x, blockIdx.x, use_tab ? range_tab : nullptr);
#endif
    if (tables_first) asm volatile("griddepcontrol.wait;" ::: "memory");
    // Stream-K: let the reduction kernel that follows in the stream be scheduled already; it does its own
    // set-up and then blocks until this whole grid has finished.
    if (p.stream_k && threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 0) TL_STAMP(1);
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
            int ks[4], km[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { ks[i] = p.ck_shift[i]; km[i] = p.ck_mask[i]; }
            while (ok && sched.next(w)) {
                const TileInfo t = decode_tile(p, prefix, row_start, w.tile);
                int bi = 0;
                while ((16 << bi) < t.rows) ++bi;
                const uint32_t a_bytes = uint32_t(16 << bi) * kAtomBytes;
                const uint32_t tx = uint32_t(kSubK) * a_bytes + uint32_t(p.kbx * p.nbx) * p.box_bytes;
                const int kc_expert = t.expert * p.k_coord_per_expert;
                int cn[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) cn[i] = ((t.n0 >> p.cn_shift[i]) & p.cn_mask[i]) + p.c_expert[i] * kc_expert;
                for (int kit = w.kbeg; kit < w.kend; ++kit) {
                    const long long cc0 = TL_CLOCK();
                    if (!mbar_wait_bounded(&empty_bar[stage], phase ^ 1, abort_ptr, p.status, kWaitProducerEmpty)) {
                        ok = false;
                        break;
                    }
                    const long long cc1 = TL_CLOCK();
                    (void)cc0; (void)cc1;
                    uint8_t* sw = stages + size_t(stage) * stage_bytes;
                    uint8_t* sa = sw + kWBytes;
                    mbar_arrive_expect_tx(&full_bar[stage], tx);
                    const int kq = t.flip ? p.k_iters - 1 - kit : kit;
                    const int k0 = (kq * kBK) << p.k_shift;         // first K element of the stage
#pragma unroll
                    for (int sub = 0; sub < kSubK; ++sub)
                        tma_load_2d(sa + size_t(sub) * p.a_rows * kAtomBytes, &p.tmap_a[bi], &full_bar[stage],
                                    k0 + ((sub * 64) << p.k_shift), t.row0);
                    if (one_box) {
                        // the usual case, one box per stage: the column part of the coordinates was worked out once
                        // for the tile, only the K part changes from stage to stage
                        tma_load_5d(sw, &p.tmap_b, &full_bar[stage], 0, ((k0 >> ks[0]) & km[0]) + cn[0],
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
                                tma_load_5d(dst, &p.tmap_b, &full_bar[stage], c[0], c[1], c[2], c[3], c[4]);
                            }
                        }
                    }
                    ++issued;
                    TL_COUNT(0, cc1 - cc0); TL_COUNT(1, TL_CLOCK() - cc1); TL_COUNT(2, 1);
                    if (++stage == uint32_t(p.num_stages)) { stage = 0; phase ^= 1; }
                }
            }
            TL_STAMP(6);
            if (!ok || *abort_ptr) {
                // Giving up: let the copies already issued land before the CTA's shared memory goes away.
                uint32_t s = stage, ph = phase;
                const uint32_t back = issued < uint32_t(p.num_stages) ? issued : uint32_t(p.num_stages);
                for (uint32_t i = 0; i < back; ++i) {
                    if (s == 0) { s = p.num_stages; ph ^= 1; }
                    --s;
                    const uint64_t t0 = global_timer_ns();
                    while (!mbar_try_wait(&full_bar[s], ph) && global_timer_ns() - t0 < 20000000ull) {}
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
            while (ok && sched.next(w)) {
                const TileInfo t = decode_tile(p, prefix, row_start, w.tile);
                const uint32_t n_mma = kWN ? uint32_t(kBN) : uint32_t((t.rows + 15) & ~15);
                // fp32 accumulate, bf16 x bf16; the weights operand is MN-major (bit 15: A, bit 16: B), the token
                // operand K-major; M = kUmmaM, N = n_mma
                const uint32_t w_major = p.w_kmajor ? 0u : (kWN ? (1u << 16) : (1u << 15));
                // (8-bit operands: format codes 0 = E4M3 in place of 1 = bf16)
                const uint32_t m_mma = kWN ? uint32_t(p.umma_m) : uint32_t(kUmmaM);
                const uint32_t idesc = (1u << 4) | (kFp8 ? 0u : (1u << 7) | (1u << 10)) | w_major |
                                       ((n_mma >> 3) << 17) | ((m_mma >> 4) << 24);
                const long long ca0 = TL_CLOCK();
                if (!mbar_wait_bounded(&acc_empty_bar[acc], acc_phase ^ 1, abort_ptr, p.status, kWaitMmaAccEmpty)) {
                    ok = false;
                    break;
                }
                TL_COUNT(4, TL_CLOCK() - ca0);
                (void)ca0;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * uint32_t(kNumN * acc_cols);
                for (int kit = w.kbeg; kit < w.kend; ++kit) {
                    const long long cm0 = TL_CLOCK();
                    if (!mbar_wait_bounded(&full_bar[stage], phase, abort_ptr, p.status, kWaitMmaFull)) {
                        ok = false;
                        break;
                    }
                    const long long cm1 = TL_CLOCK();
                    (void)cm0; (void)cm1;
                    tc_fence_after_sync();
                    TL_STAMP_ONCE(2);
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
                            if (kWN) umma_split<kFp8>(d_tmem, tok_lo0 + tok_off[j], tok_hi, w_lo, w_hi, idesc, accum);
                            else umma_split<kFp8>(d_tmem + uint32_t(u * acc_cols), w_lo, w_hi, tok_lo0 + tok_off[j], tok_hi, idesc, accum);
                        }
                    }
                    umma_commit(&empty_bar[stage]);      // frees the stage once these MMAs have read it
                    TL_COUNT(3, cm1 - cm0); TL_COUNT(5, TL_CLOCK() - cm1);
                    if (++stage == uint32_t(p.num_stages)) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                umma_commit(&acc_full_bar[acc]);         // accumulator complete
                TL_STAMP(3);
                acc ^= 1;
                if (acc == 0) acc_phase ^= 1;
            }
        }
    } else if (warp >= 6) {
        // ================================ generic-address weight loader (Section 4.4 of the paper)
        // Memory tiles whose rows are shorter than a TMA box allows are fetched with plain loads.  A stage's
        // weights are kBK/br runs of whole memory tiles, each run contiguous in the tile-major buffer, so
        // the 16-byte chunks are read in memory order (fully coalesced for any tile shape); Eq. 1 inverted
        // gives every chunk's (row, column), and the chunk (or its 16/(2 bc) row pieces) is stored where the
        // 128-byte-swizzled MN-major operand layout wants it.  Warp w fills every fourth stage.
        const int pw = warp - 6;
        const int br = 1 << p.br_log2, bc = 1 << p.bc_log2;
        const int run_bytes = bc * 2;                              // one block row
        const int G = br * run_bytes;
        const int pieces = run_bytes >= 16 ? 1 : 16 / run_bytes;  // rows held by one 16-byte chunk
        uint32_t it_global = 0;
        Work w;
        bool ok = true;
        while (ok && sched.next(w)) {
            const TileInfo t = decode_tile(p, prefix, row_start, w.tile);
            const uint8_t* Bexp = p.B + int64_t(t.expert) * p.expert_bytes;
            const int nblk0 = t.n0 >> p.bc_log2;
            for (int kit = w.kbeg; kit < w.kend; ++kit, ++it_global) {
                if ((it_global & 3u) != uint32_t(pw)) continue;
                const uint32_t stage = it_global % uint32_t(p.num_stages);
                const uint32_t phase = (it_global / uint32_t(p.num_stages)) & 1u;
                if (!mbar_wait_bounded(&empty_bar[stage], phase ^ 1, abort_ptr, p.status, kWaitProducerEmpty)) {
                    ok = false;
                    break;
                }
                uint8_t* sw = stages + size_t(stage) * stage_bytes;
                const int kq = t.flip ? p.k_iters - 1 - kit : kit;
                const int kblk0 = (kq * kBK) >> p.br_log2;
                const uint8_t* src0 = Bexp + (int64_t(kblk0) * p.blocks_per_row + nblk0) * G;
                const int k_rows_left = p.K - kq * kBK, n_cols_left = p.N - t.n0;
                const int64_t krow_stride = int64_t(p.blocks_per_row) * G;      // bytes between runs of tiles
                switch (pieces) {
                    case 1: generic_fill_stage<kBK, kBN, 1>(sw, src0, krow_stride, p.br_log2, p.bc_log2, k_rows_left, n_cols_left, lane); break;
                    case 2: generic_fill_stage<kBK, kBN, 2>(sw, src0, krow_stride, p.br_log2, p.bc_log2, k_rows_left, n_cols_left, lane); break;
                    case 4: generic_fill_stage<kBK, kBN, 4>(sw, src0, krow_stride, p.br_log2, p.bc_log2, k_rows_left, n_cols_left, lane); break;
                    default: generic_fill_stage<kBK, kBN, 8>(sw, src0, krow_stride, p.br_log2, p.bc_log2, k_rows_left, n_cols_left, lane); break;
                }
                fence_proxy_async_smem();            // generic-proxy stores -> visible to the tensor-core (async) proxy
                __syncwarp();
                if (lane == 0) mbar_arrive(&full_bar[stage]);
            }
        }
    } else {
        // =============================================================== epilogue
        const int quarter = warp & 3;                    // TMEM lanes 32*quarter .. +31
        const int et = (warp - 2) * 32 + lane;           // 0..127 among epilogue threads
        uint32_t acc = 0, acc_phase = 0;
        Work w;
        while (sched.next(w)) {
            const TileInfo t = decode_tile(p, prefix, row_start, w.tile);
            const bool full = (w.kbeg == 0 && w.kend == p.k_iters);
            const int n_mma = (t.rows + 15) & ~15;
            const long long ce0 = TL_CLOCK();
            bool ok = mbar_wait_bounded(&acc_full_bar[acc], acc_phase, abort_ptr, p.status, kWaitEpilogueAccFull);
            const long long ce1 = TL_CLOCK();
            (void)ce0; (void)ce1;
            tc_fence_after_sync();
            if (et == 0) TL_STAMP_ONCE(4);
            float* out;
            int64_t ld;
            if (full) {
                out = p.C + int64_t(t.row0) * p.ldc + t.n0;
                ld = p.ldc;
            } else {
                out = p.partials + size_t(sched.slot(sched.cta, w.tile)) * p.BM * kBN;
                ld = kBN;
            }
            if (ok && kWN) {
                // TMEM lane = token row, columns = the tile's kBN weight columns: each thread owns one row of C.
                // (MMA of 64 rows: rows 16q..16q+15 sit in the lower half of lane quarter q, the upper 16 lanes of
                // each quarter hold nothing.)
                const bool m64 = p.umma_m == 64;
                const int row = m64 ? (lane < 16 ? quarter * 16 + lane : p.BM) : quarter * 32 + lane;
                const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + acc * uint32_t(acc_cols);
                if ((m64 ? quarter * 16 : quarter * 32) < t.rows) {      // this lane quarter holds at least one real row
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
            const long long ce2 = TL_CLOCK();
            (void)ce2;
            if (et == 0) { TL_COUNT(6, ce1 - ce0); TL_COUNT(7, ce2 - ce1); TL_COUNT(9, 1); }
            acc ^= 1;
            if (acc == 0) acc_phase ^= 1;

            if (et == 0) { TL_STAMP(5); TL_COUNT(8, TL_CLOCK() - ce2); }
            if (*abort_ptr) break;
        }
    }

    // --------------------------------------------------------------- teardown
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0) { TL_COUNT(11, TL_CLOCK()); TL_COUNT(13, global_timer_ns()); }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

// Stream-K reduction.  The GEMM kernel leaves the partial sum of every (CTA, split tile) in its workspace slot
// and does no synchronisation of its own; this kernel, ordered after it by the stream, adds the partials of
// each split tile in K order (lowest CTA first) and writes C.  One CTA per boundary between two ranges of
// the GEMM grid: the boundary's tile is reduced by the first boundary that falls inside it.
__global__ void __launch_bounds__(128) streamk_reduce_kernel(const __grid_constant__ GemmParams p, int gemm_grid) {
    __shared__ int prefix[kMaxExperts + 1];
    __shared__ int row_start[kMaxExperts + 1];
    // Launched with programmatic stream serialisation, and the GEMM kernel lets its dependents launch as soon
    // as it has started: this grid is resident and has done all of its index arithmetic (which reads only
    // the call's inputs) while the GEMM grid is still running.  Nothing the GEMM kernel wrote is read before
    // griddepcontrol.wait, which returns once that grid has completed and its writes are visible.
#ifdef TL_TIMELINE
    if (threadIdx.x == 0 && g_timeline) g_timeline[(256 + blockIdx.x) * 8 + 0] = global_timer_ns();
#endif
    // The kernel after this one in the stream may start its own set-up now; it waits for this grid to complete
    // before it reads or writes anything.
    if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    load_row_starts(p, row_start);
    __syncthreads();
    if (threadIdx.x < 32) tile_prefix(p, row_start, prefix);
    __syncthreads();
    Sched sched;
    sched.init(1, p.k_iters, prefix[p.E], gemm_grid, 0, nullptr);
    const int c = int(blockIdx.x) + 1;                     // boundary between CTA c-1 and CTA c
    if (c >= sched.grid_eff) return;
    const long long b = sched.range_begin(c);
    const int tile = int(b / p.k_iters);
    const long long tile_begin = static_cast<long long>(tile) * p.k_iters;
    if (b == tile_begin) return;                           // the boundary coincides with a tile boundary
    if (sched.range_begin(c - 1) > tile_begin) return;     // an earlier boundary lies in this tile: it reduces
    const int c_lo = c - 1;
    const int c_hi = sched.owner(tile_begin + p.k_iters - 1);
    const TileInfo t = decode_tile(p, prefix, row_start, tile);
    float* dst = p.C + int64_t(t.row0) * p.ldc + t.n0;
    // slots of the contributors, computed before the wait (the load loop below must not divide)
    __shared__ int slot_of[kRangeTabMax];
    for (int j = threadIdx.x; j <= c_hi - c_lo && j < kRangeTabMax; j += blockDim.x) slot_of[j] = sched.slot(c_lo + j, tile);
    __syncthreads();
    asm volatile("griddepcontrol.wait;" ::: "memory");
#ifdef TL_TIMELINE
    if (threadIdx.x == 0 && g_timeline) g_timeline[(256 + blockIdx.x) * 8 + 1] = global_timer_ns();
#endif
    const int vec_per_row = p.BN / 4;
    const int total_vec = t.rows * vec_per_row;
    const size_t slot_floats = size_t(p.BM) * p.BN;
    for (int v0 = 0; v0 < total_vec; v0 += 4 * 128) {
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
                    const int v = v0 + q * 128 + int(threadIdx.x);
                    x[j][q] = (c_ok && v < total_vec) ? __ldcg(src + v) : make_float4(0.f, 0.f, 0.f, 0.f);
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
            const int v = v0 + q * 128 + int(threadIdx.x);
            if (v < total_vec) {
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
#ifdef TL_TIMELINE
    if (threadIdx.x == 0 && g_timeline) g_timeline[(256 + blockIdx.x) * 8 + 2] = global_timer_ns();
#endif
}

}  // namespace tl
#include "tl_gemm_pair.cuh"
namespace tl {

// ======================================================================== host

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// Encoded maps are kept: encoding costs microseconds of host time per map and the same
// (pointer, shape, box) recurs on every call of a serving loop.
struct MapKey {
    const void* base;
    int rank, dtype, swizzle;
    uint64_t dims[5], strides[5];
    uint32_t box[5];
    bool operator==(const MapKey& o) const { return memcmp(this, &o, sizeof(MapKey)) == 0; }
};
struct MapEntry {
    MapKey key;
    CUtensorMap map;
};
static constexpr int kMapCacheSize = 256;

int encode_tensor_map(CUtensorMap* out, const void* base, int dtype, int swizzle, int rank, const uint64_t* dims,
                      const uint64_t* strides_bytes, const uint32_t* box) {
    static MapEntry* cache = new MapEntry[kMapCacheSize];
    static int cache_n = 0, cache_next = 0;
    MapKey key;
    memset(&key, 0, sizeof key);
    key.base = base;
    key.rank = rank;
    key.dtype = dtype;
    key.swizzle = swizzle;
    for (int i = 0; i < rank; ++i) { key.dims[i] = dims[i]; key.strides[i] = strides_bytes[i]; key.box[i] = box[i]; }
    for (int i = 0; i < cache_n; ++i)
        if (cache[i].key == key) {
            *out = cache[i].map;
            return TL_OK;
        }
    EncodeTiledFn fn = encode_fn();
    if (!fn) {
        state().last_cuda_error = int(cudaErrorSymbolNotFound);
        return TL_ERR_CUDA;
    }
    cuuint64_t gdim[5], gstr[4];
    cuuint32_t bdim[5], estr[5];
    for (int i = 0; i < rank; ++i) { gdim[i] = dims[i]; bdim[i] = box[i]; estr[i] = 1; }
    for (int i = 0; i + 1 < rank; ++i) gstr[i] = strides_bytes[i + 1];
    CUresult r = fn(out, CUtensorMapDataType(dtype), cuuint32_t(rank), const_cast<void*>(base), gdim, gstr, bdim, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CUtensorMapSwizzle(swizzle), CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        state().last_cuda_error = int(r);
        return TL_ERR_CUDA;
    }
    const int slot = cache_n < kMapCacheSize ? cache_n++ : (cache_next++ % kMapCacheSize);
    cache[slot].key = key;
    cache[slot].map = *out;
    return TL_OK;
}

// bf16 operands of the GEMM, 128-byte swizzle
static int encode(CUtensorMap* out, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                  const uint32_t* box) {
    return encode_tensor_map(out, base, int(CU_TENSOR_MAP_DATA_TYPE_BFLOAT16), int(CU_TENSOR_MAP_SWIZZLE_128B), rank, dims,
                             strides_bytes, box);
}

static int ilog2(int64_t x) {
    int l = 0;
    while ((int64_t(1) << l) < x) ++l;
    return l;
}

struct GemmPlan {
    int BM, BN, BK;
    int umma_m, a_rows;          // see GemmParams
    int weights_on_n;     // kWN variant of the kernel
    int stream_k;
    int grid;
    int num_stages;
    size_t smem_bytes;
    size_t ws_bytes;
};

static int pick_bm(int64_t rows) {
    int bm = 16;
    while (bm < 256 && bm < rows) bm <<= 1;
    return bm;
}

// Chooses / validates the CTA tile and the schedule.  rows_max: most rows any one problem has.
// Default CTA tile (measured on B200, Llama-70B and Qwen-30B shapes).
//   up to 16 rows      16 x 256 x 64: tokens on the MMA's M side, 256 weight columns per instruction; the
//                      partial tiles of stream-K are still small (16 KB)
//   up to 128 rows     rows x 128 x 128: same orientation, narrower tile so that partial tiles stay small,
//                      deeper K step so that there are half as many barrier hand-offs
//   more rows          256 x 128 x 64 with the weights on the M side (prefill)
//   grouped            at most 32 rows per tile: most experts have a handful of rows, and a large cap costs
//                      pipeline stages and partial-tile bytes for every tile
//   narrow_scratch     (fixed-size scratch) never the 256-column tile
static void default_tile(int64_t rows_max, bool grouped, bool narrow_scratch, int* BM, int* BN, int* BK) {
    *BM = pick_bm(rows_max);
    if (grouped && *BM > 32) *BM = 32;
    if (*BM <= 16 && !narrow_scratch && !grouped) { *BN = 256; *BK = 64; }
    else if (*BM <= 128) { *BN = 128; *BK = 128; }
    else { *BN = 128; *BK = 64; }
}

static int make_plan(int64_t rows_max, int64_t tile_bound, int64_t N, int64_t K, int cta_m, int cta_n, int cta_k,
                     bool grouped, GemmPlan* plan, bool narrow_scratch = false) {
    if (int rc = ensure_device_info()) return rc;
    const int sms = state().sm_count;
    int BM = cta_m, BN = cta_n, BK = cta_k;
    if (BM == 0 && BN == 0 && BK == 0) default_tile(rows_max, grouped, narrow_scratch, &BM, &BN, &BK);
    if (BM != 16 && BM != 32 && BM != 64 && BM != 128 && BM != 256) return TL_ERR_UNSUPPORTED;
    if (BN != 64 && BN != 128 && BN != 256) return TL_ERR_UNSUPPORTED;
    if (BK != 64 && BK != 128) return TL_ERR_UNSUPPORTED;
    if (BN == 256 && BM > 128) return TL_ERR_UNSUPPORTED;   // 2 accumulators x 2 groups x BM columns <= 512
    plan->BM = BM; plan->BN = BN; plan->BK = BK;
    plan->weights_on_n = BM <= 128;                         // tokens fit the 128 rows of the MMA's M side
    // With the tokens on the M side the MMA reads 64 rows (tiles of up to 64 tokens) or 128: a stage holds that
    // many token rows per 64-wide K slice, the ones beyond BM zeroed once by the kernel.  They only feed
    // accumulator rows that are never stored.
    static const bool m128_only = getenv("TL_UMMA_M128") && atoi(getenv("TL_UMMA_M128")) != 0;    // measurement switch
    plan->umma_m = BM <= 64 && !m128_only ? 64 : 128;
    plan->a_rows = plan->weights_on_n && BM < plan->umma_m ? plan->umma_m : BM;
    const size_t stage = size_t(BK) * BN * 2 + size_t(BK / 64) * plan->a_rows * kAtomBytes;
    // 1 KB of slack to align the stages to 1024 bytes.
    // 12 KB stay free so that a CTA of the stream-K reduction kernel can be resident next to this one.
    const size_t budget = kMaxDynamicSmem - 1024 - 12 * 1024;
    int stages = int(budget / stage);
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) return TL_ERR_UNSUPPORTED;
    if (const char* e = getenv("TL_MAX_STAGES")) {          // measurement hook
        const int cap = atoi(e);
        if (cap >= 2 && cap < stages) stages = cap;
    }
    plan->num_stages = stages;
    plan->smem_bytes = size_t(stages) * stage + 1024;
    if (plan->smem_bytes < 120 * 1024) plan->smem_bytes = 120 * 1024;   // one CTA per SM: TMEM is not shared
    const int64_t k_iters = ceil_div(K, BK);
    const int64_t total_iters = tile_bound * k_iters;
    // Whole tiles when they fill the machine evenly enough, contiguous K ranges otherwise.
    const int64_t waves = ceil_div(tile_bound, sms);
    const bool even = tile_bound >= sms && double(tile_bound) / double(waves * sms) >= 0.92;
    plan->stream_k = (grouped || !even) ? 1 : 0;
    int64_t grid = plan->stream_k ? (total_iters < sms ? total_iters : sms) : (tile_bound < sms ? tile_bound : sms);
    if (grid < 1) grid = 1;
    plan->grid = int(grid);
    plan->ws_bytes = plan->stream_k ? size_t(2) * size_t(grid) * BM * BN * sizeof(float) : 0;   // two slots per CTA
    return TL_OK;
}

// Where a launch takes its scratch from when the caller of gemm_launch supplies it itself.
struct FixedScratch {
    void* ws;            // partial tiles
    size_t ws_bytes;
    uint32_t* status;    // word the kernel raises when a bounded wait expires
};

static int gemm_launch(const void* d_A, const void* d_B, float* d_C, const int32_t* d_offsets, int E,
                       int64_t rows_total, int64_t rows_max, int64_t N, int64_t K, int64_t G, int br, int bc,
                       int cta_m, int cta_n, int cta_k, cudaStream_t stream, const FixedScratch* fixed = nullptr,
                       bool kmajor = false, int elem_bytes = 2, void* d_H_swiglu = nullptr, void* d_C_bf16 = nullptr) {
    const int es = elem_bytes;                       // 2: bf16, 1: FP8 (E4M3), K-contiguous weights only
    const int k_shift = es == 1 ? 1 : 0;
    if (es != 2 && !(es == 1 && kmajor)) return TL_ERR_UNSUPPORTED;
    if (rows_total < 0 || N <= 0 || K <= 0 || E < 1) return TL_ERR_INVALID_ARG;
    if (rows_total == 0) return TL_OK;
    if (!d_A || !d_B || (!d_C && !d_H_swiglu && !d_C_bf16)) return TL_ERR_INVALID_ARG;
    if (d_C_bf16 && (N % 8 != 0 || reinterpret_cast<uintptr_t>(d_C_bf16) % 16 != 0)) return TL_ERR_INVALID_ARG;
    if (d_H_swiglu && (N % 64 != 0 || reinterpret_cast<uintptr_t>(d_H_swiglu) % 16 != 0)) return TL_ERR_INVALID_ARG;
    if (rows_total >= (int64_t(1) << 31) || N >= (int64_t(1) << 31) || K * int64_t(E) >= (int64_t(1) << 31))
        return TL_ERR_UNSUPPORTED;
    if (E > kMaxExperts) return TL_ERR_UNSUPPORTED;
    // br x bc is the memory tile of the STORED matrix: K-rows x N-columns, or N-rows x K-columns when kmajor.
    if (br != 0) {
        if (br < 0 || bc <= 0 || int64_t(br) * bc * es != G) return TL_ERR_INVALID_ARG;
        if (!is_pow2(br) || !is_pow2(bc)) return TL_ERR_UNSUPPORTED;
        if (kmajor ? (N % br != 0 || K % bc != 0) : (K % br != 0 || N % bc != 0)) return TL_ERR_INVALID_ARG;
    }
    if (kmajor) {
        // K-major operand: a tile row is one swizzle row of 128, 64 or 32 bytes; shorter rows have no path here
        if (br != 0 && bc * es < 32) return TL_ERR_UNSUPPORTED;
        if (K % (br != 0 ? 32 / es : 128 / es) != 0) return TL_ERR_UNSUPPORTED;
    }
    // One-row memory tiles are row-major (Section 3.1: the (1, G/s) extreme).
    const bool row_major = br == 0 || (!kmajor && br == 1 && N % 64 == 0);
    // TMA boxes need 128-byte rows (64 columns); narrower memory tiles take the generic-address path.
    // 16- and 32-column memory tiles (32- and 64-byte rows) are TMA-boxable with the narrower swizzles.
    const bool narrow = !kmajor && !row_major && (bc == 16 || bc == 32);
    const bool generic = !kmajor && !row_major && bc < 64 && !narrow;
    if (!kmajor && row_major && N % 64 != 0) return TL_ERR_UNSUPPORTED;
    if (generic && (G < 16 || br > 128 || bc > 256)) return TL_ERR_UNSUPPORTED;   // tile must fit the CTA tile
    if ((K * es) % 16 != 0) return TL_ERR_UNSUPPORTED;          // 16-byte row pitch of A
    if (reinterpret_cast<uintptr_t>(d_A) % 16 != 0) return TL_ERR_ALIGNMENT;
    if (reinterpret_cast<uintptr_t>(d_B) % (row_major || generic ? 16 : 128) != 0) return TL_ERR_ALIGNMENT;
    if (reinterpret_cast<uintptr_t>(d_C) % 16 != 0) return TL_ERR_ALIGNMENT;

    GemmPlan plan;
    {
        // upper bound of tiles: every expert may add one ragged m-tile
        int bm_guess = cta_m, bn_guess = cta_n, bk_guess = cta_k;
        if (cta_m == 0 && cta_n == 0 && cta_k == 0)
            default_tile(rows_max, d_offsets != nullptr, fixed != nullptr, &bm_guess, &bn_guess, &bk_guess);
        if (bm_guess <= 0 || bn_guess <= 0) return TL_ERR_UNSUPPORTED;
        const int64_t mt_bound = d_offsets ? rows_total / bm_guess + E : ceil_div(rows_total, bm_guess);
        // (the plan counts K in 2-byte units: an 8-bit stage holds twice as many elements)
        if (int rc = make_plan(rows_max, mt_bound * ceil_div(N, bn_guess), N, K >> k_shift, cta_m, cta_n, cta_k,
                               d_offsets != nullptr, &plan, fixed != nullptr))
            return rc;
    }
    if (d_offsets && K % (int64_t(plan.BK) << k_shift) != 0) return TL_ERR_UNSUPPORTED;
    if (d_H_swiglu && !plan.weights_on_n) return TL_ERR_UNSUPPORTED;        // the gated epilogue pairs columns of one token row   // a K tail would read the next expert's rows
    void* ws = nullptr;
    if (fixed) {
        if (plan.ws_bytes > fixed->ws_bytes) return TL_ERR_WORKSPACE;
        ws = plan.ws_bytes ? fixed->ws : nullptr;
        // A fixed scratch keeps the previous launch's contents; nothing in it has to start at zero: every
        // partial tile is written by the GEMM kernel before the reduction kernel reads it.
    } else {
        if (int rc = ensure_control()) return rc;
        if (int rc = get_workspace(plan.ws_bytes, &ws)) return rc;
    }

    static const bool pdl_ok = !(getenv("TL_NO_PDL") && atoi(getenv("TL_NO_PDL")) != 0);
    GemmParams p;
    memset(&p, 0, sizeof p);
    // ---- token operand A: [rows_total][K], boxes of 128 bytes of K x {16..256} rows
    const int dtype = es == 1 ? int(CU_TENSOR_MAP_DATA_TYPE_UINT8) : int(CU_TENSOR_MAP_DATA_TYPE_BFLOAT16);
    for (int i = 0; i < kNumBoxChoices; ++i) {
        const uint64_t dims[2] = {uint64_t(K), uint64_t(rows_total)};
        const uint64_t str[2] = {uint64_t(es), uint64_t(K) * es};
        const uint32_t box[2] = {uint32_t(128 / es), uint32_t(16 << i)};
        if (int rc = encode_tensor_map(&p.tmap_a[i], d_A, dtype, int(CU_TENSOR_MAP_SWIZZLE_128B), 2, dims, str, box))
            return rc;
    }
    p.fp8 = es == 1;
    p.k_shift = k_shift;
    uint32_t w_layout = 2;
    // ---- weight operand B
    const int NA = plan.BN / 64;                                  // 128-byte atoms across the CTA tile
    int RB, AB, nb_box = 1, kb_box = 1;         // box: rows, atoms, memory tiles along N and K
    int w_row_bytes = kAtomBytes;                // K-major weights: bytes of one swizzle row
    if (kmajor) {
        // Weights [N][K], K contiguous.  Tiled (Eq. 2 as printed, a = bc along K, b = br along N), with the tile
        // row cut into swizzle rows of r = min(128 bytes, tile row) holding e elements: the 5-D view
        // (e, b, E*N/b, a/e, K/a) with strides (1, a, b*K, e, a*b) elements; the box takes, for every swizzle row
        // of the stage's K range, all weight rows of the CTA tile, so the bytes land as [K row][cta_n rows][r]:
        // the canonical K-major operand in 128-, 64- or 32-byte swizzle.  Untiled: (e, E*N, 1, K/e, 1), r = 128.
        RB = plan.BK;
        AB = NA;
        const int bk_el = plan.BK << k_shift;                    // K elements per stage
        w_row_bytes = row_major ? kAtomBytes : (bc * es < kAtomBytes ? bc * es : kAtomBytes);
        const int e = w_row_bytes / es;
        const int swz = w_row_bytes == 128 ? int(CU_TENSOR_MAP_SWIZZLE_128B)
                                           : w_row_bytes == 64 ? int(CU_TENSOR_MAP_SWIZZLE_64B) : int(CU_TENSOR_MAP_SWIZZLE_32B);
        if (row_major) {
            const uint64_t big = uint64_t(K) * es * uint64_t(N) * E;
            const uint64_t dims[5] = {uint64_t(e), uint64_t(N) * E, 1, uint64_t(K / e), 1};
            const uint64_t str[5] = {uint64_t(es), uint64_t(K) * es, big, uint64_t(w_row_bytes), big};
            const uint32_t box[5] = {uint32_t(e), uint32_t(plan.BN), 1, uint32_t(bk_el / e), 1};
            if (int rc = encode_tensor_map(&p.tmap_b, d_B, dtype, swz, 5, dims, str, box)) return rc;
            p.k_coord_per_expert = int(N);
        } else {
            const int rows_box = br < plan.BN ? br : plan.BN;
            const int k_box = bc < bk_el ? bc : bk_el;
            const uint64_t dims[5] = {uint64_t(e), uint64_t(br), uint64_t(N / br) * E, uint64_t(bc / e), uint64_t(K / bc)};
            const uint64_t str[5] = {uint64_t(es), uint64_t(bc) * es, uint64_t(br) * uint64_t(K) * es, uint64_t(w_row_bytes),
                                     uint64_t(G)};
            const uint32_t box[5] = {uint32_t(e), uint32_t(rows_box), uint32_t(plan.BN / rows_box), uint32_t(k_box / e),
                                     uint32_t(bk_el / k_box)};
            if (int rc = encode_tensor_map(&p.tmap_b, d_B, dtype, swz, 5, dims, str, box)) return rc;
            p.k_coord_per_expert = int(N / br);
            p.br_log2 = ilog2(br);
            p.bc_log2 = ilog2(bc);
        }
        p.w_kmajor = 1;
        p.w_atom_log2 = ilog2(e);
        w_layout = w_row_bytes == 128 ? 2u : w_row_bytes == 64 ? 4u : 6u;
    } else if (generic) {
        // No tensor map: warps 6..9 of the kernel compute Eq. 1-2 addresses themselves and build the
        // canonical [atom][cta_k rows][64] image in shared memory.
        if (plan.BK % br != 0 || plan.BN % bc != 0) return TL_ERR_UNSUPPORTED;
        RB = plan.BK;
        AB = NA;
        p.generic_b = 1;
        p.B = static_cast<const uint8_t*>(d_B);
        p.expert_bytes = K * N * 2;
        p.blocks_per_row = int(N / bc);
        p.br_log2 = ilog2(br);
        p.bc_log2 = ilog2(bc);
    } else if (row_major) {
        // [E*K][N] seen as (64, E*K, N/64): one box covers the whole stage.
        RB = plan.BK;
        AB = NA;
        const uint64_t dims[5] = {64, uint64_t(K) * E, uint64_t(N / 64), 1, 1};
        const uint64_t str[5] = {2, uint64_t(N) * 2, 128, uint64_t(N) * 2 * uint64_t(K) * E, uint64_t(N) * 2 * uint64_t(K) * E};
        const uint32_t box[5] = {64, uint32_t(RB), uint32_t(AB), 1, 1};
        if (int rc = encode(&p.tmap_b, d_B, 5, dims, str, box)) return rc;
        p.k_coord_per_expert = int(K);
    } else {
        // Eq. 3 in the N-contiguous flavour, contiguous extent split into 64-element atoms:
        // (64, br, bc/64, N/bc, E*K/br) with strides (1, bc, 64, br*bc, br*N) elements.
        if (narrow) {
            // Tile rows of 32 or 64 bytes: one tile row is one swizzle row (32- or 64-byte swizzle), dimensions in the
            // K-inner order described below; the stage lands as [bc-column atom][cta_k rows][bc*2 bytes].
            const int rows_box = br < plan.BK ? br : plan.BK;
            RB = plan.BK;
            AB = NA;
            const uint64_t dims[5] = {uint64_t(bc), uint64_t(br), uint64_t(K / br) * E, 1, uint64_t(N / bc)};
            const uint64_t str[5] = {2, uint64_t(bc) * 2, uint64_t(br) * uint64_t(N) * 2, uint64_t(bc) * 2, uint64_t(G)};
            const uint32_t box[5] = {uint32_t(bc), uint32_t(rows_box), uint32_t(plan.BK / rows_box), 1, uint32_t(plan.BN / bc)};
            if (int rc = encode_tensor_map(&p.tmap_b, d_B, dtype, bc == 32 ? int(CU_TENSOR_MAP_SWIZZLE_64B) : int(CU_TENSOR_MAP_SWIZZLE_32B),
                                           5, dims, str, box))
                return rc;
            p.k_coord_per_expert = int(K / br);
            p.br_log2 = ilog2(br);
            p.bc_log2 = ilog2(bc);
            p.k_inner = 1;
        } else if (br < 8) {
            // Memory tiles shorter than the 8 rows of a swizzle atom: the same view with its dimensions in another
            // order, (64, br, E*K/br, bc/64, N/bc) with strides (1, bc, br*N, 64, br*bc).  The box takes all K
            // tiles of the stage before it moves to the next 64-column atom, so under every atom the stage's K
            // rows follow each other: [N tile][atom][K tile][row][64] = [atom][cta_k rows][64], canonical again.
            RB = plan.BK;
            AB = (bc < plan.BN ? bc : plan.BN) / 64;
            nb_box = NA / AB;
            const uint64_t dims[5] = {64, uint64_t(br), uint64_t(K / br) * E, uint64_t(bc / 64), uint64_t(N / bc)};
            const uint64_t str[5] = {2, uint64_t(bc) * 2, uint64_t(br) * uint64_t(N) * 2, 128, uint64_t(G)};
            const uint32_t box[5] = {64, uint32_t(br), uint32_t(plan.BK / br), uint32_t(AB), uint32_t(nb_box)};
            if (int rc = encode(&p.tmap_b, d_B, 5, dims, str, box)) return rc;
            p.k_coord_per_expert = int(K / br);
            p.br_log2 = ilog2(br);
            p.bc_log2 = ilog2(bc);
            p.k_inner = 1;
        } else {
        RB = br < plan.BK ? br : plan.BK;
        AB = (bc < plan.BN ? bc : plan.BN) / 64;
        // One TMA instruction per stage whose box is a whole number of memory tiles (box extents 3 and 4
        // count tiles along N and K).  TL_BOX_PER_BLOCK=1 issues one instruction per memory tile instead
        // (same bytes, same shared-memory image; measurably slower because instruction issue then limits).
        static const bool per_block = getenv("TL_BOX_PER_BLOCK") && atoi(getenv("TL_BOX_PER_BLOCK")) != 0;
        nb_box = per_block ? 1 : NA / AB;
        kb_box = per_block ? 1 : plan.BK / RB;
        const uint64_t dims[5] = {64, uint64_t(br), uint64_t(bc / 64), uint64_t(N / bc), uint64_t(K / br) * E};
        const uint64_t str[5] = {2, uint64_t(bc) * 2, 128, uint64_t(G), uint64_t(br) * uint64_t(N) * 2};
        const uint32_t box[5] = {64, uint32_t(RB), uint32_t(AB), uint32_t(nb_box), uint32_t(kb_box)};
        if (int rc = encode(&p.tmap_b, d_B, 5, dims, str, box)) return rc;
        p.k_coord_per_expert = int(K / br);
        p.br_log2 = ilog2(br);
        p.bc_log2 = ilog2(bc);
        }
    }
    {
        // coordinate maps (see GemmParams): which bits of k and n each tensor-map dimension takes
        auto set = [&](int i, int ks, int km, int ns, int nm, int ex) {
            p.ck_shift[i] = ks; p.ck_mask[i] = km; p.cn_shift[i] = ns; p.cn_mask[i] = nm; p.c_expert[i] = ex;
        };
        const int all = -1;
        for (int i = 0; i < 4; ++i) set(i, 0, 0, 0, 0, 0);
        if (generic) {
        } else if (kmajor && row_major) {           // (row of K-elements, N row, -, swizzle row along K, -)
            set(0, 0, 0, 0, all, 1);
            set(2, p.w_atom_log2, all, 0, 0, 0);
        } else if (kmajor) {                        // (.., row in tile, tile along N, swizzle row in tile, tile along K)
            set(0, 0, 0, 0, br - 1, 0);
            set(1, 0, 0, p.br_log2, all, 1);
            set(2, p.w_atom_log2, (bc >> p.w_atom_log2) - 1, 0, 0, 0);
            set(3, p.bc_log2, all, 0, 0, 0);
        } else if (row_major) {                     // (64 columns, K row, 64-column atom, -, -)
            set(0, 0, all, 0, 0, 1);
            set(1, 0, 0, 6, all, 0);
        } else if (p.k_inner) {                     // (.., row in tile, tile along K, atom in tile, tile along N)
            set(0, 0, br - 1, 0, 0, 0);
            set(1, p.br_log2, all, 0, 0, 1);
            set(2, 0, 0, 6, bc >= 64 ? (bc >> 6) - 1 : 0, 0);
            set(3, 0, 0, p.bc_log2, all, 0);
        } else {                                    // (.., row in tile, atom in tile, tile along N, tile along K)
            set(0, 0, br - 1, 0, 0, 0);
            set(1, 0, 0, 6, (bc >> 6) - 1, 0);
            set(2, 0, 0, p.bc_log2, all, 0);
            set(3, p.br_log2, all, 0, 0, 1);
        }
    }
    p.row_major = row_major;
    p.kbx = generic ? 0 : plan.BK / (RB * kb_box);
    p.nbx = generic ? 0 : NA / (AB * nb_box);
    p.box_rows = RB * kb_box;                                     // K rows and atoms one instruction covers
    p.box_atoms = AB * nb_box;
    p.box_bytes = uint32_t(RB) * AB * kAtomBytes * nb_box * kb_box;
    // Shared-memory image of a stage: [K box][N box][atom][row][64 elements].  Atom stride is RB*128
    // everywhere; 8-row groups are 1024 bytes apart inside a box and one box row apart across boxes.
    const uint32_t krow_bytes = uint32_t(NA) * RB * kAtomBytes;   // all boxes sharing one K range
    p.lbo = uint32_t(RB) * kAtomBytes;
    p.sbo = RB >= 16 ? 1024u : krow_bytes;
    p.ugroup_off = 2u * p.lbo;
    for (int j = 0; j < plan.BK / 16; ++j) {
        const int row = j * 16;
        p.kstep_off[j] = uint32_t(row / RB) * krow_bytes + uint32_t(row % RB) * kAtomBytes;
    }
    if (narrow) {
        // MN-major image with narrow atoms: [bc-column atom][cta_k rows][r = bc*2 bytes]; 8-row groups 8r apart, the
        // next atom cta_k rows further, a K step of 16 rows 16r further.
        const uint32_t r = uint32_t(bc) * 2u;
        p.lbo = uint32_t(plan.BK) * r;
        p.sbo = 8u * r;
        p.ugroup_off = (128u / uint32_t(bc)) * p.lbo;
        for (int j = 0; j < plan.BK / 16; ++j) p.kstep_off[j] = uint32_t(j) * 16u * r;
        p.box_rows = plan.BK;
        p.box_atoms = NA;
        p.kbx = p.nbx = 1;
        p.box_bytes = uint32_t(plan.BK) * plan.BN * 2;
        w_layout = bc == 32 ? 4u : 6u;
    }
    if (kmajor) {
        // K-major image: [swizzle row along K][cta_n rows][r bytes]; 8-row groups 8r bytes apart, a K step of one
        // instruction (32 bytes) is 32 bytes further inside the swizzle row, the next swizzle row cta_n rows further.
        const uint32_t r = uint32_t(w_row_bytes), steps_per_row = r / 32u;
        p.lbo = 16;
        p.sbo = 8u * r;
        p.ugroup_off = 128u * r;
        for (int j = 0; j < plan.BK / 16; ++j)
            p.kstep_off[j] = (uint32_t(j) / steps_per_row) * uint32_t(plan.BN) * r + (uint32_t(j) % steps_per_row) * 32u;
        p.box_rows = plan.BK << k_shift;
        p.box_atoms = NA;
        p.kbx = p.nbx = 1;
        p.box_bytes = uint32_t(plan.BK) * plan.BN * 2;
    }
    p.w_desc_hi = smem_desc_hi(p.lbo, p.sbo, w_layout);
    p.C = d_C;
    p.Cb = static_cast<__nv_bfloat16*>(d_C_bf16);
    p.epi_swiglu = d_H_swiglu != nullptr;
    p.H = static_cast<__nv_bfloat16*>(d_H_swiglu);
    p.ldh = N / 2;
    p.partials = static_cast<float*>(ws);
    p.offsets = d_offsets;
    p.status = fixed ? fixed->status : state().ctl.d_status;
    p.ldc = N;
    p.M = int(rows_total);
    p.N = int(N);
    p.K = int(K);
    p.E = E;
    p.BM = plan.BM;
    p.umma_m = plan.umma_m;
    p.a_rows = plan.a_rows;
    p.BN = plan.BN;
    p.n_tiles = int(ceil_div(N, plan.BN));
    p.k_iters = int(ceil_div(K, int64_t(plan.BK) << k_shift));
    p.stream_k = plan.stream_k;
    p.num_stages = plan.num_stages;
    static const int prefetch_env = getenv("TL_PREFETCH_STAGES") ? atoi(getenv("TL_PREFETCH_STAGES")) : -1;   // measurement hook
    // (at most four instructions: the thread that issues them holds up the CTA's first barrier for their duration)
    p.prefetch_stages = !pdl_ok ? 0 : (prefetch_env >= 0 ? prefetch_env : (plan.num_stages < 4 ? plan.num_stages : 4));

    cudaError_t err = cudaSuccess;
    // Large dense problems on TMA-readable weights: CTA pairs (cta_group::2 MMAs), see tl_gemm_pair.cuh.
    static const bool no_pair = getenv("TL_NO_PAIR") && atoi(getenv("TL_NO_PAIR")) != 0;     // measurement switch
    // Worth it once every cluster of the machine has at least one 256 x 256 tile; smaller problems keep the
    // single-CTA kernel and its stream-K split.
    if (!no_pair && !d_offsets && !generic && !d_H_swiglu && plan.BM == 256 && plan.BN == 128 && plan.BK == 64 &&
        p.kbx == 1 && p.nbx == 1 && ceil_div(rows_total, 256) * ceil_div(N, 256) * 2 >= state().sm_count) {
        static int max_clusters = -1;
        if (max_clusters < 0) {
            err = cudaFuncSetAttribute(gemm_pair_kernel<false, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynamicSmem);
            if (err == cudaSuccess)
                err = cudaFuncSetAttribute(gemm_pair_kernel<true, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynamicSmem);
            if (err == cudaSuccess)
                err = cudaFuncSetAttribute(gemm_pair_kernel<false, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynamicSmem);
            if (err == cudaSuccess)
                err = cudaFuncSetAttribute(gemm_pair_kernel<true, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynamicSmem);
            if (err != cudaSuccess) return check_cuda(err);
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(2 * state().sm_count);
            cfg.blockDim = dim3(kGemmThreads);
            cfg.dynamicSmemBytes = kMaxDynamicSmem;
            int n = 0;
            err = cudaOccupancyMaxActiveClusters(&n, gemm_pair_kernel<false, 1>, &cfg);
            if (err != cudaSuccess) return check_cuda(err);
            max_clusters = n > 0 ? n : 1;
        }
        // 512-token tiles (one weight slab per stage for two token blocks) as long as they fill whole waves of
        // clusters; what is left of the tile grid runs as 256-token tiles.  TL_PAIR_HALVES=1: 256-token tiles only.
        static const bool halves_off = getenv("TL_PAIR_HALVES") && atoi(getenv("TL_PAIR_HALVES")) == 1;
        const int64_t big_total = ceil_div(rows_total, 512) * ceil_div(N, 256);
        const int64_t big_tiles = halves_off ? 0 : (big_total / max_clusters) * max_clusters;
        const int halves = big_tiles > 0 ? 2 : 1;
        const size_t stage_bytes = 64 * 128 * 2 + size_t(halves) * 128 * kAtomBytes;
        const int stages = int((kMaxDynamicSmem - 1024) / stage_bytes);
        p.num_stages = stages < kPairStagesMax ? stages : kPairStagesMax;
        p.pair_big_tiles = int(big_tiles);
        const size_t smem = size_t(p.num_stages) * stage_bytes + 1024;
        const int64_t pair_tiles = halves == 2 ? big_tiles + 2 * (big_total - big_tiles)
                                               : ceil_div(rows_total, 256) * ceil_div(N, 256);
        const int clusters = int(pair_tiles < max_clusters ? pair_tiles : max_clusters);
        if (getenv("TL_LOG"))
            fprintf(stderr, "[tilelens] pair kernel: %lld tiles (%lld of 512 tokens), %d clusters (max active %d), %d stages, %zu B smem\n",
                    (long long)pair_tiles, (long long)big_tiles, clusters, max_clusters, p.num_stages, smem);
        if (halves == 2) {
            if (es == 1) gemm_pair_kernel<true, 2><<<2 * clusters, kGenericThreads, smem, stream>>>(p);
            else gemm_pair_kernel<false, 2><<<2 * clusters, kGenericThreads, smem, stream>>>(p);
        } else {
            if (es == 1) gemm_pair_kernel<true, 1><<<2 * clusters, kGemmThreads, smem, stream>>>(p);
            else gemm_pair_kernel<false, 1><<<2 * clusters, kGemmThreads, smem, stream>>>(p);
        }
        return check_cuda(cudaGetLastError());
    }
    // The GEMM kernel may be scheduled while its predecessor in the stream is finishing (it waits before touching
    // memory).  TL_NO_PDL=1 restores plain stream order for measurement.
    const bool pdl_gemm = pdl_ok;
#define TL_LAUNCH_GEMM_T(BK_, BN_, WN_, F8_)                                                                        \
    {                                                                                                              \
        static bool attr_set = false;                                                                              \
        if (!attr_set) {                                                                                           \
            err = cudaFuncSetAttribute(gemm_kernel<BK_, BN_, WN_, F8_>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                       kMaxDynamicSmem);                                                           \
            attr_set = err == cudaSuccess;                                                                         \
        }                                                                                                          \
        if (err == cudaSuccess) {                                                                                  \
            cudaLaunchConfig_t cfg = {};                                                                           \
            cfg.gridDim = dim3(plan.grid);                                                                         \
            cfg.blockDim = dim3(generic ? kGenericThreads : kGemmThreads);                                         \
            cfg.dynamicSmemBytes = plan.smem_bytes;                                                                \
            cfg.stream = stream;                                                                                   \
            cudaLaunchAttribute attr[1];                                                                           \
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;                                       \
            attr[0].val.programmaticStreamSerializationAllowed = 1;                                                \
            cfg.attrs = attr;                                                                                      \
            cfg.numAttrs = pdl_gemm ? 1 : 0;                                                                       \
            err = cudaLaunchKernelEx(&cfg, gemm_kernel<BK_, BN_, WN_, F8_>, p);                                    \
        }                                                                                                          \
    }
#define TL_LAUNCH_GEMM(BK_, BN_, WN_)                                                                              \
    { if (es == 1) TL_LAUNCH_GEMM_T(BK_, BN_, WN_, true) else TL_LAUNCH_GEMM_T(BK_, BN_, WN_, false) }
#define TL_LAUNCH_GEMM_BN(BK_, WN_)                                                                                \
    if (plan.BN == 64) TL_LAUNCH_GEMM(BK_, 64, WN_) else if (plan.BN == 128) TL_LAUNCH_GEMM(BK_, 128, WN_)        \
    else TL_LAUNCH_GEMM(BK_, 256, WN_)
    if (plan.weights_on_n) {
        if (plan.BK == 64) { TL_LAUNCH_GEMM_BN(64, true) } else { TL_LAUNCH_GEMM_BN(128, true) }
    } else {
        if (plan.BK == 64) { TL_LAUNCH_GEMM_BN(64, false) } else { TL_LAUNCH_GEMM_BN(128, false) }
    }
#undef TL_LAUNCH_GEMM_BN
    // stream-K: add up the partial tiles, one CTA per boundary between two CTA ranges
    if (err == cudaSuccess && plan.stream_k && plan.grid > 1) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(plan.grid - 1);
        cfg.blockDim = dim3(128);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // overlap its launch with the GEMM grid
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        err = cudaLaunchKernelEx(&cfg, streamk_reduce_kernel, p, plan.grid);
    }
#undef TL_LAUNCH_GEMM
#undef TL_LAUNCH_GEMM_T
    if (err != cudaSuccess) return check_cuda(err);
    return check_cuda(cudaGetLastError());
}

}  // namespace tl

extern "C" {

int tl_gemm(const void* d_A, const void* d_B, float* d_C, int64_t M, int64_t N, int64_t K, int64_t G, int block_rows,
            int block_cols, int cta_m, int cta_n, int cta_k, void* cuda_stream) {
    return tl::gemm_launch(d_A, d_B, d_C, nullptr, 1, M, M, N, K, G, block_rows, block_cols, cta_m, cta_n, cta_k,
                           static_cast<cudaStream_t>(cuda_stream));
}

int tl_gemm_grouped(const void* d_A_sorted, const void* d_B_experts, float* d_C, const int32_t* d_offsets, int E,
                    int64_t total_rows, int64_t N, int64_t K, int64_t G, int block_rows, int block_cols, int cta_m,
                    int cta_n, int cta_k, void* cuda_stream) {
    if (!d_offsets && total_rows > 0) return TL_ERR_INVALID_ARG;
    // Without a host copy of the offsets the largest expert is unknown: size tiles for the total.
    return tl::gemm_launch(d_A_sorted, d_B_experts, d_C, d_offsets, E, total_rows, total_rows, N, K, G, block_rows,
                           block_cols, cta_m, cta_n, cta_k, static_cast<cudaStream_t>(cuda_stream));
}

int tl_gemm_kmajor(const void* d_A, const void* d_B_nk, float* d_C, int64_t M, int64_t N, int64_t K, int64_t G, int tile_n,
                   int tile_k, int cta_m, int cta_n, int cta_k, void* cuda_stream) {
    return tl::gemm_launch(d_A, d_B_nk, d_C, nullptr, 1, M, M, N, K, G, tile_n, tile_k, cta_m, cta_n, cta_k,
                           static_cast<cudaStream_t>(cuda_stream), nullptr, true);
}

int tl_gemm_grouped_kmajor(const void* d_A_sorted, const void* d_B_experts_nk, float* d_C, const int32_t* d_offsets, int E,
                           int64_t total_rows, int64_t N, int64_t K, int64_t G, int tile_n, int tile_k, int cta_m,
                           int cta_n, int cta_k, void* cuda_stream) {
    if (!d_offsets && total_rows > 0) return TL_ERR_INVALID_ARG;
    return tl::gemm_launch(d_A_sorted, d_B_experts_nk, d_C, d_offsets, E, total_rows, total_rows, N, K, G, tile_n, tile_k,
                           cta_m, cta_n, cta_k, static_cast<cudaStream_t>(cuda_stream), nullptr, true);
}

int tl_gemm_fp8_kmajor(const void* d_A, const void* d_B_nk, float* d_C, int64_t M, int64_t N, int64_t K, int64_t G,
                       int tile_n, int tile_k, int cta_m, int cta_n, int cta_k, void* cuda_stream) {
    if (cta_k != 0 && cta_k != 128 && cta_k != 256) return TL_ERR_UNSUPPORTED;
    return tl::gemm_launch(d_A, d_B_nk, d_C, nullptr, 1, M, M, N, K, G, tile_n, tile_k, cta_m, cta_n, cta_k / 2,
                           static_cast<cudaStream_t>(cuda_stream), nullptr, true, 1);
}

int tl_gemm_grouped_fp8_kmajor(const void* d_A_sorted, const void* d_B_experts_nk, float* d_C, const int32_t* d_offsets,
                               int E, int64_t total_rows, int64_t N, int64_t K, int64_t G, int tile_n, int tile_k,
                               int cta_m, int cta_n, int cta_k, void* cuda_stream) {
    if (!d_offsets && total_rows > 0) return TL_ERR_INVALID_ARG;
    if (cta_k != 0 && cta_k != 128 && cta_k != 256) return TL_ERR_UNSUPPORTED;
    return tl::gemm_launch(d_A_sorted, d_B_experts_nk, d_C, d_offsets, E, total_rows, total_rows, N, K, G, tile_n, tile_k,
                           cta_m, cta_n, cta_k / 2, static_cast<cudaStream_t>(cuda_stream), nullptr, true, 1);
}

int tl_gemm_bf16(const void* d_A, const void* d_B, void* d_C_bf16, int64_t M, int64_t N, int64_t K, int64_t G,
                 int block_rows, int block_cols, int cta_m, int cta_n, int cta_k, void* cuda_stream) {
    if (!d_C_bf16) return TL_ERR_INVALID_ARG;
    return tl::gemm_launch(d_A, d_B, nullptr, nullptr, 1, M, M, N, K, G, block_rows, block_cols, cta_m, cta_n, cta_k,
                           static_cast<cudaStream_t>(cuda_stream), nullptr, false, 2, nullptr, d_C_bf16);
}

int tl_gemm_grouped_bf16(const void* d_A_sorted, const void* d_B_experts, void* d_C_bf16, const int32_t* d_offsets, int E,
                         int64_t total_rows, int64_t N, int64_t K, int64_t G, int block_rows, int block_cols, int cta_m,
                         int cta_n, int cta_k, void* cuda_stream) {
    if (!d_offsets && total_rows > 0) return TL_ERR_INVALID_ARG;
    if (!d_C_bf16) return TL_ERR_INVALID_ARG;
    return tl::gemm_launch(d_A_sorted, d_B_experts, nullptr, d_offsets, E, total_rows, total_rows, N, K, G, block_rows,
                           block_cols, cta_m, cta_n, cta_k, static_cast<cudaStream_t>(cuda_stream), nullptr, false, 2,
                           nullptr, d_C_bf16);
}

int tl_gemm_grouped_swiglu(const void* d_A_sorted, const void* d_B_experts_gate_up, void* d_H_bf16, const int32_t* d_offsets,
                           int E, int64_t total_rows, int64_t N, int64_t K, int64_t G, int block_rows, int block_cols,
                           int cta_m, int cta_n, int cta_k, void* cuda_stream) {
    if (!d_offsets && total_rows > 0) return TL_ERR_INVALID_ARG;
    if (!d_H_bf16) return TL_ERR_INVALID_ARG;
    return tl::gemm_launch(d_A_sorted, d_B_experts_gate_up, nullptr, d_offsets, E, total_rows, total_rows, N, K, G,
                           block_rows, block_cols, cta_m, cta_n, cta_k, static_cast<cudaStream_t>(cuda_stream), nullptr,
                           false, 2, d_H_bf16);
}

int tl_moe_ffn(const void* d_X_sorted, const void* d_W_gate_up, const void* d_W_down, void* d_H_bf16, float* d_Y,
               const int32_t* d_offsets, int E, int64_t total_rows, int64_t hidden, int64_t inter, int64_t G,
               int block_rows, int block_cols, void* cuda_stream) {
    if (hidden <= 0 || inter <= 0) return TL_ERR_INVALID_ARG;
    if (int rc = tl_gemm_grouped_swiglu(d_X_sorted, d_W_gate_up, d_H_bf16, d_offsets, E, total_rows, 2 * inter, hidden, G,
                                        block_rows, block_cols, 0, 0, 0, cuda_stream))
        return rc;
    return tl_gemm_grouped(d_H_bf16, d_W_down, d_Y, d_offsets, E, total_rows, hidden, inter, G, block_rows, block_cols, 0,
                           0, 0, cuda_stream);
}

size_t tl_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K, int cta_m, int cta_n, int cta_k) {
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    size_t need = 0;
    for (int grouped = 0; grouped < 2; ++grouped) {         // the larger of the dense and the grouped schedule
        int bm = cta_m, bn = cta_n, bk = cta_k;
        if (cta_m == 0 && cta_n == 0 && cta_k == 0) tl::default_tile(M, grouped != 0, false, &bm, &bn, &bk);
        if (bm <= 0 || bn <= 0) return 0;
        tl::GemmPlan plan;
        const int64_t mt = grouped ? M / bm + 1 : tl::ceil_div(M, bm);
        if (tl::make_plan(M, mt * tl::ceil_div(N, bn), N, K, cta_m, cta_n, cta_k, grouped != 0, &plan)) return 0;
        if (plan.ws_bytes > need) need = plan.ws_bytes;
    }
    return need;
}

}  // extern "C"

// ------------------------------------------------------------ host-buffer form
namespace tl {
static size_t align256(size_t x) { return (x + 255) & ~size_t(255); }
}

extern "C" {

size_t tl_gemm_host_scratch_bytes(int64_t M, int64_t N, int64_t K) {
    if (M < 0 || N <= 0 || K <= 0) return 0;
    return tl::align256(size_t(M) * K * 2) + 2 * tl::align256(size_t(K) * N * 2) + tl::align256(size_t(M) * N * 4);
}

int tl_gemm_host(const void* h_A, const void* h_B_rowmajor, float* h_C, int64_t M, int64_t N, int64_t K, int64_t G,
                 int block_rows, int block_cols, int cta_m, int cta_n, int cta_k, void* d_scratch,
                 size_t scratch_bytes, void* cuda_stream) {
    if (M < 0 || N <= 0 || K <= 0) return TL_ERR_INVALID_ARG;
    if (M == 0) return TL_OK;
    if (!h_A || !h_B_rowmajor || !h_C || !d_scratch) return TL_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(d_scratch) % 256 != 0) return TL_ERR_ALIGNMENT;
    if (scratch_bytes < tl_gemm_host_scratch_bytes(M, N, K)) return TL_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* base = static_cast<uint8_t*>(d_scratch);
    const size_t a_bytes = size_t(M) * K * 2, b_bytes = size_t(K) * N * 2, c_bytes = size_t(M) * N * 4;
    uint8_t* dA = base;
    uint8_t* dB_row = dA + tl::align256(a_bytes);
    uint8_t* dB_tile = dB_row + tl::align256(b_bytes);
    float* dC = reinterpret_cast<float*>(dB_tile + tl::align256(b_bytes));
    if (int rc = tl::check_cuda(cudaMemcpyAsync(dA, h_A, a_bytes, cudaMemcpyHostToDevice, stream))) return rc;
    if (int rc = tl::check_cuda(cudaMemcpyAsync(dB_row, h_B_rowmajor, b_bytes, cudaMemcpyHostToDevice, stream)))
        return rc;
    const void* dB = dB_row;
    if (block_rows != 0) {
        if (int rc = tl_relayout_on(dB_row, dB_tile, K, N, 2, G, block_rows, block_cols, TL_TO_TILE_MAJOR, stream))
            return rc;
        dB = dB_tile;
    }
    if (int rc = tl_gemm(dA, dB, dC, M, N, K, G, block_rows, block_cols, cta_m, cta_n, cta_k, stream)) return rc;
    if (int rc = tl::check_cuda(cudaMemcpyAsync(h_C, dC, c_bytes, cudaMemcpyDeviceToHost, stream))) return rc;
    return tl::check_cuda(cudaStreamSynchronize(stream));
}

}  // extern "C"

// ------------------------------------------------- scratch held in the library image
namespace tl {

// Split-K scratch of tl_gemm_noalloc: partial tiles, and in the last 256 bytes a spare word for the time-out flag when the caller passes none.  Lives in the
// module's data segment on every GPU that loads the library, from load until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[TL_NOALLOC_SCRATCH_BYTES];

// g_noalloc_scratch is a host-side handle here, not an address a kernel could use: the device address
// is looked up once per device, with that device current, and remembered.
static int noalloc_scratch_address(unsigned char** out) {
    static unsigned char* per_device[64] = {};
    int dev = -1;
    if (int rc = check_cuda(cudaGetDevice(&dev))) return rc;
    if (dev < 0 || dev >= 64) return TL_ERR_UNSUPPORTED;
    if (!per_device[dev]) {
        void* ptr = nullptr;
        if (int rc = check_cuda(cudaGetSymbolAddress(&ptr, g_noalloc_scratch))) return rc;
        if (!ptr) return TL_ERR_CUDA;
        per_device[dev] = static_cast<unsigned char*>(ptr);
    }
    *out = per_device[dev];
    return TL_OK;
}

}  // namespace tl

extern "C" int tl_gemm_noalloc(const void* d_A, const void* d_B, float* d_C, int64_t M, int64_t N, int64_t K,
                               int64_t G, int block_rows, int block_cols, int cta_m, int cta_n, int cta_k,
                               uint32_t* d_timeout_flag, void* cuda_stream) {
    if (M < 0 || N <= 0 || K <= 0) return TL_ERR_INVALID_ARG;
    if (M == 0) return TL_OK;
    unsigned char* base = nullptr;
    if (int rc = tl::noalloc_scratch_address(&base)) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    tl::FixedScratch fixed;
    fixed.ws = base;
    fixed.ws_bytes = TL_NOALLOC_SCRATCH_BYTES - 256;
    fixed.status = d_timeout_flag ? d_timeout_flag
                                  : reinterpret_cast<uint32_t*>(base + TL_NOALLOC_SCRATCH_BYTES - 256);
    return tl::gemm_launch(d_A, d_B, d_C, nullptr, 1, M, M, N, K, G, block_rows, block_cols, cta_m, cta_n, cta_k,
                           stream, &fixed);
}

#ifdef TL_TIMELINE
// Measurement builds only: d_buf holds 8 uint64 per CTA (zeroed by the caller); nullptr switches it off.
extern "C" int tl_debug_set_timeline(void* d_buf) {
    return tl::check_cuda(cudaMemcpyToSymbol(tl::g_timeline, &d_buf, sizeof d_buf));
}
extern "C" int tl_debug_set_counters(void* d_buf) {
    return tl::check_cuda(cudaMemcpyToSymbol(tl::g_counters, &d_buf, sizeof d_buf));
}
extern "C" int tl_debug_set_reverse(int on) {
    return tl::check_cuda(cudaMemcpyToSymbol(tl::g_reverse, &on, sizeof on));
}
#endif
