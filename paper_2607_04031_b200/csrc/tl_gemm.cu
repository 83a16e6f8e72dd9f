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
// Memory tiles whose rows are shorter than 32 bytes cannot be boxed as swizzle rows (the generic-address case of
// Section 4.4).  With at least 8 rows they are still fetched by the copy engine as stored, the buffer seen as plain
// bytes: tiles with 16-byte rows are core matrices of the no-swizzle MN-major operand and single-column tiles panels of
// a K-major operand, both read by the MMA as they are; tiles with 8- or 4-byte rows are transposed in place, 2 or 4
// neighbouring tiles into one with 16-byte rows, by four more warps.  Tiles of fewer rows: one more warp streams them
// into shared memory with untiled bulk copies and four more permute them into the operand image with Eq. 1-2 arithmetic.
//
// One persistent CTA per SM:
//   warp 0      TMA producer   (one lane)   ring of shared-memory stages, mbarrier expect-tx
//   warp 1      MMA issuer     (one lane)   tcgen05.mma into one of two TMEM accumulators
//   warps 2..5  epilogue                    tcgen05.ld -> fp32 -> C, or silu(gate) * up -> bf16 (expert FFN)
//   warps 6..10 in-place transpose (6..9) or generic-address weights   (only when a tile row is shorter than 16 bytes)
// Work is a list of (output tile, K range); make_plan chooses among
//   whole tiles round-robin (the tiles fill the SMs, or divide evenly over at least 3/4 of them);
//   split-K inside clusters: one tile per cluster of up to 8 CTAs, each a share of the K loop, partial tiles added
//       through distributed shared memory (decode-sized dense products; no workspace);
//   whole rounds of tiles round-robin, then the flattened (tile, K iteration) space of the rest cut into one
//       contiguous range per CTA ("stream-K"); partial tiles go to a workspace and a second small kernel
//       (streamk_reduce_kernel, launched with programmatic stream serialisation so that it is resident before this
//       one ends) adds them in K order and writes C.
// Nothing ever spins on another CTA of another cluster; every mbarrier wait is bounded (see mbar_wait_bounded).
// Large dense problems run on CTA pairs instead (tl_gemm_pair.cuh); the expert FFN can run its two products in one
// cooperative launch (tl_gemm_chain.cu).  This file: the stream-K reduction kernel, the plan, the tensor maps, the
// launches and the C entry points; the device code of the GEMM is in tl_gemm_kernel.cuh.
#include "tl_gemm_kernel.cuh"

#include <cstdio>
#include <cstdlib>
#include <cstring>

namespace tl {

__global__ void __launch_bounds__(128) streamk_reduce_kernel(const __grid_constant__ GemmParams p, int gemm_grid) {
    __shared__ int prefix[kMaxExperts + 1];
    __shared__ int row_start[kMaxExperts + 1];
    __shared__ int slot_of[kRangeTabMax];
    streamk_reduce_body<true>(p, gemm_grid, int(blockIdx.x), prefix, row_start, slot_of);
}

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
        tls().last_cuda_error = int(cudaErrorSymbolNotFound);
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
        tls().last_cuda_error = int(r);
        return TL_ERR_CUDA;
    }
    const int slot = cache_n < kMapCacheSize ? cache_n++ : (cache_next++ % kMapCacheSize);
    cache[slot].key = key;
    cache[slot].map = *out;
    return TL_OK;
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
    int cluster_k;        // > 1: clusters of that many CTAs split the K loop of one tile each (no scratch)
    int grid;
    int num_stages;
    int raw_slots;        // generic-address path: raw stage images kept in flight behind the pipeline stages
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
//   up to 64 rows      rows x 256 x 64: tokens on the MMA's M side, 256 weight columns (8 KB of weights) per
//                      instruction; few enough tiles that a no-scratch schedule exists for the usual shapes (see
//                      make_plan)
//   up to 128 rows     128 x 128 x 128: same orientation, deeper K step so that there are half as many barrier
//                      hand-offs
//   more rows          256 x 128 x 64 with the weights on the M side (prefill) when there are enough tiles for the
//                      CTA-pair kernel, else 128 x 128 x 128
//   65 to 512 rows     dense products on TMA-readable weights may take 128 x 256 x 64 instead (gemm_launch ranks the two)
//   grouped            at most 32 rows per tile (x 256 x 64): most experts have a handful of rows; caps of 64 and 128
//                      rows measured the same within 2 % on the Qwen-3 expert products (fewer passes over an
//                      expert's weights against fewer, larger pipeline stages)
//   narrow_scratch     (fixed-size scratch) never the 256-column tile
static void default_tile(int64_t rows_max, bool grouped, bool narrow_scratch, int* BM, int* BN, int* BK,
                         bool pair_sized = true) {
    *BM = pick_bm(rows_max);
    // More than 128 rows but too few tiles for the CTA-pair kernel (pair_sized == false): 128-row tiles with the
    // weights on the N side (Qwen-3 attention projections at M = 256: 14-16 us against 23-25 us with 256-row tiles).
    if (!grouped && *BM > 128 && !pair_sized) *BM = 128;
    const int group_cap = opt(TL_OPT_MOE_ROW_CAP) > 0 ? int(opt(TL_OPT_MOE_ROW_CAP)) : 32;
    if (grouped && *BM > group_cap) *BM = group_cap;
    if (*BM <= 64 && !narrow_scratch) { *BN = 256; *BK = 64; }
    else if (*BM <= 128) { *BN = 128; *BK = 128; }
    else { *BN = 128; *BK = 64; }
}

static int make_plan(int64_t rows_max, int64_t tile_bound, int64_t N, int64_t K, int cta_m, int cta_n, int cta_k,
                     bool grouped, GemmPlan* plan, bool narrow_scratch = false, bool generic = false, bool pair_sized = true,
                     int64_t rows_total = 0) {
    if (int rc = ensure_device_info()) return rc;
    int sms = dev().sm_count;
    if (opt(TL_OPT_SM_LIMIT) > 0 && opt(TL_OPT_SM_LIMIT) < sms) sms = int(opt(TL_OPT_SM_LIMIT));
    int BM = cta_m, BN = cta_n, BK = cta_k;
    if (BM == 0 && BN == 0 && BK == 0) default_tile(rows_max, grouped, narrow_scratch, &BM, &BN, &BK, pair_sized);
    if (BM != 16 && BM != 32 && BM != 64 && BM != 128 && BM != 256) return TL_ERR_UNSUPPORTED;
    if (BN != 64 && BN != 128 && BN != 256) return TL_ERR_UNSUPPORTED;
    if (BK != 64 && BK != 128) return TL_ERR_UNSUPPORTED;
    // 256 x 256 x 64: the weights-on-N kernel with two 128-row token blocks per tile, one weight slab per stage serving
    // both through the two accumulators (dense problems, whole-tile schedules only: see the end of this function)
    const bool two_blocks = BM == 256 && BN == 256 && BK == 64 && !grouped && !generic && !narrow_scratch;
    if (BN == 256 && BM > 128 && !two_blocks) return TL_ERR_UNSUPPORTED;   // 2 accumulators x 2 groups x BM columns <= 512
    plan->BM = BM; plan->BN = BN; plan->BK = BK;
    plan->weights_on_n = BM <= 128 || two_blocks;           // tokens fit the 128 rows of the MMA's M side
    // With the tokens on the M side the MMA reads 64 rows (tiles of up to 64 tokens) or 128: a stage holds that
    // many token rows per 64-wide K slice, the ones beyond BM zeroed once by the kernel.  They only feed
    // accumulator rows that are never stored.
    const bool m128_only = opt(TL_OPT_UMMA_M128) != 0;          // measurement switch
    // (umma_m == 64: per tile, 64-row instructions for tiles of up to 64 tokens and 128-row ones above)
    plan->umma_m = BM <= 128 && !m128_only ? 64 : 128;
    // (the stage must hold every token row the widest instruction of the launch reads)
    const int mma_rows_min = m128_only ? 128 : 64;
    plan->a_rows = plan->weights_on_n && BM < mma_rows_min ? mma_rows_min : BM;
    const size_t stage = size_t(BK) * BN * 2 + size_t(BK / 64) * plan->a_rows * kAtomBytes;
    // 1 KB of slack to align the stages to 1024 bytes.
    // 12 KB stay free so that a CTA of the stream-K reduction kernel can be resident next to this one.
    const size_t budget = kMaxDynamicSmem - 1024 - 12 * 1024;
    int stages = int(budget / stage);
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) return TL_ERR_UNSUPPORTED;
    plan->raw_slots = 0;
    const size_t raw_bytes = size_t(BK) * BN * 2;
    size_t table_bytes = 0;
    if (generic) {
        // Two or three operand stages; the rest of shared memory holds raw stage images (the bytes in flight).
        // (a table of one 16-bit entry per 16-byte chunk of a stage follows the ring)
        stages = stage >= 40 * 1024 ? 2 : 3;
        table_bytes = raw_bytes / 8;
        if (size_t(stages) * stage + 2 * raw_bytes + table_bytes > budget) return TL_ERR_UNSUPPORTED;
        int raw = int((budget - size_t(stages) * stage - table_bytes) / raw_bytes);
        plan->raw_slots = raw > kMaxStages ? kMaxStages : raw;
    }
    {
        const int cap = int(opt(TL_OPT_MAX_STAGES));            // measurement switch
        if (cap >= 2 && cap < stages) stages = cap;
        if (cap >= 2 && cap < plan->raw_slots) plan->raw_slots = cap;
    }
    plan->num_stages = stages;
    plan->smem_bytes = size_t(stages) * stage + size_t(plan->raw_slots) * raw_bytes + table_bytes + 1024;
    if (plan->smem_bytes < 120 * 1024) plan->smem_bytes = 120 * 1024;   // one CTA per SM: TMEM is not shared
    const int64_t k_iters = ceil_div(K, BK);
    const int64_t total_iters = tile_bound * k_iters;
    // Whole tiles when they fill the machine evenly enough, contiguous K ranges otherwise.
    const int64_t waves = ceil_div(tile_bound, sms);
    const bool even = tile_bound >= sms && double(tile_bound) / double(waves * sms) >= 0.92;
    plan->stream_k = (grouped || !even) ? 1 : 0;
    // With short tiles and enough of them the kernel cuts nothing (Sched::no_cut); where the host can tell (dense: the
    // tile count; grouped: at least ceil(rows / BM) m-tiles whatever the routing) it plans whole tiles outright: no
    // workspace, no reduction kernel.
    {
        const int64_t tiles_min = grouped ? ceil_div(rows_total, BM) * ceil_div(N, BN) : tile_bound;
        if (plan->stream_k && tiles_min * 4 >= 3 * int64_t(sms) && k_iters <= kNoCutStages) plan->stream_k = 0;
    }
    plan->cluster_k = 1;
    int64_t grid = plan->stream_k ? (total_iters < sms ? total_iters : sms) : (tile_bound < sms ? tile_bound : sms);
    // Dense decode-sized products: a schedule without partial tiles in global memory beats the stream-K cut even
    // when it leaves some SMs idle, because 110 to 130 CTAs already stream at the rate of the whole device
    // (measured: Llama gate_up, M = 8, 224 whole tiles on 112 CTAs 135 us, cut over 148 CTAs 142 us).  In order:
    //   1. whole tiles on the largest grid of at least 3/4 of the SMs that divides the tile count;
    //   2. one tile per cluster of S <= 8 CTAs which split its K loop S ways and add their partial tiles through
    //      distributed shared memory, for the S that fills most SMs (at least 3/4 of them; small problems: any number);
    //   3. the stream-K cut with its workspace and reduction kernel.
    if (plan->stream_k && !grouped && plan->weights_on_n && !generic && opt(TL_OPT_NO_SCRATCH_PLANS) != 0) {
        const int64_t lo = (3 * int64_t(sms) + 3) / 4;
        int64_t g1 = 0;
        for (int64_t g = tile_bound < sms ? tile_bound : sms; g >= lo; --g)
            if (tile_bound % g == 0) { g1 = g; break; }
        // (large partial tiles: at most 4 CTAs per cluster, the exchange through distributed shared memory measured
        // slower than the stream-K cut beyond that)
        const int s_max = size_t(BM) * (BN + 4) * 4 > 40 * 1024 ? 4 : 8;
        // every cluster of the launch must be resident at once (clusters live inside one GPC: 148 SMs hold 45 clusters of
        // 3 CTAs but only 15 of 8); a second wave of clusters costs more than any other schedule
        auto fits = [&](int s) -> bool {
            int& cap = dev().cluster_cap[s];
            if (cap == 0) {
                int n = 0;
                cap = gemm_max_active_clusters(s, &n) == TL_OK && n > 0 ? n : -1;
            }
            const int64_t limit = opt(TL_OPT_SM_LIMIT) > 0 && cap > 0 ? (int64_t(cap) * sms) / dev().sm_count : cap;
            return cap > 0 && tile_bound <= limit;
        };
        int best_s = 0;
        for (int s = 2; s <= s_max; ++s)
            if (tile_bound * s <= sms && tile_bound * s >= lo && k_iters >= s && size_t(BM) * (BN + 4) * 4 <= plan->smem_bytes - 1024 &&
                tile_bound * s > int64_t(best_s) * tile_bound && fits(s))
                best_s = s;
        // Clusters that fill fewer SMs still beat the cut while the weights are few enough: c CTAs stream at about
        // min(c x 65 GB/s, the device's 7.2 TB/s), the cut at the device's rate plus about 6 us for its partial tiles,
        // its second kernel and the wake-up (29 to 92 MB of weights on 56 to 104 CTAs: 6 to 27 % faster than the cut).
        if (g1 == 0 && best_s == 0) {
            const int64_t bytes = total_iters * BK * BN * 2;
            for (int s = s_max; s >= 2; --s) {
                const int64_t c = tile_bound * s;
                if (c > sms || k_iters < 2 * s || size_t(BM) * (BN + 4) * 4 > plan->smem_bytes - 1024 || !fits(s)) continue;
                const int64_t rate = c * 65 < 7200 ? c * 65 : 7200;                 // GB/s = bytes per ns
                if (bytes / rate <= bytes / 7200 + 6000) best_s = s;
                break;                                                              // (the largest cluster that fits, or none)
            }
        }
        // Small problems (a few MB of weights: latency, not bandwidth) that fill neither: clusters all the same, however
        // few, as long as every CTA keeps at least two K iterations.  The cut would give each of many CTAs a single
        // iteration, a partial tile in global memory each, and a second kernel to add them.
        // (Qwen-3 attention projections, 128 to 512 tokens: k / v 13.7-16.9 -> 11.4-11.6 us, o at 128 tokens 17.9 -> 14.4 us)
        if (g1 == 0 && best_s == 0 && total_iters * BK * BN * 2 <= (int64_t(16) << 20))
            for (int s = s_max; s >= 2; --s)
                if (tile_bound * s <= sms && k_iters >= 2 * s && size_t(BM) * (BN + 4) * 4 <= plan->smem_bytes - 1024 && fits(s)) {
                    best_s = s;
                    break;
                }
        if (g1 > 0) {
            plan->stream_k = 0;
            grid = g1;
        } else if (best_s > 0) {
            plan->stream_k = 0;
            plan->cluster_k = best_s;
            grid = tile_bound * best_s;
        }
    }
    if (grid < 1) grid = 1;
    plan->grid = int(grid);
    // (a tile of two token blocks owns both accumulators and is never cut: its partial tile would be 256 KB)
    if (two_blocks && (plan->stream_k || plan->cluster_k > 1)) return TL_ERR_UNSUPPORTED;
    plan->ws_bytes = plan->stream_k ? size_t(2) * size_t(grid) * BM * BN * sizeof(float) : 0;   // two slots per CTA
    return TL_OK;
}

static int launch_reduce(const GemmParams& p, int gemm_grid, cudaStream_t stream, bool pdl) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(gemm_grid - 1);
    cfg.blockDim = dim3(128);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // overlap its launch with the GEMM grid
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return check_cuda(cudaLaunchKernelEx(&cfg, streamk_reduce_kernel, p, gemm_grid));
}

// What the calling thread's last GEMM launch ran (tl_gemm_last_plan).
static tl_gemm_plan_info& last_plan() {
    static thread_local tl_gemm_plan_info info = {};
    return info;
}

// Where a launch takes its scratch from when the caller of gemm_launch supplies it itself.
struct FixedScratch {
    void* ws;            // partial tiles
    size_t ws_bytes;
    uint32_t* status;    // word the kernel raises when a bounded wait expires
};

// The CTA-pair kernel's schedule on `clusters` co-resident clusters, in units of one 256-token tile run by the
// 256-token instantiation.  It mixes whole waves of 512-token tiles with 256-token tiles for the rest (*big_tiles on
// entry: how many 512-token tiles that mix has); with few waves the mix can lose to 256-token tiles alone: a 512-token
// tile that M leaves half empty, and every 256-token tile run by the 512-token instantiation (shorter pipeline,
// accumulators not alternating), costs about 1.5 units, a full 512-token tile 1.8.  The busiest cluster of both
// schedules is worked out from the kernel's own tile order; *big_tiles is set to 0 where 256-token tiles alone are
// ahead by a tenth (Llama qkv at 640 rows: 74 + 12 tiles 172 us, 120 small ones 119 us; gate_up at 1024 rows keeps
// 444 + 8).  Returns the units of the schedule chosen.
static double pair_schedule_units(int64_t rows_total, int64_t N, int clusters, int64_t* big_tiles) {
    const int64_t n_t = ceil_div(N, 256), m_big = ceil_div(rows_total, 512), big_total = m_big * n_t;
    const int C = clusters < 1 ? 1 : (clusters < 256 ? clusters : 256);
    const double small_only = double(ceil_div(ceil_div(rows_total, 256) * n_t, int64_t(C)));
    if (*big_tiles <= 0) return small_only;
    const int64_t all = *big_tiles + 2 * (big_total - *big_tiles);
    double load[256] = {0.0};
    auto m_tile_of = [&](int64_t tile) {                            // pair_tile_coords of the kernel, m part
        const int64_t band_tiles = 8 * n_t, band = tile / band_tiles, r = tile - band * band_tiles;
        const int64_t band_rows = m_big - band * 8 < 8 ? m_big - band * 8 : 8;
        return band * 8 + r % band_rows;
    };
    for (int64_t t = 0; t < all; ++t) {
        double cost;
        if (t < *big_tiles) {
            cost = rows_total - m_tile_of(t) * 512 > 256 ? 1.8 : 1.5;
        } else {
            const int64_t sidx = t - *big_tiles, row0 = m_tile_of(*big_tiles + (sidx >> 1)) * 512 + (sidx & 1) * 256;
            cost = row0 < rows_total ? 1.5 : 0.0;
        }
        load[t % C] += cost;
    }
    double mixed = 0.0;
    for (int c = 0; c < C; ++c) mixed = load[c] > mixed ? load[c] : mixed;
    if (small_only < 0.9 * mixed) {
        *big_tiles = 0;
        return small_only;
    }
    return mixed;
}

// Rough time of a dense weights-on-N plan, for choosing between the 128- and the 256-column tile at 65 to 512 token
// rows (K in 2-byte units).  What one CTA pulls into shared memory at about 90 GB/s (measured 75-105: weight slabs and
// the token rows that come with each, most of them L2 hits), not faster than HBM delivers the weights once; plus the
// exchange of partial tiles inside a cluster (about 6 us for 128 KB tiles, 3 us for 64 KB), 12 us for the partial
// tiles and the second kernel of a stream-K cut, and a fixed 8 us.  Fitted to Llama-70B and Qwen-3 shapes at 96-512
// rows; it only has to rank two plans.
static double mid_tile_estimate_us(const GemmPlan& pl, int64_t rows, int64_t N, int64_t K) {
    const double tiles = double(ceil_div(rows, pl.BM)) * double(ceil_div(N, pl.BN));
    const double k_iters = double(ceil_div(K, pl.BK));
    const double stage = double(pl.BK) * pl.BN * 2 + double(pl.BK) * pl.a_rows * 2;
    double iters;                                           // K iterations of the busiest CTA
    if (pl.stream_k) iters = tiles * k_iters / pl.grid;
    else if (pl.cluster_k > 1) iters = double(ceil_div(int64_t(k_iters), pl.cluster_k));
    else iters = double(ceil_div(int64_t(tiles), pl.grid)) * k_iters;
    double us = iters * stage / 90e3;                       // 90 GB/s = 90e3 bytes per us
    const double hbm = double(N) * double(K) * 2 / 5.8e6;   // 5.8 TB/s with token rows in the way
    if (hbm > us) us = hbm;
    if (pl.cluster_k > 1) us += double(pl.BM) * pl.BN * 4 / 65536 * 3.0;
    if (pl.stream_k) us += 12.0;
    return us + 8.0;
}

// Token rows per tile of a grouped product whose caller left the tile to the library (0: the default of 32).  The
// 32-row tile suits routings that leave most experts a handful of rows (Qwen-3 at 256 tokens: 16 rows per expert on
// average).  With more rows per expert every further m-tile of an expert pulls the expert's weights out of L2 again,
// so the tile grows with the average: 64 rows from 25 rows per expert on, 128 from 49 on, both 256 columns wide
// (Qwen-3 gate_up / down at 1024 tokens: 194 / 129 -> 151 / 90 us; at 4096 tokens 575 / 397 -> 293 / 186 us) -- but
// only while the larger tiles still number at least one per SM: few large tiles would have to be cut along K.
// TL_OPT_MOE_ROW_CAP fixes the row count instead.
static int grouped_tile_rows(int64_t rows_total, int E, int64_t N) {
    if (opt(TL_OPT_MOE_ROW_CAP) != 0 || E < 1) return 0;
    if (ensure_device_info()) return 0;
    const int64_t avg = rows_total / E, n_tiles = ceil_div(N, 256), sms = dev().sm_count;
    if (avg > 48 && rows_total / 128 * n_tiles >= sms) return 128;
    if (avg > 24 && rows_total / 64 * n_tiles >= sms) return 64;
    return 0;
}

static int gemm_launch(const void* d_A, const void* d_B, float* d_C, const int32_t* d_offsets, int E,
                       int64_t rows_total, int64_t rows_max, int64_t N, int64_t K, int64_t G, int br, int bc,
                       int cta_m, int cta_n, int cta_k, cudaStream_t stream, const FixedScratch* fixed = nullptr,
                       bool kmajor = false, int elem_bytes = 2, void* d_H_swiglu = nullptr, void* d_C_bf16 = nullptr,
                       tl_gemm_plan_info* plan_only = nullptr, GemmParams* params_only = nullptr,
                       GemmPlan* params_plan = nullptr) {
    // params_only: everything up to the launch (checks, plan, tensor maps, workspace) and then the kernel's
    // parameters are handed back instead of being launched (the expert FFN runs two products in one kernel).
    // plan_only: no pointer is looked at, nothing is encoded or enqueued; *plan_only receives what a launch with
    // these sizes would run (the same code decides both, so the two cannot drift apart).
    const int es = elem_bytes;                       // 2: bf16, 1: FP8 (E4M3), K-contiguous weights only
    const int k_shift = es == 1 ? 1 : 0;
    if (es != 2 && !(es == 1 && kmajor)) return TL_ERR_UNSUPPORTED;
    if (rows_total < 0 || N <= 0 || K <= 0 || E < 1) return TL_ERR_INVALID_ARG;
    if (rows_total == 0 && !plan_only) return TL_OK;
    if (!plan_only) {
        if (!d_A || !d_B || (!d_C && !d_H_swiglu && !d_C_bf16)) return TL_ERR_INVALID_ARG;
        if (d_C_bf16 && (N % 8 != 0 || reinterpret_cast<uintptr_t>(d_C_bf16) % 16 != 0)) return TL_ERR_INVALID_ARG;
        if (d_H_swiglu && (N % 64 != 0 || reinterpret_cast<uintptr_t>(d_H_swiglu) % 16 != 0)) return TL_ERR_INVALID_ARG;
    }
    // fp32 C is written (by the weights-on-N epilogue and by the stream-K reduction) in 16-byte vectors: rows of C
    // must start on 16-byte boundaries and hold a whole number of vectors.
    if (!d_H_swiglu && !d_C_bf16 && N % 4 != 0) return TL_ERR_UNSUPPORTED;
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
    if (!plan_only) {
        if (reinterpret_cast<uintptr_t>(d_A) % 16 != 0) return TL_ERR_ALIGNMENT;
        if (reinterpret_cast<uintptr_t>(d_B) % (row_major || generic ? 16 : 128) != 0) return TL_ERR_ALIGNMENT;
        if (reinterpret_cast<uintptr_t>(d_C) % 16 != 0) return TL_ERR_ALIGNMENT;
    }

    // Two kinds of memory tiles that TMA cannot box as 64-column atoms can still be fetched as they are:
    //   bc == 8 (16-byte rows): the tiles are core matrices of the no-swizzle MN-major operand layout;
    //   bc == 1 (a tile = br consecutive K values of one column): the buffer is [K/br][N][br], a K-major operand
    //           in panels of br K values, swizzle rows of min(128, 2 br) bytes (no swizzle for 16-byte rows).
    const bool raw_shape = generic && bc == 8 && br >= 8 && opt(TL_OPT_GENERIC_RAW) != 0;
    const bool kcol_shape = generic && bc == 1 && br >= 8 && opt(TL_OPT_GENERIC_RAW) != 0;
    //   bc == 4 or 2 (8- or 4-byte rows), 8 <= br <= 64 or 128: fetched as stored as well, then 2 or 4 neighbouring tiles
    //           are transposed in place into one br x 8 tile with 16-byte rows (four more warps, see the kernel).
    const bool fix_shape = generic && ((bc == 4 && br >= 8 && br <= 64) || (bc == 2 && br >= 8 && br <= 128)) &&
                           opt(TL_OPT_GENERIC_RAW) != 0;
    bool raw_operand = false, kcol_operand = false, fix_operand = false;
    if (int rc = ensure_device_info()) return rc;
    // enough 256 x 256 tiles for every cluster of the CTA-pair kernel to get one
    const bool pair_sized = ceil_div(rows_total, 256) * ceil_div(N, 256) * 2 >= dev().sm_count;
    // Dense products of 65 to 512 token rows on TMA-readable weights are bound by what one SM can pull out of L2: a
    // 128-row token slab comes with every weight slab, and with 128 weight columns per tile it is half of all bytes
    // (Llama gate_up at 128 tokens: 190 us).  Twice the columns per tile (128 x 256 x 64) make it a third (167 us),
    // but halve the number of tiles.  The wider tile is taken where it has a schedule without partial tiles in global
    // memory (they are 128 KB each: down at 384 tokens, K cut over all CTAs, 213 us with the narrow tile against 289)
    // and mid_tile_estimate_us says it is ahead.  Where the default would be the CTA-pair kernel: up to 384 rows the
    // wide tile (gate_up at 256 tokens 255 against 308 us), beyond that the pair kernel.
    // (129 to 256 rows with less than 8192 weight rows and tiles for at least three quarters of the pair kernel's waves
    // stay with CTA pairs: with a short K loop their deeper pipeline and hidden epilogue count for more than the token
    // rows they load -- gate_up-shaped, 256 rows: K = 4096 132 us against 145-148, K = 1024 57 against 70-75; K = 8192 a tie)
    bool pairs_ahead = false;
    if (rows_max > 128 && rows_max <= 256 && pair_sized && (K >> k_shift) < 8192 && opt(TL_OPT_PAIR_KERNEL) != 0) {
        const int64_t tiles = ceil_div(N, 256), clusters = dev().sm_count / 2;
        pairs_ahead = 4 * tiles >= 3 * ceil_div(tiles, clusters) * clusters;
    }
    if (cta_m == 0 && cta_n == 0 && cta_k == 0 && !d_offsets && !fixed && !generic && rows_max > 64 && rows_max <= 512 &&
        !(rows_max > 384 && pair_sized) && !pairs_ahead) {
        GemmPlan wide, other;
        // 129 to 256 rows: both 128-row blocks on one weight slab per stage (256 x 256 x 64, whole tiles only), where
        // there are enough tiles: a third less out of L2 again (Llama gate_up at 256 rows 257 -> 235 us)
        if (rows_max > 128 && rows_max <= 256 &&
            make_plan(rows_max, ceil_div(N, 256), N, K >> k_shift, 256, 256, 64, false, &wide, false, false, pair_sized,
                      rows_total) == TL_OK) {
            cta_m = 256;
            cta_n = 256;
            cta_k = 64;
        } else if (make_plan(rows_max, ceil_div(rows_total, 128) * ceil_div(N, 256), N, K >> k_shift, 128, 256, 64, false, &wide,
                      false, false, pair_sized, rows_total) == TL_OK &&
            wide.stream_k == 0) {
            int bm = 0, bn = 0, bk = 0;
            default_tile(rows_max, false, false, &bm, &bn, &bk, pair_sized);
            bool take = bm > 128;                           // against the pair kernel
            if (!take && make_plan(rows_max, ceil_div(rows_total, bm) * ceil_div(N, bn), N, K >> k_shift, 0, 0, 0, false,
                                   &other, false, false, pair_sized, rows_total) == TL_OK)
                take = mid_tile_estimate_us(wide, rows_total, N, K >> k_shift) <
                       0.97 * mid_tile_estimate_us(other, rows_total, N, K >> k_shift);
            if (take) {
                cta_m = 128;
                cta_n = 256;
                cta_k = 64;
            }
        }
    }
    // More rows, where the CTA-pair kernel is the default: its 74 clusters take 256 x 256 tiles in whole waves, and a
    // tile count just above a multiple of 74 costs a whole wave more (Llama down at 1024 rows: 128 tiles, two waves,
    // 410 us).  The two-block tile does the same tile on one SM in about 1.7 units of a pair's 256-token tile; where its
    // whole-tile schedule fits the tile count better by a tenth it is taken (128 tiles on 128 CTAs: 351 us).
    if (cta_m == 0 && cta_n == 0 && cta_k == 0 && !d_offsets && !fixed && !generic && rows_max > 512 && pair_sized &&
        opt(TL_OPT_PAIR_KERNEL) != 0) {
        GemmPlan two;
        const int64_t tiles = ceil_div(rows_total, 256) * ceil_div(N, 256);
        if (make_plan(rows_max, tiles, N, K >> k_shift, 256, 256, 64, false, &two, false, false, pair_sized, rows_total) == TL_OK) {
            int clusters = dev().pair_max_clusters;
            if (clusters <= 0) clusters = dev().sm_count / 2;             // (not asked yet: at most one pair per two SMs)
            int64_t big = opt(TL_OPT_PAIR_512) == 0 ? 0 : (ceil_div(rows_total, 512) * ceil_div(N, 256) / clusters) * clusters;
            const double pair_units = pair_schedule_units(rows_total, N, clusters, &big);
            if (1.7 * double(ceil_div(tiles, int64_t(two.grid))) < 0.9 * pair_units) {
                cta_m = 256;
                cta_n = 256;
                cta_k = 64;
            }
        }
    }
    if (cta_m == 0 && cta_n == 0 && cta_k == 0 && d_offsets && !fixed && !generic) {
        if (const int rows = grouped_tile_rows(rows_total, E, N)) { cta_m = rows; cta_n = 256; cta_k = 64; }
    }
    GemmPlan plan;
    {
        // upper bound of tiles: every expert may add one ragged m-tile
        int bm_guess = cta_m, bn_guess = cta_n, bk_guess = cta_k;
        if (cta_m == 0 && cta_n == 0 && cta_k == 0)
            default_tile(rows_max, d_offsets != nullptr, fixed != nullptr, &bm_guess, &bn_guess, &bk_guess, pair_sized);
        if (bm_guess <= 0 || bn_guess <= 0) return TL_ERR_UNSUPPORTED;
        const int64_t mt_bound = d_offsets ? rows_total / bm_guess + E : ceil_div(rows_total, bm_guess);
        // (the plan counts K in 2-byte units: an 8-bit stage holds twice as many elements)
        // Memory tiles with 16-byte rows (8 bf16 columns, at least 8 rows) need no permutation: the raw tiles are
        // core matrices of the MMA's no-swizzle operand layout and the copy engine can fetch them as they are.
        // Planned like any TMA-readable weight; if the CTA tile then does not hold whole memory tiles, the permuting
        // path takes over.
        if (raw_shape) {
            const int rc = make_plan(rows_max, mt_bound * ceil_div(N, bn_guess), N, K >> k_shift, cta_m, cta_n, cta_k,
                                     d_offsets != nullptr, &plan, fixed != nullptr, false, pair_sized, rows_total);
            raw_operand = rc == TL_OK && plan.BK % br == 0 && plan.BN % bc == 0;
        }
        if (kcol_shape) {
            const int rc = make_plan(rows_max, mt_bound * ceil_div(N, bn_guess), N, K >> k_shift, cta_m, cta_n, cta_k,
                                     d_offsets != nullptr, &plan, fixed != nullptr, false, pair_sized, rows_total);
            kcol_operand = rc == TL_OK;
        }
        if (fix_shape) {
            const int rc = make_plan(rows_max, mt_bound * ceil_div(N, bn_guess), N, K >> k_shift, cta_m, cta_n, cta_k,
                                     d_offsets != nullptr, &plan, fixed != nullptr, false, pair_sized, rows_total);
            fix_operand = rc == TL_OK && plan.BK % br == 0;
        }
        if (!raw_operand && !kcol_operand && !fix_operand)
            if (int rc = make_plan(rows_max, mt_bound * ceil_div(N, bn_guess), N, K >> k_shift, cta_m, cta_n, cta_k,
                                   d_offsets != nullptr, &plan, fixed != nullptr, generic, pair_sized, rows_total))
                return rc;
    }
    if (d_offsets && K % (int64_t(plan.BK) << k_shift) != 0) return TL_ERR_UNSUPPORTED;   // a K tail would read the next expert's rows
    if (d_H_swiglu && !plan.weights_on_n) return TL_ERR_UNSUPPORTED;        // the gated epilogue pairs columns of one token row
    if (!plan_only && opt(TL_OPT_PLAN_AS_IF_SMS) != 0) return TL_ERR_INVALID_ARG;      // the planning test hook is on
    if (!fixed && !plan_only)
        if (int rc = ensure_control()) return rc;

    const bool pdl_ok = opt(TL_OPT_PDL) != 0;
    GemmParams p;
    memset(&p, 0, sizeof p);
    // (plan_only: the views are worked out as usual but not encoded)
    auto encode_tensor_map = [&](CUtensorMap* out, const void* base, int dt, int swz, int rank, const uint64_t* dims,
                                 const uint64_t* strides_bytes, const uint32_t* box) -> int {
        if (plan_only) return TL_OK;
        return tl::encode_tensor_map(out, base, dt, swz, rank, dims, strides_bytes, box);
    };
    auto encode = [&](CUtensorMap* out, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                      const uint32_t* box) -> int {
        return encode_tensor_map(out, base, int(CU_TENSOR_MAP_DATA_TYPE_BFLOAT16), int(CU_TENSOR_MAP_SWIZZLE_128B), rank,
                                 dims, strides_bytes, box);
    };
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
    uint64_t raw_chunk = 2048;                   // raw memory tiles as the operand: bytes per tensor-map row (see below)
    const bool kcol16 = kcol_operand && br == 8;      // 16-byte tiles: one run of them is a row of K-major core matrices already
    if (raw_operand || kcol16 || fix_operand)
        while ((uint64_t(plan.BN) * br * 2) % raw_chunk != 0 || (uint64_t(N) * br * 2) % raw_chunk != 0) raw_chunk >>= 1;
    // The tile-major buffer as plain bytes: (chunk of 8-byte words, chunks along a row of the tile grid, rows of the tile
    // grid); the box is the stage's cta_k/br runs of whole memory tiles, landed in memory order without swizzle.
    auto encode_byte_runs = [&]() -> int {
        const uint64_t run_full = uint64_t(plan.BN) * br * 2, grid_row = uint64_t(N) * br * 2, chunk = raw_chunk;
        const uint64_t dims[5] = {chunk / 8, grid_row / chunk, uint64_t(K / br) * E, 1, 1};
        const uint64_t str[5] = {8, chunk, grid_row, grid_row * uint64_t(K / br) * E, grid_row * uint64_t(K / br) * E};
        const uint32_t box[5] = {uint32_t(chunk / 8), uint32_t(run_full / chunk), uint32_t(plan.BK / br), 1, 1};
        return encode_tensor_map(&p.tmap_b, d_B, int(CU_TENSOR_MAP_DATA_TYPE_INT64), int(CU_TENSOR_MAP_SWIZZLE_NONE), 5, dims, str, box);
    };
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
    } else if (kcol_operand) {
        // Memory tiles of br rows x 1 column: [K/br][N][br] seen as (e, N, br/e, E*K/br) with swizzle rows of
        // r = min(128, 2 br) bytes = e elements; the box takes all swizzle rows of the stage's K range for the CTA
        // tile's columns, so the bytes land as [K row][cta_n rows][r], the canonical K-major operand.
        RB = plan.BK;
        AB = NA;
        w_row_bytes = br * 2 < kAtomBytes ? br * 2 : kAtomBytes;
        const int e = w_row_bytes / 2;
        const int swz = w_row_bytes == 128 ? int(CU_TENSOR_MAP_SWIZZLE_128B) : w_row_bytes == 64 ? int(CU_TENSOR_MAP_SWIZZLE_64B)
                        : w_row_bytes == 32 ? int(CU_TENSOR_MAP_SWIZZLE_32B) : int(CU_TENSOR_MAP_SWIZZLE_NONE);
        const int k_box = br < plan.BK ? br : plan.BK;
        const uint64_t big = uint64_t(N) * br * 2 * uint64_t(K / br) * E;
        if (kcol16) {
            // (16-byte tiles: consecutive columns' tiles already form the 128-byte core matrices, so the stage's
            // runs are fetched as plain bytes, see the next case)
            if (int rc = encode_byte_runs()) return rc;
        } else {
            const uint64_t dims[5] = {uint64_t(e), uint64_t(N), uint64_t(br / e), uint64_t(K / br) * E, 1};
            const uint64_t str[5] = {2, uint64_t(br) * 2, uint64_t(w_row_bytes), uint64_t(N) * br * 2, big};
            const uint32_t box[5] = {uint32_t(e), uint32_t(plan.BN), uint32_t(k_box / e), uint32_t(plan.BK / k_box), 1};
            if (int rc = encode_tensor_map(&p.tmap_b, d_B, dtype, swz, 5, dims, str, box)) return rc;
        }
        p.k_coord_per_expert = int(K / br);
        p.br_log2 = ilog2(br);
        p.bc_log2 = 0;
        p.w_kmajor = 1;
        p.w_atom_log2 = ilog2(e);
        w_layout = w_row_bytes == 128 ? 2u : w_row_bytes == 64 ? 4u : w_row_bytes == 32 ? 6u : 0u;
    } else if (raw_operand || fix_operand) {
        // (8- and 4-byte rows: the same view; the stage is fixed up in shared memory into the image described here)
        // Memory tiles of br rows x 16 bytes.  A stage is cta_k/br runs of cta_n/8 whole tiles, each run contiguous in
        // the tile-major buffer, so the buffer is seen as plain bytes: (chunk of 8-byte words, chunks along a row of
        // the tile grid, rows of the tile grid) with chunk = the largest power of two up to 2 KB that divides both
        // one run and a whole row of the tile grid; the box takes the stage's runs and
        // lands them in memory order, no swizzle.  Columns beyond N and rows beyond K arrive as zeros.
        RB = plan.BK;
        AB = NA;
        if (int rc = encode_byte_runs()) return rc;
        p.k_coord_per_expert = int(K / br);
        p.br_log2 = ilog2(br);
        p.bc_log2 = ilog2(bc);
        p.generic_b = fix_operand ? 2 : 0;
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
        // count tiles along N and K).  TL_OPT_BOX_PER_BLOCK issues one instruction per memory tile instead
        // (same bytes, same shared-memory image; measurably slower because instruction issue then limits).
        // tl_set_option(TL_OPT_BOX_PER_BLOCK, 1) selects it.
        const bool per_block = opt(TL_OPT_BOX_PER_BLOCK) != 0;
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
        if (kcol16) {                               // (.., chunk along the tile-grid row, tile-grid row, -, -)
            set(0, 0, 0, ilog2(int64_t(raw_chunk / 16)), all, 0);
            set(1, 3, all, 0, 0, 1);
        } else if (kcol_operand) {                  // (.., weight column, swizzle row in tile, tile along K, -)
            set(0, 0, 0, 0, all, 0);
            set(1, p.w_atom_log2, (br >> p.w_atom_log2) - 1, 0, 0, 0);
            set(2, ilog2(br), all, 0, 0, 1);
        } else if (raw_operand || fix_operand) {    // (.., chunk along the tile-grid row, tile-grid row, -, -)
            set(0, 0, 0, ilog2(int64_t(raw_chunk / (uint64_t(br) * 2))), all, 0);
            set(1, ilog2(br), all, 0, 0, 1);
        } else if (generic) {
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
    const bool permuted = generic && !raw_operand && !kcol_operand && !fix_operand;     // the generic-address path proper
    p.kbx = permuted ? 0 : plan.BK / (RB * kb_box);
    p.nbx = permuted ? 0 : NA / (AB * nb_box);
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
    if (kmajor || kcol_operand) {
        // K-major image: [swizzle row along K][cta_n rows][r bytes]; 8-row groups 8r bytes apart, a K step of one
        // instruction (32 bytes) is 32 bytes further inside the swizzle row, the next swizzle row cta_n rows further.
        // (16-byte rows, no swizzle: an instruction's K step is two rows, the second cta_n rows further.)
        const uint32_t r = uint32_t(w_row_bytes), steps_per_row = r / 32u;
        p.lbo = r == 16 ? uint32_t(plan.BN) * 16u : 16u;
        p.sbo = 8u * r;
        p.ugroup_off = 128u * r;
        for (int j = 0; j < plan.BK / 16; ++j)
            p.kstep_off[j] = r == 16 ? uint32_t(j) * 2u * uint32_t(plan.BN) * 16u
                                     : (uint32_t(j) / steps_per_row) * uint32_t(plan.BN) * r + (uint32_t(j) % steps_per_row) * 32u;
        p.box_rows = plan.BK << k_shift;
        p.box_atoms = NA;
        p.kbx = p.nbx = 1;
        p.box_bytes = uint32_t(plan.BK) * plan.BN * 2;
    }
    if (raw_operand || fix_operand) {
        // The stage holds cta_k/br runs of cta_n/8 memory tiles in memory order.  A memory tile is br/8 core matrices
        // (8 K rows x 16 bytes) one after the other: the next one along K is 128 bytes further (in the next run when
        // a tile has only 8 rows), the next one along N one memory tile further; no swizzle.
        const uint32_t run_full = uint32_t(plan.BN) * br * 2;
        p.lbo = br >= 16 ? 128u : run_full;
        p.sbo = 16u * uint32_t(br);                 // one br x 8 tile
        p.ugroup_off = 16u * p.sbo;
        for (int j = 0; j < plan.BK / 16; ++j)
            p.kstep_off[j] = uint32_t((j * 16) / br) * run_full + uint32_t((j * 16) % br) * 16u;
        w_layout = 0u;
    }
    p.w_desc_hi = smem_desc_hi(p.lbo, p.sbo, w_layout);
    p.C = d_C;
    p.Cb = static_cast<__nv_bfloat16*>(d_C_bf16);
    p.epi_swiglu = d_H_swiglu != nullptr;
    p.H = static_cast<__nv_bfloat16*>(d_H_swiglu);
    p.ldh = N / 2;
    p.offsets = d_offsets;
    p.status = fixed ? fixed->status : dev().ctl.d_status;
    p.wait_limit_ns = wait_limit_ns();
    p.reduce_split = opt(TL_OPT_REDUCE_SPLIT) != 0;
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
    p.cluster_k = plan.cluster_k;
    p.raw_slots = plan.raw_slots;
    p.smem_limit = uint32_t(plan.smem_bytes);
    p.b_bytes = int64_t(E) * K * N * es;
    p.num_stages = plan.num_stages;
    const int prefetch_env = int(opt(TL_OPT_PREFETCH_STAGES));   // measurement switch, -1: the default below
    // (at most four instructions: the thread that issues them holds up the CTA's first barrier for their duration)
    p.prefetch_stages = !pdl_ok ? 0 : (prefetch_env >= 0 ? prefetch_env : (plan.num_stages < 4 ? plan.num_stages : 4));

    cudaError_t err = cudaSuccess;
    tl_gemm_plan_info info;
    memset(&info, 0, sizeof info);
    info.cta_m = plan.BM; info.cta_n = plan.BN; info.cta_k = plan.BK << k_shift;
    info.stream_k = plan.stream_k; info.grid = plan.grid; info.stages = plan.num_stages;
    info.weights_on_n = plan.weights_on_n; info.generic_path = generic ? (permuted ? 1 : fix_operand ? 3 : 2) : 0; info.cluster_k = plan.cluster_k;
    info.workspace_bytes = plan.ws_bytes;
    // Large dense problems on TMA-readable weights: CTA pairs (cta_group::2 MMAs), see tl_gemm_pair.cuh.
    const bool no_pair = opt(TL_OPT_PAIR_KERNEL) == 0;     // measurement switch
    // Worth it once every cluster of the machine has at least one 256 x 256 tile; smaller problems keep the
    // single-CTA kernel and its stream-K split.
    if (!no_pair && !d_offsets && !permuted && !fix_operand && !d_H_swiglu && plan.BM == 256 && plan.BN == 128 && plan.BK == 64 &&
        p.kbx == 1 && p.nbx == 1 && pair_sized) {
        int& max_clusters = dev().pair_max_clusters;
        if (max_clusters < 0) {
            int n = 0;
            if (int rc = pair_max_active_clusters(&n)) return rc;
            max_clusters = n;
        }
        // 512-token tiles (one weight slab per stage for two token blocks) as long as they fill whole waves of
        // clusters; what is left of the tile grid runs as 256-token tiles.  TL_OPT_PAIR_512 = 0: 256-token tiles only.
        const bool halves_off = opt(TL_OPT_PAIR_512) == 0;
        const int64_t big_total = ceil_div(rows_total, 512) * ceil_div(N, 256);
        int64_t big_tiles = halves_off ? 0 : (big_total / max_clusters) * max_clusters;
        if (big_tiles > 0) (void)pair_schedule_units(rows_total, N, max_clusters, &big_tiles);
        const int halves = big_tiles > 0 ? 2 : 1;
        const size_t stage_bytes = 64 * 128 * 2 + size_t(halves) * 128 * kAtomBytes;
        int stages = int((kMaxDynamicSmem - 1024) / stage_bytes);
        if (stages > kPairStagesMax) stages = kPairStagesMax;
        const int stage_cap = int(opt(TL_OPT_MAX_STAGES));
        if (stage_cap >= 2 && stages > stage_cap) stages = stage_cap;
        p.num_stages = stages;
        p.pair_big_tiles = int(big_tiles);
        // behind the stages: 32 x 32 blocks of C on their way to a bulk store, one or two per epilogue warp
        const size_t out_warp_bytes = size_t(halves == 2 ? 8 : 4) * kPairStageOutBytes;
        p.out_bufs = size_t(stages) * stage_bytes + 1024 + 2 * out_warp_bytes <= size_t(kPairDynamicSmem) ? 2 : 1;
        const size_t smem = size_t(stages) * stage_bytes + 1024 + size_t(p.out_bufs) * out_warp_bytes;
        if (smem > size_t(kPairDynamicSmem)) return TL_ERR_UNSUPPORTED;
        const int64_t pair_tiles = halves == 2 ? big_tiles + 2 * (big_total - big_tiles)
                                               : ceil_div(rows_total, 256) * ceil_div(N, 256);
        const int clusters = int(pair_tiles < max_clusters ? pair_tiles : max_clusters);
        info.pair_kernel = 1;
        info.cta_m = halves == 2 ? 512 : 256;        // per CTA: its own 128 weight columns of the pair's 256
        info.stream_k = 0; info.grid = 2 * clusters; info.stages = p.num_stages; info.weights_on_n = 0;
        info.workspace_bytes = 0;
        info.pair_tiles_512 = big_tiles; info.pair_tiles_256 = pair_tiles - big_tiles;
        if (opt(TL_OPT_LOG))
            fprintf(stderr, "[tilelens] pair kernel: %lld tiles (%lld of 512 tokens), %d clusters (max active %d), %d stages, %zu B smem\n",
                    (long long)pair_tiles, (long long)big_tiles, clusters, max_clusters, p.num_stages, smem);
        if (plan_only) { *plan_only = info; return TL_OK; }
        // C as a tensor map (bulk stores need 16-byte aligned rows); otherwise the epilogue stores from registers
        p.c_tma = 0;
        {
            const void* c_base = d_C_bf16 ? d_C_bf16 : static_cast<const void*>(d_C);
            const int c_es = d_C_bf16 ? 2 : 4;
            if (opt(TL_OPT_PAIR_TMA_STORE) != 0 && reinterpret_cast<uintptr_t>(c_base) % 16 == 0 && (N * c_es) % 16 == 0) {
                const uint64_t dims[2] = {uint64_t(N), uint64_t(rows_total)}, str[2] = {uint64_t(c_es), uint64_t(N) * c_es};
                const uint32_t box[2] = {32, 32};
                if (int rc = encode_tensor_map(&p.tmap_c, c_base, d_C_bf16 ? int(CU_TENSOR_MAP_DATA_TYPE_BFLOAT16) : int(CU_TENSOR_MAP_DATA_TYPE_FLOAT32),
                                               int(CU_TENSOR_MAP_SWIZZLE_NONE), 2, dims, str, box))
                    return rc;
                p.c_tma = 1;
            }
        }
        last_plan() = info;
        return launch_gemm_pair(es == 1, halves, clusters, smem, stream, p);
    }
    if (opt(TL_OPT_LOG))
        fprintf(stderr, "[tilelens] gemm kernel: cta %d x %d x %d, weights on %s, %s, grid %d, %d stages, %zu B workspace%s\n",
                info.cta_m, info.cta_n, info.cta_k, plan.weights_on_n ? "N" : "M",
                plan.stream_k ? "stream-K" : plan.cluster_k > 1 ? "cluster split-K" : "whole tiles",
                plan.grid, plan.num_stages, plan.ws_bytes,
                raw_operand || kcol_operand ? ", raw memory tiles as the operand" : fix_operand ? ", memory tiles fixed up in place"
                                                                                    : generic ? ", generic-address weights" : "");
    if (plan_only) { *plan_only = info; return TL_OK; }
    last_plan() = info;
    // Split-K scratch (none for whole-tile schedules).  A fixed scratch keeps the previous launch's contents; nothing
    // in it has to start at zero: every partial tile is written by the GEMM kernel before the reduction kernel reads it.
    void* ws = nullptr;
    if (fixed) {
        if (plan.ws_bytes > fixed->ws_bytes) return TL_ERR_WORKSPACE;
        ws = plan.ws_bytes ? fixed->ws : nullptr;
    } else if (int rc = get_workspace(plan.ws_bytes, &ws, stream)) {
        return rc;
    }
    p.partials = static_cast<float*>(ws);
    // Test hook (TL_OPT_STALL_ONCE = 1): this launch arms the first stage of every CTA for 16 bytes more than its
    // copies deliver, so that the wait on it runs out after TL_OPT_WAIT_LIMIT_US and the kernel gives up in an orderly way.
    if (opt(TL_OPT_STALL_ONCE) == 1) {
        p.stall_extra_tx = 16;
        tl_set_option(TL_OPT_STALL_ONCE, 0);
    }
    // Test hook (TL_OPT_STALL_ONCE = 4): this grouped launch builds its provisional tables from offsets that are
    // 7 rows off, so that the check after the wait finds them wrong and the tables are built again.
    if (opt(TL_OPT_STALL_ONCE) == 4 && d_offsets) {
        p.provisional_skew = 7;
        tl_set_option(TL_OPT_STALL_ONCE, 0);
    }
    if (params_only) {
        *params_only = p;
        *params_plan = plan;
        return TL_OK;
    }
    // The GEMM kernel may be scheduled while its predecessor in the stream is finishing (it waits before touching
    // memory).  TL_OPT_PDL = 0 restores plain stream order for measurement.
    int rc = TL_OK;
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(plan.grid);
        cfg.blockDim = dim3(permuted || fix_operand ? kGenericThreads : kGemmThreads);
        cfg.dynamicSmemBytes = plan.smem_bytes;
        cfg.stream = stream;
        cudaLaunchAttribute attr[2];
        int n_attr = 0;
        if (pdl_ok) {
            attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
            ++n_attr;
        }
        if (plan.cluster_k > 1) {
            attr[n_attr].id = cudaLaunchAttributeClusterDimension;
            attr[n_attr].val.clusterDim.x = unsigned(plan.cluster_k);
            attr[n_attr].val.clusterDim.y = 1;
            attr[n_attr].val.clusterDim.z = 1;
            ++n_attr;
        }
        cfg.attrs = attr;
        cfg.numAttrs = n_attr;
        if (plan.weights_on_n) rc = es == 1 ? launch_gemm_wn_fp8(plan.BK, plan.BN, &cfg, p) : launch_gemm_wn_bf16(plan.BK, plan.BN, &cfg, p);
        else rc = es == 1 ? launch_gemm_wm_fp8(plan.BK, plan.BN, &cfg, p) : launch_gemm_wm_bf16(plan.BK, plan.BN, &cfg, p);
        if (rc == TL_ERR_CUDA && plan.cluster_k > 1) {
            // A device (or a partition of one) that cannot place clusters of this size refuses the launch; nothing was
            // enqueued.  The stream-K cut computes the same product.
            const int64_t saved = opt(TL_OPT_NO_SCRATCH_PLANS);
            tl_set_option(TL_OPT_NO_SCRATCH_PLANS, 0);
            rc = gemm_launch(d_A, d_B, d_C, d_offsets, E, rows_total, rows_max, N, K, G, br, bc, cta_m, cta_n, cta_k, stream,
                             fixed, kmajor, elem_bytes, d_H_swiglu, d_C_bf16, nullptr, nullptr, nullptr);
            tl_set_option(TL_OPT_NO_SCRATCH_PLANS, saved);
            return rc;
        }
        if (rc) return rc;
    }
    // stream-K: add up the partial tiles, one CTA per boundary between two CTA ranges
    if (plan.stream_k && plan.grid > 1) return launch_reduce(p, plan.grid, stream, pdl_ok);
    if (err != cudaSuccess) return check_cuda(err);
    return check_cuda(cudaGetLastError());
}

}  // namespace tl

extern "C" {

int tl_gemm(const void* d_A, const void* d_B, float* d_C, int64_t M, int64_t N, int64_t K, int64_t G, int block_rows,
            int block_cols, int cta_m, int cta_n, int cta_k, void* cuda_stream) {
    tl::ApiLock lock;
    return tl::gemm_launch(d_A, d_B, d_C, nullptr, 1, M, M, N, K, G, block_rows, block_cols, cta_m, cta_n, cta_k,
                           static_cast<cudaStream_t>(cuda_stream));
}

int tl_gemm_grouped(const void* d_A_sorted, const void* d_B_experts, float* d_C, const int32_t* d_offsets, int E,
                    int64_t total_rows, int64_t N, int64_t K, int64_t G, int block_rows, int block_cols, int cta_m,
                    int cta_n, int cta_k, void* cuda_stream) {
    tl::ApiLock lock;
    if (!d_offsets && total_rows > 0) return TL_ERR_INVALID_ARG;
    // Without a host copy of the offsets the largest expert is unknown: size tiles for the total.
    return tl::gemm_launch(d_A_sorted, d_B_experts, d_C, d_offsets, E, total_rows, total_rows, N, K, G, block_rows,
                           block_cols, cta_m, cta_n, cta_k, static_cast<cudaStream_t>(cuda_stream));
}

int tl_gemm_kmajor(const void* d_A, const void* d_B_nk, float* d_C, int64_t M, int64_t N, int64_t K, int64_t G, int tile_n,
                   int tile_k, int cta_m, int cta_n, int cta_k, void* cuda_stream) {
    tl::ApiLock lock;
    return tl::gemm_launch(d_A, d_B_nk, d_C, nullptr, 1, M, M, N, K, G, tile_n, tile_k, cta_m, cta_n, cta_k,
                           static_cast<cudaStream_t>(cuda_stream), nullptr, true);
}

int tl_gemm_grouped_kmajor(const void* d_A_sorted, const void* d_B_experts_nk, float* d_C, const int32_t* d_offsets, int E,
                           int64_t total_rows, int64_t N, int64_t K, int64_t G, int tile_n, int tile_k, int cta_m,
                           int cta_n, int cta_k, void* cuda_stream) {
    tl::ApiLock lock;
    if (!d_offsets && total_rows > 0) return TL_ERR_INVALID_ARG;
    return tl::gemm_launch(d_A_sorted, d_B_experts_nk, d_C, d_offsets, E, total_rows, total_rows, N, K, G, tile_n, tile_k,
                           cta_m, cta_n, cta_k, static_cast<cudaStream_t>(cuda_stream), nullptr, true);
}

int tl_gemm_fp8_kmajor(const void* d_A, const void* d_B_nk, float* d_C, int64_t M, int64_t N, int64_t K, int64_t G,
                       int tile_n, int tile_k, int cta_m, int cta_n, int cta_k, void* cuda_stream) {
    tl::ApiLock lock;
    if (cta_k != 0 && cta_k != 128 && cta_k != 256) return TL_ERR_UNSUPPORTED;
    return tl::gemm_launch(d_A, d_B_nk, d_C, nullptr, 1, M, M, N, K, G, tile_n, tile_k, cta_m, cta_n, cta_k / 2,
                           static_cast<cudaStream_t>(cuda_stream), nullptr, true, 1);
}

int tl_gemm_grouped_fp8_kmajor(const void* d_A_sorted, const void* d_B_experts_nk, float* d_C, const int32_t* d_offsets,
                               int E, int64_t total_rows, int64_t N, int64_t K, int64_t G, int tile_n, int tile_k,
                               int cta_m, int cta_n, int cta_k, void* cuda_stream) {
    tl::ApiLock lock;
    if (!d_offsets && total_rows > 0) return TL_ERR_INVALID_ARG;
    if (cta_k != 0 && cta_k != 128 && cta_k != 256) return TL_ERR_UNSUPPORTED;
    return tl::gemm_launch(d_A_sorted, d_B_experts_nk, d_C, d_offsets, E, total_rows, total_rows, N, K, G, tile_n, tile_k,
                           cta_m, cta_n, cta_k / 2, static_cast<cudaStream_t>(cuda_stream), nullptr, true, 1);
}

int tl_gemm_bf16(const void* d_A, const void* d_B, void* d_C_bf16, int64_t M, int64_t N, int64_t K, int64_t G,
                 int block_rows, int block_cols, int cta_m, int cta_n, int cta_k, void* cuda_stream) {
    tl::ApiLock lock;
    if (!d_C_bf16) return TL_ERR_INVALID_ARG;
    return tl::gemm_launch(d_A, d_B, nullptr, nullptr, 1, M, M, N, K, G, block_rows, block_cols, cta_m, cta_n, cta_k,
                           static_cast<cudaStream_t>(cuda_stream), nullptr, false, 2, nullptr, d_C_bf16);
}

int tl_gemm_grouped_bf16(const void* d_A_sorted, const void* d_B_experts, void* d_C_bf16, const int32_t* d_offsets, int E,
                         int64_t total_rows, int64_t N, int64_t K, int64_t G, int block_rows, int block_cols, int cta_m,
                         int cta_n, int cta_k, void* cuda_stream) {
    tl::ApiLock lock;
    if (!d_offsets && total_rows > 0) return TL_ERR_INVALID_ARG;
    if (!d_C_bf16) return TL_ERR_INVALID_ARG;
    return tl::gemm_launch(d_A_sorted, d_B_experts, nullptr, d_offsets, E, total_rows, total_rows, N, K, G, block_rows,
                           block_cols, cta_m, cta_n, cta_k, static_cast<cudaStream_t>(cuda_stream), nullptr, false, 2,
                           nullptr, d_C_bf16);
}

int tl_gemm_grouped_swiglu(const void* d_A_sorted, const void* d_B_experts_gate_up, void* d_H_bf16, const int32_t* d_offsets,
                           int E, int64_t total_rows, int64_t N, int64_t K, int64_t G, int block_rows, int block_cols,
                           int cta_m, int cta_n, int cta_k, void* cuda_stream) {
    tl::ApiLock lock;
    if (!d_offsets && total_rows > 0) return TL_ERR_INVALID_ARG;
    if (!d_H_bf16) return TL_ERR_INVALID_ARG;
    return tl::gemm_launch(d_A_sorted, d_B_experts_gate_up, nullptr, d_offsets, E, total_rows, total_rows, N, K, G,
                           block_rows, block_cols, cta_m, cta_n, cta_k, static_cast<cudaStream_t>(cuda_stream), nullptr,
                           false, 2, d_H_bf16);
}

int tl_moe_ffn(const void* d_X_sorted, const void* d_W_gate_up, const void* d_W_down, void* d_H_bf16, float* d_Y,
               const int32_t* d_offsets, int E, int64_t total_rows, int64_t hidden, int64_t inter, int64_t G,
               int block_rows, int block_cols, void* cuda_stream) {
    tl::ApiLock lock;
    if (hidden <= 0 || inter <= 0) return TL_ERR_INVALID_ARG;
    if (!d_offsets && total_rows > 0) return TL_ERR_INVALID_ARG;
    if (!d_H_bf16) return TL_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // One tile for both products (the smaller of what each would take by itself), so that every form of the chain runs
    // the same tiles.
    int ffn_m = 0, ffn_n = 0, ffn_k = 0;
    {
        const int r1 = tl::grouped_tile_rows(total_rows, E, 2 * inter), r2 = tl::grouped_tile_rows(total_rows, E, hidden);
        const int r = r1 < r2 ? r1 : r2;
        const bool tma_rows = block_rows == 0 || block_cols >= 16;          // (narrower memory tiles keep their own path)
        if (r > 0 && tma_rows) { ffn_m = r; ffn_n = 256; ffn_k = 64; }
        // (a routing that would grow one product's tile alone: both at the default 32 rows)
        else if ((r1 > 0 || r2 > 0) && tma_rows) { ffn_m = 32; ffn_n = 256; ffn_k = 64; }
    }
    // (Not while the stream is being captured: the barrier form counts arrivals from a base the host keeps, which a
    // replayed graph would not advance.)
    if (total_rows > 0 && tl::opt(TL_OPT_FFN_ONE_LAUNCH) != 0 && !tl::stream_is_capturing(stream)) {
        // Both products in one cooperative launch (tl_gemm_chain.cu) when they share the kernel instantiation and the
        // grid: TMA-readable weights, the default grouped tile, the stream-K schedule.  Otherwise two launches.
        tl::GemmParams p1, p2;
        tl::GemmPlan plan1, plan2;
        int rc = tl::gemm_launch(d_X_sorted, d_W_gate_up, nullptr, d_offsets, E, total_rows, total_rows, 2 * inter, hidden, G,
                                 block_rows, block_cols, ffn_m, ffn_n, ffn_k, stream, nullptr, false, 2, d_H_bf16, nullptr,
                                 nullptr, &p1, &plan1);
        if (rc) return rc;
        rc = tl::gemm_launch(d_H_bf16, d_W_down, d_Y, d_offsets, E, total_rows, total_rows, hidden, inter, G, block_rows,
                             block_cols, ffn_m, ffn_n, ffn_k, stream, nullptr, false, 2, nullptr, nullptr, nullptr, &p2, &plan2);
        if (rc) return rc;
        // (the grid is the larger of the two plans': a schedule copes with more CTAs than it has work for)
        const int grid = plan1.grid > plan2.grid ? plan1.grid : plan2.grid;
        const bool same = plan1.BM == plan2.BM && plan1.BN == plan2.BN && plan1.BK == plan2.BK &&
                          plan1.BK == 64 && plan1.BN == 256 && plan1.weights_on_n && plan2.weights_on_n &&
                          plan1.cluster_k == 1 && plan2.cluster_k == 1 && !p1.generic_b && !p2.generic_b && grid > 1 &&
                          plan1.smem_bytes <= size_t(tl::kMaxDynamicSmem - 10 * 1024) &&
                          plan2.smem_bytes <= size_t(tl::kMaxDynamicSmem - 10 * 1024);
        if (same && tl::opt(TL_OPT_FFN_ONE_LAUNCH) == 2) {
            // Per-m-tile counters instead of grid barriers (see tl_gemm_chain.cu): the first product as whole tiles
            // only, the second one as usual with its producer waiting for the rows of H it loads.  The workspace
            // holds the second product's partial tiles and, behind them, one counter per m-tile, cleared here.
            const size_t part_bytes = size_t(2) * size_t(grid) * plan2.BM * plan2.BN * sizeof(float);
            const size_t n_flags = size_t(total_rows / plan1.BM) + size_t(E) + 1;
            const size_t ws_bytes = part_bytes + n_flags * sizeof(uint32_t);
            void* ws = nullptr;
            if ((rc = tl::get_workspace(ws_bytes, &ws, stream))) return rc;
            uint32_t* flags = reinterpret_cast<uint32_t*>(static_cast<char*>(ws) + part_bytes);
            if ((rc = tl::check_cuda(cudaMemsetAsync(flags, 0, n_flags * sizeof(uint32_t), stream)))) return rc;
            p1.partials = nullptr;
            p1.stream_k = 0;
            p1.tile_flags = p2.tile_flags = flags;
            p1.tile_flags_mode = 1;
            p2.tile_flags_mode = 2;
            p2.tile_flags_target = 4u * uint32_t(p1.n_tiles);          // four epilogue warps per tile of the first product
            p2.partials = static_cast<float*>(ws);
            // Test hook (TL_OPT_STALL_ONCE = 3): CTA 0 keeps its arrivals to itself, the waits on its m-tiles run out.
            if (tl::opt(TL_OPT_STALL_ONCE) == 3) {
                p1.tile_flags_skip_cta0 = 1;
                tl_set_option(TL_OPT_STALL_ONCE, 0);
            }
            const size_t smem = plan1.smem_bytes > plan2.smem_bytes ? plan1.smem_bytes : plan2.smem_bytes;
            rc = tl::launch_gemm_chain(plan1.BK, plan1.BN, grid, smem, stream, p1, p2, tl::dev().d_grid_counter, 0, 0, false);
            if (rc) return rc;
            tl_gemm_plan_info& info = tl::last_plan();
            memset(&info, 0, sizeof info);
            info.cta_m = plan2.BM; info.cta_n = plan2.BN; info.cta_k = plan2.BK; info.stream_k = 1; info.grid = grid;
            info.stages = plan2.num_stages; info.weights_on_n = 1; info.cluster_k = 1; info.workspace_bytes = ws_bytes;
            info.chained = 2;
            info.stream_k = plan2.stream_k;
            return plan2.stream_k ? tl::launch_reduce(p2, grid, stream, false) : TL_OK;
        }
        if (same) {
            tl::DeviceState& d = tl::dev();
            // one workspace for both phases, sized for the common grid (the first product's partial tiles are summed
            // before the second one writes its own)
            const size_t ws_bytes = size_t(2) * size_t(grid) * plan1.BM * plan1.BN * sizeof(float);
            void* ws = nullptr;
            if ((rc = tl::get_workspace(ws_bytes, &ws, stream))) return rc;
            p1.partials = p2.partials = static_cast<float*>(ws);
            const unsigned long long base = d.grid_arrivals;
            const size_t smem = plan1.smem_bytes > plan2.smem_bytes ? plan1.smem_bytes : plan2.smem_bytes;
            // Test hook (TL_OPT_STALL_ONCE = 3): CTA 0 does not arrive at the first grid barrier, so every CTA's bounded
            // wait there (and at the second barrier, which then cannot fill either) runs out and is reported.
            const bool skip = tl::opt(TL_OPT_STALL_ONCE) == 3;
            if (skip) tl_set_option(TL_OPT_STALL_ONCE, 0);
            rc = tl::launch_gemm_chain(plan1.BK, plan1.BN, grid, smem, stream, p1, p2, d.d_grid_counter,
                                       base + grid, base + 2ull * grid, skip);
            if (rc) return rc;
            d.grid_arrivals = base + 2ull * grid;
            tl_gemm_plan_info& info = tl::last_plan();
            memset(&info, 0, sizeof info);
            info.cta_m = plan2.BM; info.cta_n = plan2.BN; info.cta_k = plan2.BK; info.stream_k = 1; info.grid = grid;
            info.stages = plan2.num_stages; info.weights_on_n = 1; info.cluster_k = 1; info.workspace_bytes = ws_bytes;
            info.chained = 1;
            info.stream_k = plan2.stream_k;
            return plan2.stream_k ? tl::launch_reduce(p2, grid, stream, false) : TL_OK;
        }
    }
    if (int rc = tl_gemm_grouped_swiglu(d_X_sorted, d_W_gate_up, d_H_bf16, d_offsets, E, total_rows, 2 * inter, hidden, G,
                                        block_rows, block_cols, ffn_m, ffn_n, ffn_k, cuda_stream))
        return rc;
    return tl_gemm_grouped(d_H_bf16, d_W_down, d_Y, d_offsets, E, total_rows, hidden, inter, G, block_rows, block_cols, ffn_m,
                           ffn_n, ffn_k, cuda_stream);
}

size_t tl_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K, int cta_m, int cta_n, int cta_k) {
    tl::ApiLock lock;
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    if (tl::ensure_device_info()) return 0;
    size_t need = 0;
    // the largest of the dense schedule and the grouped ones (the grouped tile grows with the rows per expert, and the
    // number of experts is not known here: 32, 64 and 128 rows are all looked at)
    for (int variant = 0; variant < 4; ++variant) {
        const bool grouped = variant != 0;
        int bm = cta_m, bn = cta_n, bk = cta_k;
        const bool pair_sized = tl::ceil_div(M, 256) * tl::ceil_div(N, 256) * 2 >= tl::dev().sm_count;
        const bool free_tile = cta_m == 0 && cta_n == 0 && cta_k == 0;
        if (!free_tile && variant > 1) break;
        if (free_tile) tl::default_tile(M, grouped, false, &bm, &bn, &bk, pair_sized);
        if (free_tile && variant == 2) { bm = 64; bn = 256; bk = 64; }
        if (free_tile && variant == 3) { bm = 128; bn = 256; bk = 64; }
        if (bm <= 0 || bn <= 0) return 0;
        tl::GemmPlan plan;
        // grouped: every expert may add a ragged m-tile and the number of experts is not known here; with the most
        // the library accepts the K ranges are cut over every SM, which is the largest scratch a launch can ask for
        const int64_t mt = grouped ? M / bm + tl::kMaxExperts : tl::ceil_div(M, bm);
        if (tl::make_plan(M, mt * tl::ceil_div(N, bn), N, K, variant > 1 ? bm : cta_m, variant > 1 ? bn : cta_n,
                          variant > 1 ? bk : cta_k, grouped, &plan, false, false, pair_sized)) {
            if (variant > 1) continue;
            return 0;
        }
        if (plan.ws_bytes > need) need = plan.ws_bytes;
    }
    return need;
}

int tl_gemm_plan(int64_t M, int64_t N, int64_t K, int64_t G, int block_rows, int block_cols, int cta_m, int cta_n,
                 int cta_k, int E, int flavour, tl_gemm_plan_info* out) {
    tl::ApiLock lock;
    if (!out || E < 0 || flavour < 0 || flavour > 2 || M <= 0) return TL_ERR_INVALID_ARG;
    if (flavour == 2 && cta_k != 0 && cta_k != 128 && cta_k != 256) return TL_ERR_UNSUPPORTED;
    // Any non-null pointer stands in for the grouped form's offsets: plan-only mode reads none of them.
    static const int32_t grouped_marker = 0;
    return tl::gemm_launch(nullptr, nullptr, nullptr, E > 0 ? &grouped_marker : nullptr, E > 0 ? E : 1, M, M, N, K, G,
                           block_rows, block_cols, cta_m, cta_n, flavour == 2 ? cta_k / 2 : cta_k, nullptr, nullptr,
                           flavour != 0, flavour == 2 ? 1 : 2, nullptr, nullptr, out);
}

int tl_gemm_last_plan(tl_gemm_plan_info* out) {
    if (!out) return TL_ERR_INVALID_ARG;
    *out = tl::last_plan();
    return TL_OK;
}

}  // extern "C"

// ------------------------------------------------------------ host-buffer form
namespace tl {
static size_t align256(size_t x) { return (x + 255) & ~size_t(255); }
}

extern "C" {

size_t tl_gemm_host_scratch_bytes(int64_t M, int64_t N, int64_t K) {
    tl::ApiLock lock;
    if (M < 0 || N <= 0 || K <= 0) return 0;
    return tl::align256(size_t(M) * K * 2) + 2 * tl::align256(size_t(K) * N * 2) + tl::align256(size_t(M) * N * 4);
}

int tl_gemm_host(const void* h_A, const void* h_B_rowmajor, float* h_C, int64_t M, int64_t N, int64_t K, int64_t G,
                 int block_rows, int block_cols, int cta_m, int cta_n, int cta_k, void* d_scratch,
                 size_t scratch_bytes, void* cuda_stream) {
    tl::ApiLock lock;
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
    tl::ApiLock lock;
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

