// Read-amplification counter (Sections 1, 2.5 and 6.5 of the paper).
//
// For the GEMM's tile schedule it counts, per weight-tile load, the distinct
// G-byte blocks that hold bytes of the cta_k x cta_n rectangle.  One warp owns
// one column of CTA tiles (one n-tile) for a group of eight K iterations: its
// lanes split the lines of every load, warp shuffles pass interval ends between
// neighbouring lines and add the pieces up.  The count is exact for any sizes:
//   tile-major  a rectangle of the matrix covers a rectangle of the block grid;
//   row-major   row r of the rectangle covers the block interval [lo_r, hi_r];
//               both ends never decrease with r, so the union grows by
//               max(0, hi_r - max(lo_r, hi_{r-1} + 1) + 1) per row;
//   col-major   the same with the roles of rows and columns exchanged.
#include "tl_common.cuh"

#include <algorithm>
#include <cmath>
#include <vector>

#include <cstdlib>
#include <cstring>

namespace tl {

struct ReadAmpParams {
    int64_t N, K;
    int64_t BN, BK;
    int64_t G, s;
    int64_t br, bc;
    int layout;
    int64_t n_tiles, k_iters;
    int64_t m_tiles;                 // multiplier for totals / replication for per-tile output
    unsigned long long* d_acc;       // [fetched, used, requests, ticket] totals (may be null); zero between launches
    unsigned long long* h_out;       // mapped pinned host memory: the last warp publishes the totals here
    unsigned long long total_ctas;
    int64_t wave_tiles;              // > 0: count per wave of this many co-resident CTA tiles (blocks shared)
    int64_t sched_m_tiles, sched_n_tiles;   // wave mode: the tile grid (tiles numbered n-tile major, m-tile minor)
    int64_t iters_per_warp;          // K iterations one warp covers
    unsigned long long* d_fetched;   // per CTA tile (may be null)
    unsigned long long* d_used;
};

__device__ __forceinline__ unsigned long long warp_sum(unsigned long long v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    return v;
}

constexpr int kItersPerWarp = 8;     // row-/column-major: K iterations one warp covers (tile-major: all of them)

// One CTA's share of one counter configuration; cta is the CTA's index within that configuration.
__device__ __forceinline__ void read_amp_body(const ReadAmpParams& p, unsigned cta) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = (cta * int64_t(blockDim.x) + threadIdx.x) >> 5;
    __shared__ unsigned long long cta_blocks[4], cta_used[4];
    const int64_t k_chunks = (p.k_iters + p.iters_per_warp - 1) / p.iters_per_warp;
    const bool has_work = warp < p.n_tiles * k_chunks;
    const int64_t tn = has_work ? warp / k_chunks : 0, kc = has_work ? warp % k_chunks : 0;
    int64_t n0 = tn * p.BN;
    int64_t n1 = n0 + p.BN < p.N ? n0 + p.BN : p.N;
    if (p.wave_tiles > 0) {
        // Wave tn holds CTA tiles [tn*P, (tn+1)*P): the n-tiles t/m_tiles of its first and last tile and all
        // between them.  Their rectangles side by side are one rectangle, whose blocks are counted once.
        const int64_t total = p.sched_m_tiles * p.sched_n_tiles;
        const int64_t t0 = tn * p.wave_tiles;
        const int64_t t1 = (t0 + p.wave_tiles < total ? t0 + p.wave_tiles : total) - 1;
        n0 = (t0 / p.sched_m_tiles) * p.BN;
        n1 = (t1 / p.sched_m_tiles + 1) * p.BN;
        if (n1 > p.N) n1 = p.N;
    }
    const int64_t it0 = kc * p.iters_per_warp;
    const int64_t it1 = !has_work ? it0 : (it0 + p.iters_per_warp < p.k_iters ? it0 + p.iters_per_warp : p.k_iters);

    unsigned long long blocks = 0;   // this lane's share of the distinct blocks of these tile loads
    if (p.layout == TL_LAYOUT_TILE_MAJOR) {
        const unsigned long long across = (unsigned long long)((n1 - 1) / p.bc - n0 / p.bc + 1);
        for (int64_t it = it0 + lane; it < it1; it += 32) {
            const int64_t k0 = it * p.BK;
            const int64_t k1 = k0 + p.BK < p.K ? k0 + p.BK : p.K;
            blocks += (unsigned long long)((k1 - 1) / p.br - k0 / p.br + 1) * across;
        }
    } else {
        // Lines of the rectangle: its rows (row-major, pitch N*s) or its columns (col-major, pitch K*s).
        const bool rowm = p.layout == TL_LAYOUT_ROW_MAJOR;
        const int64_t pitch = (rowm ? p.N : p.K) * p.s;
        for (int64_t it = it0; it < it1; ++it) {
            const int64_t k0 = it * p.BK;
            const int64_t k1 = k0 + p.BK < p.K ? k0 + p.BK : p.K;
            const int64_t line0 = rowm ? k0 : n0, line1 = rowm ? k1 : n1;   // lines of this load
            const int64_t seg0 = (rowm ? n0 : k0) * p.s;                     // first byte inside a line
            const int64_t seg1 = (rowm ? n1 : k1) * p.s - 1;                 // last byte inside a line
            for (int64_t base = line0; base < line1; base += 32) {
                const int64_t l = base + lane;
                const bool active = l < line1;
                const int64_t lo = active ? (l * pitch + seg0) / p.G : 0;
                const int64_t hi = active ? (l * pitch + seg1) / p.G : 0;
                // last block of the previous line: from the lane below, or computed by lane 0
                int64_t hi_prev = __shfl_up_sync(0xffffffffu, hi, 1);
                if (lane == 0 && l > line0) hi_prev = ((l - 1) * pitch + seg1) / p.G;
                int64_t first_new = lo;
                if (l > line0 && hi_prev + 1 > first_new) first_new = hi_prev + 1;
                if (active && hi >= first_new) blocks += (unsigned long long)(hi - first_new + 1);
            }
        }
    }
    blocks = warp_sum(blocks);
    // Everything above is arithmetic on the launch parameters.  The kernel is launched with programmatic stream
    // serialisation: only from here on does it touch memory (the accumulators shared with the previous counter
    // launch, the per-tile arrays the host has just cleared), so only here does it wait for its predecessor.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const unsigned long long fetched = blocks * (unsigned long long)p.G;
    const int64_t k_lo = it0 * p.BK, k_hi = it1 * p.BK < p.K ? it1 * p.BK : p.K;
    const unsigned long long used = has_work ? (unsigned long long)((k_hi - k_lo) * (n1 - n0) * p.s) : 0ull;
    if (lane == 0) {
        cta_blocks[threadIdx.x >> 5] = blocks;
        cta_used[threadIdx.x >> 5] = used;
        if (has_work && p.d_fetched && p.d_used) {      // zeroed by the host before the launch
            for (int64_t tm = 0; tm < p.m_tiles; ++tm) {
                atomicAdd(&p.d_fetched[tm * p.n_tiles + tn], fetched);
                atomicAdd(&p.d_used[tm * p.n_tiles + tn], used);
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0 && p.d_acc) {
        unsigned long long b = 0, u = 0;
        for (int w = 0; w < 4; ++w) { b += cta_blocks[w]; u += cta_used[w]; }
        atomicAdd(&p.d_acc[0], b * (unsigned long long)p.G * (unsigned long long)p.m_tiles);
        atomicAdd(&p.d_acc[1], u * (unsigned long long)p.m_tiles);
        atomicAdd(&p.d_acc[2], b * (unsigned long long)p.m_tiles);
        // The CTA that takes the last ticket publishes the totals to the host and leaves the
        // accumulators at zero for the next launch: no memset before and no copy after the kernel.
        __threadfence();
        if (atomicAdd(&p.d_acc[3], 1ull) == p.total_ctas - 1) {
            __threadfence();
            for (int i = 0; i < 3; ++i) p.h_out[i] = atomicExch(&p.d_acc[i], 0ull);
            p.d_acc[3] = 0;
            __threadfence_system();
        }
    }
}

__global__ void __launch_bounds__(128) read_amp_kernel(const ReadAmpParams p) {
    if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    read_amp_body(p, blockIdx.x);
}

// Up to kBatchMax configurations in one launch: CTAs [cta_begin[i], cta_begin[i+1]) work on configuration i, each
// configuration with its own accumulators and output slot.
constexpr int kBatchMax = 16;
struct ReadAmpBatch {
    int n;
    unsigned cta_begin[kBatchMax + 1];
    ReadAmpParams p[kBatchMax];
};

__global__ void __launch_bounds__(128) read_amp_batch_kernel(const __grid_constant__ ReadAmpBatch b) {
    if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    int i = 0;
    while (i + 1 < b.n && blockIdx.x >= b.cta_begin[i + 1]) ++i;
    read_amp_body(b.p[i], blockIdx.x - b.cta_begin[i]);
}

static int read_amp_validate(int64_t N, int64_t K, int cta_m, int cta_n, int cta_k, int layout, int64_t G, int br,
                             int bc, int s) {
    if (N <= 0 || K <= 0 || cta_m <= 0 || cta_n <= 0 || cta_k <= 0 || G <= 0) return TL_ERR_INVALID_ARG;
    if (s != 1 && s != 2 && s != 4) return TL_ERR_INVALID_ARG;
    if (layout == TL_LAYOUT_TILE_MAJOR) {
        if (br <= 0 || bc <= 0 || int64_t(br) * bc * s != G) return TL_ERR_INVALID_ARG;
        if (K % br != 0 || N % bc != 0) return TL_ERR_INVALID_ARG;
    } else if (layout == TL_LAYOUT_TILE_MAJOR_K) {
        if (br <= 0 || bc <= 0 || int64_t(br) * bc * s != G) return TL_ERR_INVALID_ARG;
        if (N % br != 0 || K % bc != 0) return TL_ERR_INVALID_ARG;
    } else if (layout != TL_LAYOUT_ROW_MAJOR && layout != TL_LAYOUT_COL_MAJOR) {
        return TL_ERR_INVALID_ARG;
    }
    if (G % s != 0) return TL_ERR_INVALID_ARG;   // an element never straddles two blocks
    return TL_OK;
}

// Fills the kernel parameters of one configuration; *grid = CTAs it needs (0: nothing to count).
static int read_amp_fill(int64_t m_tiles, int64_t N, int64_t K, int cta_n, int cta_k, int layout, int64_t G,
                         int br, int bc, int s, unsigned long long* d_acc, unsigned long long* d_fetched,
                         unsigned long long* d_used, int64_t wave_tiles, unsigned long long* totals_out,
                         ReadAmpParams* out, int64_t* grid_out) {
    ReadAmpParams& p = *out;
    p.N = N; p.K = K; p.BN = cta_n; p.BK = cta_k; p.G = G; p.s = s;
    p.br = br > 0 ? br : 1; p.bc = bc > 0 ? bc : 1; p.layout = layout;
    if (layout == TL_LAYOUT_TILE_MAJOR_K) {
        // Either flavour maps memory tiles one to one onto G-byte blocks, so a rectangle of the matrix covers a
        // rectangle of the tile grid: only the tile's extent along K (here block_cols) and along N (block_rows)
        // matter to the count.
        p.br = bc; p.bc = br;
        p.layout = TL_LAYOUT_TILE_MAJOR;
    }
    p.n_tiles = ceil_div(N, cta_n);
    p.k_iters = ceil_div(K, cta_k);
    p.m_tiles = m_tiles;
    p.wave_tiles = wave_tiles;
    p.sched_m_tiles = m_tiles;
    p.sched_n_tiles = p.n_tiles;
    if (wave_tiles > 0) {
        p.n_tiles = ceil_div(m_tiles * p.n_tiles, wave_tiles);      // one "column" of work per wave
        p.m_tiles = 1;
        if (d_fetched || d_used) return TL_ERR_UNSUPPORTED;
    }
    p.d_acc = d_acc; p.d_fetched = d_fetched; p.d_used = d_used;
    p.h_out = d_acc ? (totals_out ? totals_out : dev().ctl.h_acc_dev) : nullptr;
    p.iters_per_warp = p.layout == TL_LAYOUT_TILE_MAJOR ? p.k_iters : kItersPerWarp;
    *grid_out = 0;
    if (m_tiles == 0) return TL_OK;
    const int warps_per_cta = 4;
    const int64_t grid = ceil_div(p.n_tiles * ceil_div(p.k_iters, p.iters_per_warp), warps_per_cta);
    p.total_ctas = (unsigned long long)grid;
    *grid_out = grid;
    return TL_OK;
}

static int read_amp_launch(int64_t m_tiles, int64_t N, int64_t K, int cta_n, int cta_k, int layout, int64_t G,
                           int br, int bc, int s, unsigned long long* d_acc, unsigned long long* d_fetched,
                           unsigned long long* d_used, cudaStream_t stream, int64_t wave_tiles = 0,
                           unsigned long long* totals_out = nullptr) {
    ReadAmpParams p;
    int64_t grid = 0;
    if (int rc = read_amp_fill(m_tiles, N, K, cta_n, cta_k, layout, G, br, bc, s, d_acc, d_fetched, d_used, wave_tiles,
                               totals_out, &p, &grid))
        return rc;
    if (grid == 0) return TL_OK;
    const int warps_per_cta = 4;
    if (d_fetched && d_used) {
        const size_t bytes = size_t(m_tiles) * p.n_tiles * sizeof(unsigned long long);
        if (int rc = check_cuda(cudaMemsetAsync(d_fetched, 0, bytes, stream))) return rc;
        if (int rc = check_cuda(cudaMemsetAsync(d_used, 0, bytes, stream))) return rc;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(grid));
    cfg.blockDim = dim3(warps_per_cta * 32);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = opt(TL_OPT_PDL) != 0 ? 1 : 0;           // measurement switch
    return check_cuda(cudaLaunchKernelEx(&cfg, read_amp_kernel, p));
}

static int read_amp_totals(int64_t m_tiles, int64_t N, int64_t K, int cta_n, int cta_k, int layout, int64_t G,
                           int br, int bc, int s, uint64_t* fetched, uint64_t* used, uint64_t* requests,
                           int64_t wave_tiles = 0) {
    if (!fetched || !used) return TL_ERR_INVALID_ARG;
    if (int rc = ensure_control()) return rc;
    Control& ctl = dev().ctl;
    const cudaStream_t stream = tls().stream;
    if (m_tiles == 0) {
        *fetched = *used = 0;
        if (requests) *requests = 0;
        return TL_OK;
    }
    if (int rc = read_amp_launch(m_tiles, N, K, cta_n, cta_k, layout, G, br, bc, s, ctl.d_acc, nullptr, nullptr,
                                 stream, wave_tiles))
        return rc;
    // the kernel's last warp wrote the totals into mapped pinned memory; the only wait is this one
    volatile unsigned long long* h = ctl.h_acc;
    if (int rc = check_cuda(cudaStreamSynchronize(stream))) return rc;
    *fetched = h[0];
    *used = h[1];
    if (requests) *requests = h[2];
    return TL_OK;
}

}  // namespace tl

extern "C" {

int tl_read_amp(int64_t M, int64_t N, int64_t K, int cta_m, int cta_n, int cta_k, int layout, int64_t G,
                int block_rows, int block_cols, int elem_bytes, uint64_t* bytes_fetched, uint64_t* bytes_used,
                uint64_t* requests) {
    tl::ApiLock lock;
    if (M < 0) return TL_ERR_INVALID_ARG;
    if (int rc = tl::read_amp_validate(N, K, cta_m, cta_n, cta_k, layout, G, block_rows, block_cols, elem_bytes))
        return rc;
    return tl::read_amp_totals(tl::ceil_div(M, cta_m), N, K, cta_n, cta_k, layout, G, block_rows, block_cols,
                               elem_bytes, bytes_fetched, bytes_used, requests);
}

int tl_read_amp_shared(int64_t M, int64_t N, int64_t K, int cta_m, int cta_n, int cta_k, int64_t wave_ctas, int layout,
                       int64_t G, int block_rows, int block_cols, int elem_bytes, uint64_t* bytes_fetched,
                       uint64_t* bytes_needed, uint64_t* requests) {
    tl::ApiLock lock;
    if (M < 0 || wave_ctas <= 0) return TL_ERR_INVALID_ARG;
    if (int rc = tl::read_amp_validate(N, K, cta_m, cta_n, cta_k, layout, G, block_rows, block_cols, elem_bytes))
        return rc;
    return tl::read_amp_totals(tl::ceil_div(M, cta_m), N, K, cta_n, cta_k, layout, G, block_rows, block_cols,
                               elem_bytes, bytes_fetched, bytes_needed, requests, wave_ctas);
}

int64_t tl_prefetch_degree(double bandwidth_bytes_per_s, double latency_s, int64_t G, int64_t n_sm, int64_t ctas_per_sm,
                           int64_t requests_per_tile, int64_t K, int64_t cta_k, double collision_factor) {
    if (G <= 0 || n_sm <= 0 || ctas_per_sm <= 0 || requests_per_tile <= 0 || K <= 0 || cta_k <= 0) return -1;
    if (!(bandwidth_bytes_per_s >= 0.0) || !(latency_s >= 0.0) || !(collision_factor >= 0.0)) return -1;
    // requests that must be in flight to keep the bus busy, over the requests one wave issues per K iteration
    const long double in_flight = (long double)bandwidth_bytes_per_s * latency_s / (long double)G * collision_factor;
    const long double per_wave = (long double)n_sm * (long double)ctas_per_sm * (long double)requests_per_tile;
    const long double q = in_flight / per_wave;
    const int64_t cap = K / cta_k;
    if (q >= (long double)cap) return cap;
    return (int64_t)q;
}

int tl_tile_arrival_latency(const double* h_latencies, int64_t count, int64_t requests, double threshold,
                            double* first_arrival, double* last_arrival, double* p_late) {
    if (!h_latencies || count <= 0 || requests <= 0 || !first_arrival || !last_arrival) return TL_ERR_INVALID_ARG;
    std::vector<double> x(h_latencies, h_latencies + count);
    for (double v : x)
        if (!(v == v)) return TL_ERR_INVALID_ARG;          // NaN
    std::sort(x.begin(), x.end());
    // Summation by parts over the sorted sample: the largest of n draws exceeds x_(i) with probability
    // 1 - (i/N)^n, the smallest with probability ((N - i)/N)^n, so
    //   E[max] = x_(N) - sum_i (x_(i+1) - x_(i)) (i/N)^n,    E[min] = x_(1) + sum_i (x_(i+1) - x_(i)) ((N - i)/N)^n.
    const double N = double(count), n = double(requests);
    double gap_max = 0.0, gap_min = 0.0, c_max = 0.0, c_min = 0.0;      // Kahan sums
    int64_t below = 0;
    for (int64_t i = 1; i < count; ++i) {
        const double step = x[size_t(i)] - x[size_t(i) - 1];
        if (step != 0.0) {
            const double a = step * std::pow(double(i) / N, n) - c_max;
            const double t = gap_max + a;
            c_max = (t - gap_max) - a;
            gap_max = t;
            const double b = step * std::pow(double(count - i) / N, n) - c_min;
            const double u = gap_min + b;
            c_min = (u - gap_min) - b;
            gap_min = u;
        }
    }
    for (int64_t i = 0; i < count; ++i)
        if (x[size_t(i)] <= threshold) ++below;
    *last_arrival = x.back() - gap_max;
    *first_arrival = x.front() + gap_min;
    if (p_late) *p_late = 1.0 - std::pow(double(below) / N, n);
    return TL_OK;
}

int tl_read_amp_async(int64_t M, int64_t N, int64_t K, int cta_m, int cta_n, int cta_k, int layout, int64_t G,
                      int block_rows, int block_cols, int elem_bytes, uint64_t* d_totals, void* cuda_stream) {
    tl::ApiLock lock;
    if (M < 0 || !d_totals) return TL_ERR_INVALID_ARG;
    if (int rc = tl::read_amp_validate(N, K, cta_m, cta_n, cta_k, layout, G, block_rows, block_cols, elem_bytes))
        return rc;
    if (int rc = tl::ensure_control()) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (M == 0) return tl::check_cuda(cudaMemsetAsync(d_totals, 0, 3 * sizeof(uint64_t), st));
    // The accumulators are shared by all launches on the device: launches must be ordered by one stream (they
    // are between tl_read_amp* calls, which all use the stream they are given or the tl_set_stream() stream).
    return tl::read_amp_launch(tl::ceil_div(M, cta_m), N, K, cta_n, cta_k, layout, G, block_rows, block_cols, elem_bytes,
                               tl::dev().ctl.d_acc, nullptr, nullptr, st, 0,
                               reinterpret_cast<unsigned long long*>(d_totals));
}

int tl_read_amp_batch(const tl_read_amp_cfg* h_cfgs, int n, uint64_t* d_totals, void* cuda_stream) {
    tl::ApiLock lock;
    if (n < 0 || n > tl::kBatchMax || (n > 0 && (!h_cfgs || !d_totals))) return TL_ERR_INVALID_ARG;
    if (n == 0) return TL_OK;
    if (int rc = tl::ensure_control()) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    tl::ReadAmpBatch b;
    memset(&b, 0, sizeof b);
    unsigned ctas = 0;
    for (int i = 0; i < n; ++i) {
        const tl_read_amp_cfg& c = h_cfgs[i];
        if (c.M < 0) return TL_ERR_INVALID_ARG;
        if (int rc = tl::read_amp_validate(c.N, c.K, c.cta_m, c.cta_n, c.cta_k, c.layout, c.G, c.block_rows, c.block_cols,
                                           c.elem_bytes))
            return rc;
        int64_t grid = 0;
        // configuration i accumulates in its own four words of the control block and publishes to its own slot
        if (int rc = tl::read_amp_fill(tl::ceil_div(c.M, c.cta_m), c.N, c.K, c.cta_n, c.cta_k, c.layout, c.G, c.block_rows,
                                       c.block_cols, c.elem_bytes, tl::dev().ctl.d_acc + 4 * (i + 1), nullptr, nullptr, 0,
                                       reinterpret_cast<unsigned long long*>(d_totals) + 3 * i, &b.p[b.n], &grid))
            return rc;
        if (grid == 0) {                                    // M == 0: nothing is launched for it, its totals are zero
            if (int rc = tl::check_cuda(cudaMemsetAsync(d_totals + 3 * i, 0, 3 * sizeof(uint64_t), st))) return rc;
            continue;
        }
        if (grid > (1u << 30) || ctas + grid > (1u << 30)) return TL_ERR_UNSUPPORTED;
        b.cta_begin[b.n] = ctas;
        ctas += unsigned(grid);
        ++b.n;
        b.cta_begin[b.n] = ctas;
    }
    if (b.n == 0) return TL_OK;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ctas);
    cfg.blockDim = dim3(128);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return tl::check_cuda(cudaLaunchKernelEx(&cfg, tl::read_amp_batch_kernel, b));
}

int tl_read_amp_grouped(const int32_t* h_offsets, int E, int64_t N, int64_t K, int cta_m, int cta_n, int cta_k,
                        int layout, int64_t G, int block_rows, int block_cols, int elem_bytes,
                        uint64_t* bytes_fetched, uint64_t* bytes_used, uint64_t* requests) {
    tl::ApiLock lock;
    if (!h_offsets || E < 0) return TL_ERR_INVALID_ARG;
    if (int rc = tl::read_amp_validate(N, K, cta_m, cta_n, cta_k, layout, G, block_rows, block_cols, elem_bytes))
        return rc;
    // Every expert's weight has the same shape and its own G-aligned buffer, so each of its
    // m-tiles issues the loads of one tile column set: the sum over experts is a sum of m-tiles.
    int64_t m_tiles = 0;
    for (int e = 0; e < E; ++e) {
        const int64_t rows = int64_t(h_offsets[e + 1]) - int64_t(h_offsets[e]);
        if (rows < 0) return TL_ERR_INVALID_ARG;
        m_tiles += tl::ceil_div(rows, cta_m);
    }
    return tl::read_amp_totals(m_tiles, N, K, cta_n, cta_k, layout, G, block_rows, block_cols, elem_bytes,
                               bytes_fetched, bytes_used, requests);
}

int tl_read_amp_per_cta(int64_t M, int64_t N, int64_t K, int cta_m, int cta_n, int cta_k, int layout, int64_t G,
                        int block_rows, int block_cols, int elem_bytes, uint64_t* d_fetched, uint64_t* d_used,
                        void* cuda_stream) {
    tl::ApiLock lock;
    if (M < 0) return TL_ERR_INVALID_ARG;
    if (int rc = tl::read_amp_validate(N, K, cta_m, cta_n, cta_k, layout, G, block_rows, block_cols, elem_bytes))
        return rc;
    if (M == 0) return TL_OK;
    if (!d_fetched || !d_used) return TL_ERR_INVALID_ARG;
    return tl::read_amp_launch(tl::ceil_div(M, cta_m), N, K, cta_n, cta_k, layout, G, block_rows, block_cols,
                               elem_bytes, nullptr, reinterpret_cast<unsigned long long*>(d_fetched),
                               reinterpret_cast<unsigned long long*>(d_used), static_cast<cudaStream_t>(cuda_stream));
}

}  // extern "C"
