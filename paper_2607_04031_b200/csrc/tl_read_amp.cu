// Read-amplification counter (Sections 1, 2.5 and 6.5 of the paper).
//
// For the GEMM's tile schedule it counts, per weight-tile load, the distinct
// G-byte blocks that hold bytes of the cta_k x cta_n rectangle.  One warp owns
// one column of CTA tiles (one n-tile): its lanes split the work of every load
// and warp shuffles add the pieces up.  The count is exact for any sizes:
//   tile-major  a rectangle of the matrix covers a rectangle of the block grid;
//   row-major   row r of the rectangle covers the block interval [lo_r, hi_r];
//               both ends never decrease with r, so the union grows by
//               max(0, hi_r - max(lo_r, hi_{r-1} + 1) + 1) per row;
//   col-major   the same with the roles of rows and columns exchanged.
#include "tl_common.cuh"

namespace tl {

struct ReadAmpParams {
    int64_t N, K;
    int64_t BN, BK;
    int64_t G, s;
    int64_t br, bc;
    int layout;
    int64_t n_tiles, k_iters;
    int64_t m_tiles;                 // multiplier for totals / replication for per-tile output
    unsigned long long* d_acc;       // [fetched, used, requests] totals (may be null)
    unsigned long long* d_fetched;   // per CTA tile (may be null)
    unsigned long long* d_used;
};

__device__ __forceinline__ unsigned long long warp_sum(unsigned long long v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    return v;
}

__global__ void __launch_bounds__(128) read_amp_kernel(const ReadAmpParams p) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = (blockIdx.x * int64_t(blockDim.x) + threadIdx.x) >> 5;
    if (warp >= p.n_tiles) return;
    const int64_t n0 = warp * p.BN;
    const int64_t n1 = n0 + p.BN < p.N ? n0 + p.BN : p.N;

    unsigned long long blocks = 0;   // this lane's share of the distinct blocks, all K iterations
    if (p.layout == TL_LAYOUT_TILE_MAJOR) {
        const unsigned long long across = (unsigned long long)((n1 - 1) / p.bc - n0 / p.bc + 1);
        for (int64_t it = lane; it < p.k_iters; it += 32) {
            const int64_t k0 = it * p.BK;
            const int64_t k1 = k0 + p.BK < p.K ? k0 + p.BK : p.K;
            blocks += (unsigned long long)((k1 - 1) / p.br - k0 / p.br + 1) * across;
        }
    } else {
        // Lines of the rectangle: its rows (row-major, pitch N*s) or its columns (col-major, pitch K*s).
        const bool rowm = p.layout == TL_LAYOUT_ROW_MAJOR;
        const int64_t pitch = (rowm ? p.N : p.K) * p.s;
        for (int64_t it = 0; it < p.k_iters; ++it) {
            const int64_t k0 = it * p.BK;
            const int64_t k1 = k0 + p.BK < p.K ? k0 + p.BK : p.K;
            const int64_t line0 = rowm ? k0 : n0, line1 = rowm ? k1 : n1;   // lines of this load
            const int64_t seg0 = (rowm ? n0 : k0) * p.s;                     // first byte inside a line
            const int64_t seg1 = (rowm ? n1 : k1) * p.s - 1;                 // last byte inside a line
            for (int64_t l = line0 + lane; l < line1; l += 32) {
                const int64_t lo = (l * pitch + seg0) / p.G;
                const int64_t hi = (l * pitch + seg1) / p.G;
                int64_t first_new = lo;
                if (l > line0) {
                    const int64_t hi_prev = ((l - 1) * pitch + seg1) / p.G;
                    if (hi_prev + 1 > first_new) first_new = hi_prev + 1;
                }
                if (hi >= first_new) blocks += (unsigned long long)(hi - first_new + 1);
            }
        }
    }
    blocks = warp_sum(blocks);
    if (lane != 0) return;
    const unsigned long long fetched = blocks * (unsigned long long)p.G;
    const unsigned long long used = (unsigned long long)(p.K * (n1 - n0) * p.s);
    if (p.d_acc) {
        atomicAdd(&p.d_acc[0], fetched * (unsigned long long)p.m_tiles);
        atomicAdd(&p.d_acc[1], used * (unsigned long long)p.m_tiles);
        atomicAdd(&p.d_acc[2], blocks * (unsigned long long)p.m_tiles);
    }
    if (p.d_fetched && p.d_used) {
        for (int64_t tm = 0; tm < p.m_tiles; ++tm) {
            p.d_fetched[tm * p.n_tiles + warp] = fetched;
            p.d_used[tm * p.n_tiles + warp] = used;
        }
    }
}

static int read_amp_validate(int64_t N, int64_t K, int cta_m, int cta_n, int cta_k, int layout, int64_t G, int br,
                             int bc, int s) {
    if (N <= 0 || K <= 0 || cta_m <= 0 || cta_n <= 0 || cta_k <= 0 || G <= 0) return TL_ERR_INVALID_ARG;
    if (s != 1 && s != 2 && s != 4) return TL_ERR_INVALID_ARG;
    if (layout == TL_LAYOUT_TILE_MAJOR) {
        if (br <= 0 || bc <= 0 || int64_t(br) * bc * s != G) return TL_ERR_INVALID_ARG;
        if (K % br != 0 || N % bc != 0) return TL_ERR_INVALID_ARG;
    } else if (layout != TL_LAYOUT_ROW_MAJOR && layout != TL_LAYOUT_COL_MAJOR) {
        return TL_ERR_INVALID_ARG;
    }
    if (G % s != 0) return TL_ERR_INVALID_ARG;   // an element never straddles two blocks
    return TL_OK;
}

static int read_amp_launch(int64_t m_tiles, int64_t N, int64_t K, int cta_n, int cta_k, int layout, int64_t G,
                           int br, int bc, int s, unsigned long long* d_acc, unsigned long long* d_fetched,
                           unsigned long long* d_used, cudaStream_t stream) {
    ReadAmpParams p;
    p.N = N; p.K = K; p.BN = cta_n; p.BK = cta_k; p.G = G; p.s = s;
    p.br = br > 0 ? br : 1; p.bc = bc > 0 ? bc : 1; p.layout = layout;
    p.n_tiles = ceil_div(N, cta_n);
    p.k_iters = ceil_div(K, cta_k);
    p.m_tiles = m_tiles;
    p.d_acc = d_acc; p.d_fetched = d_fetched; p.d_used = d_used;
    if (m_tiles == 0) return TL_OK;
    const int warps_per_cta = 4;
    const int64_t grid = ceil_div(p.n_tiles, warps_per_cta);
    read_amp_kernel<<<unsigned(grid), warps_per_cta * 32, 0, stream>>>(p);
    return check_cuda(cudaGetLastError());
}

static int read_amp_totals(int64_t m_tiles, int64_t N, int64_t K, int cta_n, int cta_k, int layout, int64_t G,
                           int br, int bc, int s, uint64_t* fetched, uint64_t* used, uint64_t* requests) {
    if (!fetched || !used) return TL_ERR_INVALID_ARG;
    if (int rc = ensure_control()) return rc;
    State& st = state();
    if (int rc = check_cuda(cudaMemsetAsync(st.ctl.d_acc, 0, 3 * sizeof(unsigned long long), st.stream))) return rc;
    if (int rc = read_amp_launch(m_tiles, N, K, cta_n, cta_k, layout, G, br, bc, s, st.ctl.d_acc, nullptr, nullptr,
                                 st.stream))
        return rc;
    unsigned long long h[3] = {0, 0, 0};
    if (int rc = check_cuda(cudaMemcpyAsync(h, st.ctl.d_acc, sizeof h, cudaMemcpyDeviceToHost, st.stream))) return rc;
    if (int rc = check_cuda(cudaStreamSynchronize(st.stream))) return rc;
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
    if (M < 0) return TL_ERR_INVALID_ARG;
    if (int rc = tl::read_amp_validate(N, K, cta_m, cta_n, cta_k, layout, G, block_rows, block_cols, elem_bytes))
        return rc;
    return tl::read_amp_totals(tl::ceil_div(M, cta_m), N, K, cta_n, cta_k, layout, G, block_rows, block_cols,
                               elem_bytes, bytes_fetched, bytes_used, requests);
}

int tl_read_amp_grouped(const int32_t* h_offsets, int E, int64_t N, int64_t K, int cta_m, int cta_n, int cta_k,
                        int layout, int64_t G, int block_rows, int block_cols, int elem_bytes,
                        uint64_t* bytes_fetched, uint64_t* bytes_used, uint64_t* requests) {
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
