// Row-major <-> tile-major relayout (Section 3; Eq. 1 and Eq. 2 in the N-contiguous flavour; applied to the [N][K]
// array it produces the K-contiguous flavour of Eq. 2 as printed).
//
// Bandwidth-bound: every byte is read once and written once.  Three kernels:
//   relayout_tma_kernel   the copy engine does the permutation: a tensor-map box of the row-major side holds whole
//                         memory tiles, which are contiguous runs of the tile-major side and move as untiled bulk
//                         copies; one thread per CTA drives a ring of three 32 KB buffers (block rows 32 B .. 1 KB);
//   relayout_kernel<P>    32 KB tiles through shared memory with 16-byte loads and stores on both sides: the
//                         row-major side is walked in row order, the tile-major side in block order; when a block
//                         row is shorter than 16 bytes the vectors of the tile-major side are assembled from
//                         several shared-memory rows, one piece-wide access per row;
//   element-wise          for unaligned pointers or pitches.
// relayout_tma_batch_kernel is relayout_tma_kernel over the step lists of several matrices in one launch.
#include "tl_common.cuh"

#include <cstdlib>
#include <cstring>

namespace tl {

constexpr int kRelayoutThreads = 256;
constexpr int kTileBytes = 32768;                       // shared-memory tile (payload)
constexpr int kChunksPerThread = kTileBytes / 16 / kRelayoutThreads;   // 8
constexpr int kRowPad = 16;                             // bytes of padding per shared-memory row

struct RelayoutParams {
    const uint8_t* src;
    uint8_t* dst;
    int64_t rows;
    int64_t pitch;          // cols * elem_bytes
    int64_t blocks_per_row; // cols / block_cols
    int run_log2;           // log2(block_cols * elem_bytes): bytes of one block row
    int br_log2;            // log2(block_rows)
    int tile_cols_log2;     // log2(bytes of a matrix row covered by one tile)
    int tile_rows_log2;     // log2(rows covered by one tile)
    int64_t tiles_x;        // tiles along a row
    int64_t tiles_total;
    int to_tile_major;
};

__device__ __forceinline__ uint4 ld_stream(const uint8_t* p) {
    return __ldcs(reinterpret_cast<const uint4*>(p));
}
__device__ __forceinline__ void st_stream(uint8_t* p, uint4 v) {
    __stcs(reinterpret_cast<uint4*>(p), v);
}

// Byte offset in the tile-major buffer of byte column `cb` of matrix row `r` (Eq. 1 + Eq. 2,
// written on bytes: a block row is `run` contiguous bytes; shifts and masks only).
__device__ __forceinline__ int64_t tile_major_byte(const RelayoutParams& p, int64_t r, int64_t cb) {
    int64_t Tr = r >> p.br_log2, rp = r & ((int64_t(1) << p.br_log2) - 1);
    int64_t Tc = cb >> p.run_log2, cp = cb & ((int64_t(1) << p.run_log2) - 1);
    return ((((Tr * p.blocks_per_row + Tc) << p.br_log2) + rp) << p.run_log2) + cp;
}

template <int kBytes> struct PieceType { using type = uint4; };
template <> struct PieceType<8> { using type = uint2; };
template <> struct PieceType<4> { using type = uint32_t; };
template <> struct PieceType<2> { using type = uint16_t; };
template <> struct PieceType<1> { using type = uint8_t; };

// kPiece = min(16, bytes of one block row): granularity at which the tile-major side is contiguous.
template <int kPiece>
__global__ void __launch_bounds__(kRelayoutThreads, 4) relayout_kernel(const RelayoutParams p) {
    extern __shared__ __align__(16) uint8_t smem[];
    const int tile_cols = 1 << p.tile_cols_log2;        // bytes
    const int srow = tile_cols + kRowPad;               // shared-memory row pitch
    const int chunks_per_row_log2 = p.tile_cols_log2 - 4;

    // Block-order walk of the tile: index -> (block row, block col, row in block, byte in block row).
    // rin = rows of one block inside the tile, cin = bytes of one block row inside the tile.
    const int rin_log2 = min(p.tile_rows_log2, p.br_log2);
    const int cin_log2 = min(p.tile_cols_log2, p.run_log2);
    const int nbc_log2 = p.tile_cols_log2 - cin_log2;   // block columns in the tile

    for (int64_t tile = blockIdx.x; tile < p.tiles_total; tile += gridDim.x) {
        const int64_t row0 = (tile / p.tiles_x) << p.tile_rows_log2;
        const int64_t cb0 = (tile % p.tiles_x) << p.tile_cols_log2;

        uint4 v[kChunksPerThread];
        // ---- phase 1: global -> registers (all loads in flight before any use)
#pragma unroll
        for (int i = 0; i < kChunksPerThread; ++i) {
            const int idx = i * kRelayoutThreads + threadIdx.x;
            v[i] = make_uint4(0, 0, 0, 0);
            if (p.to_tile_major) {
                const int r = idx >> chunks_per_row_log2;
                const int cb = (idx & ((1 << chunks_per_row_log2) - 1)) << 4;
                if (row0 + r < p.rows && cb0 + cb < p.pitch)
                    v[i] = ld_stream(p.src + (row0 + r) * p.pitch + cb0 + cb);
            } else if (kPiece == 16) {
                // 16-byte chunk of one block row
                const int c16 = idx & ((1 << (cin_log2 - 4)) - 1);
                const int rp = (idx >> (cin_log2 - 4)) & ((1 << rin_log2) - 1);
                const int bcol = (idx >> (cin_log2 - 4 + rin_log2)) & ((1 << nbc_log2) - 1);
                const int brow = idx >> (cin_log2 - 4 + rin_log2 + nbc_log2);
                const int r = (brow << rin_log2) + rp;
                const int cb = (bcol << cin_log2) + (c16 << 4);
                if (row0 + r < p.rows && cb0 + cb < p.pitch)
                    v[i] = ld_stream(p.src + tile_major_byte(p, row0 + r, cb0 + cb));
            } else {
                // a 16-byte vector of the tile-major side holds 16/kPiece consecutive block rows
                constexpr int kRowsPerVec = 16 / kPiece;
                const int vr = idx & ((1 << rin_log2) / kRowsPerVec - 1);
                const int bcol = (idx / ((1 << rin_log2) / kRowsPerVec)) & ((1 << nbc_log2) - 1);
                const int brow = idx / ((1 << rin_log2) / kRowsPerVec) >> nbc_log2;
                const int r = (brow << rin_log2) + vr * kRowsPerVec;
                const int cb = bcol << cin_log2;
                if (row0 + r < p.rows && cb0 + cb < p.pitch)
                    v[i] = ld_stream(p.src + tile_major_byte(p, row0 + r, cb0 + cb));
            }
        }
        // ---- registers -> shared memory, always as the row-major image of the tile
#pragma unroll
        for (int i = 0; i < kChunksPerThread; ++i) {
            const int idx = i * kRelayoutThreads + threadIdx.x;
            if (p.to_tile_major) {
                const int r = idx >> chunks_per_row_log2;
                const int cb = (idx & ((1 << chunks_per_row_log2) - 1)) << 4;
                *reinterpret_cast<uint4*>(smem + r * srow + cb) = v[i];
            } else if (kPiece == 16) {
                const int c16 = idx & ((1 << (cin_log2 - 4)) - 1);
                const int rp = (idx >> (cin_log2 - 4)) & ((1 << rin_log2) - 1);
                const int bcol = (idx >> (cin_log2 - 4 + rin_log2)) & ((1 << nbc_log2) - 1);
                const int brow = idx >> (cin_log2 - 4 + rin_log2 + nbc_log2);
                const int r = (brow << rin_log2) + rp;
                const int cb = (bcol << cin_log2) + (c16 << 4);
                *reinterpret_cast<uint4*>(smem + r * srow + cb) = v[i];
            } else {
                constexpr int kRowsPerVec = 16 / kPiece;
                const int vr = idx & ((1 << rin_log2) / kRowsPerVec - 1);
                const int bcol = (idx / ((1 << rin_log2) / kRowsPerVec)) & ((1 << nbc_log2) - 1);
                const int brow = idx / ((1 << rin_log2) / kRowsPerVec) >> nbc_log2;
                const int r = (brow << rin_log2) + vr * kRowsPerVec;
                const int cb = bcol << cin_log2;
                // one piece-wide store per block row (cb and the row pitch are multiples of the piece)
                using Piece = typename PieceType<kPiece>::type;
                const Piece* pieces = reinterpret_cast<const Piece*>(&v[i]);
#pragma unroll
                for (int q = 0; q < kRowsPerVec; ++q) *reinterpret_cast<Piece*>(smem + (r + q) * srow + cb) = pieces[q];
            }
        }
        __syncthreads();
        // ---- phase 2: shared memory -> global in the order of the destination
#pragma unroll
        for (int i = 0; i < kChunksPerThread; ++i) {
            const int idx = i * kRelayoutThreads + threadIdx.x;
            if (!p.to_tile_major) {
                const int r = idx >> chunks_per_row_log2;
                const int cb = (idx & ((1 << chunks_per_row_log2) - 1)) << 4;
                if (row0 + r < p.rows && cb0 + cb < p.pitch)
                    st_stream(p.dst + (row0 + r) * p.pitch + cb0 + cb,
                              *reinterpret_cast<const uint4*>(smem + r * srow + cb));
            } else if (kPiece == 16) {
                const int c16 = idx & ((1 << (cin_log2 - 4)) - 1);
                const int rp = (idx >> (cin_log2 - 4)) & ((1 << rin_log2) - 1);
                const int bcol = (idx >> (cin_log2 - 4 + rin_log2)) & ((1 << nbc_log2) - 1);
                const int brow = idx >> (cin_log2 - 4 + rin_log2 + nbc_log2);
                const int r = (brow << rin_log2) + rp;
                const int cb = (bcol << cin_log2) + (c16 << 4);
                if (row0 + r < p.rows && cb0 + cb < p.pitch)
                    st_stream(p.dst + tile_major_byte(p, row0 + r, cb0 + cb),
                              *reinterpret_cast<const uint4*>(smem + r * srow + cb));
            } else {
                constexpr int kRowsPerVec = 16 / kPiece;
                const int vr = idx & ((1 << rin_log2) / kRowsPerVec - 1);
                const int bcol = (idx / ((1 << rin_log2) / kRowsPerVec)) & ((1 << nbc_log2) - 1);
                const int brow = idx / ((1 << rin_log2) / kRowsPerVec) >> nbc_log2;
                const int r = (brow << rin_log2) + vr * kRowsPerVec;
                const int cb = bcol << cin_log2;
                if (row0 + r < p.rows && cb0 + cb < p.pitch) {
                    using Piece = typename PieceType<kPiece>::type;
                    uint4 out;
                    Piece* pieces = reinterpret_cast<Piece*>(&out);
#pragma unroll
                    for (int q = 0; q < kRowsPerVec; ++q)
                        pieces[q] = *reinterpret_cast<const Piece*>(smem + (r + q) * srow + cb);
                    st_stream(p.dst + tile_major_byte(p, row0 + r, cb0 + cb), out);
                }
            }
        }
        __syncthreads();
    }
}

// Element-wise fallback for pitches or pointers that are not 16-byte aligned, and for G < 16.
__global__ void relayout_elementwise_kernel(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst,
                                            int64_t rows, int64_t cols, int s, int br, int bc, int to_tile_major) {
    const int64_t total = rows * cols;
    const int64_t blocks_per_row = cols / bc;
    for (int64_t e = blockIdx.x * int64_t(blockDim.x) + threadIdx.x; e < total;
         e += int64_t(gridDim.x) * blockDim.x) {
        // e walks the tile-major buffer in element order
        const int64_t blk = e / (int64_t(br) * bc), in = e % (int64_t(br) * bc);
        const int64_t r = (blk / blocks_per_row) * br + in / bc;
        const int64_t c = (blk % blocks_per_row) * bc + in % bc;
        const int64_t row_off = (r * cols + c) * s, tile_off = e * s;
        for (int b = 0; b < s; ++b) {
            if (to_tile_major) dst[tile_off + b] = src[row_off + b];
            else dst[row_off + b] = src[tile_off + b];
        }
    }
}


// ------------------------------------------------------------------ TMA path
// For block rows of 32 bytes to 1 KB and memory tiles of at most 32 KB the copy engine does the permutation by
// itself.  The row-major matrix is described as a 3-D tensor of 32-bit words (words of a block row, matrix row,
// block column): a box of (block row, br rows, nb block columns) is nb whole memory tiles, which TMA writes to
// shared memory tile after tile: exactly their image in the tile-major buffer, where they are one contiguous
// run of nb*G bytes.  So a step is one tensor copy on the row-major side and one untiled bulk copy on the
// tile-major side (load then store, in the order the direction needs), one thread per CTA driving a ring of
// 32 KB buffers.  No registers, no block-wide barriers.
#ifndef TL_TMA_TILE
#define TL_TMA_TILE 32768
#endif
#ifndef TL_TMA_STAGES
#define TL_TMA_STAGES 3
#endif
#ifndef TL_TMA_CTAS
#define TL_TMA_CTAS 2
#endif
constexpr int kTmaTileBytes = TL_TMA_TILE;
constexpr int kTmaStages = TL_TMA_STAGES;        // ring of buffers per CTA
constexpr int kTmaCtasPerSm = TL_TMA_CTAS;

struct RelayoutTmaParams {
    CUtensorMap row_map;     // row-major side
    uint8_t* tile_base;      // tile-major side
    uint32_t* status;
    uint64_t wait_limit_ns;  // bound of the wait for a buffer's load
    uint32_t stall_extra_tx; // test hook: bytes added to what the first load's barrier expects (0 in normal use)
    int64_t G;
    int br, nb;              // rows of a memory tile, memory tiles per step
    int blocks_per_row, block_rows;
    int64_t steps_x, steps_total;
    int to_tile_major;
};

__global__ void __launch_bounds__(32, kTmaCtasPerSm) relayout_tma_kernel(const __grid_constant__ RelayoutTmaParams p) {
    extern __shared__ __align__(1024) uint8_t smem_tma[];
    __shared__ __align__(8) uint64_t full_bar[kTmaStages];
    __shared__ uint32_t abort_flag;
    if (threadIdx.x != 0) return;
    uint8_t* bufs = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_tma) + 127) & ~uintptr_t(127));
    for (int s = 0; s < kTmaStages; ++s) mbar_init(&full_bar[s], 1);
    abort_flag = 0;
    fence_mbar_init();
    tma_prefetch_desc(&p.row_map);
    volatile uint32_t* abort_ptr = &abort_flag;
    // Launched with programmatic stream serialisation: the set-up above may run while the kernel before this one
    // in the stream finishes; nothing is read or written before it has completed.  The kernel after this one
    // may start its own set-up at once (it waits for this grid in the same way).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int64_t first = blockIdx.x, stride = gridDim.x;
    const int64_t mine = first < p.steps_total ? (p.steps_total - first + stride - 1) / stride : 0;
    auto issue_load = [&](int64_t i) {
        const int64_t step = first + i * stride;
        const int s = int(i % kTmaStages);
        const int64_t brow = step / p.steps_x;
        const int b0 = int(step % p.steps_x) * p.nb;
        const int nbt = p.blocks_per_row - b0 < p.nb ? p.blocks_per_row - b0 : p.nb;
        uint8_t* buf = bufs + size_t(s) * kTmaTileBytes;
        const uint32_t extra = i == 0 ? p.stall_extra_tx : 0u;      // (test hook, see RelayoutTmaParams)
        if (p.to_tile_major) {
            mbar_arrive_expect_tx(&full_bar[s], uint32_t(p.nb) * uint32_t(p.G) + extra);      // a box always counts in full
            tma_load_3d(buf, &p.row_map, &full_bar[s], 0, int(brow) * p.br, b0);
        } else {
            mbar_arrive_expect_tx(&full_bar[s], uint32_t(nbt) * uint32_t(p.G) + extra);
            bulk_load_1d(buf, p.tile_base + (brow * p.blocks_per_row + b0) * p.G, uint32_t(nbt) * uint32_t(p.G), &full_bar[s]);
        }
    };
    const int64_t ahead = mine < kTmaStages - 1 ? mine : kTmaStages - 1;
    for (int64_t i = 0; i < ahead; ++i) issue_load(i);
    for (int64_t i = 0; i < mine; ++i) {
        const int s = int(i % kTmaStages);
        if (!mbar_wait_bounded(&full_bar[s], uint32_t(i / kTmaStages) & 1u, abort_ptr, p.status, kWaitRelayoutFull, p.wait_limit_ns)) break;
        const int64_t step = first + i * stride;
        const int64_t brow = step / p.steps_x;
        const int b0 = int(step % p.steps_x) * p.nb;
        const int nbt = p.blocks_per_row - b0 < p.nb ? p.blocks_per_row - b0 : p.nb;
        const uint8_t* buf = bufs + size_t(s) * kTmaTileBytes;
        if (p.to_tile_major)
            bulk_store_1d(p.tile_base + (brow * p.blocks_per_row + b0) * p.G, buf, uint32_t(nbt) * uint32_t(p.G));
        else
            tma_store_3d(&p.row_map, buf, 0, int(brow) * p.br, b0);       // the part of the box outside the matrix is not written
        bulk_commit_group();
        // The buffer the NEXT load goes to is the one whose store was committed one step ago.
        if (i + kTmaStages - 1 < mine) {
            bulk_wait_group_read<1>();
            issue_load(i + kTmaStages - 1);
        }
    }
    bulk_wait_group_read<0>();       // shared memory must outlive the last stores' reads
}

static int relayout_tma_launch(const void* d_src, void* d_dst, int64_t rows, int64_t cols, int s, int64_t G, int br, int bc,
                               int direction, cudaStream_t stream, bool* taken) {
    *taken = false;
    const int64_t run = int64_t(bc) * s, pitch = cols * s;
    // 16-byte block rows go to the shared-memory kernel: the tensor store would write the row-major side in
    // half-sector pieces (measured 3.2-4.4 TB/s against 5.2 TB/s).
    if (run < 32 || run > 1024 || G > kTmaTileBytes || br > 256) return TL_OK;
    if (pitch % 16 != 0 || pitch >= (int64_t(1) << 40) || rows >= (int64_t(1) << 31)) return TL_OK;
    const bool to_tile = direction == TL_TO_TILE_MAJOR;
    const void* row_side = to_tile ? d_src : d_dst;
    void* tile_side = to_tile ? d_dst : const_cast<void*>(d_src);
    if (reinterpret_cast<uintptr_t>(row_side) % 16 != 0 || reinterpret_cast<uintptr_t>(tile_side) % 16 != 0) return TL_OK;
    if (int rc = ensure_control()) return rc;
    if (int rc = ensure_device_info()) return rc;
    RelayoutTmaParams p;
    memset(&p, 0, sizeof p);
    int nb = int(kTmaTileBytes / G);
    if (nb > 256) nb = 256;
    const int64_t blocks_per_row = cols / bc;
    if (nb > blocks_per_row) nb = int(blocks_per_row);
    const uint64_t dims[3] = {uint64_t(run / 4), uint64_t(rows), uint64_t(blocks_per_row)};
    const uint64_t strides[3] = {4, uint64_t(pitch), uint64_t(run)};
    const uint32_t box[3] = {uint32_t(run / 4), uint32_t(br), uint32_t(nb)};
    if (int rc = encode_tensor_map(&p.row_map, row_side, int(CU_TENSOR_MAP_DATA_TYPE_UINT32), int(CU_TENSOR_MAP_SWIZZLE_NONE), 3, dims,
                                   strides, box))
        return rc;
    p.tile_base = static_cast<uint8_t*>(tile_side);
    p.status = dev().ctl.d_status;
    p.wait_limit_ns = wait_limit_ns();
    if (opt(TL_OPT_STALL_ONCE) == 2) {           // test hook: this launch's first load per CTA never completes its barrier
        p.stall_extra_tx = 16;
        tl_set_option(TL_OPT_STALL_ONCE, 0);
    }
    p.G = G;
    p.br = br;
    p.nb = nb;
    p.blocks_per_row = int(blocks_per_row);
    p.block_rows = int(rows / br);
    p.steps_x = ceil_div(blocks_per_row, nb);
    p.steps_total = p.steps_x * (rows / br);
    p.to_tile_major = to_tile;
    const size_t smem = size_t(kTmaStages) * kTmaTileBytes + 128;
    if (int rc = ensure_smem_attr(reinterpret_cast<const void*>(relayout_tma_kernel), int(smem))) return rc;
    const int64_t max_grid = int64_t(dev().sm_count) * kTmaCtasPerSm;
    const int grid = int(p.steps_total < max_grid ? p.steps_total : max_grid);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = opt(TL_OPT_PDL) != 0 ? 1 : 0;           // measurement switch
    *taken = true;
    return check_cuda(cudaLaunchKernelEx(&cfg, relayout_tma_kernel, p));
}

// ------------------------------------------------------------------ several matrices in one launch
// The same ring of copies over the concatenated step lists of up to kBatchMax matrices that share element size,
// memory tile and direction (the weights of one layer at load time): no kernel boundary, hence no ramp and tail,
// between them.
constexpr int kBatchMax = 8;

struct RelayoutTmaBatch {
    CUtensorMap row_map[kBatchMax];
    uint8_t* tile_base[kBatchMax];
    int64_t steps_begin[kBatchMax + 1];    // first global step of each matrix
    int steps_x[kBatchMax];                // steps along a block row
    int blocks_per_row[kBatchMax];
    int nb[kBatchMax];                     // memory tiles per step (min(tile budget, blocks per row))
    uint32_t* status;
    uint64_t wait_limit_ns;
    int64_t G;
    int br, n;
    int to_tile_major;
};

__global__ void __launch_bounds__(32, kTmaCtasPerSm) relayout_tma_batch_kernel(const __grid_constant__ RelayoutTmaBatch p) {
    extern __shared__ __align__(1024) uint8_t smem_tma[];
    __shared__ __align__(8) uint64_t full_bar[kTmaStages];
    __shared__ uint32_t abort_flag;
    if (threadIdx.x != 0) return;
    uint8_t* bufs = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_tma) + 127) & ~uintptr_t(127));
    for (int s = 0; s < kTmaStages; ++s) mbar_init(&full_bar[s], 1);
    abort_flag = 0;
    fence_mbar_init();
    for (int i = 0; i < p.n; ++i) tma_prefetch_desc(&p.row_map[i]);
    volatile uint32_t* abort_ptr = &abort_flag;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int64_t first = blockIdx.x, stride = gridDim.x, total = p.steps_begin[p.n];
    const int64_t mine = first < total ? (total - first + stride - 1) / stride : 0;
    struct Step { int m; int brow; int b0; int nbt; };
    auto locate = [&](int64_t i) {
        const int64_t g = first + i * stride;
        int m = 0;
        while (m + 1 < p.n && g >= p.steps_begin[m + 1]) ++m;
        const int64_t local = g - p.steps_begin[m];
        Step st;
        st.m = m;
        st.brow = int(local / p.steps_x[m]);
        st.b0 = int(local % p.steps_x[m]) * p.nb[m];
        st.nbt = p.blocks_per_row[m] - st.b0 < p.nb[m] ? p.blocks_per_row[m] - st.b0 : p.nb[m];
        return st;
    };
    auto tile_ptr = [&](const Step& st) {
        return p.tile_base[st.m] + (int64_t(st.brow) * p.blocks_per_row[st.m] + st.b0) * p.G;
    };
    auto issue_load = [&](int64_t i) {
        const Step st = locate(i);
        const int s = int(i % kTmaStages);
        uint8_t* buf = bufs + size_t(s) * kTmaTileBytes;
        if (p.to_tile_major) {
            mbar_arrive_expect_tx(&full_bar[s], uint32_t(p.nb[st.m]) * uint32_t(p.G));     // a box always counts in full
            tma_load_3d(buf, &p.row_map[st.m], &full_bar[s], 0, st.brow * p.br, st.b0);
        } else {
            mbar_arrive_expect_tx(&full_bar[s], uint32_t(st.nbt) * uint32_t(p.G));
            bulk_load_1d(buf, tile_ptr(st), uint32_t(st.nbt) * uint32_t(p.G), &full_bar[s]);
        }
    };
    const int64_t ahead = mine < kTmaStages - 1 ? mine : kTmaStages - 1;
    for (int64_t i = 0; i < ahead; ++i) issue_load(i);
    for (int64_t i = 0; i < mine; ++i) {
        const int s = int(i % kTmaStages);
        if (!mbar_wait_bounded(&full_bar[s], uint32_t(i / kTmaStages) & 1u, abort_ptr, p.status, kWaitRelayoutFull, p.wait_limit_ns)) break;
        const Step st = locate(i);
        const uint8_t* buf = bufs + size_t(s) * kTmaTileBytes;
        if (p.to_tile_major) bulk_store_1d(tile_ptr(st), buf, uint32_t(st.nbt) * uint32_t(p.G));
        else tma_store_3d(&p.row_map[st.m], buf, 0, st.brow * p.br, st.b0);
        bulk_commit_group();
        if (i + kTmaStages - 1 < mine) {
            bulk_wait_group_read<1>();
            issue_load(i + kTmaStages - 1);
        }
    }
    bulk_wait_group_read<0>();
}

// Whether one matrix can take the copy-engine path (the conditions of relayout_tma_launch).
static bool relayout_tma_eligible(const void* d_src, const void* d_dst, int64_t rows, int64_t cols, int s, int64_t G, int br,
                                  int bc) {
    const int64_t run = int64_t(bc) * s, pitch = cols * s;
    if (run < 32 || run > 1024 || G > kTmaTileBytes || br > 256) return false;
    if (pitch % 16 != 0 || pitch >= (int64_t(1) << 40) || rows >= (int64_t(1) << 31)) return false;
    return reinterpret_cast<uintptr_t>(d_src) % 16 == 0 && reinterpret_cast<uintptr_t>(d_dst) % 16 == 0;
}

static int relayout_tma_batch_launch(int n, const void* const* srcs, void* const* dsts, const int64_t* rows,
                                     const int64_t* cols, int s, int64_t G, int br, int bc, int direction,
                                     cudaStream_t stream) {
    if (int rc = ensure_control()) return rc;
    if (int rc = ensure_device_info()) return rc;
    RelayoutTmaBatch p;
    memset(&p, 0, sizeof p);
    const bool to_tile = direction == TL_TO_TILE_MAJOR;
    const int64_t run = int64_t(bc) * s;
    int nb_max = int(kTmaTileBytes / G);
    if (nb_max > 256) nb_max = 256;
    p.steps_begin[0] = 0;
    for (int i = 0; i < n; ++i) {
        const void* row_side = to_tile ? srcs[i] : dsts[i];
        void* tile_side = to_tile ? dsts[i] : const_cast<void*>(srcs[i]);
        const int64_t blocks_per_row = cols[i] / bc, pitch = cols[i] * s;
        const int nb = nb_max > blocks_per_row ? int(blocks_per_row) : nb_max;
        const uint64_t dims[3] = {uint64_t(run / 4), uint64_t(rows[i]), uint64_t(blocks_per_row)};
        const uint64_t strides[3] = {4, uint64_t(pitch), uint64_t(run)};
        const uint32_t box[3] = {uint32_t(run / 4), uint32_t(br), uint32_t(nb)};
        if (int rc = encode_tensor_map(&p.row_map[i], row_side, int(CU_TENSOR_MAP_DATA_TYPE_UINT32), int(CU_TENSOR_MAP_SWIZZLE_NONE),
                                       3, dims, strides, box))
            return rc;
        p.tile_base[i] = static_cast<uint8_t*>(tile_side);
        p.blocks_per_row[i] = int(blocks_per_row);
        p.nb[i] = nb;
        p.steps_x[i] = int(ceil_div(blocks_per_row, nb));
        p.steps_begin[i + 1] = p.steps_begin[i] + int64_t(p.steps_x[i]) * (rows[i] / br);
    }
    p.status = dev().ctl.d_status;
    p.wait_limit_ns = wait_limit_ns();
    p.G = G;
    p.br = br;
    p.n = n;
    p.to_tile_major = to_tile;
    const size_t smem = size_t(kTmaStages) * kTmaTileBytes + 128;
    if (int rc = ensure_smem_attr(reinterpret_cast<const void*>(relayout_tma_batch_kernel), int(smem))) return rc;
    const int64_t max_grid = int64_t(dev().sm_count) * kTmaCtasPerSm, total = p.steps_begin[n];
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(total < max_grid ? total : max_grid));
    cfg.blockDim = dim3(32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = opt(TL_OPT_PDL) != 0 ? 1 : 0;           // measurement switch
    return check_cuda(cudaLaunchKernelEx(&cfg, relayout_tma_batch_kernel, p));
}

static int ilog2(int64_t x) {
    int l = 0;
    while ((int64_t(1) << l) < x) ++l;
    return l;
}

int relayout_launch(const void* d_src, void* d_dst, int64_t rows, int64_t cols, int s, int64_t G, int br, int bc,
                    int direction, cudaStream_t stream) {
    if (rows < 0 || cols < 0) return TL_ERR_INVALID_ARG;
    if (s != 1 && s != 2 && s != 4) return TL_ERR_INVALID_ARG;
    if (br <= 0 || bc <= 0 || int64_t(br) * bc * s != G) return TL_ERR_INVALID_ARG;
    if (direction != TL_TO_TILE_MAJOR && direction != TL_TO_ROW_MAJOR) return TL_ERR_INVALID_ARG;
    if (!is_pow2(br) || !is_pow2(bc)) return TL_ERR_UNSUPPORTED;
    if (rows % br != 0 || cols % bc != 0) return TL_ERR_INVALID_ARG;
    if (rows == 0 || cols == 0) return TL_OK;
    if (!d_src || !d_dst) return TL_ERR_INVALID_ARG;
    const int64_t bytes = rows * cols * s;
    const uintptr_t a = reinterpret_cast<uintptr_t>(d_src), b = reinterpret_cast<uintptr_t>(d_dst);
    if (a < b + bytes && b < a + bytes) return TL_ERR_INVALID_ARG;      // overlap
    if (int rc = ensure_device_info()) return rc;
    const int sms = dev().sm_count;

    {
        // copy-engine path when the shape allows it (TL_OPT_RELAYOUT_TMA = 0 keeps the shared-memory kernel)
        const bool no_tma = opt(TL_OPT_RELAYOUT_TMA) == 0;
        bool taken = false;
        if (!no_tma) {
            if (int rc = relayout_tma_launch(d_src, d_dst, rows, cols, s, G, br, bc, direction, stream, &taken)) return rc;
            if (taken) return TL_OK;
        }
    }
    const int64_t pitch = cols * s;
    const int64_t run = int64_t(bc) * s;
    const bool fast = (pitch % 16 == 0) && (a % 16 == 0) && (b % 16 == 0) && G >= 16;
    if (!fast) {
        const int64_t total = rows * cols;
        const int grid = int(total / 256 + 1 < int64_t(sms) * 16 ? total / 256 + 1 : int64_t(sms) * 16);
        relayout_elementwise_kernel<<<grid, 256, 0, stream>>>(static_cast<const uint8_t*>(d_src),
                                                              static_cast<uint8_t*>(d_dst), rows, cols, s, br, bc,
                                                              direction == TL_TO_TILE_MAJOR);
        return check_cuda(cudaGetLastError());
    }

    RelayoutParams p;
    p.src = static_cast<const uint8_t*>(d_src);
    p.dst = static_cast<uint8_t*>(d_dst);
    p.rows = rows;
    p.pitch = pitch;
    p.blocks_per_row = cols / bc;
    p.run_log2 = ilog2(run);
    p.br_log2 = ilog2(br);
    // Tile: as wide as one block row, but between 1 KB and 2 KB of a matrix row so that the
    // row-major side moves long contiguous strips; rows fill the rest of the 32 KB.
    int64_t tile_cols = run < 1024 ? 1024 : (run > 2048 ? 2048 : run);
    int64_t tile_rows = kTileBytes / tile_cols;
    // A 16-byte vector of the tile-major side needs 16/run block rows of the same block in the tile.
    const int piece = run >= 16 ? 16 : int(run);
    p.tile_cols_log2 = ilog2(tile_cols);
    p.tile_rows_log2 = ilog2(tile_rows);
    p.tiles_x = ceil_div(pitch, tile_cols);
    p.tiles_total = p.tiles_x * ceil_div(rows, tile_rows);
    p.to_tile_major = direction == TL_TO_TILE_MAJOR;

    const size_t smem = size_t(tile_rows) * (tile_cols + kRowPad);
    const int64_t max_grid = int64_t(sms) * 4;
    const int grid = int(p.tiles_total < max_grid ? p.tiles_total : max_grid);
    cudaError_t err = cudaSuccess;
#define TL_LAUNCH_RELAYOUT(PIECE)                                                                              \
    if (int rc = ensure_smem_attr(reinterpret_cast<const void*>(relayout_kernel<PIECE>), 48 * 1024)) return rc; \
    relayout_kernel<PIECE><<<grid, kRelayoutThreads, smem, stream>>>(p);
    switch (piece) {
        case 16: TL_LAUNCH_RELAYOUT(16) break;
        case 8: TL_LAUNCH_RELAYOUT(8) break;
        case 4: TL_LAUNCH_RELAYOUT(4) break;
        case 2: TL_LAUNCH_RELAYOUT(2) break;
        default: TL_LAUNCH_RELAYOUT(1) break;
    }
#undef TL_LAUNCH_RELAYOUT
    if (err != cudaSuccess) return check_cuda(err);
    return check_cuda(cudaGetLastError());
}

}  // namespace tl

extern "C" {

int tl_relayout_on(const void* d_src, void* d_dst, int64_t rows, int64_t cols, int elem_bytes, int64_t G,
                   int block_rows, int block_cols, int direction, void* cuda_stream) {
    tl::ApiLock lock;
    return tl::relayout_launch(d_src, d_dst, rows, cols, elem_bytes, G, block_rows, block_cols, direction,
                               static_cast<cudaStream_t>(cuda_stream));
}

int tl_relayout_batch(int n, const void* const* d_srcs, void* const* d_dsts, const int64_t* rows, const int64_t* cols,
                      int elem_bytes, int64_t G, int block_rows, int block_cols, int direction, void* cuda_stream) {
    tl::ApiLock lock;
    if (n < 0 || (n > 0 && (!d_srcs || !d_dsts || !rows || !cols))) return TL_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const bool no_tma = tl::opt(TL_OPT_RELAYOUT_TMA) == 0;
    // One launch when every matrix passes the argument checks of tl_relayout, is non-empty and can take the
    // copy-engine path; otherwise (and beyond kBatchMax matrices) one tl_relayout_on per matrix, in order.
    int i = 0;
    while (i < n) {
        int m = 0;
        while (!no_tma && i + m < n && m < tl::kBatchMax) {
            const int j = i + m;
            const int64_t bytes = rows[j] * cols[j] * elem_bytes;
            const uintptr_t a = reinterpret_cast<uintptr_t>(d_srcs[j]), b = reinterpret_cast<uintptr_t>(d_dsts[j]);
            const bool ok = (elem_bytes == 1 || elem_bytes == 2 || elem_bytes == 4) && block_rows > 0 && block_cols > 0 &&
                            int64_t(block_rows) * block_cols * elem_bytes == G && tl::is_pow2(block_rows) && tl::is_pow2(block_cols) &&
                            (direction == TL_TO_TILE_MAJOR || direction == TL_TO_ROW_MAJOR) && rows[j] > 0 && cols[j] > 0 &&
                            rows[j] % block_rows == 0 && cols[j] % block_cols == 0 && d_srcs[j] && d_dsts[j] &&
                            !(a < b + bytes && b < a + bytes) &&
                            tl::relayout_tma_eligible(d_srcs[j], d_dsts[j], rows[j], cols[j], elem_bytes, G, block_rows, block_cols);
            if (!ok) break;
            ++m;
        }
        if (m >= 2) {
            if (int rc = tl::relayout_tma_batch_launch(m, d_srcs + i, d_dsts + i, rows + i, cols + i, elem_bytes, G, block_rows,
                                                       block_cols, direction, stream))
                return rc;
            i += m;
        } else {
            if (int rc = tl::relayout_launch(d_srcs[i], d_dsts[i], rows[i], cols[i], elem_bytes, G, block_rows, block_cols,
                                             direction, stream))
                return rc;
            ++i;
        }
    }
    return TL_OK;
}

int tl_relayout(const void* d_src, void* d_dst, int64_t rows, int64_t cols, int elem_bytes, int64_t G,
                int block_rows, int block_cols, int direction) {
    tl::ApiLock lock;
    return tl::relayout_launch(d_src, d_dst, rows, cols, elem_bytes, G, block_rows, block_cols, direction,
                               tl::tls().stream);
}

}  // extern "C"
