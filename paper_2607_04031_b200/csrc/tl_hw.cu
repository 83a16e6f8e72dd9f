// Tile-major aware box loads (Section 4.3 of the paper: the proposed extension of the TMA's source-address
// computation), emulated in software.
//
// A descriptor describes a VIEW of the column-major K x N matrix the way a tensor map does (extents, strides and
// box in elements, dimension 0 contiguous) plus the two fields the section adds: the memory tile (a, b) and the
// leading stride K.  The buffer itself is tile-major (Eq. 2).  For every box the kernels do what the section
// describes for the engine:
//   phase 1  split-and-sum: coordinate x stride products with a stride below K add up to the row index i, the
//            rest to K*j; tileBase = (K*j + i*b)*s (Eq. 4);
//   phase 2  counters: the dimension whose stride is K becomes two nested counters, b steps of stride a and v/b
//            steps of stride b*K (Eq. 5); a stride below K is multiplied by b, a stride above K is kept;
//   case 2   (a wider than the box, a > u): all of the above as if the memory tile were u x b, then the bit
//            permutation (sub-tile | col | row) -> (col | sub-tile | row) inside the intra-tile offset.
// The reconfigured counters are prepared once per descriptor on the host (the part the section does at
// descriptor set-up); the per-box and per-request work runs on the GPU: one warp per box (boxes above 8 KB are cut
// into 8 KB runs of pieces taken by consecutive warps), one lane per 16-byte piece of a box row.
#include "tl_common.cuh"

namespace tl {

constexpr uint32_t kHwBadCoord = 0x900;      // status detail: a box with unaligned or out-of-range coordinates

struct HwParams {
    int rank, s_log2;
    int n_cnt;                       // counters after the split, extents of 1 dropped
    int ext[6];                      // their extents ...
    int shift[6];                    // ... log2(extent) when it is a power of two, else -1
    long long str[6];                // ... and strides (elements), dimension 0 first
    long long dims[5], strides[5], box[5];
    long long K, b;
    long long u;                     // box[0]
    int row_bits, col_bits, sub_bits;
    long long box_elems;
    long long n_boxes;
    int split_log2;                  // box_load: a box is moved by 2^split_log2 warps, each taking a run of pieces
    const int32_t* coords;           // [n_boxes][rank]
    const uint8_t* src;
    unsigned long long src_bytes;
    uint8_t* dst;                    // box_load: dense boxes, coordinate order
    unsigned long long* offsets;     // box_offsets: one byte offset per element
    uint32_t* status;
};

// Phase 1 for one box.  Returns false (and raises the status word) when Eq. 4's premise does not hold.
__device__ __forceinline__ bool hw_tile_base(const HwParams& p, const int32_t* c, long long* base_elems) {
    long long i = 0, kj = 0;
    bool ok = true;
    for (int d = 0; d < p.rank; ++d) {
        const long long x = c[d];
        ok = ok && x >= 0 && x + p.box[d] <= p.dims[d];
        if (p.strides[d] < p.K) i += x * p.strides[d];
        else kj += x * p.strides[d];
    }
    ok = ok && (i & (p.u - 1)) == 0 && kj % (p.K * p.b) == 0;
    if (!ok) {
        atomicCAS(p.status, 0u, kHwBadCoord);
        return false;
    }
    *base_elems = kj + i * p.b;          // Eq. 4, in elements
    return true;
}

// Phase 2 for the element at linear position t of the box (dimension 0 fastest): counters -> element offset,
// then the case-2 permutation.
__device__ __forceinline__ long long hw_src_elem(const HwParams& p, long long base, unsigned t) {
    long long e = base;
#pragma unroll
    for (int k = 0; k < 6; ++k) {
        if (k < p.n_cnt) {
            unsigned c;
            if (p.shift[k] >= 0) { c = t & unsigned(p.ext[k] - 1); t >>= p.shift[k]; }
            else { const unsigned q = t / unsigned(p.ext[k]); c = t - q * unsigned(p.ext[k]); t = q; }
            e += (long long)c * p.str[k];
        }
    }
    if (p.sub_bits > 0) {
        const int rc = p.row_bits + p.col_bits;
        const long long mask = (1ll << (rc + p.sub_bits)) - 1;
        const long long intra = e & mask;
        const long long row = intra & ((1ll << p.row_bits) - 1);
        const long long col = (intra >> p.row_bits) & ((1ll << p.col_bits) - 1);
        const long long sub = intra >> rc;
        e = (e & ~mask) | (col << (p.sub_bits + p.row_bits)) | (sub << p.row_bits) | row;
    }
    return e;
}

// One warp per box: lane 0 does phase 1, all lanes share phase 2.
__device__ __forceinline__ bool hw_warp_base(const HwParams& p, long long box, int lane, long long* base) {
    long long b0 = 0;
    int ok = 0;
    if (lane == 0) ok = hw_tile_base(p, p.coords + box * p.rank, &b0) ? 1 : 0;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    *base = __shfl_sync(0xffffffffu, b0, 0);
    return ok != 0;
}

__global__ void __launch_bounds__(256) hw_offsets_kernel(const HwParams p) {
    const int lane = threadIdx.x & 31;
    const long long warps = gridDim.x * 8ll;
    const unsigned n = unsigned(p.box_elems);
    for (long long box = blockIdx.x * 8ll + (threadIdx.x >> 5); box < p.n_boxes; box += warps) {
        long long base;
        const bool ok = hw_warp_base(p, box, lane, &base);
        unsigned long long* out = p.offsets + box * p.box_elems;
        for (unsigned t = lane; t < n; t += 32)
            out[t] = ok ? (unsigned long long)(hw_src_elem(p, base, t) << p.s_log2) : ~0ull;
    }
}

// kVec: bytes one thread moves at a time (16 when a box row is at least 16 bytes, else the element size).
template <int kVec>
__global__ void __launch_bounds__(256) hw_load_kernel(const HwParams p) {
    const int lane = threadIdx.x & 31;
    const long long warps = gridDim.x * 8ll;
    const unsigned pieces = unsigned((p.box_elems << p.s_log2) / kVec);
    const int piece_elems_log2 = (kVec == 16 ? 4 : p.s_log2) - p.s_log2;
    const unsigned part_pieces = pieces >> p.split_log2;
    const long long items = p.n_boxes << p.split_log2;
    for (long long item = blockIdx.x * 8ll + (threadIdx.x >> 5); item < items; item += warps) {
        const long long box = item >> p.split_log2;
        const unsigned first = unsigned(item & ((1 << p.split_log2) - 1)) * part_pieces;
        long long base;
        if (!hw_warp_base(p, box, lane, &base)) continue;
        uint8_t* dst = p.dst + box * (p.box_elems << p.s_log2);
#pragma unroll 4
        for (unsigned piece = first + lane; piece < first + part_pieces; piece += 32) {
            const unsigned long long src = (unsigned long long)(hw_src_elem(p, base, piece << piece_elems_log2) << p.s_log2);
            if (src + kVec > p.src_bytes) {
                atomicCAS(p.status, 0u, kHwBadCoord);
                continue;
            }
            uint8_t* d = dst + size_t(piece) * kVec;
            if (kVec == 16) *reinterpret_cast<uint4*>(d) = __ldg(reinterpret_cast<const uint4*>(p.src + src));
            else if (kVec == 4) *reinterpret_cast<uint32_t*>(d) = __ldg(reinterpret_cast<const uint32_t*>(p.src + src));
            else if (kVec == 2) *reinterpret_cast<uint16_t*>(d) = __ldg(reinterpret_cast<const uint16_t*>(p.src + src));
            else *d = __ldg(p.src + src);
        }
    }
}

static int ilog2_ll(long long x) {
    int l = 0;
    while ((1ll << l) < x) ++l;
    return l;
}

// Descriptor set-up: validation and the counter reconfiguration of Eq. 5.
static int hw_prepare(const tl_hw_desc* d, HwParams* p) {
    if (!d) return TL_ERR_INVALID_ARG;
    if (d->rank < 2 || d->rank > 5) return TL_ERR_INVALID_ARG;
    const int s = d->elem_bytes;
    if (s != 1 && s != 2 && s != 4) return TL_ERR_INVALID_ARG;
    const long long a = d->tile_a, b = d->tile_b, K = d->leading_stride;
    if (!is_pow2(a) || !is_pow2(b) || K <= 0 || K % a != 0 || d->strides[0] != 1) return TL_ERR_INVALID_ARG;
    const long long u = d->box[0];
    if (!is_pow2(u)) return TL_ERR_INVALID_ARG;
    if (u > a) return TL_ERR_UNSUPPORTED;                 // the section covers a == u and a > u
    memset(p, 0, sizeof *p);
    p->rank = d->rank;
    p->s_log2 = ilog2_ll(s);
    p->K = K;
    p->b = b;
    p->u = u;
    p->box_elems = 1;
    int n = 0;
    for (int k = 0; k < d->rank; ++k) {
        const long long sg = d->strides[k], v = d->box[k];
        if (d->dims[k] <= 0 || v <= 0 || v > d->dims[k] || sg <= 0) return TL_ERR_INVALID_ARG;
        p->dims[k] = d->dims[k];
        p->strides[k] = sg;
        p->box[k] = v;
        p->box_elems *= v;
        auto counter = [&](long long extent, long long stride) {
            if (extent == 1) return;
            p->ext[n] = int(extent);
            p->shift[n] = is_pow2(extent) ? ilog2_ll(extent) : -1;
            p->str[n] = stride;
            ++n;
        };
        if (k == 0) counter(u, 1);
        else if (sg == K) {
            if (v % b != 0) return TL_ERR_UNSUPPORTED;    // case 1 premise: v is a multiple of b
            counter(b, u);
            counter(v / b, b * K);
        } else if (sg < K) {
            if (sg % u != 0) return TL_ERR_UNSUPPORTED;
            counter(v, sg * b);
        } else {
            if (sg % (b * K) != 0) return TL_ERR_UNSUPPORTED;
            counter(v, sg);
        }
    }
    if (p->box_elems >= (1ll << 28)) return TL_ERR_UNSUPPORTED;
    p->n_cnt = n;
    p->row_bits = ilog2_ll(u);
    p->col_bits = ilog2_ll(b);
    p->sub_bits = ilog2_ll(a / u);
    return TL_OK;
}

// One warp per box (or per run of pieces of a box), eight warps per CTA, at most 8 CTAs per SM.
static unsigned hw_grid(long long n_boxes) {
    const long long ctas = ceil_div(n_boxes, 8);
    const long long cap = 8ll * (dev().sm_count > 0 ? dev().sm_count : 148);
    return unsigned(ctas < 1 ? 1 : (ctas < cap ? ctas : cap));
}

}  // namespace tl

extern "C" {

int tl_hw_box_offsets(const tl_hw_desc* desc, const int32_t* d_coords, int64_t n_boxes, uint64_t* d_offsets,
                      void* cuda_stream) {
    tl::ApiLock lock;
    tl::HwParams p;
    if (int rc = tl::hw_prepare(desc, &p)) return rc;
    if (n_boxes < 0) return TL_ERR_INVALID_ARG;
    if (n_boxes == 0) return TL_OK;
    if (!d_coords || !d_offsets) return TL_ERR_INVALID_ARG;
    if (int rc = tl::ensure_control()) return rc;
    if (int rc = tl::ensure_device_info()) return rc;
    p.n_boxes = n_boxes;
    p.coords = d_coords;
    p.offsets = reinterpret_cast<unsigned long long*>(d_offsets);
    p.status = tl::dev().ctl.d_status;
    tl::hw_offsets_kernel<<<tl::hw_grid(n_boxes), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(p);
    return tl::check_cuda(cudaGetLastError());
}

int tl_hw_box_load(const tl_hw_desc* desc, const void* d_src_tilemajor, uint64_t src_bytes, const int32_t* d_coords,
                   int64_t n_boxes, void* d_dst, void* cuda_stream) {
    tl::ApiLock lock;
    tl::HwParams p;
    if (int rc = tl::hw_prepare(desc, &p)) return rc;
    if (n_boxes < 0) return TL_ERR_INVALID_ARG;
    if (n_boxes == 0) return TL_OK;
    if (!d_coords || !d_src_tilemajor || !d_dst) return TL_ERR_INVALID_ARG;
    if (int rc = tl::ensure_control()) return rc;
    if (int rc = tl::ensure_device_info()) return rc;
    p.n_boxes = n_boxes;
    p.coords = d_coords;
    p.src = static_cast<const uint8_t*>(d_src_tilemajor);
    p.src_bytes = src_bytes;
    p.dst = static_cast<uint8_t*>(d_dst);
    p.status = tl::dev().ctl.d_status;
    const long long row_bytes = p.u << p.s_log2;
    const bool vec16 = row_bytes >= 16 && reinterpret_cast<uintptr_t>(d_src_tilemajor) % 16 == 0 &&
                       reinterpret_cast<uintptr_t>(d_dst) % 16 == 0;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // A warp moves at most 512 pieces (8 KB when vectorised, 16 per lane): larger boxes are cut into runs of
    // pieces taken by consecutive warps, which measured 12 % faster than one warp per 32 KB box.
    const long long pieces = (p.box_elems << p.s_log2) / (vec16 ? 16 : desc->elem_bytes);
    while (p.split_log2 < 8 && (pieces >> p.split_log2) > 512 && (pieces & ((2ll << p.split_log2) - 1)) == 0)
        ++p.split_log2;
    n_boxes <<= p.split_log2;
    if (vec16) tl::hw_load_kernel<16><<<tl::hw_grid(n_boxes), 256, 0, st>>>(p);
    else if (desc->elem_bytes == 4) tl::hw_load_kernel<4><<<tl::hw_grid(n_boxes), 256, 0, st>>>(p);
    else if (desc->elem_bytes == 2) tl::hw_load_kernel<2><<<tl::hw_grid(n_boxes), 256, 0, st>>>(p);
    else tl::hw_load_kernel<1><<<tl::hw_grid(n_boxes), 256, 0, st>>>(p);
    return tl::check_cuda(cudaGetLastError());
}

}  // extern "C"
