// Two grouped products in ONE launch: the expert FFN (gate_up with the gated epilogue, then down).
//
// The down product of an (expert, row) needs every gate_up tile of that row, so the kernel runs the two products as
// two phases of one grid with a grid-wide barrier between them:
//   phase 1   the first product through gemm_body (whole rounds of tiles + a stream-K cut of the rest);
//   barrier   every CTA's partial tiles are in the workspace;
//   sum       CTA b sums the split tile of boundary b + 1 (the body of streamk_reduce_kernel) and writes H;
//   barrier   H is complete;
//   phase 2   the second product through gemm_body; its own split tiles are summed by the ordinary
//             streamk_reduce_kernel that follows in the stream.
// The barrier is an arrival counter in global memory that only grows (the host passes each launch the values it
// waits for); every CTA arrives after a __syncthreads and a device-scope fence and then polls with a bound, after
// which it raises the status word and goes on, so the kernel always terminates.  All CTAs must be resident at the
// same time: the kernel is launched cooperatively (the launch fails rather than wait on a CTA that cannot run).
//
// A second form needs no barrier at all: the first product is scheduled as whole tiles only (no partial tiles, nothing
// to sum), every epilogue warp adds one to a counter of the m-tile whose rows of H it has stored, and the second
// product's producer waits, tile by tile and with a bound, until the counter of the m-tile it is about to load has
// reached (warps x column tiles of the first product).  A CTA that runs out of first-product tiles goes straight on
// to second-product tiles, whose experts were finished long ago: nobody waits for the slowest CTA.  No tile of the
// first product ever waits, and every CTA finishes its first-product tiles before it starts the second product, so
// the counters always fill (the cooperative launch keeps all CTAs resident); the counters are cleared by a memset
// enqueued before the launch.
//
// Measured on B200 (Qwen-3-30B-A3B expert FFN, 2048 routed rows, back-to-back calls): 203 us for the two products as
// two launches, 241 us with the barriers, 220 us with the counters (198, 216-221 and 208-210 us since short tiles are
// no longer cut along K in either product) (214 us when launched with programmatic stream
// serialisation instead of cooperatively, which is not kept: the co-residency the waits rely on would then rest on the
// grid being no larger than the SM count).  The counter form's first product cannot balance its last, partial round
// of tiles the way the stream-K cut does (the CTAs that ran one tile more finish 6 % later); giving the other CTAs a
// larger share of the second product's cut part instead made it slower still (238 us): that part then starts while
// the last experts' rows of H are still being computed, and waits.
// The boundary between two launches is already hidden by programmatic stream serialisation: with the barriers and
// the in-kernel sum compiled out the barrier form only tied with two launches; its two barriers add 12 us (every CTA
// waits for the slowest, twice) and the in-kernel sum 14 us (its index arithmetic is no longer hidden behind the first
// product's tail).  tl_moe_ffn therefore uses two launches unless TL_OPT_FFN_ONE_LAUNCH is set.
#include "tl_gemm_kernel.cuh"

namespace tl {

// Returns false when the wait ran out.
// (skip_arrival: test hook -- this CTA polls without having arrived, so that every CTA's wait runs out.)
__device__ __forceinline__ bool grid_barrier(unsigned long long* counter, unsigned long long target, uint64_t limit_ns,
                                             uint32_t* status, bool skip_arrival = false) {
    __shared__ int ok_flag;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();                                   // this CTA's writes before its arrival
        if (!skip_arrival) atomicAdd(counter, 1ull);
        bool ok = true;
        uint64_t t0 = 0;
        uint32_t polls = 0;
        while (true) {
            unsigned long long seen;
            asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(seen) : "l"(counter) : "memory");
            if (seen >= target) break;
            __nanosleep(64);                               // 148 pollers share one line of L2
            if ((++polls & 255u) == 0) {
                const uint64_t now = global_timer_ns();
                if (t0 == 0) t0 = now;
                if (now - t0 > limit_ns) {
                    atomicCAS(status, 0u, kWaitGridBarrier);
                    ok = false;
                    break;
                }
            }
        }
        __threadfence();
        ok_flag = ok;
    }
    __syncthreads();
    // what other CTAs wrote with ordinary stores is read by the copy engine next (H, as the second product's tokens)
    asm volatile("fence.proxy.async;" ::: "memory");
    return ok_flag != 0;
}

template <int kBK, int kBN>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_chain_kernel(const __grid_constant__ GemmParams p1, const __grid_constant__ GemmParams p2,
                  unsigned long long* counter, unsigned long long target1, unsigned long long target2, int skip_cta0) {
    __shared__ int prefix[kMaxExperts + 1];
    __shared__ int row_start[kMaxExperts + 1];
    __shared__ int slot_of[kRangeTabMax];
    gemm_body<kBK, kBN, true, false>(p1, true, false);
    if (p1.tile_flags_mode == 1) {
        // Per-m-tile counters instead of barriers: the first product runs whole tiles only, every CTA goes straight on to
        // its tiles of the second product, whose producer waits for the rows it is about to load (see gemm_body).
        gemm_body<kBK, kBN, true, false>(p2, false, true);
        return;
    }
    const bool ok1 = grid_barrier(counter, target1, p1.wait_limit_ns, p1.status, skip_cta0 != 0 && blockIdx.x == 0);
    if (ok1 && p1.stream_k && int(blockIdx.x) + 1 < int(gridDim.x))
        streamk_reduce_body<false>(p1, int(gridDim.x), int(blockIdx.x), prefix, row_start, slot_of);
    grid_barrier(counter, target2, p1.wait_limit_ns, p1.status);
    gemm_body<kBK, kBN, true, false>(p2, false, true);
}

int launch_gemm_chain(int bk, int bn, int grid, size_t smem, cudaStream_t stream, const GemmParams& p1,
                      const GemmParams& p2, unsigned long long* counter, unsigned long long target1,
                      unsigned long long target2, bool skip_cta0) {
    if (bk != 64 || bn != 256) return TL_ERR_UNSUPPORTED;
    auto* kernel = gemm_chain_kernel<64, 256>;
    // (this kernel's static shared memory is about 10 KB above the plain GEMM kernel's)
    if (int rc = ensure_smem_attr(reinterpret_cast<const void*>(kernel), kMaxDynamicSmem - 10 * 1024)) return rc;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return check_cuda(cudaLaunchKernelEx(&cfg, kernel, p1, p2, counter, target1, target2, int(skip_cta0)));
}

}  // namespace tl
