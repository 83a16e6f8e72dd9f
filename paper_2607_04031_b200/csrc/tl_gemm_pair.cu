// CTA-pair prefill kernel: instantiations and launcher.
#include "tl_gemm_kernel.cuh"
#include "tl_gemm_pair.cuh"

namespace tl {

int pair_max_active_clusters(int* out) {
    if (int rc = ensure_smem_attr(reinterpret_cast<const void*>(gemm_pair_kernel<false, 1>), kPairDynamicSmem)) return rc;
    if (int rc = ensure_smem_attr(reinterpret_cast<const void*>(gemm_pair_kernel<true, 1>), kPairDynamicSmem)) return rc;
    if (int rc = ensure_smem_attr(reinterpret_cast<const void*>(gemm_pair_kernel<false, 2>), kPairDynamicSmem)) return rc;
    if (int rc = ensure_smem_attr(reinterpret_cast<const void*>(gemm_pair_kernel<true, 2>), kPairDynamicSmem)) return rc;
    if (int rc = ensure_device_info()) return rc;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * dev().sm_count);
    cfg.blockDim = dim3(kPairBigThreads);
    cfg.dynamicSmemBytes = kPairDynamicSmem;
    int n = 0;
    if (int rc = check_cuda(cudaOccupancyMaxActiveClusters(&n, gemm_pair_kernel<false, 2>, &cfg))) return rc;
    *out = n > 0 ? n : 1;
    return TL_OK;
}

int launch_gemm_pair(bool fp8, int halves, int clusters, size_t smem, cudaStream_t stream, const GemmParams& p) {
    if (halves == 2) {
        if (fp8) gemm_pair_kernel<true, 2><<<2 * clusters, kPairBigThreads, smem, stream>>>(p);
        else gemm_pair_kernel<false, 2><<<2 * clusters, kPairBigThreads, smem, stream>>>(p);
    } else {
        if (fp8) gemm_pair_kernel<true, 1><<<2 * clusters, kGemmThreads, smem, stream>>>(p);
        else gemm_pair_kernel<false, 1><<<2 * clusters, kGemmThreads, smem, stream>>>(p);
    }
    return check_cuda(cudaGetLastError());
}

}  // namespace tl
