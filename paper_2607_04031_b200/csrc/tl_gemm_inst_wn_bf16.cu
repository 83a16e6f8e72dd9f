// GEMM kernel instantiations: weights on the N side of the MMA, bf16 operands.
#define TL_INST_NAME launch_gemm_wn_bf16
#define TL_INST_WN true
#define TL_INST_FP8 false
#include "tl_gemm_inst.cuh"

namespace tl {

int gemm_max_active_clusters(int size, int* out) {
    auto* kernel = gemm_kernel<64, 256, true, false>;
    if (int rc = ensure_smem_attr(reinterpret_cast<const void*>(kernel), kMaxDynamicSmem)) return rc;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(size) * 64u);
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = 160 * 1024;                      // one CTA per SM, as every plan of this kernel
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = unsigned(size);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (int rc = check_cuda(cudaOccupancyMaxActiveClusters(&n, kernel, &cfg))) return rc;
    *out = n;
    return TL_OK;
}

}  // namespace tl
