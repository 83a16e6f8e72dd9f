// Body of one instantiation unit of the GEMM kernel: the including file defines TL_INST_NAME, TL_INST_WN, TL_INST_FP8.
#include "tl_gemm_kernel.cuh"

namespace tl {

template <int kBK, int kBN>
static int launch_one(const cudaLaunchConfig_t* cfg, const GemmParams& p) {
    auto* kernel = gemm_kernel<kBK, kBN, TL_INST_WN, TL_INST_FP8>;
    if (int rc = ensure_smem_attr(reinterpret_cast<const void*>(kernel), kMaxDynamicSmem)) return rc;
    return check_cuda(cudaLaunchKernelEx(cfg, kernel, p));
}

int TL_INST_NAME(int bk, int bn, const cudaLaunchConfig_t* cfg, const GemmParams& p) {
    if (bk == 64) {
        if (bn == 64) return launch_one<64, 64>(cfg, p);
        if (bn == 128) return launch_one<64, 128>(cfg, p);
        if (bn == 256) return launch_one<64, 256>(cfg, p);
    } else if (bk == 128) {
        if (bn == 64) return launch_one<128, 64>(cfg, p);
        if (bn == 128) return launch_one<128, 128>(cfg, p);
        if (bn == 256) return launch_one<128, 256>(cfg, p);
    }
    return TL_ERR_UNSUPPORTED;
}

}  // namespace tl
