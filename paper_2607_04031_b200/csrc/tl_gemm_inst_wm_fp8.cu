// GEMM kernel instantiations: weights on the M side of the MMA, FP8 (E4M3) operands.
#define TL_INST_NAME launch_gemm_wm_fp8
#define TL_INST_WN false
#define TL_INST_FP8 true
#include "tl_gemm_inst.cuh"
