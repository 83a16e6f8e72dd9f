// GEMM kernel instantiations: weights on the M side of the MMA, bf16 operands.
#define TL_INST_NAME launch_gemm_wm_bf16
#define TL_INST_WN false
#define TL_INST_FP8 false
#include "tl_gemm_inst.cuh"
