// GEMM kernel instantiations: weights on the N side of the MMA, bf16 operands.
#define TL_INST_NAME launch_gemm_wn_bf16
#define TL_INST_WN true
#define TL_INST_FP8 false
#include "tl_gemm_inst.cuh"
