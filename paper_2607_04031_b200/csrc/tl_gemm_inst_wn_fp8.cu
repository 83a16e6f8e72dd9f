// GEMM kernel instantiations: weights on the N side of the MMA, FP8 (E4M3) operands.
#define TL_INST_NAME launch_gemm_wn_fp8
#define TL_INST_WN true
#define TL_INST_FP8 true
#include "tl_gemm_inst.cuh"
