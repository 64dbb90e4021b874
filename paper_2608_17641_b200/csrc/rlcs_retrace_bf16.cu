// The same kernels with bfloat16 tensors in global memory (fp32 arithmetic on chip).
#define RLCS_IO_BF16 1
#include "rlcs_retrace.cu"
