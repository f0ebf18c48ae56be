// The expert FFN kernel for MXFP4 expert weights: the same source as the bf16 kernel, built with the packed
// weight stage and the four expanding warps switched on (see ACM_FFN_MX in ffn.cu).
#define ACM_FFN_MX 1
#include "ffn.cu"
