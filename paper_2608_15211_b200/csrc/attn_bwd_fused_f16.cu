// The small-window tcgen05 backward kernel for fp16 activations: the same source, compiled with the fp16 element operations.
#define TERRA_ELEM_F16 1
#include "attn_bwd_fused.cu"
