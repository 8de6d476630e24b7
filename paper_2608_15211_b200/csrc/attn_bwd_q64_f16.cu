// The query side of the large-window tcgen05 backward for fp16 activations: the same source, compiled with the fp16 element operations.
#define TERRA_ELEM_F16 1
#include "attn_bwd_q64.cu"
