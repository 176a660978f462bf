// The fused BGMV kernels that start on their inputs before they join the stream order
// (plora_set_inputs_resident), in a translation unit of their own: see bgmv_lazy_kernel in bgmv.cu.
#define PLORA_BGMV_LAZY_UNIT
#include "bgmv.cu"
