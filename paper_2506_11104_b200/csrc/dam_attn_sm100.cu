#include "dam_internal.cuh"
cudaError_t dam_launch_attn_sm100(const void*, const void*, const void*, const void*, const dam_shape_t*, int, float,
                                  void*, float*, void*, cudaStream_t) { return cudaErrorNotSupported; }
