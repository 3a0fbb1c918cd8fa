#include "dam_internal.cuh"
cudaError_t dam_launch_scores_sm100(const void*, const void*, const dam_shape_t*, const DamBuildCtx&, float*,
                                    cudaStream_t) { return cudaErrorNotSupported; }
