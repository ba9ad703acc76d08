// Host-side launch entry points of the kernel families (internal to the library).
#pragma once
#include <cuda_runtime.h>

#include "mkv_common.cuh"

namespace mkv {
// returns false when no instantiation exists for (dtype, head_dim, group)
bool simt_supported(int kv_dtype, int head_dim, int group);
cudaError_t launch_simt(const Params& p, int kv_dtype, cudaStream_t stream);
// CTAs of the kernel the current device keeps resident per SM (its CTAs wait on one another:
// the grid must never exceed SM count x this)
cudaError_t simt_occupancy(int kv_dtype, int head_dim, int group, int* resident_per_sm);
bool mma_supported(int kv_dtype, int head_dim, int group);
int mma_max_stages();          // deepest ring that fits the shared memory of one CTA
cudaError_t mma_occupancy(int stages, int* resident_per_sm);   // also opts in to the ring's shared memory
cudaError_t launch_mma(const Params& p, cudaStream_t stream, bool overlap, int stages);
// recency-window diagnostics over the recorded probabilities of the last step
int diag_max_tokens();
cudaError_t launch_diag(const LayerDev& L, int cap, int window, float* mass, int32_t* count, float* curve,
                        cudaStream_t stream);
}  // namespace mkv
