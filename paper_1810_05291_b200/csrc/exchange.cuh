// Host-side declarations for the flag-ordered exchange of packed signs between workers on
// different GPUs (exchange_flags.cu) and the vote + update launch that such an exchange can call off.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/signsgd.h"

namespace ss {

// launch_vote_apply with a guard word in device memory: when it is non-zero at the time the kernel
// starts, every block returns at once and neither the parameters nor the vote words are touched
cudaError_t launch_vote_apply_guarded(const uint32_t* const* packed, int M, int64_t d, uint64_t flip,
                                      float* x, float lr, float wd, bool vec, const ss_segment* seg,
                                      int n_seg, uint32_t* vote, const uint32_t* guard, cudaStream_t st);

}  // namespace ss
