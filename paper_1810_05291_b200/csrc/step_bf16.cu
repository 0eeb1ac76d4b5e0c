// bf16-gradient instantiations of the streaming step kernel.
#include <type_traits>

#include "step_oct_kernel.cuh"

namespace ss {
cudaError_t launch_step_bf16(const StepDesc& s, cudaStream_t st) { return launch_step_dtype<BF16>(s, st); }
cudaError_t launch_signum_push_bf16(const void* g, float* v, float beta, float omb, int64_t d,
                                   uint32_t* const* dests, int n, bool vec, cudaStream_t st) {
    return launch_signum_push<BF16>(g, v, beta, omb, d, dests, n, vec, st);
}
}  // namespace ss
