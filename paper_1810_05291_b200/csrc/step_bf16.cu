// bf16-gradient instantiations of the streaming step kernel.
#include <type_traits>

#include "step_kernel.cuh"

namespace ss {
cudaError_t launch_step_bf16(const StepDesc& s, cudaStream_t st) { return launch_step_dtype<BF16>(s, st); }
}  // namespace ss
