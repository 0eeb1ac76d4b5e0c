// fp32-gradient instantiations of the streaming step kernel.
#include <type_traits>

#include "step_kernel.cuh"

namespace ss {
cudaError_t launch_step_f32(const StepDesc& s, cudaStream_t st) { return launch_step_dtype<F32>(s, st); }
}  // namespace ss
