// Kernel instances: float operands, head_dim 64.
#include "kernels.cuh"
namespace blink {
KernelSet kernels_fp32_hd64(int n_rep, bool pair) { return kernel_set_for<float, 64>(n_rep, pair); }
}  // namespace blink
