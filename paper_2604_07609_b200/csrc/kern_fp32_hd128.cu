// Kernel instances: float operands, head_dim 128.
#include "kernels.cuh"
namespace blink {
KernelSet kernels_fp32_hd128(int n_rep, bool pair) { return kernel_set_for<float, 128>(n_rep, pair); }
}  // namespace blink
