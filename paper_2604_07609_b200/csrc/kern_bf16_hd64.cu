// Kernel instances: __nv_bfloat16 operands, head_dim 64.
#include "kernels.cuh"
namespace blink {
KernelSet kernels_bf16_hd64(int n_rep, bool pair) { return kernel_set_for<__nv_bfloat16, 64>(n_rep, pair); }
}  // namespace blink
