// Kernel instances: __nv_bfloat16 operands, head_dim 128.
#include "kernels.cuh"
namespace blink {
KernelSet kernels_bf16_hd128(int n_rep, bool pair) { return kernel_set_for<__nv_bfloat16, 128>(n_rep, pair); }
}  // namespace blink
