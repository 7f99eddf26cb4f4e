// Entry points of the per-variant kernel translation units.
#pragma once
namespace blink {
// phases of one step, in execution order (per layer: NORM1 .. DOWN; then the last three)
enum Phase : int {
  PH_NORM1 = 0, PH_QKV, PH_ROPE, PH_ATTN, PH_O, PH_NORM2, PH_GU, PH_SILU, PH_DOWN,
  PH_FNORM, PH_LMHEAD, PH_SAMPLE,
  PH_MOE_GROUP,  // routed experts only: between NORM2 and the per-expert GU phases
  PH_COUNT
};

struct KernelSet {
  const void* loop;   // persistent cooperative loop: (DevCtx)
  const void* phase;  // one phase of one layer: (DevCtx, int phase, int layer, int expert)
};
KernelSet kernels_bf16_hd64(int n_rep, bool pair);
KernelSet kernels_bf16_hd128(int n_rep, bool pair);
KernelSet kernels_fp32_hd64(int n_rep, bool pair);
KernelSet kernels_fp32_hd128(int n_rep, bool pair);
}  // namespace blink
