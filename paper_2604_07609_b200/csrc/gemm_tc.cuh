// Tensor-core path of the dense contractions (tcgen05 + TMEM accumulators fed by
// TMA), bf16 operands, fp32 accumulate.
#pragma once
#include "dev_ctx.cuh"
#include "forward.cuh"

namespace blink {

enum GemmWhich : int { GEMM_QKV = 0, GEMM_O, GEMM_GU, GEMM_DOWN, GEMM_LMHEAD };

struct TcState {
  uint32_t tmem_base;
};
struct TcHost {
  int unused;
};

inline int tc_available() { return 0; }
inline size_t tc_smem_bytes() { return 0; }
inline int tc_host_setup(TcHost&, DevCtx&) { return 0; }
inline void tc_host_free(TcHost&) {}

__device__ __forceinline__ void tc_init(const DevCtx&, float*, TcState& s) { s.tmem_base = 0; }
__device__ __forceinline__ void tc_fini(const DevCtx&, TcState&) {}
__device__ __forceinline__ void phase_gemm_tc(const DevCtx&, const GemmArgs&, int, int, float*, TcState&) {}

}  // namespace blink
