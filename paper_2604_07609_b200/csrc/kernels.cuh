// The kernels of the serving loop, instantiated per (operand type, head_dim, query heads per
// kv head) so that each instance carries exactly one attention variant: the persistent
// cooperative loop and the one-phase kernel of stepped mode.
#pragma once
#include <cuda_runtime.h>

#include "../../include/blink.h"
#include "attention.cuh"
#include "control.cuh"
#include "dev_ctx.cuh"
#include "forward.cuh"
#include "gemm_tc.cuh"
#include "kernel_set.h"

namespace blink {

template <typename WT, bool PAIR>
__device__ __forceinline__ void gemm_dispatch(const DevCtx& c, const GemmArgs& a, int which, int layer, float* smem,
                                              TcState& tc) {
  if (c.gemm_tc) phase_gemm_tc<PAIR>(c, a, which, layer, smem, tc);
  else phase_gemm_simt<WT>(a);
}

// `T` = rows of the step (read once per step by the caller: it does not change between phases)
template <typename WT, int HD, int NREP, bool PAIR>
__device__ __forceinline__ void run_phase(const DevCtx& c, int phase, int layer, int sub, float* smem, TcState& tc,
                                          AttState& as, int T) {
  const size_t esz = sizeof(WT);
  switch (phase) {
    case PH_NORM1:
      if (c.fused_norm && layer > 0) phase_norm_apply<WT>(c, layer, 0, T);
      else phase_norm<WT>(c, layer, 0, smem);
      break;
    case PH_QKV: {
      GemmArgs a{c.xn, c.w_base + c.w_off[1] + (size_t)layer * c.qkv_dim * c.d * esz, c.qkv, T, c.qkv_dim, c.d,
                 c.qkv_dim, 0};
      a.w_row0 = (long long)layer * c.qkv_dim;
      if (c.fused) a.fix = FIX_ROPE_KV;
      gemm_dispatch<WT, PAIR>(c, a, GEMM_QKV, layer, smem, tc);
    } break;
    case PH_ROPE: phase_rope_kv<WT>(c, layer); break;
    case PH_ATTN:
      if constexpr (sizeof(WT) == 2) phase_attention_bf16<HD, NREP>(c, layer, smem, as);
      else phase_attention<WT, HD, NREP>(c, layer, smem);

      break;
    case PH_O: {
      GemmArgs a{c.attn, c.w_base + c.w_off[2] + (size_t)layer * c.d * c.q_dim * esz, c.h, T, c.d, c.q_dim, c.d, 1};
      a.w_row0 = (long long)layer * c.d;
      if (c.fused_norm) { a.fix = FIX_SUMSQ; a.fix_rowss = c.rowss_a; }
      gemm_dispatch<WT, PAIR>(c, a, GEMM_O, layer, smem, tc);
    } break;
    case PH_NORM2:
      if (c.fused_norm) phase_norm_apply<WT>(c, layer, 1, T);
      else phase_norm<WT>(c, layer, 1, smem);
      break;
    case PH_GU: {
      if (c.E == 0) {
        GemmArgs a{c.xn, c.w_base + c.w_off[3] + (size_t)layer * 2 * c.F * c.d * esz, c.gu, T, 2 * c.F, c.d, 2 * c.F, 0};
        a.w_row0 = (long long)layer * 2 * c.F;
        if (c.fused) { a.fix = FIX_SILU; a.fix_out = c.act; }
        gemm_dispatch<WT, PAIR>(c, a, GEMM_GU, layer, smem, tc);
      } else {
        // expert `sub` on the rows routed to it (gathered, contiguous from moe_off[sub])
        const int off = c.moe_off[sub], cnt = c.moe_off[sub + 1] - off;
        const long long we = (long long)layer * c.E + sub;
        GemmArgs a{reinterpret_cast<const char*>(c.xg) + (size_t)off * c.d * esz, c.w_base + c.w_off[3] + (size_t)we * 2 * c.F * c.d * esz,
                   c.gu + (size_t)off * 2 * c.F, cnt, 2 * c.F, c.d, 2 * c.F, 0};
        a.x_row0 = off;
        a.w_row0 = we * 2 * c.F;
        if (c.fused) { a.fix = FIX_SILU; a.fix_out = reinterpret_cast<char*>(c.act) + (size_t)off * c.F * esz; }
        gemm_dispatch<WT, PAIR>(c, a, GEMM_GU, layer, smem, tc);
      }
    } break;
    case PH_SILU:
      phase_silu_mul<WT>(c, layer, smem);
      break;
    case PH_DOWN: {
      if (c.E == 0) {
        GemmArgs a{c.act, c.w_base + c.w_off[4] + (size_t)layer * c.d * c.F * esz, c.h, T, c.d, c.F, c.d, 1};
        a.w_row0 = (long long)layer * c.d;
        if (c.fused_norm) { a.fix = FIX_SUMSQ; a.fix_rowss = c.rowss_b; }
        gemm_dispatch<WT, PAIR>(c, a, GEMM_DOWN, layer, smem, tc);
      } else {
        const int off = c.moe_off[sub], cnt = c.moe_off[sub + 1] - off;
        const long long we = (long long)layer * c.E + sub;
        GemmArgs a{reinterpret_cast<const char*>(c.act) + (size_t)off * c.F * esz, c.w_base + c.w_off[4] + (size_t)we * c.d * c.F * esz,
                   c.h, cnt, c.d, c.F, c.d, 1};
        a.x_row0 = off;
        a.w_row0 = we * c.d;
        a.row_map = c.moe_tok + off;     // result row i belongs to token moe_tok[off + i], weighted by its gate
        a.row_scale = c.moe_gate + off;
        gemm_dispatch<WT, PAIR>(c, a, GEMM_DOWN, layer, smem, tc);
      }
    } break;
    case PH_MOE_GROUP: phase_moe_group<WT>(c, smem); break;
    case PH_FNORM:
      phase_final_norm<WT>(c);
      break;
    case PH_LMHEAD: {
      GemmArgs a{c.xs, c.w_base + c.w_off[9], c.logits, c.ss->cur_rows, c.V, c.d, c.V, 0};
      gemm_dispatch<WT, PAIR>(c, a, GEMM_LMHEAD, 0, smem, tc);
    } break;
    case PH_SAMPLE: phase_sample(c, smem); break;
    default: break;
  }
}

// ---- persistent loop -----------------------------------------------------------------
template <typename WT, int HD, int NREP, bool PAIR>
__global__ void __launch_bounds__(FWD_THREADS, 1) blink_loop_kernel(const __grid_constant__ DevCtx c) {
  extern __shared__ __align__(1024) float smem[];
  unsigned long long gen = 0;   // arrivals this CTA expects at its next grid barrier
  long long launch_iters = 0;
  TcState tc;
  tc_init<PAIR>(c, smem, tc);
  AttState as;
  att_init(c, as);
  while (true) {
    if (blockIdx.x == 0) control_phase(c, launch_iters);
    if (!grid_barrier(c, gen)) break;
    if (*(volatile int*)&c.ss->cmd != CMD_RUN) break;
    if (!c.control_only) {
      bool ok = true;
      // CTA 0 keeps a per-phase-kind device time of the open iteration (a phase's time includes
      // the barrier that closes it); recorded only when per-iteration statistics are kept
      const bool timed = c.stats_cap > 0 && blockIdx.x == 0 && threadIdx.x == 0;
      uint64_t t_prev = timed ? global_timer_ns() : 0;
      const int T = __ldcg(&c.ss->cur_T);   // fixed for the whole step: one L2 read instead of one per phase
      auto step_phase = [&](int ph, int layer, int sub) {
        if (c.fused && (ph == PH_ROPE || ph == PH_SILU)) return;   // done by the epilogues of the QKV and gate/up GEMMs
        // The experts' GEMMs are independent of one another (own weights, own gathered rows; the down
        // projections add into the residual rows with reductions): one grid barrier after the last
        // expert, none in between, so every CTA streams its share of all experts back to back.  (With
        // fused epilogues the barriers stay: their tile counters are per GEMM.)
        const bool barrier = !(c.E > 0 && !c.fused && (ph == PH_GU || ph == PH_DOWN) && sub + 1 < c.E);
        run_phase<WT, HD, NREP, PAIR>(c, ph, layer, sub, smem, tc, as, T);
        if (!barrier) return;
        ok = grid_barrier(c, gen);
        if (timed) { const uint64_t t = global_timer_ns(); c.ss->cur_phase_ns[ph] += t - t_prev; t_prev = t; }
      };
      for (int layer = 0; layer < c.L && ok; ++layer) {
        for (int ph = PH_NORM1; ph <= PH_DOWN && ok; ++ph) {
          if (c.E > 0 && (ph == PH_GU || ph == PH_DOWN)) {
            if (ph == PH_GU) step_phase(PH_MOE_GROUP, layer, 0);   // routing lists and gathered rows first
            for (int e = 0; e < c.E && ok; ++e) step_phase(ph, layer, e);
          } else {
            step_phase(ph, layer, 0);
          }
        }
      }
      for (int ph = PH_FNORM; ph <= PH_SAMPLE && ok; ++ph) step_phase(ph, 0, 0);
      if (!ok) break;
    } else if (!grid_barrier(c, gen)) break;
  }
  tc_fini<PAIR>(c, tc);
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    const int aborted = *(volatile int*)&c.ss->abort_flag;
    __threadfence_system();
    c.mbox->loop_state = aborted ? (uint32_t)BLINK_LOOP_EXIT_ERROR : (uint32_t)c.ss->exit_reason;
    __threadfence_system();
  }
}

template <typename WT, int HD, int NREP, bool PAIR>
__global__ void __launch_bounds__(FWD_THREADS, 1) blink_phase_kernel(const __grid_constant__ DevCtx c, int phase, int layer, int sub) {
  extern __shared__ __align__(1024) float smem[];
  if (c.ss->cmd != CMD_RUN) return;
  TcState tc;
  tc_init<PAIR>(c, smem, tc);
  AttState as;
  att_init(c, as);
  run_phase<WT, HD, NREP, PAIR>(c, phase, layer, sub, smem, tc, as, c.ss->cur_T);
  tc_fini<PAIR>(c, tc);
}

// `pair`: the variant whose GEMMs run on CTA pairs (tcgen05 cta_group::2; launched with clusters of two).
// Built for 16-bit operands with four query heads per kv head, the shape of the large configurations.
template <typename WT, int HD>
inline KernelSet kernel_set_for(int n_rep, bool pair) {
  if (pair) {
    if constexpr (sizeof(WT) == 2) {
      if (n_rep == 4) return {(const void*)blink_loop_kernel<WT, HD, 4, true>, (const void*)blink_phase_kernel<WT, HD, 4, true>};
    }
    return {nullptr, nullptr};
  }
  switch (n_rep) {
    case 1: return {(const void*)blink_loop_kernel<WT, HD, 1, false>, (const void*)blink_phase_kernel<WT, HD, 1, false>};
    case 2: return {(const void*)blink_loop_kernel<WT, HD, 2, false>, (const void*)blink_phase_kernel<WT, HD, 2, false>};
    case 4: return {(const void*)blink_loop_kernel<WT, HD, 4, false>, (const void*)blink_phase_kernel<WT, HD, 4, false>};
    case 8: return {(const void*)blink_loop_kernel<WT, HD, 8, false>, (const void*)blink_phase_kernel<WT, HD, 8, false>};
    default: return {nullptr, nullptr};
  }
}

}  // namespace blink
