// Tensor-core path of the dense contractions: tcgen05.mma with TMEM accumulators, operands
// staged in shared memory by TMA (128-byte swizzle), bf16 x bf16 -> fp32.
//
//   out[t][n] (+)= sum_k x[t][k] * w[n][k]
//
// Operand roles are swapped relative to the usual GEMM: the 128 rows of an MMA tile are
// rows of W (output features), the MMA's N is the token tile (16..256 rows of x).  Decode
// steps have few tokens and stream every weight once, so the weight tile fills the fixed
// 128-row dimension and the token count only sets the cheap N.
//
// Work split ("stream-K"): the (n-tile, k-block) units of one GEMM are flattened and cut into
// equal contiguous ranges, one per CTA, so every SM streams the same number of weight bytes
// whatever the shape.  A CTA's range is a handful of segments (one n-tile each); a segment that
// covers the whole K of its tile stores its result, a partial one adds it with
// red.global.add.f32 (the output is zeroed or already holds the residual).  With few n-tiles
// every tile gets the same whole number of CTAs (one partial tile per CTA); with more than 256
// token rows the passes of a weight tile go to neighbouring CTAs that walk the same range at the
// same time (the tile comes from HBM once, from L2 for the other passes).
//
// Warp roles in the 256-thread CTA: warp 0 = weight producer (one lane), warp 2 = token-tile
// producer (one lane), warp 1 = MMA issuer (one lane), warps 4..7 = epilogue (TMEM -> registers
// -> global), two accumulator buffers of 256 TMEM columns so the epilogue of one segment
// overlaps the MMAs of the next; warps 0..3 store half of the CTA's last accumulator.
// Every wait is bounded: on a time-out the CTA records DEV_ERR_PIPE_TIMEOUT, raises the
// loop's abort flag and skips all further waits.
#pragma once
#include <cuda.h>

#include "control.cuh"
#include "dev_ctx.cuh"
#include "forward.cuh"

namespace blink {

enum GemmWhich : int { GEMM_QKV = 0, GEMM_O, GEMM_GU, GEMM_DOWN, GEMM_LMHEAD, GEMM_KINDS };
enum ActBuf : int { ACT_XN = 0, ACT_ATTN, ACT_ACT, ACT_XS, ACT_XG, ACT_BUFS };
constexpr int TC_BOXES = 5;  // token-tile boxes of 16, 32, 64, 128, 256 rows
constexpr int TC_MAX_STAGES = 8;
constexpr int TC_A_BYTES = 128 * 128;  // 128 weight rows x 64 bf16
constexpr int TC_TILE_BUDGET = 196608;

// Per-thread pipeline bookkeeping that survives from one GEMM phase to the next (the
// mbarriers are initialised once per kernel).  Bit s of a mask is the parity of the next
// phase to wait for on barrier s; only the thread that owns a role uses its masks.
struct TcState {
  uint32_t tmem_base;
  uint32_t fill_bits;   // producer: stages filled so far, parity per stage
  uint32_t use_bits;    // MMA issuer: stages consumed so far, parity per stage
  uint32_t acc_mma;     // MMA issuer: accumulator buffers claimed, parity per buffer
  uint32_t acc_epi;     // epilogue: accumulator buffers drained, parity per buffer
  uint32_t last_bit;    // warps 0-3: parity of the next "last accumulator complete" signal
};

struct TcShared {
  uint64_t full[TC_MAX_STAGES], empty[TC_MAX_STAGES], acc_full[2], acc_empty[2];
  uint64_t acc_last;   // completes once per GEMM phase, when the CTA's last accumulator is complete
  uint32_t tmem;
  int dead;
};
__shared__ __align__(8) TcShared g_tc;

struct TcHost {
  void* d_maps = nullptr;
};

// ---- PTX wrappers -------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  `dead` (shared) is set by whoever times out first; once set every wait returns at once.
__device__ __forceinline__ bool mbar_wait(const DevCtx& c, uint64_t* bar, uint32_t parity, volatile int* dead) {
  if (*dead) return false;
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  unsigned int spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255u) == 0) {
      if (*dead) return false;
      if ((unsigned long long)(clock64() - t0) > c.barrier_timeout_cycles) {
        *dead = 1;
        dev_fail(c, DEV_ERR_PIPE_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_u32(smem_dst)),
      "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}

// L2 policy for data that is read once per step (weights, the KV cache): evicted first, so that
// the streams do not push the step's activations out of L2.  Reductions into an evicted output
// line have to fetch it from HBM first and run several times slower.
__device__ __forceinline__ uint64_t l2_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tma_load_2d_hint(void* smem_dst, const CUtensorMap* map, int x, int y, uint64_t* bar,
                                                 uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], "
      "[%4], %5;" ::"r"(smem_u32(smem_dst)),
      "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tma_bulk_load_hint(void* smem_dst, const void* src, uint32_t bytes, uint64_t* bar,
                                                   uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
          smem_u32(smem_dst)),
      "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}

__device__ __forceinline__ void tma_bulk_load(void* smem_dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(smem_dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]^T, M = 128, K = 16 per instruction
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on `bar` once all MMAs issued so far by this thread have completed
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
// fp32 reduction into global memory, no return value (the pointer is known to be global here)
__device__ __forceinline__ void red_add_f32(float* p, float v) {
  asm volatile("red.relaxed.gpu.global.add.f32 [%0], %1;" ::"l"(__cvta_generic_to_global(p)), "f"(v) : "memory");
}
// 32 lanes x 16 consecutive 32-bit columns -> 16 registers per thread
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, "
      "[%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor: K-major tile of rows x 64 bf16 (128-byte rows), 128-byte
// swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);  // start address, 16-byte units
  d |= (uint64_t)1 << 16;                    // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;          // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                    // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                    // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 A and B (both K-major), fp32 accumulator, M = 128, N = n.
__device__ __forceinline__ uint32_t idesc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

// ---- CTA pairs (tcgen05 cta_group::2) ------------------------------------------------------------------
// Two CTAs of a cluster work on one MMA of 256 weight rows: each stages its own 128-row weight tile and
// half of the token tile (N / 2 rows), CTA 0 issues the MMAs, each CTA receives its 128 rows of the
// result in its own TMEM.  Per k-block a CTA fills 16 KiB of weights + half a token tile instead of a
// whole one.  No multicast loads: every CTA fetches its operands itself.
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrive (optionally announcing `bytes` of copies) on the barrier at the same shared-memory offset in CTA 0 of the pair
__device__ __forceinline__ void mbar_expect_tx_cta0(uint64_t* bar, uint32_t bytes) {
  asm volatile(
      "{\n\t.reg .b32 ra;\n\t"
      "mapa.shared::cluster.u32 ra, %0, 0;\n\t"
      "mbarrier.arrive.expect_tx.shared::cluster.b64 _, [ra], %1;\n\t}" ::"r"(smem_u32(bar)),
      "r"(bytes)
      : "memory");
}
__device__ __forceinline__ void mbar_arrive_cta0(uint64_t* bar) {
  asm volatile(
      "{\n\t.reg .b32 ra;\n\t"
      "mapa.shared::cluster.u32 ra, %0, 0;\n\t"
      "mbarrier.arrive.shared::cluster.b64 _, [ra];\n\t}" ::"r"(smem_u32(bar))
      : "memory");
}
// Tile copies of a pair: the bytes are counted on CTA 0's barrier (the CTA bit of the barrier's address is
// cleared), whichever CTA of the pair issues the copy and receives the data.
constexpr uint32_t PAIR_CTA0_MASK = 0xFEFFFFFFu;
__device__ __forceinline__ void tma_pair_load_2d(void* smem_dst, const CUtensorMap* map, int x, int y, uint64_t* bar,
                                                 uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%2, %3}], [%4], %5;" ::"r"(smem_u32(smem_dst)),
      "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar) & PAIR_CTA0_MASK), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tma_pair_load_3d(void* smem_dst, const CUtensorMap* map, int x, int y, int z, uint64_t* bar,
                                                 uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%2, %3, %4}], [%5], %6;" ::"r"(smem_u32(smem_dst)),
      "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar) & PAIR_CTA0_MASK), "l"(policy)
      : "memory");
}
__device__ __forceinline__ uint64_t l2_evict_normal() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
  return p;
}
// D[tmem of both CTAs] (+)= A[smem of both CTAs] * B[smem of both CTAs]^T, M = 256 (128 per CTA), K = 16
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on `bar` in both CTAs of the pair once all MMAs issued so far have completed
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
          smem_u32(bar)),
      "h"((uint16_t)3)
      : "memory");
}
__device__ __forceinline__ uint32_t idesc_bf16_pair(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}

// The same wait for warps that have nothing else to do for most of a phase: sleep between polls.
__device__ __forceinline__ bool mbar_wait_idle(const DevCtx& c, uint64_t* bar, uint32_t parity, volatile int* dead) {
  if (*dead) return false;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    __nanosleep(200);
    if (*dead) return false;
    if ((unsigned long long)(clock64() - t0) > c.barrier_timeout_cycles) {
      *dead = 1;
      dev_fail(c, DEV_ERR_PIPE_TIMEOUT);
      return false;
    }
  }
  return true;
}

// ---- TMEM allocation for the life of the kernel ---------------------------------------------
template <bool PAIR>
__device__ __forceinline__ void tc_init(const DevCtx& c, float*, TcState& s) {
  s.tmem_base = 0;
  s.fill_bits = s.use_bits = s.acc_mma = s.acc_epi = s.last_bit = 0;
  if (!c.gemm_tc) return;
  if (threadIdx.x == 32) {
    // pairs: the operands of a stage come from four producers (two per CTA), counted on CTA 0's barrier;
    // an accumulator is free again when the epilogue warps of both CTAs have drained it
    for (int i = 0; i < TC_MAX_STAGES; ++i) { mbar_init(&g_tc.full[i], PAIR ? 4 : 2); mbar_init(&g_tc.empty[i], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&g_tc.acc_full[b], 1); mbar_init(&g_tc.acc_empty[b], PAIR ? 8 : 4); }
    mbar_init(&g_tc.acc_last, 1);
    g_tc.dead = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < 32) {
    if constexpr (PAIR) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&g_tc.tmem)) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&g_tc.tmem)) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if constexpr (PAIR) cluster_sync_all();   // both CTAs' barriers exist before either touches the other's
  tc_fence_after();
  s.tmem_base = *(volatile uint32_t*)&g_tc.tmem;
}
template <bool PAIR>
__device__ __forceinline__ void tc_fini(const DevCtx& c, TcState& s) {
  if (!c.gemm_tc) return;
  tc_fence_before();
  __syncthreads();
  if constexpr (PAIR) cluster_sync_all();   // the other CTA no longer signals into this one's shared memory
  if (threadIdx.x < 32) {
    tc_fence_after();
    if constexpr (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;" ::"r"(s.tmem_base) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(s.tmem_base) : "memory");
  }
}

struct TcMaps {
  CUtensorMap w[GEMM_KINDS];
  CUtensorMap act[ACT_BUFS][TC_BOXES];
  CUtensorMap ws[GEMM_KINDS][2];   // streaming layout seen as [tiles][128][64]: box of one tile, of two consecutive tiles
};

// Where the epilogue's results go; held in registers by the warps that store (the arguments live
// in the caller's frame, and a reload after every reduction would serialise them).
struct TcEpiOut {
  float* out;
  size_t ldo;
  const int* row_map;
  const float* row_scale;
  int T, N;
  int ilv_F;               // gate/up rows interleaved in the weight tiles: row n is output column (n & 1) * F + (n >> 1)
  __nv_bfloat16* act;      // non-null: a tile whose sums are complete goes straight to act = silu(gate) * up
};
// columns [c_begin, c_end) of an accumulator (token rows t_base + column) -> out; lane = weight row n
__device__ __forceinline__ void tc_epi_columns(const TcEpiOut& e, uint32_t taddr, int n, int t_base, int c_begin, int c_end,
                                               bool plain) {
  for (int c0 = c_begin; c0 < c_end; c0 += 16) {
    float v[16];
    tmem_ld16(taddr + (uint32_t)c0, v);
    if (n < e.N) {
      const int t0 = t_base + c0;
      const int nv = min(16, e.T - t0);   // token rows of this group that exist
      const int n_out = e.ilv_F ? (n & 1) * e.ilv_F + (n >> 1) : n;
      if (e.row_map != nullptr) {
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (j < nv) red_add_f32(e.out + (size_t)e.row_map[t0 + j] * e.ldo + n_out, e.row_scale[t0 + j] * v[j]);
      } else {
        float* o = e.out + (size_t)t0 * e.ldo + n_out;
        if (plain) {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (j < nv) o[(size_t)j * e.ldo] = v[j];
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (j < nv) red_add_f32(o + (size_t)j * e.ldo, v[j]);
        }
      }
    }
  }
}
// Gate/up tile whose K is complete in this accumulator (rows interleaved: lane 2 i holds the gate row and lane
// 2 i + 1 the up row of feature n / 2): the pair of lanes exchanges its values and writes
// act = silu(gate) * up in the operand type, eight of the sixteen token columns each.  Nothing goes to the
// fp32 gate/up buffer and the SwiGLU phase skips the tile.
__device__ __forceinline__ void tc_epi_silu(const TcEpiOut& e, uint32_t taddr, int n, int t_base, int c_begin, int c_end) {
  const bool even = (n & 1) == 0;
  const int f = n >> 1;
  const int F = e.ilv_F;
  for (int c0 = c_begin; c0 < c_end; c0 += 16) {
    float v[16], o[16];
    tmem_ld16(taddr + (uint32_t)c0, v);
#pragma unroll
    for (int j = 0; j < 16; ++j) o[j] = __shfl_xor_sync(0xffffffffu, v[j], 1);
    if (n < e.N) {
      const int t0 = t_base + c0;
      const int nv = min(16, e.T - t0);
#pragma unroll
      for (int jj = 0; jj < 8; ++jj) {
        const int j = even ? jj : jj + 8;
        const float g = even ? v[jj] : o[jj + 8];
        const float u = even ? o[jj] : v[jj + 8];
        // approximate division (2 ulp before the rounding to bf16): the exact one is a call to a subroutine,
        // which costs every phase of the loop kernel, not only this one
        if (j < nv) e.act[(size_t)(t0 + j) * F + f] = __float2bfloat16_rn(__fdividef(g, 1.0f + __expf(-g)) * u);
      }
    }
  }
}
// what the gate/up GEMM of this step and layer writes beside a tile it has turned into activations
__device__ __forceinline__ unsigned long long gu_stamp(const DevCtx& c, int layer) { return c.ss->iter * (unsigned long long)c.L + (unsigned long long)layer + 1ull; }
// First column of a CTA's last accumulator that warps 0-3 store (they have no role left by
// then).  Below 128 columns the reduction is short and the extra waiting warps cost more.
__device__ __forceinline__ int tc_epi_half(int n_mma) { return n_mma >= 128 ? ((n_mma / 16 + 1) / 2) * 16 : n_mma; }

// ---- the GEMM phase -----------------------------------------------------------------------------
// Shape of one GEMM's pipeline for the current step; every role derives the same numbers.
struct TcGeom {
  int kblocks, ntiles, passes, box_id, box_rows, load_box, KPS, S;
  int pass_fixed, pdiv;   // one token pass per CTA (or -1), and the passes interleaved in its unit order
  uint32_t b_bytes, stage_bytes;
  long long u0, u1;
};
__device__ __forceinline__ TcGeom tc_geom(const DevCtx& c, int T, int N, int K, bool whole_tiles, int nb, int b, int ntiles, bool half_tokens) {
  TcGeom g;
  g.kblocks = K / 64;
  g.ntiles = ntiles;   // weight tiles of 128 rows, or pairs of them
  g.passes = (T + 255) / 256;
  g.box_id = TC_BOXES - 1;
  if (g.passes == 1) {
    g.box_id = 0;
    while ((16 << g.box_id) < T) ++g.box_id;
  }
  g.box_rows = 16 << g.box_id;
  // A stage holds one k-block, or two when the token tile is small and the weights are stored as
  // contiguous tiles (then one bulk copy brings 32 KiB): fewer, larger copies per producer step.
  g.KPS = (c.w_streaming && g.box_rows <= 128) ? 2 : 1;
  // pairs: each CTA stages half of the token rows of a pass (the box that covers n_mma / 2 rows)
  g.load_box = half_tokens ? (g.box_id > 0 ? g.box_id - 1 : 0) : g.box_id;
  g.b_bytes = (uint32_t)(16 << g.load_box) * 128u;
  g.stage_bytes = (uint32_t)g.KPS * (TC_A_BYTES + g.b_bytes);
  g.S = TC_TILE_BUDGET / (int)g.stage_bytes;
  if (g.S > TC_MAX_STAGES) g.S = TC_MAX_STAGES;
  const long long total = (long long)g.passes * g.ntiles * g.kblocks;
  g.u0 = total * b / nb;
  g.u1 = total * (b + 1) / nb;
  g.pass_fixed = -1;
  g.pdiv = g.passes;
  if (whole_tiles && g.passes == 1) {
    // every worker gets whole weight tiles (at most one more than its neighbours): no partial sums at all
    g.u0 = (long long)g.kblocks * ((long long)g.ntiles * b / nb);
    g.u1 = (long long)g.kblocks * ((long long)g.ntiles * (b + 1) / nb);
    return g;
  }
  // More than 256 token rows: the passes of a weight tile go to neighbouring workers, which walk the
  // same (weight tile, k-block) range at the same time, so the tile comes from HBM once and from
  // L2 for the others.  One worker doing the passes in turn re-reads it after the whole grid has
  // streamed more than L2 holds in between.
  if (g.passes > 1 && nb >= g.passes) {
    const int groups = nb / g.passes;
    const long long units = (long long)g.ntiles * g.kblocks;
    g.pdiv = 1;
    if (b < groups * g.passes) {
      const int grp = b / g.passes;
      g.pass_fixed = b % g.passes;
      g.u0 = units * grp / groups;
      g.u1 = units * (grp + 1) / groups;
    } else {
      g.pass_fixed = 0;
      g.u0 = g.u1 = 0;
    }
  }
  // Few weight tiles (QKV, O, down at decode sizes): give every tile the same whole number of
  // workers, so that no range crosses a tile and each has one partial tile to reduce at the
  // end instead of two.  The longest range grows by (per * nb - total) / nb k-blocks of about
  // 0.4 us each; the saved reduction takes about 0.018 us per token row.
  const int split = nb / g.ntiles;
  if (g.passes == 1 && split >= 2) {
    const int per = (g.kblocks + split - 1) / split;
    if (((long long)per * nb - total) * 23 < (long long)T * nb) {
      if (b < g.ntiles * split) {
        const int nt = b / split, part = b % split;
        g.u0 = (long long)nt * g.kblocks + (long long)g.kblocks * part / split;
        g.u1 = (long long)nt * g.kblocks + (long long)g.kblocks * (part + 1) / split;
      } else {
        g.u0 = g.u1 = 0;
      }
    }
  }
  return g;
}
// position of unit u: weight tile and token pass (the k-block is u % kblocks)
__device__ __forceinline__ int tc_unit_nt(const TcGeom& g, long long u) { return (int)(u / ((long long)g.kblocks * g.pdiv)); }
__device__ __forceinline__ int tc_unit_pass(const TcGeom& g, long long u) {
  return g.pass_fixed >= 0 ? g.pass_fixed : (int)((u / g.kblocks) % g.passes);
}
// tiles need 1024-byte alignment for the 128-byte swizzle
__device__ __forceinline__ char* tc_tiles(float* smem_f) {
  const uint32_t raw = smem_u32(smem_f);
  return reinterpret_cast<char*>(smem_f) + (((raw + 1023u) & ~1023u) - raw);
}

// In pair mode a unit names a PAIR of weight tiles (2 nt, 2 nt + 1): CTA r of the pair owns tile 2 nt + r.
template <bool PAIR>
__device__ __forceinline__ int tc_my_tile(int nt_unit, uint32_t rank) { return PAIR ? 2 * nt_unit + (int)rank : nt_unit; }

// Weight producer (one thread): stream the weight tiles of this CTA's range through the ring.
template <bool PAIR>
__device__ __forceinline__ void tc_produce_weights(const DevCtx& c, const void* w, long long w_row0, int which,
                                                   const TcGeom& g, char* tiles, TcState& tc, uint32_t rank) {
  const TcMaps* maps = reinterpret_cast<const TcMaps*>(c.tc_maps);
  const CUtensorMap* map_a = &maps->w[which];
  const int row_a0 = (int)w_row0;
  volatile int* dead = &g_tc.dead;
  const uint64_t stream_policy = l2_evict_first();
  long long u = g.u0;
  int stage = 0;
  while (u < g.u1) {
    const long long seg_end = min(g.u1, (u / g.kblocks + 1) * (long long)g.kblocks);
    const int nk = (int)min((long long)g.KPS, seg_end - u);
    const int kb = (int)(u % g.kblocks);
    const int nt = tc_my_tile<PAIR>(tc_unit_nt(g, u), rank);
    // the n-th fill of a stage waits for its (n-1)-th release
    if (!mbar_wait(c, &g_tc.empty[stage], ((tc.fill_bits >> stage) & 1u) ^ 1u, dead)) break;
    tc.fill_bits ^= 1u << stage;
    char* sa = tiles + (size_t)stage * g.stage_bytes;
    if constexpr (PAIR) {
      mbar_expect_tx_cta0(&g_tc.full[stage], (uint32_t)nk * TC_A_BYTES);
      if (c.w_streaming) {   // tile index inside the whole tensor; one or two consecutive tiles per copy
        const int tile = (int)(((w_row0 >> 7) + nt) * g.kblocks + kb);
        tma_pair_load_3d(sa, &maps->ws[which][nk - 1], 0, 0, tile, &g_tc.full[stage], stream_policy);
      } else {
        tma_pair_load_2d(sa, map_a, kb * 64, row_a0 + nt * 128, &g_tc.full[stage], stream_policy);
      }
    } else {
      mbar_expect_tx(&g_tc.full[stage], (uint32_t)nk * TC_A_BYTES);
      if (c.w_streaming) {  // contiguous tiles, already in the shared-memory operand image
        tma_bulk_load_hint(sa, reinterpret_cast<const char*>(w) + ((size_t)nt * g.kblocks + kb) * TC_A_BYTES,
                           (uint32_t)nk * TC_A_BYTES, &g_tc.full[stage], stream_policy);
      } else {
        tma_load_2d_hint(sa, map_a, kb * 64, row_a0 + nt * 128, &g_tc.full[stage], stream_policy);
      }
    }
    u += nk;
    if (++stage == g.S) stage = 0;
  }
}

// ---- consumers of finished output tiles -------------------------------------------------------------
// Every CTA adds the number of k-blocks it contributed to an output tile to that tile's counter once
// its partial sums are in memory; the CTA whose addition completes the tile (all K / 64 k-blocks; for
// gate/up the gate tile and its up tile share a counter) runs the GEMM's element-wise consumer on it:
// the finished fp32 tile is still in L2.  Counters return to zero for the next GEMM.
static __device__ __noinline__ void tc_finish_tiles(const DevCtx& c, const GemmArgs& a, const TcGeom& g, int layer) {
  constexpr int BATCH = 16;
  __shared__ int s_fin[BATCH];
  __shared__ int s_nfin;
  __shared__ long long s_next;
  // gate/up: with plain rows gate tile j and up tile j + ntiles / 2 share slot j; with interleaved rows one
  // weight tile holds gate and up of 64 features
  const bool two_tiles = a.fix == FIX_SILU && !c.w_streaming;
  const int ntiles_slot = two_tiles ? g.ntiles / 2 : g.ntiles;
  const int need = (two_tiles ? 2 : 1) * g.kblocks;
  long long u = g.u0;
  while (u < g.u1) {   // uniform over the CTA
    if (threadIdx.x == 0) {
      int n = 0;
      __threadfence();   // the CTA's partial sums (ordered before by the barrier above) before the counters
      while (u < g.u1 && n < BATCH) {
        const long long seg_end = min(g.u1, (u / g.kblocks + 1) * (long long)g.kblocks);
        const int nt = tc_unit_nt(g, u), pass = tc_unit_pass(g, u);
        const int units = (int)(seg_end - u);
        const int tile = nt % ntiles_slot;
        const int slot = (pass * ntiles_slot + tile) % TILE_CNT_SLOTS;
        const int old = atomicAdd(&c.tile_cnt[slot], units);
        if (old + units == need) {
          c.tile_cnt[slot] = 0;   // nobody touches this counter again before the next grid barrier
          s_fin[n++] = (pass << 16) | tile;
        }
        u = seg_end;
      }
      if (n > 0) __threadfence();
      s_nfin = n;
      s_next = u;
    }
    __syncthreads();
    const int n = s_nfin;
    u = s_next;
    for (int i = 0; i < n; ++i) {
      const int tile = s_fin[i] & 0xffff, pass = s_fin[i] >> 16;
      const int t0 = pass * 256, t1 = min(a.M, t0 + 256);
      if (a.fix == FIX_ROPE_KV) fixup_rope_kv<__nv_bfloat16>(c, layer, tile, t0, t1);
      else if (a.fix == FIX_SILU) fixup_silu<__nv_bfloat16>(a.out, reinterpret_cast<__nv_bfloat16*>(a.fix_out), a.N / 2, two_tiles ? tile * 128 : tile * 64, two_tiles ? 128 : 64, t0, t1);
      else fixup_sumsq(a.out, a.ldo, a.N, a.fix_rowss, tile, t0, t1);
    }
    __syncthreads();
  }
}

template <bool PAIR>
static __device__ __noinline__ void phase_gemm_tc(const DevCtx& c, const GemmArgs& a, int which, int layer, float* smem_f, TcState& tc) {
  const int T = a.M, N = a.N, K = a.K;
  if (T <= 0) return;  // uniform over the grid
  // gate/up on the streaming layout: weight rows are interleaved (gate f, up f, ...), and in a dense model
  // a tile whose sums are complete in one accumulator goes straight to the activation rows
  const int ilv_F = (which == GEMM_GU && c.w_streaming) ? c.F : 0;
  __nv_bfloat16* const act_direct = (which == GEMM_GU && gu_direct_step(c, T)) ? reinterpret_cast<__nv_bfloat16*>(c.act) : nullptr;
  const TcMaps* maps = reinterpret_cast<const TcMaps*>(c.tc_maps);
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
  const int n_tiles128 = (N + 127) / 128;
  // workers are CTAs, or CTA pairs that take two weight tiles at a time
  const TcGeom g = PAIR ? tc_geom(c, T, N, K, which == GEMM_LMHEAD && lm_head_whole_tiles(c), (int)gridDim.x / 2,
                                  (int)blockIdx.x / 2, (n_tiles128 + 1) / 2, true)
                        : tc_geom(c, T, N, K, which == GEMM_LMHEAD && lm_head_whole_tiles(c), (int)gridDim.x, (int)blockIdx.x,
                                  n_tiles128, false);
  const int kblocks = g.kblocks, KPS = g.KPS, S = g.S;
  const uint32_t b_bytes = g.b_bytes, stage_bytes = g.stage_bytes;
  const int act_id = which == GEMM_O ? ACT_ATTN : which == GEMM_DOWN ? ACT_ACT : which == GEMM_LMHEAD ? ACT_XS
                     : (which == GEMM_GU && c.E > 0) ? ACT_XG : ACT_XN;
  const CUtensorMap* map_b = &maps->act[act_id][g.load_box];
  char* tiles = tc_tiles(smem_f);
  const long long u0 = g.u0, u1 = g.u1;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* dead = &g_tc.dead;

  if (warp == 0) {
    if (lane == 0) {
      tc_produce_weights<PAIR>(c, a.w, a.w_row0, which, g, tiles, tc, rank);
    }
  } else if (warp == 2) {
    // token-tile producer: walks the same sequence of stages (nk k-blocks of one segment each)
    if (lane == 0) {
      const int x_row0 = a.x_row0;
      const uint64_t keep_policy = l2_evict_normal();
      int stage = 0;
      long long u = u0;
      while (u < u1) {
        const long long seg_end = min(u1, (u / kblocks + 1) * (long long)kblocks);
        const int nk = (int)min((long long)KPS, seg_end - u);
        const int kb = (int)(u % kblocks);
        const int pass = tc_unit_pass(g, u);
        if (!mbar_wait(c, &g_tc.empty[stage], ((tc.fill_bits >> stage) & 1u) ^ 1u, dead)) break;
        tc.fill_bits ^= 1u << stage;
        char* sa = tiles + (size_t)stage * stage_bytes;
        if constexpr (PAIR) {
          // this CTA's half of the pass: rows [rank * n_mma / 2, + n_mma / 2) (the box may reach further)
          const int n_mma = (min(256, T - pass * 256) + 15) & ~15;
          const int row0 = x_row0 + pass * 256 + (int)rank * (n_mma / 2);
          mbar_expect_tx_cta0(&g_tc.full[stage], (uint32_t)nk * b_bytes);
          for (int j = 0; j < nk; ++j)
            tma_pair_load_2d(sa + KPS * TC_A_BYTES + j * b_bytes, map_b, (kb + j) * 64, row0, &g_tc.full[stage], keep_policy);
        } else {
          mbar_expect_tx(&g_tc.full[stage], (uint32_t)nk * b_bytes);
          for (int j = 0; j < nk; ++j)
            tma_load_2d(sa + KPS * TC_A_BYTES + j * b_bytes, map_b, (kb + j) * 64, x_row0 + pass * 256, &g_tc.full[stage]);
        }
        u += nk;
        if (++stage == S) stage = 0;
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {   // pairs: CTA 0 issues the MMAs for both
      int stage = 0;
      int abuf = 0;
      long long u = u0;
      while (u < u1) {
        const long long seg_end = min(u1, (u / kblocks + 1) * (long long)kblocks);
        const int pass = tc_unit_pass(g, u);
        const int rows = min(256, T - pass * 256);
        const int n_mma = (rows + 15) & ~15;
        const uint32_t idesc = PAIR ? idesc_bf16_pair(n_mma) : idesc_bf16(n_mma);
        const uint32_t d_tmem = tc.tmem_base + (uint32_t)abuf * 256u;
        if (!mbar_wait(c, &g_tc.acc_empty[abuf], ((tc.acc_mma >> abuf) & 1u) ^ 1u, dead)) break;
        tc.acc_mma ^= 1u << abuf;
        tc_fence_after();
        bool first = true;
        bool ok = true;
        while (u < seg_end) {
          const int nk = (int)min((long long)KPS, seg_end - u);
          if (!mbar_wait(c, &g_tc.full[stage], (tc.use_bits >> stage) & 1u, dead)) { ok = false; break; }
          tc.use_bits ^= 1u << stage;
          tc_fence_after();
          const uint32_t sa = smem_u32(tiles + (size_t)stage * stage_bytes);
          for (int j = 0; j < nk; ++j) {
            const uint64_t da = smem_desc_sw128(sa + j * TC_A_BYTES);
            const uint64_t db = smem_desc_sw128(sa + KPS * TC_A_BYTES + j * b_bytes);
#pragma unroll
            for (int k16 = 0; k16 < 4; ++k16) {
              // 16 bf16 = 32 bytes further along K inside the swizzle atom: +2 in 16-byte units
              if constexpr (PAIR) umma_bf16_pair(d_tmem, da + (uint64_t)(2 * k16), db + (uint64_t)(2 * k16), idesc, (first && k16 == 0) ? 0u : 1u);
              else umma_bf16(d_tmem, da + (uint64_t)(2 * k16), db + (uint64_t)(2 * k16), idesc, (first && k16 == 0) ? 0u : 1u);
            }
            first = false;
          }
          if constexpr (PAIR) umma_commit_pair(&g_tc.empty[stage]);
          else umma_commit(&g_tc.empty[stage]);
          u += nk;
          if (++stage == S) stage = 0;
        }
        if (!ok) break;
        // Warps 0-3 take part of the CTA's last accumulator.  They cannot wait on acc_full: a parity
        // wait tells two consecutive completions apart, not the first use of a buffer in this phase
        // from its third, and they arrive here long before the epilogue warps.  A barrier of their own
        // that completes exactly once per phase has no such ambiguity.
        if constexpr (PAIR) {
          umma_commit_pair(&g_tc.acc_full[abuf]);
          if (u == u1) umma_commit_pair(&g_tc.acc_last);
        } else {
          umma_commit(&g_tc.acc_full[abuf]);
          if (u == u1) umma_commit(&g_tc.acc_last);
        }
        abuf ^= 1;
      }
    }
  } else if (warp >= 4) {
    const int q = warp & 3;  // TMEM lane quarter this warp may read
    const TcEpiOut eo{a.out, (size_t)a.ldo, a.row_map, a.row_scale, T, N, ilv_F, act_direct};
    const bool accumulate = a.accumulate != 0;
    int abuf = 0;
    long long u = u0;
    while (u < u1) {
      const long long seg_end = min(u1, (u / kblocks + 1) * (long long)kblocks);
      const int kb0 = (int)(u % kblocks);
      const int kb1 = kb0 + (int)(seg_end - u);
      const int nt = tc_my_tile<PAIR>(tc_unit_nt(g, u), rank);
      const int pass = tc_unit_pass(g, u);
      const int rows = min(256, T - pass * 256);
      const int n_mma = (rows + 15) & ~15;
      const bool plain = (kb0 == 0 && kb1 == kblocks) && !accumulate && eo.row_map == nullptr;
      if (!mbar_wait(c, &g_tc.acc_full[abuf], (tc.acc_epi >> abuf) & 1u, dead)) break;
      tc.acc_epi ^= 1u << abuf;
      tc_fence_after();
      const uint32_t taddr = tc.tmem_base + (uint32_t)abuf * 256u + ((uint32_t)(q * 32) << 16);
      // the upper columns of the CTA's last accumulator are left to warps 0-3
      const int c_end = (seg_end == u1) ? tc_epi_half(n_mma) : n_mma;
      if (plain && eo.act != nullptr) {
        tc_epi_silu(eo, taddr, nt * 128 + q * 32 + lane, pass * 256, 0, c_end);
        if (q == 0 && lane == 0 && nt * 128 < N) c.gu_done[pass * ((N + 127) / 128) + nt] = gu_stamp(c, layer);   // read after the grid barrier
      } else {
        tc_epi_columns(eo, taddr, nt * 128 + q * 32 + lane, pass * 256, 0, c_end, plain);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if constexpr (PAIR) mbar_arrive_cta0(&g_tc.acc_empty[abuf]);   // the MMA issuer sits in CTA 0
        else mbar_arrive(&g_tc.acc_empty[abuf]);
      }
      abuf ^= 1;
      u = seg_end;
    }
  }
  if (warp < 4) {
    // Producers and the MMA issuer are done once the last MMA is committed: their warps store
    // the upper columns of the last accumulator.
    __syncwarp();
    if (u0 < u1) {
      const uint32_t par = tc.last_bit;
      tc.last_bit ^= 1u;
      long long last_u = u0;
      int last_abuf = 0;
      for (long long u = u0; u < u1;) {   // find the last segment and its accumulator buffer
        last_u = u;
        u = min(u1, (u / kblocks + 1) * (long long)kblocks);
        if (u < u1) last_abuf ^= 1;
      }
      const int kb0 = (int)(last_u % kblocks);
      const int nt = tc_my_tile<PAIR>(tc_unit_nt(g, last_u), rank);
      const int pass = tc_unit_pass(g, last_u);
      const int n_mma = (min(256, T - pass * 256) + 15) & ~15;
      const int c_begin = tc_epi_half(n_mma);
      // every thread waits (also when it has no columns to store) so that its parity stays in step
      if (mbar_wait_idle(c, &g_tc.acc_last, par, dead) && c_begin < n_mma) {
        tc_fence_after();
        const TcEpiOut eo{a.out, (size_t)a.ldo, a.row_map, a.row_scale, T, N, ilv_F, act_direct};
        const bool plain = (kb0 == 0 && (long long)kb0 + (u1 - last_u) == kblocks) && a.accumulate == 0 && eo.row_map == nullptr;
        const uint32_t taddr = tc.tmem_base + (uint32_t)last_abuf * 256u + ((uint32_t)(warp * 32) << 16);
        if (plain && eo.act != nullptr) tc_epi_silu(eo, taddr, nt * 128 + warp * 32 + lane, pass * 256, c_begin, n_mma);
        else tc_epi_columns(eo, taddr, nt * 128 + warp * 32 + lane, pass * 256, c_begin, n_mma, plain);
        tc_fence_before();
      }
    }
  }
  __syncthreads();
  if constexpr (!PAIR) {
    if (a.fix != FIX_NONE) tc_finish_tiles(c, a, g, layer);
  }
}

// ---- host side: tensor maps ----------------------------------------------------------------
inline size_t tc_smem_bytes() { return (size_t)TC_TILE_BUDGET + 1024; }

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn tc_encode_fn() {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess) return nullptr;
  if (qres != cudaDriverEntryPointSuccess) return nullptr;
  return reinterpret_cast<EncodeTiledFn>(fn);
}

// bf16 row-major [rows][cols] matrix, box = box_rows x 64 columns, 128-byte swizzle
inline bool tc_make_map(EncodeTiledFn enc, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols,
                        uint32_t box_rows, bool streaming) {
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  const CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                         streaming ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// The tensor-core path needs every contraction length to be a multiple of 64 (one swizzled
// smem row) and 16-byte aligned rows.
inline int tc_shape_ok(const DevCtx& c) {
  return c.dtype == 0 && c.d % 64 == 0 && c.q_dim % 64 == 0 && c.F % 64 == 0 && c.V % 4 == 0;
}
inline int tc_available() { return tc_encode_fn() != nullptr; }
// The streaming layout needs whole 128-row panels per layer in every GEMM matrix.
inline int tc_streaming_ok(const DevCtx& c) {
  return tc_shape_ok(c) && c.qkv_dim % 128 == 0 && c.d % 128 == 0 && (2 * c.F) % 128 == 0 && c.V % 128 == 0;
}

inline int tc_host_setup(TcHost& h, DevCtx& c) {
  EncodeTiledFn enc = tc_encode_fn();
  if (!enc) return -7;
  TcMaps* hm = new TcMaps();
  const char* w = c.w_base;
  const uint64_t L = c.L;
  bool ok = true;
  ok &= tc_make_map(enc, &hm->w[GEMM_QKV], w + c.w_off[1], L * c.qkv_dim, c.d, 128, true);
  ok &= tc_make_map(enc, &hm->w[GEMM_O], w + c.w_off[2], L * c.d, c.q_dim, 128, true);
  const uint64_t E1 = c.E > 0 ? c.E : 1;
  ok &= tc_make_map(enc, &hm->w[GEMM_GU], w + c.w_off[3], L * E1 * 2 * c.F, c.d, 128, true);
  ok &= tc_make_map(enc, &hm->w[GEMM_DOWN], w + c.w_off[4], L * E1 * c.d, c.F, 128, true);
  ok &= tc_make_map(enc, &hm->w[GEMM_LMHEAD], w + c.w_off[9], c.V, c.d, 128, true);
  if (c.w_streaming) {
    // the streaming layout as a rank-3 tensor [tiles][128 rows][64 columns] of verbatim 16 KiB tile images
    // (no swizzle: the image is already the operand image), boxes of one and of two consecutive tiles
    const uint64_t rows_tot[GEMM_KINDS] = {L * c.qkv_dim, L * c.d, L * E1 * 2 * c.F, L * E1 * c.d, (uint64_t)c.V};
    const uint64_t cols_k[GEMM_KINDS] = {(uint64_t)c.d, (uint64_t)c.q_dim, (uint64_t)c.d, (uint64_t)c.F, (uint64_t)c.d};
    const int ids[GEMM_KINDS] = {1, 2, 3, 4, 9};
    for (int k = 0; k < GEMM_KINDS; ++k)
      for (int two = 0; two < 2; ++two) {
        cuuint64_t dims[3] = {64, 128, rows_tot[k] / 128 * (cols_k[k] / 64)};
        cuuint64_t strides[2] = {128, 16384};
        cuuint32_t box[3] = {64, 128, (cuuint32_t)(two + 1)};
        cuuint32_t estr[3] = {1, 1, 1};
        ok &= enc(&hm->ws[k][two], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<char*>(w + c.w_off[ids[k]]), dims, strides, box,
                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
      }
  }
  const void* bufs[ACT_BUFS] = {c.xn, c.attn, c.act, c.xs, c.xg ? c.xg : c.xn};
  const uint64_t RA = (uint64_t)c.Tmax * (c.E > 0 ? c.topE : 1);   // routed experts: one row per (token, expert)
  const uint64_t rows[ACT_BUFS] = {(uint64_t)c.Tmax, (uint64_t)c.Tmax, RA, (uint64_t)c.MB, c.xg ? RA : (uint64_t)c.Tmax};
  const uint64_t cols[ACT_BUFS] = {(uint64_t)c.d, (uint64_t)c.q_dim, (uint64_t)c.F, (uint64_t)c.d, (uint64_t)c.d};
  for (int b = 0; b < ACT_BUFS; ++b)
    for (int i = 0; i < TC_BOXES; ++i) ok &= tc_make_map(enc, &hm->act[b][i], bufs[b], rows[b], cols[b], 16u << i, false);
  int rc = 0;
  if (!ok) rc = -7;
  if (rc == 0 && cudaMalloc(&h.d_maps, sizeof(TcMaps)) != cudaSuccess) rc = -6;
  if (rc == 0 && cudaMemcpy(h.d_maps, hm, sizeof(TcMaps), cudaMemcpyHostToDevice) != cudaSuccess) rc = -7;
  delete hm;
  if (rc == 0) c.tc_maps = h.d_maps;
  return rc;
}
inline void tc_host_free(TcHost& h) {
  if (h.d_maps) cudaFree(h.d_maps);
  h.d_maps = nullptr;
}

}  // namespace blink
