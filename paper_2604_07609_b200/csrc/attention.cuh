// Paged attention of the bf16 data path (Section 4.2 / 6.1 of the paper: the engine's paged
// KV cache with decode attention and context attention inside the step).
//
// Two kinds of work share the phase:
//   * decode rows (one query token per request): a bandwidth-bound CUDA-core kernel.  All
//     (row, kv head, KV block) tiles of the step form one flat sequence that is cut into
//     sub-ranges; warps fetch sub-ranges from a counter, stream the 16-key K and V tiles
//     (contiguous in the pool) into a private shared-memory ring with bulk async copies
//     (TMA engine, mbarrier completion), and keep an online softmax per (row, kv head)
//     unit.  The query heads of a GQA group share every K/V load.  A unit cut by a
//     sub-range boundary leaves partial (m, l, acc) records; whoever finishes the last part
//     merges them in a fixed order.
//   * prefill-chunk rows (several query tokens of one request): a dense contraction, so it
//     runs on tensor cores (mma.sync m16n8k16, flash-attention style tiling): one CTA per
//     (request, block of query rows, kv head), 64-key K/V tiles through a double-buffered
//     cp.async pipeline, scores and probabilities in registers.
#pragma once
#include "gemm_tc.cuh"

namespace blink {

constexpr int ATT_NS = 3;  // ring stages per warp (decode path)
constexpr int ATT_WARPS = FWD_THREADS / 32;

struct AttShared {
  uint64_t bar[ATT_WARPS][ATT_NS];
  int ids[ATT_WARPS][8];
  int dead;
};
__shared__ __align__(8) AttShared g_att;
__shared__ int g_att_pre[MAX_BATCH + 1];   // prefix of KV blocks over the decode rows of the step
__shared__ int g_att_bslot[MAX_BATCH];
__shared__ int g_att_nctx[MAX_BATCH];
__shared__ int g_att_row[MAX_BATCH];

// per-thread state that survives from phase to phase (mbarrier parities of the warp's ring)
struct AttState {
  uint32_t par;
};

__device__ __forceinline__ void att_init(const DevCtx& c, AttState& s) {
  s.par = 0;
  if (c.dtype != 0 || c.control_only) return;
  if ((threadIdx.x & 31) == 0) {
    for (int i = 0; i < ATT_NS; ++i) mbar_init(&g_att.bar[threadIdx.x >> 5][i], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x == 0) g_att.dead = 0;
  __syncthreads();
}

__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

// packed fp32x2 arithmetic (two lanes of one 64-bit register)
__device__ __forceinline__ unsigned long long ffma2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ unsigned long long fmul2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
  return ((unsigned long long)__float_as_uint(hi) << 32) | (unsigned long long)__float_as_uint(lo);
}
__device__ __forceinline__ float lo2(unsigned long long v) { return __uint_as_float((uint32_t)v); }
__device__ __forceinline__ float hi2(unsigned long long v) { return __uint_as_float((uint32_t)(v >> 32)); }
// two bf16 in one word -> the same two values as fp32x2 (low half first)
__device__ __forceinline__ unsigned long long bf2_to_f2(uint32_t w) {
  return ((unsigned long long)(w & 0xffff0000u) << 32) | (unsigned long long)(w << 16);
}
__device__ __forceinline__ float fast_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf2(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ float ldcg_f(const float* p) {
  float v;
  asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p) : "memory");
  return v;
}

// One halving step of a butterfly reduction: the lanes of a pair (xor MASK) hold N values
// each; afterwards each holds N/2 sums (the lane with the MASK bit set keeps the upper half).
template <int N, int MASK>
__device__ __forceinline__ void halve_step(float* v, bool upper) {
#pragma unroll
  for (int i = 0; i < N / 2; ++i) {
    const float send = upper ? v[i] : v[i + N / 2];
    const float keep = upper ? v[i + N / 2] : v[i];
    v[i] = keep + __shfl_xor_sync(0xffffffffu, send, MASK);
  }
}
template <int N, int MASK>
__device__ __forceinline__ void reduce_step(float* v, bool upper) {
  if constexpr (N >= 2) {
    halve_step<N, MASK>(v, upper);
  } else {
    v[0] += __shfl_xor_sync(0xffffffffu, v[0], MASK);
  }
}

// flat tile sequence of the decode rows: unit (d, g) owns tiles [Hkv*pre[d] + g*nkb, +nkb)
struct DecCursor {
  int f, f_end;      // next tile and end of the current sub-range
  int d, g, kb, nkb; // decoded position of f
};
__device__ __forceinline__ void dec_seek(DecCursor& cur, int f, int f_end, int n_dec, int Hkv) {
  cur.f = f;
  cur.f_end = f_end;
  int lo = 0, hi = n_dec;  // last d with Hkv * pre[d] <= f
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (Hkv * g_att_pre[mid] <= f) lo = mid; else hi = mid;
  }
  cur.d = lo;
  cur.nkb = g_att_pre[lo + 1] - g_att_pre[lo];
  const int rem = f - Hkv * g_att_pre[lo];
  cur.g = rem / cur.nkb;
  cur.kb = rem - cur.g * cur.nkb;
}
__device__ __forceinline__ void dec_advance(DecCursor& cur, int n_dec, int Hkv) {
  cur.f += 1;
  if (++cur.kb == cur.nkb) {
    cur.kb = 0;
    if (++cur.g == Hkv) {
      cur.g = 0;
      cur.d += 1;
      if (cur.d < n_dec) cur.nkb = g_att_pre[cur.d + 1] - g_att_pre[cur.d];
    }
  }
}

// ---- decode rows: warp-level streaming kernel -------------------------------------------------
// Lane mapping inside a warp: every lane owns one 16-byte chunk (8 dims) of the head vector,
// LPK = head_dim / 8 lanes cover a key, so the warp reads KG = 32 / LPK keys per pass as one
// contiguous run of shared memory; pass p handles key KG * p + kg of the 16-key tile.
template <int HD, int NREP>
__device__ __forceinline__ void attn_decode_stream(const DevCtx& c, int layer, char* ring, float* sc, AttState& as) {
  constexpr int LPK = HD / 8;        // lanes per key
  constexpr int KG = 32 / LPK;       // keys per pass
  constexpr int NP = 16 / KG;        // passes per tile
  constexpr int RB = HD * 2;         // bytes per key row
  constexpr int TILE = 16 * RB;      // bytes of one K (or V) tile of a (block, kv head)
  constexpr int STAGE = 2 * TILE;
  constexpr int NV = NP * NREP;      // (pass, head) partial scores per lane per tile
  constexpr int OC = NV >= LPK ? NV / LPK : 1;
  constexpr int NA = NREP * 8;       // accumulator values per lane
  constexpr int OWN = NA / KG;       // ... and after the sum over the key groups
  constexpr int REC = NREP * HD + ((2 * NREP + 3) & ~3);  // floats per partial record, 16-byte multiple
  constexpr unsigned FULL = 0xffffffffu;
  const SchedState* ss = c.ss;
  const int n_dec = ss->cur_ndec, TT = ss->cur_TT, S = ss->cur_S;
  if (TT <= 0) return;
  const int n_sub = (TT + S - 1) / S;
  const int Hkv = c.Hkv;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int kg = lane / LPK, dc = lane % LPK;
  uint64_t* bars = g_att.bar[w];
  volatile int* dead = &g_att.dead;
  int* ctr = c.att_ctr + layer;
  const __nv_bfloat16* qb = reinterpret_cast<const __nv_bfloat16*>(c.qb);
  __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(c.attn);
  const char* kv_base = reinterpret_cast<const char*>(c.kv_base);
  const size_t kv_stride = (size_t)c.n_blocks * Hkv * TILE;  // bytes between the K and V planes of a layer
  const char* k_plane = kv_base + (size_t)layer * 2 * kv_stride;
  const float qscale = c.attn_scale * 1.4426950408889634f;

  int n_issued = 0, n_consumed = 0, p_k = 0, c_k = 0;
  bool p_done = false;
  DecCursor pc{0, 0, 0, 0, 0, 1}, cc{0, 0, 0, 0, 0, 1};
  int p_blk = 0, p_blk_d = -1, p_blk_base = -1;
  int sub_start = 0, sub_id = 0;
  bool in_unit = false;

  unsigned long long q2[NREP][4];
  unsigned long long acc2[NREP][4];
  float m[NREP], l[NREP];

  while (true) {
    // ---- producer: keep up to ATT_NS tiles in flight ----
    while (!p_done && n_issued - n_consumed < ATT_NS) {
      if (pc.f == pc.f_end) {
        int id = blockIdx.x * ATT_WARPS + w;   // first sub-range: the warp's own index
        if (p_k > 0) {
          if (lane == 0) id = atomicAdd(ctr, 1);
          id = __shfl_sync(FULL, id, 0);
        }
        if (lane == 0) g_att.ids[w][p_k & 7] = id;
        __syncwarp();
        p_k += 1;
        if (id >= n_sub) { p_done = true; break; }
        dec_seek(pc, id * S, min(TT, id * S + S), n_dec, Hkv);
      }
      if (pc.d != p_blk_d || (pc.kb & ~31) != p_blk_base) {
        p_blk_d = pc.d;
        p_blk_base = pc.kb & ~31;
        const int idx = p_blk_base + lane;
        p_blk = idx < pc.nkb ? c.block_table[(size_t)g_att_bslot[pc.d] * c.max_blocks_seq + idx] : 0;
      }
      const int blk = __shfl_sync(FULL, p_blk, pc.kb & 31);
      if (lane == 0) {
        const int s = n_issued % ATT_NS;
        const char* ksrc = k_plane + ((size_t)blk * Hkv + pc.g) * TILE;
        mbar_expect_tx(&bars[s], STAGE);
        bulk_g2s(ring + s * STAGE, ksrc, TILE, &bars[s]);
        bulk_g2s(ring + s * STAGE + TILE, ksrc + kv_stride, TILE, &bars[s]);
      }
      dec_advance(pc, n_dec, Hkv);
      n_issued += 1;
    }
    if (n_consumed == n_issued) break;

    // ---- consumer: one tile ----
    if (cc.f == cc.f_end) {
      sub_id = g_att.ids[w][c_k & 7];
      c_k += 1;
      sub_start = sub_id * S;
      dec_seek(cc, sub_start, min(TT, sub_start + S), n_dec, Hkv);
      in_unit = false;
    }
    const int t_row = g_att_row[cc.d];
    const int n_ctx = g_att_nctx[cc.d];
    if (!in_unit) {  // a unit (or this sub-range's part of it) starts here
      in_unit = true;
#pragma unroll
      for (int h = 0; h < NREP; ++h) {
        m[h] = -INFINITY;
        l[h] = 0.f;
        const __nv_bfloat16* qrow = qb + (size_t)t_row * c.q_dim + (size_t)(cc.g * NREP + h) * HD;
        const uint4 qr = *reinterpret_cast<const uint4*>(qrow + dc * 8);
        const uint32_t qw[4] = {qr.x, qr.y, qr.z, qr.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const unsigned long long f2 = bf2_to_f2(qw[i]);
          q2[h][i] = pack2(lo2(f2) * qscale, hi2(f2) * qscale);
          acc2[h][i] = 0ull;
        }
      }
    }
    const int s = n_consumed % ATT_NS;
    if (!__all_sync(FULL, mbar_wait(c, &bars[s], (as.par >> s) & 1u, dead))) break;  // uniform exit
    as.par ^= 1u << s;
    const char* kt = ring + s * STAGE;
    const char* vt = kt + TILE;
    const int key0 = cc.kb * 16;

    // scores: partial dot products over this lane's 8 dims
    float part[NV];
#pragma unroll
    for (int p = 0; p < NP; ++p) {
      const uint4 kr = *reinterpret_cast<const uint4*>(kt + (KG * p + kg) * RB + dc * 16);
      const uint32_t kw[4] = {kr.x, kr.y, kr.z, kr.w};
      unsigned long long a2[NREP];
#pragma unroll
      for (int h = 0; h < NREP; ++h) a2[h] = 0ull;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const unsigned long long k2 = bf2_to_f2(kw[i]);
#pragma unroll
        for (int h = 0; h < NREP; ++h) a2[h] = ffma2(q2[h][i], k2, a2[h]);
      }
#pragma unroll
      for (int h = 0; h < NREP; ++h) part[p * NREP + h] = lo2(a2[h]) + hi2(a2[h]);
    }
    // reduce over the LPK lanes of a key; each lane ends up owning OC complete scores
    if constexpr (LPK == 16) {
      reduce_step<NV, 8>(part, (dc & 8) != 0);
      reduce_step<NV / 2, 4>(part, (dc & 4) != 0);
      reduce_step<NV / 4, 2>(part, (dc & 2) != 0);
      reduce_step<NV / 8, 1>(part, (dc & 1) != 0);
    } else {
      reduce_step<NV, 4>(part, (dc & 4) != 0);
      reduce_step<NV / 2, 2>(part, (dc & 2) != 0);
      reduce_step<NV / 4, 1>(part, (dc & 1) != 0);
    }
    {
      const int v_base = NV >= LPK ? dc * OC : dc / (LPK / NV);
#pragma unroll
      for (int o = 0; o < OC; ++o) {
        const int v = v_base + o;
        const int p = v / NREP, h = v % NREP;
        const int key = KG * p + kg;
        sc[key * NREP + h] = (key0 + key < n_ctx) ? part[o] : -INFINITY;
      }
    }
    __syncwarp();
    float sp[NP][NREP];
    float tmax[NREP];
#pragma unroll
    for (int h = 0; h < NREP; ++h) tmax[h] = -INFINITY;
#pragma unroll
    for (int p = 0; p < NP; ++p)
#pragma unroll
      for (int h = 0; h < NREP; ++h) {
        sp[p][h] = sc[(KG * p + kg) * NREP + h];
        tmax[h] = fmaxf(tmax[h], sp[p][h]);
      }
    bool changed = false;
#pragma unroll
    for (int h = 0; h < NREP; ++h) {
      tmax[h] = fmaxf(tmax[h], __shfl_xor_sync(FULL, tmax[h], 16));
      if constexpr (KG == 4) tmax[h] = fmaxf(tmax[h], __shfl_xor_sync(FULL, tmax[h], 8));
      changed |= tmax[h] > m[h];
    }
    if (changed) {  // warp-uniform: every lane holds the same m and tmax
#pragma unroll
      for (int h = 0; h < NREP; ++h) {
        const float mn = fmaxf(m[h], tmax[h]);
        const float corr = fast_ex2(m[h] - mn);
        m[h] = mn;
        l[h] *= corr;
        const unsigned long long c2 = pack2(corr, corr);
#pragma unroll
        for (int i = 0; i < 4; ++i) acc2[h][i] = fmul2(acc2[h][i], c2);
      }
    }
    // probabilities and P.V
#pragma unroll
    for (int p = 0; p < NP; ++p) {
      const int key = KG * p + kg;
      if (key0 + key < n_ctx) {   // keys past the context hold whatever the pool held
        const uint4 vr = *reinterpret_cast<const uint4*>(vt + key * RB + dc * 16);
        const uint32_t vw[4] = {vr.x, vr.y, vr.z, vr.w};
        unsigned long long pp[NREP];
#pragma unroll
        for (int h = 0; h < NREP; ++h) {
          const float pv = fast_ex2(sp[p][h] - m[h]);
          l[h] += pv;
          pp[h] = pack2(pv, pv);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const unsigned long long v2 = bf2_to_f2(vw[i]);
#pragma unroll
          for (int h = 0; h < NREP; ++h) acc2[h][i] = ffma2(pp[h], v2, acc2[h][i]);
        }
      }
    }
    __syncwarp();  // all reads of this stage and of sc are done before they are refilled
    n_consumed += 1;

    const bool unit_ends = (cc.kb == cc.nkb - 1) || (cc.f + 1 == cc.f_end);
    if (unit_ends) {
      in_unit = false;
      // sum over the key groups: the lane ends up owning OWN accumulator values
      float a[NA];
#pragma unroll
      for (int h = 0; h < NREP; ++h)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          a[h * 8 + 2 * i] = lo2(acc2[h][i]);
          a[h * 8 + 2 * i + 1] = hi2(acc2[h][i]);
        }
      int a_base;
      if constexpr (KG == 2) {
        halve_step<NA, 16>(a, (lane & 16) != 0);
        a_base = (lane & 16) ? OWN : 0;
      } else {
        halve_step<NA, 8>(a, (lane & 8) != 0);
        halve_step<NA / 2, 16>(a, (lane & 16) != 0);
        a_base = (((lane >> 3) & 1) * 2 + ((lane >> 4) & 1)) * OWN;
      }
#pragma unroll
      for (int h = 0; h < NREP; ++h) {
        l[h] += __shfl_xor_sync(FULL, l[h], 16);
        if constexpr (KG == 4) l[h] += __shfl_xor_sync(FULL, l[h], 8);
      }
      const int us = Hkv * g_att_pre[cc.d] + cc.g * cc.nkb, ue = us + cc.nkb;
      const int j_first = us / S, j_last = (ue - 1) / S;
      if (j_first == j_last) {
#pragma unroll
        for (int o = 0; o < OWN; ++o) {
          const int ai = a_base + o;
          const int h = ai >> 3, dim = dc * 8 + (ai & 7);
          float lh = l[0];
#pragma unroll
          for (int hh = 1; hh < NREP; ++hh) lh = (h == hh) ? l[hh] : lh;
          out[(size_t)t_row * c.q_dim + (size_t)(cc.g * NREP + h) * HD + dim] = __float2bfloat16_rn(a[o] / lh);
        }
      } else {
        // partial record: [NREP][HD] accumulators, then m[NREP], then l[NREP]
        const int unit = cc.d * Hkv + cc.g;
        float* rec = c.att_part + (size_t)(2 * sub_id + (us <= sub_start ? 0 : 1)) * REC;
#pragma unroll
        for (int o = 0; o < OWN; ++o) {
          const int ai = a_base + o;
          rec[(ai >> 3) * HD + dc * 8 + (ai & 7)] = a[o];
        }
        if (lane == 0) {
#pragma unroll
          for (int h = 0; h < NREP; ++h) { rec[NREP * HD + h] = m[h]; rec[NREP * HD + NREP + h] = l[h]; }
        }
        __threadfence();
        __syncwarp();
        int old = 0;
        if (lane == 0) old = atomicAdd(&c.att_cnt[unit], 1);
        old = __shfl_sync(FULL, old, 0);
        if (old == j_last - j_first) {  // this warp delivered the last part: merge in sub-range order
          __threadfence();
          // each lane merges four consecutive dims at a time; loads of the parts are independent
          for (int i4 = lane; i4 < NREP * HD / 4; i4 += 32) {
            const int h = (i4 * 4) / HD;
            float M = -INFINITY;
#pragma unroll 4
            for (int j = j_first; j <= j_last; ++j) {
              const float* r = c.att_part + (size_t)(2 * j + (us <= j * S ? 0 : 1)) * REC;
              M = fmaxf(M, __ldcg(r + NREP * HD + h));
            }
            float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
            float den = 0.f;
#pragma unroll 4
            for (int j = j_first; j <= j_last; ++j) {
              const float* r = c.att_part + (size_t)(2 * j + (us <= j * S ? 0 : 1)) * REC;
              const float f = fast_ex2(__ldcg(r + NREP * HD + h) - M);
              const float4 a4 = __ldcg(reinterpret_cast<const float4*>(r) + i4);
              num.x += f * a4.x; num.y += f * a4.y; num.z += f * a4.z; num.w += f * a4.w;
              den += f * __ldcg(r + NREP * HD + NREP + h);
            }
            const float inv = 1.0f / den;
            uint2 o2;
            o2.x = pack_bf2(num.x * inv, num.y * inv);
            o2.y = pack_bf2(num.z * inv, num.w * inv);
            *reinterpret_cast<uint2*>(out + (size_t)t_row * c.q_dim + (size_t)(cc.g * NREP) * HD + i4 * 4) = o2;
          }
          if (lane == 0) c.att_cnt[unit] = 0;
        }
      }
    }
    dec_advance(cc, n_dec, Hkv);
  }
}

// ---- prefill-chunk rows: tensor-core tile kernel ---------------------------------------------------
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float* d, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}

// One CTA: query rows [qblk*QROWS, +QROWS) of one request's chunk, one kv head; the NREP query
// heads of the group are stacked along M (M row = head * QROWS + row), 16 M rows per warp.
// Shared memory: Q [128][HD] then two stages of K [64][HD], V [64][HD]; 16-byte chunks of a row
// are XOR-swizzled with the row index so that ldmatrix reads are conflict-free.
template <int HD, int NREP>
__device__ __forceinline__ void attn_prefill_tile(const DevCtx& c, int layer, int item, int qblk, int g, char* smem) {
  constexpr int QROWS = 128 / NREP;
  constexpr int RB = HD * 2;          // bytes per row
  constexpr int CPR = RB / 16;        // 16-byte chunks per row
  constexpr int KT = 64;              // keys per tile
  constexpr int QBYTES = 128 * RB, KVBYTES = KT * RB;
  constexpr int TILE = 16 * HD * 2;
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  const int bslot = c.it_bslot[item], start = c.it_start[item], ntok = c.it_ntok[item], qstart = c.it_qstart[item];
  const int r_base = qblk * QROWS;
  const int n_keys = start + min(ntok, r_base + QROWS);
  const int nkt = (n_keys + KT - 1) / KT;
  const int32_t* table = c.block_table + (size_t)bslot * c.max_blocks_seq;
  const __nv_bfloat16* qb = reinterpret_cast<const __nv_bfloat16*>(c.qb);
  __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(c.attn);
  const char* kv_base = reinterpret_cast<const char*>(c.kv_base);
  const size_t kv_stride = (size_t)c.n_blocks * c.Hkv * TILE;
  const char* k_plane = kv_base + (size_t)layer * 2 * kv_stride;
  const uint32_t s_q = smem_u32(smem), s_kv = s_q + QBYTES;
  const float qscale = c.attn_scale * 1.4426950408889634f;

  __syncthreads();  // the previous user of this shared memory is done
  // Q tile
  for (int id = tid; id < 128 * CPR; id += FWD_THREADS) {
    const int mrow = id / CPR, ck = id % CPR;
    const int h = mrow / QROWS, r = r_base + mrow % QROWS;
    const bool ok = r < ntok;
    const __nv_bfloat16* src = qb + (size_t)(qstart + (ok ? r : 0)) * c.q_dim + (size_t)(g * NREP + h) * HD + ck * 8;
    cp_async16(s_q + mrow * RB + ((ck ^ (mrow & 7)) << 4), src, ok ? 16u : 0u);
  }
  auto load_kv = [&](int kt, int stage) {
    const uint32_t dk = s_kv + stage * 2 * KVBYTES, dv = dk + KVBYTES;
    for (int id = tid; id < KT * CPR; id += FWD_THREADS) {
      const int key = id / CPR, ck = id % CPR;
      const int kpos = kt * KT + key;
      const bool ok = kpos < n_keys;
      const int blk = table[ok ? (kpos >> 4) : 0];
      const char* src = k_plane + ((size_t)blk * c.Hkv + g) * TILE + (size_t)(kpos & 15) * RB + ck * 16;
      const uint32_t off = key * RB + ((ck ^ (key & 7)) << 4);
      cp_async16(dk + off, src, ok ? 16u : 0u);
      cp_async16(dv + off, src + kv_stride, ok ? 16u : 0u);
    }
  };
  load_kv(0, 0);
  asm volatile("cp.async.commit_group;" ::: "memory");

  const int mrow0 = w * 16;
  const int gq = lane >> 2, tq = lane & 3;
  // positions of the two rows this lane holds in the accumulator layout
  const int pos_lo = start + r_base + (mrow0 + gq) % QROWS;
  const int pos_hi = start + r_base + (mrow0 + gq + 8) % QROWS;
  uint32_t qf[HD / 16][4];
  float o[HD / 8][4];
#pragma unroll
  for (int i = 0; i < HD / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

  for (int kt = 0; kt < nkt; ++kt) {
    const int stage = kt & 1;
    if (kt + 1 < nkt) load_kv(kt + 1, stage ^ 1);
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 1;" ::: "memory");
    __syncthreads();
    if (kt == 0) {
#pragma unroll
      for (int ks = 0; ks < HD / 16; ++ks) {
        const int row = mrow0 + (lane & 7) + ((lane >> 3) & 1) * 8;
        const int ck = ks * 2 + (lane >> 4);
        ldsm_x4(s_q + row * RB + ((ck ^ (row & 7)) << 4), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
      }
    }
    const uint32_t sk = s_kv + stage * 2 * KVBYTES, sv = sk + KVBYTES;
    // S = Q K^T for 64 keys: 8 n-tiles of 8 keys
    float sacc[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) { sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < HD / 16; ++ks) {
#pragma unroll
      for (int np = 0; np < 4; ++np) {
        const int key = np * 16 + (lane & 7) + (lane >> 4) * 8;
        const int ck = ks * 2 + ((lane >> 3) & 1);
        uint32_t b0, b1, b2, b3;
        ldsm_x4(sk + key * RB + ((ck ^ (key & 7)) << 4), b0, b1, b2, b3);
        mma_bf16_16816(sacc[2 * np], qf[ks], b0, b1);
        mma_bf16_16816(sacc[2 * np + 1], qf[ks], b2, b3);
      }
    }
    // scale, causal mask, online softmax (rows gq and gq + 8 of the warp's 16)
    float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const int k0 = kt * KT + nt * 8 + 2 * tq;
      sacc[nt][0] = (k0 <= pos_lo) ? sacc[nt][0] * qscale : -INFINITY;
      sacc[nt][1] = (k0 + 1 <= pos_lo) ? sacc[nt][1] * qscale : -INFINITY;
      sacc[nt][2] = (k0 <= pos_hi) ? sacc[nt][2] * qscale : -INFINITY;
      sacc[nt][3] = (k0 + 1 <= pos_hi) ? sacc[nt][3] * qscale : -INFINITY;
      mx_lo = fmaxf(mx_lo, fmaxf(sacc[nt][0], sacc[nt][1]));
      mx_hi = fmaxf(mx_hi, fmaxf(sacc[nt][2], sacc[nt][3]));
    }
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
    // key 0 is visible to every row, so after the first tile the maxima are finite
    const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
    const float c_lo = fast_ex2(m_lo - mn_lo), c_hi = fast_ex2(m_hi - mn_hi);
    m_lo = mn_lo; m_hi = mn_hi;
    l_lo *= c_lo; l_hi *= c_hi;
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) { o[i][0] *= c_lo; o[i][1] *= c_lo; o[i][2] *= c_hi; o[i][3] *= c_hi; }
    uint32_t pf[4][4];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const float p0 = fast_ex2(sacc[nt][0] - mn_lo), p1 = fast_ex2(sacc[nt][1] - mn_lo);
      const float p2 = fast_ex2(sacc[nt][2] - mn_hi), p3 = fast_ex2(sacc[nt][3] - mn_hi);
      l_lo += p0 + p1;
      l_hi += p2 + p3;
      pf[nt >> 1][(nt & 1) * 2] = pack_bf2(p0, p1);
      pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf2(p2, p3);
    }
    // O += P V
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
      for (int dp = 0; dp < HD / 16; ++dp) {
        const int key = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        const int ck = dp * 2 + (lane >> 4);
        uint32_t b0, b1, b2, b3;
        ldsm_x4_t(sv + key * RB + ((ck ^ (key & 7)) << 4), b0, b1, b2, b3);
        mma_bf16_16816(o[2 * dp], pf[kk], b0, b1);
        mma_bf16_16816(o[2 * dp + 1], pf[kk], b2, b3);
      }
    }
    __syncthreads();  // everyone is done with this stage before it is refilled
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
  const int h = mrow0 / QROWS;   // 16 | QROWS, so a warp's rows belong to one head
  const int r_lo = r_base + (mrow0 + gq) % QROWS, r_hi = r_base + (mrow0 + gq + 8) % QROWS;
  const float i_lo = 1.0f / l_lo, i_hi = 1.0f / l_hi;
#pragma unroll
  for (int nt = 0; nt < HD / 8; ++nt) {
    const size_t col = (size_t)(g * NREP + h) * HD + nt * 8 + 2 * tq;
    if (r_lo < ntok)
      *reinterpret_cast<uint32_t*>(out + (size_t)(qstart + r_lo) * c.q_dim + col) = pack_bf2(o[nt][0] * i_lo, o[nt][1] * i_lo);
    if (r_hi < ntok)
      *reinterpret_cast<uint32_t*>(out + (size_t)(qstart + r_hi) * c.q_dim + col) = pack_bf2(o[nt][2] * i_hi, o[nt][3] * i_hi);
  }
}

// ---- the phase ---------------------------------------------------------------------------------------
constexpr int ATT_SC_BYTES = ATT_WARPS * 16 * 8 * 4;   // per-warp score buffers, up to 8 heads per group
template <int HD>
constexpr int att_smem_bytes() {
  constexpr int ring = ATT_WARPS * ATT_NS * 2 * 16 * HD * 2 + ATT_SC_BYTES;
  constexpr int tile = 128 * HD * 2 + 2 * 2 * 64 * HD * 2;
  return ring > tile ? ring : tile;
}

template <int HD, int NREP>
__device__ __forceinline__ void phase_attention_bf16(const DevCtx& c, int layer, float* smem_f, AttState& as) {
  const SchedState* ss = c.ss;
  char* smem = reinterpret_cast<char*>(smem_f);
  const int n_pf = ss->cur_npf * c.Hkv;
  for (int u = blockIdx.x; u < n_pf; u += gridDim.x) {
    const int e = u / c.Hkv, g = u % c.Hkv;
    attn_prefill_tile<HD, NREP>(c, layer, c.pf_item[e], c.pf_qb[e], g, smem);
  }
  const int n_dec = ss->cur_ndec;
  if (n_dec > 0) {
    __syncthreads();
    for (int i = threadIdx.x; i <= n_dec; i += FWD_THREADS) {
      g_att_pre[i] = c.dec_kbpre[i];
      if (i < n_dec) { g_att_bslot[i] = c.dec_bslot[i]; g_att_nctx[i] = c.dec_nctx[i]; g_att_row[i] = c.dec_row[i]; }
    }
    __syncthreads();
    const int w = threadIdx.x >> 5;
    constexpr int STAGE = 2 * 16 * HD * 2;
    char* ring = smem + w * ATT_NS * STAGE;
    float* sc = reinterpret_cast<float*>(smem + ATT_WARPS * ATT_NS * STAGE) + w * 16 * 8;
    attn_decode_stream<HD, NREP>(c, layer, ring, sc, as);
  }
}

}  // namespace blink
