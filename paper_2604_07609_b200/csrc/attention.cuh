// Paged attention of the bf16 data path (Section 4.2 / 6.1 of the paper: the engine's paged
// KV cache with decode attention and context attention inside the step).
//
// Two kinds of work share the phase:
//   * decode rows (one query token per request): bandwidth-bound.  All (row, kv head, KV block)
//     tiles of the step form one flat sequence that is cut into sub-ranges; warps fetch
//     sub-ranges from a counter, stream the 16-key K and V tiles (contiguous in the pool) into
//     a private shared-memory ring with TMA tile copies (mbarrier completion), and keep an
//     online softmax per (row, kv head) unit.  The query heads of a GQA group share every K/V
//     load.  A unit cut by a sub-range boundary leaves partial (m, l, acc) records; whoever
//     finishes the last part merges them in a fixed order.
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

__device__ __forceinline__ float fast_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf2(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}
// one TMA tile copy from a rank-5 tensor map
__device__ __forceinline__ void tma_load_5d(void* smem_dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, int c4,
                                            uint64_t* bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4, "
      "%5, %6}], [%7], %8;" ::"r"(smem_u32(smem_dst)),
      "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
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

// ---- tensor-core and matrix-load wrappers ---------------------------------------------------------
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

// ---- decode rows: warp-level streaming kernel -------------------------------------------------
// One warp owns a (row, kv head) unit at a time and walks its 16-key tiles.  A tile's K and V
// ([16 keys][head_dim] each, contiguous in the pool) arrive through one TMA tile copy with the
// 128-byte swizzle, so both can be read with ldmatrix (at most two-way bank conflicts).  The two small contractions
// of a tile (scores and out += P V for the query heads of the group) run as m16n8k16 MMAs with
// the 16 keys (or 16 output dims) as the rows and the group's heads as the columns: written with
// CUDA-core FMAs the same loop needs about 800 instructions per tile and the SM runs out of issue
// slots at about half the HBM bandwidth; this form needs about 110.  Softmax statistics stay in
// fp32 registers and are combined with shuffles.
template <int HD, int NREP>
__device__ __noinline__ void attn_decode_stream(const DevCtx& c, int layer, char* ring, AttState& as) {
  constexpr int RB = HD * 2;         // bytes per key row
  constexpr int NBOX = HD / 64;      // 64-column boxes per tile row (128-byte swizzle span)
  constexpr int TILE = 16 * RB;      // bytes of one K (or V) tile of a (block, kv head)
  constexpr int STAGE = 2 * TILE;
  constexpr int KS = HD / 16;        // k-steps of Q K^T
  constexpr int REC = NREP * HD + ((2 * NREP + 3) & ~3);  // floats per partial record, 16-byte multiple
  constexpr unsigned FULL = 0xffffffffu;
  static_assert(NREP <= 8, "the group's heads must fit the first eight operand rows");
  const SchedState* ss = c.ss;
  const int n_dec = ss->cur_ndec, TT = ss->cur_TT, S = ss->cur_S;
  if (TT <= 0) return;
  const int n_sub = (TT + S - 1) / S;
  const int Hkv = c.Hkv;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int gq = lane >> 2, tq = lane & 3;   // operand row (= head of the group) and column pair
  const bool live = gq < NREP;   // this lane loads the q of head gq
  uint64_t* bars = g_att.bar[w];
  volatile int* dead = &g_att.dead;
  int* ctr = c.att_ctr + layer;
  const CUtensorMap* kv_map = reinterpret_cast<const CUtensorMap*>(c.kv_map);
  const __nv_bfloat16* qb = reinterpret_cast<const __nv_bfloat16*>(c.qb);
  __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(c.attn);
  const float qscale = c.attn_scale * 1.4426950408889634f;
  const uint32_t ring_s = smem_u32(ring);
  const uint64_t kv_policy = l2_evict_first();   // the cache is read once per step

  int n_issued = 0, n_consumed = 0, p_k = 0, c_k = 0;
  bool p_done = false, first_fetch = true;
  DecCursor pc{0, 0, 0, 0, 0, 1}, cc{0, 0, 0, 0, 0, 1};
  int p_blk = 0, p_blk_d = -1, p_blk_base = -1;
  int sub_start = 0, sub_id = 0;
  bool in_unit = false;

  // Both contractions are written with the 16 keys (scores) or 16 dims (output) as the M rows of
  // the MMA and the group's heads as the 8 columns, so a tile costs 8 + 8 MMAs.  Column pair
  // (2 tq, 2 tq + 1) of every accumulator belongs to this lane: two heads, softmax state for each.
  uint32_t qf[KS][2];     // B operand of the scores: q of head gq, dims 16 ks + 2 tq .. and + 8
  float o[HD / 16][4];    // out^T: dims gq + 16 i (c0, c1) and gq + 8 + 16 i (c2, c3), heads 2 tq, 2 tq + 1
  float m2[2] = {-INFINITY, -INFINITY}, l2[2] = {0.f, 0.f};

  while (true) {
    // ---- producer: keep up to ATT_NS tiles in flight ----
    while (!p_done && n_issued - n_consumed < ATT_NS) {
      if (pc.f == pc.f_end) {
        // next non-empty sub-range: the warp's own index first, then whatever the counter hands out
        int id = 0, b0 = 0, b1 = 0;
        while (true) {
          if (first_fetch) {
            id = blockIdx.x * ATT_WARPS + w;
            first_fetch = false;
          } else {
            if (lane == 0) id = atomicAdd(ctr, 1);
            id = __shfl_sync(FULL, id, 0);
          }
          if (id >= n_sub) { p_done = true; break; }
          b0 = id * S;
          b1 = min(TT, id * S + S);
          if (b0 < b1) break;
        }
        if (p_done) break;
        if (lane == 0) g_att.ids[w][p_k & 7] = id;
        __syncwarp();
        p_k += 1;
        dec_seek(pc, b0, b1, n_dec, Hkv);
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
        // one copy brings the K tile and the V tile: box {64 dims, NBOX halves, 16 keys, K and V, this layer}
        mbar_expect_tx(&bars[s], STAGE);
        tma_load_5d(ring + s * STAGE, kv_map, 0, 0, (blk * Hkv + pc.g) * 16, 0, layer, &bars[s], kv_policy);
      }
      dec_advance(pc, n_dec, Hkv);
      n_issued += 1;
    }
    if (n_consumed == n_issued) break;

    // ---- consumer: one tile ----
    while (cc.f == cc.f_end) {   // next non-empty sub-range (the producer already issued a tile of it)
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
      m2[0] = m2[1] = -INFINITY;
      l2[0] = l2[1] = 0.f;
      const __nv_bfloat16* qrow = qb + (size_t)t_row * c.q_dim + (size_t)(cc.g * NREP + (live ? gq : 0)) * HD;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        qf[ks][0] = live ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 2 * tq) : 0u;
        qf[ks][1] = live ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8 + 2 * tq) : 0u;
      }
#pragma unroll
      for (int i = 0; i < HD / 16; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    }
    const int s = n_consumed % ATT_NS;
    if (!__all_sync(FULL, mbar_wait(c, &bars[s], (as.par >> s) & 1u, dead))) break;  // uniform exit
    as.par ^= 1u << s;
    const uint32_t kt = ring_s + s * STAGE, vt = kt + TILE;
    const int key0 = cc.kb * 16;
    const int n_valid = min(16, n_ctx - key0);   // >= 1
    if (n_valid < 16) {
      // the tail of the last block holds whatever the pool held: clear those V rows (0 x NaN)
      uint4* vg = reinterpret_cast<uint4*>(ring + s * STAGE + TILE + n_valid * RB);
      for (int i = lane; i < (16 - n_valid) * RB / 16; i += 32) vg[i] = make_uint4(0u, 0u, 0u, 0u);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // before TMA refills this stage
      __syncwarp();
    }
    // The matrix loads and MMAs below are issued in program order, so all loads of an operand are
    // issued before the MMAs that use them, and V is fetched before the softmax arithmetic.
    uint32_t kf[KS][4];    // A operand of the scores: K tile, keys x dims
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const int key = (lane & 7) + ((lane >> 3) & 1) * 8;
      const int ck = ks * 2 + (lane >> 4);
      const int line = key * NBOX + (ck >> 3);   // 128-byte line of the tile; chunks are swizzled with the line index
      ldsm_x4(kt + line * 128 + (((ck & 7) ^ (line & 7)) << 4), kf[ks][0], kf[ks][1], kf[ks][2], kf[ks][3]);
    }
    uint32_t vf[HD / 16][4];   // A operand of the output: V tile transposed, dims x keys
#pragma unroll
    for (int i = 0; i < HD / 16; ++i) {
      const int key = (lane & 7) + ((lane >> 4) & 1) * 8;
      const int ck = i * 2 + ((lane >> 3) & 1);
      const int line = key * NBOX + (ck >> 3);
      ldsm_x4_t(vt + line * 128 + (((ck & 7) ^ (line & 7)) << 4), vf[i][0], vf[i][1], vf[i][2], vf[i][3]);
    }
    // scores^T [16 keys][8 heads]: four accumulators (k-step mod 4) keep the dependent chains short
    float sacc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i) { sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) mma_bf16_16816(sacc[ks & 3], kf[ks], qf[ks][0], qf[ks][1]);
    float sv[4];   // keys gq (0, 1) and gq + 8 (2, 3), heads 2 tq (0, 2) and 2 tq + 1 (1, 3)
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float v = (sacc[0][e] + sacc[1][e]) + (sacc[2][e] + sacc[3][e]);
      sv[e] = (gq + (e >> 1) * 8 < n_valid) ? v * qscale : -INFINITY;
    }
    // online softmax per head: maxima over the 16 keys live in the lanes with the same tq
    float mx0 = fmaxf(sv[0], sv[2]), mx1 = fmaxf(sv[1], sv[3]);
#pragma unroll
    for (int sh = 4; sh <= 16; sh <<= 1) {
      mx0 = fmaxf(mx0, __shfl_xor_sync(FULL, mx0, sh));
      mx1 = fmaxf(mx1, __shfl_xor_sync(FULL, mx1, sh));
    }
    const float mn0 = fmaxf(m2[0], mx0), mn1 = fmaxf(m2[1], mx1);   // finite: key 0 of the tile is always valid
    if (__any_sync(FULL, mn0 > m2[0] || mn1 > m2[1])) {
      const float c0 = fast_ex2(m2[0] - mn0), c1 = fast_ex2(m2[1] - mn1);
      l2[0] *= c0; l2[1] *= c1;
#pragma unroll
      for (int i = 0; i < HD / 16; ++i) { o[i][0] *= c0; o[i][1] *= c1; o[i][2] *= c0; o[i][3] *= c1; }
    }
    m2[0] = mn0; m2[1] = mn1;
    const float p0 = fast_ex2(sv[0] - mn0), p1 = fast_ex2(sv[1] - mn1), p2 = fast_ex2(sv[2] - mn0), p3 = fast_ex2(sv[3] - mn1);
    l2[0] += p0 + p2;
    l2[1] += p1 + p3;
    // P^T as the B operand of the output: transpose the two 8 x 8 (key, head) blocks in registers
    uint32_t pb0, pb1;
    {
      const uint32_t plo = pack_bf2(p0, p1), phi = pack_bf2(p2, p3);
      asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(pb0) : "r"(plo));
      asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(pb1) : "r"(phi));
    }
    // out^T += V^T P^T: 16 dims per MMA, one k-step of 16 keys
#pragma unroll
    for (int i = 0; i < HD / 16; ++i) mma_bf16_16816(o[i], vf[i], pb0, pb1);
    __syncwarp();  // all reads of this stage are done before it is refilled
    n_consumed += 1;

    const bool unit_ends = (cc.kb == cc.nkb - 1) || (cc.f + 1 == cc.f_end);
    if (unit_ends) {
      in_unit = false;
      float lt0 = l2[0], lt1 = l2[1];   // sums over the keys: lanes with the same tq
#pragma unroll
      for (int sh = 4; sh <= 16; sh <<= 1) {
        lt0 += __shfl_xor_sync(FULL, lt0, sh);
        lt1 += __shfl_xor_sync(FULL, lt1, sh);
      }
      const int us = Hkv * g_att_pre[cc.d] + cc.g * cc.nkb, ue = us + cc.nkb;
      const int j_first = us / S, j_last = (ue - 1) / S;
      const int h0 = 2 * tq;   // this lane's heads: h0, h0 + 1
      if (j_first == j_last) {   // the whole unit was handled here
        __nv_bfloat16* obase = out + (size_t)t_row * c.q_dim + (size_t)(cc.g * NREP) * HD;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          if (h0 + e < NREP) {
            const float inv = __fdividef(1.0f, e ? lt1 : lt0);
#pragma unroll
            for (int i = 0; i < HD / 16; ++i) {
              obase[(h0 + e) * HD + 16 * i + gq] = __float2bfloat16_rn(o[i][e] * inv);
              obase[(h0 + e) * HD + 16 * i + 8 + gq] = __float2bfloat16_rn(o[i][2 + e] * inv);
            }
          }
        }
      } else {
        // partial record: [NREP][HD] accumulators, then m[NREP], then l[NREP]
        const int unit = cc.d * Hkv + cc.g;
        float* rec = c.att_part + (size_t)(2 * sub_id + (us <= sub_start ? 0 : 1)) * REC;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          if (h0 + e < NREP) {
#pragma unroll
            for (int i = 0; i < HD / 16; ++i) {
              rec[(h0 + e) * HD + 16 * i + gq] = o[i][e];
              rec[(h0 + e) * HD + 16 * i + 8 + gq] = o[i][2 + e];
            }
            if (gq == 0) { rec[NREP * HD + h0 + e] = m2[e]; rec[NREP * HD + NREP + h0 + e] = e ? lt1 : lt0; }
          }
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
            const float inv = __fdividef(1.0f, den);
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
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}

// One CTA: query rows [qblk*QROWS, +QROWS) of one request's chunk, one kv head; the NREP query
// heads of the group are stacked along M (M row = head * QROWS + row), 16 M rows per warp.
// Shared memory: Q [128][HD] then two stages of K [64][HD], V [64][HD]; 16-byte chunks of a row
// are XOR-swizzled with the row index so that ldmatrix reads are conflict-free.
template <int HD, int NREP>
__device__ __noinline__ void attn_prefill_tile(const DevCtx& c, int layer, int item, int qblk, int g, char* smem) {
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
      uint32_t bf[4][4];   // all loads of the k-step first, then its MMAs (both are issued in program order)
#pragma unroll
      for (int np = 0; np < 4; ++np) {
        const int key = np * 16 + (lane & 7) + (lane >> 4) * 8;
        const int ck = ks * 2 + ((lane >> 3) & 1);
        ldsm_x4(sk + key * RB + ((ck ^ (key & 7)) << 4), bf[np][0], bf[np][1], bf[np][2], bf[np][3]);
      }
#pragma unroll
      for (int np = 0; np < 4; ++np) {
        mma_bf16_16816(sacc[2 * np], qf[ks], bf[np][0], bf[np][1]);
        mma_bf16_16816(sacc[2 * np + 1], qf[ks], bf[np][2], bf[np][3]);
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
      for (int d4 = 0; d4 < HD / 16; d4 += 4) {
        uint32_t bf[4][4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int key = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
          const int ck = (d4 + j) * 2 + (lane >> 4);
          ldsm_x4_t(sv + key * RB + ((ck ^ (key & 7)) << 4), bf[j][0], bf[j][1], bf[j][2], bf[j][3]);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          mma_bf16_16816(o[2 * (d4 + j)], pf[kk], bf[j][0], bf[j][1]);
          mma_bf16_16816(o[2 * (d4 + j) + 1], pf[kk], bf[j][2], bf[j][3]);
        }
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
  const float i_lo = __fdividef(1.0f, l_lo), i_hi = __fdividef(1.0f, l_hi);
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
template <int HD>
constexpr int att_smem_bytes() {
  constexpr int ring = ATT_WARPS * ATT_NS * 2 * 16 * HD * 2 + 1024;   // + alignment slack
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
    char* ring = tc_tiles(smem_f) + w * ATT_NS * STAGE;   // 1024-byte aligned: the tiles are swizzled
    attn_decode_stream<HD, NREP>(c, layer, ring, as);
  }
}

}  // namespace blink
