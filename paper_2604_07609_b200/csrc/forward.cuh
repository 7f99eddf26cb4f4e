// Data-parallel phases of one serving step (every CTA of the grid takes part):
// embedding + RMSNorm, CUDA-core reference GEMM, RoPE + paged-KV write, paged
// attention, SwiGLU gate, final norm, sampling.  Each phase is a __device__
// function that distributes its work over blockIdx.x / gridDim.x, so the same
// code runs inside the persistent loop (phases separated by grid barriers) and
// as host-launched kernels (stepped mode).
//
// Paper: the model step is the "inference engine" of Section 4.2 (paged KV cache,
// context attention, fused MLP, sampling captured inside the step); Section 6.1
// lists the engine features.  The math is the standard pre-norm decoder.
#pragma once
#include "control.cuh"
#include "dev_ctx.cuh"

namespace blink {

constexpr int FWD_THREADS = 256;

template <typename T> struct OpType;
template <> struct OpType<float> {
  static __device__ __forceinline__ float to_f(float v) { return v; }
  static __device__ __forceinline__ float from_f(float v) { return v; }
};
template <> struct OpType<__nv_bfloat16> {
  static __device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
  static __device__ __forceinline__ __nv_bfloat16 from_f(float v) { return __float2bfloat16_rn(v); }
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float block_sum(float v, float* s_red /*[8]*/) {
  v = warp_sum(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.f;
#pragma unroll
  for (int i = 0; i < FWD_THREADS / 32; ++i) t += s_red[i];
  return t;
}

template <typename WT>
__device__ __forceinline__ const WT* wptr(const DevCtx& c, int id) {
  return reinterpret_cast<const WT*>(c.w_base + c.w_off[id]);
}
__device__ __forceinline__ const float* wptr_f(const DevCtx& c, int id) {
  return reinterpret_cast<const float*>(c.w_base + c.w_off[id]);
}

// zero n_floats (a multiple of 4) floats starting at p, grid-strided
__device__ __forceinline__ void zero_floats(float* p, long long n_floats) {
  float4* q = reinterpret_cast<float4*>(p);
  const long long n4 = n_floats >> 2;
  for (long long i = (long long)blockIdx.x * FWD_THREADS + threadIdx.x; i < n4; i += (long long)gridDim.x * FWD_THREADS)
    q[i] = make_float4(0.f, 0.f, 0.f, 0.f);
}

// store four consecutive values in the operand type
template <typename WT>
__device__ __forceinline__ void store4(WT* p, float a, float b, float c, float d);
template <>
__device__ __forceinline__ void store4<float>(float* p, float a, float b, float c, float d) {
  *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d);
}
template <>
__device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16* p, float a, float b, float c, float d) {
  const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  uint2 v;
  v.x = *reinterpret_cast<const uint32_t*>(&lo);
  v.y = *reinterpret_cast<const uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = v;
}
template <typename WT>
__device__ __forceinline__ float4 load4(const WT* p);
template <>
__device__ __forceinline__ float4 load4<float>(const float* p) { return *reinterpret_cast<const float4*>(p); }
template <>
__device__ __forceinline__ float4 load4<__nv_bfloat16>(const __nv_bfloat16* p) {
  const uint2 v = *reinterpret_cast<const uint2*>(p);
  const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162*>(&v.x), hi = *reinterpret_cast<const __nv_bfloat162*>(&v.y);
  const float2 a = __bfloat1622float2(lo), b = __bfloat1622float2(hi);
  return make_float4(a.x, a.y, b.x, b.y);
}

// One CTA normalises one row: n = x / sqrt(mean(x^2) + eps) * g.  Every thread keeps its part of
// the row (16-byte vectors, up to NORM_MAXV of them: d <= 8192) in registers between the sum and
// the scaling, so the row is read once.  `src_embed` non-null: the row is first gathered from
// the embedding table into the residual stream.
constexpr int NORM_MAXV = 8;
template <typename WT>
__device__ __forceinline__ void norm_row_cta(const DevCtx& c, float* hrow, const WT* src_embed, const float* g, WT* orow,
                                             float* s_red, const float* wr = nullptr, int row_index = 0) {
  const int d = c.d;
  float4 v[NORM_MAXV];
  float ss = 0.f;
#pragma unroll
  for (int k = 0; k < NORM_MAXV; ++k) {
    const int i = (k * FWD_THREADS + threadIdx.x) * 4;
    if (i < d) {
      if (src_embed != nullptr) {
        v[k] = load4<WT>(src_embed + i);
        *reinterpret_cast<float4*>(hrow + i) = v[k];
      } else {
        v[k] = *reinterpret_cast<const float4*>(hrow + i);
      }
    }
  }
#pragma unroll
  for (int k = 0; k < NORM_MAXV; ++k) {
    const int i = (k * FWD_THREADS + threadIdx.x) * 4;
    if (i < d) {  // fixed order
      ss = fmaf(v[k].x, v[k].x, ss); ss = fmaf(v[k].y, v[k].y, ss); ss = fmaf(v[k].z, v[k].z, ss); ss = fmaf(v[k].w, v[k].w, ss);
    }
  }
  ss = block_sum(ss, s_red);
  const float inv = rsqrtf(__fdividef(ss, (float)d) + c.rms_eps);
#pragma unroll
  for (int k = 0; k < NORM_MAXV; ++k) {
    const int i = (k * FWD_THREADS + threadIdx.x) * 4;
    if (i < d) {
      const float4 gg = *reinterpret_cast<const float4*>(g + i);
      v[k] = make_float4(v[k].x * inv * gg.x, v[k].y * inv * gg.y, v[k].z * inv * gg.z, v[k].w * inv * gg.w);
      store4<WT>(orow + i, v[k].x, v[k].y, v[k].z, v[k].w);
    }
  }
  if (wr != nullptr) {
    // Router of the routed-expert FFN on the normed row in fp32 (not its 16-bit copy): logits over
    // the E experts, top-k by (logit desc, expert id asc), weights = softmax restricted to the chosen.
    __shared__ float s_rl[FWD_THREADS / 32][MAX_EXPERTS];
    const int E = c.E;
    for (int e = 0; e < E; ++e) {
      float p = 0.f;
#pragma unroll
      for (int k = 0; k < NORM_MAXV; ++k) {
        const int i = (k * FWD_THREADS + threadIdx.x) * 4;
        if (i < d) {
          const float4 w4 = *reinterpret_cast<const float4*>(wr + (size_t)e * d + i);
          p = fmaf(v[k].x, w4.x, p); p = fmaf(v[k].y, w4.y, p); p = fmaf(v[k].z, w4.z, p); p = fmaf(v[k].w, w4.w, p);
        }
      }
      p = warp_sum(p);
      if ((threadIdx.x & 31) == 0) s_rl[threadIdx.x >> 5][e] = p;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      float lg[MAX_EXPERTS];
      for (int e = 0; e < E; ++e) {
        float t = 0.f;
        for (int w = 0; w < FWD_THREADS / 32; ++w) t += s_rl[w][e];
        lg[e] = t;
      }
      int sel[MAX_EXPERTS];
      float den = 0.f, top = 0.f;
      for (int j = 0; j < c.topE; ++j) {
        int best = -1;
        for (int e = 0; e < E; ++e) {
          bool taken = false;
          for (int q = 0; q < j; ++q) taken |= sel[q] == e;
          if (!taken && (best < 0 || lg[e] > lg[best])) best = e;   // ties keep the lower id
        }
        sel[j] = best;
        if (j == 0) top = lg[best];
        den += expf(lg[best] - top);
      }
      for (int j = 0; j < c.topE; ++j) {
        c.moe_sel[(size_t)row_index * c.topE + j] = sel[j];
        c.moe_wt[(size_t)row_index * c.topE + j] = expf(lg[sel[j]] - top) / den;
      }
    }
    __syncthreads();
  }
}

// Rows of a CTA in turn, the next row on its way (asynchronous copies into shared memory, each thread reads
// back only what it copied itself) while the current one is summed and scaled: with several rows per CTA
// (steps of more rows than SMs) the phase is a chain of row latencies otherwise.  The copies hold no
// registers.  NV = d / 1024 16-byte vectors per thread.
template <typename WT, int NV>
static __device__ __noinline__ void norm_rows_pipelined(const DevCtx& c, const float* g, WT* out, int T, float* s_red, float* smem) {
  constexpr int d = NV * 1024;
  int t = blockIdx.x;
  if (t >= T) return;
  const char* stage = reinterpret_cast<const char*>(smem) + threadIdx.x * 16;   // [NV][FWD_THREADS] x 16 bytes
  const uint32_t stage_s = (uint32_t)__cvta_generic_to_shared(stage);
  const float* src = c.h + (size_t)t * d + threadIdx.x * 4;
#pragma unroll
  for (int k = 0; k < NV; ++k)
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(stage_s + k * FWD_THREADS * 16), "l"(src + k * FWD_THREADS * 4) : "memory");
  asm volatile("cp.async.commit_group;" ::: "memory");
#pragma unroll 1
  for (; t < T; t += gridDim.x) {
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    float4 cur[NV];
#pragma unroll
    for (int k = 0; k < NV; ++k) cur[k] = *reinterpret_cast<const float4*>(stage + k * FWD_THREADS * 16);
    if (t + (int)gridDim.x < T) {
      src += (size_t)gridDim.x * d;
#pragma unroll
      for (int k = 0; k < NV; ++k)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(stage_s + k * FWD_THREADS * 16), "l"(src + k * FWD_THREADS * 4) : "memory");
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
    float ss = 0.f;
#pragma unroll
    for (int k = 0; k < NV; ++k) {  // fixed order, the same as norm_row_cta
      ss = fmaf(cur[k].x, cur[k].x, ss); ss = fmaf(cur[k].y, cur[k].y, ss); ss = fmaf(cur[k].z, cur[k].z, ss); ss = fmaf(cur[k].w, cur[k].w, ss);
    }
    ss = block_sum(ss, s_red);
    const float inv = rsqrtf(ss * (1.0f / (float)d) + c.rms_eps);
    WT* orow = out + (size_t)t * d + threadIdx.x * 4;
#pragma unroll
    for (int k = 0; k < NV; ++k) {
      const float4 gg = *reinterpret_cast<const float4*>(g + (k * FWD_THREADS + threadIdx.x) * 4);
      store4<WT>(orow + k * FWD_THREADS * 4, cur[k].x * inv * gg.x, cur[k].y * inv * gg.y, cur[k].z * inv * gg.z, cur[k].w * inv * gg.w);
    }
  }
}

// ---- RMSNorm of the residual rows into the operand buffer; layer 0 gathers the
// embedding first.
template <typename WT>
static __device__ __noinline__ void phase_norm(const DevCtx& c, int layer, int which /*0: norm1, 1: norm2*/, float* smem) {
  __shared__ float s_red[FWD_THREADS / 32];
  const int T = c.ss->cur_T;
  const float* g = wptr_f(c, which == 0 ? 6 : 7) + (size_t)layer * c.d;
  WT* out = reinterpret_cast<WT*>(c.xn);
  // fused path: both sum-of-squares buffers start a step at zero (the last layer's leftovers)
  if (c.fused_norm && which == 0 && layer == 0)
    for (int i = blockIdx.x * FWD_THREADS + threadIdx.x; i < c.Tmax; i += gridDim.x * FWD_THREADS) {
      c.rowss_a[i] = 0.f;
      c.rowss_b[i] = 0.f;
    }
  const float* wr = (which == 1 && c.E > 0) ? wptr_f(c, 5) + (size_t)layer * c.E * c.d : nullptr;
  if (wr == nullptr && !(which == 0 && layer == 0) && T > (int)gridDim.x && (c.d == 4096 || c.d == 2048)) {
    if (c.d == 4096) norm_rows_pipelined<WT, 4>(c, g, out, T, s_red, smem);
    else norm_rows_pipelined<WT, 2>(c, g, out, T, s_red, smem);
    return;
  }
  for (int t = blockIdx.x; t < T; t += gridDim.x) {
    const WT* e = (which == 0 && layer == 0) ? wptr<WT>(c, 0) + (size_t)c.tok_id[t] * c.d : nullptr;
    norm_row_cta<WT>(c, c.h + (size_t)t * c.d, e, g, out + (size_t)t * c.d, s_red, wr, t);
  }
}

// The LM head gives every CTA whole weight tiles when there are at least as many tiles as CTAs: no
// partial sums, so the logits need no clearing.
__device__ __forceinline__ bool lm_head_whole_tiles(const DevCtx& c) { return (c.V + 127) / 128 >= (int)gridDim.x; }

// Fused path: the sum of squares of every residual row is already known (added up by the epilogue of
// the GEMM that completed the row), so the norm is element-wise: n = x * rsqrt(ss / d + eps) * g.
// `rows` null: rows 0 .. R-1 of h go to rows 0 .. R-1 of out; else row r of out comes from row rows[r].
template <typename WT>
__device__ __noinline__ void norm_apply_rows(const float* __restrict__ h, const float* __restrict__ rowss,
                                             const float* __restrict__ g, WT* __restrict__ out, const int32_t* rows, int R,
                                             int d, float eps) {
  constexpr int U = 4;   // items whose loads are in flight before the first store (one CTA per SM: latency-bound otherwise)
  const int d4 = d >> 2;
  const int total = R * d4;   // < 2^31
  const float inv_d = __fdividef(1.0f, (float)d);
  const int stride = gridDim.x * FWD_THREADS;
  for (int base = blockIdx.x * FWD_THREADS + threadIdx.x; base < total; base += U * stride) {
    float4 v[U], gg[U];
    float ss[U];
    int r[U], j[U];
#pragma unroll
    for (int k = 0; k < U; ++k) {
      const int idx = min(base + k * stride, total - 1);   // clamped: the tail loads a valid item twice
      r[k] = idx / d4;
      j[k] = (idx - r[k] * d4) * 4;
      const int t = rows != nullptr ? rows[r[k]] : r[k];
      v[k] = __ldcg(reinterpret_cast<const float4*>(h + (size_t)t * d + j[k]));
      ss[k] = __ldcg(rowss + t);
      gg[k] = *reinterpret_cast<const float4*>(g + j[k]);
    }
#pragma unroll
    for (int k = 0; k < U; ++k) {
      if (base + k * stride < total) {
        const float inv = rsqrtf(ss[k] * inv_d + eps);
        store4<WT>(out + (size_t)r[k] * d + j[k], v[k].x * inv * gg[k].x, v[k].y * inv * gg[k].y, v[k].z * inv * gg[k].z,
                   v[k].w * inv * gg[k].w);
      }
    }
  }
}

// Norm phases of the fused path for layers whose input rows are complete with their sums of squares:
// which 0 = first norm of layer > 0 (reads rowss_b, clears rowss_a), 1 = second norm (reads rowss_a,
// clears rowss_b).  The cleared buffer is the one the next GEMM epilogue adds into.
template <typename WT>
static __device__ __noinline__ void phase_norm_apply(const DevCtx& c, int layer, int which, int T) {
  const float* g = wptr_f(c, which == 0 ? 6 : 7) + (size_t)layer * c.d;
  float* clear = which == 0 ? c.rowss_a : c.rowss_b;
  for (int i = blockIdx.x * FWD_THREADS + threadIdx.x; i < T; i += gridDim.x * FWD_THREADS) clear[i] = 0.f;
  norm_apply_rows<WT>(c.h, which == 0 ? c.rowss_b : c.rowss_a, g, reinterpret_cast<WT*>(c.xn), nullptr, T, c.d, c.rms_eps);
}

// Final norm of the sampled rows only (the LM head runs on those rows).
template <typename WT>
static __device__ __noinline__ void phase_final_norm(const DevCtx& c) {
  __shared__ float s_red[FWD_THREADS / 32];
  const int R = c.ss->cur_rows;
  const float* g = wptr_f(c, 8);
  WT* out = reinterpret_cast<WT*>(c.xs);
  if (c.gemm_tc && !lm_head_whole_tiles(c)) zero_floats(c.logits, (long long)R * c.V);
  if (c.fused_norm) {
    norm_apply_rows<WT>(c.h, c.rowss_b, g, out, c.row_tok, R, c.d, c.rms_eps);
    return;
  }
  for (int r = blockIdx.x; r < R; r += gridDim.x)
    norm_row_cta<WT>(c, c.h + (size_t)c.row_tok[r] * c.d, nullptr, g, out + (size_t)r * c.d, s_red);
}

// ---- CUDA-core reference GEMM: out[t][n] (+)= sum_k x[t][k] * w[n][k], fp32 accumulate.
// 64x64 output tile, BK = 16, 4x4 outputs per thread.  Deterministic (no split-K).
enum GemmFix : int {
  FIX_NONE = 0,
  FIX_ROPE_KV,  // QKV: RoPE on q and k, q -> 16-bit attention operand, k and v -> paged pool; the tile is cleared
  FIX_SILU,     // gate/up: act = silu(gate) * up in the operand type; both tiles are cleared
  FIX_SUMSQ,    // O and down: add the tile's share of sum(x^2) of every residual row
};
struct GemmArgs {
  const void* x;   // [M][K] operand type
  const void* w;   // [N][K] operand type
  float* out;      // [M][ldo]
  int M, N, K, ldo;
  int accumulate;  // 1: out += result (residual), 0: out = result
  // routed experts: x rows start at row x_row0 of the activation buffer, the weights at row w_row0 of
  // the stacked weight tensor; with row_map the result row t goes to out row row_map[t], scaled by
  // row_scale[t], always added (several experts contribute to one token)
  int x_row0 = 0;
  long long w_row0 = 0;
  const int32_t* row_map = nullptr;
  const float* row_scale = nullptr;
  // tensor-core path: element-wise work that consumes the finished output tiles of this GEMM (run by
  // the CTA that delivers a tile's last partial sum, see tc_finish_tiles)
  int fix = 0;               // FIX_*
  void* fix_out = nullptr;   // FIX_SILU: the activation rows (operand type) matching `out`
  float* fix_rowss = nullptr;// FIX_SUMSQ: per-row sums of squares to add to
};

template <typename WT>
static __device__ __noinline__ void phase_gemm_simt(const GemmArgs& a) {
  constexpr int BM = 64, BN = 64, BK = 16;
  __shared__ float xs[BK][BM + 4];
  __shared__ float ws[BK][BN + 4];
  const WT* X = reinterpret_cast<const WT*>(a.x);
  const WT* W = reinterpret_cast<const WT*>(a.w);
  const int tiles_m = (a.M + BM - 1) / BM, tiles_n = (a.N + BN - 1) / BN;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;  // 16 x 16 threads
  const int lrow = threadIdx.x >> 2, lk = (threadIdx.x & 3) * 4;
  for (int tile = blockIdx.x; tile < tiles_m * tiles_n; tile += gridDim.x) {
    const int tm = tile % tiles_m, tn = tile / tiles_m;
    const int m0 = tm * BM, n0 = tn * BN;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (int k0 = 0; k0 < a.K; k0 += BK) {
      {
        const int m = m0 + lrow, n = n0 + lrow;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int k = k0 + lk + e;
          xs[lk + e][lrow] = (m < a.M && k < a.K) ? OpType<WT>::to_f(X[(size_t)m * a.K + k]) : 0.f;
          ws[lk + e][lrow] = (n < a.N && k < a.K) ? OpType<WT>::to_f(W[(size_t)n * a.K + k]) : 0.f;
        }
      }
      __syncthreads();
#pragma unroll
      for (int k = 0; k < BK; ++k) {
        float xv[4], wv[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) xv[i] = xs[k][ty * 4 + i];
#pragma unroll
        for (int j = 0; j < 4; ++j) wv[j] = ws[k][tx * 4 + j];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(xv[i], wv[j], acc[i][j]);
      }
      __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int m = m0 + ty * 4 + i;
      if (m >= a.M) continue;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int n = n0 + tx * 4 + j;
        if (n >= a.N) continue;
        if (a.row_map != nullptr) {
          atomicAdd(a.out + (size_t)a.row_map[m] * a.ldo + n, a.row_scale[m] * acc[i][j]);
        } else {
          float* o = a.out + (size_t)m * a.ldo + n;
          *o = a.accumulate ? (*o + acc[i][j]) : acc[i][j];
        }
      }
    }
  }
}

// ---- RoPE (rotate-half pairing) on q and k, then K/V into the paged pool --------------
// KV pool layout [L][2][n_blocks][Hkv][bs][hd]: one (block, kv head) tile is contiguous.
template <typename WT>
__device__ __forceinline__ WT* kv_tile(const DevCtx& c, int layer, int kv, int block, int head) {
  const size_t tile = (size_t)c.bs * c.hd;
  return reinterpret_cast<WT*>(c.kv_base) +
         ((((size_t)layer * 2 + kv) * c.n_blocks + block) * c.Hkv + head) * tile;
}

template <typename WT>
static __device__ __noinline__ void phase_rope_kv(const DevCtx& c, int layer) {
  // one thread: four consecutive rotation pairs (i .. i+3, i+half .. i+half+3) of one head of one row
  const int T = c.ss->cur_T;
  const int half = c.hd / 2, quads = half / 4;
  const int heads = c.Hq + 2 * c.Hkv;
  const int total = T * heads * quads;   // < 2^31
#pragma unroll 2
  for (int idx = blockIdx.x * FWD_THREADS + threadIdx.x; idx < total; idx += gridDim.x * FWD_THREADS) {
    const int i = (idx % quads) * 4;
    const int hh = (idx / quads) % heads;
    const int t = idx / (quads * heads);
    float* row = c.qkv + (size_t)t * c.qkv_dim + (size_t)hh * c.hd;
    const float4 x1 = *reinterpret_cast<const float4*>(row + i), x2 = *reinterpret_cast<const float4*>(row + i + half);
    if (hh < c.Hq + c.Hkv) {
      const int pos = c.tok_pos[t];
      const float4 cs = *reinterpret_cast<const float4*>(c.rope_cos + (size_t)pos * half + i);
      const float4 sn = *reinterpret_cast<const float4*>(c.rope_sin + (size_t)pos * half + i);
      // explicit fused forms: every instance of this code rounds the same way
#define BLINK_ROT1(a, b, cc, ss_) fmaf((a), (cc), -__fmul_rn((b), (ss_)))
#define BLINK_ROT2(a, b, cc, ss_) fmaf((b), (cc), __fmul_rn((a), (ss_)))
      const float4 y1 = make_float4(BLINK_ROT1(x1.x, x2.x, cs.x, sn.x), BLINK_ROT1(x1.y, x2.y, cs.y, sn.y),
                                    BLINK_ROT1(x1.z, x2.z, cs.z, sn.z), BLINK_ROT1(x1.w, x2.w, cs.w, sn.w));
      const float4 y2 = make_float4(BLINK_ROT2(x1.x, x2.x, cs.x, sn.x), BLINK_ROT2(x1.y, x2.y, cs.y, sn.y),
                                    BLINK_ROT2(x1.z, x2.z, cs.z, sn.z), BLINK_ROT2(x1.w, x2.w, cs.w, sn.w));
#undef BLINK_ROT1
#undef BLINK_ROT2
      if (hh < c.Hq) {
        if constexpr (sizeof(WT) == 2) {   // 16-bit path: q is an operand of the attention contraction
          WT* qd = reinterpret_cast<WT*>(c.qb) + (size_t)t * c.q_dim + (size_t)hh * c.hd;
          store4<WT>(qd + i, y1.x, y1.y, y1.z, y1.w);
          store4<WT>(qd + i + half, y2.x, y2.y, y2.z, y2.w);
        } else {
          *reinterpret_cast<float4*>(row + i) = y1;
          *reinterpret_cast<float4*>(row + i + half) = y2;
        }
      } else {
        const int sm = c.tok_slotmap[t];
        WT* dst = kv_tile<WT>(c, layer, 0, sm / c.bs, hh - c.Hq) + (size_t)(sm % c.bs) * c.hd;
        store4<WT>(dst + i, y1.x, y1.y, y1.z, y1.w);
        store4<WT>(dst + i + half, y2.x, y2.y, y2.z, y2.w);
      }
    } else {
      const int sm = c.tok_slotmap[t];
      WT* dst = kv_tile<WT>(c, layer, 1, sm / c.bs, hh - c.Hq - c.Hkv) + (size_t)(sm % c.bs) * c.hd;
      store4<WT>(dst + i, x1.x, x1.y, x1.z, x1.w);
      store4<WT>(dst + i + half, x2.x, x2.y, x2.z, x2.w);
    }
    if (c.gemm_tc) {   // the split-K GEMM of the next layer adds partial sums into this buffer: leave it cleared
      *reinterpret_cast<float4*>(row + i) = make_float4(0.f, 0.f, 0.f, 0.f);
      *reinterpret_cast<float4*>(row + i + half) = make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
}

// ---- element-wise consumers of finished GEMM output tiles (fused path) ----------------------------
// A tile is 128 consecutive output features of rows [t0, t1); the eight warps take rows in turn and a
// lane owns four consecutive features, so every access is one 512-byte line per row.  The fp32 sums
// were produced by reductions at L2 by several CTAs: they are read with .cg loads.

// QKV tile nt: RoPE on the q and k heads it covers (the rotation partner i + hd/2 of a feature lies in
// the same tile, hd/8 lanes away), q into the 16-bit attention operand, k and v into the paged pool;
// then the tile is cleared for the next GEMM that adds partial sums into this buffer.
constexpr int FIX_U = 8;   // rows per warp whose loads are issued before the first dependent use
constexpr int FIX_WARPS = FWD_THREADS / 32;

template <typename WT>
__device__ __noinline__ void fixup_rope_kv(const DevCtx& c, int layer, int nt, int t0, int t1) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int hd = c.hd, half = hd >> 1;
  const int f = nt * 128 + lane * 4;          // feature of this lane
  const int hh = f / hd, i0 = f - hh * hd;    // head and offset inside it
  const bool low = i0 < half;
  const int i = low ? i0 : i0 - half;         // rotation pair index
  const int partner = half >> 2;              // lanes between the two halves of a pair
  if (f >= c.qkv_dim) return;                 // whole warp: tiles are not ragged on this path
  const bool rot = hh < c.Hq + c.Hkv;
  const bool is_q = hh < c.Hq;
  const int kv = hh < c.Hq + c.Hkv ? 0 : 1;
  const int kvh = hh - c.Hq - kv * c.Hkv;
  for (int tb = t0 + w; tb < t1; tb += FIX_WARPS * FIX_U) {
    float4 x[FIX_U];
    int pos[FIX_U], sm[FIX_U];
#pragma unroll
    for (int u = 0; u < FIX_U; ++u) {
      const int t = min(tb + u * FIX_WARPS, t1 - 1);   // clamped: rows past the end repeat the last one (not stored)
      x[u] = __ldcg(reinterpret_cast<const float4*>(c.qkv + (size_t)t * c.qkv_dim + f));
      pos[u] = rot ? c.tok_pos[t] : 0;
      sm[u] = is_q ? 0 : c.tok_slotmap[t];
    }
#pragma unroll
    for (int u = 0; u < FIX_U; ++u) {
      const int t = tb + u * FIX_WARPS;
      float4 o;
      o.x = __shfl_xor_sync(0xffffffffu, x[u].x, partner);
      o.y = __shfl_xor_sync(0xffffffffu, x[u].y, partner);
      o.z = __shfl_xor_sync(0xffffffffu, x[u].z, partner);
      o.w = __shfl_xor_sync(0xffffffffu, x[u].w, partner);
      if (t >= t1) continue;   // uniform over the warp
      float4 y = x[u];
      float4 cs[FIX_U], sn[FIX_U];
      if (rot) {
        cs[u] = *reinterpret_cast<const float4*>(c.rope_cos + (size_t)pos[u] * half + i);
        sn[u] = *reinterpret_cast<const float4*>(c.rope_sin + (size_t)pos[u] * half + i);
        // the same explicit fused forms as the stand-alone RoPE phase: x1 = low half, x2 = high half
        if (low) {
          y = make_float4(fmaf(x[u].x, cs[u].x, -__fmul_rn(o.x, sn[u].x)), fmaf(x[u].y, cs[u].y, -__fmul_rn(o.y, sn[u].y)),
                          fmaf(x[u].z, cs[u].z, -__fmul_rn(o.z, sn[u].z)), fmaf(x[u].w, cs[u].w, -__fmul_rn(o.w, sn[u].w)));
        } else {
          y = make_float4(fmaf(x[u].x, cs[u].x, __fmul_rn(o.x, sn[u].x)), fmaf(x[u].y, cs[u].y, __fmul_rn(o.y, sn[u].y)),
                          fmaf(x[u].z, cs[u].z, __fmul_rn(o.z, sn[u].z)), fmaf(x[u].w, cs[u].w, __fmul_rn(o.w, sn[u].w)));
        }
      }
      WT* dst;
      if (is_q) dst = reinterpret_cast<WT*>(c.qb) + (size_t)t * c.q_dim + (size_t)hh * hd + i0;
      else dst = kv_tile<WT>(c, layer, kv, sm[u] / c.bs, kvh) + (size_t)(sm[u] % c.bs) * hd + i0;
      store4<WT>(dst, y.x, y.y, y.z, y.w);
      __stcg(reinterpret_cast<float4*>(c.qkv + (size_t)t * c.qkv_dim + f), make_float4(0.f, 0.f, 0.f, 0.f));
    }
  }
}

// gate tile j and up tile j of rows [t0, t1) of `gu` (row pitch 2F): act = silu(gate) * up; both cleared.
template <typename WT>
__device__ __noinline__ void fixup_silu(float* gu, WT* act, int F, int f0, int width, int t0, int t1) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int f = f0 + lane * 4;
  if (lane * 4 >= width || f >= F) return;
  for (int tb = t0 + w; tb < t1; tb += FIX_WARPS * FIX_U) {
    float4 g[FIX_U], u4[FIX_U];
#pragma unroll
    for (int u = 0; u < FIX_U; ++u) {
      const int t = min(tb + u * FIX_WARPS, t1 - 1);
      g[u] = __ldcg(reinterpret_cast<const float4*>(gu + (size_t)t * 2 * F + f));
      u4[u] = __ldcg(reinterpret_cast<const float4*>(gu + (size_t)t * 2 * F + F + f));
    }
#pragma unroll
    for (int u = 0; u < FIX_U; ++u) {
      const int t = tb + u * FIX_WARPS;
      if (t >= t1) continue;
      store4<WT>(act + (size_t)t * F + f, __fdividef(g[u].x, 1.0f + __expf(-g[u].x)) * u4[u].x, __fdividef(g[u].y, 1.0f + __expf(-g[u].y)) * u4[u].y,
                 __fdividef(g[u].z, 1.0f + __expf(-g[u].z)) * u4[u].z, __fdividef(g[u].w, 1.0f + __expf(-g[u].w)) * u4[u].w);
      __stcg(reinterpret_cast<float4*>(gu + (size_t)t * 2 * F + f), make_float4(0.f, 0.f, 0.f, 0.f));
      __stcg(reinterpret_cast<float4*>(gu + (size_t)t * 2 * F + F + f), make_float4(0.f, 0.f, 0.f, 0.f));
    }
  }
}

// residual tile nt of rows [t0, t1): its share of sum(x^2) per row
static __device__ __noinline__ void fixup_sumsq(const float* h, int ld, int N, float* rowss, int nt, int t0, int t1) {
  constexpr int U = 8;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int f = nt * 128 + lane * 4;
  for (int tb = t0 + w; tb < t1; tb += FIX_WARPS * U) {
    float4 x[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int t = min(tb + u * FIX_WARPS, t1 - 1);
      x[u] = f < N ? __ldcg(reinterpret_cast<const float4*>(h + (size_t)t * ld + f)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int t = tb + u * FIX_WARPS;
      float s = fmaf(x[u].x, x[u].x, fmaf(x[u].y, x[u].y, fmaf(x[u].z, x[u].z, x[u].w * x[u].w)));
      s = warp_sum(s);
      if (lane == 0 && t < t1) atomicAdd(rowss + t, s);
    }
  }
}

// ---- paged attention ---------------------------------------------------------------------
// Unit of work: (row t, kv head g): the n_rep query heads of the group share every K/V
// load.  The 8 warps of the CTA take KV blocks round-robin; within a warp a 16-byte
// vector load per lane covers whole (block, head) tiles with coalesced 512-byte rows.
// Online softmax per warp, merged across warps in shared memory at the end.
template <typename WT, int HD, int NREP>
static __device__ __noinline__ void phase_attention(const DevCtx& c, int layer, float* smem) {
  constexpr int CE = 16 / (int)sizeof(WT);  // elements per 16-byte chunk
  constexpr int LPK = HD / CE;              // lanes per key
  constexpr int KPP = 32 / LPK;             // keys per pass
  constexpr int MAXR = NREP;                // query heads per kv head
  constexpr int NW = FWD_THREADS / 32;
  static_assert(LPK <= 32 && KPP >= 1, "head_dim too large for this mapping");
  const int T = c.ss->cur_T;
  constexpr int n_rep = NREP;
  const int bs = c.bs;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int sub = lane / LPK;   // which key of the pass
  const int ch = lane % LPK;    // which 16-byte chunk of the head vector
  // shared: q [NREP][HD], per-warp m,l [NW][NREP], acc [NW][NREP][HD]
  float* s_q = smem;
  float* s_m = s_q + MAXR * HD;
  float* s_l = s_m + NW * MAXR;
  float* s_acc = s_l + NW * MAXR;
  WT* out = reinterpret_cast<WT*>(c.attn);

  const int units = T * c.Hkv;
  for (int u = blockIdx.x; u < units; u += gridDim.x) {
    const int t = u / c.Hkv, g = u % c.Hkv;
    const int item = c.tok_item[t];
    const int b = c.it_bslot[item];
    const int n_ctx = c.tok_pos[t] + 1;
    const int32_t* table = c.block_table + (size_t)b * c.max_blocks_seq;
    __syncthreads();
    for (int i = threadIdx.x; i < n_rep * HD; i += FWD_THREADS)
      s_q[i] = c.qkv[(size_t)t * c.qkv_dim + (size_t)g * n_rep * HD + i] * c.attn_scale;
    __syncthreads();
    float q[MAXR][CE];
    float acc[MAXR][CE];
    float m[MAXR], l[MAXR];
#pragma unroll
    for (int r = 0; r < MAXR; ++r) {
      m[r] = -INFINITY;
      l[r] = 0.f;
#pragma unroll
      for (int e = 0; e < CE; ++e) {
        acc[r][e] = 0.f;
        q[r][e] = (r < n_rep) ? s_q[r * HD + ch * CE + e] : 0.f;
      }
    }
    const int n_kb = (n_ctx + bs - 1) / bs;
    for (int kb = w; kb < n_kb; kb += NW) {
      const int blk = table[kb];
      const WT* kt = kv_tile<WT>(c, layer, 0, blk, g);
      const WT* vt = kv_tile<WT>(c, layer, 1, blk, g);
      for (int k0 = 0; k0 < bs; k0 += KPP) {
        const int key = k0 + sub;
        const int kpos = kb * bs + key;
        const bool valid = key < bs && kpos < n_ctx;
        float kf[CE], vf[CE];
        if (valid) {
          const uint4 kr = *reinterpret_cast<const uint4*>(kt + (size_t)key * HD + ch * CE);
          const uint4 vr = *reinterpret_cast<const uint4*>(vt + (size_t)key * HD + ch * CE);
          const WT* kp = reinterpret_cast<const WT*>(&kr);
          const WT* vp = reinterpret_cast<const WT*>(&vr);
#pragma unroll
          for (int e = 0; e < CE; ++e) { kf[e] = OpType<WT>::to_f(kp[e]); vf[e] = OpType<WT>::to_f(vp[e]); }
        } else {
#pragma unroll
          for (int e = 0; e < CE; ++e) { kf[e] = 0.f; vf[e] = 0.f; }
        }
#pragma unroll
        for (int r = 0; r < MAXR; ++r) {
          if (r >= n_rep) break;
          float s = 0.f;
#pragma unroll
          for (int e = 0; e < CE; ++e) s = fmaf(q[r][e], kf[e], s);
#pragma unroll
          for (int o = LPK / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
          if (!valid) s = -INFINITY;
          // max over the keys of this pass (lanes with different `sub`)
          float mx = s;
#pragma unroll
          for (int o = LPK; o < 32; o <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
          const float m_new = fmaxf(m[r], mx);
          if (m_new == -INFINITY) continue;   // nothing valid yet (uniform across the warp)
          const float corr = __expf(m[r] - m_new);
          const float p = valid ? __expf(s - m_new) : 0.f;
          // l and acc are per-lane partials over this lane's keys; lanes of other `sub`
          // hold the other keys and are merged at the end
          l[r] = l[r] * corr + p;
#pragma unroll
          for (int e = 0; e < CE; ++e) acc[r][e] = fmaf(p, vf[e], acc[r][e] * corr);
          m[r] = m_new;
        }
      }
    }
    // merge lanes that handled different keys (same chunk): sum over `sub`
#pragma unroll
    for (int r = 0; r < MAXR; ++r) {
      if (r >= n_rep) break;
#pragma unroll
      for (int o = LPK; o < 32; o <<= 1) {
        l[r] += __shfl_xor_sync(0xffffffffu, l[r], o);
#pragma unroll
        for (int e = 0; e < CE; ++e) acc[r][e] += __shfl_xor_sync(0xffffffffu, acc[r][e], o);
      }
      // every lane with the same `ch` now holds the warp's full partial
      if (sub == 0) {
#pragma unroll
        for (int e = 0; e < CE; ++e) s_acc[((size_t)w * MAXR + r) * HD + ch * CE + e] = acc[r][e];
        if (ch == 0) { s_m[w * MAXR + r] = m[r]; s_l[w * MAXR + r] = l[r]; }
      }
    }
    __syncthreads();
    // merge the warps: out = sum_w e^(m_w - M) acc_w / sum_w e^(m_w - M) l_w
    for (int i = threadIdx.x; i < n_rep * HD; i += FWD_THREADS) {
      const int r = i / HD, dim = i % HD;
      float M = -INFINITY;
#pragma unroll
      for (int ww = 0; ww < NW; ++ww) M = fmaxf(M, s_m[ww * MAXR + r]);
      float num = 0.f, den = 0.f;
#pragma unroll
      for (int ww = 0; ww < NW; ++ww) {
        const float mw = s_m[ww * MAXR + r];
        if (mw == -INFINITY) continue;
        const float f = __expf(mw - M);
        num += f * s_acc[((size_t)ww * MAXR + r) * HD + dim];
        den += f * s_l[ww * MAXR + r];
      }
      out[(size_t)t * c.q_dim + (size_t)(g * n_rep + r) * HD + dim] = OpType<WT>::from_f(num / den);
    }
  }
}
constexpr int ATTN_SMEM_FLOATS(int HD, int NREP) { return NREP * HD + 2 * 8 * NREP + 8 * NREP * HD; }

// ---- SwiGLU gate: act = silu(gate) * up ------------------------------------------------
// The gate/up buffer comes from HBM (the weight stream of the GEMM before has pushed it out of L2)
// and one CTA per SM leaves eight warps to cover that latency, so every thread has the loads of
// SILU_U items in flight before it stores.  A function of its own: inlined into the loop kernel
// the buffers of loaded values end up in local memory.
// silu(g) * u with the approximate division (2 ulp, then rounded to the operand type): the exact fp32 division
// took a quarter of the SwiGLU phase
template <typename WT>
__device__ __forceinline__ void silu_store(float* gu, WT* out, int t, int j, int F, const float4& g, const float4& u, bool clear) {
  store4<WT>(out + (size_t)t * F + j, __fdividef(g.x, 1.0f + __expf(-g.x)) * u.x, __fdividef(g.y, 1.0f + __expf(-g.y)) * u.y,
             __fdividef(g.z, 1.0f + __expf(-g.z)) * u.z, __fdividef(g.w, 1.0f + __expf(-g.w)) * u.w);
  if (clear) {   // consumed: the next split-K gate/up GEMM adds partial sums into a cleared buffer
    __stcg(reinterpret_cast<float4*>(gu + (size_t)t * 2 * F + j), make_float4(0.f, 0.f, 0.f, 0.f));
    __stcg(reinterpret_cast<float4*>(gu + (size_t)t * 2 * F + F + j), make_float4(0.f, 0.f, 0.f, 0.f));
  }
}
template <typename WT>
__device__ __noinline__ void silu_mul_rows(float* __restrict__ gu, WT* __restrict__ out, int T, int F, bool clear) {
  constexpr int SILU_U = 4;
  const int F4 = F / 4;
  const int total = T * F4;   // < 2^31: at most a few thousand rows
  const int stride = gridDim.x * FWD_THREADS;
  for (int base = blockIdx.x * FWD_THREADS + threadIdx.x; base < total; base += SILU_U * stride) {
    float4 g[SILU_U], u[SILU_U];
#pragma unroll
    for (int k = 0; k < SILU_U; ++k) {
      const int idx = min(base + k * stride, total - 1);   // clamped: the tail loads a valid item twice
      const int t = idx / F4, j = (idx - t * F4) * 4;
      g[k] = __ldcg(reinterpret_cast<const float4*>(gu + (size_t)t * 2 * F + j));
      u[k] = __ldcg(reinterpret_cast<const float4*>(gu + (size_t)t * 2 * F + F + j));
    }
#pragma unroll
    for (int k = 0; k < SILU_U; ++k) {
      const int idx = base + k * stride;
      if (idx < total) {
        const int t = idx / F4;
        silu_store<WT>(gu, out, t, (idx - t * F4) * 4, F, g[k], u[k], clear);
      }
    }
  }
}
// The same over the (token pass, gate/up weight tile) units that the GEMM has not already written as
// activations (a unit is up to 256 rows x 64 features; the GEMM stamps the units it wrote).  Every CTA
// compacts the pending units into shared memory once, then all threads of the grid share their items evenly.
static __device__ __noinline__ int silu_pending_units(const unsigned long long* done, unsigned long long stamp, int n_units, int* list) {
  __shared__ int s_warp[FWD_THREADS / 32];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  int count = 0;   // uniform over the CTA
  for (int b0 = 0; b0 < n_units; b0 += FWD_THREADS) {
    const int unit = b0 + threadIdx.x;
    const bool pend = unit < n_units && __ldcg(done + unit) != stamp;   // written by other SMs: not through L1
    const unsigned m = __ballot_sync(0xffffffffu, pend);
    if (lane == 0) s_warp[w] = __popc(m);
    __syncthreads();
    int off = count, tot = 0;
#pragma unroll
    for (int i = 0; i < FWD_THREADS / 32; ++i) {
      if (i < w) off += s_warp[i];
      tot += s_warp[i];
    }
    if (pend) list[off + __popc(m & ((1u << lane) - 1u))] = unit;
    count += tot;
    __syncthreads();
  }
  return count;
}
// A CTA takes a quarter of a pending unit at a time: 64 rows x 64 features, four items per thread.  The
// loads are asynchronous copies into a staging area in shared memory (each thread reads back only what it
// copied itself), so four items are in flight per thread without holding registers for them: a body that
// needs many registers here changes the register allocation of the other phase functions of the loop
// kernel, to their cost.
constexpr int SILU_STAGE_OFF = 32768 * 4;   // bytes: the staging area follows the list of pending units
template <typename WT>
__device__ __noinline__ void silu_mul_pending(float* __restrict__ gu, WT* __restrict__ out, int T, int F, const int* list, int count) {
  const int tiles = F >> 6;
  const int r_in = threadIdx.x >> 4, col = (threadIdx.x & 15) << 2;
  const char* stage = reinterpret_cast<const char*>(list) + SILU_STAGE_OFF + threadIdx.x * 16;   // [8][FWD_THREADS] x 16 bytes
  const uint32_t stage_s = (uint32_t)__cvta_generic_to_shared(stage);
  for (int q = blockIdx.x; q < count * 4; q += gridDim.x) {
    const int unit = list[q >> 2];
    const int pass = unit / tiles, tile = unit - pass * tiles;
    const int row0 = (pass << 8) + ((q & 3) << 6) + r_in, j = (tile << 6) + col;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int t = row0 + 16 * k;
      if (t < T) {
        const float* src = gu + (size_t)t * 2 * F + j;
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(stage_s + (2 * k) * FWD_THREADS * 16), "l"(src) : "memory");
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(stage_s + (2 * k + 1) * FWD_THREADS * 16), "l"(src + F) : "memory");
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int t = row0 + 16 * k;
      if (t < T) {
        const float4 g = *reinterpret_cast<const float4*>(stage + (2 * k) * FWD_THREADS * 16);
        const float4 u = *reinterpret_cast<const float4*>(stage + (2 * k + 1) * FWD_THREADS * 16);
        silu_store<WT>(gu, out, t, j, F, g, u, true);
      }
    }
  }
}
// The GEMM writes activations itself only in steps of more than one token pass: there its epilogue hides
// behind the tensor-core work of the next tile, while at decode sizes the GEMM is bound by the weight
// stream and the longer epilogue would show.
__device__ __forceinline__ bool gu_direct_step(const DevCtx& c, int T) { return c.gu_direct && T > 256; }
template <typename WT>
static __device__ __noinline__ void phase_silu_mul(const DevCtx& c, int layer, float* smem) {
  const int T = c.E > 0 ? c.ss->cur_T * c.topE : c.ss->cur_T;   // rows of the gate/up buffer
  if (T <= 0) return;
  if (gu_direct_step(c, T)) {
    int* list = reinterpret_cast<int*>(smem);
    const int count = silu_pending_units(c.gu_done, c.ss->iter * (unsigned long long)c.L + (unsigned long long)layer + 1ull, ((T + 255) >> 8) * (c.F >> 6), list);
    silu_mul_pending<WT>(c.gu, reinterpret_cast<WT*>(c.act), T, c.F, list, count);
  } else
    silu_mul_rows<WT>(c.gu, reinterpret_cast<WT*>(c.act), T, c.F, c.gemm_tc != 0);
}

// ---- routed experts: group the (token, expert) pairs by expert and gather their rows ---------
// Every CTA builds the same lists in shared memory (stable: ascending token inside an expert, so
// the order does not depend on timing), CTA 0 publishes them, and all CTAs copy the normed rows
// of the tokens into expert-contiguous order for the per-expert GEMMs.
template <typename WT>
static __device__ __noinline__ void phase_moe_group(const DevCtx& c, float* smem) {
  const int T = c.ss->cur_T, K = c.topE, E = c.E;
  const int A = T * K;   // assignments
  __shared__ int s_off[MAX_EXPERTS + 1];
  int* s_tok = reinterpret_cast<int*>(smem);          // [A] token of each gathered row
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  // counts, then offsets
  if (threadIdx.x <= E) s_off[threadIdx.x] = 0;
  __syncthreads();
  for (int a = threadIdx.x; a < A; a += FWD_THREADS) atomicAdd(&s_off[c.moe_sel[a] + 1], 1);
  __syncthreads();
  if (threadIdx.x == 0)
    for (int e = 0; e < E; ++e) s_off[e + 1] += s_off[e];
  __syncthreads();
  // stable placement: a warp walks all assignments in order for each of its experts
  for (int e = w; e < E; e += FWD_THREADS / 32) {
    int base = s_off[e];
    for (int a0 = 0; a0 < A; a0 += 32) {
      const int a = a0 + lane;
      const bool mine = a < A && c.moe_sel[a] == e;
      const unsigned m = __ballot_sync(0xffffffffu, mine);
      if (mine) {
        const int pos = base + __popc(m & ((1u << lane) - 1u));
        s_tok[pos] = a / K;
        if (blockIdx.x == 0) { c.moe_tok[pos] = a / K; c.moe_gate[pos] = c.moe_wt[a]; }
      }
      base += __popc(m);
    }
  }
  if (blockIdx.x == 0 && threadIdx.x <= E) c.moe_off[threadIdx.x] = s_off[threadIdx.x];
  __syncthreads();
  // gather: one warp per row, 16-byte vectors
  const WT* xn = reinterpret_cast<const WT*>(c.xn);
  WT* xg = reinterpret_cast<WT*>(c.xg);
  const int vec_per_row = c.d * (int)sizeof(WT) / 16;
  for (int r = blockIdx.x * (FWD_THREADS / 32) + w; r < A; r += gridDim.x * (FWD_THREADS / 32)) {
    const uint4* src = reinterpret_cast<const uint4*>(xn + (size_t)s_tok[r] * c.d);
    uint4* dst = reinterpret_cast<uint4*>(xg + (size_t)r * c.d);
    for (int i = lane; i < vec_per_row; i += 32) dst[i] = src[i];
  }
}

// ---- sampling ------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11): counter-based, so the draw for (ticket, index)
// does not depend on batch composition.
__device__ __forceinline__ uint32_t philox4x32_10_word0(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                        uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  return c0;
}

// order-preserving map float -> uint32 (larger float => larger key)
__device__ __forceinline__ uint32_t float_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// ---- top-p (nucleus) arithmetic: Section 4.2 names "Top-P with temperature" as the in-step sampler ----
// Weights are integers, q = floor(exp(z - z0) * 2^40) with z0 the largest z of the row, so that every
// sum is exact and no result depends on the order in which a parallel machine adds: the nucleus is
// the smallest prefix of the order (z desc, index asc) with cum * 2^24 >= P24 * Q (Q = total weight,
// P24 = round(top_p * 2^24) in [1, 2^24]); the draw is renormalised to its weight M: with the 24-bit
// uniform x24, the token is the first of the order with cum > (x24 * M) >> 24.
__device__ __forceinline__ unsigned long long nucleus_weight(float z, float z0) {
  return __double2ull_rd(exp((double)z - (double)z0) * 1099511627776.0);
}
__device__ __forceinline__ unsigned long long nucleus_p24(float top_p) {
  long long p = (long long)rint((double)top_p * 16777216.0);
  return (unsigned long long)(p < 1 ? 1 : (p > 16777216 ? 16777216 : p));
}
// ceil(p24 * Q / 2^24): the weight the nucleus has to reach (Q < 2^58, p24 <= 2^24)
__device__ __forceinline__ unsigned long long nucleus_need(unsigned long long p24, unsigned long long Q) {
  unsigned long long lo = p24 * Q, hi = __umul64hi(p24, Q);
  const unsigned long long lo2 = lo + 16777215ull;
  if (lo2 < lo) hi += 1;
  return (hi << 40) | (lo2 >> 24);
}
// (x24 * M) >> 24
__device__ __forceinline__ unsigned long long nucleus_target(unsigned long long x24, unsigned long long M) {
  return (__umul64hi(x24, M) << 40) | ((x24 * M) >> 24);
}

// Shared state of the whole-row nucleus search (one CTA per row).
constexpr int NUC_CAND = 1024;
struct NucShared {
  unsigned long long m0[256];   // level 0: weight per bucket of z (linear in z between the row's min and max)
  unsigned int c0[256];         //          and number of entries
  unsigned long long m[256];    // deeper levels: buckets linear in the float key inside [klo, khi]
  unsigned int cn[256];
  unsigned long long acc;       // weight of everything ahead of the current member set in the order
  unsigned long long res_cum;   // result: cumulative weight up to and including the entry found
  unsigned int klo, khi, cnt;
  int b0, first, done, res_idx, n;
  float zmin, scale;
  unsigned int chunk_cnt[FWD_THREADS];
};
__device__ __forceinline__ int nuc_bucket0(float z, float zmin, float scale) {
  const int b = (int)((z - zmin) * scale);
  return b < 0 ? 0 : (b > 255 ? 255 : b);
}

// First entry of the order (z desc, index asc) whose cumulative weight exceeds t (t < total weight).
// The member set starts as one level-0 bucket and is narrowed 256-fold per pass over the row (buckets
// over the float-key interval of the set) until it fits the candidate buffer, which is then ranked
// exactly.  A set that cannot be narrowed (more than NUC_CAND equal values) is resolved by index.
static __device__ __noinline__ void nucleus_locate(NucShared& st, const float* lg, int V, float temp, float z0,
                                                   unsigned long long t, float* s_cz, int* s_ci, float* s_sz, int* s_si) {
  const int tid = threadIdx.x;
  if (tid == 0) {
    unsigned long long acc = 0;
    int b = 255;
    for (; b > 0; --b) {
      if (acc + st.m0[b] > t) break;
      acc += st.m0[b];
    }
    st.b0 = b; st.acc = acc; st.cnt = st.c0[b]; st.klo = 0u; st.khi = 0xffffffffu; st.first = 1; st.done = 0;
  }
  __syncthreads();
  const float zmin = st.zmin, scale = st.scale;
  for (int level = 0; level < 8; ++level) {   // a level divides the key interval by 256: four suffice
    const int b0 = st.b0;
    const unsigned int klo = st.klo, khi = st.khi;
    if (st.cnt <= (unsigned)NUC_CAND) {
      // ---- gather the members, rank them exactly, walk the cumulative weights ----
      if (tid == 0) st.n = 0;
      __syncthreads();
      for (int i = tid; i < V; i += FWD_THREADS) {
        const float z = __fdiv_rn(lg[i], temp);
        const unsigned int key = float_key(z);
        if (nuc_bucket0(z, zmin, scale) == b0 && key >= klo && key <= khi) {
          const int p = atomicAdd(&st.n, 1);
          if (p < NUC_CAND) { s_cz[p] = z; s_ci[p] = i; }
        }
      }
      __syncthreads();
      const int nc = min(st.n, NUC_CAND);
      for (int a = tid; a < nc; a += FWD_THREADS) {
        const float za = s_cz[a];
        const int ia = s_ci[a];
        int rank = 0;
        for (int j = 0; j < nc; ++j) {
          const float zj = s_cz[j];
          rank += (zj > za) || (zj == za && s_ci[j] < ia);
        }
        s_sz[rank] = za; s_si[rank] = ia;
      }
      __syncthreads();
      if (tid == 0) {
        unsigned long long cum = st.acc;
        int pick = nc > 0 ? s_si[nc - 1] : 0;
        for (int j = 0; j < nc; ++j) {
          cum += nucleus_weight(s_sz[j], z0);
          if (cum > t) { pick = s_si[j]; break; }
        }
        st.res_idx = pick; st.res_cum = cum; st.done = 1;
      }
      __syncthreads();
      return;
    }
    if (st.first) {   // key interval of the level-0 bucket's members
      __syncthreads();
      if (tid == 0) { st.klo = 0xffffffffu; st.khi = 0u; }
      __syncthreads();
      for (int i = tid; i < V; i += FWD_THREADS) {
        const float z = __fdiv_rn(lg[i], temp);
        if (nuc_bucket0(z, zmin, scale) == b0) {
          const unsigned int key = float_key(z);
          atomicMin(&st.klo, key);
          atomicMax(&st.khi, key);
        }
      }
      __syncthreads();
      if (tid == 0) st.first = 0;
      __syncthreads();
      continue;   // same member set, now with its key interval
    }
    if (klo == khi) {
      // ---- more than NUC_CAND entries with one and the same z: equal weights, ordered by index ----
      const float z = __uint_as_float((klo & 0x80000000u) ? (klo & 0x7fffffffu) : ~klo);
      const unsigned long long q0 = nucleus_weight(z, z0);            // > 0: the set's weight exceeds t - acc
      const unsigned long long jl = q0 > 0 ? (t - st.acc) / q0 : 0;   // entries of the set ahead of the one sought
      const int ch = (V + FWD_THREADS - 1) / FWD_THREADS;
      const int i0 = tid * ch, i1 = min(V, i0 + ch);
      unsigned int mine = 0;
      for (int i = i0; i < i1; ++i) {
        const float zi = __fdiv_rn(lg[i], temp);
        mine += (nuc_bucket0(zi, zmin, scale) == b0 && float_key(zi) == klo) ? 1u : 0u;
      }
      st.chunk_cnt[tid] = mine;
      __syncthreads();
      unsigned long long before = 0;
      for (int k = 0; k < tid; ++k) before += st.chunk_cnt[k];
      if (jl >= before && jl < before + mine) {
        unsigned long long seen = before;
        for (int i = i0; i < i1; ++i) {
          const float zi = __fdiv_rn(lg[i], temp);
          if (nuc_bucket0(zi, zmin, scale) == b0 && float_key(zi) == klo) {
            if (seen == jl) { st.res_idx = i; st.res_cum = st.acc + (jl + 1) * q0; st.done = 1; break; }
            ++seen;
          }
        }
      }
      __syncthreads();
      if (tid == 0 && !st.done) { st.res_idx = 0; st.res_cum = st.acc; st.done = 1; }   // cannot happen for t < total
      __syncthreads();
      return;
    }
    // ---- one more level: 256 buckets over the key interval [klo, khi] ----
    st.m[tid] = 0ull;
    st.cn[tid] = 0u;
    __syncthreads();
    const unsigned long long W = (unsigned long long)khi - klo + 1ull;
    for (int i = tid; i < V; i += FWD_THREADS) {
      const float z = __fdiv_rn(lg[i], temp);
      const unsigned int key = float_key(z);
      if (nuc_bucket0(z, zmin, scale) == b0 && key >= klo && key <= khi) {
        const int b = (int)((((unsigned long long)(key - klo)) << 8) / W);
        atomicAdd(&st.m[b], nucleus_weight(z, z0));
        atomicAdd(&st.cn[b], 1u);
      }
    }
    __syncthreads();
    if (tid == 0) {
      unsigned long long acc = st.acc;
      int b = 255;
      for (; b > 0; --b) {
        if (acc + st.m[b] > t) break;
        acc += st.m[b];
      }
      st.acc = acc;
      st.cnt = st.cn[b];
      // keys of bucket b: (key - klo) * 256 / W == b
      st.klo = klo + (unsigned int)(((unsigned long long)b * W + 255ull) >> 8);
      st.khi = klo + (unsigned int)((((unsigned long long)(b + 1) * W + 255ull) >> 8) - 1ull);
    }
    __syncthreads();
  }
  if (tid == 0 && !st.done) { st.res_idx = 0; st.res_cum = st.acc; st.done = 1; }
  __syncthreads();
}

// Top-p over the whole row (no top-k cut): z = logit / T, weights and order as described above.
// The result is returned by thread 0 (other threads return -1).
static __device__ __noinline__ int sample_row_nucleus(const float* lg, int V, float temp, float top_p, unsigned long long ticket,
                                                      int gen_index, unsigned long long seed, float* smem) {
  __shared__ NucShared st;
  __shared__ float s_mx[FWD_THREADS / 32], s_mn[FWD_THREADS / 32];
  const int tid = threadIdx.x;
  float* s_cz = smem + 256;
  int* s_ci = reinterpret_cast<int*>(smem + 256 + NUC_CAND);
  float* s_sz = smem + 256 + 2 * NUC_CAND;
  int* s_si = reinterpret_cast<int*>(smem + 256 + 3 * NUC_CAND);
  __syncthreads();
  // range of the row (z is monotone in the logit, so min and max can be taken on logits)
  float lmax = -INFINITY, lmin = INFINITY;
  for (int i = tid; i < V; i += FWD_THREADS) {
    const float v = lg[i];
    lmax = fmaxf(lmax, v);
    lmin = fminf(lmin, v);
  }
  lmax = warp_max(lmax);
  lmin = -warp_max(-lmin);
  if ((tid & 31) == 0) { s_mx[tid >> 5] = lmax; s_mn[tid >> 5] = lmin; }
  st.m0[tid] = 0ull;
  st.c0[tid] = 0u;
  __syncthreads();
#pragma unroll
  for (int i = 0; i < FWD_THREADS / 32; ++i) { lmax = fmaxf(lmax, s_mx[i]); lmin = fminf(lmin, s_mn[i]); }
  const float z0 = __fdiv_rn(lmax, temp), zmin = __fdiv_rn(lmin, temp);
  const float scale = z0 > zmin ? 255.0f / (z0 - zmin) : 0.0f;
  if (tid == 0) { st.zmin = zmin; st.scale = scale; }
  // level 0: weights per bucket of z
  for (int i = tid; i < V; i += FWD_THREADS) {
    const float z = __fdiv_rn(lg[i], temp);
    const int b = nuc_bucket0(z, zmin, scale);
    atomicAdd(&st.m0[b], nucleus_weight(z, z0));
    atomicAdd(&st.c0[b], 1u);
  }
  __syncthreads();
  __shared__ unsigned long long s_t;
  if (tid == 0) {
    unsigned long long Q = 0;
    for (int b = 0; b < 256; ++b) Q += st.m0[b];
    s_t = nucleus_need(nucleus_p24(top_p), Q) - 1ull;   // first entry with cum >= need  <=>  cum > need - 1
  }
  __syncthreads();
  nucleus_locate(st, lg, V, temp, z0, s_t, s_cz, s_ci, s_sz, s_si);   // end of the nucleus: its weight is res_cum
  if (tid == 0) {
    const uint32_t x = philox4x32_10_word0((uint32_t)ticket, (uint32_t)(ticket >> 32), (uint32_t)gen_index, 0u,
                                           (uint32_t)seed, (uint32_t)(seed >> 32));
    s_t = nucleus_target((unsigned long long)(x >> 8), st.res_cum);
  }
  __syncthreads();
  nucleus_locate(st, lg, V, temp, z0, s_t, s_cz, s_ci, s_sz, s_si);
  const int result = tid == 0 ? st.res_idx : -1;
  __syncthreads();
  return result;
}

// One CTA per sampled row.  Greedy: lowest index among the maxima.  Top-k: z = logit / T
// (IEEE fp32 divide); the k largest by (z desc, index asc) are found with a radix select
// on the float keys; weights exp(z - z0) and the inverse-CDF walk run in fp64.
// The result is returned by thread 0 (other threads return -1).
static __device__ int sample_row(const float* lg, int V, int top_k, float temp, float top_p, unsigned long long ticket,
                                 int gen_index, unsigned long long seed, float* smem) {
  constexpr int CAND_MAX = 1024;
  const int tid = threadIdx.x;
  uint32_t* s_hist = reinterpret_cast<uint32_t*>(smem);             // [256]
  float* s_cz = smem + 256;                                          // [CAND_MAX]
  int* s_ci = reinterpret_cast<int*>(smem + 256 + CAND_MAX);         // [CAND_MAX]
  __shared__ float s_bv[FWD_THREADS / 32];
  __shared__ int s_bi[FWD_THREADS / 32];
  __shared__ unsigned long long s_prefix, s_mask;
  __shared__ int s_remaining, s_ncand;
  __shared__ float s_tz[MAX_TOPK];
  __shared__ int s_ti[MAX_TOPK];
  int result = -1;
  const bool nucleus = top_p > 0.f && top_p < 1.f;   // outside (0, 1): no nucleus cut
  if (top_k <= 0 && nucleus) return sample_row_nucleus(lg, V, temp, top_p, ticket, gen_index, seed, smem);
  __syncthreads();
  if (top_k <= 0) {
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int i = tid; i < V; i += FWD_THREADS) {
      const float v = lg[i];
      if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    if ((tid & 31) == 0) { s_bv[tid >> 5] = bv; s_bi[tid >> 5] = bi; }
    __syncthreads();
    if (tid == 0) {
      for (int i = 1; i < FWD_THREADS / 32; ++i)
        if (s_bv[i] > bv || (s_bv[i] == bv && s_bi[i] < bi)) { bv = s_bv[i]; bi = s_bi[i]; }
      result = bi;
    }
    __syncthreads();
    return result;
  }
  const int k = min(top_k, V);
  // Fast path.  Every thread takes the maximum of its strided share of the row; the k-th largest
  // of those 256 maxima, tau, is a lower bound of the k-th largest z of the row (k threads hold an
  // element >= tau each), so {z >= tau} contains the top k and is usually a few dozen elements.
  // z = logit / T is monotone in the logit, so the maxima can be taken on logits and divided once.
  {
    float* s_tm = smem;   // [FWD_THREADS] thread maxima of z (aliases the histogram, not live yet)
    float lmax = -INFINITY;
    const bool vec = (V & 3) == 0 && ((size_t)lg & 15) == 0;
    if (vec) {
      const float4* lg4 = reinterpret_cast<const float4*>(lg);
#pragma unroll 8
      for (int i = tid; i < V / 4; i += FWD_THREADS) {
        const float4 v = lg4[i];
        lmax = fmaxf(fmaxf(lmax, fmaxf(v.x, v.y)), fmaxf(v.z, v.w));
      }
    } else {
      for (int i = tid; i < V; i += FWD_THREADS) lmax = fmaxf(lmax, lg[i]);
    }
    const float zmax = __fdiv_rn(lmax, temp);
    s_tm[tid] = zmax;
    if (tid == 0) s_ncand = 0;
    __syncthreads();
    int rank = 0;
    for (int j = 0; j < FWD_THREADS; ++j) {
      const float zj = s_tm[j];
      rank += (zj > zmax) || (zj == zmax && j < tid);
    }
    __syncthreads();
    if (rank == k - 1) s_tm[0] = zmax;
    __syncthreads();
    const float tau = s_tm[0];
    __syncthreads();
    if (tau > -INFINITY) {
      // cheap conservative test on the logit first, the exact one on z for the survivors
      const float x = tau * temp;
      const float thr_l = x - fabsf(x) * 9.5367431640625e-7f - 1e-30f;
      auto consider = [&](float v, int i) {
        if (v >= thr_l) {
          const float z = __fdiv_rn(v, temp);
          if (z >= tau) {
            const int p = atomicAdd(&s_ncand, 1);
            if (p < CAND_MAX) { s_cz[p] = z; s_ci[p] = i; }
          }
        }
      };
      if (vec) {
        const float4* lg4 = reinterpret_cast<const float4*>(lg);
#pragma unroll 8
        for (int i = tid; i < V / 4; i += FWD_THREADS) {
          const float4 v = lg4[i];
          if (fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w)) >= thr_l) {
            consider(v.x, 4 * i); consider(v.y, 4 * i + 1); consider(v.z, 4 * i + 2); consider(v.w, 4 * i + 3);
          }
        }
      } else {
        for (int i = tid; i < V; i += FWD_THREADS) consider(lg[i], i);
      }
    }
    __syncthreads();
  }
  const bool fast_ok = s_ncand >= k && s_ncand <= CAND_MAX;
  __syncthreads();
  if (!fast_ok) {
  // Fallback (huge plateaus of equal values, or fewer than k finite thread maxima):
  // radix select over the composite key (z key, ~index): unique keys, so ties in z
  // break towards the lower index and the k-th key is exact.  Refine 8 bits at a time
  // until the set {key >= prefix} (>= k elements by construction) fits the sort buffer.
  if (tid == 0) { s_prefix = 0; s_mask = 0; s_remaining = k; }
  __syncthreads();
  for (int shift = 56; shift >= 0; shift -= 8) {
    s_hist[tid] = 0;   // FWD_THREADS == 256 bins
    __syncthreads();
    const unsigned long long prefix = s_prefix, mask = s_mask;
    for (int i = tid; i < V; i += FWD_THREADS) {
      const unsigned long long key =
          ((unsigned long long)float_key(__fdiv_rn(lg[i], temp)) << 32) | (uint32_t)(~(uint32_t)i);
      if ((key & mask) == prefix) atomicAdd(&s_hist[(unsigned)(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid == 0) {
      const int need = s_remaining;   // how many are still needed from inside the current prefix
      int bin = 255;
      uint32_t above = 0;
      for (; bin > 0; --bin) {
        if (above + s_hist[bin] >= (uint32_t)need) break;
        above += s_hist[bin];
      }
      s_remaining = need - (int)above;
      s_prefix = prefix | ((unsigned long long)bin << shift);
      s_mask = mask | (255ull << shift);
      // keys >= new prefix: those in strictly higher bins at every level so far, plus this bin
      s_ncand = (k - s_remaining) + (int)s_hist[bin];
    }
    __syncthreads();
    if (s_ncand <= CAND_MAX) break;
  }
  const unsigned long long thr = s_prefix;
  __syncthreads();
  if (tid == 0) s_ncand = 0;
  __syncthreads();
  for (int i = tid; i < V; i += FWD_THREADS) {
    const float z = __fdiv_rn(lg[i], temp);
    const unsigned long long key = ((unsigned long long)float_key(z) << 32) | (uint32_t)(~(uint32_t)i);
    if (key >= thr) {
      const int p = atomicAdd(&s_ncand, 1);
      if (p < CAND_MAX) { s_cz[p] = z; s_ci[p] = i; }
    }
  }
  __syncthreads();
  }  // fallback
  const int nc = min(s_ncand, CAND_MAX);
  // rank every candidate by (z desc, index asc); the k best land at their rank
  for (int a = tid; a < nc; a += FWD_THREADS) {
    const float za = s_cz[a];
    const int ia = s_ci[a];
    int rank = 0;
    for (int j = 0; j < nc; ++j) {
      const float zj = s_cz[j];
      rank += (zj > za) || (zj == za && s_ci[j] < ia);
    }
    if (rank < k) { s_tz[rank] = za; s_ti[rank] = ia; }
  }
  __syncthreads();
  if (tid == 0) {
    const uint32_t x = philox4x32_10_word0((uint32_t)ticket, (uint32_t)(ticket >> 32), (uint32_t)gen_index, 0u,
                                           (uint32_t)seed, (uint32_t)(seed >> 32));
    const int kk = min(k, nc);
    if (nucleus) {
      // nucleus inside the k candidates (already in the order), integer weights
      unsigned long long Q = 0;
      for (int j = 0; j < kk; ++j) Q += nucleus_weight(s_tz[j], s_tz[0]);
      const unsigned long long need = nucleus_need(nucleus_p24(top_p), Q);
      unsigned long long M = 0;
      int m = 0;
      for (; m < kk; ++m) {
        M += nucleus_weight(s_tz[m], s_tz[0]);
        if (M >= need) { ++m; break; }
      }
      const unsigned long long target = nucleus_target((unsigned long long)(x >> 8), M);
      unsigned long long cum = 0;
      int pick = s_ti[m - 1];
      for (int j = 0; j < m; ++j) {
        cum += nucleus_weight(s_tz[j], s_tz[0]);
        if (cum > target) { pick = s_ti[j]; break; }
      }
      result = pick;
    } else {
      const double u = (double)(x >> 8) * (1.0 / 16777216.0);
      double total = 0.0;
      for (int j = 0; j < kk; ++j) total += exp((double)s_tz[j] - (double)s_tz[0]);
      const double target = u * total;
      double accum = 0.0;
      int pick = s_ti[kk - 1];
      for (int j = 0; j < kk; ++j) {
        accum += exp((double)s_tz[j] - (double)s_tz[0]);
        if (accum > target) { pick = s_ti[j]; break; }
      }
      result = pick;
    }
  }
  __syncthreads();
  return result;
}

static __device__ __noinline__ void phase_sample(const DevCtx& c, float* smem) {
  const int R = c.ss->cur_rows;
  const int V = c.V;
  const int tid = threadIdx.x;
  const unsigned long long rows_before = c.ss->sample_rows_total;
  for (int r = blockIdx.x; r < R; r += gridDim.x) {
    const float* lg = c.logits + (size_t)r * V;
    const int item = c.row_item[r];
    const int b = c.it_bslot[item];
    if (c.logits_capture != nullptr && (long long)(rows_before + r) < c.capture_rows) {
      float* dst = c.logits_capture + (size_t)(rows_before + r) * V;
      for (int i = tid; i < V; i += FWD_THREADS) dst[i] = lg[i];
    }
    const int tok = sample_row(lg, V, min(c.b_topk[b], MAX_TOPK), c.b_temp[b], c.b_topp[b], (unsigned long long)c.b_ticket[b],
                               c.b_generated[b], c.b_seed[b], smem);
    if (tid == 0) c.row_sampled[r] = tok;
  }
}
constexpr int SAMPLE_SMEM_FLOATS = 256 + 4 * 1024;

}  // namespace blink
