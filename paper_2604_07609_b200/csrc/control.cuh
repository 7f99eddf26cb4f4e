// Control plane of the serving loop, executed by CTA 0 (256 threads) once per
// iteration: retire the previous step (publish tokens, free blocks), move newly
// submitted requests into the HBM ring, scan + claim, FCFS admission, step
// composition, block allocation and metadata build.
//
// Paper: Section 4.2 "Persistent scheduler" (scan, claim, launch, poll, publish),
// "Parallel slot scanning" (256 threads over contiguous slot ranges, CAS claim),
// "Continuous batching with inline prefill" (FCFS), "Ring buffer" (state machine,
// fences order the externally visible updates).
#pragma once
#include "../../include/blink.h"
#include "dev_ctx.cuh"

namespace blink {

// ---- memory-ordering helpers ------------------------------------------------------
__device__ __forceinline__ uint64_t ld_acquire_sys_u64(const volatile uint64_t* p) {
  uint64_t v;
  asm volatile("ld.acquire.sys.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t ld_relaxed_sys_u32(const volatile uint32_t* p) {
  uint32_t v;
  asm volatile("ld.relaxed.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_sys_u32(volatile uint32_t* p, uint32_t v) {
  asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire_gpu_u32(const unsigned int* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_gpu_u32(unsigned int* p, uint32_t v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void dev_fail(const DevCtx& c, int code) {
  if (atomicCAS((int*)&c.mbox->device_status, 0, code) == 0) __threadfence_system();
  atomicExch(&c.ss->abort_flag, 1);
}

__device__ __forceinline__ unsigned long long ld_acquire_gpu_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}

// Grid-wide barrier with a bounded wait: every CTA adds one to a monotone counter (reset by the
// host before each launch) and waits until it reaches the next multiple of the grid size.
// Returns false when the loop must unwind (time-out here or abort raised elsewhere).  `target`
// is the caller's private running total (thread 0 of each CTA keeps it).
__device__ __forceinline__ void fence_proxy_async_global() {
  asm volatile("fence.proxy.async.global;" ::: "memory");
}

__device__ __forceinline__ bool grid_barrier(const DevCtx& c, unsigned long long& target) {
  __shared__ int s_ok;
  // Buffers written with ordinary stores in one phase (normed rows, K/V rows, attention output, ...)
  // are read by TMA / bulk copies (the async proxy) in a later phase: every thread orders its
  // stores against that proxy before it arrives, and again before it issues copies afterwards.
  fence_proxy_async_global();
  __syncthreads();
  if (threadIdx.x == 0) {
    int ok = 1;
    SchedState* ss = c.ss;
    target += gridDim.x;
    // release at gpu scope is cumulative: the stores of the CTA's other threads, ordered before this
    // point by the barrier above, are covered without a separate fence
    asm volatile("red.release.gpu.global.add.u64 [%0], 1;" ::"l"(&ss->bar_ctr) : "memory");
    long long t0 = 0;
    unsigned int polls = 0;
    while (ld_acquire_gpu_u64(&ss->bar_ctr) < target) {
      if ((++polls & 63u) == 0) {
        if (*(volatile int*)&ss->abort_flag) { ok = 0; break; }
        if (t0 == 0) t0 = clock64();
        if ((unsigned long long)(clock64() - t0) > c.barrier_timeout_cycles) {
          dev_fail(c, DEV_ERR_BARRIER_TIMEOUT);
          ok = 0;
          break;
        }
        if (polls > 4096u) __nanosleep(200);
      }
    }
    if (*(volatile int*)&ss->abort_flag) ok = 0;
    s_ok = ok;
  }
  __syncthreads();
  fence_proxy_async_global();
  return s_ok != 0;
}

// Exclusive prefix sum over the 256 threads of the control CTA; *total gets the sum.
__device__ __forceinline__ int block_exscan(int v, int* total) {
  __shared__ int s_warp[CTRL_THREADS / 32];
  __shared__ int s_total;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  int x = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  __syncthreads();  // protects s_warp / s_total from the previous call
  if (lane == 31) s_warp[w] = x;
  __syncthreads();
  if (w == 0) {
    int t = lane < CTRL_THREADS / 32 ? s_warp[lane] : 0;
    int z = t;
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) {
      int y = __shfl_up_sync(0xffffffffu, z, o);
      if (lane >= o) z += y;
    }
    if (lane < CTRL_THREADS / 32) s_warp[lane] = z - t;
    if (lane == CTRL_THREADS / 32 - 1) s_total = z;
  }
  __syncthreads();
  *total = s_total;
  return x - v + s_warp[w];
}

__device__ __forceinline__ int32_t fake_token(unsigned long long ticket, int gen, int vocab) {
  // control-only stand-in sampler: a fixed hash of (ticket, index)
  uint32_t x = (uint32_t)(ticket * 2654435761ull + (unsigned long long)gen * 40503ull + 12345ull);
  return (int32_t)(x % (uint32_t)vocab);
}

__device__ __forceinline__ bool trace_on(const DevCtx& c) { return c.trace_cap > 0 && !c.ss->trace_off; }

// ---- step 5 of the iteration: publish, retire, free -------------------------------------
static __device__ void post_step(const DevCtx& c) {
  SchedState* ss = c.ss;
  const int tid = threadIdx.x;
  const int n_items = ss->cur_items;
  const int n_rows = ss->cur_rows;
  const bool tr = trace_on(c) && ss->cur_hdr >= 0;
  int32_t* rec_post = c.trace + ss->cur_post;
  __shared__ unsigned long long s_ptok;
  __shared__ int s_need_sum;
  if (tid == 0) { s_ptok = 0; s_need_sum = 0; }
  __syncthreads();

  int fin = 0, nfree = 0, b = -1, row = -1;
  long long ticket = 0;
  if (tid < n_items) {
    b = c.it_bslot[tid];
    const int n = c.it_ntok[tid];
    row = c.it_row[tid];
    const int slot = c.b_slot[b];
    ticket = c.b_ticket[b];
    int phase = c.b_phase[b];
    if (phase == PHASE_PREFILL) {
      c.b_prefilled[b] += n;
      atomicAdd(&s_ptok, (unsigned long long)n);
    }
    if (row >= 0) {
      const int gen = c.b_generated[b];
      const int32_t sampled = c.control_only ? fake_token((unsigned long long)ticket, gen, c.V) : c.row_sampled[row];
      const int32_t fed = (c.b_flags[b] & REQ_FLAG_FORCED) ? c.forced_arena[(size_t)slot * c.max_new + gen] : sampled;
      c.gen_arena[(size_t)slot * c.max_new + gen] = fed;
      c.b_last[b] = fed;
      c.b_generated[b] = gen + 1;
      fin = (gen + 1 == c.b_N[b]) || (c.b_eos[b] >= 0 && fed == c.b_eos[b]);
      // externally visible: token and timestamp first, then the generation count
      c.out_tokens[(size_t)slot * c.max_new + gen] = sampled;
      c.out_time[(size_t)slot * c.max_new + gen] = global_timer_ns();
      c.slot_hot[slot].generated = gen + 1;
      if (phase == PHASE_PREFILL) c.b_phase[b] = PHASE_DECODE;
      c.slot_hot[slot].state = fin ? SLOT_DECODE_COMPLETED : SLOT_DECODE_PROCESSING;
      __threadfence_system();
      c.out_count[slot] = (uint32_t)(gen + 1) | (fin ? 0x80000000u : 0u);
      if (tr) { rec_post[2 * row] = b; rec_post[2 * row + 1] = sampled; }
      if (fin) {
        nfree = c.b_have[b];
        atomicAdd(&s_need_sum, c.b_need[b]);
      }
    }
  }
  int tot_fin, tot_free;
  const int fin_idx = block_exscan(fin, &tot_fin);
  const int free_off = block_exscan(nfree, &tot_free);
  const int top = ss->free_top;
  if (fin) {
    if (tr) rec_post[2 * n_rows + fin_idx] = (int32_t)ticket;
    for (int j = 0; j < nfree; ++j) {
      const int blk = c.block_table[(size_t)b * c.max_blocks_seq + j];
      c.free_stack[top + free_off + j] = blk;
      if (tr) rec_post[2 * n_rows + tot_fin + free_off + j] = blk;
    }
    c.b_have[b] = 0;
    c.b_phase[b] = PHASE_FREE;
  }
  __syncthreads();
  // Cancellation (an early exit the host asks for): every request that is still live after the step's
  // own completions and whose slot carries the host's cancel mark is retired here, in ascending batch
  // slot, exactly as at a normal end: blocks pushed back in logical order, reservation released.
  int cfin = 0, cfree = 0, cslot = 0;
  long long cticket = 0;
  if (c.cancel != nullptr && tid < c.MB && c.b_phase[tid] != PHASE_FREE) {
    cslot = c.b_slot[tid];
    if (ld_relaxed_sys_u32(&c.cancel[cslot]) != 0u) {
      cfin = 1;
      cfree = c.b_have[tid];
      cticket = c.b_ticket[tid];
      atomicAdd(&s_need_sum, c.b_need[tid]);
    }
  }
  int tot_cfin, tot_cfree;
  const int cfin_idx = block_exscan(cfin, &tot_cfin);
  const int cfree_off = block_exscan(cfree, &tot_cfree);
  if (cfin) {
    if (tr) rec_post[2 * n_rows + tot_fin + tot_free + cfin_idx] = (int32_t)cticket;
    for (int j = 0; j < cfree; ++j) {
      const int blk = c.block_table[(size_t)tid * c.max_blocks_seq + j];
      c.free_stack[top + tot_free + cfree_off + j] = blk;
      if (tr) rec_post[2 * n_rows + tot_fin + tot_free + tot_cfin + cfree_off + j] = blk;
    }
    c.b_have[tid] = 0;
    c.b_phase[tid] = PHASE_FREE;
    c.slot_hot[cslot].state = SLOT_DECODE_COMPLETED;
    __threadfence_system();
    c.out_count[cslot] = (uint32_t)c.b_generated[tid] | 0xC0000000u;   // finished + cancelled
  }
  __syncthreads();
  if (tid == 0) {
    ss->free_top = top + tot_free + tot_cfree;
    ss->reserved -= s_need_sum;
    ss->tokens_out += (unsigned long long)n_rows;
    ss->prompt_tokens += s_ptok;
    ss->sample_rows_total += (unsigned long long)n_rows;
    const uint64_t t_end = global_timer_ns();
    if (tr) {
      // The record lists finished tickets then freed blocks; with cancellations the order is: tickets
      // that ended by themselves, their blocks, cancelled tickets, their blocks -- rewritten below into
      // the record's two lists (tickets first, then blocks) when both kinds occur.
      int32_t* hdr = c.trace + ss->cur_hdr;
      if (tot_cfin > 0 && tot_free > 0) {
        // move the cancelled tickets in front of the first group's blocks (few words, one thread)
        int32_t* base = rec_post + 2 * n_rows + tot_fin;
        for (int k = 0; k < tot_cfin; ++k) {
          const int32_t tk = base[tot_free + k];
          for (int j = tot_free + k; j > k; --j) base[j] = base[j - 1];
          base[k] = tk;
        }
      }
      hdr[6] = n_rows;
      hdr[7] = tot_fin + tot_cfin;
      hdr[8] = tot_free + tot_cfree;
      hdr[9] = ss->free_top;
      hdr[10] = ss->reserved;
      const long long end = ss->cur_post + 2 * n_rows + tot_fin + tot_cfin + tot_free + tot_cfree;
      hdr[11] = (int32_t)(end - ss->cur_hdr);
      ss->trace_pos = end;
    }
    if (c.stats_cap > 0 && (long long)ss->iter < c.stats_cap) {
      IterStat& st = c.stats[ss->iter];
      st.t_begin_ns = ss->cur_t_begin;
      st.t_forward_ns = ss->cur_t_forward;
      st.t_end_ns = t_end;
      st.n_tokens = ss->cur_T;
      st.n_decode = ss->cur_decode;
      st.n_sample_rows = n_rows;
      st.n_items = n_items;
      st.ctx_tokens = ss->cur_ctx;
      st.kv_tokens = ss->cur_kv;
      for (int i = 0; i < N_PHASE_TIMERS; ++i) st.phase_ns[i] = ss->cur_phase_ns[i];
    }
    for (int i = 0; i < N_PHASE_TIMERS; ++i) ss->cur_phase_ns[i] = 0;
    ss->iter += 1;
    ss->cur_hdr = -1;
    ss->pending_post = 0;
    c.mbox->heartbeat = ss->iter;
  }
  __syncthreads();
}

// ---- stand-in for the frontend's RDMA write: pinned submit area -> HBM ring --------------
static __device__ void ingress(const DevCtx& c, unsigned long long tail) {
  SchedState* ss = c.ss;
  const int tid = threadIdx.x;
  for (unsigned long long e = ss->seen; e < tail; ++e) {
    const SubEntry* en = &c.sub_q[e % (unsigned long long)c.n_slots];
    const uint32_t slot = en->slot;
    const uint32_t np = en->n_prompt;
    const uint32_t flags = en->flags;
    if (slot >= (uint32_t)c.n_slots || np > (uint32_t)c.max_prompt || en->ticket != e) {
      if (tid == 0) dev_fail(c, DEV_ERR_BAD_INDEX);
      break;
    }
    const int32_t* src = c.sub_tokens + (size_t)slot * c.max_prompt;
    int32_t* dst = c.in_arena + (size_t)slot * c.max_prompt;
    for (uint32_t i = tid; i < np; i += CTRL_THREADS) dst[i] = src[i];
    if (flags & REQ_FLAG_FORCED) {
      const int32_t* fs = c.sub_forced + (size_t)slot * c.max_new;
      int32_t* fd = c.forced_arena + (size_t)slot * c.max_new;
      for (uint32_t i = tid; i < en->max_new; i += CTRL_THREADS) fd[i] = fs[i];
    }
    if (tid == 0) {
      SlotCold& cold = c.slot_cold[slot];
      cold.ticket = en->ticket;
      cold.max_new = en->max_new;
      cold.top_k = en->top_k;
      cold.temperature = en->temperature;
      cold.eos_id = en->eos_id;
      cold.seed = en->seed;
      cold.user_tag = en->user_tag;
      cold.flags = flags;
      cold.top_p = en->top_p;
      SlotHot& hot = c.slot_hot[slot];
      hot.n_prompt = np;
      hot.generated = 0;
      hot.arena_off = slot;
    }
    __syncthreads();  // payload before the state flip
    if (tid == 0) {
      __threadfence();
      c.slot_hot[slot].state = SLOT_PREFILL_PENDING;
    }
  }
  __syncthreads();
  if (tid == 0) ss->seen = tail;
  __syncthreads();
}

// ---- parallel slot scan + CAS claim (Section 4.2 "Parallel slot scanning") ----------------
static __device__ void scan_and_claim(const DevCtx& c) {
  const int per = (c.n_slots + CTRL_THREADS - 1) / CTRL_THREADS;
  const int lo = threadIdx.x * per;
  const int hi = min(c.n_slots, lo + per);
  for (int s = lo; s < hi; ++s) {
    if (c.slot_hot[s].state == SLOT_PREFILL_PENDING) {
      if (atomicCAS(&c.slot_hot[s].state, (uint32_t)SLOT_PREFILL_PENDING, (uint32_t)SLOT_PREFILL_PROCESSING) ==
          SLOT_PREFILL_PENDING) {
        const unsigned long long t = c.slot_cold[s].ticket;
        c.ticket_to_slot[t % (unsigned long long)c.n_slots] = (uint32_t)s;
      }
    }
  }
  __syncthreads();
}

// ---- steps 1-3: admit, compose, allocate, build metadata ----------------------------------
// Returns the number of rows T of the composed step (0 = nothing to run).
static __device__ int schedule_step(const DevCtx& c, unsigned long long visible) {
  SchedState* ss = c.ss;
  const int tid = threadIdx.x;
  const int MB = c.MB;
  __shared__ int s_phase[MAX_BATCH];
  __shared__ long long s_ticket[MAX_BATCH];
  __shared__ int s_rem[MAX_BATCH];
  __shared__ int s_qstart[MAX_BATCH + 1];
  __shared__ int s_item_b[MAX_BATCH];
  __shared__ int s_n_admit;
  __shared__ int s_trace_ok;
  __shared__ unsigned long long s_ctx, s_kv;
  __shared__ int s_ndec;

  const uint64_t t_begin = global_timer_ns();
  s_phase[tid] = tid < MB ? c.b_phase[tid] : -1;
  if (tid == 0) { s_n_admit = 0; s_ctx = 0; s_kv = 0; s_ndec = 0; }
  __syncthreads();

  // open a trace record (header is completed later)
  long long hdr = -1;
  if (trace_on(c)) hdr = ss->trace_pos;
  int32_t* rec = c.trace + (hdr >= 0 ? hdr : 0);

  // 1. FCFS admission (serial: one decision depends on the previous one)
  if (tid == 0) {
    int n_admit = 0;
    int reserved = ss->reserved;
    int cursor = 0;
    unsigned long long na = ss->next_admit;
    // worst-case space check for the admitted section is done with the rest below
    while (na < visible) {
      const uint32_t slot = c.ticket_to_slot[na % (unsigned long long)c.n_slots];
      if (slot >= (uint32_t)c.n_slots || c.slot_cold[slot].ticket != na ||
          c.slot_hot[slot].state != SLOT_PREFILL_PROCESSING) {
        dev_fail(c, DEV_ERR_TICKET_TABLE);
        break;
      }
      const int P = (int)c.slot_hot[slot].n_prompt;
      const SlotCold cold = c.slot_cold[slot];
      const int N = (int)cold.max_new;
      const int need = (P + N - 1 + c.bs - 1) / c.bs;
      while (cursor < MB && s_phase[cursor] != PHASE_FREE) ++cursor;
      if (cursor >= MB || reserved + need > c.n_blocks) break;  // head of line blocks
      const int b = cursor;
      s_phase[b] = PHASE_PREFILL;
      c.b_phase[b] = PHASE_PREFILL;
      c.b_ticket[b] = (long long)na;
      c.b_slot[b] = (int)slot;
      c.b_P[b] = P;
      c.b_N[b] = N;
      c.b_prefilled[b] = 0;
      c.b_generated[b] = 0;
      c.b_have[b] = 0;
      c.b_need[b] = need;
      c.b_last[b] = 0;
      c.b_eos[b] = cold.eos_id;
      c.b_topk[b] = (int)cold.top_k;
      c.b_temp[b] = cold.temperature;
      c.b_topp[b] = cold.top_p;
      c.b_seed[b] = cold.seed;
      c.b_flags[b] = (int)cold.flags;
      reserved += need;
      if (hdr >= 0 && hdr + TRACE_HDR_WORDS + 2 * (n_admit + 1) <= c.trace_cap) {
        rec[TRACE_HDR_WORDS + 2 * n_admit] = (int32_t)na;
        rec[TRACE_HDR_WORDS + 2 * n_admit + 1] = b;
      }
      ++n_admit;
      ++na;
    }
    ss->next_admit = na;
    ss->reserved = reserved;
    s_n_admit = n_admit;
    __threadfence();
  }
  __syncthreads();
  const int n_admit = s_n_admit;

  // 2. compose
  int phase = PHASE_FREE, P = 0, prefilled = 0, gen = 0, have = 0, slot = 0;
  long long ticket = 0;
  if (tid < MB) {
    phase = s_phase[tid];
    if (phase != PHASE_FREE) {
      P = c.b_P[tid];
      prefilled = c.b_prefilled[tid];
      gen = c.b_generated[tid];
      have = c.b_have[tid];
      slot = c.b_slot[tid];
      ticket = c.b_ticket[tid];
    }
  }
  s_ticket[tid] = ticket;
  s_rem[tid] = (phase == PHASE_PREFILL) ? (P - prefilled) : 0;
  __syncthreads();
  int take = 0, start = 0;
  // prompt tokens already promised to earlier tickets in this iteration
  long long before = 0;
  if (phase == PHASE_PREFILL)
    for (int j = 0; j < MB; ++j)
      if (s_rem[j] > 0 && s_ticket[j] < ticket) before += s_rem[j];
  bool prefill_turn = false;
  if (c.policy == BLINK_POLICY_PAUSE_RESUME) {
    // Section 4.2 "Continuous batching with inline prefill": a step is a decode step, or a prefill step
    // for the whole prompts of the newly admitted requests while decoding is paused for this one step
    const int has_pf = __syncthreads_or(phase == PHASE_PREFILL);
    const int has_dec = __syncthreads_or(phase == PHASE_DECODE);
    prefill_turn = has_pf && (!ss->last_was_prefill || !has_dec);
    if (prefill_turn) {
      if (phase == PHASE_PREFILL && before + P <= (long long)c.chunk) take = P;   // whole prompts, nobody overtakes
      if (phase == PHASE_DECODE) c.slot_hot[slot].state = SLOT_DECODE_PAUSED;
    } else if (phase == PHASE_DECODE) {
      take = 1;
      start = P + gen - 1;
      c.slot_hot[slot].state = SLOT_DECODE_PROCESSING;
    }
  } else if (phase == PHASE_DECODE) {
    take = 1;
    start = P + gen - 1;
  } else if (phase == PHASE_PREFILL) {
    const long long left = (long long)c.chunk - before;
    take = (int)max(0ll, min((long long)(P - prefilled), left));
    start = prefilled;
  }
  const int f = take > 0;
  const int new_len = start + take;
  const int want = f ? (new_len + c.bs - 1) / c.bs - have : 0;
  const int sample = f && (phase == PHASE_DECODE || new_len == P);
  int n_items, T, n_alloc, n_rows;
  const int item = block_exscan(f, &n_items);
  const int qstart = block_exscan(take, &T);
  const int aoff = block_exscan(want, &n_alloc);
  const int row = block_exscan(sample, &n_rows);
  // blocks that post_step may free at most, and tickets that may end (completions and cancellations),
  // for the trace space check
  int tot_may_free, n_live;
  block_exscan(phase != PHASE_FREE ? have + want : 0, &tot_may_free);
  block_exscan(phase != PHASE_FREE ? 1 : 0, &n_live);
  // attention work lists: single-row requests stream their KV blocks, multi-row requests are
  // cut into blocks of 128 / n_rep query rows
  const int q_rows = 128 / c.n_rep;
  const int is_dec = f && take == 1;
  const int nkb_att = is_dec ? (new_len + c.bs - 1) / c.bs : 0;
  const int n_qb = (f && take > 1) ? (take + q_rows - 1) / q_rows : 0;
  int n_dec_att, tot_kb, n_pf;
  const int dec_idx = block_exscan(is_dec, &n_dec_att);
  const int kb_pre = block_exscan(nkb_att, &tot_kb);
  const int pf_off = block_exscan(n_qb, &n_pf);

  if (T == 0) return 0;  // uniform: every thread sees the same T

  if (tid == 0) {
    int ok = 1;
    if (hdr >= 0) {
      const long long worst = hdr + TRACE_HDR_WORDS + 2ll * n_admit + 5ll * n_items + 3ll * n_alloc + 2ll * n_rows +
                              n_live + tot_may_free;
      if (worst > c.trace_cap) {
        ok = 0;
        ss->trace_off = 1;
        atomicCAS((int*)&c.mbox->device_status, 0, DEV_ERR_TRACE_OVERFLOW);
      }
    }
    s_trace_ok = ok;
    if (ss->free_top < n_alloc) dev_fail(c, DEV_ERR_STACK_UNDERFLOW);
  }
  __syncthreads();
  if (ss->free_top < n_alloc) return 0;
  const bool tr = hdr >= 0 && s_trace_ok;
  int32_t* rec_sched = rec + TRACE_HDR_WORDS + 2 * n_admit;
  int32_t* rec_alloc = rec_sched + 5 * n_items;

  // 3. allocate: ascending batch slot, the stack pops from its top
  const int top = ss->free_top;
  if (f) {
    for (int j = 0; j < want; ++j) {
      const int blk = c.free_stack[top - 1 - (aoff + j)];
      c.block_table[(size_t)tid * c.max_blocks_seq + have + j] = blk;
      if (tr) {
        rec_alloc[3 * (aoff + j)] = tid;
        rec_alloc[3 * (aoff + j) + 1] = have + j;
        rec_alloc[3 * (aoff + j) + 2] = blk;
      }
    }
    c.b_have[tid] = have + want;
    c.it_bslot[item] = tid;
    c.it_start[item] = start;
    c.it_ntok[item] = take;
    c.it_qstart[item] = qstart;
    c.it_row[item] = sample ? row : -1;
    s_qstart[item] = qstart;
    s_item_b[item] = tid;
    if (sample) {
      c.row_tok[row] = qstart + take - 1;
      c.row_item[row] = item;
    }
    if (c.dec_row != nullptr) {
      if (is_dec) {
        c.dec_row[dec_idx] = qstart;
        c.dec_bslot[dec_idx] = tid;
        c.dec_nctx[dec_idx] = new_len;
        c.dec_kbpre[dec_idx] = kb_pre;
      }
      for (int q = 0; q < n_qb; ++q) {   // heaviest (last) row block first
        c.pf_item[pf_off + q] = item;
        c.pf_qb[pf_off + q] = n_qb - 1 - q;
      }
    }
    if (tr) {
      rec_sched[5 * item] = tid;
      rec_sched[5 * item + 1] = (int32_t)ticket;
      rec_sched[5 * item + 2] = phase;
      rec_sched[5 * item + 3] = start;
      rec_sched[5 * item + 4] = take;
    }
    unsigned long long ctx = (phase == PHASE_DECODE) ? (unsigned long long)(start + 1)
                                                     : (unsigned long long)take * start +
                                                           (unsigned long long)take * (take + 1) / 2;
    atomicAdd(&s_ctx, ctx);
    atomicAdd(&s_kv, (unsigned long long)new_len);
    if (phase == PHASE_DECODE) atomicAdd(&s_ndec, 1);
  }
  if (tid == 0) s_qstart[n_items] = T;
  __threadfence();
  __syncthreads();

  // per-row metadata: token id, position, owning item, KV slot
  // every warp of the grid starts on the sub-range of its own index; the counter hands out the rest
  if (c.att_ctr != nullptr)
    for (int i = tid; i < c.L; i += CTRL_THREADS) c.att_ctr[i] = c.n_warps_grid;
  for (int r = tid; r < T; r += CTRL_THREADS) {
    int lo = 0, hi = n_items;  // last item with qstart <= r
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (s_qstart[mid] <= r) lo = mid; else hi = mid;
    }
    const int b = s_item_b[lo];
    const int st = c.it_start[lo];
    const int pos = st + (r - s_qstart[lo]);
    int32_t tok;
    if (c.b_phase[b] == PHASE_DECODE) tok = c.b_last[b];
    else tok = c.in_arena[(size_t)c.b_slot[b] * c.max_prompt + pos];
    c.tok_id[r] = tok;
    c.tok_pos[r] = pos;
    c.tok_item[r] = lo;
    c.tok_slotmap[r] = c.block_table[(size_t)b * c.max_blocks_seq + pos / c.bs] * c.bs + pos % c.bs;
  }
  __syncthreads();
  if (tid == 0) {
    ss->free_top = top - n_alloc;
    ss->cur_T = T;
    ss->cur_items = n_items;
    ss->cur_rows = n_rows;
    ss->cur_decode = s_ndec;
    ss->cur_ctx = (long long)s_ctx;
    ss->cur_kv = (long long)s_kv;
    ss->cur_t_begin = t_begin;
    ss->pending_post = 1;
    ss->last_was_prefill = prefill_turn ? 1 : 0;
    if (c.dec_row != nullptr) {
      const long long TT = (long long)tot_kb * c.Hkv;
      // Sub-ranges: k per warp of the grid.  Every cut of a unit costs a partial record and a merge,
      // so a pure decode step takes one sub-range per warp up to 96 tiles; with prefill tiles in the
      // step the CTAs reach their decode share at different times and smaller sub-ranges (up to 48
      // tiles, the later ones handed out by the counter) even that out.
      const long long NW = c.n_warps_grid;
      const long long cap = n_pf > 0 ? 48 : 96;
      const long long k = (TT + cap * NW - 1) / (cap * NW) > 1 ? (TT + cap * NW - 1) / (cap * NW) : 1;
      long long S = (TT + k * NW - 1) / (k * NW);
      // at least 8 tiles per sub-range: a cut costs a partial record, a fence and a counter update (about the time of
      // two tiles), and a unit cut into n parts is merged by one warp in n steps; with few long rows one tile per
      // sub-range made a single 2048-token row take 120 us per layer, most of it the merge
      if (S < 8) S = 8;
      while ((TT + S - 1) / S > c.att_sub_max) S *= 2;   // cannot happen with the sizes set at create
      c.dec_kbpre[n_dec_att] = tot_kb;
      ss->cur_ndec = n_dec_att;
      ss->cur_TT = (int)TT;
      ss->cur_S = (int)S;
      ss->cur_npf = n_pf;
    }
    if (tr) {
      rec[0] = TRACE_MAGIC;
      rec[1] = (int32_t)ss->iter;
      rec[2] = (int32_t)((long long)visible - 1);
      rec[3] = n_admit;
      rec[4] = n_items;
      rec[5] = n_alloc;
      ss->cur_hdr = hdr;
      ss->cur_post = hdr + TRACE_HDR_WORDS + 2ll * n_admit + 5ll * n_items + 3ll * n_alloc;
    } else {
      ss->cur_hdr = -1;
    }
    ss->cur_t_forward = global_timer_ns();
    __threadfence();
  }
  __syncthreads();
  return T;
}

// One pass of the control plane.  `launch_iters` counts the iterations this kernel
// launch has started.  Sets ss->cmd to CMD_RUN (a step was composed), CMD_EXIT
// (leave the GPU; reason in ss->exit_reason) or CMD_NONE (stepped mode, idle).
// (a function of its own: inlined, its code shares the register allocation of the dispatcher of the loop kernel,
// which then spills more on the path of every phase: 1-1.5 % of a decode step)
static __device__ __noinline__ void control_phase(const DevCtx& c, long long& launch_iters) {
  SchedState* ss = c.ss;
  const int tid = threadIdx.x;
  __shared__ int s_cmd;
  __shared__ int s_started;
  __shared__ int s_abort;
  __shared__ unsigned long long s_tail;
  if (ss->pending_post) post_step(c);
  long long idle_t0 = clock64();
  unsigned int spins = 0;
  while (true) {
    if (tid == 0) {
      int cmd = CMD_NONE;
      if (ld_relaxed_sys_u32(&c.mbox->stop)) { cmd = CMD_EXIT; ss->exit_reason = 2; }
      else if (*(volatile int*)&ss->abort_flag) { cmd = CMD_EXIT; ss->exit_reason = 5; }
      else if (c.iteration_budget > 0 && launch_iters >= c.iteration_budget) { cmd = CMD_EXIT; ss->exit_reason = 3; }
      unsigned long long tail = ss->seen;
      const int started = !c.start_paused || ld_relaxed_sys_u32(&c.mbox->start);
      if (cmd == CMD_NONE && started) tail = ld_acquire_sys_u64(&c.mbox->sub_tail);
      s_cmd = cmd;
      s_tail = tail;
      s_started = started;
    }
    __syncthreads();
    if (s_cmd == CMD_EXIT) break;
    const unsigned long long tail = s_tail;
    const bool started = s_started != 0;
    int T = 0;
    if (started) {
      if (tail > ss->seen) ingress(c, tail);
      scan_and_claim(c);
      T = schedule_step(c, ss->seen);
    }
    __syncthreads();
    if (T > 0) {
      if (tid == 0) s_cmd = CMD_RUN;
      launch_iters += 1;
      __syncthreads();
      break;
    }
    // one thread reads the flag (another CTA may raise it at any time) so that the whole CTA
    // takes the same branch
    if (tid == 0) s_abort = *(volatile int*)&ss->abort_flag;
    __syncthreads();
    if (s_abort) {
      if (tid == 0) { s_cmd = CMD_EXIT; ss->exit_reason = 5; }
      __syncthreads();
      break;
    }
    if (c.stepped) break;  // CMD_NONE
    // idle: poll the submit mailbox, leave the GPU when nothing comes
    if ((unsigned long long)(clock64() - idle_t0) > c.idle_exit_cycles) {
      if (tid == 0) { s_cmd = CMD_EXIT; ss->exit_reason = 4; }
      __syncthreads();
      break;
    }
    if (++spins > 16) __nanosleep(1000);
    __syncthreads();
  }
  if (tid == 0) {
    ss->cmd = s_cmd;
    __threadfence();
  }
  __syncthreads();
}

}  // namespace blink
