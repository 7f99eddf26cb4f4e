// Device-visible state of the serving loop: plain structs shared by the host
// set-up code and the kernels of this library.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace blink {

// ---- slot life cycle (paper Section 4.2, "Ring buffer") ------------------------------
enum SlotState : uint32_t {
  SLOT_EMPTY = 0,
  SLOT_PREFILL_PENDING = 1,
  SLOT_PREFILL_PROCESSING = 2,
  SLOT_DECODE_PROCESSING = 3,
  SLOT_DECODE_COMPLETED = 4,
  SLOT_DECODE_PAUSED = 5,  // reserved for preemption; no policy uses it yet
};

// 16-byte hot header: n_slots * 16 B is the block the frontend would bulk-read
// (64 KB at 4096 slots, as in Section 4.4 "Token reader").
struct SlotHot {
  uint32_t state;
  uint32_t n_prompt;
  uint32_t generated;
  uint32_t arena_off;  // slot index: arenas are fixed-stride
};
struct SlotCold {
  uint64_t ticket;
  uint32_t max_new;
  uint32_t top_k;
  float temperature;
  int32_t eos_id;
  uint64_t seed;
  uint64_t user_tag;
  uint32_t flags;  // bit0: forced tokens present
  float top_p;     // outside (0, 1): no nucleus cut
};
enum { REQ_FLAG_FORCED = 1 };

// One entry of the pinned submit queue (host -> device), index = ticket % n_slots.
struct SubEntry {
  uint64_t ticket;
  uint64_t seed;
  uint64_t user_tag;
  uint32_t slot;
  uint32_t n_prompt;
  uint32_t max_new;
  uint32_t top_k;
  float temperature;
  int32_t eos_id;
  uint32_t flags;
  float top_p;
};

// Pinned control mailbox (host and device both read and write single words of it).
struct Mailbox {
  volatile uint64_t sub_tail;     // host: number of published submit entries
  volatile uint32_t stop;         // host: leave the GPU at the next iteration boundary
  volatile uint32_t start;        // host: admission may begin
  volatile uint32_t loop_state;   // device: BLINK_LOOP_*
  volatile int32_t device_status; // device: first error
  volatile uint64_t heartbeat;    // device: traced iterations so far
  volatile uint64_t clock_probe;  // device global timer sample (clock calibration)
};

enum DevError : int32_t {
  DEV_OK = 0,
  DEV_ERR_BARRIER_TIMEOUT = 1,
  DEV_ERR_TRACE_OVERFLOW = 2,  // informational: tracing stopped, loop continues
  DEV_ERR_STACK_UNDERFLOW = 3,
  DEV_ERR_BAD_INDEX = 4,
  DEV_ERR_PIPE_TIMEOUT = 5,    // a TMA / MMA mbarrier wait ran out
  DEV_ERR_TICKET_TABLE = 6,
};

enum StepCmd : int32_t { CMD_NONE = 0, CMD_RUN = 1, CMD_EXIT = 2 };
enum { PHASE_FREE = 0, PHASE_PREFILL = 1, PHASE_DECODE = 2 };

constexpr int N_PHASE_TIMERS = 16;

// Scalars of the scheduler that live in HBM and survive kernel re-instantiation.
struct SchedState {
  unsigned long long seen;          // submit entries moved into the ring
  unsigned long long next_admit;    // next ticket to admit (FCFS)
  unsigned long long iter;          // traced iterations
  unsigned long long tokens_out;
  unsigned long long prompt_tokens;
  unsigned long long sample_rows_total;
  long long trace_pos;              // words used
  long long cur_hdr;                // word offset of the open record, -1 if none
  long long cur_post;               // word offset where the post sections of the open record go
  int free_top;                     // entries in the free stack
  int reserved;                     // blocks promised to admitted requests
  int cur_T, cur_items, cur_rows, cur_decode;
  int cur_ndec;   // attention: requests with one query row in this step
  int cur_TT;     // attention: (row, kv head, KV block) tiles of those rows
  int cur_S;      // attention: tiles per sub-range of the flat tile sequence
  int cur_npf;    // attention: (request, query-row block) units of the multi-row requests
  long long cur_ctx;
  long long cur_kv;
  int cmd;
  int pending_post;                 // a forward ran and its post step is outstanding
  int trace_off;                    // tracing stopped (overflow)
  int abort_flag;
  unsigned long long bar_ctr;       // grid barrier: arrivals since the launch (the host zeroes it before a launch)
  unsigned long long cur_t_begin, cur_t_forward;
  int exit_reason;
  int last_was_prefill;             // pause-and-resume policy: the step before was a prefill step
  unsigned long long cur_phase_ns[N_PHASE_TIMERS];  // device time per phase kind of the open iteration
};

struct IterStat {
  uint64_t t_begin_ns, t_forward_ns, t_end_ns;
  int32_t n_tokens, n_decode, n_sample_rows, n_items;
  int64_t ctx_tokens;
  int64_t kv_tokens;
  uint64_t phase_ns[N_PHASE_TIMERS];
};

constexpr int TRACE_HDR_WORDS = 12;
constexpr int32_t TRACE_MAGIC = 0x424C4B31;
constexpr int CTRL_THREADS = 256;
constexpr int MAX_BATCH = 256;
constexpr int MAX_TOPK = 64;
constexpr int MAX_EXPERTS = 16;
constexpr int TILE_CNT_SLOTS = 8192;

struct DevCtx {
  // model
  int L, d, Hq, Hkv, hd, F, V, E, topE, dtype;
  int q_dim, kv_dim, qkv_dim, n_rep;
  float rope_theta, rms_eps, attn_scale;
  const char* w_base;
  unsigned long long w_off[10];
  // scheduler shape
  int MB, chunk, n_slots, max_prompt, max_new, Tmax, bs, n_blocks, max_blocks_seq, max_pos;
  int control_only, start_paused, stepped, gemm_tc;
  int policy;        // BLINK_POLICY_*: chunked prefill, or whole-prompt prefill steps that pause decoding
  int n_warps_grid;  // warps of the whole grid (attention work split)
  int w_streaming;   // GEMM matrices are stored as contiguous pre-swizzled 128 x 64 tiles
  long long iteration_budget;
  unsigned long long idle_exit_cycles, barrier_timeout_cycles;
  // ring in HBM
  SlotHot* slot_hot;
  SlotCold* slot_cold;
  int32_t* in_arena;      // [n_slots][max_prompt]
  int32_t* gen_arena;     // [n_slots][max_new]  tokens fed back (forced or sampled)
  int32_t* forced_arena;  // [n_slots][max_new]
  // pinned mailboxes (device-visible addresses)
  Mailbox* mbox;
  const SubEntry* sub_q;
  const int32_t* sub_tokens;  // [n_slots][max_prompt]
  const int32_t* sub_forced;  // [n_slots][max_new]
  int32_t* out_tokens;        // [n_slots][max_new]
  uint64_t* out_time;         // [n_slots][max_new]
  uint32_t* out_count;        // [n_slots] generated | 0x80000000 when finished | 0x40000000 when cancelled
  const uint32_t* cancel;     // [n_slots] host: non-zero = retire the request in this slot at the next step boundary
  // scheduler state in HBM
  SchedState* ss;
  uint32_t* ticket_to_slot;   // [n_slots]
  int32_t* free_stack;        // [n_blocks]
  int32_t* block_table;       // [MB][max_blocks_seq]
  // batch table, one entry per batch slot
  long long* b_ticket;
  int32_t *b_slot, *b_P, *b_N, *b_prefilled, *b_generated, *b_phase, *b_have, *b_need, *b_last, *b_eos,
      *b_topk, *b_flags;
  float *b_temp, *b_topp;
  unsigned long long* b_seed;
  // current step
  int32_t *it_bslot, *it_start, *it_ntok, *it_qstart, *it_row;  // [MB] per item
  int32_t *tok_id, *tok_pos, *tok_item, *tok_slotmap;           // [Tmax] per row
  int32_t *row_tok, *row_item, *row_sampled;                    // [MB] per sample row
  // attention work lists of the step (bf16 path)
  int32_t *dec_row, *dec_bslot, *dec_nctx, *dec_kbpre;          // [MB] (+1 for the prefix) single-row requests
  int32_t *pf_item, *pf_qb;                                     // [Tmax/16 + MB + 1] multi-row tile units
  int32_t* att_ctr;      // [L] sub-range counters, zeroed every iteration
  int32_t* att_cnt;      // [MB * Hkv] parts delivered per (row, kv head) unit; self-resetting
  float* att_part;       // partial (acc, m, l) records, two per sub-range
  long long att_sub_max; // sub-ranges the record buffer can hold
  // activations
  float* h;       // [Tmax][d]
  void* xn;       // [Tmax][d]      operand type
  float* qkv;     // [Tmax][qkv_dim]
  void* qb;       // [Tmax][q_dim]  bf16 path: q after RoPE, as the attention operand
  void* attn;     // [Tmax][q_dim]  operand type
  float* gu;      // [Tmax][2F]
  void* act;      // [Tmax][F]      operand type
  void* xs;       // [MB][d]        operand type
  // routed experts (E > 0): one row per (token, chosen expert); gu and act then have Tmax * topE rows
  void* xg;            // [Tmax*topE][d] operand type: normed rows gathered per expert
  int32_t* moe_sel;    // [Tmax][topE] chosen experts of a token, by descending router weight
  float* moe_wt;       // [Tmax][topE] their weights (sum to 1)
  int32_t* moe_off;    // [E+1] first gathered row of each expert
  int32_t* moe_tok;    // [Tmax*topE] token of a gathered row
  float* moe_gate;     // [Tmax*topE] its weight
  // fused epilogues of the tensor-core path
  float* rowss_a;      // [Tmax] sum of squares of the residual rows after the O GEMM (input of the second norm)
  float* rowss_b;      // [Tmax] the same after the down GEMM (input of the next layer's first norm / the final norm)
  int32_t* tile_cnt;   // [TILE_CNT_SLOTS] k-blocks delivered per output tile of the running GEMM; self-resetting
  int fused;           // 1: RoPE + KV write and SwiGLU run in the epilogues of the QKV and gate/up GEMMs
  int gu_direct;       // 1: gate/up tiles whose sums are complete in one accumulator are written as activations by the GEMM
  unsigned long long* gu_done;   // [token passes][gate/up weight tiles] stamp (iteration * L + layer + 1, 64 bits: never repeats) of the last such write
  int fused_norm;      // 1: the O and down epilogues add up sum(x^2) per row and the norms are element-wise
  float* logits;  // [MB][V]
  float *rope_cos, *rope_sin;  // [max_pos][hd/2]
  void* kv_base;               // [L][2][n_blocks][Hkv][bs][hd] operand type
  const void* tc_maps;         // TMA descriptors of the tensor-core path (device memory)
  const void* kv_map;          // TMA descriptor of the KV pool seen as [rows][head_dim], box 16 x 64 (device memory)
  // diagnostics
  int32_t* trace;
  long long trace_cap;
  IterStat* stats;
  long long stats_cap;
  float* logits_capture;
  long long capture_rows;
};

}  // namespace blink
