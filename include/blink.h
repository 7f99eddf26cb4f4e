/*
 * blink.h - C ABI of the GPU-resident LLM serving loop.
 *
 * The library runs the per-iteration serving loop (request pickup, FCFS
 * continuous batching, paged-KV block bookkeeping, the transformer step,
 * in-step sampling, token publication) inside one bounded-lifetime persistent
 * CUDA kernel for sm_100a.  The host appears only at set-up and as the stand-in
 * for the paper's SmartNIC frontend: it writes prompts into, and reads tokens
 * from, mapped pinned mailboxes that the kernel polls.
 *
 * Paper passages each call follows ("Blink: CPU-Free LLM Inference by Delegating
 * the Serving Stack to GPU and SmartNIC"):
 *   blink_create  - Section 4.1: the host is a provisioning plane that sets
 *                   everything up once and then leaves the inference path;
 *                   Section 4.2 "Persistent scheduler".
 *   blink_submit  - Fig. 2 steps 3-5 and Section 4.4 "RDMA datapath" / "Slot
 *                   tracker": find a free ring slot, write the tokenised prompt,
 *                   then flip the slot state so the backend can start prefill.
 *   blink_poll    - Fig. 2 step 11 and Section 4.4 "Token reader": compare each
 *                   active slot's generation count with the consumer's own and
 *                   hand out the new tokens.
 *   blink_destroy - Section 4.2 "window-based tail-launch recovery": all loop
 *                   state lives in device memory, so the kernel may leave (and be
 *                   re-instantiated) at any iteration boundary.
 *
 * Conventions: every function returns BLINK_OK (0) or a negative BLINK_E* code;
 * nothing throws, aborts or traps.  Pointers are HOST pointers unless the comment
 * says DEVICE.  Structs are plain C and start with their own size in bytes.
 * The library never frees caller-owned buffers.  No call falls back to the CPU:
 * without a CUDA device blink_create fails with BLINK_ECUDA.
 */
#ifndef BLINK_H_
#define BLINK_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  BLINK_OK = 0,
  BLINK_EAGAIN = -1,    /* no empty ring slot: back-pressure, retry later      */
  BLINK_EINVAL = -2,    /* bad argument                                         */
  BLINK_ESTOPPED = -3,  /* loop was stopped by blink_stop/blink_destroy         */
  BLINK_EDEVICE = -4,   /* the device loop reported an error (see blink_stats)  */
  BLINK_ETIMEDOUT = -5, /* a bounded wait ran out                               */
  BLINK_ENOMEM = -6,    /* allocation failed / pool too small                   */
  BLINK_ECUDA = -7,     /* a CUDA runtime or driver call failed                 */
  BLINK_ETOOBIG = -8    /* size beyond a fixed capacity (see blink_sample_noalloc) */
};

enum { BLINK_DTYPE_BF16 = 0, BLINK_DTYPE_FP32 = 1 };

/* Storage of the GEMM matrices (tensor ids 1, 2, 3, 4, 9) inside the flat weight buffer.  Tensor
 * offsets and sizes are the same in both layouts; embedding, router and norm tensors are always
 * row-major.
 *   ROW_MAJOR : [out][in], the documented exchange layout.
 *   STREAMING : bf16 only.  Each matrix is cut into panels of 128 output rows; a panel keeps its
 *     byte range but is stored as K/64 consecutive tiles of 128 rows x 64 columns (16 KiB), tile
 *     kb holding columns [64 kb, 64 kb + 64).  Inside a tile row r is at byte r * 128 and its
 *     16-byte chunk c (columns 8 c .. 8 c + 7) sits at chunk position c ^ (r % 8): the operand
 *     image the tensor cores read from shared memory, so a weight tile reaches the SM as one
 *     contiguous 16 KiB copy and every SM streams long sequential runs of HBM.  Requires every
 *     matrix to have a multiple of 128 rows per layer and a multiple of 64 columns.  The rows of
 *     each gate/up matrix (tensor 3) are first interleaved: stored row 2 f is gate row f and
 *     stored row 2 f + 1 is up row f, so one tile holds both halves of 64 features and the GEMM
 *     that owns all of a tile's K writes silu(gate) * up itself.
 * blink_convert_weights switches a buffer between the two, in place. */
enum { BLINK_WEIGHTS_ROW_MAJOR = 0, BLINK_WEIGHTS_STREAMING = 1 };

/* how the iteration is executed */
enum {
  BLINK_EXEC_PERSISTENT = 0, /* one cooperative kernel loops on the device (product mode)           */
  BLINK_EXEC_STEPPED = 1,    /* same device code, one host launch per phase (profiling, debugging)  */
  BLINK_EXEC_MANUAL = 2,     /* the cooperative loop kernel, launched only by blink_run (measurement) */
  /* Host-driven comparison arms (Section 6.1 baselines keep the host in the loop; Section 6.3 "Interference"):
   * the same device code as STEPPED, but a thread of the library launches one iteration at a time and waits
   * for it before it launches the next, as a host-resident serving loop does.  HOST_GRAPH launches the
   * iteration as one pre-captured CUDA graph, HOST_LAUNCHES as one kernel launch per phase.  blink_submit,
   * blink_poll and blink_cancel work as in PERSISTENT; blink_step and blink_run are refused. */
  BLINK_EXEC_HOST_GRAPH = 3,
  BLINK_EXEC_HOST_LAUNCHES = 4
};

/* which kernels run the dense contractions */
enum {
  BLINK_GEMM_AUTO = 0, /* tensor cores for bf16, CUDA cores for fp32 */
  BLINK_GEMM_SIMT = 1, /* CUDA-core reference kernels                */
  BLINK_GEMM_TC = 2,   /* tcgen05 / TMEM / TMA kernels (bf16 only)   */
  BLINK_GEMM_TC_PAIR = 3 /* the same on CTA pairs (tcgen05 cta_group::2, kernels launched with clusters of two): each
                          CTA stages its own weight tile and half of the token tile.  bf16, four query heads per
                          kv head, separate element-wise phases; BLINK_EINVAL otherwise */
};

/* where RoPE + KV write, SwiGLU and the norms' sums of squares run (tensor-core path only) */
enum {
  BLINK_FUSION_AUTO = 0, /* the faster of the two for the model shape (currently: separate phases)        */
  BLINK_FUSION_OFF = 1,  /* phases of their own between grid barriers                                     */
  BLINK_FUSION_ON = 2    /* in the GEMM epilogues: the CTA that completes an output tile consumes it      */
};

/* how prompts enter a running batch */
enum {
  BLINK_POLICY_CHUNKED = 0,      /* chunked prefill: every step carries all decode rows plus up to
                                    prefill_chunk_tokens prompt tokens, in ticket order              */
  BLINK_POLICY_PAUSE_RESUME = 1  /* the paper's inline prefill (Section 4.2 "Continuous batching with inline
                                    prefill"): a step is either a decode step or a prefill step that runs the
                                    whole prompts of the newly admitted requests (in ticket order, as many as
                                    fit into prefill_chunk_tokens, which must be >= max_prompt) while the
                                    decode requests are paused (slot state DECODE_PAUSED) for that one step */
};

/* why the device loop is not running (blink_stats.loop_state) */
enum {
  BLINK_LOOP_NOT_STARTED = 0,
  BLINK_LOOP_RUNNING = 1,
  BLINK_LOOP_EXIT_STOP = 2,   /* host asked                              */
  BLINK_LOOP_EXIT_BUDGET = 3, /* iteration budget of this launch used up */
  BLINK_LOOP_EXIT_IDLE = 4,   /* nothing to do for idle_exit_us          */
  BLINK_LOOP_EXIT_ERROR = 5   /* device_status != 0                      */
};

typedef struct blink_ctx blink_ctx;

/* Decoder-only transformer shape (pre-norm, RMSNorm, rotate-half RoPE, grouped-query
 * attention, SwiGLU FFN or top-k routed experts) and its weights. */
typedef struct blink_model_cfg {
  uint32_t size;
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ff, vocab;
  int32_t n_experts;     /* 0 = dense FFN, else up to 16 routed experts */
  int32_t top_k_experts; /* experts per token when n_experts > 0 */
  float rope_theta;
  float rms_eps;
  int32_t dtype;         /* BLINK_DTYPE_*: storage type of matrices, KV pool and GEMM operands */
  int32_t weights_layout;/* BLINK_WEIGHTS_*: how the five GEMM matrices are stored inside `weights` */
  const void* weights;   /* DEVICE, caller-owned, layout: see blink_weight_offset; may be NULL when control_only */
  uint64_t weights_bytes;
} blink_model_cfg;

typedef struct blink_sched_cfg {
  uint32_t size;
  int32_t max_batch;            /* 1..256 requests in the running batch                         */
  int32_t prefill_chunk_tokens; /* prompt tokens scheduled per iteration, over all requests     */
  int32_t n_slots;              /* ring slots (the paper uses 4096)                             */
  int32_t max_prompt;           /* longest accepted prompt                                      */
  int32_t max_new;              /* largest accepted max_new_tokens                              */
  int32_t exec_mode;            /* BLINK_EXEC_*                                                 */
  int32_t gemm_impl;            /* BLINK_GEMM_*                                                 */
  int32_t control_only;         /* 1: no model math, tokens come from a fixed hash (trace tests) */
  int32_t start_paused;         /* 1: the loop admits nothing until blink_start                 */
  int32_t wait_limit_ms;        /* bound of every wait inside the kernel (grid barrier, copy / MMA pipeline
                                   barriers): a wait that lasts longer ends the loop with device_status
                                   set and BLINK_LOOP_EXIT_ERROR.  0 = idle_exit_us + 3 s.  CTAs wait at a
                                   grid barrier while the control plane polls an empty queue, so a limit
                                   below idle_exit_us turns an idle period into a time-out error          */
  int64_t iteration_budget;     /* iterations per kernel launch, 0 = unbounded                  */
  int64_t idle_exit_us;         /* leave the GPU after this long without work, 0 = 2 s          */
  int64_t trace_capacity_words; /* int32 words of scheduling trace kept on the device, 0 = off  */
  int64_t stats_capacity_iters; /* per-iteration timing records kept on the device, 0 = off     */
  float* logits_capture;        /* DEVICE, caller-owned [logits_capture_rows][vocab] or NULL: row r
                                   receives the logits of the r-th sampled row since create      */
  int64_t logits_capture_rows;
  int32_t epilogue_fusion;      /* BLINK_FUSION_*                                               */
  int32_t policy;               /* BLINK_POLICY_*                                               */
} blink_sched_cfg;

/* Caller-owned DEVICE memory for the paged KV cache.  The library derives
 * n_blocks = bytes / (n_layers * 2 * n_kv_heads * block_size * head_dim * elem). */
typedef struct blink_kv_pool {
  uint32_t size;
  int32_t block_size; /* tokens per block (16) */
  void* base;         /* DEVICE, 256-byte aligned */
  uint64_t bytes;
} blink_kv_pool;

typedef struct blink_request {
  uint32_t size;
  int32_t n_prompt;
  const int32_t* prompt;        /* HOST, copied before return                                   */
  int32_t max_new_tokens;
  int32_t top_k;                /* 0 = greedy, else 1..64                                       */
  float temperature;            /* used when top_k > 0; must be > 0                             */
  int32_t eos_id;               /* -1 = none                                                    */
  uint64_t seed;                /* sampling stream key                                          */
  uint64_t user_tag;            /* returned with every event                                    */
  const int32_t* forced_tokens; /* HOST or NULL.  Teacher forcing for tests: max_new_tokens ids
                                   that are fed back instead of the sampled ones; the sampled ones
                                   are still the ones reported.                                 */
  float top_p;                  /* nucleus sampling (Section 4.2: Top-P with temperature): in (0, 1) the
                                   draw is restricted to the smallest set of most likely tokens whose
                                   probability reaches top_p (taken among the top_k largest when top_k > 0,
                                   else over the whole vocabulary); 0 or >= 1 = no cut.  Needs
                                   temperature > 0                                              */
  int32_t reserved0;
} blink_request;

typedef struct blink_token_event {
  uint64_t ticket;
  uint64_t user_tag;
  int32_t index;        /* 0-based index of this token in the request's output */
  int32_t token;
  int32_t is_first, is_last;
  uint64_t t_device_ns; /* device global timer when the token was published    */
  uint64_t t_host_ns;   /* host CLOCK_MONOTONIC when blink_poll saw it         */
  uint64_t t_submit_ns; /* host CLOCK_MONOTONIC when the request was submitted */
} blink_token_event;

typedef struct blink_stats {
  uint32_t size;
  int32_t loop_state;     /* BLINK_LOOP_*                                         */
  int32_t device_status;  /* 0 = fine, else first error the device loop recorded  */
  int32_t n_blocks;       /* KV blocks in the pool                                */
  int64_t iterations;     /* traced (non-idle) iterations since create            */
  int64_t launches;       /* kernel launches issued by the library since create   */
  int64_t tokens_out;     /* tokens published since create                        */
  int64_t prompt_tokens;  /* prompt tokens prefetched since create                */
  int64_t trace_words;    /* valid words in the trace                             */
  int64_t device_clock_offset_ns; /* host CLOCK_MONOTONIC minus device global timer at create */
  int32_t free_blocks, reserved_blocks, batch_live, reserved1;
  int64_t bytes_to_device;   /* bytes blink_submit wrote into the mapped submit areas (entries, prompts,
                                forced tokens) since create                                          */
  int64_t bytes_from_device; /* bytes the device wrote into the mapped host mirrors for the tokens blink_poll
                                has handed out since create (token, timestamp and count word: 16 each) */
} blink_stats;

/* One record per traced iteration, for throughput / roofline arithmetic. */
typedef struct blink_iter_stat {
  uint64_t t_begin_ns;    /* device timer: scheduling of this iteration starts */
  uint64_t t_forward_ns;  /* scheduling done, forward starts                   */
  uint64_t t_end_ns;      /* tokens of this iteration published                */
  int32_t n_tokens;       /* rows in the step (decode + prefill chunk)         */
  int32_t n_decode;       /* decode rows                                       */
  int32_t n_sample_rows;  /* rows that went through LM head + sampler          */
  int32_t n_items;        /* requests in the step                              */
  int64_t ctx_tokens;     /* sum over rows of keys attended (attention flops)  */
  int64_t kv_tokens;      /* sum over requests in the step of their context length after the
                             step: KV tokens an ideal kernel reads once per step              */
  uint64_t phase_ns[16];  /* persistent / manual mode: device time per phase kind, summed over the
                             layers, each including the grid barrier that closes it.  Index:
                             0 norm1(+embedding) 1 QKV 2 RoPE+KV write 3 attention 4 O 5 norm2
                             6 gate/up 7 SwiGLU 8 down 9 final norm 10 LM head 11 sampling
                             12 expert grouping + gather (routed experts); 13..15 unused (zero)                                             */
} blink_iter_stat;

/* Bytes of the flat weight buffer for a model shape (dtype taken from cfg). */
uint64_t blink_weights_bytes(const blink_model_cfg* cfg);

/* Byte offset of tensor `tensor_id` in the flat weight buffer, or UINT64_MAX.
 * ids: 0 embed[V,d], 1 wqkv[L,(Hq+2Hkv)*hd,d] (q rows, k rows, v rows),
 * 2 wo[L,d,Hq*hd], 3 wgu[L,E',2F,d] (gate rows then up rows; E' = max(1,E)),
 * 4 wd[L,E',d,F], 5 wr[L,E,d] fp32, 6 norm1[L,d] fp32, 7 norm2[L,d] fp32,
 * 8 normf[d] fp32, 9 lm_head[V,d].  All matrices row-major [out, in]; every tensor
 * starts on a 256-byte boundary. */
uint64_t blink_weight_offset(const blink_model_cfg* cfg, int tensor_id);

/* Convert the GEMM matrices of `weights` (DEVICE, caller-owned, blink_weights_bytes(cfg) bytes)
 * in place from cfg->weights_layout to `to_layout`.  Part of set-up (the provisioning plane of
 * Section 4.1: the host prepares the engine once, then leaves the inference path).  Synchronous;
 * uses temporary device scratch of one 128-row panel per SM and of one gate/up matrix.  BLINK_EINVAL when the shape does
 * not admit the streaming layout or the dtype is not bf16; a no-op when the layouts are equal.
 * No context may be using the buffer meanwhile. */
int blink_convert_weights(const blink_model_cfg* cfg, void* weights, int to_layout);

/* KV blocks a pool of `bytes` yields for this model shape and block size. */
int64_t blink_kv_blocks_for_bytes(const blink_model_cfg* cfg, int block_size, uint64_t bytes);

/* Set up ring, arenas, tables and mailboxes (library-owned), and launch the loop
 * (persistent mode).  On failure *out is NULL and nothing stays allocated. */
int blink_create(const blink_model_cfg* model, const blink_sched_cfg* sched, const blink_kv_pool* kv,
                 blink_ctx** out);

/* Let a loop created with start_paused begin admitting (everything submitted
 * before this call is visible to its first iteration). */
int blink_start(blink_ctx* ctx);

/* Non-blocking, thread-safe.  Copies the prompt, stamps the next ticket (FCFS
 * order), publishes the request to the device.  BLINK_EAGAIN when every slot is
 * in use, BLINK_EINVAL for lengths/ids/sampling parameters out of range or a
 * request whose worst-case KV need exceeds the whole pool. */
int blink_submit(blink_ctx* ctx, const blink_request* req, uint64_t* ticket_out);

/* Collect up to max_events new tokens; waits at most timeout_us for the first one.
 * Returns the number of events (>= 0) or a negative error.  Events of one request
 * arrive in index order.  Never makes the device wait.  Also re-launches a loop
 * that left the GPU (budget, idle) while work is outstanding. */
int blink_poll(blink_ctx* ctx, blink_token_event* out, int max_events, int timeout_us);

/* Ask the loop to drop a request (the paper lists early exits among what the serving path has to handle,
 * Section 1; it gives no mechanism).  The device retires it at the end of the step in which it sees the mark:
 * its KV blocks return to the free list, its reservation and batch slot are released, no further token is
 * produced.  Tokens published before that are still delivered; then blink_poll hands out one closing event
 * for the request with token = -1, index = number of tokens it produced, and is_last set (no other event of
 * a cancelled request carries is_last).  A request that was still waiting for admission is admitted first and
 * retired at the end of its first step.  BLINK_EINVAL when the ticket is unknown or the request has already
 * delivered its last token.  Thread-safe, non-blocking. */
int blink_cancel(blink_ctx* ctx, uint64_t ticket);

/* Stepped mode only: run `n_iterations` iterations, one host launch per phase,
 * and wait for them. */
int blink_step(blink_ctx* ctx, int n_iterations);

/* Manual mode only: launch the loop kernel once with an iteration budget of
 * `n_iterations`, wait until it has left the GPU (budget used up, or nothing left to do
 * for idle_exit_us) and report the launch's duration measured with CUDA events on the
 * library's stream.  One launch = up to n_iterations whole steps of the hot path. */
int blink_run(blink_ctx* ctx, int64_t n_iterations, float* elapsed_ms);

/* Ask the loop to leave the GPU and wait (bounded) until it has. State stays
 * intact; blink_poll / blink_submit / blink_start re-launch it when needed
 * unless `final` is non-zero. */
int blink_stop(blink_ctx* ctx, int final, int timeout_ms);

/* Stop the loop (bounded wait), free library-owned memory.  BLINK_ETIMEDOUT, and
 * nothing freed, if the kernel has not left in time. */
int blink_destroy(blink_ctx* ctx, int timeout_ms);

int blink_get_stats(blink_ctx* ctx, blink_stats* out);

/* Copy up to `capacity` int32 words of the scheduling trace into `out` (HOST);
 * *n_words receives the number of valid words on the device.  One variable-length
 * record per traced (non-idle) iteration:
 *   header, 12 words: magic 0x424C4B31, iteration, W (highest ticket visible to this
 *     iteration), n_admitted, n_scheduled, n_allocated, n_sampled, n_finished, n_freed,
 *     free blocks after the iteration, reserved blocks after the iteration, record words;
 *   admitted  : (ticket, batch slot) pairs, in admission order;
 *   scheduled : (batch slot, ticket, phase 1=prefill 2=decode, start position, n tokens),
 *               ascending batch slot;
 *   allocated : (batch slot, logical block index, physical block) in allocation order;
 *   sampled   : (batch slot, token) ascending batch slot;
 *   finished  : tickets, ascending batch slot;  freed: physical blocks in push order. */
int blink_get_trace(blink_ctx* ctx, int32_t* out, int64_t capacity, int64_t* n_words);

/* Copy up to `capacity` per-iteration records into `out` (HOST). */
int blink_get_iter_stats(blink_ctx* ctx, blink_iter_stat* out, int64_t capacity, int64_t* n_records);

/* Test aid: the in-step sampler alone (Section 4.2, sampling captured inside the step).
 * `logits` is a DEVICE array [rows][vocab] (fp32); the per-row parameter arrays and `out`
 * are HOST arrays of length rows.  Row r is sampled exactly as the loop samples token
 * gen_index[r] of request ticket[r]: greedy when top_k[r] == 0, else top-k (<= 64) with
 * temperature and the counter-based random draw keyed by seed[r].  Synchronous; allocates
 * and frees a small device scratch. */
int blink_sample(const float* logits, int rows, int vocab, const int32_t* top_k, const float* temperature,
                 const uint64_t* ticket, const int32_t* gen_index, const uint64_t* seed, int32_t* out);

/* blink_sample with the nucleus cut of Section 4.2 ("Top-P with temperature"): `top_p` is a HOST array of
 * length rows; row r is sampled as the loop samples a request with top_k[r], temperature[r] and
 * top_p[r] (see blink_request.top_p).  Arithmetic, so that results do not depend on the order of a
 * parallel sum: integer weights floor(exp(z - z_max) * 2^40), the nucleus is the shortest prefix of the
 * order (z desc, index asc) whose weight times 2^24 reaches round(top_p * 2^24) times the total weight,
 * and the 24-bit uniform draw is scaled to the nucleus' weight. */
int blink_sample_top_p(const float* logits, int rows, int vocab, const int32_t* top_k, const float* temperature,
                       const float* top_p, const uint64_t* ticket, const int32_t* gen_index, const uint64_t* seed,
                       int32_t* out);

/* blink_sample for callers that cannot allocate.  The paper has no counterpart: this is a
 * convenience of this library.  Some callers must not call cudaMalloc / cudaFree once they
 * are running: a server that handed all free device memory to the KV pool at start-up (a
 * later allocation can simply fail), or code on a path where the implicit device-wide
 * synchronisation of cudaFree is not acceptable.  This variant computes exactly what
 * blink_sample computes, row for row, but keeps its per-row parameters and results in a
 * fixed scratch array that is part of the library image (32 KiB of device memory on every
 * GPU that loads the library, held until the process exits) instead of a temporary
 * allocation.  It calls no cudaMalloc, cudaFree or other allocating routine.
 *
 * Arguments as for blink_sample (`logits` DEVICE [rows][vocab] fp32; the parameter arrays and
 * `out` HOST, length rows).  rows must not exceed BLINK_SAMPLE_NOALLOC_MAX_ROWS: a larger
 * value is refused with BLINK_ETOOBIG before anything is touched; split the rows over
 * several calls instead.
 *
 * The first call on each device does the set-up: it looks up the device address of the scratch
 * array (one runtime query, with that device current) and creates the stream the call works on
 * (a driver object, no device memory from the allocator); make that first call before any
 * stream capture begins.  Every later call only enqueues copies and one kernel on that stream
 * and waits for the stream: it neither uses the legacy default stream nor synchronises the
 * device, so other streams keep running.  Consequences for the caller: `logits` must be
 * complete before the call (synchronise the stream that produced it); and the kernel needs
 * SMs like any other launch, so while a persistent serving loop of this library occupies every
 * SM of the GPU the call waits until that loop leaves (stop it, or let it reach its idle exit).
 *
 * All calls on a device share the one scratch array and it keeps the previous call's
 * contents: every call overwrites the part it uses before the kernel reads it, nothing has
 * to start at zero.  Calls that overlap on the same GPU (from several threads or processes
 * sharing a context) would race on the array: the library serialises its own callers with a
 * mutex, and the call is synchronous, so a single process is safe. */
#define BLINK_SAMPLE_NOALLOC_MAX_ROWS 1024
int blink_sample_noalloc(const float* logits, int rows, int vocab, const int32_t* top_k, const float* temperature,
                         const uint64_t* ticket, const int32_t* gen_index, const uint64_t* seed, int32_t* out);

const char* blink_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* BLINK_H_ */
