// libblink: kernels of the GPU-resident serving loop and the C ABI around them.
//
// Persistent mode: one cooperative kernel (one CTA per SM) loops on the device;
// CTA 0 runs the control plane, then all CTAs run the phases of the step
// separated by grid barriers.  Stepped mode runs the very same device functions
// as one host launch per phase (for profilers and debugging).
#include <cuda_runtime.h>
#include <stdio.h>
#include <string.h>
#include <time.h>

#include <atomic>
#include <chrono>
#include <cmath>
#include <deque>
#include <mutex>
#include <new>
#include <thread>
#include <vector>

#include "../../include/blink.h"
#include "control.cuh"
#include "dev_ctx.cuh"
#include "forward.cuh"
#include "gemm_tc.cuh"
#include "attention.cuh"
#include "kernel_set.h"

namespace blink {

// ---- stepped mode ----------------------------------------------------------------------
__global__ void __launch_bounds__(CTRL_THREADS, 1) blink_control_kernel(const __grid_constant__ DevCtx c, int post_only) {
  if (post_only) {
    if (c.ss->pending_post) post_step(c);
    if (threadIdx.x == 0) c.ss->cmd = CMD_NONE;
    return;
  }
  long long li = 0;
  control_phase(c, li);
}

// Sampler alone over caller-provided logits (one CTA per row).
__global__ void __launch_bounds__(FWD_THREADS, 1)
blink_sample_kernel(const float* logits, int rows, int V, const int* top_k, const float* temp,
                    const unsigned long long* ticket, const int* gen_index, const unsigned long long* seed, int* out,
                    const float* top_p) {
  extern __shared__ __align__(1024) float smem[];
  for (int r = blockIdx.x; r < rows; r += gridDim.x) {
    const int tok = sample_row(logits + (size_t)r * V, V, min(top_k[r], MAX_TOPK), temp[r], top_p ? top_p[r] : 0.f, ticket[r],
                               gen_index[r], seed[r], smem);
    if (threadIdx.x == 0) out[r] = tok;
  }
}

// In-place conversion of one GEMM matrix between row-major and the streaming tile layout.
// A 128-row panel keeps its byte range; one CTA copies the panel to its scratch slot, then
// writes it back in the other layout.
__global__ void __launch_bounds__(256) blink_retile_kernel(char* base, long long n_panels, int K, char* scratch,
                                                           int to_streaming) {
  const size_t panel_bytes = (size_t)128 * K * 2;
  const int cpr = K / 8;  // 16-byte chunks per row
  uint4* tmp = reinterpret_cast<uint4*>(scratch + (size_t)blockIdx.x * panel_bytes);
  for (long long p = blockIdx.x; p < n_panels; p += gridDim.x) {
    uint4* panel = reinterpret_cast<uint4*>(base + (size_t)p * panel_bytes);
    const int n16 = 128 * cpr;
    for (int i = threadIdx.x; i < n16; i += blockDim.x) tmp[i] = panel[i];
    __syncthreads();
    for (int i = threadIdx.x; i < n16; i += blockDim.x) {
      const int r = i / cpr, cc = i % cpr;
      const int kb = cc >> 3, c8 = cc & 7;
      const int tiled = kb * 1024 + r * 8 + (c8 ^ (r & 7));  // in 16-byte units
      if (to_streaming) panel[tiled] = tmp[i];
      else panel[i] = tmp[tiled];
    }
    __syncthreads();
  }
}

// Row permutation of one gate/up matrix ([2F][K], gate rows first): the streaming layout stores it with
// gate row f and up row f adjacent (rows 2f and 2f + 1), so that one 128-row weight tile holds both
// halves of 64 features and the GEMM epilogue can form silu(gate) * up from one accumulator.
__global__ void __launch_bounds__(256) blink_interleave_rows_kernel(uint4* __restrict__ dst, const uint4* __restrict__ src,
                                                                    long long F, int cpr, int interleave) {
  const long long total = 2 * F * cpr;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long r = i / cpr;
    const int cc = (int)(i - r * cpr);
    const long long sr = interleave ? ((r & 1) * F + (r >> 1)) : (r < F ? 2 * r : 2 * (r - F) + 1);
    dst[i] = src[sr * cpr + cc];
  }
}

__global__ void blink_clock_probe_kernel(Mailbox* mb) {
  mb->clock_probe = global_timer_ns();
  __threadfence_system();
}

}  // namespace blink

// =========================================================================================
// Host side
// =========================================================================================
using namespace blink;

namespace {

uint64_t now_ns() {
  timespec ts;
  clock_gettime(CLOCK_MONOTONIC, &ts);
  return (uint64_t)ts.tv_sec * 1000000000ull + (uint64_t)ts.tv_nsec;
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Layout {
  uint64_t off[10];
  uint64_t total;
};

bool model_ok(const blink_model_cfg* m) {
  if (!m || m->size != sizeof(blink_model_cfg)) return false;
  if (m->n_layers < 1 || m->d_model < 16 || m->n_q_heads < 1 || m->n_kv_heads < 1 || m->vocab < 2 || m->d_ff < 16)
    return false;
  if (m->head_dim != 64 && m->head_dim != 128) return false;
  if (m->n_q_heads % m->n_kv_heads) return false;
  const int rep = m->n_q_heads / m->n_kv_heads;
  if (rep != 1 && rep != 2 && rep != 4 && rep != 8) return false;
  if (m->dtype != BLINK_DTYPE_BF16 && m->dtype != BLINK_DTYPE_FP32) return false;
  if (m->n_experts < 0 || (m->n_experts > 0 && (m->top_k_experts < 1 || m->top_k_experts > m->n_experts))) return false;
  if (m->d_model % 8 || m->d_model > 8192 || m->d_ff % 8) return false;   // rows move as 16-byte vectors
  return true;
}

Layout weight_layout(const blink_model_cfg* m) {
  Layout lo;
  const uint64_t esz = m->dtype == BLINK_DTYPE_BF16 ? 2 : 4;
  const uint64_t L = m->n_layers, d = m->d_model, V = m->vocab, F = m->d_ff;
  const uint64_t qd = (uint64_t)m->n_q_heads * m->head_dim, kvd = (uint64_t)m->n_kv_heads * m->head_dim;
  const uint64_t E1 = m->n_experts > 0 ? m->n_experts : 1, E = m->n_experts;
  const uint64_t n[10] = {V * d, L * (qd + 2 * kvd) * d, L * d * qd, L * E1 * 2 * F * d, L * E1 * d * F,
                          L * E * d, L * d, L * d, d, V * d};
  const uint64_t es[10] = {esz, esz, esz, esz, esz, 4, 4, 4, 4, esz};
  uint64_t off = 0;
  for (int i = 0; i < 10; ++i) {
    lo.off[i] = off;
    off += align_up(n[i] * es[i], 256);
  }
  lo.total = off;
  return lo;
}

}  // namespace

struct SlotInfo {
  uint64_t ticket = 0, user_tag = 0, t_submit_ns = 0;
  int32_t max_new = 0, consumed = 0;
  bool busy = false;
};

struct blink_ctx {
  DevCtx dc;
  blink_model_cfg model;
  blink_sched_cfg sched;
  cudaStream_t stream = nullptr, copy_stream = nullptr;
  std::vector<void*> dev_allocs, host_allocs;
  Mailbox* mbox = nullptr;       // host view
  SubEntry* sub_q = nullptr;
  int32_t *sub_tokens = nullptr, *sub_forced = nullptr, *out_tokens = nullptr;
  uint64_t* out_time = nullptr;
  uint32_t* out_count = nullptr;
  uint32_t* cancel = nullptr;    // host view of the cancel marks
  std::mutex mu;
  std::vector<SlotInfo> slots;
  std::deque<int> active;
  int hint = 0;
  uint64_t next_ticket = 0;
  std::atomic<int64_t> launches{0};
  int64_t bytes_to_device = 0, bytes_from_device = 0;
  int64_t clock_offset = 0;
  bool final_stop = false;
  int n_sms = 1;
  size_t smem_bytes = 0;
  int grid = 1;
  TcHost tc_host;
  KernelSet ks{nullptr, nullptr};
  bool manual = false;
  bool pair = false;   // GEMMs on CTA pairs: kernels launched with clusters of two
  cudaEvent_t ev0 = nullptr, ev1 = nullptr;
  // host-driven comparison arms: a thread of the library launches one iteration at a time
  int host_driven = 0;                 // 0, BLINK_EXEC_HOST_GRAPH or BLINK_EXEC_HOST_LAUNCHES
  int device = 0;                      // the device of the context: the driver thread selects it
  cudaGraphExec_t iter_graph = nullptr;
  std::thread driver;
  std::atomic<bool> driver_stop{false};
  std::atomic<int> driver_error{0};
};

namespace {

template <typename T>
int dev_alloc(blink_ctx* x, T** p, size_t n, bool zero = true) {
  void* q = nullptr;
  if (cudaMalloc(&q, n * sizeof(T) > 0 ? n * sizeof(T) : 16) != cudaSuccess) return BLINK_ENOMEM;
  if (zero && cudaMemset(q, 0, n * sizeof(T) > 0 ? n * sizeof(T) : 16) != cudaSuccess) return BLINK_ECUDA;
  x->dev_allocs.push_back(q);
  *p = reinterpret_cast<T*>(q);
  return BLINK_OK;
}

template <typename T>
int pinned_alloc(blink_ctx* x, T** host, T** dev, size_t n) {
  void* q = nullptr;
  const size_t bytes = n * sizeof(T) > 0 ? n * sizeof(T) : 16;
  if (cudaHostAlloc(&q, bytes, cudaHostAllocMapped | cudaHostAllocPortable) != cudaSuccess) return BLINK_ENOMEM;
  memset(q, 0, bytes);
  void* d = nullptr;
  if (cudaHostGetDevicePointer(&d, q, 0) != cudaSuccess) return BLINK_ECUDA;
  x->host_allocs.push_back(q);
  *host = reinterpret_cast<T*>(q);
  *dev = reinterpret_cast<T*>(d);
  return BLINK_OK;
}

void free_all(blink_ctx* x) {
  for (void* p : x->dev_allocs) cudaFree(p);
  for (void* p : x->host_allocs) cudaFreeHost(p);
  x->dev_allocs.clear();
  x->host_allocs.clear();
  tc_host_free(x->tc_host);
  if (x->ev0) cudaEventDestroy(x->ev0);
  if (x->ev1) cudaEventDestroy(x->ev1);
  x->ev0 = x->ev1 = nullptr;
  if (x->iter_graph) cudaGraphExecDestroy(x->iter_graph);
  x->iter_graph = nullptr;
  if (x->stream) cudaStreamDestroy(x->stream);
  if (x->copy_stream) cudaStreamDestroy(x->copy_stream);
  x->stream = x->copy_stream = nullptr;
}

size_t phase_smem_bytes(const blink_ctx* x) {
  size_t a = sizeof(float) * (size_t)ATTN_SMEM_FLOATS(x->dc.hd, x->dc.n_rep);
  size_t s = sizeof(float) * (size_t)SAMPLE_SMEM_FLOATS;
  size_t m = a > s ? a : s;
  if (x->dc.gemm_tc && tc_smem_bytes() > m) m = tc_smem_bytes();
  const size_t moe = x->dc.E > 0 ? (size_t)x->dc.Tmax * x->dc.topE * sizeof(int) : 0;   // routing lists of a step
  if (moe > m) m = moe;
  if (x->dc.dtype == BLINK_DTYPE_BF16) {
    const size_t ab = x->dc.hd == 64 ? (size_t)att_smem_bytes<64>() : (size_t)att_smem_bytes<128>();
    if (ab > m) m = ab;
  }
  return m;
}

int launch_loop(blink_ctx* x) {
  x->mbox->stop = 0;
  x->mbox->loop_state = BLINK_LOOP_RUNNING;
  std::atomic_thread_fence(std::memory_order_seq_cst);
  void* args[] = {(void*)&x->dc};
  const void* fn = x->ks.loop;
  // the grid barrier counts arrivals from zero in every launch
  if (cudaMemsetAsync(&x->dc.ss->bar_ctr, 0, sizeof(unsigned long long), x->stream) != cudaSuccess) return BLINK_ECUDA;
  cudaError_t e;
  if (x->pair) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(x->grid); cfg.blockDim = dim3(FWD_THREADS); cfg.dynamicSmemBytes = x->smem_bytes; cfg.stream = x->stream;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension; at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeCooperative; at[1].val.cooperative = 1;
    cfg.attrs = at; cfg.numAttrs = 2;
    e = cudaLaunchKernelExC(&cfg, fn, args);
  } else {
    e = cudaLaunchCooperativeKernel(fn, dim3(x->grid), dim3(FWD_THREADS), args, x->smem_bytes, x->stream);
  }
  if (e != cudaSuccess) {
    x->mbox->loop_state = BLINK_LOOP_EXIT_ERROR;
    fprintf(stderr, "blink: persistent launch failed: %s\n", cudaGetErrorString(e));
    return BLINK_ECUDA;
  }
  x->launches += 1;
  return BLINK_OK;
}

// Re-instantiate a loop that left the GPU while work is outstanding (caller holds mu).
int pump(blink_ctx* x) {
  if (x->host_driven) return x->driver_error.load(std::memory_order_acquire) != 0 ? BLINK_EDEVICE : BLINK_OK;
  if (x->dc.stepped || x->manual) return BLINK_OK;
  const uint32_t st = x->mbox->loop_state;
  if (st == BLINK_LOOP_RUNNING) return BLINK_OK;
  if (st == BLINK_LOOP_EXIT_ERROR) return BLINK_EDEVICE;
  if (x->final_stop) return BLINK_ESTOPPED;
  const bool work = !x->active.empty();
  if (!work && st != BLINK_LOOP_NOT_STARTED) return BLINK_OK;
  if (cudaStreamSynchronize(x->stream) != cudaSuccess) return BLINK_ECUDA;
  return launch_loop(x);
}

void launch_phase(blink_ctx* x, int phase, int layer, int sub = 0) {
  void* args[] = {(void*)&x->dc, (void*)&phase, (void*)&layer, (void*)&sub};
  if (x->pair) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(x->grid); cfg.blockDim = dim3(FWD_THREADS); cfg.dynamicSmemBytes = x->smem_bytes; cfg.stream = x->stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension; at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    cudaLaunchKernelExC(&cfg, x->ks.phase, args);
  } else {
    cudaLaunchKernel(x->ks.phase, dim3(x->grid), dim3(FWD_THREADS), args, x->smem_bytes, x->stream);
  }
  x->launches += 1;
}

int step_once(blink_ctx* x) {
  blink_control_kernel<<<1, CTRL_THREADS, 0, x->stream>>>(x->dc, 0);
  x->launches += 1;
  if (!x->dc.control_only) {
    for (int l = 0; l < x->dc.L; ++l)
      for (int ph = PH_NORM1; ph <= PH_DOWN; ++ph) {
        if (x->dc.E > 0 && (ph == PH_GU || ph == PH_DOWN)) {
          if (ph == PH_GU) launch_phase(x, PH_MOE_GROUP, l);
          for (int e = 0; e < x->dc.E; ++e) launch_phase(x, ph, l, e);
        } else if (!(x->dc.fused && (ph == PH_ROPE || ph == PH_SILU))) {   // fused into the GEMM epilogues
          launch_phase(x, ph, l);
        }
      }
    for (int ph = PH_FNORM; ph <= PH_SAMPLE; ++ph) launch_phase(x, ph, 0);
  }
  return cudaGetLastError() == cudaSuccess ? BLINK_OK : BLINK_ECUDA;
}

// The host-resident serving loop of the comparison arms: while requests are outstanding, launch one iteration
// and wait for it (the host is on the critical path of every token, as in the stacks of Section 6.1).
void driver_loop(blink_ctx* x) {
  if (cudaSetDevice(x->device) != cudaSuccess) {
    x->driver_error.store(BLINK_ECUDA, std::memory_order_release);
    return;
  }
  while (!x->driver_stop.load(std::memory_order_acquire)) {
    bool work;
    {
      std::lock_guard<std::mutex> g(x->mu);
      work = !x->active.empty() && (!x->dc.start_paused || x->mbox->start != 0);
    }
    if (!work) {
      std::this_thread::sleep_for(std::chrono::microseconds(50));
      continue;
    }
    int rc = BLINK_OK;
    if (x->iter_graph) {
      if (cudaGraphLaunch(x->iter_graph, x->stream) != cudaSuccess) rc = BLINK_ECUDA;
      x->launches += 1;
    } else {
      rc = step_once(x);
    }
    if (rc == BLINK_OK && cudaStreamSynchronize(x->stream) != cudaSuccess) rc = BLINK_ECUDA;
    if (rc == BLINK_OK && x->mbox->device_status > 0 && x->mbox->device_status != DEV_ERR_TRACE_OVERFLOW) rc = BLINK_EDEVICE;
    if (rc != BLINK_OK) {
      x->driver_error.store(rc, std::memory_order_release);
      return;
    }
  }
}

void driver_start(blink_ctx* x) {
  if (!x->host_driven || x->driver.joinable() || x->driver_error.load() != 0) return;
  x->driver_stop.store(false, std::memory_order_release);
  x->driver = std::thread(driver_loop, x);
}

// never called with x->mu held: the driver takes it between iterations
void driver_join(blink_ctx* x) {
  if (!x->driver.joinable()) return;
  x->driver_stop.store(true, std::memory_order_release);
  x->driver.join();
}

}  // namespace

extern "C" {

const char* blink_strerror(int code) {
  switch (code) {
    case BLINK_OK: return "ok";
    case BLINK_EAGAIN: return "no empty ring slot (back-pressure)";
    case BLINK_EINVAL: return "invalid argument";
    case BLINK_ESTOPPED: return "loop stopped";
    case BLINK_EDEVICE: return "device loop reported an error";
    case BLINK_ETIMEDOUT: return "timed out";
    case BLINK_ENOMEM: return "out of memory or pool too small";
    case BLINK_ECUDA: return "CUDA call failed";
    case BLINK_ETOOBIG: return "size exceeds a fixed capacity";
    default: return "unknown error";
  }
}

uint64_t blink_weights_bytes(const blink_model_cfg* cfg) {
  if (!model_ok(cfg)) return 0;
  return weight_layout(cfg).total;
}

uint64_t blink_weight_offset(const blink_model_cfg* cfg, int tensor_id) {
  if (!model_ok(cfg) || tensor_id < 0 || tensor_id > 9) return UINT64_MAX;
  return weight_layout(cfg).off[tensor_id];
}

int blink_convert_weights(const blink_model_cfg* cfg, void* weights, int to_layout) {
  if (!model_ok(cfg) || !weights || ((uintptr_t)weights & 255)) return BLINK_EINVAL;
  if (to_layout != BLINK_WEIGHTS_ROW_MAJOR && to_layout != BLINK_WEIGHTS_STREAMING) return BLINK_EINVAL;
  if (cfg->weights_layout != BLINK_WEIGHTS_ROW_MAJOR && cfg->weights_layout != BLINK_WEIGHTS_STREAMING) return BLINK_EINVAL;
  if (cfg->weights_layout == to_layout) return BLINK_OK;
  if (cfg->dtype != BLINK_DTYPE_BF16) return BLINK_EINVAL;
  const long long L = cfg->n_layers, d = cfg->d_model, F = cfg->d_ff, V = cfg->vocab;
  const long long qd = (long long)cfg->n_q_heads * cfg->head_dim, kvd = (long long)cfg->n_kv_heads * cfg->head_dim;
  const long long E1 = cfg->n_experts > 0 ? cfg->n_experts : 1;
  // (tensor id, rows per layer slice, total rows, columns)
  const long long rows_per[5] = {qd + 2 * kvd, d, 2 * F, d, V};
  const long long rows_tot[5] = {L * (qd + 2 * kvd), L * d, L * E1 * 2 * F, L * E1 * d, V};
  const long long cols[5] = {d, qd, d, F, d};
  const int ids[5] = {1, 2, 3, 4, 9};
  long long max_k = 0;
  for (int i = 0; i < 5; ++i) {
    if (rows_per[i] % 128 || cols[i] % 64) return BLINK_EINVAL;
    if (cols[i] > max_k) max_k = cols[i];
  }
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return BLINK_ECUDA;
  char* scratch = nullptr;
  if (cudaMalloc(&scratch, (size_t)sms * 128 * max_k * 2) != cudaSuccess) return BLINK_ENOMEM;
  const Layout lo = weight_layout(cfg);
  const bool to_streaming = to_layout == BLINK_WEIGHTS_STREAMING;
  const size_t gu_bytes = (size_t)2 * F * d * 2;
  char* gu_tmp = nullptr;
  if (cudaMalloc(&gu_tmp, gu_bytes) != cudaSuccess) { cudaFree(scratch); return BLINK_ENOMEM; }
  int rc = BLINK_OK;
  // gate/up rows are interleaved in the streaming layout: permute each [2F][d] matrix while it is row-major
  auto permute_gate_up = [&]() {
    for (long long m = 0; m < L * E1 && rc == BLINK_OK; ++m) {
      char* mat = static_cast<char*>(weights) + lo.off[3] + (size_t)m * gu_bytes;
      if (cudaMemcpyAsync(gu_tmp, mat, gu_bytes, cudaMemcpyDeviceToDevice, 0) != cudaSuccess) rc = BLINK_ECUDA;
      blink_interleave_rows_kernel<<<sms * 8, 256>>>(reinterpret_cast<uint4*>(mat), reinterpret_cast<const uint4*>(gu_tmp), F,
                                                     (int)(d / 8), to_streaming);
      if (cudaGetLastError() != cudaSuccess) rc = BLINK_ECUDA;
    }
  };
  if (to_streaming) permute_gate_up();
  for (int i = 0; i < 5 && rc == BLINK_OK; ++i) {
    blink_retile_kernel<<<sms, 256>>>(static_cast<char*>(weights) + lo.off[ids[i]], rows_tot[i] / 128, (int)cols[i], scratch,
                                      to_streaming);
    if (cudaGetLastError() != cudaSuccess) rc = BLINK_ECUDA;
  }
  if (!to_streaming) permute_gate_up();
  if (cudaDeviceSynchronize() != cudaSuccess) rc = BLINK_ECUDA;
  cudaFree(scratch);
  cudaFree(gu_tmp);
  return rc;
}

int64_t blink_kv_blocks_for_bytes(const blink_model_cfg* cfg, int block_size, uint64_t bytes) {
  if (!model_ok(cfg) || block_size < 1) return BLINK_EINVAL;
  const uint64_t esz = cfg->dtype == BLINK_DTYPE_BF16 ? 2 : 4;
  const uint64_t per = (uint64_t)cfg->n_layers * 2 * cfg->n_kv_heads * block_size * cfg->head_dim * esz;
  return (int64_t)(bytes / per);
}

static int sample_impl(const float* logits, int rows, int vocab, const int32_t* top_k, const float* temperature,
                       const float* top_p, const uint64_t* ticket, const int32_t* gen_index, const uint64_t* seed,
                       int32_t* out) {
  if (!logits || rows < 1 || vocab < 2 || !top_k || !temperature || !ticket || !gen_index || !seed || !out)
    return BLINK_EINVAL;
  for (int r = 0; r < rows; ++r) {
    const bool nucleus = top_p && top_p[r] > 0.f && top_p[r] < 1.f;
    if (top_k[r] < 0 || top_k[r] > MAX_TOPK || ((top_k[r] > 0 || nucleus) && !(temperature[r] > 0.f))) return BLINK_EINVAL;
    if (top_p && !(top_p[r] >= 0.f)) return BLINK_EINVAL;
  }
  char* d = nullptr;
  const size_t n = (size_t)rows;
  const size_t bytes = n * (4 + 4 + 8 + 4 + 8 + 4 + 4);
  if (cudaMalloc(&d, bytes) != cudaSuccess) return BLINK_ENOMEM;
  unsigned long long* d_ticket = (unsigned long long*)d;
  unsigned long long* d_seed = d_ticket + n;
  int* d_topk = (int*)(d_seed + n);
  float* d_temp = (float*)(d_topk + n);
  int* d_gen = (int*)(d_temp + n);
  int* d_out = d_gen + n;
  float* d_topp = (float*)(d_out + n);
  int rc = BLINK_OK;
  if (top_p && cudaMemcpy(d_topp, top_p, n * 4, cudaMemcpyHostToDevice) != cudaSuccess) rc = BLINK_ECUDA;
  if (cudaMemcpy(d_ticket, ticket, n * 8, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(d_seed, seed, n * 8, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(d_topk, top_k, n * 4, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(d_temp, temperature, n * 4, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(d_gen, gen_index, n * 4, cudaMemcpyHostToDevice) != cudaSuccess)
    rc = BLINK_ECUDA;
  if (rc == BLINK_OK) {
    const int grid = rows < 1184 ? rows : 1184;
    blink_sample_kernel<<<grid, FWD_THREADS, SAMPLE_SMEM_FLOATS * sizeof(float)>>>(
        logits, rows, vocab, d_topk, d_temp, d_ticket, d_gen, d_seed, d_out, top_p ? d_topp : nullptr);
    if (cudaDeviceSynchronize() != cudaSuccess) rc = BLINK_ECUDA;
    else if (cudaMemcpy(out, d_out, n * 4, cudaMemcpyDeviceToHost) != cudaSuccess) rc = BLINK_ECUDA;
  }
  cudaFree(d);
  return rc;
}

int blink_sample(const float* logits, int rows, int vocab, const int32_t* top_k, const float* temperature,
                 const uint64_t* ticket, const int32_t* gen_index, const uint64_t* seed, int32_t* out) {
  return sample_impl(logits, rows, vocab, top_k, temperature, nullptr, ticket, gen_index, seed, out);
}

int blink_sample_top_p(const float* logits, int rows, int vocab, const int32_t* top_k, const float* temperature,
                       const float* top_p, const uint64_t* ticket, const int32_t* gen_index, const uint64_t* seed,
                       int32_t* out) {
  if (!top_p) return BLINK_EINVAL;
  return sample_impl(logits, rows, vocab, top_k, temperature, top_p, ticket, gen_index, seed, out);
}

// ---- sampler for callers that cannot allocate --------------------------------------------------
// Per-row parameters and results live in a fixed array inside the library image.  In host code
// the symbol below is only a handle: the device address comes from cudaGetSymbolAddress, once
// per device, with that device current.
namespace {
constexpr size_t NOALLOC_ROW_BYTES = 8 + 8 + 4 + 4 + 4 + 4;  // ticket, seed, top_k, temperature, gen_index, out
constexpr int NOALLOC_MAX_DEVICES = 64;
}  // namespace
static __device__ __align__(256) unsigned char g_sample_scratch[BLINK_SAMPLE_NOALLOC_MAX_ROWS * NOALLOC_ROW_BYTES];
namespace {
std::mutex g_noalloc_mu;
void* g_noalloc_ptr[NOALLOC_MAX_DEVICES] = {nullptr};
cudaStream_t g_noalloc_stream[NOALLOC_MAX_DEVICES] = {nullptr};
}  // namespace

int blink_sample_noalloc(const float* logits, int rows, int vocab, const int32_t* top_k, const float* temperature,
                         const uint64_t* ticket, const int32_t* gen_index, const uint64_t* seed, int32_t* out) {
  if (!logits || rows < 1 || vocab < 2 || !top_k || !temperature || !ticket || !gen_index || !seed || !out)
    return BLINK_EINVAL;
  if (rows > BLINK_SAMPLE_NOALLOC_MAX_ROWS) {
    fprintf(stderr, "blink_sample_noalloc: %d rows exceed the fixed scratch capacity of %d rows; split the call\n", rows,
            BLINK_SAMPLE_NOALLOC_MAX_ROWS);
    return BLINK_ETOOBIG;
  }
  for (int r = 0; r < rows; ++r)
    if (top_k[r] < 0 || top_k[r] > MAX_TOPK || (top_k[r] > 0 && !(temperature[r] > 0.f))) return BLINK_EINVAL;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NOALLOC_MAX_DEVICES) return BLINK_ECUDA;
  std::lock_guard<std::mutex> g(g_noalloc_mu);  // one user of the shared scratch at a time
  if (!g_noalloc_ptr[dev]) {
    // first call on this device: the address of the scratch array, and a stream of the call's own so
    // that it neither joins the legacy default stream nor synchronises the whole device
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_sample_scratch);
    if (e != cudaSuccess || !p) {
      fprintf(stderr, "blink_sample_noalloc: cudaGetSymbolAddress failed: %s\n", cudaGetErrorString(e));
      return BLINK_ECUDA;
    }
    cudaStream_t st = nullptr;
    if (cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking) != cudaSuccess) return BLINK_ECUDA;
    g_noalloc_stream[dev] = st;
    g_noalloc_ptr[dev] = p;
  }
  cudaStream_t st = g_noalloc_stream[dev];
  // carve the scratch with the capacity as stride, so every sub-array stays naturally aligned
  char* d = static_cast<char*>(g_noalloc_ptr[dev]);
  const size_t cap = BLINK_SAMPLE_NOALLOC_MAX_ROWS, n = (size_t)rows;
  unsigned long long* d_ticket = reinterpret_cast<unsigned long long*>(d);
  unsigned long long* d_seed = d_ticket + cap;
  int* d_topk = reinterpret_cast<int*>(d_seed + cap);
  float* d_temp = reinterpret_cast<float*>(d_topk + cap);
  int* d_gen = reinterpret_cast<int*>(d_temp + cap);
  int* d_out = d_gen + cap;
  if (cudaMemcpyAsync(d_ticket, ticket, n * 8, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(d_seed, seed, n * 8, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(d_topk, top_k, n * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(d_temp, temperature, n * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(d_gen, gen_index, n * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemsetAsync(d_out, 0xff, n * 4, st) != cudaSuccess)  // results of an earlier call must not show through
    return BLINK_ECUDA;
  const int grid = rows < 1184 ? rows : 1184;
  blink_sample_kernel<<<grid, FWD_THREADS, SAMPLE_SMEM_FLOATS * sizeof(float), st>>>(logits, rows, vocab, d_topk, d_temp,
                                                                                     d_ticket, d_gen, d_seed, d_out, nullptr);
  if (cudaGetLastError() != cudaSuccess) return BLINK_ECUDA;
  if (cudaMemcpyAsync(out, d_out, n * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return BLINK_ECUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return BLINK_ECUDA;
  return BLINK_OK;
}

int blink_create(const blink_model_cfg* model, const blink_sched_cfg* sched, const blink_kv_pool* kv,
                 blink_ctx** out) {
  if (!out) return BLINK_EINVAL;
  *out = nullptr;
  if (!model_ok(model) || !sched || sched->size != sizeof(blink_sched_cfg) || !kv || kv->size != sizeof(blink_kv_pool))
    return BLINK_EINVAL;
  if (sched->max_batch < 1 || sched->max_batch > MAX_BATCH || sched->prefill_chunk_tokens < 1 || sched->n_slots < 1 ||
      sched->max_prompt < 1 || sched->max_new < 1 || sched->wait_limit_ms < 0)
    return BLINK_EINVAL;
  if (kv->block_size != 16) return BLINK_EINVAL;
  if (!sched->control_only && (model->weights == nullptr || model->weights_bytes < blink_weights_bytes(model)))
    return BLINK_EINVAL;
  if (model->n_experts > MAX_EXPERTS) return BLINK_EINVAL;
  if (((uintptr_t)kv->base & 255) || ((uintptr_t)model->weights & 255)) return BLINK_EINVAL;
  int dev_count = 0;
  if (cudaGetDeviceCount(&dev_count) != cudaSuccess || dev_count < 1) return BLINK_ECUDA;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return BLINK_ECUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return BLINK_ECUDA;
  if (prop.major != 10) {
    fprintf(stderr, "blink: built for sm_100a, device is sm_%d%d\n", prop.major, prop.minor);
    return BLINK_ECUDA;
  }
  const int64_t nb = blink_kv_blocks_for_bytes(model, kv->block_size, kv->bytes);
  if (nb < 1 || (!sched->control_only && kv->base == nullptr)) return BLINK_ENOMEM;

  blink_ctx* x = new (std::nothrow) blink_ctx();
  if (!x) return BLINK_ENOMEM;
  x->model = *model;
  x->sched = *sched;
  x->n_sms = prop.multiProcessorCount;
  DevCtx& c = x->dc;
  memset(&c, 0, sizeof(c));
  c.L = model->n_layers; c.d = model->d_model; c.Hq = model->n_q_heads; c.Hkv = model->n_kv_heads;
  c.hd = model->head_dim; c.F = model->d_ff; c.V = model->vocab; c.E = model->n_experts; c.topE = model->top_k_experts;
  c.dtype = model->dtype;
  c.q_dim = c.Hq * c.hd; c.kv_dim = c.Hkv * c.hd; c.qkv_dim = c.q_dim + 2 * c.kv_dim; c.n_rep = c.Hq / c.Hkv;
  c.rope_theta = model->rope_theta; c.rms_eps = model->rms_eps; c.attn_scale = 1.0f / sqrtf((float)c.hd);
  c.w_base = reinterpret_cast<const char*>(model->weights);
  const Layout lo = weight_layout(model);
  for (int i = 0; i < 10; ++i) c.w_off[i] = lo.off[i];
  c.MB = sched->max_batch; c.chunk = sched->prefill_chunk_tokens; c.n_slots = sched->n_slots;
  c.max_prompt = sched->max_prompt; c.max_new = sched->max_new; c.Tmax = c.MB + c.chunk; c.bs = kv->block_size;
  c.n_blocks = (int)(nb > 0x7fffffff ? 0x7fffffff : nb);
  c.max_pos = c.max_prompt + c.max_new;
  c.max_blocks_seq = (c.max_pos + c.bs - 1) / c.bs;
  c.control_only = sched->control_only; c.start_paused = sched->start_paused;
  if (sched->exec_mode < BLINK_EXEC_PERSISTENT || sched->exec_mode > BLINK_EXEC_HOST_LAUNCHES) { delete x; return BLINK_EINVAL; }
  x->host_driven = sched->exec_mode >= BLINK_EXEC_HOST_GRAPH ? sched->exec_mode : 0;
  x->device = dev;
  c.stepped = sched->exec_mode == BLINK_EXEC_STEPPED || x->host_driven != 0;
  x->manual = sched->exec_mode == BLINK_EXEC_MANUAL;
  c.gemm_tc = 0;
  if (!c.control_only && model->dtype == BLINK_DTYPE_BF16 && sched->gemm_impl != BLINK_GEMM_SIMT)
    c.gemm_tc = tc_available() && tc_shape_ok(c);
  if ((sched->gemm_impl == BLINK_GEMM_TC || sched->gemm_impl == BLINK_GEMM_TC_PAIR) && !c.gemm_tc) { delete x; return BLINK_EINVAL; }
  if (sched->gemm_impl < BLINK_GEMM_AUTO || sched->gemm_impl > BLINK_GEMM_TC_PAIR) { delete x; return BLINK_EINVAL; }
  // CTA pairs: built for four query heads per kv head, need an even grid and separate element-wise phases
  const bool pair_ok = c.gemm_tc && c.n_rep == 4 && !(x->n_sms & 1) && sched->epilogue_fusion != BLINK_FUSION_ON;
  if (sched->gemm_impl == BLINK_GEMM_TC_PAIR && !pair_ok) { delete x; return BLINK_EINVAL; }
  x->pair = pair_ok && (sched->gemm_impl == BLINK_GEMM_TC_PAIR || sched->gemm_impl == BLINK_GEMM_AUTO);   // measured faster
  // epilogue fusion needs whole 128-feature tiles that do not straddle q|k|v or gate|up
  if (sched->policy != BLINK_POLICY_CHUNKED && sched->policy != BLINK_POLICY_PAUSE_RESUME) { delete x; return BLINK_EINVAL; }
  if (sched->policy == BLINK_POLICY_PAUSE_RESUME && sched->prefill_chunk_tokens < sched->max_prompt) { delete x; return BLINK_EINVAL; }
  c.policy = sched->policy;
  if (sched->epilogue_fusion < BLINK_FUSION_AUTO || sched->epilogue_fusion > BLINK_FUSION_ON) { delete x; return BLINK_EINVAL; }
  c.fused = sched->epilogue_fusion == BLINK_FUSION_ON && c.gemm_tc && c.qkv_dim % 128 == 0 && c.q_dim % 128 == 0 && c.kv_dim % 128 == 0 && c.F % 128 == 0 &&
            c.d % 128 == 0 && 128 % c.hd == 0;
  c.fused_norm = c.fused && c.E == 0;
  c.w_streaming = model->weights_layout == BLINK_WEIGHTS_STREAMING;
  if (model->weights_layout != BLINK_WEIGHTS_ROW_MAJOR && model->weights_layout != BLINK_WEIGHTS_STREAMING) { delete x; return BLINK_EINVAL; }
  // the streaming layout is read by the tensor-core path only
  if (c.w_streaming && !c.control_only && (!c.gemm_tc || !tc_streaming_ok(c))) { delete x; return BLINK_EINVAL; }
  c.iteration_budget = c.stepped ? 0 : sched->iteration_budget;
  const double cyc_per_us = 2000.0;  // upper bound on the SM clock: time-outs only get longer at lower clocks
  const int64_t idle_us = sched->idle_exit_us > 0 ? sched->idle_exit_us : 2000000;
  c.idle_exit_cycles = (unsigned long long)(idle_us * cyc_per_us);
  c.barrier_timeout_cycles = sched->wait_limit_ms > 0 ? (unsigned long long)(sched->wait_limit_ms * 1000.0 * cyc_per_us)
                                                      : (unsigned long long)((idle_us + 3000000) * cyc_per_us);
  c.kv_base = kv->base;
  c.trace_cap = sched->trace_capacity_words;
  c.stats_cap = sched->stats_capacity_iters;
  c.logits_capture = sched->logits_capture;
  c.capture_rows = sched->logits_capture ? sched->logits_capture_rows : 0;

  int rc = BLINK_OK;
  auto fail = [&](int code) { free_all(x); delete x; return code; };
  if (cudaStreamCreateWithFlags(&x->stream, cudaStreamNonBlocking) != cudaSuccess) return fail(BLINK_ECUDA);
  if (cudaStreamCreateWithFlags(&x->copy_stream, cudaStreamNonBlocking) != cudaSuccess) return fail(BLINK_ECUDA);

#define TRY(expr) do { rc = (expr); if (rc != BLINK_OK) return fail(rc); } while (0)
  const size_t S = c.n_slots, MB = c.MB, TM = c.Tmax;
  const size_t esz = c.dtype == BLINK_DTYPE_BF16 ? 2 : 4;
  TRY(dev_alloc(x, &c.slot_hot, S));
  TRY(dev_alloc(x, &c.slot_cold, S));
  TRY(dev_alloc(x, &c.in_arena, S * c.max_prompt, false));
  TRY(dev_alloc(x, &c.gen_arena, S * c.max_new, false));
  TRY(dev_alloc(x, &c.forced_arena, S * c.max_new, false));
  TRY(dev_alloc(x, &c.ss, 1));
  TRY(dev_alloc(x, &c.ticket_to_slot, S));
  TRY(dev_alloc(x, &c.free_stack, (size_t)c.n_blocks, false));
  TRY(dev_alloc(x, &c.block_table, MB * c.max_blocks_seq));
  TRY(dev_alloc(x, &c.b_ticket, MB)); TRY(dev_alloc(x, &c.b_slot, MB)); TRY(dev_alloc(x, &c.b_P, MB));
  TRY(dev_alloc(x, &c.b_N, MB)); TRY(dev_alloc(x, &c.b_prefilled, MB)); TRY(dev_alloc(x, &c.b_generated, MB));
  TRY(dev_alloc(x, &c.b_phase, MB)); TRY(dev_alloc(x, &c.b_have, MB)); TRY(dev_alloc(x, &c.b_need, MB));
  TRY(dev_alloc(x, &c.b_last, MB)); TRY(dev_alloc(x, &c.b_eos, MB)); TRY(dev_alloc(x, &c.b_topk, MB));
  TRY(dev_alloc(x, &c.b_flags, MB)); TRY(dev_alloc(x, &c.b_temp, MB)); TRY(dev_alloc(x, &c.b_topp, MB)); TRY(dev_alloc(x, &c.b_seed, MB));
  TRY(dev_alloc(x, &c.it_bslot, MB)); TRY(dev_alloc(x, &c.it_start, MB)); TRY(dev_alloc(x, &c.it_ntok, MB));
  TRY(dev_alloc(x, &c.it_qstart, MB)); TRY(dev_alloc(x, &c.it_row, MB));
  TRY(dev_alloc(x, &c.tok_id, TM)); TRY(dev_alloc(x, &c.tok_pos, TM)); TRY(dev_alloc(x, &c.tok_item, TM));
  TRY(dev_alloc(x, &c.tok_slotmap, TM));
  TRY(dev_alloc(x, &c.row_tok, MB)); TRY(dev_alloc(x, &c.row_item, MB)); TRY(dev_alloc(x, &c.row_sampled, MB));
  if (!c.control_only) {
    char* p;
    TRY(dev_alloc(x, &c.h, TM * c.d));
    TRY(dev_alloc(x, &p, TM * c.d * esz)); c.xn = p;
    TRY(dev_alloc(x, &c.qkv, TM * c.qkv_dim));
    if (c.dtype == BLINK_DTYPE_BF16) {
      TRY(dev_alloc(x, &p, TM * c.q_dim * esz)); c.qb = p;
      c.n_warps_grid = x->n_sms * (FWD_THREADS / 32);
      c.att_sub_max = 2ll * c.n_warps_grid + (long long)MB * c.Hkv * c.max_blocks_seq / 24 + 8;
      TRY(dev_alloc(x, &c.dec_row, MB)); TRY(dev_alloc(x, &c.dec_bslot, MB)); TRY(dev_alloc(x, &c.dec_nctx, MB));
      TRY(dev_alloc(x, &c.dec_kbpre, MB + 1));
      TRY(dev_alloc(x, &c.pf_item, TM / 16 + MB + 1)); TRY(dev_alloc(x, &c.pf_qb, TM / 16 + MB + 1));
      TRY(dev_alloc(x, &c.att_ctr, (size_t)c.L)); TRY(dev_alloc(x, &c.att_cnt, MB * c.Hkv));
      {  // the KV pool as a rank-5 tensor {64 dims, hd/64 halves, n_blocks*Hkv*16 keys, K|V, L}; one box = the
         // K and V tiles of a (layer, block, kv head): {64, hd/64, 16, 2, 1}, 128-byte swizzle
        EncodeTiledFn enc = tc_encode_fn();
        const uint64_t rows = (uint64_t)c.n_blocks * c.Hkv * 16, rb = (uint64_t)c.hd * 2;
        if (!enc || rows > 0x7fffffffull) return fail(BLINK_EINVAL);
        CUtensorMap hm;
        cuuint64_t dims[5] = {64, (cuuint64_t)(c.hd / 64), rows, 2, (cuuint64_t)c.L};
        cuuint64_t strides[4] = {128, rb, rows * rb, 2 * rows * rb};
        cuuint32_t box[5] = {64, (cuuint32_t)(c.hd / 64), 16, 2, 1};
        cuuint32_t estr[5] = {1, 1, 1, 1, 1};
        if (enc(&hm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, c.kv_base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
          return fail(BLINK_ECUDA);
        void* dm = nullptr;
        TRY(dev_alloc(x, reinterpret_cast<char**>(&dm), sizeof(CUtensorMap), false));
        if (cudaMemcpy(dm, &hm, sizeof(CUtensorMap), cudaMemcpyHostToDevice) != cudaSuccess) return fail(BLINK_ECUDA);
        c.kv_map = dm;
      }
      TRY(dev_alloc(x, &c.att_part, (size_t)(2 * c.att_sub_max) * (c.n_rep * c.hd + ((2 * c.n_rep + 3) & ~3)), false));
    }
    TRY(dev_alloc(x, &p, TM * c.q_dim * esz)); c.attn = p;
    const size_t RA = TM * (c.E > 0 ? (size_t)c.topE : 1);   // routed experts: one FFN row per (token, expert)
    TRY(dev_alloc(x, &c.gu, RA * 2 * c.F));
    TRY(dev_alloc(x, &p, RA * c.F * esz)); c.act = p;
    if (c.E > 0) {
      TRY(dev_alloc(x, &p, RA * c.d * esz)); c.xg = p;
      TRY(dev_alloc(x, &c.moe_sel, RA)); TRY(dev_alloc(x, &c.moe_wt, RA)); TRY(dev_alloc(x, &c.moe_off, (size_t)c.E + 1));
      TRY(dev_alloc(x, &c.moe_tok, RA)); TRY(dev_alloc(x, &c.moe_gate, RA));
    }
    TRY(dev_alloc(x, &p, MB * c.d * esz)); c.xs = p;
    TRY(dev_alloc(x, &c.rowss_a, TM)); TRY(dev_alloc(x, &c.rowss_b, TM)); TRY(dev_alloc(x, &c.tile_cnt, (size_t)TILE_CNT_SLOTS));
    // one stamp per (256-row token pass, gate/up weight tile); the SwiGLU phase lists the units in shared memory
    const size_t gu_units = ((TM + 255) / 256) * (size_t)((c.F + 63) / 64);
    c.gu_direct = c.w_streaming && c.gemm_tc && c.E == 0 && !c.fused && gu_units <= 32768;
    TRY(dev_alloc(x, &c.gu_done, gu_units));
    TRY(dev_alloc(x, &c.logits, MB * c.V));
    TRY(dev_alloc(x, &c.rope_cos, (size_t)c.max_pos * (c.hd / 2), false));
    TRY(dev_alloc(x, &c.rope_sin, (size_t)c.max_pos * (c.hd / 2), false));
    std::vector<float> cs((size_t)c.max_pos * (c.hd / 2)), sn(cs.size());
    for (int i = 0; i < c.hd / 2; ++i) {
      const double inv = std::pow((double)c.rope_theta, -2.0 * i / c.hd);
      for (int p2 = 0; p2 < c.max_pos; ++p2) {
        cs[(size_t)p2 * (c.hd / 2) + i] = (float)std::cos(p2 * inv);
        sn[(size_t)p2 * (c.hd / 2) + i] = (float)std::sin(p2 * inv);
      }
    }
    if (cudaMemcpy(c.rope_cos, cs.data(), cs.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess) return fail(BLINK_ECUDA);
    if (cudaMemcpy(c.rope_sin, sn.data(), sn.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess) return fail(BLINK_ECUDA);
  }
  if (c.trace_cap > 0) TRY(dev_alloc(x, &c.trace, (size_t)c.trace_cap, false));
  if (c.stats_cap > 0) TRY(dev_alloc(x, &c.stats, (size_t)c.stats_cap));
  // free stack: pop takes from the top; first pops return 0, 1, 2, ...
  {
    std::vector<int32_t> st((size_t)c.n_blocks);
    for (int i = 0; i < c.n_blocks; ++i) st[(size_t)c.n_blocks - 1 - i] = i;
    if (cudaMemcpy(c.free_stack, st.data(), st.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess) return fail(BLINK_ECUDA);
    SchedState s0;
    memset(&s0, 0, sizeof(s0));
    s0.free_top = c.n_blocks;
    s0.cur_hdr = -1;
    if (cudaMemcpy(c.ss, &s0, sizeof(s0), cudaMemcpyHostToDevice) != cudaSuccess) return fail(BLINK_ECUDA);
  }
  // pinned mailboxes
  {
    Mailbox* md; SubEntry* qd; int32_t *td, *fd, *od; uint64_t* tmd; uint32_t* cd;
    TRY(pinned_alloc(x, &x->mbox, &md, 1)); c.mbox = md;
    TRY(pinned_alloc(x, &x->sub_q, &qd, S)); c.sub_q = qd;
    TRY(pinned_alloc(x, &x->sub_tokens, &td, S * c.max_prompt)); c.sub_tokens = td;
    TRY(pinned_alloc(x, &x->sub_forced, &fd, S * c.max_new)); c.sub_forced = fd;
    TRY(pinned_alloc(x, &x->out_tokens, &od, S * c.max_new)); c.out_tokens = od;
    TRY(pinned_alloc(x, &x->out_time, &tmd, S * c.max_new)); c.out_time = tmd;
    TRY(pinned_alloc(x, &x->out_count, &cd, S)); c.out_count = cd;
    { uint32_t* cn; TRY(pinned_alloc(x, &x->cancel, &cn, S)); c.cancel = cn; }
  }
  if (c.gemm_tc) TRY(tc_host_setup(x->tc_host, c));
#undef TRY
  x->slots.resize(S);

  // clock calibration: host CLOCK_MONOTONIC vs device global timer
  {
    const uint64_t t0 = now_ns();
    blink_clock_probe_kernel<<<1, 1, 0, x->stream>>>(c.mbox);
    if (cudaStreamSynchronize(x->stream) != cudaSuccess) return fail(BLINK_ECUDA);
    const uint64_t t1 = now_ns();
    x->clock_offset = (int64_t)((t0 + t1) / 2) - (int64_t)x->mbox->clock_probe;
  }

  x->smem_bytes = phase_smem_bytes(x);
  x->grid = c.control_only ? 1 : x->n_sms;
  auto pick_kernels = [&]() {
    x->ks = c.dtype == BLINK_DTYPE_BF16 ? (c.hd == 64 ? kernels_bf16_hd64(c.n_rep, x->pair) : kernels_bf16_hd128(c.n_rep, x->pair))
                                        : (c.hd == 64 ? kernels_fp32_hd64(c.n_rep, false) : kernels_fp32_hd128(c.n_rep, false));
  };
  pick_kernels();
  if (x->pair) {   // every cluster of two must be resident at once (the loop's grid barrier needs the whole grid)
    bool fits = x->ks.loop != nullptr;
    if (fits) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(x->grid); cfg.blockDim = dim3(FWD_THREADS); cfg.dynamicSmemBytes = x->smem_bytes;
      cudaLaunchAttribute at[1];
      at[0].id = cudaLaunchAttributeClusterDimension; at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
      cfg.attrs = at; cfg.numAttrs = 1;
      int ncl = 0;
      fits = cudaFuncSetAttribute(x->ks.loop, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)x->smem_bytes) == cudaSuccess &&
             cudaOccupancyMaxActiveClusters(&ncl, x->ks.loop, &cfg) == cudaSuccess && 2 * ncl >= x->grid;
    }
    if (!fits) {
      if (sched->gemm_impl == BLINK_GEMM_TC_PAIR) return fail(BLINK_EINVAL);
      x->pair = false;   // chosen automatically: fall back to single CTAs
      pick_kernels();
    }
  }
  const void* loop_fn = x->ks.loop;
  const void* ph_fn = x->ks.phase;
  if (!loop_fn || !ph_fn) return fail(BLINK_EINVAL);
  if (cudaFuncSetAttribute(loop_fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)x->smem_bytes) != cudaSuccess ||
      cudaFuncSetAttribute(ph_fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)x->smem_bytes) != cudaSuccess)
    return fail(BLINK_ECUDA);
  int occ = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, loop_fn, FWD_THREADS, x->smem_bytes) != cudaSuccess || occ < 1)
    return fail(BLINK_ECUDA);
  if (cudaDeviceSynchronize() != cudaSuccess) return fail(BLINK_ECUDA);
  if (!c.stepped && !x->manual) {
    rc = launch_loop(x);
    if (rc != BLINK_OK) return fail(rc);
  } else {
    x->mbox->loop_state = BLINK_LOOP_NOT_STARTED;
  }
  if (x->host_driven == BLINK_EXEC_HOST_GRAPH) {
    // one iteration (control plane + every phase) captured once: shapes come from device metadata, so the
    // same graph serves every step
    cudaGraph_t g = nullptr;
    if (cudaStreamBeginCapture(x->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) return fail(BLINK_ECUDA);
    const int src = step_once(x);
    if (cudaStreamEndCapture(x->stream, &g) != cudaSuccess || src != BLINK_OK || g == nullptr) return fail(BLINK_ECUDA);
    const cudaError_t ie = cudaGraphInstantiate(&x->iter_graph, g, 0);
    cudaGraphDestroy(g);
    if (ie != cudaSuccess) return fail(BLINK_ECUDA);
    x->launches = 0;
  }
  *out = x;
  if (x->host_driven && !c.start_paused) driver_start(x);
  return BLINK_OK;
}

int blink_start(blink_ctx* x) {
  if (!x) return BLINK_EINVAL;
  {
    std::lock_guard<std::mutex> g(x->mu);
    std::atomic_thread_fence(std::memory_order_seq_cst);
    x->mbox->start = 1;
    if (!x->host_driven) return pump(x) == BLINK_EDEVICE ? BLINK_EDEVICE : BLINK_OK;
  }
  driver_start(x);
  return x->driver_error.load() != 0 ? x->driver_error.load() : BLINK_OK;
}

int blink_submit(blink_ctx* x, const blink_request* r, uint64_t* ticket_out) {
  if (!x || !r || r->size != sizeof(blink_request) || !r->prompt) return BLINK_EINVAL;
  const DevCtx& c = x->dc;
  if (r->n_prompt < 1 || r->n_prompt > c.max_prompt || r->max_new_tokens < 1 || r->max_new_tokens > c.max_new)
    return BLINK_EINVAL;
  if (!(r->top_p >= 0.f)) return BLINK_EINVAL;
  const bool nucleus = r->top_p > 0.f && r->top_p < 1.f;
  if (r->top_k < 0 || r->top_k > MAX_TOPK || ((r->top_k > 0 || nucleus) && !(r->temperature > 0.f))) return BLINK_EINVAL;
  if (r->eos_id >= c.V) return BLINK_EINVAL;
  for (int i = 0; i < r->n_prompt; ++i)
    if (r->prompt[i] < 0 || r->prompt[i] >= c.V) return BLINK_EINVAL;
  if (r->forced_tokens)
    for (int i = 0; i < r->max_new_tokens; ++i)
      if (r->forced_tokens[i] < 0 || r->forced_tokens[i] >= c.V) return BLINK_EINVAL;
  const long long need = ((long long)r->n_prompt + r->max_new_tokens - 1 + c.bs - 1) / c.bs;
  if (need > c.n_blocks) return BLINK_EINVAL;  // could never be admitted: would block the queue for good

  std::lock_guard<std::mutex> g(x->mu);
  if (x->final_stop) return BLINK_ESTOPPED;
  if (x->mbox->loop_state == BLINK_LOOP_EXIT_ERROR || x->mbox->device_status > 0) {
    if (x->mbox->device_status != DEV_ERR_TRACE_OVERFLOW) return BLINK_EDEVICE;
  }
  // slot tracker: circular scan from a hint over the local availability cache
  int slot = -1;
  for (int k = 0; k < c.n_slots; ++k) {
    const int s = (x->hint + k) % c.n_slots;
    if (!x->slots[s].busy) { slot = s; break; }
  }
  if (slot < 0) return BLINK_EAGAIN;
  x->hint = (slot + 1) % c.n_slots;
  const uint64_t ticket = x->next_ticket++;
  memcpy(x->sub_tokens + (size_t)slot * c.max_prompt, r->prompt, (size_t)r->n_prompt * 4);
  if (r->forced_tokens) memcpy(x->sub_forced + (size_t)slot * c.max_new, r->forced_tokens, (size_t)r->max_new_tokens * 4);
  x->out_count[slot] = 0;
  x->cancel[slot] = 0;
  SubEntry& e = x->sub_q[ticket % (uint64_t)c.n_slots];
  e.ticket = ticket; e.seed = r->seed; e.user_tag = r->user_tag; e.slot = (uint32_t)slot;
  e.n_prompt = (uint32_t)r->n_prompt; e.max_new = (uint32_t)r->max_new_tokens; e.top_k = (uint32_t)r->top_k;
  e.temperature = r->temperature; e.eos_id = r->eos_id; e.flags = r->forced_tokens ? REQ_FLAG_FORCED : 0; e.top_p = r->top_p;
  SlotInfo& si = x->slots[slot];
  si.busy = true; si.ticket = ticket; si.user_tag = r->user_tag; si.max_new = r->max_new_tokens; si.consumed = 0;
  si.t_submit_ns = now_ns();
  x->bytes_to_device += (int64_t)sizeof(SubEntry) + 8 + (int64_t)r->n_prompt * 4 + (r->forced_tokens ? (int64_t)r->max_new_tokens * 4 : 0);
  x->active.push_front(slot);  // new slots are looked at first by the token reader
  // payload first, then the tail that makes it visible
  std::atomic_thread_fence(std::memory_order_release);
  __atomic_store_n((uint64_t*)&x->mbox->sub_tail, ticket + 1, __ATOMIC_RELEASE);
  if (ticket_out) *ticket_out = ticket;
  const int prc = pump(x);
  return prc == BLINK_EDEVICE ? BLINK_EDEVICE : BLINK_OK;
}

int blink_poll(blink_ctx* x, blink_token_event* out, int max_events, int timeout_us) {
  if (!x || !out || max_events < 1) return BLINK_EINVAL;
  const DevCtx& c = x->dc;
  const uint64_t deadline = now_ns() + (uint64_t)(timeout_us > 0 ? timeout_us : 0) * 1000ull;
  while (true) {
    int n = 0;
    {
      std::lock_guard<std::mutex> g(x->mu);
      const int prc = pump(x);
      if (prc == BLINK_EDEVICE) return BLINK_EDEVICE;
      const uint64_t t_now = now_ns();
      for (auto it = x->active.begin(); it != x->active.end() && n < max_events;) {
        const int slot = *it;
        SlotInfo& si = x->slots[slot];
        const uint32_t cnt = __atomic_load_n(&x->out_count[slot], __ATOMIC_ACQUIRE);
        const int have = (int)(cnt & 0x3fffffffu);
        const bool fin = (cnt >> 31) != 0;
        const bool cancelled = (cnt & 0x40000000u) != 0;
        while (si.consumed < have && n < max_events) {
          blink_token_event& ev = out[n++];
          const size_t idx = (size_t)slot * c.max_new + si.consumed;
          ev.ticket = si.ticket; ev.user_tag = si.user_tag; ev.index = si.consumed;
          ev.token = x->out_tokens[idx];
          ev.is_first = si.consumed == 0;
          ev.is_last = fin && !cancelled && si.consumed + 1 == have;
          ev.t_device_ns = x->out_time[idx];
          ev.t_host_ns = t_now;
          ev.t_submit_ns = si.t_submit_ns;
          si.consumed += 1;
          x->bytes_from_device += 16;   // what the device wrote into the host mirrors for it: token, timestamp, count word
        }
        if (fin && cancelled && si.consumed == have) {
          if (n >= max_events) { ++it; continue; }   // no room for the closing event in this call
          blink_token_event& ev = out[n++];           // a cancelled request ends with an event of its own
          ev.ticket = si.ticket; ev.user_tag = si.user_tag; ev.index = have; ev.token = -1;
          ev.is_first = 0; ev.is_last = 1; ev.t_device_ns = 0; ev.t_host_ns = t_now; ev.t_submit_ns = si.t_submit_ns;
        }
        if (fin && si.consumed == have) {
          si.busy = false;  // DECODE_COMPLETED -> EMPTY: the frontend owns this transition
          it = x->active.erase(it);
        } else {
          ++it;
        }
      }
    }
    if (n > 0 || now_ns() >= deadline) return n;
    std::this_thread::sleep_for(std::chrono::microseconds(20));
  }
}

int blink_cancel(blink_ctx* x, uint64_t ticket) {
  if (!x) return BLINK_EINVAL;
  std::lock_guard<std::mutex> g(x->mu);
  for (int slot : x->active) {
    SlotInfo& si = x->slots[slot];
    if (si.busy && si.ticket == ticket) {
      __atomic_store_n(&x->cancel[slot], 1u, __ATOMIC_RELEASE);
      return BLINK_OK;
    }
  }
  return BLINK_EINVAL;   // unknown, or all of its tokens have been handed out already
}

int blink_step(blink_ctx* x, int n_iterations) {
  if (!x || n_iterations < 0) return BLINK_EINVAL;
  if (!x->dc.stepped || x->host_driven) return BLINK_EINVAL;
  std::lock_guard<std::mutex> g(x->mu);
  for (int i = 0; i < n_iterations; ++i) {
    const int rc = step_once(x);
    if (rc != BLINK_OK) return rc;
  }
  blink_control_kernel<<<1, CTRL_THREADS, 0, x->stream>>>(x->dc, 1);
  x->launches += 1;
  if (cudaStreamSynchronize(x->stream) != cudaSuccess) return BLINK_ECUDA;
  return x->mbox->device_status > 0 && x->mbox->device_status != DEV_ERR_TRACE_OVERFLOW ? BLINK_EDEVICE : BLINK_OK;
}

int blink_run(blink_ctx* x, int64_t n_iterations, float* elapsed_ms) {
  if (!x || n_iterations < 1) return BLINK_EINVAL;
  if (!x->manual) return BLINK_EINVAL;
  std::lock_guard<std::mutex> g(x->mu);
  if (x->final_stop) return BLINK_ESTOPPED;
  if (x->mbox->device_status > 0 && x->mbox->device_status != DEV_ERR_TRACE_OVERFLOW) return BLINK_EDEVICE;
  if (!x->ev0 && (cudaEventCreate(&x->ev0) != cudaSuccess || cudaEventCreate(&x->ev1) != cudaSuccess)) return BLINK_ECUDA;
  x->dc.iteration_budget = n_iterations;
  if (cudaEventRecord(x->ev0, x->stream) != cudaSuccess) return BLINK_ECUDA;
  const int rc = launch_loop(x);
  if (rc != BLINK_OK) return rc;
  if (cudaEventRecord(x->ev1, x->stream) != cudaSuccess) return BLINK_ECUDA;
  if (cudaEventSynchronize(x->ev1) != cudaSuccess) return BLINK_ECUDA;
  float ms = 0.f;
  if (cudaEventElapsedTime(&ms, x->ev0, x->ev1) != cudaSuccess) return BLINK_ECUDA;
  if (elapsed_ms) *elapsed_ms = ms;
  return x->mbox->loop_state == BLINK_LOOP_EXIT_ERROR ? BLINK_EDEVICE : BLINK_OK;
}

int blink_stop(blink_ctx* x, int final, int timeout_ms) {
  if (!x) return BLINK_EINVAL;
  if (x->host_driven) driver_join(x);   // leaves between iterations; blink_start brings it back
  std::lock_guard<std::mutex> g(x->mu);
  if (final) x->final_stop = true;
  if (x->dc.stepped) return cudaStreamSynchronize(x->stream) == cudaSuccess ? BLINK_OK : BLINK_ECUDA;
  const uint64_t deadline = now_ns() + (uint64_t)(timeout_ms > 0 ? timeout_ms : 0) * 1000000ull;
  if (x->mbox->loop_state == BLINK_LOOP_RUNNING) {
    std::atomic_thread_fence(std::memory_order_seq_cst);
    x->mbox->stop = 1;
  }
  while (true) {
    const cudaError_t q = cudaStreamQuery(x->stream);
    if (q == cudaSuccess) break;
    if (q != cudaErrorNotReady) return BLINK_ECUDA;
    if (now_ns() >= deadline) return BLINK_ETIMEDOUT;
    std::this_thread::sleep_for(std::chrono::microseconds(50));
  }
  return BLINK_OK;
}

int blink_destroy(blink_ctx* x, int timeout_ms) {
  if (!x) return BLINK_EINVAL;
  const int rc = blink_stop(x, 1, timeout_ms);
  if (rc == BLINK_ETIMEDOUT) return rc;
  free_all(x);
  delete x;
  return rc == BLINK_ECUDA ? BLINK_ECUDA : BLINK_OK;
}

static int read_ss(blink_ctx* x, SchedState* s) {
  if (cudaMemcpyAsync(s, x->dc.ss, sizeof(SchedState), cudaMemcpyDeviceToHost, x->copy_stream) != cudaSuccess) return BLINK_ECUDA;
  if (cudaStreamSynchronize(x->copy_stream) != cudaSuccess) return BLINK_ECUDA;
  return BLINK_OK;
}

int blink_get_stats(blink_ctx* x, blink_stats* out) {
  if (!x || !out || out->size != sizeof(blink_stats)) return BLINK_EINVAL;
  std::lock_guard<std::mutex> g(x->mu);
  SchedState s;
  const int rc = read_ss(x, &s);
  if (rc != BLINK_OK) return rc;
  out->loop_state = (int32_t)x->mbox->loop_state;
  out->device_status = x->mbox->device_status;
  out->n_blocks = x->dc.n_blocks;
  out->iterations = (int64_t)s.iter;
  out->launches = x->launches;
  out->tokens_out = (int64_t)s.tokens_out;
  out->prompt_tokens = (int64_t)s.prompt_tokens;
  out->trace_words = s.trace_pos;
  out->device_clock_offset_ns = x->clock_offset;
  out->free_blocks = s.free_top;
  out->reserved_blocks = s.reserved;
  std::vector<int32_t> ph((size_t)x->dc.MB);
  if (cudaMemcpyAsync(ph.data(), x->dc.b_phase, ph.size() * 4, cudaMemcpyDeviceToHost, x->copy_stream) != cudaSuccess ||
      cudaStreamSynchronize(x->copy_stream) != cudaSuccess)
    return BLINK_ECUDA;
  int live = 0;
  for (int v : ph) live += v != PHASE_FREE;
  out->batch_live = live;
  out->reserved1 = 0;
  out->bytes_to_device = x->bytes_to_device;
  out->bytes_from_device = x->bytes_from_device;
  return BLINK_OK;
}

int blink_get_trace(blink_ctx* x, int32_t* out, int64_t capacity, int64_t* n_words) {
  if (!x || !n_words || capacity < 0 || (capacity > 0 && !out)) return BLINK_EINVAL;
  std::lock_guard<std::mutex> g(x->mu);
  SchedState s;
  const int rc = read_ss(x, &s);
  if (rc != BLINK_OK) return rc;
  *n_words = s.trace_pos;
  const int64_t n = s.trace_pos < capacity ? s.trace_pos : capacity;
  if (n > 0) {
    if (cudaMemcpyAsync(out, x->dc.trace, (size_t)n * 4, cudaMemcpyDeviceToHost, x->copy_stream) != cudaSuccess ||
        cudaStreamSynchronize(x->copy_stream) != cudaSuccess)
      return BLINK_ECUDA;
  }
  return BLINK_OK;
}

int blink_get_iter_stats(blink_ctx* x, blink_iter_stat* out, int64_t capacity, int64_t* n_records) {
  if (!x || !n_records || capacity < 0 || (capacity > 0 && !out)) return BLINK_EINVAL;
  static_assert(sizeof(blink_iter_stat) == sizeof(IterStat), "iter stat layout");
  std::lock_guard<std::mutex> g(x->mu);
  SchedState s;
  const int rc = read_ss(x, &s);
  if (rc != BLINK_OK) return rc;
  int64_t have = (int64_t)s.iter < x->dc.stats_cap ? (int64_t)s.iter : x->dc.stats_cap;
  *n_records = have;
  const int64_t n = have < capacity ? have : capacity;
  if (n > 0) {
    if (cudaMemcpyAsync(out, x->dc.stats, (size_t)n * sizeof(IterStat), cudaMemcpyDeviceToHost, x->copy_stream) != cudaSuccess ||
        cudaStreamSynchronize(x->copy_stream) != cudaSuccess)
      return BLINK_ECUDA;
  }
  return BLINK_OK;
}

}  // extern "C"
