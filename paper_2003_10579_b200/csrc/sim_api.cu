// C-ABI of the straggler-SGD simulator: handle, argument checks, memory, kernel dispatch.
// See include/straggler_sim.h for the contract of every entry point.
#include "../../include/straggler_sim.h"

#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "linear_kernel.cuh"
#include "softmax_kernel.cuh"
#include "softmax_ws_kernel.cuh"
#include "mlp_tc_kernel.cuh"
#include "eval_kernel.cuh"

using namespace ssim;

namespace {

thread_local std::string g_last_error;

struct TraceBuffers {
  double* t = nullptr;
  float* loss = nullptr;
  float* dist2 = nullptr;
  uint16_t* K_used = nullptr;
  uint16_t* worker = nullptr;
  uint32_t* stale = nullptr;
  uint32_t* seq = nullptr;
  uint8_t* snap_slot = nullptr;
  uint8_t* new_slot = nullptr;
};

}  // namespace

struct sim_handle {
  sim_problem prob{};
  int P = 0, K = 0, variant = 0, m = 0, R = 0;
  sim_delay delay{};
  float eta = 0.f;
  uint64_t seed = 0;
  uint32_t replica_base = 0;
  cudaStream_t stream = nullptr;
  int device = 0;
  int K0 = 0;
  double t_interval = 0.0;
  int K_stride = 0;
  bool is_async = false;
  bool uses_pool = false;     // parameters live in a version pool (asynchronous variants, and the MLP always)
  int n_slots = 0;
  long long n_params = 0;
  long long slot_stride = 0;  // floats between versions in the pool (16-byte aligned slots)
  long long n_updates = 0, cap = 0;
  int tune_stages = 0, tune_rows = 0, tune_threads = 0;
  // device state
  uint32_t* s = nullptr;
  uint32_t* tau = nullptr;
  double* f = nullptr;
  uint8_t* wslot = nullptr;
  uint8_t* cur_slot = nullptr;
  uint8_t* begin_slot = nullptr;
  double* clock = nullptr;
  float* w_state = nullptr;   // synchronous: [R][n_params]
  float* pool = nullptr;      // asynchronous: [R][n_slots][n_params]
  MlpScratch mlp{};
  MlpMaps mlp_maps{};
  int* err = nullptr;
  double* eval_partial = nullptr;   // [row blocks][R], made on the first sim_eval_loss
  // loss-driven K (Algorithm 1): per-replica progress and K, risks at w_0 and at the last pause
  bool ada_loss = false, F0_ready = false;
  float* F0 = nullptr; float* Fcur = nullptr;
  long long* done = nullptr; long long* run_j0 = nullptr; long long* run_iters = nullptr; long long* q_last = nullptr;
  int* K_cur = nullptr; int* want_eval = nullptr; int* remaining = nullptr;
  // full-data risk recorded inside sim_run: entry 0 is F(w_0), entry i the risk after i * eval_every updates
  long long eval_every = 0, n_evals = 0, risk_cap = 0;
  float* risk = nullptr;            // [risk_cap][R]
  float* mlp_eval_part = nullptr;   // MLP: per 32-row group partial loss sums of one evaluation
  TraceBuffers tr;
  bool poisoned = false;
  bool in_arena = false;      // buffers come from the creating thread's DeviceArena and are not freed one by one
  mutable std::string last_error;
};

namespace {

sim_status fail(const sim_handle* h, sim_status st, const std::string& msg) {
  if (h) h->last_error = msg; else g_last_error = msg;
  return st;
}

#define CUDA_TRY(h, expr)                                                                   \
  do {                                                                                      \
    cudaError_t e_ = (expr);                                                                \
    if (e_ != cudaSuccess)                                                                  \
      return fail(h, e_ == cudaErrorMemoryAllocation ? SIM_ERR_ALLOC : SIM_ERR_CUDA,       \
                  std::string(#expr) + ": " + cudaGetErrorString(e_));                      \
  } while (0)

// Device memory for many short-lived handles at once (sim_sweep_host): buffers are carved out of a few
// large chunks instead of one cudaMalloc / cudaFree each (a cudaFree waits for the whole device).  While
// a host thread has an arena installed, every handle it creates takes its buffers from it and frees
// none of them; the arena's owner releases the chunks after the handles are gone.
struct DeviceArena {
  std::vector<void*> chunks;
  char* cur = nullptr;
  size_t left = 0;
  cudaError_t take(void** p, size_t bytes) {
    bytes = (bytes + 255) & ~(size_t)255;
    if (bytes > left) {
      const size_t chunk = bytes > ((size_t)64 << 20) ? bytes : ((size_t)64 << 20);
      void* c = nullptr;
      const cudaError_t e = cudaMalloc(&c, chunk);
      if (e != cudaSuccess) return e;
      chunks.push_back(c);
      cur = static_cast<char*>(c);
      left = chunk;
    }
    *p = cur;
    cur += bytes;
    left -= bytes;
    return cudaSuccess;
  }
  void release() {
    for (void* c : chunks) cudaFree(c);
    chunks.clear(); cur = nullptr; left = 0;
  }
};
thread_local DeviceArena* t_arena = nullptr;

template <typename T>
cudaError_t dev_alloc(T** p, size_t count, cudaStream_t st, bool zero = true) {
  *p = nullptr;
  if (count == 0) return cudaSuccess;
  cudaError_t e = t_arena ? t_arena->take(reinterpret_cast<void**>(p), count * sizeof(T))
                          : cudaMalloc(reinterpret_cast<void**>(p), count * sizeof(T));
  if (e != cudaSuccess) { *p = nullptr; return e; }
  if (zero) e = cudaMemsetAsync(*p, 0, count * sizeof(T), st);
  return e;
}

long long model_params(const sim_problem& p) {
  switch (p.model) {
    case SIM_LSQ: case SIM_LOGISTIC: return p.d;
    case SIM_SOFTMAX: return (long long)p.n_classes * p.d;
    case SIM_MLP2: return (long long)p.d * p.hidden + p.hidden + (long long)p.hidden * p.n_classes + p.n_classes;
    default: return 0;
  }
}

sim_status check_delay(const sim_handle* h, const sim_delay& dl) {
  if (dl.kind != SIM_DELAY_EXP && dl.kind != SIM_DELAY_SHIFTED_EXP && dl.kind != SIM_DELAY_PARETO2)
    return fail(h, SIM_ERR_ARG, "unknown delay kind");
  if (dl.kind == SIM_DELAY_PARETO2) {
    if (dl.mu != 2.0) return fail(h, SIM_ERR_ARG, "the Pareto law is built for shape mu = 2 only");
    if (!(dl.shift > 0.0 && std::isfinite(dl.shift))) return fail(h, SIM_ERR_ARG, "the Pareto scale (shift) must be finite and > 0");
    return SIM_OK;
  }
  if (!(dl.mu > 0.0)) return fail(h, SIM_ERR_ARG, "delay rate mu must be > 0");
  if (dl.kind == SIM_DELAY_SHIFTED_EXP && !(dl.shift >= 0.0 && std::isfinite(dl.shift)))
    return fail(h, SIM_ERR_ARG, "delay shift must be finite and >= 0");
  return SIM_OK;
}

// tiled_dH / H: for the MLP the first tiled_dH parameters (W1) are stored block-tiled inside the pool
__global__ void broadcast_params_kernel(const float* w0, float* dst, long long n_params, long long stride, int R,
                                        long long tiled_dH, int H) {
  const long long total = n_params * R;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long r = i / n_params, p = i % n_params;
    const long long q = p < tiled_dH ? w1_tiled_index(p / H, p % H, H) : p;
    dst[r * stride + q] = w0[p];
  }
}

__global__ void gather_params_kernel(const float* pool, const uint8_t* cur_slot, float* out, long long n_params, long long slot_stride,
                                     int n_slots, int R, long long tiled_dH, int H) {
  const long long total = n_params * R;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long r = i / n_params, p = i % n_params;
    const long long q = p < tiled_dH ? w1_tiled_index(p / H, p % H, H) : p;
    out[i] = pool[(r * n_slots + cur_slot[r]) * slot_stride + q];
  }
}

template <typename T>
sim_status regrow(sim_handle* h, T** buf, size_t per_update, long long new_cap, bool zero) {
  T* nb = nullptr;
  CUDA_TRY(h, dev_alloc(&nb, (size_t)h->R * new_cap * per_update, h->stream, zero));
  if (*buf && h->n_updates > 0) {
    CUDA_TRY(h, cudaMemcpy2DAsync(nb, (size_t)new_cap * per_update * sizeof(T), *buf,
                                  (size_t)h->cap * per_update * sizeof(T),
                                  (size_t)h->n_updates * per_update * sizeof(T), h->R,
                                  cudaMemcpyDeviceToDevice, h->stream));
  }
  if (*buf && !h->in_arena) { CUDA_TRY(h, cudaStreamSynchronize(h->stream)); cudaFree(*buf); }
  *buf = nb;
  return SIM_OK;
}

sim_status ensure_capacity(sim_handle* h, long long need) {
  if (need <= h->cap) return SIM_OK;
  long long nc = h->cap * 2 > need ? h->cap * 2 : need;
  const size_t Ks = (size_t)h->K_stride;
  sim_status st;
  if ((st = regrow(h, &h->tr.t, 1, nc, false)) != SIM_OK) return st;
  if ((st = regrow(h, &h->tr.loss, 1, nc, true)) != SIM_OK) return st;
  if ((st = regrow(h, &h->tr.dist2, 1, nc, true)) != SIM_OK) return st;
  if ((st = regrow(h, &h->tr.K_used, 1, nc, false)) != SIM_OK) return st;
  if ((st = regrow(h, &h->tr.worker, Ks, nc, false)) != SIM_OK) return st;
  if ((st = regrow(h, &h->tr.stale, Ks, nc, false)) != SIM_OK) return st;
  if ((st = regrow(h, &h->tr.seq, Ks, nc, false)) != SIM_OK) return st;
  if (h->is_async) {
    if ((st = regrow(h, &h->tr.snap_slot, Ks, nc, false)) != SIM_OK) return st;
    if ((st = regrow(h, &h->tr.new_slot, 1, nc, false)) != SIM_OK) return st;
  }
  h->cap = nc;
  return SIM_OK;
}

// ---- dispatch of the single-output linear kernel by feature count ----
template <int NT, int CHUNKS, int T>
sim_status launch_linear1(sim_handle* h, NumericArgs& a) {
  const int d = a.d;
  const size_t row_bytes = (size_t)d * 4;
  int S = h->tune_stages;
  if (S <= 0) {
    if (a.R > 296) {
      // more than two replicas per SM: what counts is how many CTAs fit an SM, so two stages - more only while 32 CTAs
      // still fit (tiny rows).  Measured: 65536 replicas of 64 features 212 -> 306 M updates/s with three stages instead
      // of eight; rows of 2048 features 7.4 -> 7.7 TB/s with two stages instead of three.
      S = (int)(((size_t)7 << 10) / ((size_t)T * row_bytes));
    } else {
      // small rows: several CTAs per SM; long rows: one CTA per SM, or two when there are more replicas than SMs
      const size_t budget = d <= 1024 ? (36u << 10) : (a.R > 148 ? (100u << 10) : (200u << 10));
      S = (int)(budget / ((size_t)T * row_bytes));
    }
  }
  if (S < 2) S = 2;
  if (S > 8) S = 8;
  size_t smem = linear1_smem_bytes(NT, T, S, d, a.m);
  while (smem > (size_t)(226 << 10) && S > 2) { --S; smem = linear1_smem_bytes(NT, T, S, d, a.m); }
  if (smem > (size_t)(226 << 10))
    return fail(h, SIM_ERR_ARG, "the row staging buffers (d) and the minibatch index table (m) do not fit in shared memory with this tuning");
  a.stages = S;
  auto kern = a.is_async ? linear1_kernel<NT, CHUNKS, T, true> : linear1_kernel<NT, CHUNKS, T, false>;
  CUDA_TRY(h, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  kern<<<a.R, NT, smem, h->stream>>>(a);
  CUDA_TRY(h, cudaGetLastError());
  return SIM_OK;
}

sim_status run_linear1(sim_handle* h, NumericArgs& a) {
  const int d4 = a.d / 4;
  // up to 32 column chunks: with few replicas (at most two per SM the run is a chain of latencies) a second warp that only
  // produces overlaps drawing indices and issuing copies with the arithmetic; with many, one warp per replica packs better
  if (d4 <= 32 && a.R > 296) return launch_linear1<32, 1, 8>(h, a);
  if (d4 <= 64) return (a.R > 296 && !h->tune_rows && !h->tune_threads) ? launch_linear1<32, 2, 8>(h, a) : launch_linear1<64, 1, 8>(h, a);
  // With more than two replicas per SM narrow blocks with more column chunks a thread win (fewer warps meet at a tile's
  // barrier - none in a one-warp block - and more blocks fit an SM).  Measured with eight simulations of 1024 replicas on
  // concurrent streams, K = 8, m = 32: rows of 512 features 5.5 -> 7.1 TB/s, 1024 features 7.0 -> 8.1, 2048 features 6.2 -> 7.7.
  const bool many = a.R > 296 && !h->tune_rows && !h->tune_threads;
  if (d4 <= 128) {
    if (many && linear1_smem_bytes(32, 8, 2, a.d, a.m) <= (size_t)(226 << 10)) return launch_linear1<32, 4, 8>(h, a);
    return launch_linear1<128, 1, 4>(h, a);
  }
  if (d4 <= 256) {
    // one warp per replica with eight column chunks a thread: six such CTAs fit an SM (two 16 KB stages each) where five
    // of 128 threads did, and the K-sweep workload runs 15 % faster; with few replicas the wider block is quicker per replica
    if (many) return launch_linear1<32, 8, 4>(h, a);
    const int rows = h->tune_rows ? h->tune_rows : 4;
    if (h->tune_threads == 256) return rows == 8 ? launch_linear1<256, 1, 8>(h, a) : launch_linear1<256, 1, 4>(h, a);
    return rows == 8 ? launch_linear1<128, 2, 8>(h, a) : rows == 2 ? launch_linear1<128, 2, 2>(h, a) : launch_linear1<128, 2, 4>(h, a);
  }
  if (d4 <= 512) return many ? launch_linear1<64, 8, 4>(h, a) : launch_linear1<256, 2, 4>(h, a);
  if (d4 <= 1024) {
    const int rows = h->tune_rows ? h->tune_rows : (a.R > 148 ? 2 : 4), threads = h->tune_threads ? h->tune_threads : 256;
    if (threads == 512 && d4 <= 1024) return rows == 2 ? launch_linear1<512, 2, 2>(h, a) : launch_linear1<512, 2, 4>(h, a);
    // more than one replica per SM: four warps x eight chunks a thread (half as many warps meet at the tile's barrier;
    // the asynchronous logistic workload runs 7 % faster than with eight warps x four chunks)
    if (rows == 2) return h->tune_threads == 256 ? launch_linear1<256, 4, 2>(h, a) : launch_linear1<128, 8, 2>(h, a);
    return launch_linear1<256, 4, 4>(h, a);
  }
  if (d4 <= 2048) return launch_linear1<512, 4, 2>(h, a);
  return fail(h, SIM_ERR_ARG, "d > 8192 is not supported by the linear-model kernel");
}

// Shared memory the linear-model kernel needs at its smallest ring (two stages) with the tile shape the
// dispatch above picks for d when no tuning is set: rows of the ring plus the m-entry index table.
size_t linear1_min_smem(int d, int m, int R) {
  const int d4 = d / 4;
  int NT = 512, T = 2;
  if (d4 <= 64) { NT = 64; T = 8; }       // (a block of 32 threads needs no more)
  else if (d4 <= 128) { NT = 128; T = 4; }
  else if (d4 <= 256) { NT = 128; T = 4; }
  else if (d4 <= 512) { NT = 256; T = 4; }
  else if (d4 <= 1024) { NT = 256; T = R > 148 ? 2 : 4; }
  return linear1_smem_bytes(NT, T, 2, d, m);
}

sim_status device_error(const sim_handle* h) {
  int e = 0;
  CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  CUDA_TRY(h, cudaMemcpy(&e, h->err, sizeof(int), cudaMemcpyDeviceToHost));
  if (e == ERR_NONE) return SIM_OK;
  const_cast<sim_handle*>(h)->poisoned = true;
  if (e == ERR_WAIT_TIMEOUT) return fail(h, SIM_ERR_TIMEOUT, "a bounded device-side wait ran out");
  return fail(h, SIM_ERR_INTERNAL, "device-side consistency check failed (code " + std::to_string(e) + ")");
}

void free_all(sim_handle* h) {
  mlp_scratch_free(h->mlp);
  if (h->in_arena) return;          // the arena's owner frees the chunks
  cudaFree(h->s); cudaFree(h->tau); cudaFree(h->f); cudaFree(h->wslot); cudaFree(h->cur_slot);
  cudaFree(h->begin_slot); cudaFree(h->clock); cudaFree(h->w_state); cudaFree(h->pool); cudaFree(h->err);
  cudaFree(h->eval_partial); cudaFree(h->F0); cudaFree(h->Fcur); cudaFree(h->done); cudaFree(h->run_j0);
  cudaFree(h->run_iters); cudaFree(h->q_last); cudaFree(h->K_cur); cudaFree(h->want_eval); cudaFree(h->remaining);
  cudaFree(h->tr.t); cudaFree(h->tr.loss); cudaFree(h->tr.dist2); cudaFree(h->tr.K_used);
  cudaFree(h->tr.worker); cudaFree(h->tr.stale); cudaFree(h->tr.seq); cudaFree(h->tr.snap_slot);
  cudaFree(h->tr.new_slot); cudaFree(h->risk); cudaFree(h->mlp_eval_part);
}

// MLP: bf16 copy of the data, per-update scratch and the bf16 shadow of the initial W1, made on first use
cudaError_t ensure_mlp_scratch(sim_handle* h) {
  if (h->mlp.Xq) return cudaSuccess;
  cudaError_t ce = mlp_scratch_alloc(h->mlp, h->prob.X, h->prob.n, h->prob.d, h->prob.hidden, h->prob.n_classes, h->m,
                                     h->K_stride, h->R, h->n_slots, h->stream);
  if (ce == cudaSuccess) ce = mlp_after_set_params(h->mlp, h->pool, h->slot_stride, h->stream);
  return ce;
}

sim_status eval_into(sim_handle* h, float* loss) {
  const sim_model mdl = h->prob.model;
  if (mdl == SIM_MLP2) {
    // forward pass of the tensor-core kernel over the whole data set, every replica at its current version
    const int blocks = (int)((h->prob.n + 127) / 128);
    if (!h->mlp_eval_part) CUDA_TRY(h, dev_alloc(&h->mlp_eval_part, (size_t)h->R * blocks * 4, h->stream, false));
    CUDA_TRY(h, ensure_mlp_scratch(h));
    NumericArgs a{};
    a.X = h->prob.X; a.y = h->prob.label; a.n = (uint64_t)h->prob.n; a.d = h->prob.d; a.m = h->m; a.model = (int)mdl;
    a.n_classes = h->prob.n_classes; a.replica_base = h->replica_base; a.R = h->R; a.is_async = h->is_async ? 1 : 0;
    a.n_slots = h->n_slots; a.n_params = h->n_params; a.slot_stride = h->slot_stride; a.pool = h->pool; a.err = h->err;
    const char* why = nullptr;
    const cudaError_t ce = run_mlp_eval(a, h->mlp, h->mlp_maps, h->is_async ? h->cur_slot : nullptr, (int)(h->n_updates & 1),
                                        h->mlp_eval_part, loss, h->stream, &why);
    if (why) return fail(h, SIM_ERR_ARG, why);
    CUDA_TRY(h, ce);
    return SIM_OK;
  }
  if (mdl != SIM_LSQ && mdl != SIM_LOGISTIC && mdl != SIM_SOFTMAX)
    return fail(h, SIM_ERR_ARG, "the full-data risk needs a model (LSQ, logistic, softmax or the MLP)");
  EvalArgs e{};
  e.X = h->prob.X;
  e.y = mdl == SIM_LSQ ? static_cast<const void*>(h->prob.y) : static_cast<const void*>(h->prob.label);
  e.n = h->prob.n; e.d = h->prob.d; e.C = mdl == SIM_SOFTMAX ? h->prob.n_classes : 1; e.model = (int)mdl; e.R = h->R;
  e.RB = EV_BN / e.C;
  e.w_state = h->uses_pool ? nullptr : h->w_state;
  e.pool = h->uses_pool ? h->pool : nullptr;
  e.cur_slot = h->cur_slot; e.n_slots = h->n_slots; e.n_params = h->n_params; e.slot_stride = h->slot_stride;
  e.row_blocks = (int)((h->prob.n + EV_BM - 1) / EV_BM);
  if (!h->eval_partial) CUDA_TRY(h, dev_alloc(&h->eval_partial, (size_t)e.row_blocks * h->R, h->stream, false));
  e.partial = h->eval_partial; e.out = loss;
  dim3 grid((unsigned)e.row_blocks, (unsigned)((h->R + e.RB - 1) / e.RB));
  CUDA_TRY(h, cudaFuncSetAttribute(eval_loss_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)EV_SMEM_BYTES));
  eval_loss_kernel<<<grid, 256, EV_SMEM_BYTES, h->stream>>>(e);
  CUDA_TRY(h, cudaGetLastError());
  eval_loss_finish_kernel<<<(h->R + 127) / 128, 128, 0, h->stream>>>(e);
  CUDA_TRY(h, cudaGetLastError());
  return SIM_OK;
}

// Self-test of the timeout path: a wait on a barrier that nobody arrives at, with a limit of `limit` polls.  It runs out,
// the block votes on it and reports through the handle's error word - the steps a numeric kernel takes when one of
// its bounded waits gives up.  The kernel returns by itself; nothing is left waiting.
__global__ void wait_timeout_selftest_kernel(int* err, uint32_t limit) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) { mbar_init(smem_addr(&bar), 1); mbar_fence_init(); }
  __syncthreads();
  const bool ok = mbar_wait(smem_addr(&bar), 0u, limit);
  if (__syncthreads_or(!ok) && threadIdx.x == 0) atomicExch(err, ERR_WAIT_TIMEOUT);
}

// risk trace [evals][R] (as recorded) -> [R][evals] for the caller, with the clock of each evaluation: entry 0 is
// F(w_0) at time 0, entry i the risk after i * every updates, i.e. at the time recorded for update i * every - 1
__global__ void risk_trace_out_kernel(const float* risk, const double* t, long long cap, long long every, int R, long long E,
                                      float* risk_out, double* t_out) {
  const long long total = (long long)R * E;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long r = i / E, e = i % E;
    if (risk_out) risk_out[i] = risk[e * R + r];
    if (t_out) t_out[i] = e == 0 ? 0.0 : t[r * cap + e * every - 1];
  }
}

// Mean over replicas of F(w) - f_star at the replica's last evaluation completed by grid time g (one block per grid
// point, binary search over the evaluation times, fp64 tree sum in a fixed order).
__global__ void __launch_bounds__(256) risk_curve_kernel(const float* risk, const double* t, long long cap, long long every, int R,
                                                         long long E, const double* grid, float f_star, float* mean, int* count) {
  __shared__ double sum_s[256];
  __shared__ int cnt_s[256];
  const double g = grid[blockIdx.x];
  double s = 0.0;
  int c = 0;
  for (int r = threadIdx.x; r < R; r += 256) {
    const double* tr = t + (size_t)r * cap;
    long long lo = 0, hi = E;                 // first evaluation with time > g (evaluation 0 is at time 0)
    while (lo < hi) {
      const long long mid = (lo + hi) >> 1;
      const double tm = mid == 0 ? 0.0 : tr[mid * every - 1];
      if (tm <= g) lo = mid + 1; else hi = mid;
    }
    if (lo > 0) { s += (double)risk[(lo - 1) * R + r] - (double)f_star; ++c; }
  }
  sum_s[threadIdx.x] = s; cnt_s[threadIdx.x] = c;
  __syncthreads();
  for (int off = 128; off > 0; off >>= 1) {
    if ((int)threadIdx.x < off) { sum_s[threadIdx.x] += sum_s[threadIdx.x + off]; cnt_s[threadIdx.x] += cnt_s[threadIdx.x + off]; }
    __syncthreads();
  }
  if (threadIdx.x == 0) { count[blockIdx.x] = cnt_s[0]; mean[blockIdx.x] = cnt_s[0] ? (float)(sum_s[0] / cnt_s[0]) : 0.f; }
}

// Lower envelope of n curves on one grid: at each grid point the smallest value among the curves that have data
// there (count > 0), and which curve it belongs to (lowest index on ties; -1 and 0 where no curve has data).
__global__ void envelope_kernel(const float* curves, const int* counts, int n, int G, float* env, int* best) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= G) return;
  float v = 0.f;
  int b = -1;
  for (int c = 0; c < n; ++c)
    if (counts[(size_t)c * G + i] > 0 && (b < 0 || curves[(size_t)c * G + i] < v)) { v = curves[(size_t)c * G + i]; b = c; }
  env[i] = v;
  best[i] = b;
}

__global__ void fill_int_kernel(int* p, int v, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = v;
}

}  // namespace

// One stretch of `iters` updates of every replica: the arrival process, then the arithmetic along it (in rounds when
// the loss-driven K rule pauses replicas at interval boundaries).  Capacity has been checked by the caller.
static sim_status run_span(sim_handle* h, int64_t iters) {
  sim_status st = SIM_OK;
  ScheduleArgs sa{};
  sa.variant = h->variant; sa.P = h->P; sa.K_fixed = h->K; sa.K0 = h->K0; sa.t_interval = h->t_interval;
  sa.law.kind = (int)h->delay.kind; sa.law.mu = h->delay.mu; sa.law.shift = h->delay.shift;
  sa.seed = h->seed; sa.R = h->R; sa.replica_base = h->replica_base;
  sa.j0 = h->n_updates; sa.iters = iters; sa.cap = h->cap; sa.K_stride = h->K_stride; sa.n_slots = h->n_slots;
  sa.s = h->s; sa.tau = h->tau; sa.f = h->f; sa.wslot = h->wslot; sa.cur_slot = h->cur_slot;
  sa.begin_slot = h->begin_slot; sa.clock = h->clock;
  sa.t = h->tr.t; sa.K_used = h->tr.K_used; sa.worker = h->tr.worker; sa.stale = h->tr.stale; sa.seq = h->tr.seq;
  sa.snap_slot = h->tr.snap_slot; sa.new_slot = h->tr.new_slot; sa.err = h->err;
  // Loss-driven K: replicas pause where an update starts in a new interval and K may still grow; each
  // round schedules every replica up to its next pause (or the target), runs the arithmetic that far,
  // evaluates the full-data risk and sets the paused replicas' new K.  Rounds = interval crossings + 1.
  const bool adaptive = h->ada_loss && h->t_interval > 0.0;
  if (adaptive) {
    if (!h->F0_ready) { if ((st = eval_into(h, h->F0)) != SIM_OK) return st; h->F0_ready = true; }
    sa.adaptive = 1; sa.target = h->n_updates + iters; sa.done = h->done; sa.run_j0 = h->run_j0; sa.run_iters = h->run_iters;
    sa.K_cur = h->K_cur; sa.q_last = h->q_last; sa.want_eval = h->want_eval;
  }
  for (long long round = 0;; ++round) {
  CUDA_TRY(h, launch_schedule(sa, h->stream));

  if (h->prob.model != SIM_NONE) {
    NumericArgs a{};
    if (adaptive) { a.run_j0 = h->run_j0; a.run_iters = h->run_iters; }
    a.X = h->prob.X;
    a.y = h->prob.model == SIM_LSQ ? static_cast<const void*>(h->prob.y) : static_cast<const void*>(h->prob.label);
    a.w_ref = h->prob.w_ref; a.n = (uint64_t)h->prob.n; a.d = h->prob.d; a.m = h->m; a.model = (int)h->prob.model;
    a.n_classes = h->prob.n_classes; a.eta = h->eta; a.seed = h->seed; a.replica_base = h->replica_base; a.R = h->R;
    a.j0 = h->n_updates; a.iters = iters; a.cap = h->cap; a.K_stride = h->K_stride; a.is_async = h->is_async ? 1 : 0;
    a.n_slots = h->n_slots; a.n_params = h->n_params; a.slot_stride = h->slot_stride;
    a.K_used = h->tr.K_used; a.worker = h->tr.worker; a.seq = h->tr.seq; a.snap_slot = h->tr.snap_slot;
    a.new_slot = h->tr.new_slot; a.begin_slot = h->begin_slot; a.loss = h->tr.loss; a.dist2 = h->tr.dist2;
    a.w_state = h->w_state; a.pool = h->pool; a.err = h->err;
    const char* why = nullptr;
    cudaError_t ce = cudaSuccess;
    switch (h->prob.model) {
      case SIM_LSQ: case SIM_LOGISTIC: st = run_linear1(h, a); break;
      case SIM_SOFTMAX:
        ce = run_softmax_any(a, h->tune_stages, h->stream, &why);
        st = why ? fail(h, SIM_ERR_ARG, why) : SIM_OK;
        break;
      case SIM_MLP2:
        ce = ensure_mlp_scratch(h);
        if (ce == cudaSuccess) ce = run_mlp(a, h->mlp, h->mlp_maps, h->P, h->stream, &why);
        if (ce == cudaSuccess && !h->is_async)   // synchronous variants ping-pong between two slots
          ce = cudaMemsetAsync(h->cur_slot, (int)((h->n_updates + iters) & 1), (size_t)h->R, h->stream);
        st = why ? fail(h, SIM_ERR_ARG, why) : SIM_OK;
        break;
      default: st = fail(h, SIM_ERR_ARG, "unknown model");
    }
    if (ce != cudaSuccess) st = fail(h, SIM_ERR_CUDA, std::string("numeric kernel launch: ") + cudaGetErrorString(ce));
    if (st != SIM_OK) { h->poisoned = true; return st; }
  }
  if (!adaptive) break;
  if ((st = eval_into(h, h->Fcur)) != SIM_OK) { h->poisoned = true; return st; }
  CUDA_TRY(h, cudaMemsetAsync(h->remaining, 0, sizeof(int), h->stream));
  adasync_update_kernel<<<(h->R + 127) / 128, 128, 0, h->stream>>>(h->variant, h->P, h->K0, h->t_interval, h->R, sa.target, h->F0,
                                                                  h->Fcur, h->clock, h->done, h->K_cur, h->q_last, h->want_eval,
                                                                  h->remaining);
  CUDA_TRY(h, cudaGetLastError());
  int remaining = 0;
  CUDA_TRY(h, cudaMemcpyAsync(&remaining, h->remaining, sizeof(int), cudaMemcpyDeviceToHost, h->stream));
  CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  if (remaining == 0) break;
  if (round > iters + 8) { h->poisoned = true; return fail(h, SIM_ERR_INTERNAL, "loss-driven K: no progress"); }
  }
  h->n_updates += iters;
  return SIM_OK;
}


extern "C" {

sim_status sim_create(const sim_problem* problem, int32_t P, int32_t K, sim_variant variant,
                      sim_delay delay, float eta, int32_t m, uint64_t seed, int32_t n_replicas,
                      int64_t replica_base, void* cuda_stream, sim_handle** out) {
  if (!out) return fail(nullptr, SIM_ERR_ARG, "out is NULL");
  *out = nullptr;
  if (P < 1 || P > SIM_MAX_P) return fail(nullptr, SIM_ERR_ARG, "P must be in [1, SIM_MAX_P]");
  if (K < 1 || K > P) return fail(nullptr, SIM_ERR_ARG, "K must be in [1, P]");
  if ((int)variant < 0 || (int)variant > 3) return fail(nullptr, SIM_ERR_ARG, "unknown variant");
  if (m < 1) return fail(nullptr, SIM_ERR_ARG, "m must be >= 1");
  // the index stream packs draw q as chunk q / 4 into 24 bits of the counter
  if (m > (1 << 26)) return fail(nullptr, SIM_ERR_ARG, "m must be at most 2^26 (the minibatch index stream has 2^24 chunks of four draws)");
  if (n_replicas < 1) return fail(nullptr, SIM_ERR_ARG, "n_replicas must be >= 1");
  if (replica_base < 0 || replica_base + (int64_t)n_replicas > (int64_t)1 << 32)
    return fail(nullptr, SIM_ERR_ARG, "global replica ids must fit in 32 bits");
  sim_status st = check_delay(nullptr, delay);
  if (st != SIM_OK) return st;
  if (!(eta == eta) || std::isinf(eta)) return fail(nullptr, SIM_ERR_ARG, "eta must be finite");

  sim_problem prob{};
  prob.model = SIM_NONE;
  if (problem) prob = *problem;
  if (prob.model != SIM_NONE) {
    if ((int)prob.model < 0 || (int)prob.model > (int)SIM_MLP2) return fail(nullptr, SIM_ERR_ARG, "unknown model");
    if (prob.n < 1 || prob.n > (int64_t)1 << 32) return fail(nullptr, SIM_ERR_ARG, "n must be in [1, 2^32]");
    if (prob.d < 4 || prob.d % 4 != 0) return fail(nullptr, SIM_ERR_ARG, "d must be a positive multiple of 4");
    if (!prob.X || (reinterpret_cast<uintptr_t>(prob.X) & 15u)) return fail(nullptr, SIM_ERR_ARG, "X must be a 16-byte aligned device pointer");
    if (prob.model == SIM_LSQ && !prob.y) return fail(nullptr, SIM_ERR_ARG, "least squares needs y");
    if (prob.model != SIM_LSQ && !prob.label) return fail(nullptr, SIM_ERR_ARG, "classification models need label");
    if (prob.w_ref && (reinterpret_cast<uintptr_t>(prob.w_ref) & 15u)) return fail(nullptr, SIM_ERR_ARG, "w_ref must be 16-byte aligned");
    if (prob.model == SIM_SOFTMAX || prob.model == SIM_MLP2) {
      if (prob.n_classes < 2 || prob.n_classes > SIM_MAX_CLASSES) return fail(nullptr, SIM_ERR_ARG, "n_classes must be in [2, SIM_MAX_CLASSES]");
    }
    if (prob.model == SIM_SOFTMAX) {
      const char* why = softmax_ws_supported(prob.d, prob.n_classes, m) ? nullptr : softmax_shape_unsupported(prob.d, prob.n_classes, m);
      if (why) return fail(nullptr, SIM_ERR_ARG, why);
    }
    if (prob.model == SIM_MLP2) {
      const char* why = mlp_shape_unsupported(prob.d, prob.hidden, prob.n_classes, m);
      if (why) return fail(nullptr, SIM_ERR_ARG, why);
    }
    if ((prob.model == SIM_LSQ || prob.model == SIM_LOGISTIC) && prob.d > 8192)
      return fail(nullptr, SIM_ERR_ARG, "d > 8192 is not supported by the linear-model kernel");
    if ((prob.model == SIM_LSQ || prob.model == SIM_LOGISTIC) && linear1_min_smem(prob.d, m, n_replicas) > (size_t)(226 << 10))
      return fail(nullptr, SIM_ERR_ARG, "m is too large for this d: the kernel keeps two tiles of sample rows and an m-entry index table "
                                        "(4 m bytes) in shared memory");
  }

  sim_handle* h = new (std::nothrow) sim_handle();
  if (h) h->in_arena = t_arena != nullptr;
  if (!h) return fail(nullptr, SIM_ERR_ALLOC, "host allocation failed");
  h->prob = prob; h->P = P; h->K = K; h->variant = (int)variant; h->delay = delay; h->eta = eta;
  h->m = m; h->seed = seed; h->R = n_replicas; h->replica_base = (uint32_t)replica_base;
  h->stream = static_cast<cudaStream_t>(cuda_stream);
  h->K_stride = K;
  h->is_async = variant == SIM_KASYNC || variant == SIM_KBATCHASYNC;
  h->uses_pool = h->is_async || prob.model == SIM_MLP2;
  h->n_slots = h->is_async ? P + 2 : (prob.model == SIM_MLP2 ? 2 : 0);
  h->n_params = model_params(prob);
  h->slot_stride = (h->n_params + 3) & ~3ll;

  cudaError_t e = cudaGetDevice(&h->device);
  const size_t RP = (size_t)h->R * P;
  if (e == cudaSuccess) e = dev_alloc(&h->s, RP, h->stream);
  if (e == cudaSuccess) e = dev_alloc(&h->tau, RP, h->stream);
  if (e == cudaSuccess) e = dev_alloc(&h->f, RP, h->stream);
  if (e == cudaSuccess) e = dev_alloc(&h->wslot, RP, h->stream);
  if (e == cudaSuccess) e = dev_alloc(&h->cur_slot, (size_t)h->R, h->stream);
  if (e == cudaSuccess) e = dev_alloc(&h->begin_slot, (size_t)h->R, h->stream);
  if (e == cudaSuccess) e = dev_alloc(&h->clock, (size_t)h->R, h->stream);
  if (e == cudaSuccess) e = dev_alloc(&h->err, 1, h->stream);
  if (e == cudaSuccess && h->n_params > 0) {
    if (h->uses_pool) e = dev_alloc(&h->pool, (size_t)h->R * h->n_slots * h->slot_stride, h->stream);
    else e = dev_alloc(&h->w_state, (size_t)h->R * h->n_params, h->stream);
  }
  if (e != cudaSuccess) {
    const sim_status code = e == cudaErrorMemoryAllocation ? SIM_ERR_ALLOC : SIM_ERR_CUDA;
    std::string msg = std::string("sim_create: ") + cudaGetErrorString(e);
    free_all(h);
    delete h;
    cudaGetLastError();
    return fail(nullptr, code, msg);
  }
  *out = h;
  return SIM_OK;
}

sim_status sim_set_params(sim_handle* h, const float* w0) {
  if (!h) return fail(nullptr, SIM_ERR_ARG, "handle is NULL");
  if (!w0) return fail(h, SIM_ERR_ARG, "w0 is NULL");
  if (h->n_updates > 0) return fail(h, SIM_ERR_STATE, "sim_set_params is only allowed before the first sim_run");
  if (h->n_params == 0) return SIM_OK;
  float* dst = h->uses_pool ? h->pool : h->w_state;
  const long long stride = h->uses_pool ? (long long)h->n_slots * h->slot_stride : h->n_params;
  const bool mlp = h->prob.model == SIM_MLP2;
  broadcast_params_kernel<<<1184, 256, 0, h->stream>>>(w0, dst, h->n_params, stride, h->R,
                                                        mlp ? (long long)h->prob.d * h->prob.hidden : 0, mlp ? h->prob.hidden : 1);
  CUDA_TRY(h, cudaGetLastError());
  // the caller's buffer is read by enqueued work: finish it before returning
  CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  return SIM_OK;
}

sim_status sim_set_adasync(sim_handle* h, int32_t K0, double t_interval) {
  if (!h) return fail(nullptr, SIM_ERR_ARG, "handle is NULL");
  if (h->n_updates > 0 || h->cap > 0) return fail(h, SIM_ERR_STATE, "sim_set_adasync is only allowed before sim_reserve / sim_run");
  if (t_interval > 0.0) {
    if (K0 < 1 || K0 > h->P) return fail(h, SIM_ERR_ARG, "K0 must be in [1, P]");
    h->K0 = K0; h->t_interval = t_interval; h->K_stride = h->P; h->ada_loss = false;
  } else {
    // switching the schedule off also switches off the loss-driven rule: with no interval there is nothing to
    // pause at, and the trace rows go back to K entries
    h->K0 = 0; h->t_interval = 0.0; h->K_stride = h->K; h->ada_loss = false; h->F0_ready = false;
  }
  return SIM_OK;
}

sim_status sim_set_tuning(sim_handle* h, int32_t stages, int32_t tile_rows, int32_t threads) {
  if (!h) return fail(nullptr, SIM_ERR_ARG, "handle is NULL");
  if (stages < 0 || stages == 1 || stages > 8) return fail(h, SIM_ERR_ARG, "stages must be 0 (automatic) or in [2, 8]");
  if (tile_rows != 0 && tile_rows != 2 && tile_rows != 4 && tile_rows != 8) return fail(h, SIM_ERR_ARG, "tile_rows must be 0, 2, 4 or 8");
  if (threads != 0 && threads != 256 && threads != 512) return fail(h, SIM_ERR_ARG, "threads must be 0, 256 or 512");
  h->tune_stages = stages; h->tune_rows = tile_rows; h->tune_threads = threads;
  return SIM_OK;
}

sim_status sim_reserve(sim_handle* h, int64_t total_updates) {
  if (!h) return fail(nullptr, SIM_ERR_ARG, "handle is NULL");
  if (total_updates < 0) return fail(h, SIM_ERR_ARG, "total_updates must be >= 0");
  return ensure_capacity(h, total_updates);
}

sim_status sim_run(sim_handle* h, int64_t iters) {
  if (!h) return fail(nullptr, SIM_ERR_ARG, "handle is NULL");
  if (iters < 0) return fail(h, SIM_ERR_ARG, "iters must be >= 0");
  if (h->poisoned) return fail(h, SIM_ERR_STATE, "the handle failed earlier and cannot run");
  if (iters == 0) return SIM_OK;
  if (h->n_updates + iters > (1ll << 31)) return fail(h, SIM_ERR_ARG, "more than 2^31 updates");
  sim_status st = ensure_capacity(h, h->n_updates + iters);
  if (st != SIM_OK) return st;
  if (h->eval_every <= 0) return run_span(h, iters);

  // with a risk trace: stop at every multiple of eval_every and evaluate F(w_j) there (entry 0 is F(w_0))
  const long long every = h->eval_every, need = 1 + (h->n_updates + iters) / every;
  if (need > h->risk_cap) {
    const long long nc = h->risk_cap * 2 > need ? h->risk_cap * 2 : need;
    float* nb = nullptr;
    CUDA_TRY(h, dev_alloc(&nb, (size_t)nc * h->R, h->stream, false));
    if (h->risk && h->n_evals > 0)
      CUDA_TRY(h, cudaMemcpyAsync(nb, h->risk, (size_t)h->n_evals * h->R * sizeof(float), cudaMemcpyDeviceToDevice, h->stream));
    if (h->risk && !h->in_arena) { CUDA_TRY(h, cudaStreamSynchronize(h->stream)); cudaFree(h->risk); }
    h->risk = nb; h->risk_cap = nc;
  }
  if (h->n_evals == 0) {
    if ((st = eval_into(h, h->risk)) != SIM_OK) { h->poisoned = true; return st; }
    h->n_evals = 1;
  }
  for (long long left = iters; left > 0;) {
    const long long mark = (h->n_updates / every + 1) * every;
    const long long seg = left < mark - h->n_updates ? left : mark - h->n_updates;
    if ((st = run_span(h, seg)) != SIM_OK) return st;
    left -= seg;
    if (h->n_updates == mark) {
      if ((st = eval_into(h, h->risk + (size_t)h->n_evals * h->R)) != SIM_OK) { h->poisoned = true; return st; }
      ++h->n_evals;
    }
  }
  return SIM_OK;
}

sim_status sim_trace_size(const sim_handle* h, int64_t* n_updates, int32_t* K_max) {
  if (!h) return fail(nullptr, SIM_ERR_ARG, "handle is NULL");
  sim_status st = device_error(h);
  if (st != SIM_OK) return st;
  if (n_updates) *n_updates = h->n_updates;
  if (K_max) *K_max = h->K_stride;
  return SIM_OK;
}

sim_status sim_get_trace(const sim_handle* h, double* t, float* loss, float* dist2, uint16_t* K_used,
                         uint16_t* worker, uint32_t* stale, uint32_t* seq) {
  if (!h) return fail(nullptr, SIM_ERR_ARG, "handle is NULL");
  sim_status st = device_error(h);
  if (st != SIM_OK) return st;
  const long long J = h->n_updates;
  if (J == 0) return SIM_OK;
  const size_t Ks = (size_t)h->K_stride;
  auto copy = [&](void* dst, const void* src, size_t elem) -> cudaError_t {
    if (!dst) return cudaSuccess;
    return cudaMemcpy2DAsync(dst, (size_t)J * elem, src, (size_t)h->cap * elem, (size_t)J * elem, h->R,
                             cudaMemcpyDeviceToDevice, h->stream);
  };
  CUDA_TRY(h, copy(t, h->tr.t, 8));
  CUDA_TRY(h, copy(loss, h->tr.loss, 4));
  CUDA_TRY(h, copy(dist2, h->tr.dist2, 4));
  CUDA_TRY(h, copy(K_used, h->tr.K_used, 2));
  CUDA_TRY(h, copy(worker, h->tr.worker, 2 * Ks));
  CUDA_TRY(h, copy(stale, h->tr.stale, 4 * Ks));
  CUDA_TRY(h, copy(seq, h->tr.seq, 4 * Ks));
  CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  return SIM_OK;
}

sim_status sim_get_params(const sim_handle* h, float* w) {
  if (!h) return fail(nullptr, SIM_ERR_ARG, "handle is NULL");
  if (!w) return fail(h, SIM_ERR_ARG, "w is NULL");
  sim_status st = device_error(h);
  if (st != SIM_OK) return st;
  if (h->n_params == 0) return SIM_OK;
  if (h->uses_pool) {
    gather_params_kernel<<<1184, 256, 0, h->stream>>>(h->pool, h->cur_slot, w, h->n_params, h->slot_stride, h->n_slots, h->R,
                                                       h->prob.model == SIM_MLP2 ? (long long)h->prob.d * h->prob.hidden : 0,
                                                       h->prob.model == SIM_MLP2 ? h->prob.hidden : 1);
    CUDA_TRY(h, cudaGetLastError());
  } else {
    CUDA_TRY(h, cudaMemcpyAsync(w, h->w_state, (size_t)h->R * h->n_params * sizeof(float), cudaMemcpyDeviceToDevice, h->stream));
  }
  CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  return SIM_OK;
}

sim_status sim_eval_loss(sim_handle* h, float* loss) {
  if (!h) return fail(nullptr, SIM_ERR_ARG, "handle is NULL");
  if (!loss) return fail(h, SIM_ERR_ARG, "loss is NULL");
  if (h->poisoned) return fail(h, SIM_ERR_STATE, "the handle failed earlier");
  return eval_into(h, loss);
}

sim_status sim_set_adasync_loss(sim_handle* h, int32_t K0, double t_interval) {
  if (!h) return fail(nullptr, SIM_ERR_ARG, "handle is NULL");
  if (h->n_updates > 0 || h->cap > 0) return fail(h, SIM_ERR_STATE, "sim_set_adasync_loss is only allowed before sim_reserve / sim_run");
  if (!(t_interval > 0.0)) return fail(h, SIM_ERR_ARG, "t_interval must be > 0");
  if (K0 < 1 || K0 > h->P) return fail(h, SIM_ERR_ARG, "K0 must be in [1, P]");
  if (h->eval_every > 0) return fail(h, SIM_ERR_STATE, "the loss-driven K rule cannot be combined with the risk trace (sim_set_eval_every)");
  const sim_model mdl = h->prob.model;
  if (mdl != SIM_LSQ && mdl != SIM_LOGISTIC && mdl != SIM_SOFTMAX)
    return fail(h, SIM_ERR_ARG, "the loss-driven K rule needs the full-data risk: LSQ, logistic or softmax");
  const size_t R = (size_t)h->R;
  if (!h->F0) {
    CUDA_TRY(h, dev_alloc(&h->F0, R, h->stream)); CUDA_TRY(h, dev_alloc(&h->Fcur, R, h->stream));
    CUDA_TRY(h, dev_alloc(&h->done, R, h->stream)); CUDA_TRY(h, dev_alloc(&h->run_j0, R, h->stream));
    CUDA_TRY(h, dev_alloc(&h->run_iters, R, h->stream)); CUDA_TRY(h, dev_alloc(&h->q_last, R, h->stream));
    CUDA_TRY(h, dev_alloc(&h->K_cur, R, h->stream)); CUDA_TRY(h, dev_alloc(&h->want_eval, R, h->stream));
    CUDA_TRY(h, dev_alloc(&h->remaining, 1, h->stream));
  }
  fill_int_kernel<<<(h->R + 127) / 128, 128, 0, h->stream>>>(h->K_cur, K0, h->R);
  CUDA_TRY(h, cudaGetLastError());
  h->ada_loss = true; h->F0_ready = false;
  h->K0 = K0; h->t_interval = t_interval; h->K_stride = h->P;
  return SIM_OK;
}

sim_status sim_error_curve(const sim_handle* h, const double* grid, int32_t n_grid, float* mean_loss, int32_t* count) {
  if (!h) return fail(nullptr, SIM_ERR_ARG, "handle is NULL");
  if (!grid || !mean_loss || !count || n_grid < 1) return fail(h, SIM_ERR_ARG, "grid, mean_loss, count and n_grid >= 1 are required");
  sim_status st = device_error(h);
  if (st != SIM_OK) return st;
  if (h->n_updates == 0) return fail(h, SIM_ERR_STATE, "no updates have been simulated yet");
  error_curve_kernel<<<n_grid, 256, 0, h->stream>>>(h->tr.t, h->tr.loss, h->cap, h->n_updates, h->R, grid, mean_loss, count);
  CUDA_TRY(h, cudaGetLastError());
  CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  return SIM_OK;
}

sim_status sim_set_eval_every(sim_handle* h, int64_t every) {
  if (!h) return fail(nullptr, SIM_ERR_ARG, "handle is NULL");
  if (every < 0) return fail(h, SIM_ERR_ARG, "every must be >= 0");
  if (h->n_updates > 0) return fail(h, SIM_ERR_STATE, "sim_set_eval_every is only allowed before the first sim_run");
  if (every > 0 && h->prob.model == SIM_NONE) return fail(h, SIM_ERR_ARG, "a clock-only simulation has no risk to record");
  if (every > 0 && h->ada_loss) return fail(h, SIM_ERR_STATE, "the risk trace cannot be combined with the loss-driven K rule");
  h->eval_every = every;
  return SIM_OK;
}

sim_status sim_risk_trace_size(const sim_handle* h, int64_t* n_evals) {
  if (!h) return fail(nullptr, SIM_ERR_ARG, "handle is NULL");
  if (n_evals) *n_evals = h->n_evals;
  return SIM_OK;
}

sim_status sim_get_risk_trace(const sim_handle* h, float* risk, double* t) {
  if (!h) return fail(nullptr, SIM_ERR_ARG, "handle is NULL");
  sim_status st = device_error(h);
  if (st != SIM_OK) return st;
  if (h->n_evals == 0 || (!risk && !t)) return SIM_OK;
  risk_trace_out_kernel<<<296, 256, 0, h->stream>>>(h->risk, h->tr.t, h->cap, h->eval_every, h->R, h->n_evals, risk, t);
  CUDA_TRY(h, cudaGetLastError());
  CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  return SIM_OK;
}

sim_status sim_risk_curve(const sim_handle* h, const double* grid, int32_t n_grid, float f_star, float* mean_err, int32_t* count) {
  if (!h) return fail(nullptr, SIM_ERR_ARG, "handle is NULL");
  if (!grid || !mean_err || !count || n_grid < 1) return fail(h, SIM_ERR_ARG, "grid, mean_err, count and n_grid >= 1 are required");
  sim_status st = device_error(h);
  if (st != SIM_OK) return st;
  if (h->n_evals == 0) return fail(h, SIM_ERR_STATE, "no risk has been recorded (sim_set_eval_every, then sim_run)");
  risk_curve_kernel<<<n_grid, 256, 0, h->stream>>>(h->risk, h->tr.t, h->cap, h->eval_every, h->R, h->n_evals, grid, f_star, mean_err, count);
  CUDA_TRY(h, cudaGetLastError());
  CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  return SIM_OK;
}

sim_status sim_risk_envelope(sim_handle* const* handles, int32_t n_handles, const double* grid, int32_t n_grid, float f_star,
                             float* env, int32_t* best) {
  if (!handles || n_handles < 1 || n_handles > 4096) return fail(nullptr, SIM_ERR_ARG, "sim_risk_envelope: handles and 1 <= n_handles <= 4096 are required");
  if (!grid || !env || !best || n_grid < 1) return fail(nullptr, SIM_ERR_ARG, "sim_risk_envelope: grid, env, best and n_grid >= 1 are required");
  for (int i = 0; i < n_handles; ++i)
    if (!handles[i]) return fail(nullptr, SIM_ERR_ARG, "sim_risk_envelope: a handle is NULL");
  float* curves = nullptr;
  int* counts = nullptr;
  const size_t cells = (size_t)n_handles * n_grid;
  cudaError_t ce = cudaMalloc(&curves, cells * sizeof(float));
  if (ce == cudaSuccess) ce = cudaMalloc(&counts, cells * sizeof(int));
  sim_status st = ce == cudaSuccess ? SIM_OK : fail(nullptr, SIM_ERR_ALLOC, std::string("sim_risk_envelope: ") + cudaGetErrorString(ce));
  std::string msg;
  for (int i = 0; i < n_handles && st == SIM_OK; ++i) {      // each curve on its handle's stream; the call waits for it
    st = sim_risk_curve(handles[i], grid, n_grid, f_star, curves + (size_t)i * n_grid, counts + (size_t)i * n_grid);
    if (st != SIM_OK) msg = sim_last_error(handles[i]);
  }
  if (st == SIM_OK && msg.empty()) {
    cudaStream_t stream = handles[0]->stream;
    envelope_kernel<<<(n_grid + 127) / 128, 128, 0, stream>>>(curves, counts, n_handles, n_grid, env, best);
    ce = cudaGetLastError();
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(stream);
    if (ce != cudaSuccess) { st = SIM_ERR_CUDA; msg = cudaGetErrorString(ce); }
  }
  cudaFree(curves);
  cudaFree(counts);
  if (st != SIM_OK && !msg.empty()) return fail(nullptr, st, "sim_risk_envelope: " + msg);
  return st;
}

sim_status sim_selftest_wait_timeout(sim_handle* h) {
  if (!h) return fail(nullptr, SIM_ERR_ARG, "handle is NULL");
  wait_timeout_selftest_kernel<<<1, 64, 0, h->stream>>>(h->err, 1u << 10);
  CUDA_TRY(h, cudaGetLastError());
  return SIM_OK;
}

int64_t sim_n_params(const sim_handle* h) { return h ? h->n_params : 0; }

const char* sim_last_error(const sim_handle* h) { return h ? h->last_error.c_str() : g_last_error.c_str(); }

void sim_destroy(sim_handle* h) {
  if (!h) return;
  cudaStreamSynchronize(h->stream);
  free_all(h);
  delete h;
}

sim_status sim_draw_delays(sim_delay delay, uint64_t seed, int64_t replica_base, int32_t n_replicas,
                           int32_t P, int32_t n_seq, double* out, void* cuda_stream) {
  sim_status st = check_delay(nullptr, delay);
  if (st != SIM_OK) return st;
  if (!out || n_replicas < 1 || P < 1 || n_seq < 1 || replica_base < 0 || replica_base + (int64_t)n_replicas > (int64_t)1 << 32)
    return fail(nullptr, SIM_ERR_ARG, "sim_draw_delays: bad argument");
  DelayLaw law{(int)delay.kind, delay.mu, delay.shift};
  draw_delays_kernel<<<592, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(law, seed, (uint32_t)replica_base, n_replicas, P, n_seq, out);
  CUDA_TRY(nullptr, cudaGetLastError());
  return SIM_OK;
}

sim_status sim_draw_indices(uint64_t seed, int64_t replica_base, int32_t n_replicas, int32_t P,
                            int32_t n_seq, int64_t n, int32_t m, uint32_t* out, void* cuda_stream) {
  if (!out || n_replicas < 1 || P < 1 || n_seq < 1 || m < 1 || n < 1 || n > (int64_t)1 << 32 || replica_base < 0 ||
      replica_base + (int64_t)n_replicas > (int64_t)1 << 32)
    return fail(nullptr, SIM_ERR_ARG, "sim_draw_indices: bad argument");
  draw_indices_kernel<<<592, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(seed, (uint32_t)replica_base, n_replicas, P, n_seq, (uint64_t)n, m, out);
  CUDA_TRY(nullptr, cudaGetLastError());
  return SIM_OK;
}

sim_status sim_simulate_host(const sim_problem* problem, int32_t P, int32_t K, sim_variant variant,
                             sim_delay delay, float eta, int32_t m, uint64_t seed, int32_t n_replicas,
                             int64_t replica_base, const float* w0, int32_t K0, double t_interval,
                             int64_t iters, double* t, float* loss, float* dist2, uint16_t* K_used,
                             uint16_t* worker, uint32_t* stale, uint32_t* seq, float* w_final) {
  if (iters < 0) return fail(nullptr, SIM_ERR_ARG, "iters must be >= 0");
  sim_problem dp{};
  dp.model = SIM_NONE;
  std::vector<void*> owned;
  sim_handle* h = nullptr;
  sim_status st = SIM_OK;
  std::string msg;
  auto up = [&](const void* src, size_t bytes, void** dst) -> bool {
    *dst = nullptr;
    if (!src || bytes == 0) return true;
    cudaError_t e = cudaMalloc(dst, bytes);
    if (e == cudaSuccess) { owned.push_back(*dst); e = cudaMemcpyAsync(*dst, src, bytes, cudaMemcpyHostToDevice, nullptr); }
    if (e != cudaSuccess) { st = e == cudaErrorMemoryAllocation ? SIM_ERR_ALLOC : SIM_ERR_CUDA; msg = cudaGetErrorString(e); return false; }
    return true;
  };
  auto down = [&](void* host, size_t bytes, auto getter) -> bool {
    if (!host || bytes == 0) return true;
    void* dev = nullptr;
    cudaError_t e = cudaMalloc(&dev, bytes);
    if (e != cudaSuccess) { st = SIM_ERR_ALLOC; msg = cudaGetErrorString(e); return false; }
    owned.push_back(dev);
    st = getter(dev);
    if (st != SIM_OK) { msg = sim_last_error(h); return false; }
    e = cudaMemcpy(host, dev, bytes, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) { st = SIM_ERR_CUDA; msg = cudaGetErrorString(e); return false; }
    return true;
  };
  do {
    void* dw0 = nullptr;
    long long np = 0;
    if (problem && problem->model != SIM_NONE) {
      dp = *problem;
      if (dp.n < 1 || dp.d < 1 || !dp.X) { st = SIM_ERR_ARG; msg = "bad problem"; break; }
      np = model_params(dp);
      void *X, *y, *lab, *wr;
      if (!up(problem->X, (size_t)dp.n * dp.d * 4, &X)) break;
      if (!up(problem->y, (size_t)dp.n * 4, &y)) break;
      if (!up(problem->label, (size_t)dp.n * 4, &lab)) break;
      if (!up(problem->w_ref, (size_t)np * 4, &wr)) break;
      dp.X = (const float*)X; dp.y = (const float*)y; dp.label = (const int32_t*)lab; dp.w_ref = (const float*)wr;
      if (!up(w0, (size_t)np * 4, &dw0)) break;
    }
    st = sim_create(&dp, P, K, variant, delay, eta, m, seed, n_replicas, replica_base, nullptr, &h);
    if (st != SIM_OK) { msg = g_last_error; break; }
    if (t_interval > 0.0 && (st = sim_set_adasync(h, K0, t_interval)) != SIM_OK) { msg = sim_last_error(h); break; }
    if (dw0 && (st = sim_set_params(h, (const float*)dw0)) != SIM_OK) { msg = sim_last_error(h); break; }
    if ((st = sim_run(h, iters)) != SIM_OK) { msg = sim_last_error(h); break; }
    const size_t RJ = (size_t)n_replicas * iters, Ks = (size_t)h->K_stride;
    if (!down(t, RJ * 8, [&](void* p) { return sim_get_trace(h, (double*)p, 0, 0, 0, 0, 0, 0); })) break;
    if (!down(loss, RJ * 4, [&](void* p) { return sim_get_trace(h, 0, (float*)p, 0, 0, 0, 0, 0); })) break;
    if (!down(dist2, RJ * 4, [&](void* p) { return sim_get_trace(h, 0, 0, (float*)p, 0, 0, 0, 0); })) break;
    if (!down(K_used, RJ * 2, [&](void* p) { return sim_get_trace(h, 0, 0, 0, (uint16_t*)p, 0, 0, 0); })) break;
    if (!down(worker, RJ * Ks * 2, [&](void* p) { return sim_get_trace(h, 0, 0, 0, 0, (uint16_t*)p, 0, 0); })) break;
    if (!down(stale, RJ * Ks * 4, [&](void* p) { return sim_get_trace(h, 0, 0, 0, 0, 0, (uint32_t*)p, 0); })) break;
    if (!down(seq, RJ * Ks * 4, [&](void* p) { return sim_get_trace(h, 0, 0, 0, 0, 0, 0, (uint32_t*)p); })) break;
    if (np > 0 && !down(w_final, (size_t)n_replicas * np * 4, [&](void* p) { return sim_get_params(h, (float*)p); })) break;
    if (st == SIM_OK) st = device_error(h);
    if (st != SIM_OK) msg = sim_last_error(h);
  } while (0);
  if (h) sim_destroy(h); else cudaDeviceSynchronize();
  for (void* p : owned) cudaFree(p);
  if (st != SIM_OK) return fail(nullptr, st, "sim_simulate_host: " + msg);
  return SIM_OK;
}

sim_status sim_sweep_host(const sim_problem* problem, int32_t P, int32_t n_runs, const int32_t* variants,
                          const int32_t* Ks, sim_delay delay, float eta, int32_t m, uint64_t seed,
                          int32_t n_replicas, int64_t replica_base, const float* w0, int64_t iters,
                          double* t, float* loss, float* dist2) {
  if (!problem || problem->model == SIM_NONE || !problem->X) return fail(nullptr, SIM_ERR_ARG, "sim_sweep_host needs a problem");
  if (n_runs < 1 || n_runs > 256 || !variants || !Ks) return fail(nullptr, SIM_ERR_ARG, "n_runs must be in [1, 256] with variants and Ks given");
  if (iters < 1) return fail(nullptr, SIM_ERR_ARG, "iters must be >= 1");
  if (problem->n < 1 || problem->d < 1) return fail(nullptr, SIM_ERR_ARG, "bad problem");
  sim_problem dp = *problem;
  const long long np = model_params(dp);
  std::vector<void*> owned;
  std::vector<sim_handle*> hs((size_t)n_runs, nullptr);
  std::vector<cudaStream_t> streams((size_t)n_runs, nullptr);
  sim_status st = SIM_OK;
  std::string msg;
  auto up = [&](const void* src, size_t bytes, void** dst) -> bool {
    *dst = nullptr;
    if (!src || bytes == 0) return true;
    cudaError_t e = cudaMalloc(dst, bytes);
    if (e == cudaSuccess) { owned.push_back(*dst); e = cudaMemcpyAsync(*dst, src, bytes, cudaMemcpyHostToDevice, nullptr); }
    if (e != cudaSuccess) { st = e == cudaErrorMemoryAllocation ? SIM_ERR_ALLOC : SIM_ERR_CUDA; msg = cudaGetErrorString(e); return false; }
    return true;
  };
  const size_t RJ = (size_t)n_replicas * (size_t)iters;
  DeviceArena arena;                    // the runs' state, parameters and traces: a few chunks instead of hundreds of buffers
  t_arena = &arena;
  cudaEvent_t uploaded = nullptr;
  do {
    void *X, *y, *lab, *wr, *dw0;
    if (!up(problem->X, (size_t)dp.n * dp.d * 4, &X)) break;
    if (!up(problem->y, (size_t)dp.n * 4, &y)) break;
    if (!up(problem->label, (size_t)dp.n * 4, &lab)) break;
    if (!up(problem->w_ref, (size_t)np * 4, &wr)) break;
    if (!up(w0, (size_t)np * 4, &dw0)) break;
    dp.X = (const float*)X; dp.y = (const float*)y; dp.label = (const int32_t*)lab; dp.w_ref = (const float*)wr;
    // the copies above are in flight on the default stream; the runs' streams wait for them on the device, so that the host
    // sets the runs up meanwhile
    if (cudaEventCreateWithFlags(&uploaded, cudaEventDisableTiming) != cudaSuccess || cudaEventRecord(uploaded, nullptr) != cudaSuccess) {
      st = SIM_ERR_CUDA; msg = "upload failed"; break;
    }
    // every run gets its own stream: the runs are independent and overlap on the device
    for (int i = 0; i < n_runs && st == SIM_OK; ++i) {
      if (cudaStreamCreateWithFlags(&streams[i], cudaStreamNonBlocking) != cudaSuccess ||
          cudaStreamWaitEvent(streams[i], uploaded, 0) != cudaSuccess) { st = SIM_ERR_CUDA; msg = "stream creation failed"; break; }
      st = sim_create(&dp, P, Ks[i], (sim_variant)variants[i], delay, eta, m, seed, n_replicas, replica_base, streams[i], &hs[i]);
      if (st != SIM_OK) { msg = g_last_error; break; }
      if ((st = sim_reserve(hs[i], iters)) != SIM_OK) { msg = sim_last_error(hs[i]); break; }
      if (dw0 && (st = sim_set_params(hs[i], (const float*)dw0)) != SIM_OK) { msg = sim_last_error(hs[i]); break; }
    }
    if (st != SIM_OK) break;
    for (int i = 0; i < n_runs && st == SIM_OK; ++i)
      if ((st = sim_run(hs[i], iters)) != SIM_OK) msg = sim_last_error(hs[i]);
    if (st != SIM_OK) break;
    // traces come back run by run, straight from each handle's buffers (row pitch = capacity = iters)
    for (int i = 0; i < n_runs && st == SIM_OK; ++i) {
      sim_handle* h = hs[i];
      if ((st = device_error(h)) != SIM_OK) { msg = sim_last_error(h); break; }
      cudaError_t e = cudaSuccess;
      if (t) e = cudaMemcpy2D(t + (size_t)i * RJ, (size_t)iters * 8, h->tr.t, (size_t)h->cap * 8, (size_t)iters * 8, n_replicas, cudaMemcpyDeviceToHost);
      if (e == cudaSuccess && loss) e = cudaMemcpy2D(loss + (size_t)i * RJ, (size_t)iters * 4, h->tr.loss, (size_t)h->cap * 4, (size_t)iters * 4, n_replicas, cudaMemcpyDeviceToHost);
      if (e == cudaSuccess && dist2) e = cudaMemcpy2D(dist2 + (size_t)i * RJ, (size_t)iters * 4, h->tr.dist2, (size_t)h->cap * 4, (size_t)iters * 4, n_replicas, cudaMemcpyDeviceToHost);
      if (e != cudaSuccess) { st = SIM_ERR_CUDA; msg = cudaGetErrorString(e); }
    }
  } while (0);
  for (int i = 0; i < n_runs; ++i) {
    if (hs[i]) sim_destroy(hs[i]);
    if (streams[i]) cudaStreamDestroy(streams[i]);
  }
  t_arena = nullptr;
  cudaDeviceSynchronize();
  if (uploaded) cudaEventDestroy(uploaded);
  arena.release();
  for (void* p : owned) cudaFree(p);
  if (st != SIM_OK) return fail(nullptr, st, "sim_sweep_host: " + msg);
  return SIM_OK;
}

}  // extern "C"
