// sim_schedule_noalloc: the arrival process (clock-only simulation) for callers that must not
// allocate device memory.
//
// Some callers cannot call cudaMalloc at all: code that runs inside a latency-critical service
// loop where an allocation would serialise the whole device, code that runs under a memory pool
// whose owner forbids side allocations, or a host thread that shares the GPU with a job that has
// already claimed the memory it is allowed to use.  For them this file offers one entry point
// that allocates nothing: the per-replica worker state that the regular path keeps in
// cudaMalloc'ed buffers (tasks launched, version fetched, finish time of the running task, the
// replica's clock) lives in a fixed array that is part of the library image.
//
// The array is a file-scope `static __device__` object.  Its name is usable directly in device
// code; in host code the name is only a stand-in for the symbol, not a device address, so the
// host asks the runtime for the real address once per device (cudaGetSymbolAddress, with that
// device current) and hands that pointer to the kernel.
//
// Consequences the caller must know:
//   * every GPU that loads this library holds SIM_NOALLOC_SCRATCH_BYTES (about 1.04 MiB) of
//     device memory until the process exits;
//   * the first call on a device performs the address look-up; make that first call outside any
//     stream capture;
//   * all calls on a device share the one array.  It keeps the previous call's contents, so each
//     call clears the part it uses before its first kernel; two calls whose work overlaps on the
//     GPU (different streams, or different host threads) race on it - serialise them;
//   * sizes beyond the fixed maximum are refused with SIM_ERR_ARG, nothing is launched.
#include "../../include/straggler_sim.h"

#include <cmath>
#include <mutex>
#include <string>

#include "device_rng.cuh"

namespace {

using namespace ssim;

constexpr int NA_MAX_REPLICAS = SIM_NOALLOC_MAX_REPLICAS;             // 4096
constexpr int NA_MAX_TASKS = SIM_NOALLOC_MAX_REPLICA_WORKERS;         // 65536 = replicas x P
constexpr size_t NA_OFF_F = 0;                                         // double [NA_MAX_TASKS]
constexpr size_t NA_OFF_S = NA_OFF_F + sizeof(double) * NA_MAX_TASKS;  // uint32 [NA_MAX_TASKS]
constexpr size_t NA_OFF_TAU = NA_OFF_S + sizeof(uint32_t) * NA_MAX_TASKS;
constexpr size_t NA_OFF_CLOCK = NA_OFF_TAU + sizeof(uint32_t) * NA_MAX_TASKS;   // double [NA_MAX_REPLICAS]
constexpr size_t NA_BYTES = NA_OFF_CLOCK + sizeof(double) * NA_MAX_REPLICAS;
static_assert(NA_BYTES <= SIM_NOALLOC_SCRATCH_BYTES, "scratch layout exceeds the stated size");

static __device__ __align__(256) unsigned char g_noalloc_scratch[SIM_NOALLOC_SCRATCH_BYTES];

thread_local std::string g_noalloc_error;

struct NaArgs {
  int variant, P, K_fixed, K0;
  double t_interval;
  DelayLaw law;
  uint64_t seed;
  int R;
  uint32_t replica_base;
  long long j0, iters, J;   // updates done before this launch, updates in this launch, row length of the outputs
  int K_stride;
  unsigned char* scratch;   // device address of g_noalloc_scratch
  double* t;
  uint16_t* K_used;
  uint16_t* worker;
  uint32_t* stale;
  uint32_t* seq;
};

__device__ __forceinline__ bool na_before(double va, int ia, double vb, int ib) {
  return va < vb || (va == vb && ia < ib);
}

// Variant of the arrival-process kernel: one warp per replica, one lane per worker, state carried
// between launches in the static scratch array instead of library-allocated buffers.  No version
// pool bookkeeping (there are no parameters in a clock-only run).
__global__ void __launch_bounds__(128) noalloc_schedule_kernel(NaArgs a) {
  const int lane = threadIdx.x & 31;
  const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (r >= a.R) return;
  const int P = a.P;
  const bool active = lane < P;
  const uint32_t rid = a.replica_base + (uint32_t)r;
  const bool async = a.variant == 2 || a.variant == 3;
  const double INF = __longlong_as_double(0x7FF0000000000000ll);
  double* st_f = reinterpret_cast<double*>(a.scratch + NA_OFF_F);
  uint32_t* st_s = reinterpret_cast<uint32_t*>(a.scratch + NA_OFF_S);
  uint32_t* st_tau = reinterpret_cast<uint32_t*>(a.scratch + NA_OFF_TAU);
  double* st_clock = reinterpret_cast<double*>(a.scratch + NA_OFF_CLOCK);

  uint32_t s = active ? st_s[r * P + lane] : 0u;
  uint32_t tau = active ? st_tau[r * P + lane] : 0u;
  double f = (active && async) ? st_f[r * P + lane] : INF;
  double clock = st_clock[r];
  if (async && a.j0 == 0 && active) {
    f = __dadd_rn(0.0, draw_delay(a.law, a.seed, rid, lane, s)); s += 1; tau = 0;
  }

  for (long long u = 0; u < a.iters; ++u) {
    const long long j = a.j0 + u;
    int K = a.K_fixed;
    if (a.t_interval > 0.0) {
      const double q = floor(__ddiv_rn(clock, a.t_interval));
      K = a.K0;
      for (double i = 0.0; i < q && K < P; i += 1.0) K *= 2;
      K = K < P ? K : P;
    }
    const long long row = (long long)r * a.J + j;
    uint16_t* wk = a.worker + row * a.K_stride;
    uint32_t* sl = a.stale + row * a.K_stride;
    uint32_t* sq = a.seq + row * a.K_stride;
    for (int l = lane; l < a.K_stride; l += 32)
      if (l >= K) { wk[l] = 0xFFFFu; sl[l] = 0xFFFFFFFFu; sq[l] = 0xFFFFFFFFu; }

    if (a.variant == 0 || a.variant == 2) {
      // K-sync: fresh draws, offsets from the iteration start; K-async: running finish times
      double v = INF;
      if (a.variant == 0) { if (active) { v = draw_delay(a.law, a.seed, rid, lane, s); s += 1; } }
      else v = f;
      int rank = 0;
      for (int o = 0; o < P; ++o) {
        const double vo = __shfl_sync(0xFFFFFFFFu, v, o);
        rank += na_before(vo, o, v, lane) ? 1 : 0;
      }
      const bool mine = active && rank < K;
      if (mine) {
        wk[rank] = (uint16_t)lane;
        sl[rank] = a.variant == 0 ? 0u : (uint32_t)(j - (long long)tau);
        sq[rank] = s - 1u;
      }
      const unsigned who = __ballot_sync(0xFFFFFFFFu, active && rank == K - 1);
      const double vK = __shfl_sync(0xFFFFFFFFu, v, __ffs(who) - 1);
      if (a.variant == 0) {
        clock = __dadd_rn(clock, vK);
      } else {
        clock = vK;
        if (mine) { tau = (uint32_t)(j + 1); f = __dadd_rn(clock, draw_delay(a.law, a.seed, rid, lane, s)); s += 1; }
      }
    } else {
      // the two batch variants: K rounds of "earliest finisher pushes and starts another minibatch"
      double c = f;
      if (a.variant == 1) { c = INF; if (active) { c = draw_delay(a.law, a.seed, rid, lane, s); s += 1; } }
      double last = 0.0;
      for (int l = 0; l < K; ++l) {
        double bv = c; int bi = lane;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
          const double ov = __shfl_xor_sync(0xFFFFFFFFu, bv, off);
          const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, off);
          if (na_before(ov, oi, bv, bi)) { bv = ov; bi = oi; }
        }
        last = bv;
        if (lane == bi) {
          wk[l] = (uint16_t)lane; sq[l] = s - 1u;
          if (a.variant == 1) {
            sl[l] = 0u;
            if (l + 1 < K) { c = __dadd_rn(c, draw_delay(a.law, a.seed, rid, lane, s)); s += 1; }
          } else {
            sl[l] = (uint32_t)(j - (long long)tau);
            tau = (l + 1 == K) ? (uint32_t)(j + 1) : (uint32_t)j;
            c = __dadd_rn(c, draw_delay(a.law, a.seed, rid, lane, s)); s += 1;
          }
        }
      }
      if (a.variant == 1) clock = __dadd_rn(clock, last);
      else { clock = last; f = c; }
    }
    if (lane == 0) { a.t[row] = clock; a.K_used[row] = (uint16_t)K; }
  }

  if (active) { st_s[r * P + lane] = s; st_tau[r * P + lane] = tau; if (async) st_f[r * P + lane] = f; }
  if (lane == 0) st_clock[r] = clock;
}

sim_status na_fail(sim_status st, const std::string& msg) {
  g_noalloc_error = msg;
  return st;
}

// Device address of the scratch array, looked up once per device.
constexpr int NA_MAX_DEVICES = 64;
std::mutex g_na_mutex;
unsigned char* g_na_ptr[NA_MAX_DEVICES] = {};

sim_status scratch_address(unsigned char** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return na_fail(SIM_ERR_CUDA, std::string("cudaGetDevice: ") + cudaGetErrorString(e));
  if (dev < 0 || dev >= NA_MAX_DEVICES) return na_fail(SIM_ERR_ARG, "device ordinal beyond 63");
  std::lock_guard<std::mutex> lock(g_na_mutex);
  if (!g_na_ptr[dev]) {
    unsigned char* p = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_noalloc_scratch);
    if (e != cudaSuccess || !p)
      return na_fail(SIM_ERR_CUDA, std::string("cudaGetSymbolAddress(scratch): ") + cudaGetErrorString(e));
    g_na_ptr[dev] = p;
  }
  *out = g_na_ptr[dev];
  return SIM_OK;
}

}  // namespace

extern "C" {

sim_status sim_schedule_noalloc(int32_t P, int32_t K, sim_variant variant, sim_delay delay, uint64_t seed,
                                int64_t replica_base, int32_t n_replicas, int32_t K0, double t_interval,
                                int64_t iters, double* t, uint16_t* K_used, uint16_t* worker,
                                uint32_t* stale, uint32_t* seq, void* cuda_stream) {
  if (P < 1 || P > SIM_NOALLOC_MAX_P) return na_fail(SIM_ERR_ARG, "P must be in [1, SIM_NOALLOC_MAX_P]");
  if ((int)variant < 0 || (int)variant > 3) return na_fail(SIM_ERR_ARG, "unknown variant");
  const bool growing = t_interval > 0.0;
  if (growing ? (K0 < 1 || K0 > P) : (K < 1 || K > P)) return na_fail(SIM_ERR_ARG, "K (or K0) must be in [1, P]");
  if (n_replicas < 1 || n_replicas > NA_MAX_REPLICAS)
    return na_fail(SIM_ERR_ARG, "n_replicas exceeds SIM_NOALLOC_MAX_REPLICAS (the fixed scratch array cannot hold more)");
  if ((int64_t)n_replicas * P > NA_MAX_TASKS)
    return na_fail(SIM_ERR_ARG, "n_replicas * P exceeds SIM_NOALLOC_MAX_REPLICA_WORKERS (the fixed scratch array cannot hold more)");
  if (iters < 1 || iters > ((int64_t)1 << 31)) return na_fail(SIM_ERR_ARG, "iters must be in [1, 2^31]");
  if (replica_base < 0 || replica_base + (int64_t)n_replicas > (int64_t)1 << 32)
    return na_fail(SIM_ERR_ARG, "global replica ids must fit in 32 bits");
  if (delay.kind != SIM_DELAY_EXP && delay.kind != SIM_DELAY_SHIFTED_EXP && delay.kind != SIM_DELAY_PARETO2)
    return na_fail(SIM_ERR_ARG, "unknown delay kind");
  if (delay.kind == SIM_DELAY_PARETO2 && !(delay.mu == 2.0 && delay.shift > 0.0 && std::isfinite(delay.shift)))
    return na_fail(SIM_ERR_ARG, "the Pareto law needs shape mu = 2 and a finite scale (shift) > 0");
  if (!(delay.mu > 0.0)) return na_fail(SIM_ERR_ARG, "delay rate mu must be > 0");
  if (delay.kind == SIM_DELAY_SHIFTED_EXP && !(delay.shift >= 0.0 && std::isfinite(delay.shift)))
    return na_fail(SIM_ERR_ARG, "delay shift must be finite and >= 0");
  if (!t || !K_used || !worker || !stale || !seq) return na_fail(SIM_ERR_ARG, "all five output buffers are required");

  unsigned char* scratch = nullptr;
  sim_status st = scratch_address(&scratch);
  if (st != SIM_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

  // the array still holds the previous call's state: everything this call reads must start at zero
  cudaError_t e = cudaMemsetAsync(scratch, 0, NA_BYTES, stream);
  if (e != cudaSuccess) return na_fail(SIM_ERR_CUDA, std::string("cudaMemsetAsync(scratch): ") + cudaGetErrorString(e));

  NaArgs a{};
  a.variant = (int)variant; a.P = P; a.K_fixed = K; a.K0 = growing ? K0 : 0; a.t_interval = growing ? t_interval : 0.0;
  a.law.kind = (int)delay.kind; a.law.mu = delay.mu; a.law.shift = delay.shift;
  a.seed = seed; a.R = n_replicas; a.replica_base = (uint32_t)replica_base; a.J = iters;
  a.K_stride = growing ? P : K; a.scratch = scratch;
  a.t = t; a.K_used = K_used; a.worker = worker; a.stale = stale; a.seq = seq;
  // long runs go out as several launches; the worker state crosses launches in the scratch array
  const long long chunk = 8192;
  for (long long j0 = 0; j0 < iters; j0 += chunk) {
    a.j0 = j0;
    a.iters = iters - j0 < chunk ? iters - j0 : chunk;
    noalloc_schedule_kernel<<<(n_replicas + 3) / 4, 128, 0, stream>>>(a);
    e = cudaGetLastError();
    if (e != cudaSuccess) return na_fail(SIM_ERR_CUDA, std::string("launch: ") + cudaGetErrorString(e));
  }
  return SIM_OK;
}

const char* sim_noalloc_last_error(void) { return g_noalloc_error.c_str(); }

}  // extern "C"
