// Arrival process of the four SGD variants of Section 2.2: one warp per replica, one lane per
// worker (P <= 32).  The process depends on the delay stream only, never on parameter values,
// so it runs ahead of the numeric kernels and leaves them a compact schedule:
//   per update j: clock t_{j+1} (fp64), K_j, and for each contributor in arrival order its
//   worker id, task sequence number, staleness j - tau and (asynchronous variants) the slot of
//   the version pool that holds the parameters it fetched, plus the slot w_{j+1} is written to.
//
// Selection is exact: the K smallest of (time, worker id) by an all-pairs rank over the warp
// (K-sync, K-async) or K rounds of a warp arg-min with redraw (the two batch variants).
#pragma once
#include "device_rng.cuh"

namespace ssim {

enum : int { V_KSYNC = 0, V_KBATCHSYNC = 1, V_KASYNC = 2, V_KBATCHASYNC = 3 };
enum : int { ERR_NONE = 0, ERR_WAIT_TIMEOUT = 1, ERR_NO_FREE_SLOT = 2, ERR_BAD_INDEX = 3 };

struct ScheduleArgs {
  int variant, P, K_fixed, K0;
  double t_interval;
  DelayLaw law;
  uint64_t seed;
  int R;
  uint32_t replica_base;
  long long j0, iters;       // updates already done, updates to do now
  long long cap;             // trace capacity in updates (row stride)
  int K_stride;              // contributors per trace row
  int n_slots;               // version-pool slots per replica (asynchronous variants)
  // per-replica state
  uint32_t* s;               // [R][P] tasks launched by each worker
  uint32_t* tau;             // [R][P] version each worker last fetched
  double* f;                 // [R][P] absolute finish time of the running task
  uint8_t* wslot;            // [R][P] pool slot of the version each worker holds
  uint8_t* cur_slot;         // [R]    pool slot of w_j
  uint8_t* begin_slot;       // [R]    pool slot of w_{j0} (what cur_slot was when this launch began)
  double* clock;             // [R]    simulated time of the last update
  // trace
  double* t;                 // [R][cap]
  uint16_t* K_used;          // [R][cap]
  uint16_t* worker;          // [R][cap][K_stride]
  uint32_t* stale;
  uint32_t* seq;
  uint8_t* snap_slot;        // [R][cap][K_stride] (asynchronous variants, else null)
  uint8_t* new_slot;         // [R][cap]
  int* err;
  // loss-driven K (Algorithm 1): a replica's K changes only when an update starts in a later interval
  // than the one K was last set in; the arrival process then pauses there until the risk is known
  int adaptive;
  long long target;          // every replica is advanced to this many updates in total
  long long* done;           // [R] updates scheduled so far
  long long* run_j0;         // [R] out: first update and number of updates scheduled by this launch
  long long* run_iters;
  int* K_cur;                // [R] K in force
  long long* q_last;         // [R] interval index K was last set in
  int* want_eval;            // [R] out: 1 if the replica paused because it needs a new K
};

// K in force for an update that starts at simulated time t (doubling once per elapsed interval).
__device__ __forceinline__ int k_for_time(const ScheduleArgs& a, double t) {
  if (!(a.t_interval > 0.0)) return a.K_fixed;
  const double q = floor(__ddiv_rn(t, a.t_interval));
  int K = a.K0;
  for (double i = 0.0; i < q && K < a.P; i += 1.0) K *= 2;
  return K < a.P ? K : a.P;
}

__device__ __forceinline__ bool before(double va, int ia, double vb, int ib) {
  return va < vb || (va == vb && ia < ib);
}

// number of workers that arrive strictly before (v, lane)
__device__ __forceinline__ int arrival_rank(double v, int lane, int P) {
  int rank = 0;
  for (int o = 0; o < P; ++o) {
    const double vo = __shfl_sync(0xFFFFFFFFu, v, o);
    rank += before(vo, o, v, lane) ? 1 : 0;
  }
  return rank;
}

__device__ __forceinline__ void warp_argmin(double v, int lane, double& bv, int& bi) {
  bv = v; bi = lane;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const double ov = __shfl_xor_sync(0xFFFFFFFFu, bv, off);
    const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, off);
    if (before(ov, oi, bv, bi)) { bv = ov; bi = oi; }
  }
}

__device__ __forceinline__ unsigned long long warp_or64(unsigned long long m) {
  const uint32_t lo = __reduce_or_sync(0xFFFFFFFFu, (uint32_t)m);
  const uint32_t hi = __reduce_or_sync(0xFFFFFFFFu, (uint32_t)(m >> 32));
  return ((unsigned long long)hi << 32) | lo;
}

__global__ void __launch_bounds__(128) schedule_kernel(ScheduleArgs a) {
  const int lane = threadIdx.x & 31;
  const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (r >= a.R) return;
  const int P = a.P;
  const bool active = lane < P;
  const uint32_t rid = a.replica_base + (uint32_t)r;
  const bool async = a.variant == V_KASYNC || a.variant == V_KBATCHASYNC;
  const double INF = __longlong_as_double(0x7FF0000000000000ll);

  uint32_t s = active ? a.s[r * P + lane] : 0u;
  uint32_t tau = active ? a.tau[r * P + lane] : 0u;
  double f = (active && async) ? a.f[r * P + lane] : INF;
  int slot = (active && async) ? a.wslot[r * P + lane] : 0;
  int cur = async ? a.cur_slot[r] : 0;
  double clock = a.clock[r];

  long long j = a.adaptive ? a.done[r] : a.j0;
  const long long j_begin = j, j_end = a.adaptive ? a.target : a.j0 + a.iters;
  int K_now = a.adaptive ? a.K_cur[r] : 0, want = 0;
  long long q_last = a.adaptive ? a.q_last[r] : 0;
  if (async && j == 0 && __all_sync(0xFFFFFFFFu, s == 0u)) {   // every worker fetches w_0 and starts its first minibatch at t = 0
    if (active) { f = __dadd_rn(0.0, draw_delay(a.law, a.seed, rid, lane, s)); s += 1; tau = 0; slot = 0; }
    cur = 0;
  }
  if (async && lane == 0) a.begin_slot[r] = (uint8_t)cur;

  for (; j < j_end; ++j) {
    int K;
    if (a.adaptive) {
      const double qd = floor(__ddiv_rn(clock, a.t_interval));
      const long long q = qd > 9.0e18 ? 0x7FFFFFFFFFFFFFFFll : (long long)qd;
      if (q > q_last) {
        if (K_now < P) { want = 1; break; }     // the risk of w_j decides the next K
        q_last = q;
      }
      K = K_now;
    } else {
      K = k_for_time(a, clock);
    }
    const long long row = (long long)r * a.cap + j;
    uint16_t* wk = a.worker + row * a.K_stride;
    uint32_t* sl = a.stale + row * a.K_stride;
    uint32_t* sq = a.seq + row * a.K_stride;
    uint8_t* ss = async ? a.snap_slot + row * a.K_stride : nullptr;
    for (int l = lane; l < a.K_stride; l += 32) {
      if (l >= K) { wk[l] = 0xFFFFu; sl[l] = 0xFFFFFFFFu; sq[l] = 0xFFFFFFFFu; if (ss) ss[l] = 0xFF; }
    }

    if (a.variant == V_KSYNC) {
      double x = INF;
      if (active) { x = draw_delay(a.law, a.seed, rid, lane, s); s += 1; }
      const int rank = arrival_rank(x, lane, P);
      if (active && rank < K) { wk[rank] = (uint16_t)lane; sl[rank] = 0u; sq[rank] = s - 1u; }
      const unsigned who = __ballot_sync(0xFFFFFFFFu, active && rank == K - 1);
      const double T = __shfl_sync(0xFFFFFFFFu, x, __ffs(who) - 1);
      clock = __dadd_rn(clock, T);
    } else if (a.variant == V_KBATCHSYNC) {
      double c = INF;
      if (active) { c = draw_delay(a.law, a.seed, rid, lane, s); s += 1; }
      double T = 0.0;
      for (int l = 0; l < K; ++l) {
        double bv; int bi;
        warp_argmin(c, lane, bv, bi);
        T = bv;
        if (lane == bi) {
          wk[l] = (uint16_t)lane; sl[l] = 0u; sq[l] = s - 1u;
          if (l + 1 < K) { c = __dadd_rn(c, draw_delay(a.law, a.seed, rid, lane, s)); s += 1; }
        }
      }
      clock = __dadd_rn(clock, T);
    } else if (a.variant == V_KASYNC) {
      const int rank = arrival_rank(f, lane, P);
      const bool mine = active && rank < K;
      if (mine) { wk[rank] = (uint16_t)lane; sl[rank] = (uint32_t)(j - (long long)tau); sq[rank] = s - 1u; ss[rank] = (uint8_t)slot; }
      const unsigned who = __ballot_sync(0xFFFFFFFFu, active && rank == K - 1);
      clock = __shfl_sync(0xFFFFFFFFu, f, __ffs(who) - 1);
      // w_{j+1} goes to a slot that no worker holds and that is not w_j
      const unsigned long long used = warp_or64(active ? (1ull << slot) : 0ull) | (1ull << cur);
      int fresh = __ffsll((long long)~used) - 1;
      if (fresh < 0 || fresh >= a.n_slots) { if (lane == 0) atomicExch(a.err, ERR_NO_FREE_SLOT); fresh = 0; }
      if (lane == 0) a.new_slot[row] = (uint8_t)fresh;
      if (mine) {
        tau = (uint32_t)(j + 1); slot = fresh;
        f = __dadd_rn(clock, draw_delay(a.law, a.seed, rid, lane, s)); s += 1;
      }
      cur = fresh;
    } else {  // V_KBATCHASYNC
      unsigned long long read_now = 0ull;   // slots whose parameters this update's gradients read
      for (int l = 0; l < K; ++l) {
        double bv; int bi;
        warp_argmin(f, lane, bv, bi);
        const int bslot = __shfl_sync(0xFFFFFFFFu, slot, bi);
        read_now |= 1ull << bslot;
        int fresh = cur;
        if (l + 1 == K) {
          clock = bv;
          const unsigned long long used = warp_or64(active ? (1ull << slot) : 0ull) | (1ull << cur) | read_now;
          fresh = __ffsll((long long)~used) - 1;
          if (fresh < 0 || fresh >= a.n_slots) { if (lane == 0) atomicExch(a.err, ERR_NO_FREE_SLOT); fresh = 0; }
          if (lane == 0) a.new_slot[row] = (uint8_t)fresh;
        }
        if (lane == bi) {
          wk[l] = (uint16_t)lane; sl[l] = (uint32_t)(j - (long long)tau); sq[l] = s - 1u; ss[l] = (uint8_t)slot;
          // the pusher fetches what the server holds after its push was counted
          tau = (l + 1 == K) ? (uint32_t)(j + 1) : (uint32_t)j;
          slot = fresh;
          f = __dadd_rn(f, draw_delay(a.law, a.seed, rid, lane, s)); s += 1;
        }
        if (l + 1 == K) cur = fresh;
      }
    }
    if (lane == 0) { a.t[row] = clock; a.K_used[row] = (uint16_t)K; }
  }

  if (active) {
    a.s[r * P + lane] = s;
    a.tau[r * P + lane] = tau;
    if (async) { a.f[r * P + lane] = f; a.wslot[r * P + lane] = (uint8_t)slot; }
  }
  if (lane == 0) {
    a.clock[r] = clock;
    if (async) a.cur_slot[r] = (uint8_t)cur;
    if (a.adaptive) {
      a.run_j0[r] = j_begin; a.run_iters[r] = j - j_begin; a.done[r] = j;
      a.q_last[r] = q_last; a.want_eval[r] = want;
    }
  }
}

// After the risk of the paused replicas is known: the rule of Section 6 / Algorithm 1.
//   K-batch-sync, K-async, K-batch-async:  K = K0 sqrt(F(w_0) / F(w_start))
//   K-sync:  K^2 / (P - K) = K0^2 / (P - K0) * F(w_0) / F(w_start)   (positive root)
// rounded half up, never decreasing, at most P; F <= 0 (F* reached) gives P.  fp64 with explicit
// round-to-nearest operations on the fp32 risks, so that the integer is reproducible elsewhere.
__global__ void adasync_update_kernel(int variant, int P, int K0, double t_interval, int R, long long target,
                                      const float* F0, const float* F, const double* clock, const long long* done,
                                      int* K_cur, long long* q_last, int* want_eval, int* remaining) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= R) return;
  if (want_eval[r]) {
    const double f0 = (double)F0[r], f = (double)F[r];
    int K = P;
    if (f > 0.0 && isfinite(f) && isfinite(f0)) {
      const double ratio = __ddiv_rn(f0, f);
      double k_real;
      if (variant == V_KSYNC) {
        if (K0 >= P) k_real = (double)P;
        else {
          const double c = __dmul_rn(__ddiv_rn((double)(K0 * K0), (double)(P - K0)), ratio);
          const double disc = __dadd_rn(__dmul_rn(c, c), __dmul_rn(__dmul_rn(4.0, c), (double)P));
          k_real = __dmul_rn(__dadd_rn(__dsqrt_rn(disc), -c), 0.5);
        }
      } else {
        k_real = __dmul_rn((double)K0, __dsqrt_rn(ratio));
      }
      K = k_real < 1e9 ? (int)floor(__dadd_rn(k_real, 0.5)) : P;
    }
    const int prev = K_cur[r];
    K = K < prev ? prev : K;
    K_cur[r] = K > P ? P : K;
    const double qd = floor(__ddiv_rn(clock[r], t_interval));
    q_last[r] = qd > 9.0e18 ? 0x7FFFFFFFFFFFFFFFll : (long long)qd;
    want_eval[r] = 0;
  }
  if (done[r] < target) atomicAdd(remaining, 1);
}

// The raw draws, for checking the stream against another implementation.
__global__ void draw_delays_kernel(DelayLaw law, uint64_t seed, uint32_t replica_base, int R, int P,
                                   int n_seq, double* out) {
  const long long total = (long long)R * P * n_seq;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int sq = (int)(i % n_seq);
    const int w = (int)((i / n_seq) % P);
    const int r = (int)(i / ((long long)n_seq * P));
    out[i] = draw_delay(law, seed, replica_base + (uint32_t)r, (uint32_t)w, (uint32_t)sq);
  }
}

__global__ void draw_indices_kernel(uint64_t seed, uint32_t replica_base, int R, int P, int n_seq,
                                    uint64_t n, int m, uint32_t* out) {
  const long long total = (long long)R * P * n_seq * m;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int q = (int)(i % m);
    const long long task = i / m;
    const int sq = (int)(task % n_seq);
    const int w = (int)((task / n_seq) % P);
    const int r = (int)(task / ((long long)n_seq * P));
    out[i] = draw_index(seed, replica_base + (uint32_t)r, (uint32_t)w, (uint32_t)sq, (uint32_t)q, n);
  }
}

}  // namespace ssim
