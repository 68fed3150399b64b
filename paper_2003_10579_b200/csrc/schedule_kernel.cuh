// Arrival process of the four SGD variants of Section 2.2: one warp per replica, one lane per
// worker for P <= 32, two or four workers per lane for P <= 64 / P <= 128.  The process depends on the delay stream only, never on parameter values,
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

// Lane `lane` owns workers lane, lane + 32, ..., lane + 32 (I - 1): I = 1 for P <= 32, 2 for P <= 64,
// 4 for P <= 128.  Everything below is unrolled over the I items, so I = 1 is the one-lane-per-worker code.

// rank[i] = number of workers that arrive strictly before worker lane + 32 i
template <int I>
__device__ __forceinline__ void arrival_ranks(const double (&v)[I], int lane, int P, int (&rank)[I]) {
#pragma unroll
  for (int i = 0; i < I; ++i) rank[i] = 0;
#pragma unroll
  for (int ob = 0; ob < I; ++ob) {
    for (int o = 0; o < 32 && ob * 32 + o < P; ++o) {
      const double vo = __shfl_sync(0xFFFFFFFFu, v[ob], o);
#pragma unroll
      for (int i = 0; i < I; ++i) rank[i] += before(vo, ob * 32 + o, v[i], lane + 32 * i) ? 1 : 0;
    }
  }
}

// value and worker id of the earliest (time, id) over all workers of the warp
template <int I>
__device__ __forceinline__ void warp_argmin(const double (&v)[I], int lane, double& bv, int& bi) {
  bv = v[0]; bi = lane;
#pragma unroll
  for (int i = 1; i < I; ++i)
    if (before(v[i], lane + 32 * i, bv, bi)) { bv = v[i]; bi = lane + 32 * i; }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const double ov = __shfl_xor_sync(0xFFFFFFFFu, bv, off);
    const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, off);
    if (before(ov, oi, bv, bi)) { bv = ov; bi = oi; }
  }
}

// the value item `id >> 5` of lane `id & 31` holds
template <int I>
__device__ __forceinline__ int item_of_worker(const int (&x)[I], int id) {
  int out = 0;
#pragma unroll
  for (int i = 0; i < I; ++i) {
    const int t = __shfl_sync(0xFFFFFFFFu, x[i], id & 31);
    if ((id >> 5) == i) out = t;
  }
  return out;
}
template <int I>
__device__ __forceinline__ double item_of_worker(const double (&x)[I], int id) {
  double out = 0.0;
#pragma unroll
  for (int i = 0; i < I; ++i) {
    const double t = __shfl_sync(0xFFFFFFFFu, x[i], id & 31);
    if ((id >> 5) == i) out = t;
  }
  return out;
}

// Set of version-pool slots (at most 32 I + 2 of them) as I + 1 words.
template <int I>
struct SlotSet {
  uint32_t w[I + 1];
  __device__ __forceinline__ void clear() {
#pragma unroll
    for (int k = 0; k <= I; ++k) w[k] = 0u;
  }
  __device__ __forceinline__ void add(int slot) {
#pragma unroll
    for (int k = 0; k <= I; ++k) if ((slot >> 5) == k) w[k] |= 1u << (slot & 31);
  }
  __device__ __forceinline__ void warp_union() {
#pragma unroll
    for (int k = 0; k <= I; ++k) w[k] = __reduce_or_sync(0xFFFFFFFFu, w[k]);
  }
  __device__ __forceinline__ void join(const SlotSet& o) {
#pragma unroll
    for (int k = 0; k <= I; ++k) w[k] |= o.w[k];
  }
  __device__ __forceinline__ int first_free() const {     // lowest slot not in the set, or 32 (I + 1)
    int out = 32 * (I + 1);
#pragma unroll
    for (int k = I; k >= 0; --k) if (~w[k]) out = 32 * k + __ffs((int)~w[k]) - 1;
    return out;
  }
};

template <int I>
__global__ void __launch_bounds__(128) schedule_kernel(ScheduleArgs a) {
  const int lane = threadIdx.x & 31;
  const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (r >= a.R) return;
  const int P = a.P;
  const uint32_t rid = a.replica_base + (uint32_t)r;
  const bool async = a.variant == V_KASYNC || a.variant == V_KBATCHASYNC;
  const double INF = __longlong_as_double(0x7FF0000000000000ll);

  bool active[I];
  uint32_t s[I], tau[I];
  double f[I];
  int slot[I];
  bool fresh_start = true;
#pragma unroll
  for (int i = 0; i < I; ++i) {
    const int id = lane + 32 * i;
    active[i] = id < P;
    s[i] = active[i] ? a.s[r * P + id] : 0u;
    tau[i] = active[i] ? a.tau[r * P + id] : 0u;
    f[i] = (active[i] && async) ? a.f[r * P + id] : INF;
    slot[i] = (active[i] && async) ? a.wslot[r * P + id] : 0;
    fresh_start = fresh_start && s[i] == 0u;
  }
  int cur = async ? a.cur_slot[r] : 0;
  double clock = a.clock[r];

  long long j = a.adaptive ? a.done[r] : a.j0;
  const long long j_begin = j, j_end = a.adaptive ? a.target : a.j0 + a.iters;
  int K_now = a.adaptive ? a.K_cur[r] : 0, want = 0;
  long long q_last = a.adaptive ? a.q_last[r] : 0;
  if (async && j == 0 && __all_sync(0xFFFFFFFFu, fresh_start)) {   // every worker fetches w_0 and starts its first minibatch at t = 0
#pragma unroll
    for (int i = 0; i < I; ++i)
      if (active[i]) { f[i] = __dadd_rn(0.0, draw_delay(a.law, a.seed, rid, lane + 32 * i, s[i])); s[i] += 1; tau[i] = 0; slot[i] = 0; }
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
      double x[I];
      int rank[I];
#pragma unroll
      for (int i = 0; i < I; ++i) {
        x[i] = INF;
        if (active[i]) { x[i] = draw_delay(a.law, a.seed, rid, lane + 32 * i, s[i]); s[i] += 1; }
      }
      arrival_ranks<I>(x, lane, P, rank);
      double T = 0.0;
#pragma unroll
      for (int i = 0; i < I; ++i) {
        if (active[i] && rank[i] < K) { wk[rank[i]] = (uint16_t)(lane + 32 * i); sl[rank[i]] = 0u; sq[rank[i]] = s[i] - 1u; }
        const unsigned who = __ballot_sync(0xFFFFFFFFu, active[i] && rank[i] == K - 1);
        const double Ti = __shfl_sync(0xFFFFFFFFu, x[i], who ? __ffs(who) - 1 : 0);
        if (who) T = Ti;
      }
      clock = __dadd_rn(clock, T);
    } else if (a.variant == V_KBATCHSYNC) {
      double c[I];
#pragma unroll
      for (int i = 0; i < I; ++i) {
        c[i] = INF;
        if (active[i]) { c[i] = draw_delay(a.law, a.seed, rid, lane + 32 * i, s[i]); s[i] += 1; }
      }
      double T = 0.0;
      for (int l = 0; l < K; ++l) {
        double bv; int bi;
        warp_argmin<I>(c, lane, bv, bi);
        T = bv;
#pragma unroll
        for (int i = 0; i < I; ++i) {
          if (bi == lane + 32 * i) {
            wk[l] = (uint16_t)bi; sl[l] = 0u; sq[l] = s[i] - 1u;
            if (l + 1 < K) { c[i] = __dadd_rn(c[i], draw_delay(a.law, a.seed, rid, bi, s[i])); s[i] += 1; }
          }
        }
      }
      clock = __dadd_rn(clock, T);
    } else if (a.variant == V_KASYNC) {
      int rank[I];
      arrival_ranks<I>(f, lane, P, rank);
      bool mine[I];
      double t_new = 0.0;
      SlotSet<I> used;
      used.clear();
#pragma unroll
      for (int i = 0; i < I; ++i) {
        mine[i] = active[i] && rank[i] < K;
        if (mine[i]) {
          wk[rank[i]] = (uint16_t)(lane + 32 * i); sl[rank[i]] = (uint32_t)(j - (long long)tau[i]); sq[rank[i]] = s[i] - 1u;
          ss[rank[i]] = (uint8_t)slot[i];
        }
        const unsigned who = __ballot_sync(0xFFFFFFFFu, active[i] && rank[i] == K - 1);
        const double ti = __shfl_sync(0xFFFFFFFFu, f[i], who ? __ffs(who) - 1 : 0);
        if (who) t_new = ti;
        if (active[i]) used.add(slot[i]);
      }
      clock = t_new;
      // w_{j+1} goes to a slot that no worker holds and that is not w_j
      used.warp_union();
      used.add(cur);
      int fresh = used.first_free();
      if (fresh >= a.n_slots) { if (lane == 0) atomicExch(a.err, ERR_NO_FREE_SLOT); fresh = 0; }
      if (lane == 0) a.new_slot[row] = (uint8_t)fresh;
#pragma unroll
      for (int i = 0; i < I; ++i) {
        if (mine[i]) {
          tau[i] = (uint32_t)(j + 1); slot[i] = fresh;
          f[i] = __dadd_rn(clock, draw_delay(a.law, a.seed, rid, lane + 32 * i, s[i])); s[i] += 1;
        }
      }
      cur = fresh;
    } else {  // V_KBATCHASYNC
      SlotSet<I> read_now;                  // slots whose parameters this update's gradients read
      read_now.clear();
      for (int l = 0; l < K; ++l) {
        double bv; int bi;
        warp_argmin<I>(f, lane, bv, bi);
        const int bslot = item_of_worker<I>(slot, bi);
        read_now.add(bslot);
        int fresh = cur;
        if (l + 1 == K) {
          clock = bv;
          SlotSet<I> used;
          used.clear();
#pragma unroll
          for (int i = 0; i < I; ++i) if (active[i]) used.add(slot[i]);
          used.warp_union();
          used.add(cur);
          used.join(read_now);
          fresh = used.first_free();
          if (fresh >= a.n_slots) { if (lane == 0) atomicExch(a.err, ERR_NO_FREE_SLOT); fresh = 0; }
          if (lane == 0) a.new_slot[row] = (uint8_t)fresh;
        }
#pragma unroll
        for (int i = 0; i < I; ++i) {
          if (bi == lane + 32 * i) {
            wk[l] = (uint16_t)bi; sl[l] = (uint32_t)(j - (long long)tau[i]); sq[l] = s[i] - 1u; ss[l] = (uint8_t)slot[i];
            // the pusher fetches what the server holds after its push was counted
            tau[i] = (l + 1 == K) ? (uint32_t)(j + 1) : (uint32_t)j;
            slot[i] = fresh;
            f[i] = __dadd_rn(f[i], draw_delay(a.law, a.seed, rid, bi, s[i])); s[i] += 1;
          }
        }
        if (l + 1 == K) cur = fresh;
      }
    }
    if (lane == 0) { a.t[row] = clock; a.K_used[row] = (uint16_t)K; }
  }

#pragma unroll
  for (int i = 0; i < I; ++i) {
    const int id = lane + 32 * i;
    if (active[i]) {
      a.s[r * P + id] = s[i];
      a.tau[r * P + id] = tau[i];
      if (async) { a.f[r * P + id] = f[i]; a.wslot[r * P + id] = (uint8_t)slot[i]; }
    }
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

inline cudaError_t launch_schedule(const ScheduleArgs& a, cudaStream_t stream) {
  const int grid = (a.R + 3) / 4;
  if (a.P <= 32) schedule_kernel<1><<<grid, 128, 0, stream>>>(a);
  else if (a.P <= 64) schedule_kernel<2><<<grid, 128, 0, stream>>>(a);
  else schedule_kernel<4><<<grid, 128, 0, stream>>>(a);
  return cudaGetLastError();
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
