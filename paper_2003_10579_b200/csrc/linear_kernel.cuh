// Gradient / update kernel for the single-output linear models (least squares, logistic).
//
// One CTA per replica walks the replica's schedule: for each update j, for each contributor l
// in arrival order, the m rows of its minibatch (indices re-derived from the Philox stream) are
// staged into shared memory by bulk asynchronous copies (one 4d-byte copy per row, completion
// counted on an mbarrier), several tiles ahead of the arithmetic - the rows never depend on w,
// so the row stream can be prefetched across contributor and update boundaries.  Per tile of T
// rows:   z_q = x_q . w_tau        (each thread owns a fixed set of columns; block reduction)
//         a_q = dl/dz(z_q, y_q)    (x.w - y, or sigmoid(x.w) - b)
//         g  += sum_q a_q x_q      (column owner accumulates, no reduction needed)
// and at the end of the update  w_{j+1} = w_j - (eta / (K m)) g   (Eq. 2 / Eq. 3), the minibatch
// loss and |w_{j+1} - w_ref|^2 are recorded.  w_j, w_tau and g live in registers; for the
// asynchronous variants every version is also written to the replica's version pool, from
// which stale snapshots w_tau are read back.
#pragma once
#include "schedule_kernel.cuh"

namespace ssim {

enum : int { M_NONE = 0, M_LSQ = 1, M_LOGISTIC = 2, M_SOFTMAX = 3, M_MLP2 = 4 };

struct NumericArgs {
  const float* X;            // [n][d]
  const void* y;             // [n] float targets (lsq) or int32 labels
  const float* w_ref;        // [n_params] or null
  uint64_t n;
  int d, m, model, n_classes;
  float eta;
  uint64_t seed;
  uint32_t replica_base;
  int R;
  long long j0, iters, cap;
  const long long* run_j0;   // optional per-replica [R] first update / update count of this launch (loss-driven K:
  const long long* run_iters; // replicas pause at different updates); null: j0 / iters for all
  int K_stride;
  int is_async;
  int n_slots;
  long long n_params;
  long long slot_stride;     // floats between versions in the pool: n_params rounded up to a multiple of 4
  const uint16_t* K_used;    // schedule, see schedule_kernel.cuh
  const uint16_t* worker;
  const uint32_t* seq;
  const uint8_t* snap_slot;
  const uint8_t* new_slot;
  const uint8_t* begin_slot; // [R] slot of w_{j0}
  float* loss;               // [R][cap]
  float* dist2;              // [R][cap]
  float* w_state;            // synchronous variants: [R][n_params]
  float* pool;               // asynchronous variants: [R][n_slots][n_params]
  int stages;                // shared-memory ring depth
  int* err;
};

// Where the MLP keeps element (k, n) of W1 inside a version of the pool.  The update kernel moves W1
// one 128-row x 32-column block at a time; stored block by block - [d/128][H/32][128][32] - a block is
// 16 KB contiguous (one bulk copy each way), a tile of the kernel a contiguous run of blocks.  Inside a
// row of a block the eight 16-byte pieces are XOR-swizzled with the row number, so that a thread per row
// reads its row from shared memory without bank conflicts.  Callers see the row-major order:
// sim_set_params / sim_get_params convert.
__host__ __device__ __forceinline__ long long w1_tiled_index(long long k, long long n, int H) {
  return (((k >> 7) * (H >> 5) + (n >> 5)) << 12) + ((k & 127) << 5) + (((((n & 31) >> 2) ^ (k & 7)) << 2) | (n & 3));
}

// ---- shared-memory barrier and bulk-copy primitives ------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: gives up after `limit` polls (the default is a few seconds' worth) and reports it.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t limit = 1u << 24) {
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (i > 4096) __nanosleep(128);
  }
  return false;
}
// After a wait has run out: before the block gives up its shared memory, give the row copies that are still in flight
// a bounded time to land.  At tile (st, parity) the producer is at most one ring ahead: stages st.. complete phase
// `parity`, stages below st the next one.  A stage that was never issued simply uses up its (short) limit.
__device__ __forceinline__ void drain_ring(uint64_t* full, int S, int st, uint32_t parity) {
  for (int s = 0; s < S; ++s) mbar_wait((uint32_t)__cvta_generic_to_shared(&full[s]), s >= st ? parity : parity ^ 1u, 1u << 14);
}
// global -> shared bulk copy of `bytes` (multiple of 16, both addresses 16-byte aligned)
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// 4-byte asynchronous copy whose completion is counted as one arrival on `bar`
__device__ __forceinline__ void word_g2s_arrive(uint32_t dst, const void* src, uint32_t bar) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
  return v;
}

// ---- the producer's walk over the schedule ---------------------------------------------------
enum : int { TILE_FIRST_OF_TASK = 1, TILE_LAST_OF_TASK = 2, TILE_LAST_OF_UPDATE = 4, TILE_LAST_OF_RUN = 8 };

struct TileInfo { int flags, rows, K, snap, fresh; };   // 5 ints per stage in shared memory

struct TaskDesc { uint32_t worker, seq, snap, fresh, K; };

struct ScheduleWalk {
  long long j, j_end, row0;   // current update, end of run, r * cap
  int l, k, tiles_per_task;
  TaskDesc cur, nxt;
  bool done;

  __device__ __forceinline__ TaskDesc load(const NumericArgs& a, long long jj, int ll) const {
    TaskDesc t;
    const long long row = row0 + jj;
    t.worker = a.worker[row * a.K_stride + ll];
    t.seq = a.seq[row * a.K_stride + ll];
    t.K = a.K_used[row];
    t.snap = a.is_async ? a.snap_slot[row * a.K_stride + ll] : 0u;
    t.fresh = a.is_async ? a.new_slot[row] : 0u;
    return t;
  }
  __device__ __forceinline__ void prefetch_next(const NumericArgs& a) {
    long long nj = j; int nl = l + 1;
    if (nl >= (int)cur.K) { nl = 0; nj = j + 1; }
    if (nj < j_end) nxt = load(a, nj, nl);
  }
  __device__ __forceinline__ void start(const NumericArgs& a, int r, long long first, long long count) {
    row0 = (long long)r * a.cap; j = first; j_end = first + count; l = 0; k = 0;
    tiles_per_task = (a.m + 0) ;   // set by caller (depends on T)
    done = count <= 0;
    if (!done) { cur = load(a, j, 0); prefetch_next(a); }
  }
  __device__ __forceinline__ void advance(const NumericArgs& a) {
    if (++k < tiles_per_task) return;
    k = 0;
    if (++l >= (int)cur.K) { l = 0; ++j; }
    if (j >= j_end) { done = true; return; }
    cur = nxt;
    prefetch_next(a);
  }
};

template <int NT, int CHUNKS, int T, bool ASYNC>
__global__ void __launch_bounds__(NT) linear1_kernel(NumericArgs a) {
  constexpr int NW = NT / 32;
  constexpr int E = 4 * CHUNKS;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r = blockIdx.x;
  const int d = a.d, d4 = d >> 2, S = a.stages, m = a.m;
  const uint32_t rid = a.replica_base + (uint32_t)r;
  const uint32_t row_bytes = (uint32_t)d * 4u;
  const long long my_j0 = a.run_j0 ? a.run_j0[r] : a.j0, my_iters = a.run_iters ? a.run_iters[r] : a.iters;

  extern __shared__ __align__(128) unsigned char smem[];
  // layout: [S] barriers | [S] TileInfo | y_stage [S][T] | red [2][NW][T] | misc [NW] | rows [S][T][d]
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);
  TileInfo* info_s = reinterpret_cast<TileInfo*>(smem + 8 * S);
  uint32_t* y_s = reinterpret_cast<uint32_t*>(info_s + S);
  float* red_s = reinterpret_cast<float*>((reinterpret_cast<uintptr_t>(y_s + S * T) + 15) & ~(uintptr_t)15);   // read as vectors
  float* misc_s = red_s + 2 * NW * T;
  const size_t head = (size_t)((unsigned char*)(misc_s + NW) - smem);
  float* rows_s = reinterpret_cast<float*>(smem + ((head + 127) & ~(size_t)127));
  uint32_t* pidx_s = reinterpret_cast<uint32_t*>(rows_s + (size_t)S * T * d);   // [m] sample rows of the producer's task

  // the row slots start as zeros: the long-row path reads every slot of a tile, also those a ragged tile leaves unfilled
  if (CHUNKS >= 4)
    for (int i = tid; i < S * T * d4; i += NT) reinterpret_cast<float4*>(rows_s)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (tid == 0) {
    for (int s = 0; s < S; ++s) mbar_init(smem_addr(&full[s]), (uint32_t)T + 1u);
    mbar_fence_init();
  }
  __syncthreads();

  // ---- parameters in registers: thread owns float4 chunks tid + NT*c ----
  float w_cur[E], w_tau[E], g[E];
  int cur_slot = ASYNC ? (int)a.begin_slot[r] : 0;
  {
    const float* src = ASYNC ? a.pool + ((size_t)r * a.n_slots + cur_slot) * (size_t)d
                             : a.w_state + (size_t)r * d;
#pragma unroll
    for (int c = 0; c < CHUNKS; ++c) {
      const int ci = tid + NT * c;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (ci < d4) v = reinterpret_cast<const float4*>(src)[ci];
      w_cur[4 * c] = v.x; w_cur[4 * c + 1] = v.y; w_cur[4 * c + 2] = v.z; w_cur[4 * c + 3] = v.w;
    }
#pragma unroll
    for (int e = 0; e < E; ++e) { g[e] = 0.f; w_tau[e] = w_cur[e]; }
  }

  // ---- producer (the last warp; thread 0 of the first records losses and distances): stage tiles of rows ahead of the
  //      arithmetic.  For the narrowest rows the block has one warp more than the columns need, so that drawing indices
  //      and issuing copies overlaps the arithmetic instead of taking turns with it ----
  ScheduleWalk walk;
  walk.done = true;
  int prod_st = 0;
  auto issue_tile = [&](long long) {
    // called by all lanes of the producer warp; the stage's previous contents have been consumed
    if (walk.done) return;
    const int st = prod_st;   // tiles are issued in order: a counter, not a 64-bit modulo per tile
    if (++prod_st == S) prod_st = 0;
    const uint32_t bar = smem_addr(&full[st]);
    const int rows = min(T, m - walk.k * T);
    if (walk.k == 0) {   // a new task: its m sample rows are drawn once, 32 at a time (only this warp uses the table)
      __syncwarp();
      for (int q = lane; q < m; q += 32) {
        uint32_t idx = draw_index(a.seed, rid, walk.cur.worker, walk.cur.seq, (uint32_t)q, a.n);
        if ((uint64_t)idx >= a.n) { atomicExch(a.err, ERR_BAD_INDEX); idx = 0; }
        pidx_s[q] = idx;
      }
      __syncwarp();
    }
    if (lane == 0) {
      TileInfo ti;
      ti.rows = rows; ti.K = (int)walk.cur.K; ti.snap = (int)walk.cur.snap; ti.fresh = (int)walk.cur.fresh;
      ti.flags = (walk.k == 0 ? TILE_FIRST_OF_TASK : 0) | (walk.k == walk.tiles_per_task - 1 ? TILE_LAST_OF_TASK : 0);
      if ((ti.flags & TILE_LAST_OF_TASK) && walk.l == (int)walk.cur.K - 1) {
        ti.flags |= TILE_LAST_OF_UPDATE;
        if (walk.j == walk.j_end - 1) ti.flags |= TILE_LAST_OF_RUN;
      }
      info_s[st] = ti;
      mbar_arrive_expect_tx(bar, (uint32_t)rows * row_bytes);
    }
    __syncwarp();
    if (lane < T) {
      if (lane < rows) {
        const uint32_t idx = pidx_s[walk.k * T + lane];
        bulk_g2s(smem_addr(rows_s + ((size_t)st * T + lane) * d), a.X + (size_t)idx * d, row_bytes, bar);
        word_g2s_arrive(smem_addr(&y_s[st * T + lane]), reinterpret_cast<const uint32_t*>(a.y) + idx, bar);
      } else {
        mbar_arrive(bar);
      }
    }
    walk.advance(a);
  };
  if (warp == NW - 1) {
    walk.start(a, r, my_j0, my_iters);
    walk.tiles_per_task = (m + T - 1) / T;
    for (int s = 0; s < S - 1; ++s) issue_tile(s);
  }
  __syncthreads();
  if (my_iters <= 0) return;

  float loss_acc = 0.f;
  long long j = my_j0;
  bool failed = false;
  int st = 0;             // stage and phase parity of tile `it`, kept as counters (it % S and it / S are 64-bit divisions)
  uint32_t parity = 0;
  for (long long it = 0;; ++it, parity ^= (uint32_t)(st + 1 == S), st = (st + 1 == S ? 0 : st + 1)) {
    // A thread whose wait runs out does not leave: the others may already be on their way to the tile's block barrier.
    // It stops waiting for good and follows the block through the rest of the run in step - same barriers, arithmetic on
    // whatever the stages hold - and reports at the end.  The control flow cannot split: it is steered by the tile's
    // descriptor, which the producer wrote at least one block barrier before any thread reads it, whether or not the
    // tile's copies ever land; so all threads of the block take the same branches by construction.
    const bool ok = !failed && mbar_wait(smem_addr(&full[st]), parity);
    failed = failed || !ok;
    const TileInfo ti = info_s[st];
    const float* tile = rows_s + (size_t)st * T * d;

    if (ASYNC && (ti.flags & TILE_FIRST_OF_TASK)) {
      if (ti.snap == cur_slot) {
#pragma unroll
        for (int e = 0; e < E; ++e) w_tau[e] = w_cur[e];
      } else {
        const float4* src = reinterpret_cast<const float4*>(a.pool + ((size_t)r * a.n_slots + ti.snap) * (size_t)d);
#pragma unroll
        for (int c = 0; c < CHUNKS; ++c) {
          const int ci = tid + NT * c;
          float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
          if (ci < d4) v = src[ci];
          w_tau[4 * c] = v.x; w_tau[4 * c + 1] = v.y; w_tau[4 * c + 2] = v.z; w_tau[4 * c + 3] = v.w;
        }
      }
    }

    // ---- z_q = x_q . w_tau: per-thread partial over own columns, then block reduction ----
    // Long rows (four chunks a thread) take both passes branch-free over rows and columns: a chunk index past
    // the row is clamped (its weights are zero and its gradient is never stored), and every row slot of the tile
    // is read (slots start as zeros; a row a ragged tile does not have gets a_q = 0).  Measured: +8 % on
    // 4096-feature rows, -5 % on 1024-feature rows (the compiler then hoists more loads than five CTAs per SM
    // leave registers for), hence the switch.
    constexpr bool BF = CHUNKS >= 4;
    float part[T];
#pragma unroll
    for (int q = 0; q < T; ++q) part[q] = 0.f;
    const float4* tile4 = reinterpret_cast<const float4*>(tile);
#pragma unroll
    for (int c = 0; c < CHUNKS; ++c) {
      const int ci = BF ? min(tid + NT * c, d4 - 1) : tid + NT * c;
      if (BF || ci < d4) {
#pragma unroll
        for (int q = 0; q < T; ++q) {
          if (BF || q < ti.rows) {
            const float4 x = tile4[q * d4 + ci];
            const float* wt = ASYNC ? &w_tau[4 * c] : &w_cur[4 * c];
            part[q] = fmaf(x.x, wt[0], part[q]);
            part[q] = fmaf(x.y, wt[1], part[q]);
            part[q] = fmaf(x.z, wt[2], part[q]);
            part[q] = fmaf(x.w, wt[3], part[q]);
          }
        }
      }
    }
#pragma unroll
    for (int q = 0; q < T; ++q) part[q] = warp_sum(part[q]);
    if (lane == 0) {
#pragma unroll
      for (int q = 0; q < T; ++q) red_s[((it & 1) * NW + warp) * T + q] = part[q];
    }
    __syncthreads();
    // every thread is past its reads of the previous tile's stage: refill it
    if (warp == NW - 1) issue_tile(it + S - 1);

    // ---- a_q = dl/dz and the loss ----
    float aq[T], zq[T];
#pragma unroll
    for (int q = 0; q < T; ++q) zq[q] = 0.f;
    {   // the warps' partial sums of all T rows, a vector load per warp
      constexpr int V = T % 4 == 0 ? 4 : 2;
      static_assert(T % 2 == 0, "tile rows are read in pairs");
      const float* rp = red_s + (it & 1) * NW * T;
#pragma unroll
      for (int w = 0; w < NW; ++w) {
#pragma unroll
        for (int q = 0; q < T; q += V) {
          if (V == 4) {
            const float4 v = *reinterpret_cast<const float4*>(rp + w * T + q);
            zq[q] += v.x; zq[q + 1] += v.y; zq[q + 2] += v.z; zq[q + 3] += v.w;
          } else {
            const float2 v = *reinterpret_cast<const float2*>(rp + w * T + q);
            zq[q] += v.x; zq[q + 1] += v.y;
          }
        }
      }
    }
#pragma unroll
    for (int q = 0; q < T; ++q) {
      aq[q] = 0.f;
      if (q < ti.rows) {
        const float z = zq[q];
        const uint32_t yraw = y_s[st * T + q];
        if (a.model == M_LSQ) {
          const float res = z - __uint_as_float(yraw);
          aq[q] = res;
          loss_acc = fmaf(0.5f * res, res, loss_acc);
        } else {  // logistic, label b in {0,1}: f = softplus(z) - b z, df/dz = sigmoid(z) - b
          const float b = (float)(int)yraw;
          const float ez = expf(-fabsf(z));
          // sigmoid(z) - b without cancellation: sigma - 1 is formed directly for b = 1
          const float inv = __frcp_rn(1.f + ez);   // the correctly rounded 1 / (1 + ez), without the division's slow path
          const float sig = z >= 0.f ? inv : ez * inv;
          const float sig_m1 = z >= 0.f ? -ez * inv : -inv;
          aq[q] = b != 0.f ? sig_m1 : sig;
          if (tid == 0) loss_acc += fmaxf(z, 0.f) + log1pf(ez) - b * z;   // only thread 0 records the loss
        }
      }
    }
    // ---- g += sum_q a_q x_q over own columns ----
#pragma unroll
    for (int c = 0; c < CHUNKS; ++c) {
      const int ci = BF ? min(tid + NT * c, d4 - 1) : tid + NT * c;
      if (BF || ci < d4) {
#pragma unroll
        for (int q = 0; q < T; ++q) {
          if (BF || q < ti.rows) {
            const float4 x = tile4[q * d4 + ci];
            g[4 * c] = fmaf(aq[q], x.x, g[4 * c]);
            g[4 * c + 1] = fmaf(aq[q], x.y, g[4 * c + 1]);
            g[4 * c + 2] = fmaf(aq[q], x.z, g[4 * c + 2]);
            g[4 * c + 3] = fmaf(aq[q], x.w, g[4 * c + 3]);
          }
        }
      }
    }

    if (ti.flags & TILE_LAST_OF_UPDATE) {
      // w_{j+1} = w_j - (eta / (K m)) sum of the K m per-sample gradients
      const float scale = (float)((double)a.eta / ((double)ti.K * (double)m));
      float dd = 0.f;
#pragma unroll
      for (int c = 0; c < CHUNKS; ++c) {
        const int ci = tid + NT * c;
        if (ci < d4) {
#pragma unroll
          for (int e = 0; e < 4; ++e) { w_cur[4 * c + e] = fmaf(-scale, g[4 * c + e], w_cur[4 * c + e]); g[4 * c + e] = 0.f; }
          if (ASYNC) {
            float4* dst = reinterpret_cast<float4*>(a.pool + ((size_t)r * a.n_slots + ti.fresh) * (size_t)d);
            dst[ci] = make_float4(w_cur[4 * c], w_cur[4 * c + 1], w_cur[4 * c + 2], w_cur[4 * c + 3]);
          }
          if (a.w_ref) {
            const float4 wr = reinterpret_cast<const float4*>(a.w_ref)[ci];
            const float e0 = w_cur[4 * c] - wr.x, e1 = w_cur[4 * c + 1] - wr.y, e2 = w_cur[4 * c + 2] - wr.z, e3 = w_cur[4 * c + 3] - wr.w;
            dd = fmaf(e0, e0, dd); dd = fmaf(e1, e1, dd); dd = fmaf(e2, e2, dd); dd = fmaf(e3, e3, dd);
          }
        }
      }
      if (ASYNC) cur_slot = ti.fresh;
      if (a.w_ref) {
        dd = warp_sum(dd);
        if (lane == 0) misc_s[warp] = dd;
        __syncthreads();
        if (tid == 0) {
          float tot = 0.f;
          for (int w = 0; w < NW; ++w) tot += misc_s[w];
          a.dist2[(size_t)r * a.cap + j] = tot;
        }
      } else if (tid == 0) {
        a.dist2[(size_t)r * a.cap + j] = 0.f;
      }
      if (tid == 0) a.loss[(size_t)r * a.cap + j] = loss_acc / ((float)ti.K * (float)m);
      loss_acc = 0.f;
      ++j;
    }
    if (ti.flags & TILE_LAST_OF_RUN) break;
  }

  if (failed) {
    if (tid == 0) {
      atomicExch(a.err, ERR_WAIT_TIMEOUT);
      drain_ring(full, S, st, parity);
    }
    __syncthreads();
    return;
  }
  if (!ASYNC) {
    float4* dst = reinterpret_cast<float4*>(a.w_state + (size_t)r * d);
#pragma unroll
    for (int c = 0; c < CHUNKS; ++c) {
      const int ci = tid + NT * c;
      if (ci < d4) dst[ci] = make_float4(w_cur[4 * c], w_cur[4 * c + 1], w_cur[4 * c + 2], w_cur[4 * c + 3]);
    }
  }
}

// shared-memory bytes of linear1_kernel for a given shape
inline size_t linear1_smem_bytes(int NT, int T, int S, int d, int m) {
  size_t head = 8 * (size_t)S + sizeof(TileInfo) * (size_t)S + 4 * (size_t)S * T + 16 + 4 * (size_t)2 * (NT / 32) * T + 4 * (size_t)(NT / 32);
  head = (head + 127) & ~(size_t)127;
  return head + (size_t)S * T * d * 4 + (size_t)m * 4;
}

}  // namespace ssim
