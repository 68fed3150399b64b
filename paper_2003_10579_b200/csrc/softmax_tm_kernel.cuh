// Gradient / update kernel for softmax regression with up to 10 classes, W in R^{C x d}: the
// parameters live in TENSOR MEMORY, not in shared memory.
//
// One CTA of NT = 128 NG threads per replica, same producer / schedule walk as the other numeric
// kernels (rows staged by bulk asynchronous copies, a ring of tiles of T = NG TG rows).
//
// Ownership.  The d/2 pairs of adjacent features are dealt to the threads: thread t owns pairs
// t + NT k (k < KP).  For its pairs and all classes it keeps the gradient accumulator G in registers
// for the whole update and the parameters W_tau in 20 KP columns of its own tensor-memory lane
// (lane t mod 128, columns 20 KP (t / 128) ...; column 20 k + 2 c + h holds W[c][feature h of pair k]).
// Tensor memory is used as a 120 KB register-file extension with its own read path: no MMA is issued.
// The update W <- W - (eta / (K m)) G (Eq. 2 / Eq. 3) is thread-local: tcgen05.ld, FMA, tcgen05.st.
//
// Per tile:
//   logits    Z = X_tile W_tau^T.  The NG thread groups of four warps take different rows (TG each);
//             thread (lane L of the 128, group g) walks the whole of tensor-memory lane L - the columns
//             of all NG owners - i.e. it covers 2 KP NG features of its rows.  Splitting the rows over
//             the groups divides the number of partial logits to reduce across threads by NG against a
//             mapping where every thread works on every row; one warp transposition reduce
//             (<= 31 shuffles for TG x 10 values) and a four-way sum in shared memory finish it.
//   softmax   D = softmax(Z) - onehot(label), loss: 16 lanes per row.
//   gradient  G += D^T X_tile: every thread, every row, own pairs, packed fp32x2 FMAs (the two
//             features of a pair); D is stored once and paired by register moves (see there).
// Plain fp32 FMAs: at 20 FMA per 4-byte feature this path sits at the fp32 ridge, and the 1e-5
// parity bound on the parameters rules out reduced-precision tensor-core operands.
#pragma once
#include "softmax_kernel.cuh"

#ifndef SMX_TM_NG
#define SMX_TM_NG 3
#endif
#ifndef SMX_TM_TG
#define SMX_TM_TG 3
#endif

namespace ssim {

constexpr int SMT_CP = 10;            // classes the layout is built for
constexpr int SMT_WC = 2 * SMT_CP;    // tensor-memory columns per feature pair
constexpr int SMT_DSTR = 12;          // floats per row of D in shared memory (10 classes, padded to whole 16-byte loads)
constexpr int SMT_HEAD_BYTES = 4096;
constexpr uint32_t SMT_TMEM_COLS = 256;

struct TmTileInfo { int flags, rows, K, snap, fresh, next_snap; };

__device__ __forceinline__ void tm_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tm_ld4(uint32_t taddr, float* v) {
  uint32_t r[4];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr) : "memory");
#pragma unroll
  for (int i = 0; i < 4; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tm_st16(uint32_t taddr, const float* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
        "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
        "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
        "r"(__float_as_uint(v[15])) : "memory");
}
__device__ __forceinline__ void tm_st4(uint32_t taddr, const float* v) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1,%2,%3,%4};"
               ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
                 "r"(__float_as_uint(v[3])) : "memory");
}
// the 20 columns of one feature pair
__device__ __forceinline__ void tm_ld20(uint32_t taddr, float* v) { tm_ld16(taddr, v); tm_ld4(taddr + 16, v + 16); }
__device__ __forceinline__ void tm_st20(uint32_t taddr, const float* v) { tm_st16(taddr, v); tm_st4(taddr + 16, v + 16); }
__device__ __forceinline__ void tm_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tm_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tm_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tm_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tm_alloc(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tm_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// Transposition reduce of S values per lane over the warp: every step halves the values a lane holds
// (padding an odd count with a zero) and doubles the lanes each value has been summed over.
template <int O, int S>
__device__ __forceinline__ void tm_reduce_steps(float* v, int lane) {
  if constexpr (O >= 1) {
    constexpr int E = S + (S & 1), H = E / 2;
    if (S & 1) v[S] = 0.f;
    const bool up = (lane & O) != 0;
#pragma unroll
    for (int i = 0; i < H; ++i) {
      const float send = up ? v[i] : v[i + H];
      const float keep = up ? v[i + H] : v[i];
      v[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, O);
    }
    tm_reduce_steps<O / 2, H>(v, lane);
  }
}
// Which of the N original values lane `lane` holds in v[0] after tm_reduce_steps<16, N> (-1: padding).
template <int N>
__device__ __forceinline__ int tm_reduce_index(int lane) {
  static_assert(N <= 32, "one value per lane at most");
  int idx = 0, real = N, s = N;
#pragma unroll
  for (int O = 16; O >= 1; O >>= 1) {
    const int h = (s + (s & 1)) / 2;
    if (lane & O) { idx += h; real -= h; } else { real = min(real, h); }
    s = h;
  }
  return real >= 1 ? idx : -1;
}

template <int NG, int KP, int TG, bool ASYNC>
__global__ void __launch_bounds__(128 * NG) softmax_tm_kernel(NumericArgs a) {
  constexpr int NT = 128 * NG, NW = 4 * NG, T = NG * TG, CP = SMT_CP, WC = SMT_WC, OWN = KP * WC, NV = TG * CP;
  constexpr int DS = 2 * NT * KP;      // floats between row slots: every thread can read its pairs without a bounds test
  static_assert(NG * OWN <= (int)SMT_TMEM_COLS, "the parameters must fit the allocated columns");
  constexpr int SW = (16 * T + 31) / 32;   // warps of the softmax stage: whole warps, it shuffles with a full mask
  static_assert(32 * SW <= NT && T <= 32 && NV <= 32, "tile shape");
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int grp = tid >> 7, L = tid & 127;
  const int r = blockIdx.x;
  const int d = a.d, dp = d >> 1, m = a.m, C = a.n_classes;
  const uint32_t rid = a.replica_base + (uint32_t)r;
  const uint32_t row_bytes = (uint32_t)d * 4u;
  const size_t np = (size_t)C * d;
  const long long my_j0 = a.run_j0 ? a.run_j0[r] : a.j0, my_iters = a.run_iters ? a.run_iters[r] : a.iters;

  extern __shared__ __align__(128) unsigned char smem[];
  // head (ring of S <= 4 tiles): barriers [4] @0 | tmem base @32 | first snapshot @36 | TileInfo [4] @48 | y [4][T] @160
  //       | lossrow [T] @352 | misc [NW] @480 | delta [T][12] @576 | red [NW][32] @2048
  const int S = a.stages;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 32);
  int* first_snap_s = reinterpret_cast<int*>(smem + 36);
  TmTileInfo* info_s = reinterpret_cast<TmTileInfo*>(smem + 48);
  uint32_t* y_s = reinterpret_cast<uint32_t*>(smem + 160);
  float* lossrow_s = reinterpret_cast<float*>(smem + 352);
  float* misc_s = reinterpret_cast<float*>(smem + 480);
  float* delta_s = reinterpret_cast<float*>(smem + 576);
  float* red_s = reinterpret_cast<float*>(smem + 2048);
  static_assert(48 + 4 * sizeof(TmTileInfo) <= 160 && 160 + 16 * T <= 352 && 352 + 4 * T <= 480 && 480 + 4 * NW <= 576 &&
                576 + 8 * T * CP <= 2048 && 2048 + 128 * NW <= SMT_HEAD_BYTES, "head layout");
  float* rows_s = reinterpret_cast<float*>(smem + SMT_HEAD_BYTES);
  uint32_t* pidx_s = reinterpret_cast<uint32_t*>(rows_s + (size_t)S * T * DS);   // [m] sample rows of the producer's task

  if (tid == 0) {
    for (int s = 0; s < S; ++s) mbar_init(smem_addr(&full[s]), (uint32_t)T + 1u);
    mbar_fence_init();
  }
  if (warp == 1) tm_alloc(smem_addr(tmem_slot), SMT_TMEM_COLS);
  // The arithmetic reads whole row slots and whole tiles: features past d and rows past the end of a ragged tile
  // must hold finite numbers (they meet zero parameters / zero softmax terms), so the slots start as zeros.
  for (int i = tid; i < S * T * DS / 4; i += NT) reinterpret_cast<float4*>(rows_s)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();

  ScheduleWalk walk;
  walk.done = true;
  int prod_st = 0;      // tiles are issued in order: the producer's stage is a counter
  auto issue_tile = [&]() {
    if (walk.done) return;
    const int st = prod_st;
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
      TmTileInfo ti;
      ti.rows = rows; ti.K = (int)walk.cur.K; ti.snap = (int)walk.cur.snap; ti.fresh = (int)walk.cur.fresh;
      ti.next_snap = (int)walk.nxt.snap;
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
        bulk_g2s(smem_addr(rows_s + ((size_t)st * T + lane) * DS), a.X + (size_t)idx * d, row_bytes, bar);
        word_g2s_arrive(smem_addr(&y_s[st * T + lane]), reinterpret_cast<const uint32_t*>(a.y) + idx, bar);
      } else {
        mbar_arrive(bar);
      }
    }
    walk.advance(a);
  };
  if (warp == 0) {
    walk.start(a, r, my_j0, my_iters);
    walk.tiles_per_task = (m + T - 1) / T;
    if (lane == 0) *first_snap_s = walk.done ? 0 : (int)walk.cur.snap;
    for (int s = 0; s < S; ++s) issue_tile();
  }
  tm_fence_before();
  __syncthreads();
  tm_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;
  const uint32_t t_own = tmem + lane_base + (uint32_t)(grp * OWN);    // this thread's own columns
  const uint32_t t_lane = tmem + lane_base;                           // all columns of its lane

  // parameters of this thread's pairs: global (row-major [C][d]) -> tensor memory, zero where there is no such pair / class
  auto load_w = [&](const float* src) {
#pragma unroll
    for (int k = 0; k < KP; ++k) {
      const int p = tid + NT * k;
      float w[WC];
#pragma unroll
      for (int c = 0; c < CP; ++c) {
        float2 v = make_float2(0.f, 0.f);
        if (p < dp && c < C) v = reinterpret_cast<const float2*>(src + (size_t)c * d)[p];
        w[2 * c] = v.x; w[2 * c + 1] = v.y;
      }
      tm_st20(t_own + k * WC, w);
    }
    tm_wait_st();
  };
  if (my_iters > 0) {
    load_w(ASYNC ? a.pool + ((size_t)r * a.n_slots + *first_snap_s) * np : a.w_state + (size_t)r * np);
    tm_fence_before();
    __syncthreads();
    tm_fence_after();
  }

  uint64_t G[CP][KP];      // the two features of a pair
#pragma unroll
  for (int c = 0; c < CP; ++c)
#pragma unroll
    for (int k = 0; k < KP; ++k) G[c][k] = 0ull;
  float loss_acc = 0.f;      // meaningful in the row-leader threads of the softmax stage
  long long j = my_j0;
  bool failed = false;
  int cur_slot = ASYNC ? (int)a.begin_slot[r] : 0;
  const int st_tid = tid - (NT - 32 * SW);         // the last warps serve the softmax stage (warp 0 is the producer)
  const int sq = st_tid >> 4, sc = st_tid & 15;    // 16 lanes per row
  const int red_idx = tm_reduce_index<NV>(lane);

  int st = 0;                // stage and phase parity of tile `it`, as counters
  uint32_t parity = 0;
  for (long long it = 0; my_iters > 0; ++it, parity ^= (uint32_t)(st + 1 == S), st = (st + 1 == S ? 0 : st + 1)) {
    const bool ok = mbar_wait(smem_addr(&full[st]), parity);
    const TmTileInfo ti = info_s[st];
    const float* tile = rows_s + (size_t)st * T * DS;

    // ---- logits of this group's rows (row grp + NG s of the tile, s < TG) over the features of its lane ----
    {
      float acc[NV + 2];
#pragma unroll
      for (int i = 0; i < NV + 2; ++i) acc[i] = 0.f;
      const float2* rowp = reinterpret_cast<const float2*>(tile + grp * DS) + L;
#pragma unroll
      for (int ck = 0; ck < NG * KP; ++ck) {
        const int gp = ck / KP, k = ck % KP;
        float w[WC];
        tm_ld20(t_lane + ck * WC, w);
        float2 x[TG];
#pragma unroll
        for (int s = 0; s < TG; ++s) x[s] = rowp[s * NG * (DS / 2) + 128 * gp + NT * k];
        tm_wait_ld();
#pragma unroll
        for (int s = 0; s < TG; ++s)
#pragma unroll
          for (int c = 0; c < CP; ++c)
            acc[s * CP + c] = fmaf(x[s].y, w[2 * c + 1], fmaf(x[s].x, w[2 * c], acc[s * CP + c]));
      }
      tm_reduce_steps<16, NV>(acc, lane);
      if (red_idx >= 0) red_s[warp * 32 + red_idx] = acc[0];
    }
    tm_fence_before();
    if (__syncthreads_or(!ok)) { failed = true; break; }   // (A) partial logits published; everyone is past the previous tile
    tm_fence_after();
    if (warp == 0 && it >= 1) issue_tile();                // tile it + S - 1, into the stage of tile it - 1

    // ---- softmax stage: thread (sq, sc) owns logit (row sq, class sc) ----
    float loss_term = 0.f, loss_s1 = 0.f;
    if (st_tid >= 0) {
      float z = -INFINITY;
      const bool live = sc < C && sq < ti.rows;
      int label = 0;
      if (sq < ti.rows) label = (int)y_s[st * T + sq];
      if (live) {
        const int g = sq % NG, s = sq / NG;
        float acc = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) acc += red_s[(4 * g + w) * 32 + s * CP + sc];
        z = acc;
      }
      float zmax = z;
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) zmax = fmaxf(zmax, __shfl_xor_sync(0xFFFFFFFFu, zmax, off));
      // sum of exponentials without the maximal class (whose term is exactly 1): log(1 + s) and
      // p_max - 1 = -s / (1 + s) stay accurate when the sample is classified with a wide margin
      const unsigned at_max = __ballot_sync(0xFFFFFFFFu, live && z == zmax);
      const int cmax = __ffs((at_max >> (lane & 16)) & 0xFFFFu) - 1;
      const bool is_max = sc == cmax;
      const float ez = (live && !is_max) ? expf(z - zmax) : 0.f;
      float sexcl = ez;
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) sexcl += __shfl_xor_sync(0xFFFFFFFFu, sexcl, off);
      const float inv = __frcp_rn(1.f + sexcl);   // one correctly rounded reciprocal instead of a division per case
      const float zlab = __shfl_sync(0xFFFFFFFFu, z, (lane & 16) + label);
      float dl = 0.f;
      if (live) {
        if (is_max) dl = sc == label ? -sexcl * inv : inv;
        else dl = ez * inv - (sc == label ? 1.f : 0.f);
      }
      if (sc < SMT_DSTR && sq < T) delta_s[sq * SMT_DSTR + sc] = dl;
      loss_term = (sc == 0 && sq < ti.rows) ? zmax - zlab : 0.f;
      loss_s1 = (sc == 0 && sq < ti.rows) ? sexcl : 0.f;
    }
    __syncthreads();   // (B)
    if (st_tid >= 0) loss_acc += log1pf(loss_s1) + loss_term;   // off the path the other warps wait on

    // ---- G += D^T X over own pairs ----
    // (every row of the tile: the softmax stage wrote zeros for the rows a ragged tile does not have)
    {
      const uint64_t* xp = reinterpret_cast<const uint64_t*>(tile) + tid;
#pragma unroll
      for (int q = 0; q < T; ++q) {
        uint64_t x2[KP];
#pragma unroll
        for (int k = 0; k < KP; ++k) x2[k] = xp[q * (DS / 2) + NT * k];
        // D of the row: a shared-memory load delivers 4 bytes per lane and wavefront whatever its width, also when
        // all lanes read the same address, so D is stored once (not as ready-made pairs) and paired by a register move
        float dv[SMT_DSTR];
#pragma unroll
        for (int c4 = 0; c4 < 2; ++c4) {
          const float4 v = reinterpret_cast<const float4*>(delta_s)[q * (SMT_DSTR / 4) + c4];
          dv[4 * c4] = v.x; dv[4 * c4 + 1] = v.y; dv[4 * c4 + 2] = v.z; dv[4 * c4 + 3] = v.w;
        }
        {
          const float2 v = reinterpret_cast<const float2*>(delta_s)[q * (SMT_DSTR / 2) + 4];
          dv[8] = v.x; dv[9] = v.y;
        }
#pragma unroll
        for (int c = 0; c < CP; ++c) {
          const uint64_t dd = pack2(dv[c], dv[c]);
#pragma unroll
          for (int k = 0; k < KP; ++k) G[c][k] = ffma2(dd, x2[k], G[c][k]);
        }
      }
    }

    const bool last_of_update = (ti.flags & TILE_LAST_OF_UPDATE) != 0;
    const bool reload = ASYNC && (ti.flags & TILE_LAST_OF_TASK) && !(ti.flags & TILE_LAST_OF_RUN);
    if (last_of_update) {
      const float scale = (float)((double)a.eta / ((double)ti.K * (double)m));
      float dd = 0.f;
      const float* w_from = ASYNC ? a.pool + ((size_t)r * a.n_slots + cur_slot) * np : nullptr;
      float* w_to = ASYNC ? a.pool + ((size_t)r * a.n_slots + ti.fresh) * np : nullptr;
#pragma unroll
      for (int k = 0; k < KP; ++k) {
        const int p = tid + NT * k;
        float w[WC];
        if (!ASYNC) { tm_ld20(t_own + k * WC, w); tm_wait_ld(); }
#pragma unroll
        for (int c = 0; c < CP; ++c) {
          float g0, g1;
          unpack2(G[c][k], g0, g1);
          G[c][k] = 0ull;
          if (ASYNC) {
            if (p < dp && c < C) {
              float2 v = reinterpret_cast<const float2*>(w_from + (size_t)c * d)[p];
              v.x = fmaf(-scale, g0, v.x);
              v.y = fmaf(-scale, g1, v.y);
              reinterpret_cast<float2*>(w_to + (size_t)c * d)[p] = v;
              w[2 * c] = v.x; w[2 * c + 1] = v.y;
            }
          } else {
            w[2 * c] = fmaf(-scale, g0, w[2 * c]);
            w[2 * c + 1] = fmaf(-scale, g1, w[2 * c + 1]);
          }
          if (a.w_ref && p < dp && c < C) {
            const float2 wr = reinterpret_cast<const float2*>(a.w_ref + (size_t)c * d)[p];
            const float e0 = w[2 * c] - wr.x, e1 = w[2 * c + 1] - wr.y;
            dd = fmaf(e0, e0, dd); dd = fmaf(e1, e1, dd);
          }
        }
        if (!ASYNC) tm_st20(t_own + k * WC, w);
      }
      if (ASYNC) cur_slot = ti.fresh;
      dd = warp_sum(dd);
      if (lane == 0) misc_s[warp] = dd;
      if (st_tid >= 0 && sc == 0 && sq < T) lossrow_s[sq] = loss_acc;
    }
    if (reload) load_w(a.pool + ((size_t)r * a.n_slots + ti.next_snap) * np);   // the next task's snapshot (own elements only)
    if (last_of_update || reload) {
      tm_wait_st();
      tm_fence_before();
      __syncthreads();   // (C) the parameters in tensor memory are the next tile's
      tm_fence_after();
    }
    if (last_of_update) {
      if (tid == 0) {
        float tot = 0.f, ls = 0.f;
        for (int w = 0; w < NW; ++w) tot += misc_s[w];
        for (int q = 0; q < T; ++q) ls += lossrow_s[q];
        a.dist2[(size_t)r * a.cap + j] = a.w_ref ? tot : 0.f;
        a.loss[(size_t)r * a.cap + j] = ls / ((float)ti.K * (float)m);
      }
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
  } else if (!ASYNC && my_iters > 0) {
    float* dst = a.w_state + (size_t)r * np;
#pragma unroll
    for (int k = 0; k < KP; ++k) {
      const int p = tid + NT * k;
      float w[WC];
      tm_ld20(t_own + k * WC, w);
      tm_wait_ld();
#pragma unroll
      for (int c = 0; c < CP; ++c)
        if (p < dp && c < C) reinterpret_cast<float2*>(dst + (size_t)c * d)[p] = make_float2(w[2 * c], w[2 * c + 1]);
    }
  }
  tm_fence_before();
  __syncthreads();
  if (warp == 1) tm_dealloc(tmem, SMT_TMEM_COLS);
}

inline size_t softmax_tm_smem_bytes(int S, int T, int d, int m) {
  const int nt = 128 * SMX_TM_NG, kp = (d / 2 + nt - 1) / nt;
  const size_t need = (size_t)SMT_HEAD_BYTES + (size_t)S * T * (2 * nt * kp) * 4 + (size_t)m * 4;
  // one CTA per SM, whatever the shape: two CTAs' tensor-memory allocations would still fit, a third would wait
  return need < (size_t)(116 << 10) ? (size_t)(116 << 10) : need;
}

// Shapes this kernel takes; the others go to softmax_kernel.
inline bool softmax_tm_supported(int d, int C, int m) {
  constexpr int NT = 128 * SMX_TM_NG, T = SMX_TM_NG * SMX_TM_TG;
  const int kp = (d / 2 + NT - 1) / NT;
  return C <= SMT_CP && kp * SMX_TM_NG * SMT_WC <= (int)SMT_TMEM_COLS && softmax_tm_smem_bytes(2, T, d, m) <= (size_t)(226 << 10);
}

template <int KP>
cudaError_t launch_softmax_tm(NumericArgs& a, cudaStream_t stream) {
  constexpr int NG = SMX_TM_NG, TG = SMX_TM_TG;
  auto kern = a.is_async ? softmax_tm_kernel<NG, KP, TG, true> : softmax_tm_kernel<NG, KP, TG, false>;
  int S = 4;   // tiles in the ring: as many as shared memory holds, two at least
  while (S > 2 && softmax_tm_smem_bytes(S, NG * TG, a.d, a.m) > (size_t)(226 << 10)) --S;
  const size_t smem = softmax_tm_smem_bytes(S, NG * TG, a.d, a.m);
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  a.stages = S;
  kern<<<a.R, 128 * NG, smem, stream>>>(a);
  return cudaGetLastError();
}

inline cudaError_t run_softmax_tm_any(NumericArgs& a, int tune_stages, cudaStream_t stream, const char** why) {
  *why = nullptr;
  if (softmax_tm_supported(a.d, a.n_classes, a.m)) {
    const int kp = (a.d / 2 + 128 * SMX_TM_NG - 1) / (128 * SMX_TM_NG);
    switch (kp) {
      case 1: return launch_softmax_tm<1>(a, stream);
      case 2: return launch_softmax_tm<2>(a, stream);
      case 3: return launch_softmax_tm<3>(a, stream);
#if SMX_TM_NG == 3
      case 4: return launch_softmax_tm<4>(a, stream);
#endif
      default: break;
    }
  }
  return run_softmax(a, tune_stages, stream, why);
}

}  // namespace ssim
