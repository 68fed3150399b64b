// Gradient / update kernel for softmax regression with up to 10 classes, warp-specialised: twelve
// warps do nothing but the two FMA passes; a fourth warpgroup stages rows (one warp) and forms the
// softmax terms (three warps), on a small share of the registers.
//
// Ownership.  The d/2 pairs of adjacent features are dealt to the 384 FMA threads: thread t owns pairs
// t + 384 k (k < KP).  For its pairs and all classes it keeps the gradient accumulator G in registers
// for the whole update and the parameters W_tau in 20 KP columns of its own tensor-memory lane
// (lane t mod 128, columns 20 KP (t / 128) ...; column 20 k + 2 c + h holds W[c][feature h of pair k]):
// tensor memory serves as a 120 KB register-file extension with its own read path, no MMA is issued.
// The update W <- W - (eta / (K m)) G (Eq. 2 / Eq. 3) is thread-local: tcgen05.ld, FMA, tcgen05.st.
// Per tile:
//   logits    Z = X_tile W_tau^T.  The three groups of four warps take different rows (TG each); thread
//             (lane L of the 128, group g) walks the whole of tensor-memory lane L - the columns of all
//             three owners.  One warp transposition reduce and a four-way sum finish the logits.
//   softmax   D = softmax(Z) - onehot(label), loss: 16 lanes per row.
//   gradient  G += D^T X_tile: every FMA thread, every row, own pairs, packed fp32x2 FMAs (the two
//             features of a pair), for nine of the ten class slots - the rows of D sum to zero, so the
//             tenth slot's gradient is minus the sum of the others and is formed once per update.
// Plain fp32 FMAs: the 1e-5 parity bound on the parameters rules out reduced-precision tensor-core operands.
//
// Who waits for whom.  This path is
// bound by instruction issue (20 FMA per 4-byte feature, every other instruction costs an FMA
// slot), and in a kernel where all warps walk through "logits, barrier, softmax, barrier,
// gradient" together the FMA pipe idles while a few lanes form the softmax terms and while one
// warp issues the next tile's copies.  Here:
//   FMA warps 0-11, tile t:   logits of tile t  ->  publish the partial sums  ->  gradient of tile
//                             t - 1 (whose softmax terms were formed meanwhile)  ->  free its stage.
//                             No block barrier inside an update: the warps drift apart and cover one
//                             another's latencies.
//   softmax warps 13-15:      wait for the twelve partial logit vectors of tile t, form
//                             D = softmax(Z) - onehot(label) and the rows' losses (two rows a warp, 16 lanes
//                             a row), publish D.
//   producer warp 12:         refills the stage of tile t - 1 as soon as its gradient pass is through.
// The block is launched with 128 registers a thread; the three FMA warpgroups then take 152 each and the helper
// warpgroup keeps 56 (setmaxnreg; 3 x 128 x 152 + 128 x 56 = 512 x 128, the whole allocation and no more).
// Tiles are 3 TG rows in a ring of S stages (6 rows x 3 stages for 3072 features): tile t + 1 is
// read for logits while tile t still waits for its gradient pass and tile t + 2 is in flight.
// Where the parameters change - the end of an update (Eq. 2 / Eq. 3) and, for the asynchronous
// variants, the start of a task with another snapshot - the pipeline drains: the twelve FMA warps
// meet at a barrier of their own before and after tensor memory is rewritten.
// Every wait (on row copies, partial logits, softmax terms, free stages, the FMA warps' barrier) is
// a bounded poll of an mbarrier; a wait that runs out raises a flag in shared memory that ends all
// other waits early, and the error word is set.
#pragma once
#include "tmem_util.cuh"

namespace ssim {

constexpr int SWS_NG = 3;                       // thread groups of four warps (one per tensor-memory lane quarter each)
constexpr int SWS_FMA_THREADS = 128 * SWS_NG;   // 384
constexpr int SWS_THREADS = SWS_FMA_THREADS + 128;   // + one helper warpgroup: producer warp, three softmax warps
constexpr int SWS_LAUNCH_REGS = 128, SWS_FMA_REGS = 152, SWS_HELPER_REGS = 56;
static_assert(SWS_FMA_THREADS * SWS_FMA_REGS + 128 * SWS_HELPER_REGS <= SWS_THREADS * SWS_LAUNCH_REGS, "the register split must fit the launch allocation");
constexpr int SWS_MAX_S = 6;
constexpr int SWS_HEAD_BYTES = 5120;

// bounded wait that also gives up when another role has raised the abort flag
__device__ __forceinline__ bool sws_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < (1u << 24); ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (i > 2048) {
      if (*abort_flag) return false;
      __nanosleep(64);
    }
  }
  return false;
}

// Parameters of a thread's pairs: global (row-major [C][d]) -> its own tensor-memory columns, zero where there is no such
// pair / class.  Not inlined on purpose: in the asynchronous variants it is called inside the tile loop (a task with
// another snapshot), and inlined there its loads in flight competed with the gradient accumulator for registers on every
// tile; as a call the accumulator is saved and restored around it, where it is needed once per task.
template <int KP>
__device__ __noinline__ void sws_load_params(const float* src, int d, int C, int tid, uint32_t t_own) {
  constexpr int NT = SWS_FMA_THREADS, CP = SMT_CP, WC = SMT_WC;
  const int dp = d >> 1;
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
}

// Eq. 3 for the asynchronous variants: w_{j+1} = w_j - scale G goes from one version of the pool to another in global
// memory (the snapshot in tensor memory is some worker's stale one, not w_j).  Gm holds the nine accumulated class slots of
// the thread's pairs ([slot][pair]); the tenth is minus their sum.  Returns the thread's share of |w_{j+1} - w_ref|^2.
// Not inlined, and fed through local memory, for the reason given at sws_load_params: once per update, never per tile.
template <int KP>
__device__ __noinline__ float sws_async_update(const uint64_t* Gm, const float* w_from, float* w_to, const float* w_ref, float scale,
                                               int d, int C, int tid) {
  constexpr int NT = SWS_FMA_THREADS, CP = SMT_CP, GC = CP - 1;
  const int dp = d >> 1;
  float dd = 0.f;
#pragma unroll
  for (int k = 0; k < KP; ++k) {
    const int p = tid + NT * k;
    if (p >= dp) continue;
    float s0 = 0.f, s1 = 0.f;      // sum of the nine accumulated slots, in slot order
#pragma unroll
    for (int c = 0; c < CP; ++c) {
      float g0, g1;
      if (c < GC) {
        unpack2(Gm[c * KP + k], g0, g1);
        s0 += g0; s1 += g1;
      } else {
        g0 = C == CP ? -s0 : 0.f;
        g1 = C == CP ? -s1 : 0.f;
      }
      if (c < C) {
        float2 v = reinterpret_cast<const float2*>(w_from + (size_t)c * d)[p];
        v.x = fmaf(-scale, g0, v.x);
        v.y = fmaf(-scale, g1, v.y);
        reinterpret_cast<float2*>(w_to + (size_t)c * d)[p] = v;
        if (w_ref) {
          const float2 wr = reinterpret_cast<const float2*>(w_ref + (size_t)c * d)[p];
          const float e0 = v.x - wr.x, e1 = v.y - wr.y;
          dd = fmaf(e0, e0, dd); dd = fmaf(e1, e1, dd);
        }
      }
    }
  }
  return dd;
}

template <int KP, int TG, bool ASYNC>
__global__ void __launch_bounds__(SWS_THREADS, 1) softmax_ws_kernel(NumericArgs a) {
  constexpr int NG = SWS_NG, NT = SWS_FMA_THREADS, NW = NT / 32, T = NG * TG, CP = SMT_CP, WC = SMT_WC, OWN = KP * WC, NV = TG * CP;
  constexpr int DS = 2 * NT * KP;      // floats between row slots: every thread can read its pairs without a bounds test
  static_assert(NG * OWN <= (int)SMT_TMEM_COLS, "the parameters must fit the allocated columns");
  static_assert(T == 6 && NV <= 32, "three softmax warps take two rows each; one reduce per tile");
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r = blockIdx.x;
  const int d = a.d, dp = d >> 1, m = a.m, C = a.n_classes, S = a.stages;
  const uint32_t rid = a.replica_base + (uint32_t)r;
  const uint32_t row_bytes = (uint32_t)d * 4u;
  const size_t np = (size_t)C * d;
  const long long my_j0 = a.run_j0 ? a.run_j0[r] : a.j0, my_iters = a.run_iters ? a.run_iters[r] : a.iters;

  extern __shared__ __align__(128) unsigned char smem[];
  // head: full[6] @0 | empty[6] @64 | zready[2] @128 | dready[2] @144 | cbar @160 | tmem base @176 | first snapshot @180
  //       | abort @184 | TileInfo[6] @192 | y [6][T] @384 | lossrow [T] @528 | misc [12] @576 | delta [2][T][12] @640
  //       | red [2][12][32] @2048
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);
  uint64_t* empty = reinterpret_cast<uint64_t*>(smem + 64);
  uint64_t* zready = reinterpret_cast<uint64_t*>(smem + 128);
  uint64_t* dready = reinterpret_cast<uint64_t*>(smem + 144);
  uint64_t* cbar = reinterpret_cast<uint64_t*>(smem + 160);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 176);
  int* first_snap_s = reinterpret_cast<int*>(smem + 180);
  volatile int* abort_s = reinterpret_cast<volatile int*>(smem + 184);
  TmTileInfo* info_s = reinterpret_cast<TmTileInfo*>(smem + 192);
  uint32_t* y_s = reinterpret_cast<uint32_t*>(smem + 384);
  float* lossrow_s = reinterpret_cast<float*>(smem + 528);
  float* misc_s = reinterpret_cast<float*>(smem + 576);
  float* delta_s = reinterpret_cast<float*>(smem + 640);
  float* red_s = reinterpret_cast<float*>(smem + 2048);
  static_assert(192 + SWS_MAX_S * sizeof(TmTileInfo) <= 384 && 384 + 4 * SWS_MAX_S * T <= 528 && 528 + 4 * T <= 576 && 576 + 4 * NW <= 640 &&
                640 + 4 * 2 * T * SMT_DSTR <= 2048 && 2048 + 4 * 2 * NW * 32 <= SWS_HEAD_BYTES, "head layout");
  float* rows_s = reinterpret_cast<float*>(smem + SWS_HEAD_BYTES);
  uint32_t* pidx_s = reinterpret_cast<uint32_t*>(rows_s + (size_t)S * T * DS);   // [m] sample rows of the producer's task

  if (tid == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(smem_addr(&full[s]), (uint32_t)T + 1u); mbar_init(smem_addr(&empty[s]), (uint32_t)NW); }
    for (int b = 0; b < 2; ++b) { mbar_init(smem_addr(&zready[b]), (uint32_t)NW); mbar_init(smem_addr(&dready[b]), 96u); }
    mbar_init(smem_addr(cbar), (uint32_t)NW);
    *abort_s = 0;
    mbar_fence_init();
  }
  if (warp == NW) { tm_alloc(smem_addr(tmem_slot), SMT_TMEM_COLS); tm_fence_before(); }
  if (tid < T) lossrow_s[tid] = 0.f;
  // The arithmetic reads whole row slots and whole tiles: features past d and rows past the end of a ragged tile
  // must hold finite numbers (they meet zero parameters / zero softmax terms), so the slots start as zeros.
  for (int i = tid; i < S * T * DS / 4; i += SWS_THREADS) reinterpret_cast<float4*>(rows_s)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int i = tid; i < 2 * T * SMT_DSTR; i += SWS_THREADS) delta_s[i] = 0.f;
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();

  const int tiles_per_task = (m + T - 1) / T;
  bool failed = false;

  if (warp >= NW) {
  // the helper warpgroup gives registers up in one instruction that all four of its warps execute, then splits into roles
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(SWS_HELPER_REGS));
  if (warp == NW) {
    // =============================== producer warp: rows in ===============================
    ScheduleWalk walk;
    walk.done = true;
    int prod_st = 0;      // tiles are issued in order: the producer's stage is a counter
    auto issue_tile = [&]() {
      const int st = prod_st;
      if (++prod_st == S) prod_st = 0;
      const uint32_t bar = smem_addr(&full[st]);
      const int rows = min(T, m - walk.k * T);
      if (walk.k == 0) {   // a new task: its m sample rows are drawn once, 32 at a time
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
    walk.start(a, r, my_j0, my_iters);
    walk.tiles_per_task = tiles_per_task;
    if (lane == 0) *first_snap_s = walk.done ? 0 : (int)walk.cur.snap;
    for (int s = 0; s < S && !walk.done; ++s) issue_tile();
    __syncthreads();      // (1) first snapshot known, tensor memory allocated
    __syncthreads();      // (2) the FMA warps have loaded the parameters
    // tile n + S goes into the stage of tile n once the twelve FMA warps are through tile n's gradient pass
    int st = 0;
    uint32_t par_empty = 0;
    while (!walk.done) {
      if (!sws_wait(smem_addr(&empty[st]), par_empty, abort_s)) { failed = true; break; }
      issue_tile();
      if (++st == S) { st = 0; par_empty ^= 1u; }
    }
  } else {
    // =============================== softmax warps: two rows of the tile each ===============================
    __syncthreads();      // (1)
    __syncthreads();      // (2)
    const int sq = 2 * (warp - NW - 1) + (lane >> 4), sc = lane & 15;      // row of the tile, class; 16 lanes per row
    const int g = sq % NG, srow = sq / NG;                                 // the row was summed by group g as its srow-th row
    float loss_acc = 0.f;                           // in lanes 0 and 16: their row slot's losses of the current update
    int st = 0;
    uint32_t par_full = 0;
    for (long long it = 0; my_iters > 0; ++it) {
      const int buf = (int)(it & 1);
      if (!sws_wait(smem_addr(&zready[buf]), (uint32_t)((it >> 1) & 1), abort_s)) { failed = true; break; }
      const TmTileInfo ti = info_s[st];
      const float* red = red_s + buf * NW * 32;
      const bool live = sc < C && sq < ti.rows;
      int label = 0;
      if (sq < ti.rows) label = (int)y_s[st * T + sq];
      float z = -INFINITY;
      if (live) {
        float acc = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) acc += red[(4 * g + w) * 32 + srow * CP + sc];
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
      if (sc < SMT_DSTR) delta_s[(buf * T + sq) * SMT_DSTR + sc] = dl;
      const bool row_leader = sc == 0 && sq < ti.rows;
      if (row_leader) loss_acc += log1pf(sexcl) + (zmax - zlab);
      if (ti.flags & TILE_LAST_OF_UPDATE) {          // the row slot's share of the update's loss; thread 0 adds the shares up
        if (sc == 0) lossrow_s[sq] = loss_acc;
        loss_acc = 0.f;
      }
      mbar_arrive(smem_addr(&dready[buf]));          // every lane after its own stores
      if (ti.flags & TILE_LAST_OF_RUN) break;
      if (++st == S) { st = 0; par_full ^= 1u; }
    }
    (void)par_full;
  }
  } else {
    // =============================== FMA warps ===============================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(SWS_FMA_REGS));
    const int grp = tid >> 7, L = tid & 127;
    __syncthreads();      // (1)
    tm_fence_after();
    const uint32_t tmem = *tmem_slot;
    const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;
    const uint32_t t_own = tmem + lane_base + (uint32_t)(grp * OWN);    // this thread's own columns
    const uint32_t t_lane = tmem + lane_base;                           // all columns of its lane

    auto load_w = [&](const float* src) { sws_load_params<KP>(src, d, C, tid, t_own); };
    if (my_iters > 0) load_w(ASYNC ? a.pool + ((size_t)r * a.n_slots + *first_snap_s) * np : a.w_state + (size_t)r * np);
    tm_fence_before();
    __syncthreads();      // (2)
    tm_fence_after();

    // barrier of the twelve FMA warps alone (bounded, like every wait here)
    uint32_t cpar = 0;
    auto fma_barrier = [&]() -> bool {
      tm_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_addr(cbar));
      const bool ok = sws_wait(smem_addr(cbar), cpar, abort_s);
      cpar ^= 1u;
      tm_fence_after();
      return ok;
    };

    // Gradient accumulator of the first nine class slots only.  The rows of D = softmax(Z) - onehot sum to zero over the
    // classes, hence so do the rows of the gradient D^T X: the tenth slot is minus the sum of the other nine, formed
    // once per update instead of being accumulated with a tenth of the gradient pass's FMAs (with fewer than ten classes
    // the tenth slot is padding and its gradient is zero).
    constexpr int GC = CP - 1;
    uint64_t G[GC][KP];      // the two features of a pair
#pragma unroll
    for (int c = 0; c < GC; ++c)
#pragma unroll
      for (int k = 0; k < KP; ++k) G[c][k] = 0ull;
    long long j = my_j0;
    int cur_slot = ASYNC ? (int)a.begin_slot[r] : 0;
    const int red_idx = tm_reduce_index<NV>(lane);

    // G += D^T X over own pairs for the tile in stage `gst`, softmax terms in buffer `gbuf`; then the stage is free
    auto gradient_pass = [&](int gst, int gbuf) {
      const uint64_t* xp = reinterpret_cast<const uint64_t*>(rows_s + (size_t)gst * T * DS) + tid;
      const float* delta = delta_s + gbuf * T * SMT_DSTR;
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
          const float4 v = reinterpret_cast<const float4*>(delta)[q * (SMT_DSTR / 4) + c4];
          dv[4 * c4] = v.x; dv[4 * c4 + 1] = v.y; dv[4 * c4 + 2] = v.z; dv[4 * c4 + 3] = v.w;
        }
        dv[8] = delta[q * SMT_DSTR + 8];
#pragma unroll
        for (int c = 0; c < GC; ++c) {
          const uint64_t dd = pack2(dv[c], dv[c]);
#pragma unroll
          for (int k = 0; k < KP; ++k) G[c][k] = ffma2(dd, x2[k], G[c][k]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_addr(&empty[gst]));
    };

    // logits of this group's rows (row grp + NG s of the tile, s < TG) over the features of its lane, for the tile in stage
    // `lst`; the warp's partial sums go to buffer `lbuf` and are published
    auto logit_pass = [&](int lst, int lbuf) {
      const float* tile = rows_s + (size_t)lst * T * DS;
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
        for (int s = 0; s < TG; ++s) {
#pragma unroll
          for (int c = 0; c < CP; ++c)
            acc[s * CP + c] = fmaf(x[s].y, w[2 * c + 1], fmaf(x[s].x, w[2 * c], acc[s * CP + c]));
        }
      }
      tm_reduce_steps<16, NV>(acc, lane);
      if (red_idx >= 0) red_s[(lbuf * NW + warp) * 32 + red_idx] = acc[0];
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_addr(&zready[lbuf]));
    };
    // loss and distance of the update that ends with a tile of K contributors, recorded by thread 0 after the barrier
    auto record = [&](int K_of_update) {
      if (tid == 0) {
        float tot = 0.f, ls = 0.f;
        for (int w = 0; w < NW; ++w) tot += misc_s[w];
        for (int q = 0; q < T; ++q) ls += lossrow_s[q];      // published with the update's last softmax terms
        a.dist2[(size_t)r * a.cap + j] = a.w_ref ? tot : 0.f;
        a.loss[(size_t)r * a.cap + j] = ls / ((float)K_of_update * (float)m);
      }
      ++j;
    };

    int st = 0;
    uint32_t par_full = 0;
    bool pending = false;     // tile it - 1 still waits for its gradient pass
    int st_prev = 0;
    if (!ASYNC) {
      // ---- synchronous variants: one flat loop; the parameters change once per update, in tensor memory ----
      for (long long it = 0; my_iters > 0; ++it) {
        const int buf = (int)(it & 1);
        if (!sws_wait(smem_addr(&full[st]), par_full, abort_s)) { failed = true; break; }
        const TmTileInfo ti = info_s[st];
        logit_pass(st, buf);
        // gradient pass of the previous tile, whose softmax terms were formed while this one's logits ran
        if (pending) {
          if (!sws_wait(smem_addr(&dready[buf ^ 1]), (uint32_t)(((it - 1) >> 1) & 1), abort_s)) { failed = true; break; }
          gradient_pass(st_prev, buf ^ 1);
        }
        pending = true;
        st_prev = st;
        if (ti.flags & TILE_LAST_OF_UPDATE) {
          // the update needs this tile's gradient too: the pipeline drains here
          if (!sws_wait(smem_addr(&dready[buf]), (uint32_t)((it >> 1) & 1), abort_s)) { failed = true; break; }
          gradient_pass(st, buf);
          pending = false;
          if (!fma_barrier()) { failed = true; break; }     // every warp is through the logit pass that read these parameters
          const float scale = (float)((double)a.eta / ((double)ti.K * (double)m));
          float dd = 0.f;
#pragma unroll
          for (int k = 0; k < KP; ++k) {
            const int p = tid + NT * k;
            float w[WC];
            tm_ld20(t_own + k * WC, w);
            tm_wait_ld();
            float s0 = 0.f, s1 = 0.f;      // sum of the nine accumulated slots, in slot order
#pragma unroll
            for (int c = 0; c < CP; ++c) {
              float g0, g1;
              if (c < GC) {
                unpack2(G[c][k], g0, g1);
                G[c][k] = 0ull;
                s0 += g0; s1 += g1;
              } else {
                g0 = C == CP ? -s0 : 0.f;
                g1 = C == CP ? -s1 : 0.f;
              }
              w[2 * c] = fmaf(-scale, g0, w[2 * c]);
              w[2 * c + 1] = fmaf(-scale, g1, w[2 * c + 1]);
              if (a.w_ref && p < dp && c < C) {
                const float2 wr = reinterpret_cast<const float2*>(a.w_ref + (size_t)c * d)[p];
                const float e0 = w[2 * c] - wr.x, e1 = w[2 * c + 1] - wr.y;
                dd = fmaf(e0, e0, dd); dd = fmaf(e1, e1, dd);
              }
            }
            tm_st20(t_own + k * WC, w);
          }
          dd = warp_sum(dd);
          if (lane == 0) misc_s[warp] = dd;
          tm_wait_st();
          if (!fma_barrier()) { failed = true; break; }     // the parameters in tensor memory are the next tile's
          record(ti.K);
        }
        if (ti.flags & TILE_LAST_OF_RUN) break;
        if (++st == S) { st = 0; par_full ^= 1u; }
      }
    } else {
      // ---- asynchronous variants: every task brings another snapshot, so the parameters change every few tiles.  The
      //      tile loop is kept free of the reload's and the update's calls and global traffic: with them inside it, the
      //      loop's own state lived on the stack (17 local loads and stores a tile, 40 % more time per row) ----
      long long it = 0;
      bool running = my_iters > 0;
      while (running) {
        TmTileInfo ti;
        int buf;
        for (;;) {
          buf = (int)(it & 1);
          if (!sws_wait(smem_addr(&full[st]), par_full, abort_s)) { failed = true; break; }
          ti = info_s[st];
          logit_pass(st, buf);
          if (pending) {
            if (!sws_wait(smem_addr(&dready[buf ^ 1]), (uint32_t)(((it - 1) >> 1) & 1), abort_s)) { failed = true; break; }
            gradient_pass(st_prev, buf ^ 1);
          }
          pending = true;
          st_prev = st;
          if (ti.flags & TILE_LAST_OF_TASK) break;          // (the last tile of an update or of the run is the last of a task)
          ++it;
          if (++st == S) { st = 0; par_full ^= 1u; }
        }
        if (failed) break;
        const bool last_of_update = (ti.flags & TILE_LAST_OF_UPDATE) != 0;
        const bool reload = !(ti.flags & TILE_LAST_OF_RUN);
        if (last_of_update) {
          if (!sws_wait(smem_addr(&dready[buf]), (uint32_t)((it >> 1) & 1), abort_s)) { failed = true; break; }
          gradient_pass(st, buf);
          pending = false;
        }
        if (!fma_barrier()) { failed = true; break; }       // every warp is through the logit pass that read these parameters
        if (last_of_update) {
          // the accumulator goes through local memory into a call (see sws_async_update) and starts again at zero
          const float scale = (float)((double)a.eta / ((double)ti.K * (double)m));
          uint64_t Gm[GC * KP];
#pragma unroll
          for (int c = 0; c < GC; ++c)
#pragma unroll
            for (int k = 0; k < KP; ++k) { Gm[c * KP + k] = G[c][k]; G[c][k] = 0ull; }
          float dd = sws_async_update<KP>(Gm, a.pool + ((size_t)r * a.n_slots + cur_slot) * np,
                                          a.pool + ((size_t)r * a.n_slots + ti.fresh) * np, a.w_ref, scale, d, C, tid);
          cur_slot = ti.fresh;
          dd = warp_sum(dd);
          if (lane == 0) misc_s[warp] = dd;
        }
        if (reload) load_w(a.pool + ((size_t)r * a.n_slots + ti.next_snap) * np);   // the next task's snapshot (own elements only)
        tm_wait_st();
        if (!fma_barrier()) { failed = true; break; }       // the parameters in tensor memory are the next tile's
        if (last_of_update) record(ti.K);
        if (ti.flags & TILE_LAST_OF_RUN) running = false;
        ++it;
        if (++st == S) { st = 0; par_full ^= 1u; }
      }
    }

    if (!failed && !ASYNC && my_iters > 0) {
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
  }

  if (failed) {
    *abort_s = 1;                                    // ends the other roles' waits early
    if (lane == 0) atomicExch(a.err, ERR_WAIT_TIMEOUT);
  }
  tm_fence_before();
  __syncthreads();
  if (warp == NW) {
    if (*abort_s && lane == 0) {                     // copies still in flight get a bounded time to land before shared memory is given up
      for (int s = 0; s < S; ++s)
        for (uint32_t par = 0; par < 2; ++par) mbar_wait(smem_addr(&full[s]), par, 1u << 12);
    }
    __syncwarp();
    tm_dealloc(*tmem_slot, SMT_TMEM_COLS);
  }
}

inline size_t softmax_ws_smem_bytes(int S, int T, int d, int m) {
  const int kp = (d / 2 + SWS_FMA_THREADS - 1) / SWS_FMA_THREADS;
  const size_t need = (size_t)SWS_HEAD_BYTES + (size_t)S * T * (2 * SWS_FMA_THREADS * kp) * 4 + (size_t)m * 4;
  // one CTA per SM, whatever the shape: two CTAs' tensor-memory allocations would still fit, a third would wait
  return need < (size_t)(116 << 10) ? (size_t)(116 << 10) : need;
}

// Shapes this kernel takes; the others go to softmax_kernel.
inline bool softmax_ws_supported(int d, int C, int m) {
  const int kp = (d / 2 + SWS_FMA_THREADS - 1) / SWS_FMA_THREADS;
  return C <= SMT_CP && kp >= 1 && kp <= 4 && kp * SWS_NG * SMT_WC <= (int)SMT_TMEM_COLS &&
         softmax_ws_smem_bytes(3, 6, d, m) <= (size_t)(226 << 10);
}

// *fits is set to false (and nothing is launched) if the block's register allocation, as compiled, could not cover the
// split the kernel asks for: the FMA warpgroups would then wait for registers that never come.
template <int KP>
cudaError_t launch_softmax_ws(NumericArgs& a, cudaStream_t stream, bool* fits) {
  constexpr int TG = 2, T = SWS_NG * TG;
  auto kern = a.is_async ? softmax_ws_kernel<KP, TG, true> : softmax_ws_kernel<KP, TG, false>;
  cudaFuncAttributes attr;
  cudaError_t e0 = cudaFuncGetAttributes(&attr, kern);
  if (e0 != cudaSuccess) return e0;
  *fits = attr.numRegs * SWS_THREADS >= SWS_FMA_THREADS * SWS_FMA_REGS + 128 * SWS_HELPER_REGS;
  if (!*fits) return cudaSuccess;
  int S = SWS_MAX_S;   // tiles in the ring: as many as shared memory holds, three at least
  while (S > 3 && softmax_ws_smem_bytes(S, T, a.d, a.m) > (size_t)(226 << 10)) --S;
  const size_t smem = softmax_ws_smem_bytes(S, T, a.d, a.m);
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  a.stages = S;
  kern<<<a.R, SWS_THREADS, smem, stream>>>(a);
  return cudaGetLastError();
}

inline cudaError_t run_softmax_any(NumericArgs& a, int tune_stages, cudaStream_t stream, const char** why) {
  *why = nullptr;
  if (softmax_ws_supported(a.d, a.n_classes, a.m)) {
    const int kp = (a.d / 2 + SWS_FMA_THREADS - 1) / SWS_FMA_THREADS;
    bool fits = true;
    cudaError_t e = cudaSuccess;
    switch (kp) {
      case 1: e = launch_softmax_ws<1>(a, stream, &fits); break;
      case 2: e = launch_softmax_ws<2>(a, stream, &fits); break;
      case 3: e = launch_softmax_ws<3>(a, stream, &fits); break;
      default: e = launch_softmax_ws<4>(a, stream, &fits); break;
    }
    if (!fits) *why = "softmax: the kernel was built with fewer registers per thread than its register split needs";
    return e;
  }
  return run_softmax(a, tune_stages, stream, why);
}

}  // namespace ssim
