// Gradient / update kernel for softmax regression, W in R^{C x d} (C <= 16).
//
// One CTA of 384 threads per replica, same producer / schedule walk as the single-output kernel
// (rows staged by bulk asynchronous copies, several tiles ahead).  W_tau stays in shared memory
// for a whole task (for the synchronous variants it is w_j itself and is updated in place);
// each thread owns a fixed set of columns and keeps the C x (its columns) block of the gradient
// accumulator G in registers for the whole update.  Per tile of 4 rows:
//   x (own columns) -> registers, the stage is handed back to the producer at once
//   Z = X_tile W_tau^T   partial over own columns, classes in two halves; warp transposition
//                        reduce (31 shuffles per half), cross-warp sum by 64 threads
//   D = softmax(Z) - onehot(label), loss                       (those 64 threads, 16 lanes a row)
//   G += D^T X_tile      from the registers that still hold x
// and at the end of the update W <- W - (eta / (K m)) G  (Eq. 2 / Eq. 3).
// Plain fp32 FMAs: at 20 FMA per 4-byte feature this path sits at the fp32 ridge, not on the
// tensor cores.
#pragma once
#include "linear_kernel.cuh"

namespace ssim {

constexpr int SMX_NT = 384;
constexpr int SMX_T = 4;
constexpr int SMX_HEAD_BYTES = 3840;   // multiple of 128

template <int O, int N>
__device__ __forceinline__ void transpose_reduce_step(float (&v)[32], int lane) {
  const bool up = (lane & O) != 0;
#pragma unroll
  for (int i = 0; i < N / 2; ++i) {
    const float send = up ? v[i] : v[i + N / 2];
    const float keep = up ? v[i + N / 2] : v[i];
    v[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, O);
  }
}
// After the call, v[0] on lane L is the sum over the warp of the callers' v[L].
__device__ __forceinline__ void warp_transpose_reduce(float (&v)[32], int lane) {
  transpose_reduce_step<16, 32>(v, lane);
  transpose_reduce_step<8, 16>(v, lane);
  transpose_reduce_step<4, 8>(v, lane);
  transpose_reduce_step<2, 4>(v, lane);
  transpose_reduce_step<1, 2>(v, lane);
}

// Two fp32 FMAs in one instruction (each half rounds like fmaf): halves the issue slots of the two products.
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
  return d;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }

template <int CHUNKS, int CP, bool ASYNC>
__global__ void __launch_bounds__(SMX_NT) softmax_kernel(NumericArgs a) {
  constexpr int NT = SMX_NT, NW = NT / 32, T = SMX_T, E = 4 * CHUNKS, CH = CP / 2;
  static_assert(CP % 2 == 0 && T * CH <= 32, "class halves must fit one transposition reduce");
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r = blockIdx.x;
  const int d = a.d, d4 = d >> 2, S = a.stages, m = a.m, C = a.n_classes;
  const uint32_t rid = a.replica_base + (uint32_t)r;
  const uint32_t row_bytes = (uint32_t)d * 4u;
  const size_t np = (size_t)C * d;
  const long long my_j0 = a.run_j0 ? a.run_j0[r] : a.j0, my_iters = a.run_iters ? a.run_iters[r] : a.iters;

  extern __shared__ __align__(128) unsigned char smem[];
  // fixed head (S <= 8), every array on a 16-byte boundary:
  //   barriers [8] @0 | delta [T][16] @64 | red [NW][64] @320 | misc [NW] | lossrow [T] | y [8][T] | TileInfo [8]
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);
  float* delta_s = reinterpret_cast<float*>(smem + 64);
  float* red_s = delta_s + T * 16;
  float* misc_s = red_s + NW * 64;
  float* lossrow_s = misc_s + NW;
  uint32_t* y_s = reinterpret_cast<uint32_t*>(lossrow_s + T);
  TileInfo* info_s = reinterpret_cast<TileInfo*>(y_s + 8 * T);
  static_assert(64 + 4 * (T * 16 + NW * 64 + NW + T + 8 * T) + 8 * sizeof(TileInfo) <= SMX_HEAD_BYTES, "head too small");
  float* W_s = reinterpret_cast<float*>(smem + SMX_HEAD_BYTES);
  float* rows_s = W_s + np;
  uint32_t* pidx_s = reinterpret_cast<uint32_t*>(rows_s + (size_t)S * T * d);   // [m] sample rows of the producer's task

  if (tid == 0) {
    for (int s = 0; s < S; ++s) mbar_init(smem_addr(&full[s]), (uint32_t)T + 1u);
    mbar_fence_init();
  }
  int cur_slot = ASYNC ? (int)a.begin_slot[r] : 0;
  if (!ASYNC) {
    const float4* src = reinterpret_cast<const float4*>(a.w_state + (size_t)r * np);
    for (size_t i = tid; i < np / 4; i += NT) reinterpret_cast<float4*>(W_s)[i] = src[i];
  }
  __syncthreads();

  ScheduleWalk walk;
  walk.done = true;
  int prod_st = 0;
  auto issue_tile = [&](long long) {
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
  if (warp == 0) {
    walk.start(a, r, my_j0, my_iters);
    walk.tiles_per_task = (m + T - 1) / T;
    for (int s = 0; s < S; ++s) issue_tile(s);
  }
  __syncthreads();
  if (my_iters <= 0) return;

  uint64_t G[CP][E / 2];      // pairs of adjacent columns
#pragma unroll
  for (int c = 0; c < CP; ++c)
#pragma unroll
    for (int e = 0; e < E / 2; ++e) G[c][e] = 0ull;
  float loss_acc = 0.f;      // meaningful in the row-leader threads of the softmax stage
  long long j = my_j0;
  bool failed = false;
  // role in the softmax stage: 16 lanes per row
  const int st_tid = tid - (NT - 16 * T);          // the last two warps serve the softmax stage (warp 0 is the producer)
  const int sq = st_tid >> 4, sc = st_tid & 15;

  int st = 0;             // stage and phase parity of tile `it`, kept as counters (it % S and it / S are 64-bit divisions)
  uint32_t parity = 0;
  for (long long it = 0;; ++it, parity ^= (uint32_t)(st + 1 == S), st = (st + 1 == S ? 0 : st + 1)) {
    // a wait that runs out is voted on by the whole block, so that every thread drains or none does
    if (__syncthreads_or(!mbar_wait(smem_addr(&full[st]), parity))) { failed = true; break; }
    const TileInfo ti = info_s[st];
    const float* tile = rows_s + (size_t)st * T * d;

    if (ASYNC && (ti.flags & TILE_FIRST_OF_TASK)) {
      const float4* src = reinterpret_cast<const float4*>(a.pool + ((size_t)r * a.n_slots + ti.snap) * np);
      for (size_t i = tid; i < np / 4; i += NT) reinterpret_cast<float4*>(W_s)[i] = src[i];
      __syncthreads();
    }

    // ---- x of own columns -> registers; label of the row this thread serves in the softmax stage ----
    uint64_t x[T][E / 2];      // pairs of adjacent columns, as the 16-byte loads deliver them
#pragma unroll
    for (int c = 0; c < CHUNKS; ++c) {
      const int ci = tid + NT * c;
#pragma unroll
      for (int q = 0; q < T; ++q) {
        ulonglong2 v = make_ulonglong2(0ull, 0ull);
        if (ci < d4 && q < ti.rows) v = reinterpret_cast<const ulonglong2*>(tile + (size_t)q * d)[ci];
        x[q][2 * c] = v.x; x[q][2 * c + 1] = v.y;
      }
    }
    int label = 0;
    if (st_tid >= 0 && sq < ti.rows) label = (int)y_s[st * T + sq];

    // ---- Z partials over own columns, one half of the classes at a time ----
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      float v[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = 0.f;
#pragma unroll
      for (int c = 0; c < CHUNKS; ++c) {
        const int ci = tid + NT * c;
        if (ci < d4) {
#pragma unroll
          for (int cc = 0; cc < CH; ++cc) {
            const int cls = h * CH + cc;
            if (cls < C) {
              const float4 w = reinterpret_cast<const float4*>(W_s + (size_t)cls * d)[ci];
#pragma unroll
              for (int q = 0; q < T; ++q) {
                float x0, x1, x2, x3;
                unpack2(x[q][2 * c], x0, x1);
                unpack2(x[q][2 * c + 1], x2, x3);
                float acc = v[q * CH + cc];
                acc = fmaf(x0, w.x, acc);
                acc = fmaf(x1, w.y, acc);
                acc = fmaf(x2, w.z, acc);
                acc = fmaf(x3, w.w, acc);
                v[q * CH + cc] = acc;
              }
            }
          }
        }
      }
      warp_transpose_reduce(v, lane);
      red_s[warp * 64 + h * 32 + lane] = v[0];
    }
    __syncthreads();   // (A) partial logits published; this tile's stage is free again
    if (warp == 0) issue_tile(it + S);

    // ---- softmax stage: thread (sq, sc) owns logit (row sq, class sc) ----
    if (st_tid >= 0) {
      float z = -INFINITY;
      const bool live = sc < C && sq < ti.rows;
      if (live) {
        const int h = sc / CH, cc = sc - h * CH;
        float acc = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) acc += red_s[w * 64 + h * 32 + sq * CH + cc];
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
      const float ssum = 1.f + sexcl;
      const float zlab = __shfl_sync(0xFFFFFFFFu, z, (lane & 16) + label);
      float dl = 0.f;
      if (live) {
        if (is_max) dl = sc == label ? -sexcl / ssum : 1.f / ssum;
        else dl = ez / ssum - (sc == label ? 1.f : 0.f);
      }
      delta_s[sq * 16 + sc] = dl;
      if (sc == 0 && sq < ti.rows) loss_acc += log1pf(sexcl) + (zmax - zlab);
    }
    __syncthreads();   // (B)

    // ---- G += D^T X over own columns ----
#pragma unroll
    for (int q = 0; q < T; ++q) {
      if (q < ti.rows) {
#pragma unroll
        for (int c4 = 0; c4 < (CP + 3) / 4; ++c4) {
          const float4 dv = reinterpret_cast<const float4*>(delta_s + q * 16)[c4];
          const float dl[4] = {dv.x, dv.y, dv.z, dv.w};
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int cls = 4 * c4 + k;
            if (cls < CP) {
              const uint64_t dd2 = pack2(dl[k], dl[k]);
#pragma unroll
              for (int e = 0; e < E / 2; ++e) G[cls][e] = ffma2(dd2, x[q][e], G[cls][e]);
            }
          }
        }
      }
    }

    if (ti.flags & TILE_LAST_OF_UPDATE) {
      const float scale = (float)((double)a.eta / ((double)ti.K * (double)m));
      float dd = 0.f;
      const float* w_from = ASYNC ? a.pool + ((size_t)r * a.n_slots + cur_slot) * np : W_s;
      float* w_to = ASYNC ? a.pool + ((size_t)r * a.n_slots + ti.fresh) * np : W_s;
#pragma unroll
      for (int c = 0; c < CHUNKS; ++c) {
        const int ci = tid + NT * c;
        if (ci < d4) {
#pragma unroll
          for (int cls = 0; cls < CP; ++cls) {
            if (cls < C) {
              float4 w = reinterpret_cast<const float4*>(w_from + (size_t)cls * d)[ci];
              float g0, g1, g2, g3;
              unpack2(G[cls][2 * c], g0, g1);
              unpack2(G[cls][2 * c + 1], g2, g3);
              w.x = fmaf(-scale, g0, w.x);
              w.y = fmaf(-scale, g1, w.y);
              w.z = fmaf(-scale, g2, w.z);
              w.w = fmaf(-scale, g3, w.w);
              reinterpret_cast<float4*>(w_to + (size_t)cls * d)[ci] = w;
              if (a.w_ref) {
                const float4 wr = reinterpret_cast<const float4*>(a.w_ref + (size_t)cls * d)[ci];
                const float e0 = w.x - wr.x, e1 = w.y - wr.y, e2 = w.z - wr.z, e3 = w.w - wr.w;
                dd = fmaf(e0, e0, dd); dd = fmaf(e1, e1, dd); dd = fmaf(e2, e2, dd); dd = fmaf(e3, e3, dd);
              }
            }
            G[cls][2 * c] = 0ull; G[cls][2 * c + 1] = 0ull;
          }
        }
      }
      if (ASYNC) cur_slot = ti.fresh;
      dd = warp_sum(dd);
      if (lane == 0) misc_s[warp] = dd;
      if (st_tid >= 0 && sc == 0) lossrow_s[sq] = loss_acc;
      __syncthreads();   // (C)
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
    __syncthreads();
    return;
  }
  if (!ASYNC) {
    __syncthreads();
    float4* dst = reinterpret_cast<float4*>(a.w_state + (size_t)r * np);
    for (size_t i = tid; i < np / 4; i += NT) dst[i] = reinterpret_cast<const float4*>(W_s)[i];
  }
}

inline size_t softmax_smem_bytes(int S, int d, int C, int m) {
  return (size_t)SMX_HEAD_BYTES + (size_t)C * d * 4 + (size_t)S * SMX_T * d * 4 + (size_t)m * 4;
}

inline const char* softmax_shape_unsupported(int d, int C, int m) {
  const int d4 = d / 4;
  if (C <= 10 && d4 > 2 * SMX_NT) return "softmax: d > 3072 is not supported for up to 10 classes";
  if (C > 10 && d4 > SMX_NT) return "softmax: d > 1536 is not supported for more than 10 classes";
  if (softmax_smem_bytes(2, d, C, m) > (size_t)(226 << 10)) return "softmax: W and two row tiles do not fit in shared memory";
  return nullptr;
}

template <int CHUNKS, int CP>
cudaError_t launch_softmax(NumericArgs& a, int S, size_t smem, cudaStream_t stream) {
  auto kern = a.is_async ? softmax_kernel<CHUNKS, CP, true> : softmax_kernel<CHUNKS, CP, false>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kern<<<a.R, SMX_NT, smem, stream>>>(a);
  return cudaGetLastError();
}

inline cudaError_t run_softmax(NumericArgs& a, int tune_stages, cudaStream_t stream, const char** why) {
  *why = softmax_shape_unsupported(a.d, a.n_classes, a.m);
  if (*why) return cudaSuccess;
  int S = tune_stages > 0 ? tune_stages : 8;
  while (S > 2 && softmax_smem_bytes(S, a.d, a.n_classes, a.m) > (size_t)(226 << 10)) --S;
  const size_t smem = softmax_smem_bytes(S, a.d, a.n_classes, a.m);
  a.stages = S;
  const int d4 = a.d / 4;
  if (a.n_classes <= 10) return d4 <= SMX_NT ? launch_softmax<1, 10>(a, S, smem, stream) : launch_softmax<2, 10>(a, S, smem, stream);
  return launch_softmax<1, 16>(a, S, smem, stream);
}

}  // namespace ssim
