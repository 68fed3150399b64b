// Two-layer relu MLP (d - H - C, softmax cross-entropy) under the simulated schedule.
//
// Parameters per version: [W1 (d x H), b1 (H), W2 (H x C row-major), b2 (C)], fp32, kept in a pool of
// immutable versions per replica (W1 block-tiled inside the pool, see w1_tiled_index; row-major to
// callers), plus a bf16 shadow of W1 per version and a bf16 copy of the data set.  The two products over d take bf16 operands and accumulate in fp32
// on the tensor cores:
//     A1 = bf16(X_b) bf16(W1)          (forward,  [m x d] [d x H])
//     dW1 = bf16(X_b)^T bf16(delta1)   (backward, [d x m] [m x H])
// everything else (bias, relu, layer 2, softmax, loss, update) is fp32.
//
// All replicas advance in lock step, one update at a time, with four launches per update (rows,
// forward, head, dw1):
//   forward   (mlp_tc_kernel.cuh) one CTA per (replica, contributor, 128-sample block): A1 = X_b W1 on
//             tcgen05 with the accumulator in tensor memory, then h = relu(A1 + b1), logits, softmax,
//             delta2, delta1 = (delta2 W2^T) . [h > 0]; writes h, delta2, bf16(delta1), partial db1, loss
//   head      one CTA per (replica, 32 hidden units): dW2 = h^T delta2, db2 and db1 summed over the K
//             contributors in a fixed order, b1 / W2 / b2 updated in the same CTA, loss recorded
//   dw1       (mlp_tc_kernel.cuh) persistent, tiles of 128 rows of W1 x up to 256 columns: accumulates
//             X^T delta1 over all K m samples of the update in tensor memory (tcgen05, MN-major
//             operands) and applies W1 <- W1 - (eta/(K m)) dW1 in its epilogue (Eq. 2 / Eq. 3), writing
//             the new version and its transposed bf16 shadow: dW1 never exists in memory
#pragma once
#include <cuda_bf16.h>

#include "linear_kernel.cuh"

namespace ssim {

struct MlpScratch {
  __nv_bfloat16* Xq = nullptr;     // [n][d]                   bf16 copy of the data set
  __nv_bfloat16* W1qT = nullptr;   // [R][n_slots][d/64][H][64] bf16 shadow of every W1 version, transposed and tiled: the
                                   //                          64 k-values of a k-block are contiguous per hidden unit, so the
                                   //                          [H x 64] operand tile of one k-block is one contiguous block
  __nv_bfloat16* D1q = nullptr;    // [R][Kmax][m][H]          bf16(delta1) of the current update
  float* Hact = nullptr;           // [R][Kmax][m][H]          h
  float* D2 = nullptr;             // [R][Kmax][m][16]         delta2
  float* db1_part = nullptr;       // [R][Kmax][m/32][H]       column sums of delta1 per 32-row group
  float* loss_part = nullptr;      // [R][Kmax][m/32]
  int* rows_tab = nullptr;         // [R][Kmax][m]             sample row of every minibatch draw of the current update
  // |w_{j+1} - w_ref|^2 of the current update, in pieces: one partial per (W1 tile, epilogue group) from the dW1 kernel,
  // one per 32 hidden units ([b1 | W2 | b2] part) from the head kernel; the last piece to arrive adds them in index order
  float* dist_w1 = nullptr;        // [R][(d/128) (H/Hn) 2]
  float* dist_head = nullptr;      // [R][H/32]
  int* dist_cnt = nullptr;         // [R] W1 pieces that have arrived
  int H = 0, C = 0, d = 0, m = 0, Kmax = 0, n_slots = 0, R = 0;
  long long n = 0;
};

struct MlpArgs {
  NumericArgs na;
  MlpScratch sc;
  int H, P;
  long long j;            // update being processed
  // forward-only evaluation of the full-data risk (the forward kernel's EVAL form): consecutive 128-row blocks of the
  // data set instead of minibatches, every replica at its current version
  int eval_blocks;              // ceil(n / 128)
  const uint8_t* eval_slot;     // [R] pool slot of the current version (asynchronous variants) or null:
  int eval_parity;              //     then every replica's current version sits in slot eval_parity
  float* eval_part;             // [R][eval_blocks][4] loss sums per 32-row group
};

inline const char* mlp_shape_unsupported(int d, int H, int C, int m) {
  if (H < 64 || H > 512 || H % 64 != 0) return "mlp: hidden width must be a multiple of 64 in [64, 512]";
  if (d % 128 != 0) return "mlp: d must be a multiple of 128";
  if (m % 128 != 0) return "mlp: m must be a multiple of 128";
  if (C < 2 || C > 16) return "mlp: n_classes must be in [2, 16]";
  return nullptr;
}

// ---- small device helpers ---------------------------------------------------------------------
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// slot bookkeeping shared by the kernels: synchronous variants ping-pong between two slots
__device__ __forceinline__ int mlp_cur_slot(const NumericArgs& a, int r, long long j) {
  if (!a.is_async) return (int)(j & 1);
  return j == a.j0 ? (int)a.begin_slot[r] : (int)a.new_slot[(size_t)r * a.cap + (j - 1)];
}
__device__ __forceinline__ int mlp_fresh_slot(const NumericArgs& a, int r, long long j) {
  if (!a.is_async) return (int)((j + 1) & 1);
  return (int)a.new_slot[(size_t)r * a.cap + j];
}
__device__ __forceinline__ int mlp_snap_slot(const NumericArgs& a, int r, long long j, int l) {
  if (!a.is_async) return (int)(j & 1);
  return (int)a.snap_slot[((size_t)r * a.cap + j) * a.K_stride + l];
}

// ---- data preparation ---------------------------------------------------------------------------
__global__ void to_bf16_kernel(const float* src, __nv_bfloat16* dst, long long count) {
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < count; i += (long long)gridDim.x * blockDim.x)
    dst[i] = __float2bfloat16_rn(src[i]);
}
// transposed, k-block-tiled bf16 shadow of W1 in pool slot `slot` of every replica:
// element (k, n) of W1 goes to [(k / 64) * H + n] * 64 + k % 64
__global__ void shadow_w1_kernel(const float* pool, __nv_bfloat16* W1qT, long long slot_stride, int d, int H, int n_slots, int slot, int R) {
  const long long dH = (long long)d * H, total = dH * R;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long r = i / dH, p = i % dH;
    const long long kb = p / (64ll * H), n = (p / 64) % H, kk = p % 64;
    W1qT[((size_t)r * n_slots + slot) * dH + p] =
        __float2bfloat16_rn(pool[((size_t)r * n_slots + slot) * slot_stride + w1_tiled_index(kb * 64 + kk, n, H)]);
  }
}

// ---- sample rows of the update's minibatches, drawn once for all kernels of the update ----------
__global__ void mlp_rows_kernel(MlpArgs g) {
  const NumericArgs& a = g.na;
  const MlpScratch& sc = g.sc;
  const int l = blockIdx.x % sc.Kmax, r = blockIdx.x / sc.Kmax;
  const int K = (int)a.K_used[(size_t)r * a.cap + g.j];
  if (l == 0 && threadIdx.x == 0) sc.dist_cnt[r] = 0;
  if (l >= K) return;
  const size_t ent = ((size_t)r * a.cap + g.j) * a.K_stride + l;
  const uint32_t worker = a.worker[ent], seq = a.seq[ent];
  for (int q = threadIdx.x; q < sc.m; q += blockDim.x) {
    uint32_t idx = draw_index(a.seed, a.replica_base + (uint32_t)r, worker, seq, (uint32_t)q, a.n);
    if ((uint64_t)idx >= a.n) { atomicExch(a.err, ERR_BAD_INDEX); idx = 0; }
    sc.rows_tab[((size_t)r * sc.Kmax + l) * sc.m + q] = (int)idx;
  }
}

// ---- dW2 = h^T delta2, db2, db1 summed over the update's K contributors; b1, W2, b2 update; loss record ----
// One CTA per (replica, 32 hidden columns): the K*m sample rows of the update are dealt to the eight warps
// in chunks of 32 rows; a lane owns one column, holds the chunk's 32 activations in registers (32 loads
// in flight) and reads the rows' delta2 from a per-warp shared-memory copy.  The eight warps' sums are
// added in warp order, then the CTA applies Eq. 2 / Eq. 3 to its 32 rows of W2 and 32 entries of b1; the
// CTA of columns 0..31 also owns b2 and the loss record.  Every sum has a fixed order.
constexpr int MLP_HEAD_THREADS = 256;
__global__ void __launch_bounds__(MLP_HEAD_THREADS, 3) mlp_head_kernel(MlpArgs g) {
  const NumericArgs& a = g.na;
  const MlpScratch& sc = g.sc;
  const int H = sc.H, C = sc.C, m = sc.m, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ncb = H / 32, cb = blockIdx.x % ncb, r = blockIdx.x / ncb;
  const long long j = g.j;
  const int K = (int)a.K_used[(size_t)r * a.cap + j];
  const size_t row_base = (size_t)r * sc.Kmax * m;          // contributors l < K are consecutive blocks of m rows
  const int n_chunks = K * m / 32;
  __shared__ __align__(16) float d2_s[8][32][16];             // per warp: delta2 of the chunk's rows; later the warps' sums
  float accw[16], accb = 0.f;
#pragma unroll
  for (int c = 0; c < 16; ++c) accw[c] = 0.f;
  for (int ch = warp; ch < n_chunks; ch += 8) {
    const size_t row0 = row_base + (size_t)ch * 32;
    float hv[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) hv[i] = sc.Hact[(row0 + i) * H + cb * 32 + lane];
    float4 dl[4];
#pragma unroll
    for (int c4 = 0; c4 < 4; ++c4) dl[c4] = reinterpret_cast<const float4*>(sc.D2 + (row0 + lane) * 16)[c4];
    __syncwarp();
#pragma unroll
    for (int c4 = 0; c4 < 4; ++c4) reinterpret_cast<float4*>(&d2_s[warp][lane][0])[c4] = dl[c4];
    __syncwarp();
    if (cb == 0 && lane < 16) {                               // db2: lane c sums class c over the chunk's rows
#pragma unroll 8
      for (int i = 0; i < 32; ++i) accb += d2_s[warp][i][lane];
    }
#pragma unroll
    for (int i = 0; i < 32; ++i) {
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4) {
        const float4 dv = reinterpret_cast<const float4*>(&d2_s[warp][i][0])[c4];
        accw[4 * c4] = fmaf(hv[i], dv.x, accw[4 * c4]); accw[4 * c4 + 1] = fmaf(hv[i], dv.y, accw[4 * c4 + 1]);
        accw[4 * c4 + 2] = fmaf(hv[i], dv.z, accw[4 * c4 + 2]); accw[4 * c4 + 3] = fmaf(hv[i], dv.w, accw[4 * c4 + 3]);
      }
    }
  }
  __syncwarp();
#pragma unroll
  for (int c4 = 0; c4 < 4; ++c4)
    reinterpret_cast<float4*>(&d2_s[warp][lane][0])[c4] = make_float4(accw[4 * c4], accw[4 * c4 + 1], accw[4 * c4 + 2], accw[4 * c4 + 3]);
  __shared__ float b2_s[8][16];
  if (cb == 0 && lane < 16) b2_s[warp][lane] = accb;
  __syncthreads();

  const long long dH = (long long)sc.d * H;
  const int cur = mlp_cur_slot(a, r, j), fresh = mlp_fresh_slot(a, r, j);
  const float scale = (float)((double)a.eta / ((double)K * (double)m));
  const float* wc = a.pool + ((size_t)r * a.n_slots + cur) * a.slot_stride + dH;      // [b1 | W2 | b2] of w_j
  float* wn = a.pool + ((size_t)r * a.n_slots + fresh) * a.slot_stride + dH;
  // with a reference vector: this CTA's share of |w_{j+1} - w_ref|^2 (its entries of b1, W2, b2), summed in a fixed order
  const float* wref = a.w_ref ? a.w_ref + dH : nullptr;
  float dd = 0.f;
  auto dist_term = [&](size_t p, float w_new) { if (wref) { const float e = w_new - wref[p]; dd = fmaf(e, e, dd); } };
  // W2 rows cb*32 .. cb*32+31: 32 x C consecutive parameters
  for (int e = tid; e < 32 * C; e += MLP_HEAD_THREADS) {
    const int col = e / C, c = e % C;
    float gsum = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) gsum += d2_s[w][col][c];
    const size_t p = (size_t)H + (size_t)(cb * 32) * C + e;
    const float w_new = fmaf(-scale, gsum, wc[p]);
    wn[p] = w_new;
    dist_term(p, w_new);
  }
  if (tid < 32) {                                             // b1: partial column sums of delta1 written by the forward kernel
    const int col = cb * 32 + tid, parts = m / 32;
    float gsum = 0.f;
    for (int q = 0; q < K * parts; ++q) gsum += sc.db1_part[((size_t)r * sc.Kmax * parts + q) * H + col];
    const float w_new = fmaf(-scale, gsum, wc[col]);
    wn[col] = w_new;
    dist_term((size_t)col, w_new);
  }
  if (cb == 0 && warp == 1) {
    if (lane < C) {
      float gsum = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) gsum += b2_s[w][lane];
      const size_t p = (size_t)H + (size_t)H * C + lane;
      const float w_new = fmaf(-scale, gsum, wc[p]);
      wn[p] = w_new;
      dist_term(p, w_new);
    }
    if (lane == 31) {
      const int parts = m / 32;
      float ls = 0.f;
      for (int q = 0; q < K * parts; ++q) ls += sc.loss_part[(size_t)r * sc.Kmax * parts + q];
      a.loss[(size_t)r * a.cap + j] = ls / ((float)K * (float)m);
      if (!wref) a.dist2[(size_t)r * a.cap + j] = 0.f;      // otherwise the dW1 kernel records it once W1 is updated
    }
  }
  if (wref) {
    __shared__ float dist_s[8];
    dd = warp_sum(dd);
    if (lane == 0) dist_s[warp] = dd;
    __syncthreads();
    if (tid == 0) {
      float tot = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) tot += dist_s[w];
      sc.dist_head[(size_t)r * ncb + cb] = tot;
    }
  }
}

// ---- host side -----------------------------------------------------------------------------------
inline void mlp_scratch_free(MlpScratch& s) {
  cudaFree(s.rows_tab); cudaFree(s.Xq); cudaFree(s.W1qT); cudaFree(s.D1q); cudaFree(s.Hact); cudaFree(s.D2);
  cudaFree(s.db1_part); cudaFree(s.loss_part); cudaFree(s.dist_w1); cudaFree(s.dist_head); cudaFree(s.dist_cnt);
  s = MlpScratch{};
}

inline cudaError_t mlp_scratch_alloc(MlpScratch& s, const float* X, long long n, int d, int H, int C, int m, int Kmax, int R,
                                     int n_slots, cudaStream_t stream) {
  s.H = H; s.C = C; s.d = d; s.m = m; s.Kmax = Kmax; s.n_slots = n_slots; s.R = R; s.n = n;
  const size_t tasks = (size_t)R * Kmax;
  cudaError_t e;
#define MLP_ALLOC(ptr, count) \
  if ((e = cudaMalloc(reinterpret_cast<void**>(&(ptr)), (count) * sizeof(*(ptr)))) != cudaSuccess) return e; \
  if ((e = cudaMemsetAsync((ptr), 0, (count) * sizeof(*(ptr)), stream)) != cudaSuccess) return e;
  MLP_ALLOC(s.Xq, (size_t)n * d)
  MLP_ALLOC(s.W1qT, (size_t)R * n_slots * d * H)
  MLP_ALLOC(s.D1q, tasks * m * H)
  MLP_ALLOC(s.Hact, tasks * m * H)
  MLP_ALLOC(s.D2, tasks * m * 16)
  MLP_ALLOC(s.db1_part, tasks * (m / 32) * H)
  MLP_ALLOC(s.loss_part, tasks * (m / 32))
  MLP_ALLOC(s.rows_tab, tasks * m)
  MLP_ALLOC(s.dist_w1, (size_t)R * (d / 128) * (H / 64) * 2)      // at most H/64 column parts per 128-row slab
  MLP_ALLOC(s.dist_head, (size_t)R * (H / 32))
  MLP_ALLOC(s.dist_cnt, (size_t)R)
#undef MLP_ALLOC
  to_bf16_kernel<<<1184, 256, 0, stream>>>(X, s.Xq, (long long)n * d);
  return cudaGetLastError();
}

// after the initial parameters went into slot 0 of every replica
inline cudaError_t mlp_after_set_params(MlpScratch& s, const float* pool, long long slot_stride, cudaStream_t stream) {
  shadow_w1_kernel<<<1184, 256, 0, stream>>>(pool, s.W1qT, slot_stride, s.d, s.H, s.n_slots, 0, s.R);
  return cudaGetLastError();
}

}  // namespace ssim
