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
//   forward   (mlp_tc_kernel.cuh) persistent, tiles of one (replica, contributor, 128-sample block) x up to
//             256 hidden units: A1 = X_b W1 on tcgen05 with the accumulator double-buffered in tensor
//             memory; the epilogue of one tile (h = relu(A1 + b1) and the tile's share of the logits h W2)
//             runs under the next tile's main loop; writes h and the partial logits
//   head      one CTA per (replica, 32 hidden units): logits = b2 + partial logits, softmax, delta2, loss;
//             dW2 = h^T delta2, delta1 = (delta2 W2^T) . [h > 0] (stored in bf16 for the dw1 kernel), db2 and
//             db1 summed over the K contributors in a fixed order, b1 / W2 / b2 updated in the same CTA
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
  float* ZP = nullptr;             // [R][Kmax][m][halves][16] h W2 over each half of the hidden units (one half if H <= 256)
  int* rows_tab = nullptr;         // [R][Kmax][m]             sample row of every minibatch draw of the current update
  int* label_tab = nullptr;        // [R][Kmax][m]             and its label
  // |w_{j+1} - w_ref|^2 of the current update, in pieces: one partial per (W1 tile, epilogue group) from the dW1 kernel,
  // one per 64 hidden units ([b1 | W2 | b2] part) from the head kernel; the last piece to arrive adds them in index order
  float* dist_w1 = nullptr;        // [R][(d/128) (H/Hn) 2]
  float* dist_head = nullptr;      // [R][H/64]
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
    sc.label_tab[((size_t)r * sc.Kmax + l) * sc.m + q] = reinterpret_cast<const int*>(a.y)[idx];
  }
}

// Softmax cross-entropy of one sample from its logits z[0..C) (C <= 16): returns the sample's loss and, if wanted,
// delta2 = softmax(z) - onehot(lab) in d2 (zeros past C).  Exponentials without the maximal class keep log(1 + s) and
// p_max - 1 = -s / (1 + s) accurate for wide margins.  z is overwritten.
template <bool WANT_D2>
__device__ __forceinline__ float mlp_row_softmax(float (&z)[16], int C, int lab, float (&d2)[16]) {
  float zmax = -INFINITY;
#pragma unroll
  for (int c = 0; c < 16; ++c) { if (c >= C) z[c] = -INFINITY; zmax = fmaxf(zmax, z[c]); }
  int cmax = 0;
#pragma unroll
  for (int c = 15; c >= 0; --c) if (c < C && z[c] == zmax) cmax = c;
  float zl = 0.f;
#pragma unroll
  for (int c = 0; c < 16; ++c) if (c == lab) zl = z[c];
  float sexcl = 0.f;
#pragma unroll
  for (int c = 0; c < 16; ++c) { z[c] = (c < C && c != cmax) ? expf(z[c] - zmax) : 0.f; sexcl += z[c]; }
  if (WANT_D2) {
    const float ssum = 1.f + sexcl;
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      float dl = 0.f;
      if (c < C) {
        if (c == cmax) dl = c == lab ? -sexcl / ssum : 1.f / ssum;
        else dl = z[c] / ssum - (c == lab ? 1.f : 0.f);
      }
      d2[c] = dl;
    }
  }
  return log1pf(sexcl) + (zmax - zl);
}

// ---- layer 2 and the small parameters: logits, softmax, delta2, loss; dW2 = h^T delta2, delta1, db1, db2 summed over
//      the update's K contributors; b1, W2, b2 update; loss record ----
// One CTA per (replica, 64 hidden columns): the K*m sample rows of the update are dealt to the eight warps
// in chunks of 32 rows.  For a chunk a lane first takes one row: logits = (b2 + partial logits of the first half of the
// hidden units) + those of the second, softmax, delta2 into a per-warp shared-memory copy (every CTA of the replica
// repeats this cheap step rather than wait for one that does it).  Then a lane owns two neighbouring columns: it holds
// their activations of 8 rows in registers, with the next 8 rows' already requested, and their rows of the contributor's W2, and forms for
// every row its terms of dW2 and delta1 = (delta2 . W2 row) [h > 0], which leaves in bf16 for the dW1 kernel and in fp32
// for db1.  Two columns a lane because every row's delta2 is a broadcast read of shared memory, whose return path moves
// 128 B a clock: with one column the kernel was bound by it.  The eight warps' sums are added in warp order, then the CTA
// applies Eq. 2 / Eq. 3 to its 64 rows of W2 and 64 entries of b1; the CTA of columns 0..63 also owns b2 and the loss
// record.  Every sum has a fixed order.  C4 = ceil(C / 4), the float4 groups of a class vector that are in use.
constexpr int MLP_HEAD_THREADS = 256;
constexpr int MLP_HEAD_COLS = 64;
template <int C4>
__global__ void __launch_bounds__(MLP_HEAD_THREADS, 2) mlp_head_kernel(MlpArgs g) {
  const NumericArgs& a = g.na;
  const MlpScratch& sc = g.sc;
  const int H = sc.H, C = sc.C, m = sc.m, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ncb = H / MLP_HEAD_COLS, cb = blockIdx.x % ncb, r = blockIdx.x / ncb;
  const int n_halves = H > 256 ? 2 : 1;
  const long long j = g.j;
  const long long dH = (long long)sc.d * H;
  const int K = (int)a.K_used[(size_t)r * a.cap + j];
  const size_t row_base = (size_t)r * sc.Kmax * m;          // contributors l < K are consecutive blocks of m rows
  const int n_chunks = K * m / 32;
  const int col0 = cb * MLP_HEAD_COLS + 2 * lane;             // this lane's columns: col0, col0 + 1
  // per warp: delta2 of the chunk's rows; after the row loop the same bytes take the warps' sums of dW2
  constexpr int D2W = 4 * C4;
  constexpr int BUF_FLOATS = 8 * MLP_HEAD_COLS * D2W > 8 * 32 * D2W ? 8 * MLP_HEAD_COLS * D2W : 8 * 32 * D2W;
  __shared__ __align__(16) float buf_s[BUF_FLOATS];
  float (*d2_s)[32][D2W] = reinterpret_cast<float (*)[32][D2W]>(buf_s);
  float (*sum_s)[MLP_HEAD_COLS][D2W] = reinterpret_cast<float (*)[MLP_HEAD_COLS][D2W]>(buf_s);
  __shared__ float b2_s[8][16], b1_s[8][MLP_HEAD_COLS], loss_s[8];
  float accw[2][D2W], accb = 0.f, accb1[2] = {0.f, 0.f}, lossw = 0.f;
#pragma unroll
  for (int c = 0; c < D2W; ++c) { accw[0][c] = 0.f; accw[1][c] = 0.f; }
  // activations of 8 rows of this lane's two columns; two such groups are in flight, one being used, one on its way
  auto load_h = [&](float2 (&hv)[8], size_t rows) {
#pragma unroll
    for (int i = 0; i < 8; ++i) hv[i] = *reinterpret_cast<const float2*>(sc.Hact + (rows + i) * H + col0);
  };
  float2 hv[8], hvn[8];
  if (warp < n_chunks) load_h(hv, row_base + (size_t)warp * 32);
  for (int ch = warp; ch < n_chunks; ch += 8) {
    const size_t row0 = row_base + (size_t)ch * 32;
    const int l = (ch * 32) / m;
    const float* wsnap = a.pool + ((size_t)r * a.n_slots + mlp_snap_slot(a, r, j, l)) * a.slot_stride + dH;   // [b1 | W2 | b2] the contributor read
    float w2r[2][D2W];                                        // the contributor's W2 rows of this lane's columns
#pragma unroll
    for (int c = 0; c < D2W; ++c) {
      w2r[0][c] = c < C ? wsnap[(size_t)H + (size_t)col0 * C + c] : 0.f;
      w2r[1][c] = c < C ? wsnap[(size_t)H + (size_t)(col0 + 1) * C + c] : 0.f;
    }
    {
      // lane = row: logits in the order b2 + first half + second half, then softmax
      const float4* zp = reinterpret_cast<const float4*>(sc.ZP + (row0 + lane) * n_halves * 16);
      const float* b2 = wsnap + (size_t)H + (size_t)H * C;
      float z[16], d2[16];
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4) {
        if (c4 < C4) {
          const float4 p0 = zp[c4];
          z[4 * c4] = (4 * c4 < C ? b2[4 * c4] : 0.f) + p0.x;
          z[4 * c4 + 1] = (4 * c4 + 1 < C ? b2[4 * c4 + 1] : 0.f) + p0.y;
          z[4 * c4 + 2] = (4 * c4 + 2 < C ? b2[4 * c4 + 2] : 0.f) + p0.z;
          z[4 * c4 + 3] = (4 * c4 + 3 < C ? b2[4 * c4 + 3] : 0.f) + p0.w;
          if (n_halves == 2) {
            const float4 p1 = zp[4 + c4];
            z[4 * c4] += p1.x; z[4 * c4 + 1] += p1.y; z[4 * c4 + 2] += p1.z; z[4 * c4 + 3] += p1.w;
          }
        } else {
          z[4 * c4] = 0.f; z[4 * c4 + 1] = 0.f; z[4 * c4 + 2] = 0.f; z[4 * c4 + 3] = 0.f;
        }
      }
      const float rowloss = mlp_row_softmax<true>(z, C, sc.label_tab[row0 + lane], d2);
      if (cb == 0) lossw += warp_sum(rowloss);
      __syncwarp();
#pragma unroll
      for (int c4 = 0; c4 < C4; ++c4)
        reinterpret_cast<float4*>(&d2_s[warp][lane][0])[c4] = make_float4(d2[4 * c4], d2[4 * c4 + 1], d2[4 * c4 + 2], d2[4 * c4 + 3]);
      __syncwarp();
    }
    if (cb == 0 && lane < D2W) {                              // db2: lane c sums class c over the chunk's rows
#pragma unroll 8
      for (int i = 0; i < 32; ++i) accb += d2_s[warp][i][lane];
    }
    // groups of 8 rows; the loop is kept rolled (one copy of the 8-row body: the instruction cache holds it)
#pragma unroll 1
    for (int grp = 0; grp < 4; ++grp) {
      if (grp < 3) load_h(hvn, row0 + 8 * (grp + 1));
      else if (ch + 8 < n_chunks) load_h(hvn, row0 + 8 * 32);   // the next chunk's first rows, on their way during its softmax step
      __nv_bfloat162* dout = reinterpret_cast<__nv_bfloat162*>(sc.D1q + (row0 + 8 * grp) * H + col0);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float a0 = 0.f, a1 = 0.f;
#pragma unroll
        for (int c4 = 0; c4 < C4; ++c4) {
          const float4 dv = reinterpret_cast<const float4*>(&d2_s[warp][8 * grp + i][0])[c4];
          accw[0][4 * c4] = fmaf(hv[i].x, dv.x, accw[0][4 * c4]); accw[0][4 * c4 + 1] = fmaf(hv[i].x, dv.y, accw[0][4 * c4 + 1]);
          accw[0][4 * c4 + 2] = fmaf(hv[i].x, dv.z, accw[0][4 * c4 + 2]); accw[0][4 * c4 + 3] = fmaf(hv[i].x, dv.w, accw[0][4 * c4 + 3]);
          accw[1][4 * c4] = fmaf(hv[i].y, dv.x, accw[1][4 * c4]); accw[1][4 * c4 + 1] = fmaf(hv[i].y, dv.y, accw[1][4 * c4 + 1]);
          accw[1][4 * c4 + 2] = fmaf(hv[i].y, dv.z, accw[1][4 * c4 + 2]); accw[1][4 * c4 + 3] = fmaf(hv[i].y, dv.w, accw[1][4 * c4 + 3]);
          a0 = fmaf(dv.x, w2r[0][4 * c4], a0); a0 = fmaf(dv.y, w2r[0][4 * c4 + 1], a0);
          a0 = fmaf(dv.z, w2r[0][4 * c4 + 2], a0); a0 = fmaf(dv.w, w2r[0][4 * c4 + 3], a0);
          a1 = fmaf(dv.x, w2r[1][4 * c4], a1); a1 = fmaf(dv.y, w2r[1][4 * c4 + 1], a1);
          a1 = fmaf(dv.z, w2r[1][4 * c4 + 2], a1); a1 = fmaf(dv.w, w2r[1][4 * c4 + 3], a1);
        }
        const float d0 = hv[i].x > 0.f ? a0 : 0.f, d1 = hv[i].y > 0.f ? a1 : 0.f;
        dout[(size_t)i * (H / 2)] = __floats2bfloat162_rn(d0, d1);
        accb1[0] += d0; accb1[1] += d1;
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) hv[i] = hvn[i];
    }
  }
  __syncthreads();                                            // every warp is done with its delta2 rows
#pragma unroll
  for (int c4 = 0; c4 < C4; ++c4) {
    reinterpret_cast<float4*>(&sum_s[warp][2 * lane][0])[c4] = make_float4(accw[0][4 * c4], accw[0][4 * c4 + 1], accw[0][4 * c4 + 2], accw[0][4 * c4 + 3]);
    reinterpret_cast<float4*>(&sum_s[warp][2 * lane + 1][0])[c4] = make_float4(accw[1][4 * c4], accw[1][4 * c4 + 1], accw[1][4 * c4 + 2], accw[1][4 * c4 + 3]);
  }
  if (cb == 0 && lane < 16) b2_s[warp][lane] = accb;
  b1_s[warp][2 * lane] = accb1[0];
  b1_s[warp][2 * lane + 1] = accb1[1];
  if (lane == 0) loss_s[warp] = lossw;
  __syncthreads();

  const int cur = mlp_cur_slot(a, r, j), fresh = mlp_fresh_slot(a, r, j);
  const float scale = (float)((double)a.eta / ((double)K * (double)m));
  const float* wc = a.pool + ((size_t)r * a.n_slots + cur) * a.slot_stride + dH;      // [b1 | W2 | b2] of w_j
  float* wn = a.pool + ((size_t)r * a.n_slots + fresh) * a.slot_stride + dH;
  // with a reference vector: this CTA's share of |w_{j+1} - w_ref|^2 (its entries of b1, W2, b2), summed in a fixed order
  const float* wref = a.w_ref ? a.w_ref + dH : nullptr;
  float dd = 0.f;
  auto dist_term = [&](size_t p, float w_new) { if (wref) { const float e = w_new - wref[p]; dd = fmaf(e, e, dd); } };
  // W2 rows cb*64 .. cb*64+63: 64 x C consecutive parameters
  for (int e = tid; e < MLP_HEAD_COLS * C; e += MLP_HEAD_THREADS) {
    const int col = e / C, c = e % C;
    float gsum = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) gsum += sum_s[w][col][c];
    const size_t p = (size_t)H + (size_t)(cb * MLP_HEAD_COLS) * C + e;
    const float w_new = fmaf(-scale, gsum, wc[p]);
    wn[p] = w_new;
    dist_term(p, w_new);
  }
  if (tid < MLP_HEAD_COLS) {                                  // b1
    const int col = cb * MLP_HEAD_COLS + tid;
    float gsum = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) gsum += b1_s[w][tid];
    const float w_new = fmaf(-scale, gsum, wc[col]);
    wn[col] = w_new;
    dist_term((size_t)col, w_new);
  }
  if (cb == 0 && warp == 2) {
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
      float ls = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) ls += loss_s[w];
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
inline void launch_mlp_head(const MlpArgs& g, cudaStream_t stream) {
  const int grid = g.na.R * (g.sc.H / MLP_HEAD_COLS), C4 = (g.sc.C + 3) / 4;
  if (C4 == 1) mlp_head_kernel<1><<<grid, MLP_HEAD_THREADS, 0, stream>>>(g);
  else if (C4 == 2) mlp_head_kernel<2><<<grid, MLP_HEAD_THREADS, 0, stream>>>(g);
  else if (C4 == 3) mlp_head_kernel<3><<<grid, MLP_HEAD_THREADS, 0, stream>>>(g);
  else mlp_head_kernel<4><<<grid, MLP_HEAD_THREADS, 0, stream>>>(g);
}

// ---- host side -----------------------------------------------------------------------------------
inline void mlp_scratch_free(MlpScratch& s) {
  cudaFree(s.rows_tab); cudaFree(s.label_tab); cudaFree(s.Xq); cudaFree(s.W1qT); cudaFree(s.D1q); cudaFree(s.Hact); cudaFree(s.ZP);
  cudaFree(s.dist_w1); cudaFree(s.dist_head); cudaFree(s.dist_cnt);
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
  MLP_ALLOC(s.ZP, tasks * m * (H > 256 ? 2 : 1) * 16)
  MLP_ALLOC(s.rows_tab, tasks * m)
  MLP_ALLOC(s.label_tab, tasks * m)
  MLP_ALLOC(s.dist_w1, (size_t)R * (d / 128) * (H / 64) * 2)      // at most H/64 column parts per 128-row slab
  MLP_ALLOC(s.dist_head, (size_t)R * (H / MLP_HEAD_COLS))
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
