// Two-layer relu MLP (d - H - C, softmax cross-entropy) under the simulated schedule.
//
// Parameters per version: [W1 (d x H row-major), b1 (H), W2 (H x C row-major), b2 (C)], fp32,
// kept in a pool of immutable versions per replica, plus a bf16 shadow of W1 per version and a
// bf16 copy of the data set.  The two products over d take bf16 operands and accumulate in fp32
// on the tensor cores:
//     A1 = bf16(X_b) bf16(W1)          (forward,  [m x d] [d x H])
//     dW1 = bf16(X_b)^T bf16(delta1)   (backward, [d x m] [m x H])
// everything else (bias, relu, layer 2, softmax, loss, update) is fp32.
//
// All replicas advance in lock step, one update at a time, with four launches per update:
//   forward   one CTA per (replica, contributor, 64-sample half): A1 tile 64 x H by mma.sync
//             m16n8k16 (cp.async 3-stage ring, XOR-swizzled shared memory, ldmatrix), then
//             h = relu(A1 + b1), logits, softmax, delta2, delta1 = (delta2 W2^T) . [h > 0];
//             writes h, delta2, bf16(delta1), partial db1 and the loss of its rows
//   head      one CTA per (replica, contributor): dW2 = h^T delta2, db2
//   dw1       one CTA per (replica, 64-row slab of W1): accumulates X^T delta1 over all K m samples
//             of the update in registers and applies W1 <- W1 - (eta/(K m)) dW1 in its epilogue
//             (Eq. 2 / Eq. 3), writing the new version and its bf16 shadow: dW1 never exists in memory
//   small     b1, W2, b2 update from the partials (fixed summation order), loss record
#pragma once
#include <cuda_bf16.h>

#include "linear_kernel.cuh"

namespace ssim {

struct MlpScratch {
  __nv_bfloat16* Xq = nullptr;     // [n][d]                   bf16 copy of the data set
  __nv_bfloat16* W1q = nullptr;    // [R][n_slots][d*H]        bf16 shadow of every W1 version
  __nv_bfloat16* D1q = nullptr;    // [R][Kmax][m][H]          bf16(delta1) of the current update
  float* Hact = nullptr;           // [R][Kmax][m][H]          h
  float* D2 = nullptr;             // [R][Kmax][m][16]         delta2
  float* db1_part = nullptr;       // [R][Kmax][m/64][H]
  float* dW2_part = nullptr;       // [R][Kmax][H*C]
  float* db2_part = nullptr;       // [R][Kmax][16]
  float* loss_part = nullptr;      // [R][Kmax][m/64]
  int H = 0, C = 0, d = 0, m = 0, Kmax = 0, n_slots = 0, R = 0;
  long long n = 0;
};

struct MlpArgs {
  NumericArgs na;
  MlpScratch sc;
  int H, P;
  long long j;            // update being processed
};

constexpr int MLP_BM = 64;          // rows of the output tile per CTA
constexpr int MLP_BK = 64;          // reduction chunk
constexpr int MLP_PITCH_B = 1024;   // bytes per k-row of the B tile (H <= 512 bf16)
constexpr int MLP_STAGE_A = MLP_BM * 128;              // 64 rows x 128 B
constexpr int MLP_STAGE_B = MLP_BK * MLP_PITCH_B;      // 64 k-rows x 1024 B
constexpr int MLP_STAGES = 3;
constexpr int MLP_SMEM = MLP_STAGES * (MLP_STAGE_A + MLP_STAGE_B) + 1024;

inline const char* mlp_shape_unsupported(int d, int H, int C, int m) {
  if (H < 64 || H > 512 || H % 64 != 0) return "mlp: hidden width must be a multiple of 64 in [64, 512]";
  if (d % 64 != 0) return "mlp: d must be a multiple of 64";
  if (m % 64 != 0) return "mlp: m must be a multiple of 64";
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

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

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

// One BK-deep step of the 64 x (8 warps x 64) tile: A fragments of the 4 row blocks, B fragments
// of the warp's 8 column blocks, 32 MMAs.  A_KM: the A tile is stored [k][m] (transposed).
template <bool A_KM>
__device__ __forceinline__ void mlp_tile_mma(float (&acc)[4][8][4], uint32_t As, uint32_t Bs, int warp, int lane, int ncols) {
  if (warp * 64 >= ncols) return;
#pragma unroll
  for (int k16 = 0; k16 < MLP_BK / 16; ++k16) {
    uint32_t af[4][4];
#pragma unroll
    for (int mt = 0; mt < 4; ++mt) {
      if (!A_KM) {
        const int row = mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        const int chunk = k16 * 2 + (lane >> 4);
        ldmatrix_x4(af[mt], As + row * 128 + ((chunk ^ (row & 7)) << 4));
      } else {
        const int krow = k16 * 16 + (lane & 7) + (lane >> 4) * 8;
        const int chunk = mt * 2 + ((lane >> 3) & 1);
        ldmatrix_x4_trans(af[mt], As + krow * 128 + ((chunk ^ (krow & 7)) << 4));
      }
    }
#pragma unroll
    for (int np = 0; np < 4; ++np) {
      uint32_t bf[4];
      const int krow = k16 * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
      const int chunk = warp * 8 + np * 2 + (lane >> 4);
      ldmatrix_x4_trans(bf, Bs + krow * MLP_PITCH_B + ((chunk ^ (krow & 7)) << 4));
#pragma unroll
      for (int mt = 0; mt < 4; ++mt) {
        mma_bf16(acc[mt][2 * np], af[mt], bf[0], bf[1]);
        mma_bf16(acc[mt][2 * np + 1], af[mt], bf[2], bf[3]);
      }
    }
  }
}

// ---- data preparation ---------------------------------------------------------------------------
__global__ void to_bf16_kernel(const float* src, __nv_bfloat16* dst, long long count) {
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < count; i += (long long)gridDim.x * blockDim.x)
    dst[i] = __float2bfloat16_rn(src[i]);
}
// bf16 shadow of W1 of pool slot `slot` of every replica
__global__ void shadow_w1_kernel(const float* pool, __nv_bfloat16* W1q, long long n_params, long long dH, int n_slots, int slot, int R) {
  const long long total = dH * R;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long r = i / dH, p = i % dH;
    W1q[((size_t)r * n_slots + slot) * dH + p] = __float2bfloat16_rn(pool[((size_t)r * n_slots + slot) * n_params + p]);
  }
}

// ---- forward + backward down to delta1 -------------------------------------------------------
__global__ void __launch_bounds__(256, 1) mlp_forward_kernel(MlpArgs g) {
  const NumericArgs& a = g.na;
  const MlpScratch& sc = g.sc;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int H = sc.H, C = sc.C, d = sc.d, m = sc.m;
  const int halves = m / MLP_BM;
  const int half = blockIdx.x % halves;
  const int l = (blockIdx.x / halves) % sc.Kmax;
  const int r = blockIdx.x / (halves * sc.Kmax);
  const long long j = g.j;
  const int K = (int)a.K_used[(size_t)r * a.cap + j];
  if (l >= K) return;
  const size_t ent = ((size_t)r * a.cap + j) * a.K_stride + l;
  const uint32_t worker = a.worker[ent], seq = a.seq[ent];
  const int snap = mlp_snap_slot(a, r, j, l);
  const uint32_t rid = a.replica_base + (uint32_t)r;
  const size_t task = (size_t)r * sc.Kmax + l;
  const long long dH = (long long)d * H;
  const float* wsnap = a.pool + ((size_t)r * a.n_slots + snap) * a.n_params;
  const __nv_bfloat16* W1q = sc.W1q + ((size_t)r * sc.n_slots + snap) * dH;

  extern __shared__ __align__(128) unsigned char smem[];
  unsigned long long* rowptr_s = reinterpret_cast<unsigned long long*>(smem);   // [64] source rows (element offsets)
  int* label_s = reinterpret_cast<int*>(smem + 512);                            // [64]
  unsigned char* stages = smem + 1024;
  const uint32_t stages_addr = smem_addr(stages);

  if (tid < MLP_BM) {
    uint32_t idx = draw_index(a.seed, rid, worker, seq, (uint32_t)(half * MLP_BM + tid), a.n);
    if ((uint64_t)idx >= a.n) { atomicExch(a.err, ERR_BAD_INDEX); idx = 0; }
    rowptr_s[tid] = (unsigned long long)idx * (unsigned long long)d;
    label_s[tid] = reinterpret_cast<const int*>(a.y)[idx];
  }
  __syncthreads();

  auto load_stage = [&](int kc) {
    const int st = kc % MLP_STAGES;
    const uint32_t As = stages_addr + st * (MLP_STAGE_A + MLP_STAGE_B);
    const uint32_t Bs = As + MLP_STAGE_A;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int c = tid + 256 * i, row = c >> 3, ch = c & 7;
      cp_async16(As + row * 128 + ((ch ^ (row & 7)) << 4), sc.Xq + rowptr_s[row] + (size_t)kc * MLP_BK + ch * 8);
    }
    const int nch = H / 8;   // 16-byte chunks per k-row
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const int c = tid + 256 * i, krow = c >> 6, ch = c & 63;
      if (ch < nch)
        cp_async16(Bs + krow * MLP_PITCH_B + ((ch ^ (krow & 7)) << 4), W1q + ((size_t)kc * MLP_BK + krow) * H + ch * 8);
    }
  };

  float acc[4][8][4];
#pragma unroll
  for (int mt = 0; mt < 4; ++mt)
#pragma unroll
    for (int nt = 0; nt < 8; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[mt][nt][e] = 0.f;

  const int nk = d / MLP_BK;
  for (int s = 0; s < MLP_STAGES - 1; ++s) { if (s < nk) load_stage(s); cp_async_commit(); }
  for (int kc = 0; kc < nk; ++kc) {
    cp_async_wait<MLP_STAGES - 2>();
    __syncthreads();
    if (kc + MLP_STAGES - 1 < nk) load_stage(kc + MLP_STAGES - 1);
    cp_async_commit();
    const int st = kc % MLP_STAGES;
    const uint32_t As = stages_addr + st * (MLP_STAGE_A + MLP_STAGE_B);
    mlp_tile_mma<false>(acc, As, As + MLP_STAGE_A, warp, lane, H);
  }
  cp_async_wait<0>();
  __syncthreads();

  // ---- epilogue: the stage buffers are free; reuse them ----
  float* W2_s = reinterpret_cast<float*>(stages);                 // [H][16]
  float* zpart_s = W2_s + 512 * 16;                                // [8 warps][64 rows][16]
  float* d2_s = zpart_s + 8 * 64 * 16;                             // [64][16]
  const float* b1 = wsnap + dH;
  const float* W2 = b1 + H;
  const float* b2 = W2 + (size_t)H * C;
  for (int i = tid; i < H * 16; i += 256) {
    const int col = i >> 4, c = i & 15;
    W2_s[i] = c < C ? W2[(size_t)col * C + c] : 0.f;
  }
  const int g8 = lane >> 2, tig = lane & 3;
  const bool wactive = warp * 64 < H;
  // h = relu(A1 + b1); keep in acc; write to the scratch for the head kernel
  if (wactive) {
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const int col = warp * 64 + nt * 8 + 2 * tig;
      const float bb0 = b1[col], bb1 = b1[col + 1];
#pragma unroll
      for (int mt = 0; mt < 4; ++mt) {
#pragma unroll
        for (int rh = 0; rh < 2; ++rh) {
          const int row = mt * 16 + g8 + rh * 8;
          const float h0 = fmaxf(acc[mt][nt][2 * rh] + bb0, 0.f), h1 = fmaxf(acc[mt][nt][2 * rh + 1] + bb1, 0.f);
          acc[mt][nt][2 * rh] = h0; acc[mt][nt][2 * rh + 1] = h1;
          *reinterpret_cast<float2*>(sc.Hact + (task * m + half * MLP_BM + row) * H + col) = make_float2(h0, h1);
        }
      }
    }
  }
  __syncthreads();   // W2_s ready
  // partial logits over this warp's 64 hidden units
#pragma unroll
  for (int mt = 0; mt < 4; ++mt) {
#pragma unroll
    for (int rh = 0; rh < 2; ++rh) {
      const int row = mt * 16 + g8 + rh * 8;
      float zp[16];
#pragma unroll
      for (int c = 0; c < 16; ++c) zp[c] = 0.f;
      if (wactive) {
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int col = warp * 64 + nt * 8 + 2 * tig + e;
            const float hv = acc[mt][nt][2 * rh + e];
            const float4* wr = reinterpret_cast<const float4*>(W2_s + col * 16);
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
              const float4 w = wr[c4];
              zp[4 * c4] = fmaf(hv, w.x, zp[4 * c4]); zp[4 * c4 + 1] = fmaf(hv, w.y, zp[4 * c4 + 1]);
              zp[4 * c4 + 2] = fmaf(hv, w.z, zp[4 * c4 + 2]); zp[4 * c4 + 3] = fmaf(hv, w.w, zp[4 * c4 + 3]);
            }
          }
        }
      }
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        zp[c] += __shfl_xor_sync(0xFFFFFFFFu, zp[c], 1);
        zp[c] += __shfl_xor_sync(0xFFFFFFFFu, zp[c], 2);
      }
      if (tig == 0) {
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4)
          reinterpret_cast<float4*>(zpart_s + (warp * 64 + row) * 16)[c4] = make_float4(zp[4 * c4], zp[4 * c4 + 1], zp[4 * c4 + 2], zp[4 * c4 + 3]);
      }
    }
  }
  __syncthreads();
  // softmax, loss and delta2: one thread per row
  if (tid < MLP_BM) {
    const int row = tid, lab = label_s[row];
    float z[16], zmax = -INFINITY;
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      float s = 0.f;
      for (int w = 0; w < 8; ++w) s += zpart_s[(w * 64 + row) * 16 + c];
      z[c] = c < C ? s + b2[c] : -INFINITY;
      zmax = fmaxf(zmax, z[c]);
    }
    // exponentials without the maximal class (its term is exactly 1): log(1 + s) and
    // p_max - 1 = -s / (1 + s) stay accurate for samples classified with a wide margin
    int cmax = 0;
#pragma unroll
    for (int c = 15; c >= 0; --c) if (c < C && z[c] == zmax) cmax = c;
    float zl = 0.f;
#pragma unroll
    for (int c = 0; c < 16; ++c) if (c == lab) zl = z[c];
    float sexcl = 0.f;
#pragma unroll
    for (int c = 0; c < 16; ++c) { z[c] = (c < C && c != cmax) ? expf(z[c] - zmax) : 0.f; sexcl += z[c]; }
    const float ssum = 1.f + sexcl;
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      float dl = 0.f;
      if (c < C) {
        if (c == cmax) dl = c == lab ? -sexcl / ssum : 1.f / ssum;
        else dl = z[c] / ssum - (c == lab ? 1.f : 0.f);
      }
      d2_s[row * 16 + c] = dl;
      sc.D2[(task * m + half * MLP_BM + row) * 16 + c] = dl;
    }
    float rowloss = log1pf(sexcl) + (zmax - zl);
    rowloss += __shfl_xor_sync(0xFFFFFFFFu, rowloss, 16);
    rowloss += __shfl_xor_sync(0xFFFFFFFFu, rowloss, 8);
    rowloss += __shfl_xor_sync(0xFFFFFFFFu, rowloss, 4);
    rowloss += __shfl_xor_sync(0xFFFFFFFFu, rowloss, 2);
    rowloss += __shfl_xor_sync(0xFFFFFFFFu, rowloss, 1);
    if (lane == 0) d2_s[MLP_BM * 16 + warp] = rowloss;     // rows 0..31 and rows 32..63
  }
  __syncthreads();
  if (tid == 0) sc.loss_part[task * halves + half] = d2_s[MLP_BM * 16] + d2_s[MLP_BM * 16 + 1];
  // delta1 = (delta2 W2^T) . [h > 0]; db1 partial; bf16 store
  if (wactive) {
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      float colsum[2] = {0.f, 0.f};
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int col = warp * 64 + nt * 8 + 2 * tig + e;
        float w2[16];
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) {
          const float4 w = reinterpret_cast<const float4*>(W2_s + col * 16)[c4];
          w2[4 * c4] = w.x; w2[4 * c4 + 1] = w.y; w2[4 * c4 + 2] = w.z; w2[4 * c4 + 3] = w.w;
        }
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) {
#pragma unroll
          for (int rh = 0; rh < 2; ++rh) {
            const int row = mt * 16 + g8 + rh * 8;
            float dv = 0.f;
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
              const float4 dl = reinterpret_cast<const float4*>(d2_s + row * 16)[c4];
              dv = fmaf(dl.x, w2[4 * c4], dv); dv = fmaf(dl.y, w2[4 * c4 + 1], dv);
              dv = fmaf(dl.z, w2[4 * c4 + 2], dv); dv = fmaf(dl.w, w2[4 * c4 + 3], dv);
            }
            dv = acc[mt][nt][2 * rh + e] > 0.f ? dv : 0.f;
            acc[mt][nt][2 * rh + e] = dv;
            colsum[e] += dv;
          }
        }
      }
      const int col = warp * 64 + nt * 8 + 2 * tig;
#pragma unroll
      for (int mt = 0; mt < 4; ++mt) {
#pragma unroll
        for (int rh = 0; rh < 2; ++rh) {
          const int row = mt * 16 + g8 + rh * 8;
          *reinterpret_cast<__nv_bfloat162*>(sc.D1q + (task * m + half * MLP_BM + row) * H + col) =
              __floats2bfloat162_rn(acc[mt][nt][2 * rh], acc[mt][nt][2 * rh + 1]);
        }
      }
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        colsum[e] += __shfl_xor_sync(0xFFFFFFFFu, colsum[e], 4);
        colsum[e] += __shfl_xor_sync(0xFFFFFFFFu, colsum[e], 8);
        colsum[e] += __shfl_xor_sync(0xFFFFFFFFu, colsum[e], 16);
      }
      if (g8 == 0) {
        sc.db1_part[(task * halves + half) * H + col] = colsum[0];
        sc.db1_part[(task * halves + half) * H + col + 1] = colsum[1];
      }
    }
  }
}

// ---- dW2 = h^T delta2, db2 (per contributor) --------------------------------------------------
__global__ void __launch_bounds__(512) mlp_head_kernel(MlpArgs g) {
  const NumericArgs& a = g.na;
  const MlpScratch& sc = g.sc;
  const int l = blockIdx.x % sc.Kmax, r = blockIdx.x / sc.Kmax;
  const int K = (int)a.K_used[(size_t)r * a.cap + g.j];
  if (l >= K) return;
  const int H = sc.H, C = sc.C, m = sc.m, tid = threadIdx.x;
  const size_t task = (size_t)r * sc.Kmax + l;
  extern __shared__ __align__(128) unsigned char smem[];
  float* d2_s = reinterpret_cast<float*>(smem);   // [m][16]
  for (int i = tid; i < m * 16; i += blockDim.x) d2_s[i] = sc.D2[task * m * 16 + i];
  __syncthreads();
  if (tid < H) {
    float accw[16];
#pragma unroll
    for (int c = 0; c < 16; ++c) accw[c] = 0.f;
    for (int row = 0; row < m; ++row) {
      const float hv = sc.Hact[(task * m + row) * H + tid];
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4) {
        const float4 dl = reinterpret_cast<const float4*>(d2_s + row * 16)[c4];
        accw[4 * c4] = fmaf(hv, dl.x, accw[4 * c4]); accw[4 * c4 + 1] = fmaf(hv, dl.y, accw[4 * c4 + 1]);
        accw[4 * c4 + 2] = fmaf(hv, dl.z, accw[4 * c4 + 2]); accw[4 * c4 + 3] = fmaf(hv, dl.w, accw[4 * c4 + 3]);
      }
    }
    for (int c = 0; c < C; ++c) sc.dW2_part[task * H * C + (size_t)tid * C + c] = accw[c];
  }
  if (tid < 16) {
    float s = 0.f;
    for (int row = 0; row < m; ++row) s += d2_s[row * 16 + tid];
    sc.db2_part[task * 16 + tid] = s;
  }
}

// ---- dW1 = X^T delta1 over all contributors of the update, fused with the W1 update ------------
__global__ void __launch_bounds__(256, 1) mlp_dw1_update_kernel(MlpArgs g) {
  const NumericArgs& a = g.na;
  const MlpScratch& sc = g.sc;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int H = sc.H, d = sc.d, m = sc.m;
  const int slabs = d / MLP_BM;
  const int slab = blockIdx.x % slabs, r = blockIdx.x / slabs;
  const long long j = g.j;
  const int K = (int)a.K_used[(size_t)r * a.cap + j];
  const uint32_t rid = a.replica_base + (uint32_t)r;
  const long long dH = (long long)d * H;
  const int blocks_per_task = m / MLP_BK;
  const int nk = K * blocks_per_task;

  extern __shared__ __align__(128) unsigned char smem[];
  unsigned long long* rowptr_s = reinterpret_cast<unsigned long long*>(smem);   // [3 stages][64]... one set per stage
  unsigned char* stages = smem + 2048;
  const uint32_t stages_addr = smem_addr(stages);

  auto draw_rows = [&](int kc) {   // sample rows of reduction block kc -> rowptr_s[kc % 3]
    if (tid < MLP_BK) {
      const int l = kc / blocks_per_task, blk = kc % blocks_per_task;
      const size_t ent = ((size_t)r * a.cap + j) * a.K_stride + l;
      uint32_t idx = draw_index(a.seed, rid, a.worker[ent], a.seq[ent], (uint32_t)(blk * MLP_BK + tid), a.n);
      if ((uint64_t)idx >= a.n) { atomicExch(a.err, ERR_BAD_INDEX); idx = 0; }
      rowptr_s[(kc % MLP_STAGES) * 64 + tid] = (unsigned long long)idx * (unsigned long long)d;
    }
  };
  auto load_stage = [&](int kc) {
    const int st = kc % MLP_STAGES;
    const int l = kc / blocks_per_task, blk = kc % blocks_per_task;
    const uint32_t As = stages_addr + st * (MLP_STAGE_A + MLP_STAGE_B);
    const uint32_t Bs = As + MLP_STAGE_A;
    // A tile stored [k = sample][m = 64 columns of this slab]
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int c = tid + 256 * i, krow = c >> 3, ch = c & 7;
      cp_async16(As + krow * 128 + ((ch ^ (krow & 7)) << 4), sc.Xq + rowptr_s[st * 64 + krow] + (size_t)slab * MLP_BM + ch * 8);
    }
    const __nv_bfloat16* D1 = sc.D1q + (((size_t)r * sc.Kmax + l) * m + (size_t)blk * MLP_BK) * H;
    const int nch = H / 8;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const int c = tid + 256 * i, krow = c >> 6, ch = c & 63;
      if (ch < nch) cp_async16(Bs + krow * MLP_PITCH_B + ((ch ^ (krow & 7)) << 4), D1 + (size_t)krow * H + ch * 8);
    }
  };

  float acc[4][8][4];
#pragma unroll
  for (int mt = 0; mt < 4; ++mt)
#pragma unroll
    for (int nt = 0; nt < 8; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[mt][nt][e] = 0.f;

  // the row indices of a block are drawn one iteration before its loads are issued
  for (int s = 0; s < MLP_STAGES - 1; ++s) if (s < nk) draw_rows(s);
  __syncthreads();
  for (int s = 0; s < MLP_STAGES - 1; ++s) { if (s < nk) load_stage(s); cp_async_commit(); }
  if (MLP_STAGES - 1 < nk) draw_rows(MLP_STAGES - 1);
  for (int kc = 0; kc < nk; ++kc) {
    cp_async_wait<MLP_STAGES - 2>();
    __syncthreads();
    if (kc + MLP_STAGES - 1 < nk) load_stage(kc + MLP_STAGES - 1);
    cp_async_commit();
    const int st = kc % MLP_STAGES;
    const uint32_t As = stages_addr + st * (MLP_STAGE_A + MLP_STAGE_B);
    mlp_tile_mma<true>(acc, As, As + MLP_STAGE_A, warp, lane, H);
    // rows for block kc + STAGES go to slot kc % STAGES of rowptr_s: its last readers were the loads of
    // block kc (issued two iterations ago); the next reader, load_stage(kc + STAGES), runs after the
    // barrier at the top of the next iteration
    if (kc + MLP_STAGES < nk) draw_rows(kc + MLP_STAGES);
  }
  cp_async_wait<0>();

  // ---- epilogue: W1 <- W1 - (eta/(K m)) dW1 for this slab, new version + bf16 shadow ----
  if (warp * 64 >= H) return;
  const int cur = mlp_cur_slot(a, r, j), fresh = mlp_fresh_slot(a, r, j);
  const float scale = (float)((double)a.eta / ((double)K * (double)m));
  const float* wc = a.pool + ((size_t)r * a.n_slots + cur) * a.n_params;
  float* wn = a.pool + ((size_t)r * a.n_slots + fresh) * a.n_params;
  __nv_bfloat16* wq = sc.W1q + ((size_t)r * sc.n_slots + fresh) * dH;
  const int g8 = lane >> 2, tig = lane & 3;
#pragma unroll
  for (int mt = 0; mt < 4; ++mt) {
#pragma unroll
    for (int rh = 0; rh < 2; ++rh) {
      const size_t row = (size_t)slab * MLP_BM + mt * 16 + g8 + rh * 8;
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        const int col = warp * 64 + nt * 8 + 2 * tig;
        const float2 w = *reinterpret_cast<const float2*>(wc + row * H + col);
        const float n0 = fmaf(-scale, acc[mt][nt][2 * rh], w.x), n1 = fmaf(-scale, acc[mt][nt][2 * rh + 1], w.y);
        *reinterpret_cast<float2*>(wn + row * H + col) = make_float2(n0, n1);
        *reinterpret_cast<__nv_bfloat162*>(wq + row * H + col) = __floats2bfloat162_rn(n0, n1);
      }
    }
  }
}

// ---- b1, W2, b2 update and the loss record -------------------------------------------------------
__global__ void __launch_bounds__(256) mlp_small_update_kernel(MlpArgs g) {
  const NumericArgs& a = g.na;
  const MlpScratch& sc = g.sc;
  const int r = blockIdx.x, tid = threadIdx.x;
  const long long j = g.j;
  const int K = (int)a.K_used[(size_t)r * a.cap + j];
  const int H = sc.H, C = sc.C, m = sc.m, halves = m / MLP_BM;
  const long long dH = (long long)sc.d * H;
  const int cur = mlp_cur_slot(a, r, j), fresh = mlp_fresh_slot(a, r, j);
  const float scale = (float)((double)a.eta / ((double)K * (double)m));
  const float* wc = a.pool + ((size_t)r * a.n_slots + cur) * a.n_params + dH;
  float* wn = a.pool + ((size_t)r * a.n_slots + fresh) * a.n_params + dH;
  const int tail = H + H * C + C;
  for (int p = tid; p < tail; p += blockDim.x) {
    float gsum = 0.f;
    for (int l = 0; l < K; ++l) {
      const size_t task = (size_t)r * sc.Kmax + l;
      if (p < H) { for (int hf = 0; hf < halves; ++hf) gsum += sc.db1_part[(task * halves + hf) * H + p]; }
      else if (p < H + H * C) gsum += sc.dW2_part[task * H * C + (p - H)];
      else gsum += sc.db2_part[task * 16 + (p - H - H * C)];
    }
    wn[p] = fmaf(-scale, gsum, wc[p]);
  }
  if (tid == 0) {
    float ls = 0.f;
    for (int l = 0; l < K; ++l)
      for (int hf = 0; hf < halves; ++hf) ls += sc.loss_part[((size_t)r * sc.Kmax + l) * halves + hf];
    a.loss[(size_t)r * a.cap + j] = ls / ((float)K * (float)m);
    a.dist2[(size_t)r * a.cap + j] = 0.f;
  }
}

// ---- host side -----------------------------------------------------------------------------------
inline void mlp_scratch_free(MlpScratch& s) {
  cudaFree(s.Xq); cudaFree(s.W1q); cudaFree(s.D1q); cudaFree(s.Hact); cudaFree(s.D2);
  cudaFree(s.db1_part); cudaFree(s.dW2_part); cudaFree(s.db2_part); cudaFree(s.loss_part);
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
  MLP_ALLOC(s.W1q, (size_t)R * n_slots * d * H)
  MLP_ALLOC(s.D1q, tasks * m * H)
  MLP_ALLOC(s.Hact, tasks * m * H)
  MLP_ALLOC(s.D2, tasks * m * 16)
  MLP_ALLOC(s.db1_part, tasks * (m / MLP_BM) * H)
  MLP_ALLOC(s.dW2_part, tasks * H * C)
  MLP_ALLOC(s.db2_part, tasks * 16)
  MLP_ALLOC(s.loss_part, tasks * (m / MLP_BM))
#undef MLP_ALLOC
  to_bf16_kernel<<<1184, 256, 0, stream>>>(X, s.Xq, (long long)n * d);
  return cudaGetLastError();
}

// after the initial parameters went into slot 0 of every replica
inline cudaError_t mlp_after_set_params(MlpScratch& s, const float* pool, long long n_params, cudaStream_t stream) {
  shadow_w1_kernel<<<1184, 256, 0, stream>>>(pool, s.W1q, n_params, (long long)s.d * s.H, s.n_slots, 0, s.R);
  return cudaGetLastError();
}

inline cudaError_t run_mlp(NumericArgs& a, MlpScratch& s, int P, cudaStream_t stream, const char** why) {
  *why = nullptr;
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(mlp_forward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, MLP_SMEM)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(mlp_dw1_update_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, MLP_SMEM + 1024)) != cudaSuccess) return e;
  MlpArgs g{};
  g.na = a; g.sc = s; g.H = s.H; g.P = P;
  const int halves = s.m / MLP_BM;
  for (long long u = 0; u < a.iters; ++u) {
    g.j = a.j0 + u;
    mlp_forward_kernel<<<a.R * s.Kmax * halves, 256, MLP_SMEM, stream>>>(g);
    mlp_head_kernel<<<a.R * s.Kmax, 512, (size_t)s.m * 16 * 4, stream>>>(g);
    mlp_dw1_update_kernel<<<a.R * (s.d / MLP_BM), 256, MLP_SMEM + 1024, stream>>>(g);
    mlp_small_update_kernel<<<a.R, 256, 0, stream>>>(g);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace ssim
