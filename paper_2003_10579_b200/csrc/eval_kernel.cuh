// Full-data empirical risk F(w) = (1/N) sum_n f(w, xi_n) (Eq. 1) of every replica's current
// parameters, for the linear models: the quantity behind the paper's error-versus-wall-clock
// curves and behind the rule that raises K in Algorithm 1.
//
// The logits of all replicas are one dense product Z = X W^T (n x d times d x (R*C)), so the data
// set is read once per 128 (replica, class) columns instead of once per replica.  fp32 FMAs
// (a loss at its noise floor needs the full fp32 mantissa of the logits, so no tf32 / bf16 tensor
// path), shared-memory tiling: block = 128 rows x 128 columns, 256 threads x (8 x 8).
// The per-sample losses are summed in fp64 in a fixed order (warp tree, then row blocks in
// sequence in a second kernel): the result does not vary from run to run.
#pragma once
#include "linear_kernel.cuh"

namespace ssim {

constexpr int EV_BM = 128, EV_BN = 128, EV_BK = 16;
constexpr int EV_LDA = EV_BM + 4, EV_LDB = EV_BN + 4;   // padded leading dimensions of the operand tiles [k][row], [k][column]
constexpr int EV_OPERAND_FLOATS = 2 * EV_BK * (EV_LDA + EV_LDB);   // A and B, two buffers each
constexpr int EV_CG = EV_BN / 64;                       // groups of four columns per thread
constexpr int EV_Z_FLOATS = EV_BM * (EV_BN + 1);
constexpr size_t EV_SMEM_BYTES = sizeof(float) * (EV_Z_FLOATS > EV_OPERAND_FLOATS ? EV_Z_FLOATS : EV_OPERAND_FLOATS);

struct EvalArgs {
  const float* X;
  const void* y;
  long long n;
  int d, C, model, R;
  int RB;                       // replicas per column block: floor(EV_BN / C)
  const float* w_state;         // [R][n_params] or null
  const float* pool;            // [R][n_slots][slot_stride] or null
  const uint8_t* cur_slot;      // [R] (pool)
  int n_slots;
  long long n_params, slot_stride;
  double* partial;              // [row blocks][R]
  int row_blocks;
  float* out;                   // [R]
};

__device__ __forceinline__ const float* eval_params(const EvalArgs& a, int r) {
  if (a.pool) return a.pool + ((size_t)r * a.n_slots + a.cur_slot[r]) * a.slot_stride;
  return a.w_state + (size_t)r * a.n_params;
}

// Block = 128 rows x 128 (replica, class) columns, 256 threads x (8 x 8) accumulators, two blocks per SM.  (At 128 B/clk
// of shared-memory return bandwidth against 128 FMA/clk an 8 x 8 register tile needs one byte per FMA, so the two pipes
// are about equally loaded; 8 x 16 tiles at one block per SM need 0.75 but were slower: 41 against 44 TFLOP/s, the
// second block's warps hide more than the saved loads buy.)  Both operands are stored with k
// contiguous (rows of X, rows of W), so a tile is read as float4s along k into registers and written transposed into
// shared memory ([k][row], [k][column]); the next tile's global loads are in flight while the current one is multiplied
// (register prefetch, two shared-memory buffers, one block barrier per k-tile).  A thread's eight rows and eight columns
// are groups of four, 64 apart, so that its float4 reads of a k-row are conflict-free.  After the k loop the logits go
// to shared memory (over the operand buffers) and the per-sample losses are formed and summed as before.
__global__ void __launch_bounds__(256, 2) eval_loss_kernel(EvalArgs a) {
  extern __shared__ __align__(16) float ev_smem[];
  __shared__ double sums_s[EV_BN][4];
  float* As = ev_smem;                                   // [2][EV_BK][EV_LDA]
  float* Bs = ev_smem + 2 * EV_BK * EV_LDA;              // [2][EV_BK][EV_LDB]
  float* Zs = ev_smem;                                   // [EV_BM][EV_BN + 1], after the k loop
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const long long row0 = (long long)blockIdx.x * EV_BM;
  const int rep0 = blockIdx.y * a.RB;
  const int d = a.d, C = a.C;

  // global -> register mapping of a tile: thread takes k-quad kq of rows lr, lr + 64 and columns lr + 64 i, i < EV_CG
  const int lr = tid >> 2, kq = tid & 3;
  const float* aptr[2];
  const float* bptr[EV_CG];
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const long long row = row0 + lr + 64 * i;
    aptr[i] = row < a.n ? a.X + (size_t)row * d : nullptr;
  }
#pragma unroll
  for (int i = 0; i < EV_CG; ++i) {
    const int col = lr + 64 * i;                         // column of the block = (replica rep0 + col / C, class col % C)
    const int rep = rep0 + col / C;
    bptr[i] = (col < a.RB * C && rep < a.R) ? eval_params(a, rep) + (size_t)(col % C) * d : nullptr;
  }
  auto fetch = [&](int k0, float4 (&av)[2], float4 (&bv)[EV_CG]) {
    const bool in = k0 + 4 * kq < d;                     // d is a multiple of 4: a quad is inside or outside
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      av[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (in && aptr[i]) av[i] = *reinterpret_cast<const float4*>(aptr[i] + k0 + 4 * kq);
    }
#pragma unroll
    for (int i = 0; i < EV_CG; ++i) {
      bv[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (in && bptr[i]) bv[i] = *reinterpret_cast<const float4*>(bptr[i] + k0 + 4 * kq);
    }
  };
  auto stash = [&](int buf, const float4 (&av)[2], const float4 (&bv)[EV_CG]) {
    float* A_ = As + buf * EV_BK * EV_LDA;
    float* B_ = Bs + buf * EV_BK * EV_LDB;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int rc = lr + 64 * i;
      A_[(4 * kq) * EV_LDA + rc] = av[i].x; A_[(4 * kq + 1) * EV_LDA + rc] = av[i].y;
      A_[(4 * kq + 2) * EV_LDA + rc] = av[i].z; A_[(4 * kq + 3) * EV_LDA + rc] = av[i].w;
    }
#pragma unroll
    for (int i = 0; i < EV_CG; ++i) {
      const int rc = lr + 64 * i;
      B_[(4 * kq) * EV_LDB + rc] = bv[i].x; B_[(4 * kq + 1) * EV_LDB + rc] = bv[i].y;
      B_[(4 * kq + 2) * EV_LDB + rc] = bv[i].z; B_[(4 * kq + 3) * EV_LDB + rc] = bv[i].w;
    }
  };

  float acc[8][4 * EV_CG];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int jn = 0; jn < 4 * EV_CG; ++jn) acc[i][jn] = 0.f;

  float4 av[2], bv[EV_CG];
  fetch(0, av, bv);
  stash(0, av, bv);
  __syncthreads();
  const int n_tiles = (d + EV_BK - 1) / EV_BK;
  for (int kt = 0; kt < n_tiles; ++kt) {
    const int buf = kt & 1;
    if (kt + 1 < n_tiles) fetch((kt + 1) * EV_BK, av, bv);
    const float* A_ = As + buf * EV_BK * EV_LDA;
    const float* B_ = Bs + buf * EV_BK * EV_LDB;
#pragma unroll
    for (int k = 0; k < EV_BK; ++k) {
      const float4 a0 = *reinterpret_cast<const float4*>(A_ + k * EV_LDA + ty * 4);
      const float4 a1 = *reinterpret_cast<const float4*>(A_ + k * EV_LDA + 64 + ty * 4);
      const float ar[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
#pragma unroll
      for (int g = 0; g < EV_CG; ++g) {
        const float4 b = *reinterpret_cast<const float4*>(B_ + k * EV_LDB + 64 * g + tx * 4);
        const float br[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
          for (int jn = 0; jn < 4; ++jn) acc[i][4 * g + jn] = fmaf(ar[i], br[jn], acc[i][4 * g + jn]);
      }
    }
    if (kt + 1 < n_tiles) stash(buf ^ 1, av, bv);
    __syncthreads();
  }
  // logits to shared memory (the operand buffers are free after the last barrier)
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int jn = 0; jn < 4 * EV_CG; ++jn)
      Zs[((i >> 2) * 64 + ty * 4 + (i & 3)) * (EV_BN + 1) + (jn >> 2) * 64 + tx * 4 + (jn & 3)] = acc[i][jn];
  __syncthreads();

  // per-sample losses: pair p = (replica rr, row): consecutive threads take consecutive rows
  const int lane = tid & 31;
  for (int p = tid; p < a.RB * EV_BM; p += 256) {
    const int rr = p / EV_BM, row = p % EV_BM;
    double f = 0.0;
    if (row0 + row < a.n && rep0 + rr < a.R) {
      const float* z = &Zs[row * (EV_BN + 1) + rr * C];
      if (a.model == M_LSQ) {
        const float res = z[0] - reinterpret_cast<const float*>(a.y)[row0 + row];
        f = 0.5 * (double)res * (double)res;
      } else if (a.model == M_LOGISTIC) {
        const float b = (float)reinterpret_cast<const int*>(a.y)[row0 + row];
        f = (double)(fmaxf(z[0], 0.f) + log1pf(expf(-fabsf(z[0]))) - b * z[0]);
      } else {
        const int lab = reinterpret_cast<const int*>(a.y)[row0 + row];
        float zmax = z[0];
        int cmax = 0;
        for (int c = 1; c < C; ++c) if (z[c] > zmax) { zmax = z[c]; cmax = c; }
        float sexcl = 0.f;
        for (int c = 0; c < C; ++c) if (c != cmax) sexcl += expf(z[c] - zmax);
        f = (double)(log1pf(sexcl) + (zmax - z[lab]));
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) f += __shfl_xor_sync(0xFFFFFFFFu, f, off);
    if (lane == 0) sums_s[rr][(row >> 5)] = f;
  }
  __syncthreads();
  if (tid < a.RB && rep0 + tid < a.R)
    a.partial[(size_t)blockIdx.x * a.R + rep0 + tid] = sums_s[tid][0] + sums_s[tid][1] + sums_s[tid][2] + sums_s[tid][3];
}

__global__ void eval_loss_finish_kernel(EvalArgs a) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= a.R) return;
  double s = 0.0;
  for (int b = 0; b < a.row_blocks; ++b) s += a.partial[(size_t)b * a.R + r];
  a.out[r] = (float)(s / (double)a.n);
}

// Error against simulated wall clock on a common time grid: at grid time g a replica contributes the
// loss recorded at its last update with t <= g (binary search in its clock trace); the mean is over the
// replicas that have completed an update by then.  One block per grid point, fp64 tree sum (fixed order).
__global__ void __launch_bounds__(256) error_curve_kernel(const double* t, const float* err, long long cap, long long J, int R,
                                                          const double* grid, float* mean, int* count) {
  __shared__ double sum_s[256];
  __shared__ int cnt_s[256];
  const double g = grid[blockIdx.x];
  double s = 0.0;
  int c = 0;
  for (int r = threadIdx.x; r < R; r += 256) {
    const double* tr = t + (size_t)r * cap;
    long long lo = 0, hi = J;                 // first index with t > g
    while (lo < hi) { const long long mid = (lo + hi) >> 1; if (tr[mid] <= g) lo = mid + 1; else hi = mid; }
    if (lo > 0) { s += (double)err[(size_t)r * cap + lo - 1]; ++c; }
  }
  sum_s[threadIdx.x] = s; cnt_s[threadIdx.x] = c;
  __syncthreads();
  for (int off = 128; off > 0; off >>= 1) {
    if ((int)threadIdx.x < off) { sum_s[threadIdx.x] += sum_s[threadIdx.x + off]; cnt_s[threadIdx.x] += cnt_s[threadIdx.x + off]; }
    __syncthreads();
  }
  if (threadIdx.x == 0) { count[blockIdx.x] = cnt_s[0]; mean[blockIdx.x] = cnt_s[0] ? (float)(sum_s[0] / cnt_s[0]) : 0.f; }
}

}  // namespace ssim
