// Full-data empirical risk F(w) = (1/N) sum_n f(w, xi_n) (Eq. 1) of every replica's current
// parameters, for the linear models: the quantity behind the paper's error-versus-wall-clock
// curves and behind the rule that raises K in Algorithm 1.
//
// The logits of all replicas are one dense product Z = X W^T (n x d times d x (R*C)), so the data
// set is read once per 64 (replica, class) columns instead of once per replica.  fp32 FMAs
// (a loss at its noise floor needs the full fp32 mantissa of the logits, so no tf32 / bf16 tensor
// path), classic shared-memory tiling: block = 128 rows x 64 columns, 256 threads x (8 x 4).
// The per-sample losses are summed in fp64 in a fixed order (warp tree, then row blocks in
// sequence in a second kernel): the result does not vary from run to run.
#pragma once
#include "linear_kernel.cuh"

namespace ssim {

constexpr int EV_BM = 128, EV_BN = 64, EV_BK = 16;

struct EvalArgs {
  const float* X;
  const void* y;
  long long n;
  int d, C, model, R;
  int RB;                       // replicas per column block: floor(64 / C)
  const float* w_state;         // [R][n_params] or null
  const float* pool;            // [R][n_slots][slot_stride] or null
  const uint8_t* cur_slot;      // [R] (pool)
  int n_slots;
  long long n_params, slot_stride;
  double* partial;              // [row_blocks][R]
  int row_blocks;
  float* out;                   // [R]
};

__device__ __forceinline__ const float* eval_params(const EvalArgs& a, int r) {
  if (a.pool) return a.pool + ((size_t)r * a.n_slots + a.cur_slot[r]) * a.slot_stride;
  return a.w_state + (size_t)r * a.n_params;
}

__global__ void __launch_bounds__(256) eval_loss_kernel(EvalArgs a) {
  __shared__ float As[EV_BK][EV_BM + 4];
  __shared__ float Bs[EV_BK][EV_BN + 4];
  __shared__ float Zs[EV_BM][EV_BN + 1];
  __shared__ double sums_s[EV_BN][4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const long long row0 = (long long)blockIdx.x * EV_BM;
  const int rep0 = blockIdx.y * a.RB;
  const int d = a.d, C = a.C;

  // B operand: column c of the block = (replica rep0 + c / C, class c % C)
  const int bcol = tid >> 2, bkq = tid & 3;
  const int brep = rep0 + bcol / C, bcls = bcol % C;
  const bool bvalid = bcol < a.RB * C && brep < a.R;
  const float* bptr = bvalid ? eval_params(a, brep) + (size_t)bcls * d : nullptr;

  float acc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int jn = 0; jn < 4; ++jn) acc[i][jn] = 0.f;

  for (int k0 = 0; k0 < d; k0 += EV_BK) {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int row = (tid >> 2) + 64 * i, kq = tid & 3;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (row0 + row < a.n && k0 + 4 * kq < d) v = *reinterpret_cast<const float4*>(a.X + (size_t)(row0 + row) * d + k0 + 4 * kq);
      As[4 * kq][row] = v.x; As[4 * kq + 1][row] = v.y; As[4 * kq + 2][row] = v.z; As[4 * kq + 3][row] = v.w;
    }
    {
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (bvalid && k0 + 4 * bkq < d) v = *reinterpret_cast<const float4*>(bptr + k0 + 4 * bkq);
      Bs[4 * bkq][bcol] = v.x; Bs[4 * bkq + 1][bcol] = v.y; Bs[4 * bkq + 2][bcol] = v.z; Bs[4 * bkq + 3][bcol] = v.w;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < EV_BK; ++k) {
      float av[8], bv[4];
      const float4 a0 = *reinterpret_cast<const float4*>(&As[k][ty * 8]);
      const float4 a1 = *reinterpret_cast<const float4*>(&As[k][ty * 8 + 4]);
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
      av[0] = a0.x; av[1] = a0.y; av[2] = a0.z; av[3] = a0.w; av[4] = a1.x; av[5] = a1.y; av[6] = a1.z; av[7] = a1.w;
      bv[0] = b0.x; bv[1] = b0.y; bv[2] = b0.z; bv[3] = b0.w;
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int jn = 0; jn < 4; ++jn) acc[i][jn] = fmaf(av[i], bv[jn], acc[i][jn]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int jn = 0; jn < 4; ++jn) Zs[ty * 8 + i][tx * 4 + jn] = acc[i][jn];
  __syncthreads();

  // per-sample losses: pair p = (replica rr, row): consecutive threads take consecutive rows
  const int lane = tid & 31;
  for (int p = tid; p < a.RB * EV_BM; p += 256) {
    const int rr = p / EV_BM, row = p % EV_BM;
    double f = 0.0;
    if (row0 + row < a.n && rep0 + rr < a.R) {
      const float* z = &Zs[row][rr * C];
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
