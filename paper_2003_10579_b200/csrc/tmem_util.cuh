// Tensor memory used as a register-file extension by the softmax-regression kernel: allocation, 32x32b loads and
// stores of a thread's own lane (thread t of a warp reads lane 32 (warp % 4) + t), the fences that order them against
// thread synchronisation, and the warp transposition reduce of the partial logits.  No MMA is issued on this path.
#pragma once
#include "softmax_kernel.cuh"

namespace ssim {

constexpr int SMT_CP = 10;            // classes the layout is built for
constexpr int SMT_WC = 2 * SMT_CP;    // tensor-memory columns per feature pair
constexpr int SMT_DSTR = 12;          // floats per row of D in shared memory (10 classes, padded to whole 16-byte loads)
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

}  // namespace ssim
