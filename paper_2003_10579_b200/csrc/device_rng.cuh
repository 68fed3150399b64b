// Counter-based random stream of the simulation, device side.
//
// Philox4x32 with 10 rounds (Salmon et al., SC'11), key = the 64-bit seed, counter =
// ((tag << 24) | chunk, task sequence number, worker, global replica id).  tag 0 / chunk 0 gives
// the delay of a task, tag 1 / chunk c gives minibatch draws 4c .. 4c+3 of that task.
//
// A third law, Pareto with shape 2 (the heavy-tailed case of the paper's runtime simulations), is
// X = x_m / sqrt(u) with the same u.
// The delay X = shift + E / mu uses E = -ln(u) evaluated by a fixed sequence of integer
// operations and round-to-nearest fp64 operations (explicit intrinsics, so that the compiler
// neither contracts nor reorders them): the same inputs give the same bits on any IEEE machine,
// which is what makes the simulated arrival order reproducible elsewhere.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace ssim {

struct U4 { uint32_t x, y, z, w; };

__device__ __forceinline__ U4 philox4x32_10(uint32_t k0, uint32_t k1, uint32_t c0, uint32_t c1,
                                            uint32_t c2, uint32_t c3) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  return U4{c0, c1, c2, c3};
}

__device__ __forceinline__ U4 stream_block(uint64_t seed, uint32_t tag, uint32_t chunk,
                                           uint32_t replica, uint32_t worker, uint32_t seq) {
  return philox4x32_10((uint32_t)seed, (uint32_t)(seed >> 32), (tag << 24) | chunk, seq, worker,
                       replica);
}

// E = -ln(u), u = (2k+1) / 2^53, k = top 52 bits of (x0:x1).
//   2k+1 = f 2^b with f in (sqrt(1/2), sqrt(2)];  ln f = 2 atanh(s), s = (f-1)/(f+1);
//   atanh(s)/s = sum_{i<12} s^(2i)/(2i+1) by Horner with fused multiply-adds;
//   E = (53 - b) ln2 - ln f with one fused multiply-add.
__device__ __forceinline__ double neg_log_uniform(uint32_t x0, uint32_t x1) {
  const unsigned long long k = ((unsigned long long)x0 << 20) | ((unsigned long long)x1 >> 12);
  const unsigned long long n = 2ull * k + 1ull;
  int b = 63 - __clzll((long long)n);
  unsigned long long fb = 0x3FF0000000000000ull | ((n << (52 - b)) & 0x000FFFFFFFFFFFFFull);
  if (fb > 0x3FF6A09E667F3BCDull) { fb -= 0x0010000000000000ull; b += 1; }
  const double f = __longlong_as_double((long long)fb);
  const double s = __ddiv_rn(__dsub_rn(f, 1.0), __dadd_rn(f, 1.0));
  const double z = __dmul_rn(s, s);
  double p = 1.0 / 23.0;
  p = __fma_rn(p, z, 1.0 / 21.0);
  p = __fma_rn(p, z, 1.0 / 19.0);
  p = __fma_rn(p, z, 1.0 / 17.0);
  p = __fma_rn(p, z, 1.0 / 15.0);
  p = __fma_rn(p, z, 1.0 / 13.0);
  p = __fma_rn(p, z, 1.0 / 11.0);
  p = __fma_rn(p, z, 1.0 / 9.0);
  p = __fma_rn(p, z, 1.0 / 7.0);
  p = __fma_rn(p, z, 1.0 / 5.0);
  p = __fma_rn(p, z, 1.0 / 3.0);
  p = __fma_rn(p, z, 1.0);
  const double lnf = __dmul_rn(__dmul_rn(2.0, s), p);
  return __fma_rn((double)(53 - b), __longlong_as_double(0x3FE62E42FEFA39EFll), -lnf);
}

// kind: 0 = Exp(mu), 1 = shift + Exp(mu), 2 = Pareto of shape 2 and scale `shift`
struct DelayLaw { int kind; double mu; double shift; };

__device__ __forceinline__ double draw_delay(const DelayLaw& law, uint64_t seed, uint32_t replica,
                                             uint32_t worker, uint32_t seq) {
  const U4 x = stream_block(seed, 0u, 0u, replica, worker, seq);
  if (law.kind == 2) {   // Pareto(2, x_m): X = x_m / sqrt(u), u = (2k+1)/2^53 exact; sqrt and divide are IEEE
    const unsigned long long k = ((unsigned long long)x.x << 20) | ((unsigned long long)x.y >> 12);
    const double u = __dmul_rn((double)(2ull * k + 1ull), 1.1102230246251565e-16 /* 2^-53 */);
    return __ddiv_rn(law.shift, __dsqrt_rn(u));
  }
  const double e = neg_log_uniform(x.x, x.y);
  return __dadd_rn(law.kind == 1 ? law.shift : 0.0, __ddiv_rn(e, law.mu));
}

// Draw q of the minibatch of task (replica, worker, seq): floor(u32 * n / 2^32), n <= 2^32.
__device__ __forceinline__ uint32_t draw_index(uint64_t seed, uint32_t replica, uint32_t worker,
                                               uint32_t seq, uint32_t q, uint64_t n) {
  const U4 x = stream_block(seed, 1u, q >> 2, replica, worker, seq);
  const uint32_t sel = q & 3u;
  const uint32_t v = sel == 0 ? x.x : sel == 1 ? x.y : sel == 2 ? x.z : x.w;
  return (uint32_t)(((uint64_t)v * n) >> 32);
}

}  // namespace ssim
