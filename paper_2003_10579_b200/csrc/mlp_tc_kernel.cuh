// The MLP's two products over d on the 5th-generation tensor cores (tcgen05), accumulators in tensor memory:
// mlp_forward_tc_kernel (training, persistent), mlp_risk_tc_kernel (forward-only, full-data risk), mlp_dw1_tc_kernel.
// Every mbarrier wait is bounded; a wait that runs out sets the error word and the CTA drains.
#pragma once
#include <cuda.h>

#include "mlp_kernel.cuh"
#include "softmax_kernel.cuh"

namespace ssim {

constexpr int TC_BK = 64;                       // k per stage: one 128-byte swizzle atom of bf16
constexpr int TC_A_BYTES = 128 * 128;           // 128 rows x 128 B
constexpr int TC_THREADS = 320;      // warp 0 B producer, warp 1 MMA, warps 2-5 A producers + epilogue, warps 6-9 epilogue helpers

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
// named barrier `id` (1..15) over `threads` threads (a multiple of 32)
__device__ __forceinline__ void group_barrier(int id, int threads) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_alloc(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]),
        "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]),
        "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]),
        "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle.  K-major operand: rows (M or N) are 128 B
// apart, 8-row groups 1024 B apart (stride byte offset); the leading byte offset is unused.
__device__ __forceinline__ uint64_t tc_desc_kmajor(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}
// bf16 x bf16 -> f32, M = 128, N = n, both operands K-major
__device__ __forceinline__ uint32_t tc_idesc(int n, int a_mn_major, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

constexpr int FWD_LAG = 2;    // k-blocks of A in flight per producer thread before the oldest is signalled
struct TcLayout {   // shared-memory plan of the forward kernel (offsets from a 1024-byte aligned base)
  int sa, sb, b_bytes, off_b, off_w2, off_b1, off_b2, off_rows, off_labels, off_zx, off_bars, off_tmem, total;
};
// The operands have rings of their own: A (128 samples x 64 k, 16 KB) in `sa` slots; B in `sb` slots of
// [n_inst x 64 k], n_inst = H (H <= 256) or H/2 - half a k-block of W1 per slot, so that several loads of
// 32 KB are in flight instead of one of 64 KB.  The main loop is bound by the latency of those loads, i.e. by the bytes
// in flight, so everything the epilogue alone needs (W2 padded to 16 classes, the partial logits) lives in the A ring's
// bytes, which are free once the last MMA has completed, and the B ring gets the room.
inline __host__ __device__ TcLayout tc_forward_layout(int H) {
  TcLayout L;
  L.b_bytes = (H > 256 ? H / 2 : H) * 128;
  L.sa = 4;
  L.sb = 4;
  L.off_w2 = 0;                                   // [H][16] floats, after the main loop
  L.off_zx = L.off_w2 + H * 16 * 4;               // partial logits of the two column halves: [2][128][16], after the main loop
  L.off_b = L.sa * TC_A_BYTES;
  L.off_b1 = L.off_b + L.sb * L.b_bytes;
  L.off_b2 = L.off_b1 + H * 4;
  L.off_rows = L.off_b2 + 64;
  L.off_labels = L.off_rows + 128 * 4;
  L.off_bars = L.off_labels + 128 * 4;
  L.off_tmem = L.off_bars + 8 * (2 * L.sa + 2 * L.sb + 1);
  L.total = L.off_tmem + 16 + 1024;   // slack for the manual 1024-byte alignment
  return L;
}
static_assert(512 * 16 * 4 + 2 * 128 * 16 * 4 <= 4 * TC_A_BYTES, "W2 and the partial logits must fit the A ring's bytes");

// Forward-only pass for the full-data risk F(w) of Eq. 1: one CTA per (replica, 128 consecutive rows of the data set),
// A1[128 x H] = bf16(X_b)[128 x d] bf16(W1)[d x H] with the replica's current version; only the rows' losses leave the CTA.
//   warp 0   B producer: TMA tensor loads of W1 from the transposed, k-block-tiled bf16 shadow (K-major B
//            operand, 128-byte swizzle), half a k-block ([H/2 x 64], contiguous in the shadow) per ring
//            slot; the first slots are requested before the block's opening barrier
//   warps 2-5  A producer during the main loop: the 128 sample rows of a k-block are 1024
//            16-byte pieces, copied with cp.async into the same 128-byte-swizzle pattern, made visible to the
//            tensor core's asynchronous proxy with a proxy fence before the slot is signalled
//   warp 1   allocates tensor memory; one elected lane issues tcgen05.mma (M=128, N<=256, K=16)
//            and commits slot-free / accumulator-ready mbarriers
//   warps 6-9  during the main loop: stage b1, W2 (padded to 16 classes) and b2
//   warps 2-9  epilogue: tcgen05.ld gives each thread one sample's row of A1 - warps 2-5 the first
//            half of the hidden units, warps 6-9 the second - so bias, relu and the partial logits
//            need no cross-thread reduction; the two partial logit vectors of a row meet in shared
//            memory and the row's softmax cross-entropy is summed per warp
__global__ void __launch_bounds__(TC_THREADS, 1)
mlp_risk_tc_kernel(const __grid_constant__ CUtensorMap tmW, MlpArgs g) {
  const NumericArgs& a = g.na;
  const MlpScratch& sc = g.sc;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int H = sc.H, C = sc.C, d = sc.d;
  const int mtiles = g.eval_blocks;
  const int mt = blockIdx.x % mtiles;
  const int r = blockIdx.x / mtiles;
  const int snap = g.eval_slot ? (int)g.eval_slot[r] : g.eval_parity;
  const long long dH = (long long)d * H;
  const float* wsnap = a.pool + ((size_t)r * a.n_slots + snap) * a.slot_stride;
  const int n_halves = H > 256 ? 2 : 1;
  const int n_inst = H / n_halves;
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < H) tmem_cols <<= 1;

  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw_addr = smem_addr(smem_raw);
  const uint32_t base_addr = (raw_addr + 1023u) & ~1023u;
  unsigned char* base = smem_raw + (base_addr - raw_addr);
  const TcLayout L = tc_forward_layout(H);
  const int SA = L.sa, SB = L.sb;
  float* W2_s = reinterpret_cast<float*>(base + L.off_w2);
  float* b1_s = reinterpret_cast<float*>(base + L.off_b1);
  float* b2_s = reinterpret_cast<float*>(base + L.off_b2);
  int* rows_s = reinterpret_cast<int*>(base + L.off_rows);
  int* label_s = reinterpret_cast<int*>(base + L.off_labels);
  float* zx_s = reinterpret_cast<float*>(base + L.off_zx);
  const uint32_t bars = base_addr + L.off_bars;            // afull[SA] | aempty[SA] | bfull[SB] | bempty[SB] | acc_ready
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base + L.off_tmem);
  auto afull = [&](int s) { return bars + 8u * s; };
  auto aempty = [&](int s) { return bars + 8u * (SA + s); };
  auto bfull = [&](int s) { return bars + 8u * (2 * SA + s); };
  auto bempty = [&](int s) { return bars + 8u * (2 * SA + SB + s); };
  const uint32_t acc_bar = bars + 8u * (2 * SA + 2 * SB);

  if (tid == 0) {
    // an A slot is full after its 128 producer threads arrived, a B slot after the TMA bytes (one arrival with expect_tx)
    for (int s = 0; s < SA; ++s) { mbar_init(afull(s), 128); mbar_init(aempty(s), 1); }
    for (int s = 0; s < SB; ++s) { mbar_init(bfull(s), 1); mbar_init(bempty(s), 1); }
    mbar_init(acc_bar, 1);
    mbar_fence_init();
  }
  const int nk = d / TC_BK;
  const long long w_blk0 = ((long long)r * sc.n_slots + snap) * (d / TC_BK);     // first k-block of this W1^T shadow
  const int n_first = min(SB, nk * n_halves);       // B loads that need no free slot: issued before the block barrier
  if (tid == 0) {
    for (int n = 0; n < n_first; ++n) {
      mbar_arrive_expect_tx(bfull(n), (uint32_t)L.b_bytes);
      tma_load_2d(base_addr + L.off_b + (uint32_t)n * L.b_bytes, &tmW, 0, (int)((w_blk0 + n / n_halves) * H + (n % n_halves) * n_inst), bfull(n));
    }
  }
  if (warp == 1) tc_alloc(smem_addr(tmem_slot), tmem_cols);
  if (tid >= 64 && tid < 192) {                     // sample rows and labels (the A producers need them first)
    const int t = tid - 64;
    // consecutive rows; a row past the end of the data set repeats the last one and is left out of the sum
    const uint64_t want = (uint64_t)mt * 128 + t;
    const uint32_t idx = (uint32_t)(want < a.n ? want : a.n - 1);
    rows_s[t] = (int)idx;
    label_s[t] = reinterpret_cast<const int*>(a.y)[idx];
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  bool failed = false;

  if (warp == 0) {
    // ---- B producer ----
    if (lane == 0) {
      for (int n = n_first; n < nk * n_halves; ++n) {
        const int s = n % SB, kc = n / n_halves, hf = n % n_halves;
        if (!mbar_wait(bempty(s), (uint32_t)(((n / SB) & 1) ^ 1))) { failed = true; break; }
        mbar_arrive_expect_tx(bfull(s), (uint32_t)L.b_bytes);
        tma_load_2d(base_addr + L.off_b + (uint32_t)s * L.b_bytes, &tmW, 0, (int)((w_blk0 + kc) * H + hf * n_inst), bfull(s));
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---- MMA issuer ----
    const uint32_t idesc = tc_idesc(n_inst, 0, 0);
    for (int kc = 0; kc < nk && !failed; ++kc) {
      const int sa = kc % SA;
      if (!mbar_wait(afull(sa), (uint32_t)((kc / SA) & 1))) { failed = true; break; }
      const uint32_t As = base_addr + (uint32_t)sa * TC_A_BYTES;
      for (int hf = 0; hf < n_halves; ++hf) {
        const int n = kc * n_halves + hf, s = n % SB;
        if (!mbar_wait(bfull(s), (uint32_t)((n / SB) & 1))) { failed = true; break; }
        tc_fence_after();
        if (lane == 0) {
          const uint32_t Bs = base_addr + L.off_b + (uint32_t)s * L.b_bytes;
#pragma unroll
          for (int k16 = 0; k16 < TC_BK / 16; ++k16)
            tc_mma_bf16(tmem_base + (uint32_t)hf * n_inst, tc_desc_kmajor(As + k16 * 32), tc_desc_kmajor(Bs + k16 * 32), idesc,
                        (kc > 0 || k16 > 0) ? 1u : 0u);
          tc_commit(bempty(s));                     // the slot may be refilled once these MMAs have read it
          if (hf == n_halves - 1) {
            tc_commit(aempty(sa));
            if (kc == nk - 1) tc_commit(acc_bar);   // accumulator complete
          }
        }
        __syncwarp();
      }
    }
  } else {
    // ---- warps 2-9: thread = one sample row and one half of the hidden units in the epilogue ----
    const int q = warp & 3;                         // the TMEM lane quarter this warp may read
    const int ehalf = warp >= 6 ? 1 : 0;            // hidden units [ehalf * H/2, +H/2)
    const int row = 32 * q + lane;
    if (ehalf) {
      // ---- helpers: b1 and b2 of the snapshot during the main loop; W2 (rows padded to 16 classes) goes into the A
      //      ring's bytes once the last MMA has read them (its values wait in registers meanwhile) ----
      const int t = tid - 192;
      const float* b1 = wsnap + dH;
      const float* W2 = b1 + H;
      const float* b2 = W2 + (size_t)H * C;
      for (int i = t; i < H; i += 128) b1_s[i] = b1[i];
      if (t < 16) b2_s[t] = t < C ? b2[t] : 0.f;
      float w2v[64];                                 // H * 16 / 128 <= 64 entries per thread
#pragma unroll
      for (int u = 0; u < 64; ++u) {
        const int i = t + 128 * u, col = i >> 4, c = i & 15;
        w2v[u] = (i < H * 16 && c < C) ? W2[(size_t)col * C + c] : 0.f;
      }
      if (!mbar_wait(acc_bar, 0)) failed = true;
#pragma unroll
      for (int u = 0; u < 64; ++u) {
        const int i = t + 128 * u;
        if (i < H * 16) W2_s[i] = w2v[u];
      }
    } else
    // ---- A producer: thread t copies 16-byte piece (t & 7) of rows (t >> 3) + 16 i, i < 8.  A k-block is
    //      signalled FWD_LAG k-blocks after it was issued; the ring is deeper than that (SA > FWD_LAG + 1), so
    //      the signal never waits for a slot whose release depends on the k-block just before the signalled one.
    {
      const int t = tid - 64, ch = t & 7, row0 = t >> 3;
      auto signal = [&](int kc2) {          // pieces of k-block kc2 have landed: publish to the async proxy
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_arrive(afull(kc2 % SA));
      };
      int signalled = 0;
      for (int kc = 0; kc < nk && !failed; ++kc) {
        const int s = kc % SA;
        if (!mbar_wait(aempty(s), (uint32_t)(((kc / SA) & 1) ^ 1))) { failed = true; break; }
        const uint32_t As = base_addr + (uint32_t)s * TC_A_BYTES;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int rw = row0 + 16 * i;
          cp_async16(As + rw * 128 + ((ch ^ (rw & 7)) << 4), sc.Xq + (size_t)rows_s[rw] * d + (size_t)kc * TC_BK + ch * 8);
        }
        cp_async_commit();
        if (kc >= FWD_LAG) {
          cp_async_wait<FWD_LAG>();
          signal(signalled++);
        }
      }
      cp_async_wait<0>();
      if (!failed) while (signalled < nk) signal(signalled++);
    }
    group_barrier(1, 256);                          // b1 / W2 / b2 are in shared memory (all eight warps, failed or not)
    if (!failed && !mbar_wait(acc_bar, 0)) failed = true;
    tc_fence_after();
    const uint32_t trow = tmem_base + ((uint32_t)(32 * q) << 16);
    const int ch0 = ehalf * (H / 64), ch1 = ch0 + H / 64;
    float z[16];
    uint32_t v[32];
    if (!failed) {
#pragma unroll
      for (int c = 0; c < 16; ++c) z[c] = 0.f;
      for (int ch = ch0; ch < ch1; ++ch) {
        tc_ld32(trow + ch * 32, v);
#pragma unroll
        for (int i4 = 0; i4 < 8; ++i4) {
          float hv[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int col = ch * 32 + i4 * 4 + e;
            hv[e] = fmaxf(__uint_as_float(v[i4 * 4 + e]) + b1_s[col], 0.f);
            const float4* wr = reinterpret_cast<const float4*>(W2_s + col * 16);
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
              if (4 * c4 < C) {
                const float4 w = wr[c4];
                z[4 * c4] = fmaf(hv[e], w.x, z[4 * c4]); z[4 * c4 + 1] = fmaf(hv[e], w.y, z[4 * c4 + 1]);
                z[4 * c4 + 2] = fmaf(hv[e], w.z, z[4 * c4 + 2]); z[4 * c4 + 3] = fmaf(hv[e], w.w, z[4 * c4 + 3]);
              }
            }
          }
        }
      }
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4)
        reinterpret_cast<float4*>(zx_s + (ehalf * 128 + row) * 16)[c4] = make_float4(z[4 * c4], z[4 * c4 + 1], z[4 * c4 + 2], z[4 * c4 + 3]);
    }
    group_barrier(1, 256);                          // both halves of every row's logits are published
    if (!failed) {
      // logits = b2 + half 0 + half 1
#pragma unroll
      for (int c = 0; c < 16; ++c) z[c] = (b2_s[c] + zx_s[row * 16 + c]) + zx_s[(128 + row) * 16 + c];
      if (!ehalf) {
        float d2[16];
        const bool real = (uint64_t)mt * 128 + row < a.n;
        const float loss = mlp_row_softmax<false>(z, C, label_s[row], d2);
        const float rowloss = warp_sum(real ? loss : 0.f);
        if (lane == 0) g.eval_part[((size_t)r * g.eval_blocks + mt) * 4 + q] = rowloss;
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tc_dealloc(tmem_base, tmem_cols);
  if (failed && lane == 0) atomicExch(a.err, ERR_WAIT_TIMEOUT);
}



// Position in a ring of n slots: slot and phase parity of use number u, stepped as counters (u % n and u / n with a
// run-time n and a 64-bit u are a division subroutine each, on the critical path of single-thread roles).
struct RingPos {
  int s;
  uint32_t ph;
  __device__ __forceinline__ void step(int n, int by = 1) { s += by; if (s >= n) { s -= n; ph ^= 1u; } }
};


// ---- training forward pass: persistent kernel --------------------------------------------------------------------
// Tiles of one (replica, contributor, 128-sample block) x Hn hidden units (Hn = H, or H/2 for H > 256) are dealt round-robin
// to one CTA per SM; the two halves of a block are neighbours in that order, so that the second reader of the block's
// sample rows finds them in L2.  The accumulator is double-buffered in tensor memory: the epilogue of one tile runs under
// the loads and MMAs of the next.  The epilogue gives each thread one sample's row of A1 (tcgen05.ld 32x32b), so bias, relu
// and the tile's share of the logits h W2 need no cross-thread reduction; h and the partial logits go to global memory and
// the head kernel takes it from there (softmax needs all hidden units of a row, which no single tile has).
//   warp 0      TMA producer of B: [Hn x 64] blocks of the transposed, k-block-tiled bf16 shadow of W1 (K-major operand,
//               128-byte swizzle), one ring slot per k-block
//   warp 1      allocates tensor memory; one elected lane issues tcgen05.mma (M = 128, N = Hn, K = 16) and commits the
//               slot-free / accumulator-ready mbarriers
//   warps 2-5   A producers: the 128 gathered sample rows of a k-block are 1024 16-byte pieces, copied with cp.async into
//               the 128-byte-swizzle pattern (one-row TMA boxes of 128 B were limited by the TMA instruction rate) and
//               made visible to the tensor core's asynchronous proxy with a proxy fence before the slot is signalled
//   warps 6-9   epilogue (one warp per tensor-memory lane quarter): stage b1 and W2 (rows padded to 16 classes) of the
//               tile's snapshot and hidden units in shared memory, wait for the accumulator, form h and the partial logits
struct TcFwdLayout { int sa, sb, b_bytes, off_b, off_w2, off_b1, off_bars, off_tmem, off_fail, total; };
inline __host__ __device__ TcFwdLayout tc_fwd_layout(int H) {
  TcFwdLayout L;
  const int Hn = H > 256 ? H / 2 : H;
  const int budget = 226 << 10;
  L.b_bytes = Hn * 128;
  L.sa = 4;
  const int fixed = L.sa * TC_A_BYTES + Hn * 64 + Hn * 4 + 8 * (2 * L.sa + 2 * 8 + 4) + 32 + 1024;
  L.sb = (budget - fixed) / L.b_bytes;
  if (L.sb > 8) L.sb = 8;
  L.off_b = L.sa * TC_A_BYTES;
  L.off_w2 = L.off_b + L.sb * L.b_bytes;          // [Hn][16] floats
  L.off_b1 = L.off_w2 + Hn * 64;
  L.off_bars = L.off_b1 + Hn * 4;
  L.off_tmem = L.off_bars + 8 * (2 * L.sa + 2 * L.sb + 4);
  L.off_fail = L.off_tmem + 16;
  L.total = L.off_fail + 16 + 1024;               // slack for the manual 1024-byte alignment
  return L;
}

__global__ void __launch_bounds__(TC_THREADS, 1)
mlp_forward_tc_kernel(const __grid_constant__ CUtensorMap tmW, MlpArgs g) {
  const NumericArgs& a = g.na;
  const MlpScratch& sc = g.sc;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int H = sc.H, C = sc.C, d = sc.d, m = sc.m;
  const int mtiles = m / 128, n_halves = H > 256 ? 2 : 1, Hn = H / n_halves;
  const int n_tiles = a.R * sc.Kmax * mtiles * n_halves;
  const int nk = d / TC_BK;
  const long long j = g.j;
  const long long dH = (long long)d * H;
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < 2 * Hn) tmem_cols <<= 1;

  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw_addr = smem_addr(smem_raw);
  const uint32_t base_addr = (raw_addr + 1023u) & ~1023u;
  unsigned char* base = smem_raw + (base_addr - raw_addr);
  const TcFwdLayout L = tc_fwd_layout(H);
  const int SA = L.sa, SB = L.sb;
  float* W2_s = reinterpret_cast<float*>(base + L.off_w2);
  float* b1_s = reinterpret_cast<float*>(base + L.off_b1);
  const uint32_t bars = base_addr + L.off_bars;      // afull[SA] | aempty[SA] | bfull[SB] | bempty[SB] | acc_full[2] | acc_empty[2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base + L.off_tmem);
  volatile int* fail_s = reinterpret_cast<volatile int*>(base + L.off_fail);
  auto afull = [&](int s) { return bars + 8u * s; };
  auto aempty = [&](int s) { return bars + 8u * (SA + s); };
  auto bfull = [&](int s) { return bars + 8u * (2 * SA + s); };
  auto bempty = [&](int s) { return bars + 8u * (2 * SA + SB + s); };
  auto acc_full = [&](int b) { return bars + 8u * (2 * SA + 2 * SB + b); };
  auto acc_empty = [&](int b) { return bars + 8u * (2 * SA + 2 * SB + 2 + b); };

  if (tid == 0) {
    // an A slot is full after its 128 producer threads arrived, a B slot after the TMA bytes (one arrival with expect_tx)
    for (int s = 0; s < SA; ++s) { mbar_init(afull(s), 128); mbar_init(aempty(s), 1); }
    for (int s = 0; s < SB; ++s) { mbar_init(bfull(s), 1); mbar_init(bempty(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), 4); }
    fail_s[0] = 0;
    mbar_fence_init();
  }
  if (warp == 1) tc_alloc(smem_addr(tmem_slot), tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  bool failed = false;
  // tile t -> (replica r, contributor l, sample block mt, half hf of the hidden units); false for a contributor the
  // update does not have (l >= K), which every role skips alike
  auto tile_of = [&](int t, int& r, int& l, int& mt, int& hf) {
    hf = t % n_halves;
    int x = t / n_halves;
    mt = x % mtiles; x /= mtiles;
    l = x % sc.Kmax;
    r = x / sc.Kmax;
    return l < (int)a.K_used[(size_t)r * a.cap + j];
  };

  if (warp == 0) {
    // ---- B producer ----
    if (lane == 0) {
      RingPos rp{0, 0u};
      for (int t = blockIdx.x; t < n_tiles && !failed; t += gridDim.x) {
        int r, l, mt, hf;
        if (!tile_of(t, r, l, mt, hf)) continue;
        const long long w_blk0 = ((long long)r * sc.n_slots + mlp_snap_slot(a, r, j, l)) * nk;     // first k-block of this W1^T shadow
        for (int kc = 0; kc < nk; ++kc, rp.step(SB)) {
          const int s = rp.s;
          if (!mbar_wait(bempty(s), rp.ph ^ 1u)) { failed = true; break; }
          mbar_arrive_expect_tx(bfull(s), (uint32_t)L.b_bytes);
          tma_load_2d(base_addr + L.off_b + (uint32_t)s * L.b_bytes, &tmW, 0, (int)((w_blk0 + kc) * H + hf * Hn), bfull(s));
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---- MMA issuer ----
    const uint32_t idesc = tc_idesc(Hn, 0, 0);
    RingPos ra{0, 0u}, rb{0, 0u};
    int i = 0;
    for (int t = blockIdx.x; t < n_tiles && !failed; t += gridDim.x) {
      int r, l, mt, hf;
      if (!tile_of(t, r, l, mt, hf)) continue;
      const int buf = i & 1;
      if (!mbar_wait(acc_empty(buf), (uint32_t)(((i >> 1) & 1) ^ 1))) { failed = true; break; }
      tc_fence_after();
      for (int kc = 0; kc < nk; ++kc, ra.step(SA), rb.step(SB)) {
        if (!mbar_wait(afull(ra.s), ra.ph) || !mbar_wait(bfull(rb.s), rb.ph)) { failed = true; break; }
        tc_fence_after();
        if (lane == 0) {
          const uint32_t As = base_addr + (uint32_t)ra.s * TC_A_BYTES, Bs = base_addr + L.off_b + (uint32_t)rb.s * L.b_bytes;
#pragma unroll
          for (int k16 = 0; k16 < TC_BK / 16; ++k16)
            tc_mma_bf16(tmem_base + (uint32_t)(buf * Hn), tc_desc_kmajor(As + k16 * 32), tc_desc_kmajor(Bs + k16 * 32), idesc,
                        (kc > 0 || k16 > 0) ? 1u : 0u);
          tc_commit(bempty(rb.s));                  // the slots may be refilled once these MMAs have read them
          tc_commit(aempty(ra.s));
          if (kc == nk - 1) tc_commit(acc_full(buf));
        }
        __syncwarp();
      }
      ++i;
    }
  } else if (warp < 6) {
    // ---- A producers: thread p copies 16-byte piece (p & 7) of rows (p >> 3) + 16 i, i < 8.  A k-block is
    //      signalled FWD_LAG k-blocks after it was issued; the ring is deeper than that (SA > FWD_LAG + 1), so
    //      the signal never waits for a slot whose release depends on the k-block just before the signalled one.
    const int p = tid - 64, piece = p & 7, row0 = p >> 3;
    long long it = 0, signalled = 0;
    RingPos rp{0, 0u}, sig{0, 0u};
    auto signal = [&]() {                 // the oldest unsignalled k-block has landed: publish to the async proxy
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(afull(sig.s));
      sig.step(SA);
      ++signalled;
    };
    for (int t = blockIdx.x; t < n_tiles && !failed; t += gridDim.x) {
      int r, l, mt, hf;
      if (!tile_of(t, r, l, mt, hf)) continue;
      const int* rows = sc.rows_tab + ((size_t)r * sc.Kmax + l) * m + (size_t)mt * 128;
      const __nv_bfloat16* src[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) src[i] = sc.Xq + (size_t)rows[row0 + 16 * i] * d + piece * 8;
      for (int kc = 0; kc < nk; ++kc, ++it, rp.step(SA)) {
        if (!mbar_wait(aempty(rp.s), rp.ph ^ 1u)) { failed = true; break; }
        const uint32_t As = base_addr + (uint32_t)rp.s * TC_A_BYTES;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int rw = row0 + 16 * i;
          cp_async16(As + rw * 128 + ((piece ^ (rw & 7)) << 4), src[i] + (size_t)kc * TC_BK);
        }
        cp_async_commit();
        if (it >= FWD_LAG) {
          cp_async_wait<FWD_LAG>();
          signal();
        }
      }
    }
    cp_async_wait<0>();
    if (!failed) while (signalled < it) signal();
  } else {
    // ---- epilogue: thread = one sample row of the tile ----
    const int q = warp & 3;                         // the tensor-memory lane quarter this warp may read
    const int row = 32 * q + lane, e0 = tid - 192;
    for (int e = e0; e < Hn * 16; e += 128) W2_s[e] = 0.f;      // the padding classes stay zero
    group_barrier(1, 128);
    int i = 0;
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x) {
      int r, l, mt, hf;
      if (!tile_of(t, r, l, mt, hf)) continue;
      const int buf = i & 1;
      const float* b1 = a.pool + ((size_t)r * a.n_slots + mlp_snap_slot(a, r, j, l)) * a.slot_stride + dH + hf * Hn;
      const float* W2 = b1 + (H - hf * Hn) + (size_t)hf * Hn * C;
      for (int e = e0; e < Hn; e += 128) b1_s[e] = b1[e];
      for (int e = e0; e < Hn * C; e += 128) {
        const int col = e / C;
        W2_s[col * 16 + (e - col * C)] = W2[e];
      }
      if (!mbar_wait(acc_full(buf), (uint32_t)((i >> 1) & 1))) fail_s[0] = 1;
      group_barrier(1, 128);                        // b1 / W2 are staged; the four warps give up together or not at all
      if (fail_s[0]) { failed = true; break; }
      tc_fence_after();
      const size_t grow = ((size_t)r * sc.Kmax + l) * m + (size_t)mt * 128 + row;
      const uint32_t trow = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * Hn);
      float z[16];
#pragma unroll
      for (int c = 0; c < 16; ++c) z[c] = 0.f;
      for (int ch = 0; ch < Hn / 32; ++ch) {
        uint32_t v[32];
        tc_ld32(trow + ch * 32, v);
        float4* hout = reinterpret_cast<float4*>(sc.Hact + grow * H + hf * Hn + ch * 32);
#pragma unroll
        for (int i4 = 0; i4 < 8; ++i4) {
          float hv[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int col = ch * 32 + i4 * 4 + e;
            hv[e] = fmaxf(__uint_as_float(v[i4 * 4 + e]) + b1_s[col], 0.f);
            const float4* wr = reinterpret_cast<const float4*>(W2_s + col * 16);
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
              if (4 * c4 < C) {
                const float4 w = wr[c4];
                z[4 * c4] = fmaf(hv[e], w.x, z[4 * c4]); z[4 * c4 + 1] = fmaf(hv[e], w.y, z[4 * c4 + 1]);
                z[4 * c4 + 2] = fmaf(hv[e], w.z, z[4 * c4 + 2]); z[4 * c4 + 3] = fmaf(hv[e], w.w, z[4 * c4 + 3]);
              }
            }
          }
          hout[i4] = make_float4(hv[0], hv[1], hv[2], hv[3]);
        }
      }
      tc_fence_before();                            // this warp's reads of the buffer are done: hand it back
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty(buf));
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4)
        reinterpret_cast<float4*>(sc.ZP + (grow * n_halves + hf) * 16)[c4] = make_float4(z[4 * c4], z[4 * c4 + 1], z[4 * c4 + 2], z[4 * c4 + 3]);
      group_barrier(1, 128);                        // b1 / W2 may be overwritten for the next tile
      ++i;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tc_dealloc(tmem_base, tmem_cols);
  if (failed && lane == 0) atomicExch(a.err, ERR_WAIT_TIMEOUT);
}

// Shared-memory matrix descriptor, 128-byte swizzle, MN-major operand (the M or N index is the
// contiguous one): 64-element (128-byte) runs along MN, 8 such k-rows form a 1024-byte atom;
// the next 8 k-rows are `sbo` bytes on (stride byte offset), the next 64 MN elements `lbo` bytes on
// (leading byte offset).
__device__ __forceinline__ uint64_t tc_desc_mnmajor(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}

// ---- dW1 = bf16(X)^T bf16(delta1), fused with the update of W1: persistent kernel -----------------
// Tiles of 128 rows of W1 x Hn columns (Hn <= 256) are dealt round-robin to one CTA per SM.  The
// accumulator is double-buffered in tensor memory, so the epilogue of one tile overlaps the loads and
// MMAs of the next.  Both operands are MN-major and used exactly as stored: a stage holds 64 samples;
// A = their features [slab*128, +128) gathered from the bf16 data set (cp.async by four producer warps
// into the 128-byte-swizzle atom layout), B = the same samples' bf16 delta1 columns (TMA boxes of
// 64 x 64).  dW1 itself never exists in memory.
// The epilogue never touches global memory from a register: w_j streams in as 16 KB blocks (128 rows x 32
// columns, contiguous in the pool) by bulk copies into a ring of shared-memory slots, a group of four
// warps (thread = row) applies Eq. 2 / Eq. 3 in place from the accumulator, writes the bf16 shadow of the
// block beside it, and one thread sends both out with bulk stores.
//   warp 0      TMA producer of B          warp 1      tcgen05.mma issuer, owns tensor memory
//   warps 2-5   cp.async producers of A    warps 6-13  epilogue: two groups of four warps (one per tensor-
//   warp 14     bulk-copy producer of w_j               memory lane quarter), blocks of a tile dealt alternately
constexpr int DW1_THREADS = 480;
constexpr int DW1_WBLOCK = 16384;        // one block of W1 in fp32
constexpr int DW1_QSTAGE = 8192;         // its bf16 shadow: two k-blocks of 32 columns x 64 rows

// columns per tile: the largest H/p that is at most 256 and a multiple of 64
inline __host__ __device__ int tc_dw1_cols(int H) {
  for (int p = 1; p <= 8; ++p)
    if (H % p == 0 && H / p <= 256 && (H / p) % 64 == 0) return H / p;
  return 64;
}
struct TcDw1Layout { int stages, stage_bytes, wslots, off_w, off_q, off_bars, off_tmem, off_fail, off_dist, total; };
inline __host__ __device__ TcDw1Layout tc_dw1_layout(int H) {
  TcDw1Layout L;
  const int budget = 224 << 10;
  L.stage_bytes = TC_A_BYTES + tc_dw1_cols(H) * 128;     // A: 64 samples x 128 features; B: 64 samples x Hn
  L.stages = (budget - 2 * DW1_QSTAGE - 3 * DW1_WBLOCK) / L.stage_bytes;
  if (L.stages > 4) L.stages = 4;
  L.wslots = (budget - 2 * DW1_QSTAGE - L.stages * L.stage_bytes) / DW1_WBLOCK;
  if (L.wslots > 6) L.wslots = 6;
  L.off_w = L.stages * L.stage_bytes;
  L.off_q = L.off_w + L.wslots * DW1_WBLOCK;
  L.off_bars = L.off_q + 2 * DW1_QSTAGE;
  L.off_tmem = L.off_bars + 8 * (2 * L.stages + 4 + 2 * L.wslots);
  L.off_fail = L.off_tmem + 16;
  L.off_dist = L.off_fail + 16;        // [2 groups][4 warps] partial distances
  L.total = L.off_dist + 32 + 1024;
  return L;
}

__device__ __forceinline__ void bulk_s2g(void* dst, uint32_t src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__global__ void __launch_bounds__(DW1_THREADS, 1)
mlp_dw1_tc_kernel(const __grid_constant__ CUtensorMap tmD, MlpArgs g) {
  const NumericArgs& a = g.na;
  const MlpScratch& sc = g.sc;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int H = sc.H, d = sc.d, m = sc.m;
  const int slabs = d / 128, Hn = tc_dw1_cols(H), parts = H / Hn;
  const int n_tiles = a.R * slabs * parts;
  const long long j = g.j;
  const long long dH = (long long)d * H;
  const int blocks_per_task = m / TC_BK;
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < 2 * Hn) tmem_cols <<= 1;

  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw_addr = smem_addr(smem_raw);
  const uint32_t base_addr = (raw_addr + 1023u) & ~1023u;
  unsigned char* base = smem_raw + (base_addr - raw_addr);
  const TcDw1Layout L = tc_dw1_layout(H);
  const int S = L.stages;
  const int NB = L.wslots;
  const uint32_t bars = base_addr + L.off_bars;     // full[S] | empty[S] | acc_full[2] | acc_empty[2] | wfull[NB] | wempty[NB]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base + L.off_tmem);
  volatile int* fail_s = reinterpret_cast<volatile int*>(base + L.off_fail);     // one flag per epilogue group
  float* dist_s = reinterpret_cast<float*>(base + L.off_dist);
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (S + s); };
  auto acc_full = [&](int b) { return bars + 8u * (2 * S + b); };
  auto acc_empty = [&](int b) { return bars + 8u * (2 * S + 2 + b); };
  auto wfull = [&](int s) { return bars + 8u * (2 * S + 4 + s); };
  auto wempty = [&](int s) { return bars + 8u * (2 * S + 4 + NB + s); };

  if (tid == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1 + 128); mbar_init(empty_bar(s), 1); }    // B's expect_tx arrival + A's 128 producer threads
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), 8); }
    for (int s = 0; s < NB; ++s) { mbar_init(wfull(s), 1); mbar_init(wempty(s), 1); }
    fail_s[0] = 0; fail_s[1] = 0;
    mbar_fence_init();
  }
  if (warp == 1) tc_alloc(smem_addr(tmem_slot), tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  bool failed = false;
  const uint32_t ATOM = 8192;     // one 64-wide MN block of a 64-sample stage: 64 k-rows x 128 B
  // tile t -> (replica, slab, column part); the number of 64-sample stages depends on the replica's K
  auto tile_r = [&](int t) { return t / (parts * slabs); };
  auto tile_nk = [&](int t) { return (int)a.K_used[(size_t)tile_r(t) * a.cap + j] * blocks_per_task; };

  if (warp == 0) {
    // ---- B producer: delta1 rows of 64 samples, Hn/64 boxes of 64 x 64 ----
    if (lane == 0) {
      RingPos rp{0, 0u};
      for (int t = blockIdx.x; t < n_tiles && !failed; t += gridDim.x) {
        const int r = tile_r(t), part = t % parts, nk = tile_nk(t);
        for (int kc = 0; kc < nk; ++kc, rp.step(S)) {
          const int s = rp.s;
          if (!mbar_wait(empty_bar(s), rp.ph ^ 1u)) { failed = true; break; }
          const uint32_t Bs = base_addr + (uint32_t)s * L.stage_bytes + TC_A_BYTES;
          const int row0 = (int)((size_t)r * sc.Kmax * m + (size_t)kc * TC_BK);
          mbar_arrive_expect_tx(full_bar(s), (uint32_t)(Hn * 128));
          for (int b = 0; b < Hn / 64; ++b) tma_load_2d(Bs + (uint32_t)b * ATOM, &tmD, part * Hn + b * 64, row0, full_bar(s));
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---- MMA issuer ----
    const uint32_t idesc = tc_idesc(Hn, 1, 1);
    const uint32_t lbo = ATOM, sbo = 1024u;   // next 64 MN elements: one atom block on; next 8 samples: 1024 B on
    RingPos rp{0, 0u};
    int i = 0;
    for (int t = blockIdx.x; t < n_tiles && !failed; t += gridDim.x, ++i) {
      const int nk = tile_nk(t), buf = i & 1;
      if (!mbar_wait(acc_empty(buf), (uint32_t)(((i >> 1) & 1) ^ 1))) { failed = true; break; }
      tc_fence_after();
      for (int kc = 0; kc < nk; ++kc, rp.step(S)) {
        const int s = rp.s;
        if (!mbar_wait(full_bar(s), rp.ph)) { failed = true; break; }
        tc_fence_after();
        if (lane == 0) {
          const uint32_t As = base_addr + (uint32_t)s * L.stage_bytes, Bs = As + TC_A_BYTES;
#pragma unroll
          for (int k16 = 0; k16 < TC_BK / 16; ++k16) {      // 16 samples = two 8-row groups = 2048 B
            const uint64_t ad = tc_desc_mnmajor(As + k16 * 2048, lbo, sbo);
            const uint64_t bd = tc_desc_mnmajor(Bs + k16 * 2048, lbo, sbo);
            tc_mma_bf16(tmem_base + (uint32_t)buf * Hn, ad, bd, idesc, (kc > 0 || k16 > 0) ? 1u : 0u);
          }
          tc_commit(empty_bar(s));
          if (kc == nk - 1) tc_commit(acc_full(buf));
        }
        __syncwarp();
      }
    }
  } else if (warp < 6) {
    // ---- A producers: thread p copies 16-byte piece (p & 15) of sample rows (p >> 4) + 8 i, i < 8.  A stage is
    //      signalled `lag` stages after it was issued, lag = S - 2: the signal then never waits for a slot
    //      whose release depends on the stage just before the signalled one.
    const int p = tid - 64, piece = p & 15, k0 = p >> 4;
    const int lag = S > 2 ? S - 2 : 1;
    long long it = 0, signalled = 0;
    RingPos rp{0, 0u}, sig{0, 0u};
    auto signal = [&](long long) {      // stages are signalled in order
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(full_bar(sig.s));
      sig.step(S);
    };
    for (int t = blockIdx.x; t < n_tiles && !failed; t += gridDim.x) {
      const int r = tile_r(t), slab = (t / parts) % slabs, nk = tile_nk(t);
      const int* rows = sc.rows_tab + (size_t)r * sc.Kmax * m;
      for (int kc = 0; kc < nk; ++kc, ++it, rp.step(S)) {
        const int s = rp.s;
        int rid[8];                     // issued before the wait: the ring is usually full, the latency hides there
#pragma unroll
        for (int i = 0; i < 8; ++i) rid[i] = rows[kc * TC_BK + k0 + 8 * i];
        if (!mbar_wait(empty_bar(s), rp.ph ^ 1u)) { failed = true; break; }
        const uint32_t As = base_addr + (uint32_t)s * L.stage_bytes + (uint32_t)(piece >> 3) * ATOM;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int k = k0 + 8 * i;
          cp_async16(As + (k >> 3) * 1024 + (k & 7) * 128 + (((piece & 7) ^ (k & 7)) << 4),
                     sc.Xq + (size_t)rid[i] * d + (size_t)slab * 128 + piece * 8);
        }
        cp_async_commit();
        if (it >= lag) {                // the group issued `lag` stages ago has landed
          if (lag == 1) cp_async_wait<1>(); else cp_async_wait<2>();
          signal(signalled++);
        }
      }
    }
    cp_async_wait<0>();
    if (!failed) while (signalled < it) signal(signalled++);
  } else if (warp < 14) {
    // ---- epilogue: thread = one row of the 128-row block; group grp takes blocks grp, grp + 2, ... of a tile ----
    const int q = warp & 3, grp = (warp - 6) >> 2;      // q: the tensor-memory lane quarter this warp may read
    const int rloc = 32 * q + lane, nb = Hn / 32;
    const bool leader = ((warp - 6) & 3) == 0 && lane == 0;
    unsigned char* qstage = base + L.off_q + grp * DW1_QSTAGE;
    // shadow element (k, n) lives at [(k / 64) * H + n] * 64 + k % 64: in the staging copy of a block,
    // [k / 64][n - first column][k % 64]
    __nv_bfloat16* qrow = reinterpret_cast<__nv_bfloat16*>(qstage) + (rloc >> 6) * 2048 + (rloc & 63);
    RingPos wp{grp % NB, (uint32_t)((grp / NB) & 1)};   // ring position of this group's running block number grp, grp + 2, ...
    int i = 0;
    for (int t = blockIdx.x; t < n_tiles && !failed; t += gridDim.x, ++i) {
      const int r = tile_r(t), slab = (t / parts) % slabs, part = t % parts, buf = i & 1;
      const int K = (int)a.K_used[(size_t)r * a.cap + j];
      const int fresh = mlp_fresh_slot(a, r, j);
      const float scale = (float)((double)a.eta / ((double)K * (double)m));
      float* wn = a.pool + ((size_t)r * a.n_slots + fresh) * a.slot_stride + (((size_t)slab * (H >> 5) + ((part * Hn) >> 5)) << 12);
      __nv_bfloat16* wq = sc.W1qT + ((size_t)r * sc.n_slots + fresh) * dH + ((size_t)(2 * slab) * H + part * Hn) * 64;
      const uint32_t trow = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * Hn);
      // reference parameters of this thread's row (row-major [d][H], as the caller gave them) for |w_{j+1} - w_ref|^2
      const float4* wref_row = a.w_ref ? reinterpret_cast<const float4*>(a.w_ref + (size_t)(slab * 128 + rloc) * H + part * Hn) : nullptr;
      float dd = 0.f;
      for (int b = grp; b < nb; b += 2, wp.step(NB, 2)) {
        const int s = wp.s;
        float4 wr[8];                                   // requested before the waits below, so that their latency hides there
        if (wref_row) {
#pragma unroll
          for (int i4 = 0; i4 < 8; ++i4) wr[i4] = wref_row[b * 8 + i4];
        }
        bool ok = mbar_wait(wfull(s), wp.ph);
        if (ok && b == grp) ok = mbar_wait(acc_full(buf), (uint32_t)((i >> 1) & 1));
        if (!ok) fail_s[grp] = 1;
        group_barrier(1 + grp, 128);                    // the four warps give up together or not at all
        if (fail_s[grp]) { failed = true; break; }
        tc_fence_after();
        uint32_t v[32];
        tc_ld32(trow + b * 32, v);
        float4* wrow = reinterpret_cast<float4*>(base + L.off_w + s * DW1_WBLOCK + rloc * 128);
#pragma unroll
        for (int i4 = 0; i4 < 8; ++i4) {
          float4 w = wrow[i4 ^ (rloc & 7)];
          w.x = fmaf(-scale, __uint_as_float(v[4 * i4]), w.x);
          w.y = fmaf(-scale, __uint_as_float(v[4 * i4 + 1]), w.y);
          w.z = fmaf(-scale, __uint_as_float(v[4 * i4 + 2]), w.z);
          w.w = fmaf(-scale, __uint_as_float(v[4 * i4 + 3]), w.w);
          wrow[i4 ^ (rloc & 7)] = w;
          qrow[(4 * i4) * 64] = __float2bfloat16_rn(w.x);
          qrow[(4 * i4 + 1) * 64] = __float2bfloat16_rn(w.y);
          qrow[(4 * i4 + 2) * 64] = __float2bfloat16_rn(w.z);
          qrow[(4 * i4 + 3) * 64] = __float2bfloat16_rn(w.w);
          if (wref_row) {
            const float e0 = w.x - wr[i4].x, e1 = w.y - wr[i4].y, e2 = w.z - wr[i4].z, e3 = w.w - wr[i4].w;
            dd = fmaf(e0, e0, dd); dd = fmaf(e1, e1, dd); dd = fmaf(e2, e2, dd); dd = fmaf(e3, e3, dd);
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        group_barrier(1 + grp, 128);
        if (leader) {
          bulk_s2g(wn + (size_t)b * 4096, base_addr + L.off_w + s * DW1_WBLOCK, DW1_WBLOCK);
          bulk_s2g(wq + (size_t)b * 2048, base_addr + L.off_q + grp * DW1_QSTAGE, 4096);
          bulk_s2g(wq + (size_t)H * 64 + (size_t)b * 2048, base_addr + L.off_q + grp * DW1_QSTAGE + 4096, 4096);
          bulk_commit();
          bulk_wait_read_all();                         // shared memory read out (a fraction of a microsecond): slot and staging are free
          mbar_arrive(wempty(s));
        }
      }
      if (failed) break;
      tc_fence_before();                 // this warp's reads of the buffer are done: hand it back
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty(buf));
      if (wref_row) {
        // This group's share of the tile goes to its own entry; the group that delivers a replica's last entry
        // adds all of them, and the head kernel's, in index order and records the distance (fixed order of sums).
        dd = warp_sum(dd);
        if (lane == 0) dist_s[grp * 4 + q] = dd;
        group_barrier(1 + grp, 128);
        if (leader) {
          const int per_r = slabs * parts * 2;
          float* mine = sc.dist_w1 + (size_t)r * per_r;
          mine[(slab * parts + part) * 2 + grp] = (dist_s[grp * 4] + dist_s[grp * 4 + 1]) + (dist_s[grp * 4 + 2] + dist_s[grp * 4 + 3]);
          __threadfence();
          if (atomicAdd(sc.dist_cnt + r, 1) == per_r - 1) {
            __threadfence();
            float tot = 0.f;
            for (int i2 = 0; i2 < per_r; ++i2) tot += __ldcg(mine + i2);
            for (int i2 = 0; i2 < H / MLP_HEAD_COLS; ++i2) tot += __ldcg(sc.dist_head + (size_t)r * (H / MLP_HEAD_COLS) + i2);
            a.dist2[(size_t)r * a.cap + j] = tot;
          }
        }
        group_barrier(1 + grp, 128);     // dist_s may be overwritten by the next tile
      }
    }
    if (leader) bulk_wait_all();
  } else {
    // ---- w_j producer: the tile's blocks are consecutive 16 KB runs of the current version ----
    if (lane == 0) {
      auto tile_src = [&](int t) {
        const int r = tile_r(t), slab = (t / parts) % slabs, part = t % parts;
        return a.pool + ((size_t)r * a.n_slots + mlp_cur_slot(a, r, j)) * a.slot_stride +
               (((size_t)slab * (H >> 5) + ((part * Hn) >> 5)) << 12);
      };
      const int nb = Hn / 32;
      RingPos wp{0, 0u};
      for (int t = blockIdx.x; t < n_tiles && !failed; t += gridDim.x) {
        const float* src = tile_src(t);
        for (int b = 0; b < nb; ++b, wp.step(NB)) {
          const int s = wp.s;
          if (!mbar_wait(wempty(s), wp.ph ^ 1u)) { failed = true; break; }
          mbar_arrive_expect_tx(wfull(s), DW1_WBLOCK);
          bulk_g2s(base_addr + L.off_w + s * DW1_WBLOCK, src + (size_t)b * 4096, DW1_WBLOCK, wfull(s));
        }
      }
    }
    __syncwarp();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tc_dealloc(tmem_base, tmem_cols);
  if (failed && lane == 0) atomicExch(a.err, ERR_WAIT_TIMEOUT);
}

// ---- host: tensor maps ----------------------------------------------------------------------------
typedef CUresult (*PFN_encodeTiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                    const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline PFN_encodeTiled tc_encode_fn() {
  static PFN_encodeTiled fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess && qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<PFN_encodeTiled>(p);
  }
  return fn;
}

// 2-D bf16 tensor [rows][cols] (cols contiguous), box = box_cols x box_rows, 128-byte swizzle
inline bool tc_make_map(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_cols, uint32_t box_rows) {
  PFN_encodeTiled fn = tc_encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {box_cols, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct MlpMaps { CUtensorMap tmW, tmD; bool ready = false; };

inline bool mlp_make_maps(MlpScratch& s, MlpMaps& maps) {
  if (maps.ready) return true;
  const int n_halves = s.H > 256 ? 2 : 1;
  if (!tc_make_map(&maps.tmW, s.W1qT, (uint64_t)s.R * s.n_slots * (s.d / TC_BK) * s.H, (uint64_t)TC_BK, TC_BK, (uint32_t)(s.H / n_halves)) ||
      !tc_make_map(&maps.tmD, s.D1q, (uint64_t)s.R * s.Kmax * s.m, (uint64_t)s.H, 64, 64))
    return false;
  maps.ready = true;
  return true;
}

// sum of a replica's per-group loss sums, in fp64 and a fixed order (lane-strided, then a shuffle tree), over n samples
__global__ void mlp_eval_finish_kernel(const float* part, int R, int per_replica, long long n, float* out) {
  const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (r >= R) return;
  double s = 0.0;
  for (int i = lane; i < per_replica; i += 32) s += (double)part[(size_t)r * per_replica + i];
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
  if (lane == 0) out[r] = (float)(s / (double)n);
}

// Full-data risk of every replica's current version: the forward kernel over all rows of the data set, losses only.
inline cudaError_t run_mlp_eval(NumericArgs& a, MlpScratch& s, MlpMaps& maps, const uint8_t* cur_slot, int parity, float* part,
                                float* out, cudaStream_t stream, const char** why) {
  *why = nullptr;
  if (!mlp_make_maps(s, maps)) { *why = "mlp: could not encode the TMA tensor maps"; return cudaSuccess; }
  cudaError_t e;
  const TcLayout L = tc_forward_layout(s.H);
  if ((e = cudaFuncSetAttribute(mlp_risk_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L.total)) != cudaSuccess) return e;
  MlpArgs g{};
  g.na = a; g.sc = s; g.H = s.H; g.P = 0; g.j = 0;
  g.eval_blocks = (int)((s.n + 127) / 128); g.eval_slot = cur_slot; g.eval_parity = parity; g.eval_part = part;
  if ((long long)a.R * g.eval_blocks > 0x7FFFFFFFll) { *why = "mlp: replicas x 128-row blocks of the data set exceed the grid limit 2^31 - 1"; return cudaSuccess; }
  mlp_risk_tc_kernel<<<a.R * g.eval_blocks, TC_THREADS, L.total, stream>>>(maps.tmW, g);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  mlp_eval_finish_kernel<<<(a.R + 3) / 4, 128, 0, stream>>>(part, a.R, g.eval_blocks * 4, s.n, out);
  return cudaGetLastError();
}

inline cudaError_t run_mlp(NumericArgs& a, MlpScratch& s, MlpMaps& maps, int P, cudaStream_t stream, const char** why) {
  *why = nullptr;
  cudaError_t e;
  if (!mlp_make_maps(s, maps)) {
    *why = "mlp: could not encode the TMA tensor maps";
    return cudaSuccess;
  }
  const TcFwdLayout L = tc_fwd_layout(s.H);
  if ((e = cudaFuncSetAttribute(mlp_forward_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L.total)) != cudaSuccess) return e;
  const TcDw1Layout LD = tc_dw1_layout(s.H);
  if ((e = cudaFuncSetAttribute(mlp_dw1_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, LD.total)) != cudaSuccess) return e;
  int dev = 0, sms = 148;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  const int dw1_tiles = a.R * (s.d / 128) * (s.H / tc_dw1_cols(s.H));
  const int dw1_grid = dw1_tiles < sms ? dw1_tiles : sms;      // one persistent CTA per SM
  MlpArgs g{};
  g.na = a; g.sc = s; g.H = s.H; g.P = P;
  const int fwd_tiles = a.R * s.Kmax * (s.m / 128) * (s.H > 256 ? 2 : 1);
  const int fwd_grid = fwd_tiles < sms ? fwd_tiles : sms;
  for (long long u = 0; u < a.iters; ++u) {
    g.j = a.j0 + u;
    mlp_rows_kernel<<<a.R * s.Kmax, 128, 0, stream>>>(g);
    mlp_forward_tc_kernel<<<fwd_grid, TC_THREADS, L.total, stream>>>(maps.tmW, g);
    launch_mlp_head(g, stream);
    mlp_dw1_tc_kernel<<<dw1_grid, DW1_THREADS, LD.total, stream>>>(maps.tmD, g);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace ssim
