// Fused LM-head + verification: the large model's logits z = hidden x W^T are produced by a tcgen05 GEMM
// (bf16 operands staged by TMA into 128-byte-swizzled shared memory, fp32 accumulators in tensor memory)
// and consumed in the epilogue by the same per-row arithmetic as the logits path (Sec. 3.1-3.2 for one
// model pair), so the large model's logits never reach HBM.
//
// The Jensen-Shannon terms need the large model's normaliser before they can be formed, and 256 x V fp32
// logits fit nowhere on chip, so the GEMM runs twice:
//   sweep 1  per (row, 128-column tile): partial (max, sum-exp) of the large logits (from the accumulator)
//            and of the small logits (bf16, read from HBM);          -> lmhead_reduce_kernel -> per-row lse
//   sweep 2  per (row, tile): sum of divergence terms, sum max(p,q), residual mass, mass of p
//   final    per sequence: row totals, accept bits, accepted prefix, and the residual draw: the tile is found
//            from the per-tile residual masses, and only that tile's 128 logits of the rejected row are
//            recomputed (128 dot products) to place the token.
//
// One CTA = 10 warps: warp 0 lane 0 issues TMA loads, warp 1 lane 0 issues the MMAs (and owns the tensor
// memory allocation), warps 2..9 are the epilogue (warp e reads TMEM lanes 32*(e%4).. of accumulator
// e/4). Tile: M = 256 rows (two M=128 accumulators sharing one B tile) x N = 128 columns, K in steps of
// 64; 4-stage shared-memory ring; two accumulator buffers (512 TMEM columns) so that the epilogue of one
// tile overlaps the MMAs of the next. CTAs are persistent over the N tiles (tile = blockIdx.x + i*grid).
// Every mbarrier wait is bounded; on giving up a thread raises the status word and stops waiting.
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "rowstats_cluster.cuh"   // mbarrier wrappers, psi_poly, packed helpers

namespace psd {

constexpr int kLmM = 256;            // rows per CTA tile (the whole batch of positions)
constexpr int kLmN = 128;            // columns per tile
constexpr int kLmK = 64;             // K elements per stage (128 bytes of bf16: one swizzle row)
constexpr int kLmStages = 4;
constexpr int kLmABytes = kLmM * kLmK * 2;   // 32 KB
constexpr int kLmBBytes = kLmN * kLmK * 2;   // 16 KB
constexpr int kLmStageBytes = kLmABytes + kLmBBytes;
constexpr int kLmThreads = 320;
constexpr int kLmEpiWarps = 8;
constexpr size_t kLmSmemBytes = static_cast<size_t>(kLmStages) * kLmStageBytes + 1024 /*alignment*/ + 256 /*barriers*/;
constexpr unsigned kLmSpinLimit = 1u << 24;

struct LmParams {
  const __nv_bfloat16* small;     // [M, V] bf16 logits of the small model
  const int32_t* tokens;          // [M]
  int M, d, V, n_tiles;
  int row0;                       // first row of the 256-row block this launch works on
  float c;                        // log2(e) / T
  float2* part_large;             // sweep 1: [M][n_tiles] (max in scaled base-2 domain, sum)
  float2* part_small;
  float4* row_lse;                // [M] (m2_small, l2s_small, m2_large, l2s_large)
  float4* part_div;               // sweep 2: [M][n_tiles] (js bits, sum max(p,q), residual mass, mass of p)
  int* status;
  // KL(large || small) needs no second sweep for the divergence itself: sum_i p_i (log2 p_i - log2 q_i) =
  // (1 / S_l) sum_i P_i (z_i - x_i) c - (lse_l - lse_s) with P_i = 2^(z_i c - m), which sweep 1 accumulates per
  // tile next to (m, S_l), rescaled online like the sum.
  float* part_t;                  // KL, sweep 1: [M][n_tiles] sum of P_i (z_i - x_i) c against the tile's own max
  float* row_div;                 // KL: [M] the row's divergence in nats, written by the row reduction
  int* need_sweep2;               // KL: set by the accept scan when a residual mass is needed after all; sweep 2 leaves at once if 0
};

// ---- tcgen05 / TMA wrappers -----------------------------------------------------------------------------
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, int x, int y, unsigned long long* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(smem_u32(smem_dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tmem_alloc(unsigned* smem_result, unsigned ncols) {   // whole warp
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(unsigned taddr, unsigned ncols) {         // whole warp
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(unsigned long long* bar) {   // one thread
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 x bf16 -> fp32, one thread issues
__device__ __forceinline__ void tc_mma_bf16(unsigned tmem_d, unsigned long long desc_a, unsigned long long desc_b, unsigned idesc,
                                            unsigned accumulate) {
  asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
               ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld32(unsigned taddr, float (&v)[32]) {
  unsigned r[32];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
               "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
                 "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
                 "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
                 "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
               : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes, 128-byte swizzled:
// start address >> 4 in bits [0,14); leading byte offset (unused for swizzled K-major, 1) in [16,30);
// stride byte offset = 8 rows x 128 B = 1024 B >> 4 in [32,46); descriptor version 1 in [46,48);
// layout type SWIZZLE_128B = 2 in [61,64).
__device__ __forceinline__ unsigned long long umma_desc_k128(unsigned smem_addr) {
  unsigned long long d = 0;
  d |= static_cast<unsigned long long>((smem_addr >> 4) & 0x3fffu);
  d |= static_cast<unsigned long long>(1u) << 16;
  d |= static_cast<unsigned long long>(1024u >> 4) << 32;
  d |= static_cast<unsigned long long>(1u) << 46;
  d |= static_cast<unsigned long long>(2u) << 61;
  return d;
}
// Instruction descriptor: D fp32 (bits [4,6) = 1), A and B bf16 ([7,10) = 1, [10,13) = 1), both K-major
// ([15], [16] = 0), N >> 3 in [17,23), M >> 4 in [24,29).
__host__ __device__ constexpr unsigned umma_idesc_bf16(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<unsigned>(n >> 3) << 17) | (static_cast<unsigned>(m >> 4) << 24);
}

struct LmBarriers {
  unsigned long long full[kLmStages], empty[kLmStages], tmem_full[2], tmem_empty[2];
  unsigned tmem_base;
};

// ---- epilogues ------------------------------------------------------------------------------------------
// Sweep 1: online (max, sum) of one row over the tile's columns, in the scaled base-2 domain.
struct OnlineLse {
  float m, s;
  __device__ __forceinline__ void init() { m = -1e30f; s = 0.f; }
  template <int N>
  __device__ __forceinline__ void add(const float (&z)[N], float c, int n_valid) {
    float gm = -INFINITY;
#pragma unroll
    for (int i = 0; i < N; ++i) gm = fmaxf(gm, (i < n_valid) ? z[i] : -INFINITY);
    const float nm = fmaxf(m, fmaxf(gm * c, -1e30f));
    s *= ex2_approx(m - nm);
    m = nm;
    float t = 0.f;
#pragma unroll
    for (int i = 0; i < N; ++i) t += (i < n_valid) ? ex2_approx(fmaf(z[i], c, -m)) : 0.f;
    s += t;   // NaN and +inf logits poison s, as they should
  }
};

__device__ __forceinline__ void load_small32(const __nv_bfloat16* p, bool aligned, int n_valid, float (&x)[32]) {
  if (aligned && n_valid == 32) {
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      const uint4 u = __ldg(reinterpret_cast<const uint4*>(p) + v);
      Elem<__nv_bfloat16>::unpack(u, x + v * 8);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 32; ++i) x[i] = (i < n_valid) ? Elem<__nv_bfloat16>::load(p, i) : -INFINITY;
  }
}

// What one thread (= one row) leaves per 128-column tile.
struct LmTilePartial {
  float2 large, small;   // sweep 1: (max, sum) of both models
  float kl_t;            // sweep 1, KL: sum of P_i (z_i - x_i) c against `large.x`
  float4 div;            // sweep 2: (js bits, sum max(p,q), residual mass, mass of p)
};

// The epilogue of one 128-column tile for this thread's row: reads the accumulator from tensor memory 32
// columns at a time (all 32 lanes execute the loads, whatever row_ok says) and the small model's logits
// from global memory.
template <int SWEEP, bool KL = false>
__device__ __forceinline__ void lm_epilogue_tile(unsigned tacc, int n0, bool row_ok, const __nv_bfloat16* small_row, float c,
                                                 float off_l, float off_s, int V, LmTilePartial& out) {
  OnlineLse ol, os;
  ol.init(); os.init();
  float js = 0.f, big = 0.f, resid = 0.f, pmass = 0.f, kl_t = 0.f;
#pragma unroll 1
  for (int cb = 0; cb < kLmN / 32; ++cb) {
    float z[32], x[32];
    tmem_ld32(tacc + static_cast<unsigned>(cb * 32), z);
    const int col0 = n0 + cb * 32;
    const int nv = min(32, V - col0);   // columns of this group inside the vocabulary (<= 0: none)
    if (row_ok && nv > 0) {
      const __nv_bfloat16* sp = small_row + col0;
      load_small32(sp, (reinterpret_cast<uintptr_t>(sp) & 15u) == 0, nv, x);
      if (SWEEP == 1) {
        const float m_before = ol.m;
        ol.add<32>(z, c, nv);
        os.add<32>(x, c, nv);
        if (KL) {
          kl_t *= ex2_approx(m_before - ol.m);   // the group may have raised the tile's max
          float t = 0.f;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            if (i < nv) {
              const float e = ex2_approx(fmaf(z[i], c, -ol.m));
              if (e > 0.f) t = fmaf(e, (z[i] - x[i]) * c, t);   // q_i = 0 under p_i > 0 gives +inf, as it should
            }
          }
          kl_t += t;
        }
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          if (i < nv) {
            const float a = fmaxf(fmaf(z[i], c, -off_l), -125.f), b = fmaxf(fmaf(x[i], c, -off_s), -125.f);   // log2 p, log2 q
            const float E = ex2_approx(fmaxf(a, b));
            const float dd = a - b;
            const float u = ex2_approx(-fabsf(dd));
            const float2 ps = psi_poly<7>(make_float2(u, u));
            js = fmaf(E, fmaf(u, -fabsf(dd), ps.x), js);
            big += E;
            const float lo = E * u;                       // min(p, q)
            resid += (dd > 0.f) ? E - lo : 0.f;           // max(0, p - q)
            pmass += (dd >= 0.f) ? E : lo;                // p
          }
        }
      }
    }
  }
  out.large = make_float2(ol.m, ol.s);
  out.small = make_float2(os.m, os.s);
  out.kl_t = kl_t;
  out.div = make_float4(js, big, resid, pmass);
}

template <int SWEEP, bool KL = false>
__device__ __forceinline__ void lm_store_partial(const LmParams& P, size_t idx, const LmTilePartial& part) {
  if (SWEEP == 1) {
    P.part_large[idx] = part.large;
    P.part_small[idx] = part.small;
    if (KL) P.part_t[idx] = part.kl_t;
  } else {
    P.part_div[idx] = part.div;
  }
}

template <int SWEEP, bool KL = false>
__global__ void __launch_bounds__(kLmThreads, 1)
lmhead_sweep_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const LmParams P) {
  extern __shared__ unsigned char lm_smem_raw[];
  // KL: the second sweep only serves residual masses; when the accept scan found no use for them every CTA leaves
  // here, before it has set up anything (the flag was written by an earlier kernel: the same answer for all)
  if (SWEEP == 2 && P.need_sweep2 != nullptr && *reinterpret_cast<volatile const int*>(P.need_sweep2) == 0) return;
  unsigned char* tiles = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(lm_smem_raw) + 1023) & ~uintptr_t(1023));
  LmBarriers* bars = reinterpret_cast<LmBarriers*>(tiles + static_cast<size_t>(kLmStages) * kLmStageBytes);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int k_steps = P.d / kLmK;

  if (tid == 0) {
    for (int s = 0; s < kLmStages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&bars->tmem_full[b], 1); mbar_init(&bars->tmem_empty[b], kLmEpiWarps); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(&bars->tmem_base, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const unsigned tmem_base = bars->tmem_base;

  bool dead = false;
  auto wait_phase = [&](unsigned long long* bar, unsigned parity) {
    if (mbar_test(bar, parity)) return;
    unsigned spins = 0;
    while (!dead && !mbar_try(bar, parity))
      if (++spins > kLmSpinLimit) { dead = true; atomicExch(P.status, 1); }
  };

  if (warp == 0) {
    // ================================ TMA producer ================================
    if (lane == 0) {
      unsigned stage = 0, fills = 0;
      for (int tile = blockIdx.x; tile < P.n_tiles && !dead; tile += gridDim.x) {
        for (int ks = 0; ks < k_steps; ++ks) {
          if (fills > 0) wait_phase(&bars->empty[stage], (fills - 1u) & 1u);
          if (dead) break;   // the stage never came back: nothing more is copied into this ring
          unsigned char* sa = tiles + static_cast<size_t>(stage) * kLmStageBytes;
          mbar_arrive_expect_tx(&bars->full[stage], kLmStageBytes);
          tma_load_2d(sa, &map_a, ks * kLmK, P.row0, &bars->full[stage]);                 // 256 hidden rows of the block
          tma_load_2d(sa + kLmABytes, &map_b, ks * kLmK, tile * kLmN, &bars->full[stage]);  // W^T rows tile*128..
          if (++stage == kLmStages) { stage = 0; ++fills; }
        }
      }
      // When a wait gave up somewhere in the CTA the consumers no longer wait for the copies issued above: this
      // thread sees each of them land (bounded) before the shared memory goes away.
      if (dead || *reinterpret_cast<volatile int*>(P.status) != 0) {
        for (unsigned s = 0; s < static_cast<unsigned>(kLmStages); ++s) {
          const unsigned turns = fills + (s < stage ? 1u : 0u);
          if (turns == 0) continue;
          unsigned spins = 0;
          while (!mbar_try(&bars->full[s], (turns - 1u) & 1u) && ++spins <= kLmSpinLimit) {}
        }
      }
    }
  } else if (warp == 1) {
    // ================================ MMA issuer ================================
    if (lane == 0) {
      constexpr unsigned idesc = umma_idesc_bf16(128, kLmN);
      unsigned stage = 0, par = 0;
      int it = 0;
      for (int tile = blockIdx.x; tile < P.n_tiles; tile += gridDim.x, ++it) {
        const int buf = it & 1;
        if (it >= 2) wait_phase(&bars->tmem_empty[buf], ((it >> 1) - 1) & 1u);   // the epilogue has drained this buffer
        if (dead) break;
        tc_fence_after();
        const unsigned acc0 = tmem_base + static_cast<unsigned>(buf) * 256u, acc1 = acc0 + 128u;
        for (int ks = 0; ks < k_steps; ++ks) {
          wait_phase(&bars->full[stage], par);
          if (dead) break;   // no MMA on operands that have not arrived
          tc_fence_after();
          const unsigned sa = smem_u32(tiles + static_cast<size_t>(stage) * kLmStageBytes);
          const unsigned long long da0 = umma_desc_k128(sa), da1 = umma_desc_k128(sa + 128 * 128), db = umma_desc_k128(sa + kLmABytes);
#pragma unroll
          for (int kk = 0; kk < kLmK / 16; ++kk) {
            // 16 bf16 = 32 bytes further along K inside the swizzled row: +2 in the descriptor's 16-byte units
            const unsigned acc = (ks | kk) != 0 ? 1u : 0u;
            tc_mma_bf16(acc0, da0 + 2ull * kk, db + 2ull * kk, idesc, acc);
            tc_mma_bf16(acc1, da1 + 2ull * kk, db + 2ull * kk, idesc, acc);
          }
          tc_commit(&bars->empty[stage]);   // arrives when the MMAs that read this stage have completed
          if (++stage == kLmStages) { stage = 0; par ^= 1u; }
        }
        if (dead) break;
        tc_commit(&bars->tmem_full[buf]);   // the accumulators of this tile are complete
      }
    }
  } else {
    // ================================ epilogue ================================
    // a warp reads the TMEM lanes 32 * (its index in the CTA mod 4) ..; warps 2..5 take accumulator 0, 6..9 accumulator 1
    const int quarter = warp & 3, half = (warp - 2) >> 2;
    const int row = P.row0 + half * 128 + quarter * 32 + lane;   // this thread's row (TMEM lane + 128*half of the block)
    const bool row_ok = row < P.M;
    const float c = P.c;
    const __nv_bfloat16* small_row = P.small + static_cast<size_t>(row_ok ? row : 0) * P.V;
    float4 lse = make_float4(0.f, 0.f, 0.f, 0.f);
    if (SWEEP == 2 && row_ok) lse = P.row_lse[row];
    const float off_s = lse.x + lse.y, off_l = lse.z + lse.w;
    int it = 0;
    for (int tile = blockIdx.x; tile < P.n_tiles; tile += gridDim.x, ++it) {
      const int buf = it & 1;
      wait_phase(&bars->tmem_full[buf], (it >> 1) & 1u);
      tc_fence_after();
      const unsigned tacc = tmem_base + static_cast<unsigned>(buf) * 256u + static_cast<unsigned>(half) * 128u +
                            (static_cast<unsigned>(quarter * 32) << 16);
      const int n0 = tile * kLmN;
      LmTilePartial part;
      lm_epilogue_tile<SWEEP, KL>(tacc, n0, row_ok, small_row, c, off_l, off_s, P.V, part);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->tmem_empty[buf]);   // this warp has read its part of the accumulator
      if (row_ok) lm_store_partial<SWEEP, KL>(P, static_cast<size_t>(row) * P.n_tiles + tile, part);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// ---- two-SM variant -------------------------------------------------------------------------------------
// A pair of CTAs (cluster of 2) shares one 256 x 256 tile: tcgen05.mma.cta_group::2 with M = 256 takes rows
// 0..127 of A from the even CTA's shared memory and rows 128..255 from the odd one's, and the two halves of
// the 256 B rows likewise; each CTA keeps its 128 rows of the fp32 accumulator in its own tensor memory
// (256 columns, two buffers). Per K step a CTA stages 16 KB of A and 16 KB of B (six stages), so the hidden
// matrix crosses L2 -> SM once per 256 columns instead of once per 128, and the ring holds 1.5x the K steps.
// The even CTA issues the MMAs; both CTAs' TMA loads count their bytes on the even CTA's "full" barrier,
// tcgen05.commit (multicast to both CTAs) frees the stages and publishes the accumulators, and the odd CTA's
// epilogue warps arrive remotely on the even CTA's "accumulator drained" barrier.
constexpr int kLm2N = 256;
constexpr int kLm2Stages = 6;
constexpr int kLm2HalfBytes = 128 * kLmK * 2;              // 16 KB: 128 rows x 64 bf16
constexpr int kLm2StageBytes = 2 * kLm2HalfBytes;          // A half + B half
constexpr size_t kLm2SmemBytes = static_cast<size_t>(kLm2Stages) * kLm2StageBytes + 1024 + 256;

struct Lm2Barriers {
  unsigned long long full[kLm2Stages], empty[kLm2Stages], tmem_full[2], tmem_empty[2];
  unsigned tmem_base;
};

__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const CUtensorMap* map, int x, int y, unsigned long long* bar) {
  // the barrier address with the peer bit cleared names the even CTA's barrier at the same offset
  asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(smem_u32(smem_dst)), "l"(map), "r"(smem_u32(bar) & 0xFEFFFFFFu), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(unsigned* smem_result, unsigned ncols) {   // same warp index in both CTAs
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(unsigned taddr, unsigned ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_commit_pair(unsigned long long* bar) {   // arrives on this barrier in both CTAs
  const unsigned short mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(smem_u32(bar)), "h"(mask) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(unsigned tmem_d, unsigned long long desc_a, unsigned long long desc_b, unsigned idesc,
                                                 unsigned accumulate) {
  const unsigned z = 0;
  asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
               " tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n}"
               ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(z) : "memory");
}
__device__ __forceinline__ void mbar_arrive_remote_release(unsigned cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

template <int SWEEP, bool KL = false>
__global__ void __launch_bounds__(kLmThreads, 1)
lmhead_sweep2sm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const LmParams P) {
  extern __shared__ unsigned char lm_smem_raw[];
  if (SWEEP == 2 && P.need_sweep2 != nullptr && *reinterpret_cast<volatile const int*>(P.need_sweep2) == 0) return;   // as in the one-SM kernel
  unsigned char* tiles = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(lm_smem_raw) + 1023) & ~uintptr_t(1023));
  Lm2Barriers* bars = reinterpret_cast<Lm2Barriers*>(tiles + static_cast<size_t>(kLm2Stages) * kLm2StageBytes);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const unsigned rank = cluster_rank();          // 0: issues the MMAs; 1: its peer
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int k_steps = P.d / kLmK;
  const int n_tiles2 = (P.n_tiles + 1) / 2;      // 256-column tiles

  if (tid == 0) {
    for (int s = 0; s < kLm2Stages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&bars->tmem_full[b], 1); mbar_init(&bars->tmem_empty[b], 2 * kLmEpiWarps); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc_pair(&bars->tmem_base, 512);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();        // both CTAs' barriers and allocations exist before either signals the other
  tc_fence_after();
  const unsigned tmem_base = bars->tmem_base;

  bool dead = false;
  auto wait_phase = [&](unsigned long long* bar, unsigned parity) {
    if (mbar_test(bar, parity)) return;
    unsigned spins = 0;
    while (!dead && !mbar_try(bar, parity))
      if (++spins > kLmSpinLimit) { dead = true; atomicExch(P.status, 1); }
  };

  if (warp == 0) {
    // ================================ TMA producer (both CTAs) ================================
    if (lane == 0) {
      unsigned stage = 0, fills = 0;
      for (int tile = pair; tile < n_tiles2 && !dead; tile += n_pairs) {
        for (int ks = 0; ks < k_steps; ++ks) {
          if (fills > 0) wait_phase(&bars->empty[stage], (fills - 1u) & 1u);
          if (dead) break;   // the stage never came back: nothing more is copied into this ring
          unsigned char* sa = tiles + static_cast<size_t>(stage) * kLm2StageBytes;
          // the even CTA's barrier counts the bytes of both CTAs
          if (rank == 0) mbar_arrive_expect_tx(&bars->full[stage], 2u * kLm2StageBytes);
          tma_load_2d_pair(sa, &map_a, ks * kLmK, P.row0 + static_cast<int>(rank) * 128, &bars->full[stage]);
          tma_load_2d_pair(sa + kLm2HalfBytes, &map_b, ks * kLmK, tile * kLm2N + static_cast<int>(rank) * 128, &bars->full[stage]);
          if (++stage == kLm2Stages) { stage = 0; ++fills; }
        }
      }
      // After a wait gave up, the even CTA (whose barriers count both CTAs' bytes) sees every copy issued so far
      // land, bounded, before it enters the final cluster barrier that keeps both CTAs' shared memory alive.
      if (rank == 0 && (dead || *reinterpret_cast<volatile int*>(P.status) != 0)) {
        for (unsigned s = 0; s < static_cast<unsigned>(kLm2Stages); ++s) {
          const unsigned turns = fills + (s < stage ? 1u : 0u);
          if (turns == 0) continue;
          unsigned spins = 0;
          while (!mbar_try(&bars->full[s], (turns - 1u) & 1u) && ++spins <= kLmSpinLimit) {}
        }
      }
    }
  } else if (warp == 1) {
    // ================================ MMA issuer (even CTA only) ================================
    if (lane == 0 && rank == 0) {
      constexpr unsigned idesc = umma_idesc_bf16(256, kLm2N);
      unsigned stage = 0, par = 0;
      int it = 0;
      for (int tile = pair; tile < n_tiles2; tile += n_pairs, ++it) {
        const int buf = it & 1;
        if (it >= 2) wait_phase(&bars->tmem_empty[buf], ((it >> 1) - 1) & 1u);   // both CTAs' epilogues have drained this buffer
        if (dead) break;
        tc_fence_after();
        const unsigned acc = tmem_base + static_cast<unsigned>(buf) * 256u;
        for (int ks = 0; ks < k_steps; ++ks) {
          wait_phase(&bars->full[stage], par);
          if (dead) break;   // no MMA on operands that have not arrived
          tc_fence_after();
          const unsigned sa = smem_u32(tiles + static_cast<size_t>(stage) * kLm2StageBytes);
          const unsigned long long da = umma_desc_k128(sa), db = umma_desc_k128(sa + kLm2HalfBytes);
#pragma unroll
          for (int kk = 0; kk < kLmK / 16; ++kk)
            tc_mma_bf16_pair(acc, da + 2ull * kk, db + 2ull * kk, idesc, (ks | kk) != 0 ? 1u : 0u);
          tc_commit_pair(&bars->empty[stage]);   // frees the stage in both CTAs once these MMAs have read it
          if (++stage == kLm2Stages) { stage = 0; par ^= 1u; }
        }
        if (dead) break;
        tc_commit_pair(&bars->tmem_full[buf]);   // the accumulators of this tile are complete, in both CTAs
      }
    }
  } else {
    // ================================ epilogue (both CTAs) ================================
    const int quarter = warp & 3, half = (warp - 2) >> 2;          // TMEM lanes 32*quarter.., columns 128*half..
    const int row = P.row0 + static_cast<int>(rank) * 128 + quarter * 32 + lane;
    const bool row_ok = row < P.M;
    const float c = P.c;
    const __nv_bfloat16* small_row = P.small + static_cast<size_t>(row_ok ? row : 0) * P.V;
    float4 lse = make_float4(0.f, 0.f, 0.f, 0.f);
    if (SWEEP == 2 && row_ok) lse = P.row_lse[row];
    const float off_s = lse.x + lse.y, off_l = lse.z + lse.w;
    const unsigned drained = map_to_rank(&bars->tmem_empty[0], 0);   // the even CTA's barriers
    int it = 0;
    for (int tile = pair; tile < n_tiles2; tile += n_pairs, ++it) {
      const int buf = it & 1;
      wait_phase(&bars->tmem_full[buf], (it >> 1) & 1u);
      tc_fence_after();
      const unsigned tacc = tmem_base + static_cast<unsigned>(buf) * 256u + static_cast<unsigned>(half) * 128u +
                            (static_cast<unsigned>(quarter * 32) << 16);
      const int tile128 = tile * 2 + half;
      LmTilePartial part;
      lm_epilogue_tile<SWEEP, KL>(tacc, tile128 * kLmN, row_ok, small_row, c, off_l, off_s, P.V, part);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_remote_release(drained + static_cast<unsigned>(buf) * 8u);
      if (row_ok && tile128 < P.n_tiles) lm_store_partial<SWEEP, KL>(P, static_cast<size_t>(row) * P.n_tiles + tile128, part);
    }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();        // nobody frees tensor memory or leaves while the peer can still touch it
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, 512);
  }
}

// Per row: combine the tiles' (max, sum) partials into the row's log-sum-exp (base 2), both models; with the KL
// partials also the row's divergence KL(large || small) = ln 2 * (T / S_l - (lse_l - lse_s)), T rescaled to the
// row's max like S_l.
__global__ void __launch_bounds__(256) lmhead_reduce_kernel(const LmParams P) {
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= P.M) return;
  const bool kl = P.part_t != nullptr;
  float ml = -1e30f, sl = 0.f, ms = -1e30f, ss = 0.f;
  for (int t = lane; t < P.n_tiles; t += 32) {
    const float2 a = P.part_large[static_cast<size_t>(row) * P.n_tiles + t], b = P.part_small[static_cast<size_t>(row) * P.n_tiles + t];
    lse_merge(ml, sl, a.x, a.y);
    lse_merge(ms, ss, b.x, b.y);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    lse_merge(ml, sl, __shfl_xor_sync(0xffffffffu, ml, o), __shfl_xor_sync(0xffffffffu, sl, o));
    lse_merge(ms, ss, __shfl_xor_sync(0xffffffffu, ms, o), __shfl_xor_sync(0xffffffffu, ss, o));
  }
  const float l2sl = lg2_approx(sl), l2ss = lg2_approx(ss);
  if (lane == 0) P.row_lse[row] = make_float4(ms, l2ss, ml, l2sl);
  if (kl) {
    float tt = 0.f;   // sum over the tiles of T_t * 2^(m_t - ml): ml is the row's max after the merge above
    for (int t = lane; t < P.n_tiles; t += 32) {
      const float tv = P.part_t[static_cast<size_t>(row) * P.n_tiles + t];
      const float f = ex2_approx(P.part_large[static_cast<size_t>(row) * P.n_tiles + t].x - ml);
      if (f > 0.f) tt = fmaf(tv, f, tt);   // a tile without mass contributes nothing (0 * inf otherwise)
    }
    tt = warp_reduce<OpSum>(tt);
    if (lane == 0) P.row_div[row] = fmaxf(kLn2 * (__fdiv_rn(tt, sl) - ((ml + l2sl) - (ms + l2ss))), 0.f);
  }
}

// ---- final kernel: one CTA per sequence ------------------------------------------------------------------
struct LmFinalParams {
  LmParams lm;
  const __nv_bfloat16* hidden;   // [M, d]
  const __nv_bfloat16* w_t;      // [V, d]
  int B, K;
  float threshold;
  int mode;
  unsigned long long seed, offset;
  long long seq_base;   // index of sequence 0 in the whole batch (Philox row counter)
  int32_t* out_accept_len;
  int32_t* out_next_token;
  float* out_div;        // [B, K] or null
  float* out_resid;      // [B, K] or null
  // KL: 0 = the usual pass over the second sweep's partials. 1 = accept scan only, before the second sweep: raises
  // lm.need_sweep2 when some rejected row needs residual masses. 2 = full pass after a second sweep that may not
  // have run (then every draw comes from p_large, whose tile masses the first sweep left).
  int kl_phase;
};

// dot(hidden[row], w_t[col]) by one warp, fp32 accumulation in index order per lane then a shuffle tree
__device__ __forceinline__ float lm_dot(const __nv_bfloat16* h, const __nv_bfloat16* w, int d, int lane) {
  float acc = 0.f;
  for (int j = lane * 8; j < d; j += 256) {
    float a[8], b[8];
    Elem<__nv_bfloat16>::unpack(__ldg(reinterpret_cast<const uint4*>(h + j)), a);
    Elem<__nv_bfloat16>::unpack(__ldg(reinterpret_cast<const uint4*>(w + j)), b);
#pragma unroll
    for (int i = 0; i < 8; ++i) acc = fmaf(a[i], b[i], acc);
  }
  return warp_reduce<OpSum>(acc);
}

__global__ void __launch_bounds__(256) lmhead_final_kernel(const LmFinalParams F) {
  __shared__ float sh_div[32], sh_res[32], sh_px[32], sh_qx[32], sh_pm[32];
  __shared__ int sh_flag[32];
  __shared__ float sh_w[kLmN];
  __shared__ double sh_seg[256];
  __shared__ int sh_L, sh_tile, sh_token;
  __shared__ float sh_target, sh_u2;
  const LmParams& P = F.lm;
  const int b = blockIdx.x, K = F.K, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nwarps = blockDim.x >> 5;
  const float c = P.c;

  // per row: totals over the tiles, and the probabilities of the row's token
  for (int k = warp; k < K; k += nwarps) {
    const int r = b * K + k;
    double js = 0.0, big = 0.0, res = 0.0, pm = 0.0;
    // KL: the divergence comes from the row reduction; the second sweep's partials exist only if it ran
    const bool have2 = F.kl_phase == 0 || (F.kl_phase == 2 && *reinterpret_cast<volatile const int*>(P.need_sweep2) != 0);
    if (have2) {
      for (int t = lane; t < P.n_tiles; t += 32) {
        const float4 v = P.part_div[static_cast<size_t>(r) * P.n_tiles + t];
        js += v.x; big += v.y; res += v.z; pm += v.w;
      }
    }
    js = warp_reduce<OpSum>(js); res = warp_reduce<OpSum>(res); pm = warp_reduce<OpSum>(pm);
    const float4 lse = P.row_lse[r];
    const int x = P.tokens[r];
    (void)big;
    int flags = 0;
    if (!(fabsf(lse.x + lse.y) < INFINITY)) flags |= kFlagSmallNonfinite;
    if (!(fabsf(lse.z + lse.w) < INFINITY)) flags |= kFlagLargeNonfinite;
    if (x < 0 || x >= P.V) flags |= kFlagTokenRange;
    float px = 0.f, qx = 0.f;
    if (!flags) {
      const float zx = lm_dot(F.hidden + static_cast<size_t>(r) * P.d, F.w_t + static_cast<size_t>(x) * P.d, P.d, lane);
      px = ex2_approx(fmaf(zx, c, -lse.z) - lse.w);
      qx = ex2_approx(fmaf(Elem<__nv_bfloat16>::load(P.small + static_cast<size_t>(r) * P.V, x), c, -lse.x) - lse.y);
    }
    if (lane == 0) {
      sh_div[k] = F.kl_phase != 0 ? P.row_div[r] : fmaxf(static_cast<float>(0.5 * 0.6931471805599453 * js), 0.f);
      sh_res[k] = have2 ? fmaxf(static_cast<float>(res), 0.f) : __int_as_float(0x7fc00000);
      sh_pm[k] = static_cast<float>(pm);
      sh_px[k] = px; sh_qx[k] = qx; sh_flag[k] = flags;
      const bool no_dist = (flags & (kFlagSmallNonfinite | kFlagLargeNonfinite)) != 0;   // a bad token leaves D and R intact
      if (F.kl_phase != 1) {
        if (F.out_div) F.out_div[r] = no_dist ? __int_as_float(0x7fc00000) : sh_div[k];
        if (F.out_resid) F.out_resid[r] = no_dist ? __int_as_float(0x7fc00000) : sh_res[k];
      }
    }
  }
  __syncthreads();
  // accept bits and prefix: lane k of warp 0 owns position k
  float u2 = 0.f;
  if (warp == 0) {
    bool acc = true;
    float u = 0.f, uu2 = 0.f;
    if (lane < K) {
      row_uniforms(F.seed, F.offset, static_cast<unsigned>((F.seq_base + b) * K + lane), &u, &uu2);
      const float px = sh_px[lane], qx = sh_qx[lane];
      const float rho = (qx > 0.f) ? __fdiv_rn(px, qx) : (px > 0.f ? INFINITY : 0.f);
      const bool coin_ok = u < fminf(1.f, rho);
      const bool fuzzy_ok = sh_div[lane] <= F.threshold;
      if (F.mode == kModeFuzzy) acc = fuzzy_ok;
      else if (F.mode == kModeStrict || F.mode == kModeAssisted) acc = coin_ok;
      else acc = fuzzy_ok || coin_ok;
      if (sh_flag[lane]) acc = false;
    }
    const unsigned rejected = ~__ballot_sync(0xffffffffu, acc);
    const int L = rejected ? (__ffs(rejected) - 1) : K;
    const float u2L = __shfl_sync(0xffffffffu, uu2, min(L, 31));
    if (lane == 0) { sh_L = L; sh_u2 = u2L; }
  }
  __syncthreads();
  const int L = sh_L;
  u2 = sh_u2;
  if (F.kl_phase == 1) {
    // scan only: a rejected row with a distribution draws from the residual unless the mode is the assisted one
    if (tid == 0 && L < K && !(sh_flag[L] & (kFlagSmallNonfinite | kFlagLargeNonfinite)) && F.mode != kModeAssisted)
      atomicExch(P.need_sweep2, 1);
    return;
  }
  const bool have2 = F.kl_phase == 0 || *reinterpret_cast<volatile const int*>(P.need_sweep2) != 0;
  int next = -1;
  if (L < K) {
    if (sh_flag[L] & (kFlagSmallNonfinite | kFlagLargeNonfinite)) {
      next = -2;
    } else {
      const int r = b * K + L;
      const bool from_large = (F.mode == kModeAssisted) || !have2 || !(sh_res[L] > 0.f);
      const float4 lse_r = P.row_lse[r];
      // weight of tile t: the second sweep's residual mass or mass of p; without a second sweep the mass of p from
      // the first sweep's (max, sum) of the tile
      auto tile_weight = [&](int t) -> double {
        if (have2) {
          const float4 v = P.part_div[static_cast<size_t>(r) * P.n_tiles + t];
          return from_large ? v.w : v.z;
        }
        const float2 a = P.part_large[static_cast<size_t>(r) * P.n_tiles + t];
        return static_cast<double>(a.y) * static_cast<double>(ex2_approx((a.x - lse_r.z) - lse_r.w));
      };
      // the tile that holds the target mass: first tile whose inclusive cumulative weight exceeds it. Two levels:
      // every thread sums a run of consecutive tiles, one thread walks the 256 run sums and then the chosen run.
      const int per = (P.n_tiles + static_cast<int>(blockDim.x) - 1) / static_cast<int>(blockDim.x);
      {
        double run = 0.0;
        const int t0 = tid * per, t1 = min(P.n_tiles, t0 + per);
        for (int t = t0; t < t1; ++t) run += tile_weight(t);
        sh_seg[tid] = run;
      }
      __syncthreads();
      if (tid == 0) {
        double total = 0.0;
        for (int g = 0; g < static_cast<int>(blockDim.x); ++g) total += sh_seg[g];
        const double target = static_cast<double>(u2) * total;
        int seg = -1, last_seg = -1;
        double cum = 0.0, before_seg = 0.0, before_last_seg = 0.0;
        for (int g = 0; g < static_cast<int>(blockDim.x); ++g) {
          const double wgt = sh_seg[g];
          if (wgt > 0.0) { last_seg = g; before_last_seg = cum; }
          if (seg < 0 && cum + wgt > target && wgt > 0.0) { seg = g; before_seg = cum; }
          cum += wgt;
        }
        if (seg < 0) { seg = last_seg; before_seg = before_last_seg; }
        int pick = -1, last_pos = -1;
        double before_pick = 0.0, before_last = 0.0;
        if (seg >= 0) {
          cum = before_seg;
          for (int t = seg * per; t < min(P.n_tiles, (seg + 1) * per); ++t) {
            const double wgt = tile_weight(t);
            if (wgt > 0.0) { last_pos = t; before_last = cum; }
            if (pick < 0 && cum + wgt > target && wgt > 0.0) { pick = t; before_pick = cum; }
            cum += wgt;
          }
          if (pick < 0) { pick = last_pos; before_pick = before_last; }
        }
        sh_tile = pick;
        sh_target = static_cast<float>(target - before_pick);
        sh_token = -1;
      }
      __syncthreads();
      const int tile = sh_tile;
      if (tile >= 0) {
        // recompute the rejected row's logits of that tile only, and the weights from them
        const float4 lse = P.row_lse[r];
        for (int j = warp; j < kLmN; j += nwarps) {
          const int col = tile * kLmN + j;
          float w = 0.f;
          if (col < P.V) {
            const float z = lm_dot(F.hidden + static_cast<size_t>(r) * P.d, F.w_t + static_cast<size_t>(col) * P.d, P.d, lane);
            const float p = ex2_approx(fmaf(z, c, -lse.z) - lse.w);
            const float q = ex2_approx(fmaf(Elem<__nv_bfloat16>::load(P.small + static_cast<size_t>(r) * P.V, col), c, -lse.x) - lse.y);
            w = from_large ? p : fmaxf(p - q, 0.f);
          }
          if (lane == 0) sh_w[j] = w;
        }
        __syncthreads();
        if (tid == 0) {
          const float t3 = sh_target;
          float run = 0.f;
          int choice = -1, last_pos = -1;
          for (int j = 0; j < kLmN; ++j) {
            run += sh_w[j];
            if (sh_w[j] > 0.f) {
              last_pos = j;
              if (choice < 0 && run > t3) choice = j;
            }
          }
          if (choice < 0) choice = last_pos;
          sh_token = (choice >= 0) ? tile * kLmN + choice : -1;
        }
        __syncthreads();
        next = sh_token;
      }
    }
  }
  if (tid == 0) {
    F.out_accept_len[b] = L;
    F.out_next_token[b] = next;
  }
}

}  // namespace psd
