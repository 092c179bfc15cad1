// Cluster row-statistics kernel: the HBM-streaming hot loop of one verification stage (Sec. 3.1-3.2).
//
// One thread-block cluster owns one (sequence, position) row pair at a time; CTA `rank` of the cluster
// owns the vocabulary slice [rank*SL, (rank+1)*SL). Every CTA is persistent and walks a static list of
// rows. The slice of both models' logits is brought into a shared-memory ring by 1-D bulk copies
// (cp.async.bulk + mbarrier complete_tx) exactly once, and is read twice from there:
//   pass A  per-thread streaming log-sum-exp of both models (one ex2 per logit);
//   pass B  with the row's normalisers known: p, q, the Jensen-Shannon terms and the residual mass.
// Pass B of a row needs the normalisers of the WHOLE row, so the CTAs of a cluster exchange their
// (reference, sum) partials through distributed shared memory. Nothing waits on that exchange in line:
// the ring holds more than one row slice, the pass-A warps run ahead of the pass-B warps for as long as
// loaded chunks are available, and an agent warp carries partials between CTAs. Warps are independent
// of each other; they meet only on mbarriers (chunk landed / chunk free / row partials complete), and
// every one of those waits is a blocking mbarrier wait on a single condition.
//
// Roles: warps 0..7 run pass A, warps 8..15 run pass B (each warp owns 2 x 32 16-byte vectors of every
// chunk and model; the hardware scheduler interleaves the two instruction streams on each SM
// sub-partition), warp 16 lane 0 issues the bulk copies, warps 17 and 18 are the agents (they reduce the
// warps' partials and talk to the peers; on rank 0 the second one also writes the row's RowStats). Every
// wait is bounded: on giving up a thread records PSD_ERR_TIMEOUT in the status word and stops waiting, so
// the kernel always terminates.
//
// Streamed-twice variant (template flag RS). Clusters of one or two CTAs are the only ones that fill every
// SM, but for a large vocabulary their slice does not fit the ring. There the slice is copied in twice:
// part of the ring feeds pass A and is handed back by pass A, the rest feeds pass B, which runs one row
// behind and gets its copy out of L2; a second loader thread (warp 19) serves pass B's ring. The
// arithmetic and its order are those of the resident variant.
//
// Three-row form of the streamed-twice variant (template flag TRI), for the two-stage wrapper. Stage 2 of the
// pyramid scores the window with the qualifier's distribution in the draft's place (Fig. 1), so for a position
// k < K_q the qualifier row is the large model of the stage-1 pair and the small model of the stage-2 pair. A
// TRI launch walks one work item per stage-1 row: positions k < K_q are row triples (draft, qualifier, target)
// -- three log-sum-exps in pass A, the two pairs' divergence terms in pass B, the qualifier row read, widened
// and normalised once -- and positions k >= K_q are ordinary pairs. A triple moves one chunk of three rows per
// ring slot, a pair two chunks of two rows; each model's sums and each pair's terms are taken in the order of
// the two-row form, so both forms return the same bits.
#pragma once

#include <type_traits>

#include "common.cuh"

namespace psd {

constexpr int kClAWarps = 8;                       // warps running pass A (0 .. kClAWarps - 1)
constexpr int kClBWarps = 8;                       // warps running pass B (the next kClBWarps)
constexpr int kClConsumerWarps = kClAWarps + kClBWarps;
constexpr int kClConsumers = kClConsumerWarps * 32;
constexpr int kClThreads = kClConsumers + 96;      // + loader warp + two agent warps
constexpr int kClSubRS = 2;                        // chunks per slot of the streamed-twice variant (measured: 2 beats 1, 3 and 4)
constexpr int kClThreadsRS = kClThreads + 32;      // the streamed-twice variant has a loader warp per pass
constexpr int kClHalfBytes = 8192;                 // one model's part of a chunk: 256 threads x 2 x 16 bytes
constexpr int kClAVec = 16 / kClAWarps;            // 16-byte vectors per lane, chunk and model in pass A
constexpr int kClBVec = 16 / kClBWarps;            // ... and in pass B
static_assert(kClAVec * kClAWarps == 16 && kClBVec * kClBWarps == 16, "the 512 vectors of a chunk must split evenly");
constexpr int kClSlotBytes = 2 * kClHalfBytes;
constexpr int kClSlots = 13;                       // ring slots
constexpr int kClDepth = 4;                        // rows of exchange buffers in flight
constexpr int kClMaxRanks = 16;
// Registers per thread by role in the streamed-twice variant (640 threads start with 96 each). Its five groups of
// four warps trade registers at the role split (setmaxnreg): the pass-A warps and the loader / agent warps give
// some up, the pass-B warps, whose inner loop holds two vectors of three models in flight, take them.
// 8 x 32 x 80 + 8 x 32 x 128 + 4 x 32 x 56 = 60416 <= 640 x 96. Measured against 96 everywhere: config 4's
// statistics launch 0.558 -> 0.539 ms, config 3 unchanged; 72 / 136 / 56 and 64 / 136 / 64 spill in pass A.
constexpr int kClRegsA = 80, kClRegsB = 128, kClRegsService = 56;
static_assert(kClThreadsRS == 640 && kClAWarps == 8 && kClBWarps == 8, "the register split above is for 8 + 8 + 4 warps");
constexpr int kClLag = 3;   // streamed twice: rows pass A's loader may be ahead of the row pass B has finished (measured: 3 costs
                            // nothing at V = 128256 and gains 4 % at V = 152064 bf16; 2 and 1 starve pass A)
constexpr unsigned kClSpinLimit = 1u << 22;        // polls before a wait gives up (a fraction of a second at the least)

struct ClusterGeom {
  int cs;        // CTAs per cluster
  int slice;     // vocabulary indices per CTA (multiple of the 16-byte vector)
  int chunks;    // chunks per slice
  int ring;      // ring slots in use: min(kClSlots, 3 * chunks - 1), at least chunks + 1
  int n_clusters;
  int ra;        // 0: a slice stays in the ring from pass A to pass B. > 0 (slice larger than the ring): the
                 // slice is streamed twice through slots of two chunks each, slots [0, ra) feed pass A and
                 // slots [ra, ring) feed pass B
  int lead;      // streamed twice: pass A hands row n to the agent once row n - lead has been released to pass B
  int tri;       // 1: the launch walks the two-stage wrapper's rows as triples (k < K2) and pairs, one item per stage-1 row
};

// Per-row constants of pass B: -log2 of the normalisers in the scaled base-2 domain and the clamp floors.
struct __align__(16) RowConsts {
  float off_small, off_large;        // log2(sum_i exp(z_i / T)) of each model
  float floor_small, floor_large;    // logits below these would give log2 p < -125
  unsigned floor2_small, floor2_large;   // the same floors as packed bf16 pairs
  unsigned floor2_third;             // row triples: the third model (the target)
  unsigned pad0;
  float off_third, floor_third;
  unsigned pad1, pad2;
};

// Shared-memory control block behind the ring.
struct __align__(16) ClusterCtl {
  unsigned long long full[kClSlots];
  unsigned long long empty[kClSlots];
  unsigned long long a_done[kClDepth], b_done[kClDepth], lse_ready[kClDepth], fin_ready[kClDepth], b_go[kClDepth];
  float4 a_part[kClDepth][kClAWarps];              // (ref_small, sum_small, ref_large, sum_large) per pass-A warp
  float4 b_part[kClDepth][kClBWarps];              // (divergence sum in bits, sum max(p,q), rows differ, unused) per pass-B warp
  float4 row_lse[kClDepth];                        // (m2_small, l2s_small, m2_large, l2s_large) of the row
  RowConsts row_consts[kClDepth];                  // what pass B needs of the row, published by the agent
  float4 lse_in[kClDepth][kClMaxRanks];            // partials received from every rank of the cluster
  float4 fin_in[kClDepth][kClMaxRanks];            // pass-B partials received (rank 0 only)
  // row triples: the third model's log-sum-exp partials and the second pair's pass-B partials
  float4 a_part3[kClDepth][kClAWarps];             // (ref_third, sum_third, unused, unused)
  float4 b_part2[kClDepth][kClBWarps];
  float4 row_lse3[kClDepth];                       // (m2_third, l2s_third, unused, unused)
  float4 lse_in3[kClDepth][kClMaxRanks];
  float4 fin_in2[kClDepth][kClMaxRanks];
  int rows_closed;                                 // rows whose pass-B partials the second agent has dealt with
};

constexpr size_t kClSmemBytes = static_cast<size_t>(kClSlots) * kClSlotBytes + sizeof(ClusterCtl) + 128;

// ---- PTX wrappers -----------------------------------------------------------------------------------
__device__ __forceinline__ unsigned smem_u32(const void* p) { return static_cast<unsigned>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// non-blocking: has the phase with this parity completed?
__device__ __forceinline__ bool mbar_test(unsigned long long* bar, unsigned parity) {
  unsigned ok;
  asm volatile("{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// may suspend the thread for a hardware-chosen time before answering
__device__ __forceinline__ bool mbar_try(unsigned long long* bar, unsigned parity) {
  unsigned ok;
  asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned map_to_rank(const void* local, unsigned rank) {
  unsigned r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(local)), "r"(rank));
  return r;
}
// 16 bytes into another CTA's shared memory; the bytes are counted on that CTA's mbarrier when they land,
// so the receiver needs no fence: a completed phase means the data is there.
__device__ __forceinline__ void remote_post_f4(unsigned cluster_addr, float4 v, unsigned cluster_bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
               ::"r"(cluster_addr), "r"(__float_as_uint(v.x)), "r"(__float_as_uint(v.y)), "r"(__float_as_uint(v.z)),
                 "r"(__float_as_uint(v.w)), "r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, unsigned bytes, unsigned long long* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// The same copy with an L2 eviction priority: the streamed-twice variant asks L2 to keep what pass A's copy
// brought in (pass B's copy of the same bytes follows a row slice later) and to drop pass B's copy first.
__device__ __forceinline__ unsigned long long l2_policy_keep() {
  unsigned long long p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ unsigned long long l2_policy_drop() {
  unsigned long long p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void bulk_load_hint(void* smem_dst, const void* gsrc, unsigned bytes, unsigned long long* bar,
                                               unsigned long long policy) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
               ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)), "l"(policy) : "memory");
}
__device__ __forceinline__ unsigned cluster_rank() {
  unsigned r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint4 lds128(const void* p) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(smem_u32(p)));
  return v;
}

// ---- row walk ---------------------------------------------------------------------------------------
// Every role of every CTA of a cluster walks the same list: rows q, q + n_clusters, ... of the [B*K]
// grid, skipping positions at or beyond the sequence's n_valid. `n` counts the rows taken so far.
// Three-row launches walk one item per stage-1 row instead, position-major, with the positions taken in an
// order that alternates triples (k < K2) and pairs (k >= K2), so that whatever the number of clusters and
// the batch size have in common every cluster gets its share of both.
struct RowWalk {
  int next_r, stride, rows, rows1, K, K2, B;
  const int32_t* n_valid;
  bool tri_mode;
  int n;     // ordinal of the current row among the rows this cluster takes
  int r;     // current row index (valid after advance() returned true)
  int r2;    // row triples: index of the stage-2 row, b * K2 + k
  bool tri;  // the current item is a row triple
  __device__ void init(const StageParams& P, int cluster_id, int n_clusters, bool three_row) {
    next_r = cluster_id; stride = n_clusters; rows1 = P.B * P.K; K = P.K; K2 = P.K2; B = P.B;
    tri_mode = three_row;
    rows = three_row ? rows1 : P.B * (P.K + P.K2);
    n_valid = P.n_valid; n = -1; r = -1; r2 = -1; tri = false;
  }
  __device__ bool advance() {
    if (tri_mode) {
      if (next_r >= rows) return false;
      const int cand = next_r;
      next_r += stride;
      const int j = cand / B, b = cand - j * B;
      // j-th position in the alternating order: 0, K2, 1, K2 + 1, ... until one kind runs out
      const int n_pair = K - K2, both = 2 * (K2 < n_pair ? K2 : n_pair);
      int k;
      if (j < both) k = (j & 1) ? K2 + (j >> 1) : (j >> 1);
      else k = (K2 > n_pair) ? (both >> 1) + (j - both) : K2 + (both >> 1) + (j - both);
      r = b * K + k; tri = k < K2; r2 = b * K2 + k; ++n;
      return true;
    }
    while (next_r < rows) {
      const int cand = next_r;
      next_r += stride;
      if (n_valid != nullptr && cand < rows1) {   // n_valid speaks of the first row set only
        // candidates are taken position-major (all sequences' position 0, then position 1, ...): the early
        // positions, which are the ones that are usually valid, then spread evenly over the clusters
        // whatever the number of clusters and K have in common
        const int k = cand / B, b = cand - k * B;
        if (k >= n_valid[b]) continue;
        r = b * K + k; ++n;
        return true;
      }
      r = cand; ++n;
      return true;
    }
    return false;
  }
};

template <typename T>
__device__ __forceinline__ const T* row_ptr(const void* base, long long seq_stride, int r, int K, int V) {
  const int b = r / K, k = r - b * K;
  return static_cast<const T*>(base) + b * seq_stride + static_cast<long long>(k) * V;
}

// ---- packed fp32 pairs: float2 through the sm_100 packed add / mul / fma (one issue slot for two lanes) ----
__device__ __forceinline__ float2 splat2(float v) { return make_float2(v, v); }
__device__ __forceinline__ float2 ex2_2(float2 v) { return make_float2(ex2_approx(v.x), ex2_approx(v.y)); }

// One 16-byte vector of logits as packed pairs of consecutive vocabulary indices.
template <typename T> struct Pairs;
template <> struct Pairs<float> {
  static constexpr int kN = 2;
  __device__ static __forceinline__ void load(const uint4& u, float2 (&x)[2]) {
    x[0] = make_float2(__uint_as_float(u.x), __uint_as_float(u.y));
    x[1] = make_float2(__uint_as_float(u.z), __uint_as_float(u.w));
  }
  // the same with every logit raised to at least `floor_x`
  __device__ static __forceinline__ void load_clamped(const uint4& u, float floor_x, unsigned, float2 (&x)[2]) {
    x[0] = make_float2(fmaxf(__uint_as_float(u.x), floor_x), fmaxf(__uint_as_float(u.y), floor_x));
    x[1] = make_float2(fmaxf(__uint_as_float(u.z), floor_x), fmaxf(__uint_as_float(u.w), floor_x));
  }
  __device__ static __forceinline__ unsigned floor_bits(float) { return 0u; }
};
template <> struct Pairs<__nv_bfloat16> {
  static constexpr int kN = 4;
  // bf16 is the upper half of a binary32: widen by shifting / masking
  __device__ static __forceinline__ float2 widen(unsigned w) {
    return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
  }
  __device__ static __forceinline__ void load(const uint4& u, float2 (&x)[4]) {
    x[0] = widen(u.x); x[1] = widen(u.y); x[2] = widen(u.z); x[3] = widen(u.w);
  }
  __device__ static __forceinline__ unsigned max_bf16x2(unsigned a, unsigned b) {
    unsigned r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
  }
  // the clamp runs on the packed bf16 words, one instruction per two logits
  __device__ static __forceinline__ void load_clamped(const uint4& u, float, unsigned floor2, float2 (&x)[4]) {
    x[0] = widen(max_bf16x2(u.x, floor2)); x[1] = widen(max_bf16x2(u.y, floor2));
    x[2] = widen(max_bf16x2(u.z, floor2)); x[3] = widen(max_bf16x2(u.w, floor2));
  }
  // `floor_x` rounded up to bf16, in both halves of a word
  __device__ static __forceinline__ unsigned floor_bits(float floor_x) {
    unsigned b = __float_as_uint(floor_x);
    if (floor_x == floor_x && fabsf(floor_x) < INFINITY) {
      const unsigned low = b & 0xffffu;
      b &= 0xffff0000u;
      if (low != 0u && floor_x > 0.f) b += 0x10000u;   // towards +inf; negative values round up by truncation
    } else {
      b = 0xff800000u;                                  // no usable floor: -inf clamps nothing
    }
    return (b >> 16) | (b & 0xffff0000u);
  }
};

// ---- pass A: streaming log-sum-exp -------------------------------------------------------------------
// State per warp and model: a reference `ref` in the scaled base-2 domain, the same in every lane, and
// per lane the sum S of 2^(x*c - ref). No running maximum is kept: the exps of one vector are summed on
// their own, and only when some lane's vector sum is not finite (a logit more than 2^127 above the
// reference, which includes the first finite vector of a row because the reference starts at -1e30, or a
// NaN / +inf logit) does the warp take the slow path, which moves the reference to the warp's maximum of
// that vector and redoes it. The finite starting reference makes -inf logits (masked vocabulary)
// contribute exactly 0. With one reference per warp the row-end reduction is a plain sum.
struct LseState {
  float ref, s;
  __device__ __forceinline__ void reset() { ref = -1e30f; s = 0.f; }
};

// sum of 2^(x*c - ref) over one 16-byte vector; `live` false (vector outside the slice) gives 0
template <typename T>
__device__ __forceinline__ float lse_vector_sum(const uint4& u, float c, float ref) {
  constexpr int N = Pairs<T>::kN;
  float2 x[N];
  Pairs<T>::load(u, x);
  const float2 cc = splat2(c), nref = splat2(-ref);
  float2 v = ex2_2(__ffma2_rn(x[0], cc, nref));
#pragma unroll
  for (int j = 1; j < N; ++j) v = __fadd2_rn(v, ex2_2(__ffma2_rn(x[j], cc, nref)));
  return v.x + v.y;
}

// the same as a packed pair of partial sums (their total is the vector sum)
template <typename T>
__device__ __forceinline__ float2 lse_vector_sum2(const uint4& u, float c, float ref) {
  constexpr int N = Pairs<T>::kN;
  float2 x[N];
  Pairs<T>::load(u, x);
  const float2 cc = splat2(c), nref = splat2(-ref);
  float2 v = ex2_2(__ffma2_rn(x[0], cc, nref));
#pragma unroll
  for (int j = 1; j < N; ++j) v = __fadd2_rn(v, ex2_2(__ffma2_rn(x[j], cc, nref)));
  return v;
}

// Warp-wide: move the reference up to the largest logit of this vector (over the live lanes) and
// return this lane's vector sum against the new reference.
template <typename T>
__device__ __noinline__ float lse_slow_path(uint4 u, bool live, float c, float ref_in, float s_in, float* ref_out,
                                            float* s_out) {
  constexpr int N = Pairs<T>::kN;
  float2 x[N];
  Pairs<T>::load(u, x);
  float gm = -INFINITY;
  if (live) {
#pragma unroll
    for (int j = 0; j < N; ++j) gm = fmaxf(gm, fmaxf(x[j].x, x[j].y));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) gm = fmaxf(gm, __shfl_xor_sync(0xffffffffu, gm, o));
  const float nr = gm * c;
  float ref = ref_in, s = s_in;
  if (nr > ref) {   // false for NaN; +inf poisons the sum below, as it should
    s *= ex2_approx(ref - nr);
    ref = nr;
  }
  float t = 0.f;
  if (live) {
#pragma unroll
    for (int j = 0; j < N; ++j) t += ex2_approx(fmaf(x[j].x, c, -ref)) + ex2_approx(fmaf(x[j].y, c, -ref));
  }
  *ref_out = ref;
  *s_out = s;
  return t;
}

// Largest logit of one vector (-inf when the vector lies outside the slice), NaN ignored.
template <typename T>
__device__ __forceinline__ float vector_max(const uint4& u, bool live) {
  constexpr int N = Pairs<T>::kN;
  float2 x[N];
  Pairs<T>::load(u, x);
  float gm = fmaxf(x[0].x, x[0].y);
#pragma unroll
  for (int j = 1; j < N; ++j) gm = fmaxf(gm, fmaxf(x[j].x, x[j].y));
  return live ? gm : -INFINITY;
}

// Add one vector sum, taken against `ref_used`, to the state; all 32 lanes call this together. When an
// earlier vector of the same step has moved the reference the sum is taken again, so that the result
// does not depend on how many vectors a step happened to group.
template <typename T>
__device__ __forceinline__ void lse_commit(float t, float ref_used, const uint4& u, bool live, float c, LseState& st) {
  if (st.ref != ref_used) t = lse_vector_sum<T>(u, c, st.ref);
  if (__any_sync(0xffffffffu, live && !(t < INFINITY))) {
    float r2, s2;
    t = lse_slow_path<T>(u, live, c, st.ref, st.s, &r2, &s2);
    st.ref = r2;
    st.s = s2;
  }
  st.s += live ? t : 0.f;
}

// Combine (ref, S) partials: returns the pair for the union. Fixed order, NaN-preserving in S.
__device__ __forceinline__ void lse_merge(float& ref, float& s, float oref, float os) {
  const float m = fmaxf(ref, oref);
  s = s * ex2_approx(ref - m) + os * ex2_approx(oref - m);
  ref = m;
}

// ---- pass B ------------------------------------------------------------------------------------------
// With a = log2 p and b = log2 q (both linear in the logits once the normalisers are known), each
// vocabulary index adds to the Jensen-Shannon divergence, in bits and before the factor 1/2,
//     p lg p + q lg q - (p + q) lg((p + q) / 2)  =  2^M * h(d),   M = max(a, b),  d = -|a - b|,
//     h(d) = u d + psi(u),   u = 2^d in (0, 1],   psi(u) = (1 + u) (1 - lg(1 + u)),
// which costs two ex2 (2^M and 2^d) and a polynomial for psi instead of two ex2 and one lg2 plus
// cancelling sums: every term is >= 0 (h(0) = 0 for equal probabilities, h -> 1 when one side vanishes).
// 2^M is max(p, q), so the residual mass sum max(0, p - q) = sum max(p, q) - 1 falls out of the same ex2.
// psi is a minimax polynomial on [0, 1] (least-squares/Remez fits): degree 7 with max abs error 5.6e-8;
// degrees 5 and 4, fitted with psi(0) = 1 and psi(1) = 0 held exactly so that vanishing and equal
// probabilities add no bias, with 4.4e-6 and 4.0e-5.
// Logits arrive clamped from below so that a, b >= -125: nothing is -inf, NaN cannot arise, and the terms
// clamped away are below 2^-125.
template <int DEG>
__device__ __forceinline__ float2 psi_poly(float2 u) {
  if (DEG == 7) {
    float2 p = __ffma2_rn(splat2(3.571110749e-03f), u, splat2(-1.966644044e-02f));
    p = __ffma2_rn(p, u, splat2(5.437676601e-02f));
    p = __ffma2_rn(p, u, splat2(-1.133036196e-01f));
    p = __ffma2_rn(p, u, splat2(2.388960843e-01f));
    p = __ffma2_rn(p, u, splat2(-7.211711122e-01f));
    p = __ffma2_rn(p, u, splat2(-4.427027888e-01f));
    p = __ffma2_rn(p, u, splat2(1.000000056e+00f));
    return p;
  } else if (DEG == 5) {
    float2 p = __ffma2_rn(splat2(1.597597450e-02f), u, splat2(-7.831134647e-02f));
    p = __ffma2_rn(p, u, splat2(2.232717425e-01f));
    p = __ffma2_rn(p, u, splat2(-7.180256248e-01f));
    p = __ffma2_rn(p, u, splat2(-4.429107606e-01f));
    p = __ffma2_rn(p, u, splat2(1.0f));
    return p;
  } else {
    float2 p = __ffma2_rn(splat2(-3.877525777e-02f), u, splat2(1.896598488e-01f));
    p = __ffma2_rn(p, u, splat2(-7.068237066e-01f));
    p = __ffma2_rn(p, u, splat2(-4.440608621e-01f));
    p = __ffma2_rn(p, u, splat2(1.0f));
    return p;
  }
}

// Degree by logits type: fp32 logits are held to 1e-5 on the divergence and take degree 7; bf16 logits are
// held to 2e-3 and take degree 4, whose error adds at most 0.35 * 4e-5 * sum max(p, q) < 3e-5 to D (measured
// against a double-precision reference on peaked, flat, near-equal and far-apart row pairs: at most 1.6e-5,
// against 1e-6 with degree 7), for three of the polynomial's seven instructions.
constexpr int kPsiDegBf16 = 4;

struct DivAcc {
  float2 js, big;    // sum 2^M h(d); sum 2^M
  unsigned differ;   // OR of (small bits XOR large bits)
  __device__ __forceinline__ void reset() { js = big = make_float2(0.f, 0.f); differ = 0u; }
};

template <int DIV, int N, int PSI = 7>
__device__ __forceinline__ void div_accumulate(const float2 (&xl)[N], const float2 (&xs)[N], float c, float off_l,
                                               float off_s, DivAcc& acc) {
  const float2 cc = splat2(c), nl = splat2(-off_l), ns = splat2(-off_s);
#pragma unroll
  for (int j = 0; j < N; ++j) {
    const float2 a = __ffma2_rn(xl[j], cc, nl), b = __ffma2_rn(xs[j], cc, ns);   // log2 p, log2 q
    if (DIV == kDivKL) {
      // KL(large || small) on unclamped logits: q == 0 with p > 0 gives +inf, as it should
      const float2 p = ex2_2(a), q = ex2_2(b);
      acc.big = __fadd2_rn(acc.big, make_float2(fmaxf(p.x, q.x), fmaxf(p.y, q.y)));
      if (p.x > 0.f) acc.js.x = (q.x > 0.f) ? fmaf(p.x, a.x - b.x, acc.js.x) : INFINITY;
      if (p.y > 0.f) acc.js.y = (q.y > 0.f) ? fmaf(p.y, a.y - b.y, acc.js.y) : INFINITY;
    } else {
      const float2 e = make_float2(ex2_approx(fmaxf(a.x, b.x)), ex2_approx(fmaxf(a.y, b.y)));   // max(p, q)
      acc.big = __fadd2_rn(acc.big, e);
      if (DIV == kDivJS) {
        const float2 dd = __ffma2_rn(b, splat2(-1.f), a);
        const float2 u = make_float2(ex2_approx(-fabsf(dd.x)), ex2_approx(-fabsf(dd.y)));
        const float2 ps = psi_poly<PSI>(u);
        const float2 h = make_float2(fmaf(u.x, -fabsf(dd.x), ps.x), fmaf(u.y, -fabsf(dd.y), ps.y));
        acc.js = __ffma2_rn(e, h, acc.js);
      }
    }
  }
}

template <typename V>
__device__ __forceinline__ V warp_sum(V v) { return warp_reduce<OpSum>(v); }

// A next launch that was made a programmatic dependent of this one (the finalisation) may be scheduled once every
// warp of every CTA has been here; it still waits for this grid's end before it reads a statistic. Every warp comes
// here after it has traded its registers, so no CTA placed early can be in the way of that trade.
__device__ __forceinline__ void release_dependent_launch() { asm volatile("griddepcontrol.launch_dependents;"); }

// ---- the kernel -------------------------------------------------------------------------------------
// RS = false: a CTA's slice of a row fits the ring and is copied in once. RS = true ("re-stream"): the slice is
// larger than the ring (small clusters, which is what fills every SM of the device), so it is copied in
// twice -- once for each pass, the second copy coming out of L2 -- through two rings of their own.
// TRI (with RS only): the launch is a two-stage wrapper's, walked as row triples and pairs (see the top).
template <typename T, int DIV, bool RS, bool TRI>
__global__ void __launch_bounds__(RS ? kClThreadsRS : kClThreads, 1) rowstats_cluster_kernel(const StageParams P, const ClusterGeom G) {
  static_assert(RS || !TRI, "row triples are streamed twice");
  extern __shared__ unsigned char smem_raw[];
  unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  ClusterCtl* ctl = reinterpret_cast<ClusterCtl*>(ring + static_cast<size_t>(kClSlots) * kClSlotBytes);

  constexpr int E = Elem<T>::kPerVec;              // logits per 16-byte vector
  constexpr int CH = kClHalfBytes / sizeof(T);     // logits per chunk and model
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const unsigned rank = cluster_rank();
  const int cluster_id = blockIdx.x / G.cs;
  const int V = P.V, K = P.K;
  const int slice_begin = static_cast<int>(rank) * G.slice;
  const int slice_len = max(0, min(G.slice, V - slice_begin));   // logits this CTA owns
  const int C = G.chunks, R = G.ring;
  const int RA = RS ? G.ra : R;        // slots pass A cycles through
  const int RB0 = RS ? G.ra : 0;       // first slot of pass B
  // The streamed-twice variant moves two chunks per barrier (a slot of 2 x 16 KB): its rings need no chunk
  // granularity to hold a row, and every hand-off costs the two instruction streams issue slots. A row triple
  // moves one chunk of its three rows (24 KB of the same slot).
  constexpr int SUB = RS ? kClSubRS : 1;
  constexpr int kSlotStride = SUB * kClSlotBytes;
  static_assert(!TRI || kSlotStride >= 3 * kClHalfBytes, "a slot holds one chunk of three rows");
  const int CS = (C + SUB - 1) / SUB;  // barrier steps per row slice of a pair
  auto steps_of = [&](bool tri) { return tri ? C : CS; };

  if (tid == 0) {
    ctl->rows_closed = 0;
    for (int s = 0; s < kClSlots; ++s) {
      mbar_init(&ctl->full[s], 1);
      mbar_init(&ctl->empty[s], (RS && s < RA) ? kClAWarps : kClBWarps);   // the warps that hand the slot back
    }
    for (int d = 0; d < kClDepth; ++d) {
      mbar_init(&ctl->a_done[d], kClAWarps);
      mbar_init(&ctl->b_done[d], kClBWarps);
      mbar_init(&ctl->lse_ready[d], 1);   // the local agent's arrive; the peers' partials count as bytes
      mbar_init(&ctl->fin_ready[d], 1);
      mbar_init(&ctl->b_go[d], 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  cluster_sync_all();   // every CTA's barriers exist before anyone arrives on them remotely

  bool dead = false;    // this thread gave up on a wait: stop waiting, just run to the end
  auto give_up = [&]() {
    dead = true;
    atomicExch(P.status, 1);
  };
  // blocking wait on one mbarrier phase, bounded
  auto wait_phase = [&](unsigned long long* bar, unsigned parity) {
    if (mbar_test(bar, parity)) return;   // the common case: already complete, no suspension
    unsigned spins = 0;
    while (!dead && !mbar_try(bar, parity))
      if (++spins > kClSpinLimit) give_up();
  };
  const int rows1 = P.B * K;
  // base of this CTA's slice of model m (0 small, 1 large, 2 third) of the walk's current item
  auto model_row = [&](const RowWalk& w, int m) -> const T* {
    if (TRI) {
      if (m == 0) return row_ptr<T>(P.small, P.seq_stride_small, w.r, K, V) + slice_begin;
      if (m == 1) return row_ptr<T>(P.large, P.seq_stride_large, w.r, K, V) + slice_begin;
      return row_ptr<T>(P.large2, P.seq_stride_large2, w.r2, P.K2, V) + slice_begin;
    }
    const bool second = w.r >= rows1;   // second row set: stage 2 of the wrapper
    if (m == 0) return (second ? row_ptr<T>(P.small2, P.seq_stride_small2, w.r - rows1, P.K2, V)
                               : row_ptr<T>(P.small, P.seq_stride_small, w.r, K, V)) + slice_begin;
    return (second ? row_ptr<T>(P.large2, P.seq_stride_large2, w.r - rows1, P.K2, V)
                   : row_ptr<T>(P.large, P.seq_stride_large, w.r, K, V)) + slice_begin;
  };

  if (warp < kClConsumerWarps) {
    const float c = P.c;
    const bool is_a = warp < kClAWarps;
    const int pw = is_a ? warp : warp - kClAWarps;    // index among the warps of this pass
    const int pass_warps = is_a ? kClAWarps : kClBWarps;
    // vectors pw*32 + lane + i * pass_warps * 32 of every chunk; `len[i]` > chunk offset while vector i lies inside the slice
    const unsigned char* my = ring + (pw * 32 + lane) * 16;
    constexpr int kMaxVec = kClAVec > kClBVec ? kClAVec : kClBVec;
    int len[kMaxVec];
#pragma unroll
    for (int i = 0; i < kMaxVec; ++i) len[i] = slice_len - (pw * 32 + lane + i * pass_warps * 32) * E;
    RowWalk w;
    w.init(P, cluster_id, G.n_clusters, TRI);
    unsigned slot = 0, par = 0;

    if (is_a) {
      if (RS) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kClRegsA));
      release_dependent_launch();
      constexpr int kVecStride = kClAWarps * 32 * 16;   // bytes between a lane's vectors
      // ================================ pass A ================================
      // A row is summed optimistically against one reference per model, taken from the warp's first
      // vectors: no vote and no dependent branch per chunk, so the exps of consecutive chunks pipeline
      // freely. Only if some lane's row sum comes out non-finite (a logit more than 2^127 above that
      // reference, or NaN / +inf) is the row redone through the careful per-vector commits -- its chunks
      // are all still in the ring, because pass B cannot enter the row before pass A has left it.
      bool landed = false;   // the answer of a test of the next chunk's barrier, asked one chunk early
      // one row of NM models, SUBN chunks per slot
      auto row_a = [&](auto nm_c, auto sub_c) {
        constexpr int NM = decltype(nm_c)::value, SUBN = decltype(sub_c)::value;
        const int steps = (C + SUBN - 1) / SUBN;
        LseState st[NM];
        float2 v[NM];
#pragma unroll
        for (int m = 0; m < NM; ++m) { st[m].reset(); v[m] = make_float2(0.f, 0.f); }
        const unsigned slot0 = slot;   // where the row starts in the ring
        int off = 0;   // chunk offset inside the slice, in logits
        for (int step = 0; step < steps; ++step) {
          if (!landed) wait_phase(&ctl->full[slot], par);
          const unsigned char* sbase = my + slot * kSlotStride;
          const unsigned used = slot;
          if (++slot == static_cast<unsigned>(RA)) { slot = 0; par ^= 1u; }
          landed = mbar_test(&ctl->full[slot], par);   // its latency hides behind this step's arithmetic
#pragma unroll
          for (int sub = 0; sub < SUBN; ++sub, off += CH) {   // a chunk beyond the slice (odd count) has no live vector
            const unsigned char* base = sbase + sub * kClSlotBytes;
            uint4 u[NM][kClAVec];
#pragma unroll
            for (int i = 0; i < kClAVec; ++i)
#pragma unroll
              for (int m = 0; m < NM; ++m) u[m][i] = lds128(base + m * kClHalfBytes + i * kVecStride);
            if (step == 0 && sub == 0) {
              // the warp's largest logit of its first vectors (the floor keeps rows that start with -inf at 0)
              float g[NM];
#pragma unroll
              for (int m = 0; m < NM; ++m) g[m] = vector_max<T>(u[m][0], len[0] > 0);
#pragma unroll
              for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                for (int m = 0; m < NM; ++m) g[m] = fmaxf(g[m], __shfl_xor_sync(0xffffffffu, g[m], o));
#pragma unroll
              for (int m = 0; m < NM; ++m) st[m].ref = fmaxf(g[m] * c, -1e30f);
            }
#pragma unroll
            for (int i = 0; i < kClAVec; ++i) {
              const bool live = len[i] > off;
#pragma unroll
              for (int m = 0; m < NM; ++m) {
                const float2 ps = lse_vector_sum2<T>(u[m][i], c, st[m].ref);
                v[m] = __fadd2_rn(v[m], live ? ps : make_float2(0.f, 0.f));
              }
            }
          }
          if (RS) {   // pass A is this slot's only reader: hand it back
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl->empty[used]);
          }
        }
        float tot = 0.f;
#pragma unroll
        for (int m = 0; m < NM; ++m) { st[m].s = v[m].x + v[m].y; tot += st[m].s; }
        if (__any_sync(0xffffffffu, !(tot < INFINITY))) {
          // careful second go over the row's chunks, vector by vector, moving the references as needed
#pragma unroll
          for (int m = 0; m < NM; ++m) st[m].s = 0.f;
          unsigned sl2 = slot0;
          off = 0;
          // when the slice is streamed twice its chunks have left the ring: take the vectors from global memory
          const T* g[NM];
#pragma unroll
          for (int m = 0; m < NM; ++m) g[m] = model_row(w, m);
#pragma unroll 1
          for (int cidx = 0; cidx < C; ++cidx, off += CH) {
            const unsigned char* base = my + sl2 * kClSlotBytes;
#pragma unroll 1
            for (int i = 0; i < kClAVec; ++i) {
              const int e = off + (pw * 32 + lane + i * kClAWarps * 32) * E;   // first logit of the vector, in the slice
              const bool live = e < slice_len;
#pragma unroll
              for (int m = 0; m < NM; ++m) {
                uint4 v4 = make_uint4(0u, 0u, 0u, 0u);
                if (RS) {
                  if (live) v4 = *reinterpret_cast<const uint4*>(g[m] + e);
                } else {
                  v4 = lds128(base + m * kClHalfBytes + i * kVecStride);
                }
                // a NaN "reference used" makes the commit take the vector sum afresh
                lse_commit<T>(0.f, __int_as_float(0x7fc00000), v4, live, c, st[m]);
              }
            }
            if (++sl2 == static_cast<unsigned>(R)) sl2 = 0;
          }
        }
        // row finished: the warp's partial (one reference, summed S) -> a_part, then tell the agent
        float sums[NM];
#pragma unroll
        for (int m = 0; m < NM; ++m) sums[m] = warp_reduce<OpSum>(st[m].s);
        const int d = w.n % kClDepth;
        // With a ring of its own pass A could run rows ahead of pass B and of the agents (a resident slice
        // cannot: its slots come back from pass B). The exchange buffers are kClDepth rows deep, so row n is
        // handed over only once row n - kClDepth has been released to pass B, which is after the agent has
        // read that row's partials out of this buffer.
        if (RS && w.n >= G.lead) {
          const int m = w.n - G.lead;   // 1 <= lead <= kClDepth
          wait_phase(&ctl->b_go[m % kClDepth], (m / kClDepth) & 1u);
        }
        if (lane == 0) {
          ctl->a_part[d][pw] = make_float4(st[0].ref, sums[0], st[1].ref, sums[1]);
          if (NM == 3) ctl->a_part3[d][pw] = make_float4(st[NM - 1].ref, sums[NM - 1], 0.f, 0.f);
          mbar_arrive(&ctl->a_done[d]);
        }
      };
      while (w.advance()) {
        if (TRI && w.tri) row_a(std::integral_constant<int, 3>{}, std::integral_constant<int, 1>{});
        else row_a(std::integral_constant<int, 2>{}, std::integral_constant<int, SUB>{});
      }
    } else {
      // ================================ pass B ================================
      if (RS) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kClRegsB));
      release_dependent_launch();
      constexpr int N = Pairs<T>::kN;
      constexpr int PSI = sizeof(T) == 2 ? kPsiDegBf16 : 7;
      constexpr int kVecStride = kClBWarps * 32 * 16;   // bytes between a lane's vectors
      if (RS) slot = static_cast<unsigned>(RB0);
      bool landed = false;   // as in pass A: the next chunk's barrier is tested one chunk early
      auto row_b = [&](auto nm_c, auto sub_c) {
        constexpr int NM = decltype(nm_c)::value, SUBN = decltype(sub_c)::value;
        const int steps = (C + SUBN - 1) / SUBN;
        const int d = w.n % kClDepth;
        wait_phase(&ctl->b_go[d], (w.n / kClDepth) & 1u);   // the row's constants are published: pass A is through
        const RowConsts rc = ctl->row_consts[d];
        DivAcc acc, acc2;   // the pair (small, large); for a triple also the pair (large, third)
        acc.reset(); acc2.reset();
        int off = 0;
        for (int step = 0; step < steps; ++step) {
          if (RS && !landed) wait_phase(&ctl->full[slot], par);   // pass B's own copy of the chunks
          const unsigned char* sbase = my + slot * kSlotStride;
          if (RS) {
            unsigned nslot = slot + 1u, npar = par;
            if (nslot == static_cast<unsigned>(R)) { nslot = static_cast<unsigned>(RB0); npar ^= 1u; }
            landed = mbar_test(&ctl->full[nslot], npar);
          }
#pragma unroll
          for (int sub = 0; sub < SUBN; ++sub, off += CH) {
            const unsigned char* base = sbase + sub * kClSlotBytes;
            uint4 u[NM][kClBVec];
#pragma unroll
            for (int i = 0; i < kClBVec; ++i)
#pragma unroll
              for (int m = 0; m < NM; ++m) u[m][i] = lds128(base + m * kClHalfBytes + i * kVecStride);
#pragma unroll
            for (int i = 0; i < kClBVec; ++i) {
              float2 xs[N], xl[N];
              Pairs<T>::load_clamped(u[0][i], rc.floor_small, rc.floor2_small, xs);
              Pairs<T>::load_clamped(u[1][i], rc.floor_large, rc.floor2_large, xl);
              DivAcc local;
              local.reset();
              local.differ = (u[0][i].x ^ u[1][i].x) | (u[0][i].y ^ u[1][i].y) | (u[0][i].z ^ u[1][i].z) | (u[0][i].w ^ u[1][i].w);
              div_accumulate<DIV, N, PSI>(xl, xs, c, rc.off_large, rc.off_small, local);
              const bool live = len[i] > off;   // a vector beyond the slice adds nothing
              if (live) {
                acc.js = __fadd2_rn(acc.js, local.js);
                acc.big = __fadd2_rn(acc.big, local.big);
                acc.differ |= local.differ;
              }
              if (NM == 3) {
                float2 xt[N];
                Pairs<T>::load_clamped(u[NM - 1][i], rc.floor_third, rc.floor2_third, xt);
                DivAcc local2;
                local2.reset();
                local2.differ = (u[1][i].x ^ u[NM - 1][i].x) | (u[1][i].y ^ u[NM - 1][i].y) | (u[1][i].z ^ u[NM - 1][i].z) |
                                (u[1][i].w ^ u[NM - 1][i].w);
                div_accumulate<DIV, N, PSI>(xt, xl, c, rc.off_third, rc.off_large, local2);
                if (live) {
                  acc2.js = __fadd2_rn(acc2.js, local2.js);
                  acc2.big = __fadd2_rn(acc2.big, local2.big);
                  acc2.differ |= local2.differ;
                }
              }
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(&ctl->empty[slot]);   // this warp is done with the slot
          if (++slot == static_cast<unsigned>(R)) { slot = static_cast<unsigned>(RB0); par ^= 1u; }
        }
        const float js = warp_reduce<OpSum>(acc.js.x + acc.js.y);
        const float big = warp_reduce<OpSum>(acc.big.x + acc.big.y);
        const unsigned differ = __reduce_or_sync(0xffffffffu, acc.differ);
        float js2 = 0.f, big2 = 0.f;
        unsigned differ2 = 0u;
        if (NM == 3) {
          js2 = warp_reduce<OpSum>(acc2.js.x + acc2.js.y);
          big2 = warp_reduce<OpSum>(acc2.big.x + acc2.big.y);
          differ2 = __reduce_or_sync(0xffffffffu, acc2.differ);
        }
        if (lane == 0) {
          ctl->b_part[d][pw] = make_float4(js, big, differ ? 1.f : 0.f, 0.f);
          if (NM == 3) ctl->b_part2[d][pw] = make_float4(js2, big2, differ2 ? 1.f : 0.f, 0.f);
          mbar_arrive(&ctl->b_done[d]);
        }
      };
      while (w.advance()) {
        if (TRI && w.tri) row_b(std::integral_constant<int, 3>{}, std::integral_constant<int, 1>{});
        else row_b(std::integral_constant<int, 2>{}, std::integral_constant<int, SUB>{});
      }
    }
  } else if (warp == kClConsumerWarps || warp == kClConsumerWarps + 3) {
    if (RS) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kClRegsService));
    release_dependent_launch();
    // ================================ loader ================================
    // One thread per ring: the whole ring, or (slice streamed twice) pass A's slots [0, RA) from this warp and
    // pass B's slots [RA, R) from the last warp. The two streams run freely; pass B's copy of a chunk is
    // asked for about one row slice after pass A's and is served by L2.
    const bool for_b = warp != kClConsumerWarps;
    const unsigned lo = for_b ? static_cast<unsigned>(RB0) : 0u, hi = static_cast<unsigned>(for_b ? R : RA);
    if (lane == 0) {
      RowWalk w;
      w.init(P, cluster_id, G.n_clusters, TRI);
      const unsigned long long policy = RS ? (for_b ? l2_policy_drop() : l2_policy_keep()) : 0ull;
      // step `step` of a row slice (`sub_n` chunks of `nm` models) into `slot`, once the slot's readers of
      // `fills` ring turns ago are through
      auto fill = [&](const T* const (&src)[3], int nm, int sub_n, int step, unsigned slot, unsigned fills) {
        if (fills > 0) wait_phase(&ctl->empty[slot], (fills - 1u) & 1u);
        if (dead) return false;   // the slot was never handed back: nothing more is copied into this ring
        unsigned total = 0;
        for (int sub = 0; sub < sub_n; ++sub) total += static_cast<unsigned>(max(0, min(CH, slice_len - (step * sub_n + sub) * CH)));
        if (total > 0) {
          mbar_arrive_expect_tx(&ctl->full[slot], static_cast<unsigned>(nm) * total * static_cast<unsigned>(sizeof(T)));
          for (int sub = 0; sub < sub_n; ++sub) {
            const int e0 = (step * sub_n + sub) * CH;
            const int n = min(CH, slice_len - e0);
            if (n > 0) {
              const unsigned bytes = static_cast<unsigned>(n) * sizeof(T);
              unsigned char* dst = ring + static_cast<size_t>(slot) * kSlotStride + sub * kClSlotBytes;
              for (int m = 0; m < nm; ++m) {
                if (RS) bulk_load_hint(dst + m * kClHalfBytes, src[m] + e0, bytes, &ctl->full[slot], policy);
                else bulk_load(dst + m * kClHalfBytes, src[m] + e0, bytes, &ctl->full[slot]);
              }
            }
          }
        } else {
          mbar_arrive(&ctl->full[slot]);   // nothing of this step falls into this CTA's slice
        }
        return true;
      };
      unsigned slot = lo, fills = 0;   // ring position; how often the ring has wrapped
      while (!dead && w.advance()) {
        const bool tri = TRI && w.tri;
        if (RS && !for_b) {
          // Pass A is the lighter pass; left alone it runs rows ahead of pass B until the exchange buffers stop it,
          // and pass B's copy of the same bytes then finds part of them gone from L2. Its loader starts row n only
          // once pass B is through row n - kClLag.
          unsigned spins = 0;
          while (!dead && *reinterpret_cast<volatile int*>(&ctl->rows_closed) < w.n - kClLag + 1) {
            __nanosleep(200);
            if (++spins > kClSpinLimit) give_up();
          }
        }
        const T* const src[3] = {model_row(w, 0), model_row(w, 1), tri ? model_row(w, 2) : nullptr};
        const int steps = steps_of(tri);
        for (int step = 0; step < steps; ++step) {
          if (!fill(src, tri ? 3 : 2, tri ? 1 : SUB, step, slot, fills)) break;
          if (++slot == hi) { slot = lo; ++fills; }
        }
      }
      // Every copy issued above is waited for by its consumers before they leave -- unless a wait gave up
      // somewhere in the CTA. Then this thread has stopped issuing, and it sees every copy it did issue land
      // before the CTA's shared memory goes away: each slot's barrier is polled (bounded) for its latest phase.
      if (dead || *reinterpret_cast<volatile int*>(P.status) != 0) {
        for (unsigned s = lo; s < hi; ++s) {
          const unsigned turns = fills + (s < slot ? 1u : 0u);   // phases of this slot's barrier armed so far
          if (turns == 0) continue;
          unsigned spins = 0;
          while (!mbar_try(&ctl->full[s], (turns - 1u) & 1u) && ++spins <= kClSpinLimit) {}
        }
      }
    }
  } else {
    // ================================ agent ================================
    // Four kinds of events per row:
    //   a(n)  the warps' pass-A partials of row n are in    -> merge, send the CTA's partial to every rank
    //   g(n)  every rank's partial of row n has arrived     -> row constants for pass B, release the consumers
    //   b(n)  the warps' pass-B partials of row n are in    -> sum, send to rank 0
    //   f(n)  (rank 0) every rank's pass-B partial arrived  -> write the row's statistics
    // shared by two agent warps: one takes a(n), g(n) in row order (the path that releases pass B), the other
    // b(n), f(n). Every wait is a blocking wait on one barrier, so the agents cost the consumer warps that
    // share their issue ports next to nothing. The exchange buffers are kClDepth rows deep; nothing of row m
    // can be produced anywhere in the cluster before a(m) has been sent, a(m) comes after g(m-1), and the
    // first agent holds a(m) back until the second one has closed row m - kClDepth + 1.
    // A row triple carries a second 16-byte record through every step (third model / second pair).
    if (RS) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kClRegsService));
    release_dependent_launch();
    const float inv_c = 1.f / P.c;

    auto event_a = [&](int n, bool tri) {
      const int d = n % kClDepth;
      wait_phase(&ctl->a_done[d], (n / kClDepth) & 1u);
      // merge the warps' partials (every lane does the same arithmetic, warp order) ...
      float ms = -1e30f, ml = -1e30f, mt = -1e30f;
#pragma unroll
      for (int k = 0; k < kClAWarps; ++k) { ms = fmaxf(ms, ctl->a_part[d][k].x); ml = fmaxf(ml, ctl->a_part[d][k].z); }
      float ss = 0.f, sl = 0.f, stt = 0.f;
#pragma unroll
      for (int k = 0; k < kClAWarps; ++k) {
        const float4 v = ctl->a_part[d][k];
        ss = fmaf(v.y, ex2_approx(v.x - ms), ss);
        sl = fmaf(v.w, ex2_approx(v.z - ml), sl);
      }
      if (TRI && tri) {
#pragma unroll
        for (int k = 0; k < kClAWarps; ++k) mt = fmaxf(mt, ctl->a_part3[d][k].x);
#pragma unroll
        for (int k = 0; k < kClAWarps; ++k) {
          const float4 v = ctl->a_part3[d][k];
          stt = fmaf(v.y, ex2_approx(v.x - mt), stt);
        }
      }
      // ... open this row's phase of the local barrier for one partial per rank, and post ours to every rank
      if (lane == 0) mbar_arrive_expect_tx(&ctl->lse_ready[d], static_cast<unsigned>(G.cs) * ((TRI && tri) ? 32u : 16u));
      if (lane < G.cs) {
        remote_post_f4(map_to_rank(&ctl->lse_in[d][rank], lane), make_float4(ms, ss, ml, sl),
                       map_to_rank(&ctl->lse_ready[d], lane));
        if (TRI && tri)
          remote_post_f4(map_to_rank(&ctl->lse_in3[d][rank], lane), make_float4(mt, stt, 0.f, 0.f),
                         map_to_rank(&ctl->lse_ready[d], lane));
      }
    };
    auto event_g = [&](int n, bool tri) {
      const int d = n % kClDepth;
      wait_phase(&ctl->lse_ready[d], (n / kClDepth) & 1u);
      // rank order, so that every CTA of the cluster gets the same bits; four ranks at a time keeps the
      // loads and exps of a group independent of each other (this sits on the path that releases pass B)
      float ms = -1e30f, ml = -1e30f, ss = 0.f, sl = 0.f;
      for (int j0 = 0; j0 < G.cs; j0 += 4) {
        float4 v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = (j0 + j < G.cs) ? ctl->lse_in[d][j0 + j] : make_float4(-1e30f, 0.f, -1e30f, 0.f);
        const float gs = fmaxf(fmaxf(v[0].x, v[1].x), fmaxf(v[2].x, v[3].x));
        const float gl = fmaxf(fmaxf(v[0].z, v[1].z), fmaxf(v[2].z, v[3].z));
        const float ns = fmaxf(ms, gs), nl = fmaxf(ml, gl);
        ss *= ex2_approx(ms - ns);
        sl *= ex2_approx(ml - nl);
        ms = ns; ml = nl;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          ss = fmaf(v[j].y, ex2_approx(v[j].x - ms), ss);
          sl = fmaf(v[j].w, ex2_approx(v[j].z - ml), sl);
        }
      }
      float mt = -1e30f, stt = 0.f;
      if (TRI && tri) {   // the third model, the same way (its partials sit in the x, y fields)
        for (int j0 = 0; j0 < G.cs; j0 += 4) {
          float4 v[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) v[j] = (j0 + j < G.cs) ? ctl->lse_in3[d][j0 + j] : make_float4(-1e30f, 0.f, -1e30f, 0.f);
          const float gt = fmaxf(fmaxf(v[0].x, v[1].x), fmaxf(v[2].x, v[3].x));
          const float nt = fmaxf(mt, gt);
          stt *= ex2_approx(mt - nt);
          mt = nt;
#pragma unroll
          for (int j = 0; j < 4; ++j) stt = fmaf(v[j].y, ex2_approx(v[j].x - mt), stt);
        }
      }
      const float l2ss = lg2_approx(ss), l2sl = lg2_approx(sl), l2st = lg2_approx(stt);
      if (lane == 0) {
        RowConsts rc;
        rc.off_small = ms + l2ss;
        rc.off_large = ml + l2sl;
        // logits below the floors give log2 p < -125; the KL variant needs true zeros and clamps nothing
        rc.floor_small = (DIV == kDivKL) ? -INFINITY : (rc.off_small - 125.f) * inv_c;
        rc.floor_large = (DIV == kDivKL) ? -INFINITY : (rc.off_large - 125.f) * inv_c;
        rc.floor2_small = Pairs<T>::floor_bits(rc.floor_small);
        rc.floor2_large = Pairs<T>::floor_bits(rc.floor_large);
        rc.off_third = mt + l2st;
        rc.floor_third = (DIV == kDivKL) ? -INFINITY : (rc.off_third - 125.f) * inv_c;
        rc.floor2_third = Pairs<T>::floor_bits(rc.floor_third);
        rc.pad0 = rc.pad1 = rc.pad2 = 0u;
        ctl->row_consts[d] = rc;
        ctl->row_lse[d] = make_float4(ms, l2ss, ml, l2sl);
        if (TRI) ctl->row_lse3[d] = make_float4(mt, l2st, 0.f, 0.f);
        mbar_arrive(&ctl->b_go[d]);
      }
    };
    auto event_b = [&](int n, bool tri) {
      const int d = n % kClDepth;
      wait_phase(&ctl->b_done[d], (n / kClDepth) & 1u);
      float js = 0.f, big = 0.f, differ = 0.f, js2 = 0.f, big2 = 0.f, differ2 = 0.f;
#pragma unroll
      for (int k = 0; k < kClBWarps; ++k) {   // warp order
        const float4 v = ctl->b_part[d][k];
        js += v.x; big += v.y; differ += v.z;
      }
      if (TRI && tri) {
#pragma unroll
        for (int k = 0; k < kClBWarps; ++k) {
          const float4 v = ctl->b_part2[d][k];
          js2 += v.x; big2 += v.y; differ2 += v.z;
        }
      }
      if (lane == 0) {
        if (rank == 0) mbar_arrive_expect_tx(&ctl->fin_ready[d], static_cast<unsigned>(G.cs) * ((TRI && tri) ? 32u : 16u));
        remote_post_f4(map_to_rank(&ctl->fin_in[d][rank], 0), make_float4(js, big, differ, 0.f),
                       map_to_rank(&ctl->fin_ready[d], 0));
        if (TRI && tri)
          remote_post_f4(map_to_rank(&ctl->fin_in2[d][rank], 0), make_float4(js2, big2, differ2, 0.f),
                         map_to_rank(&ctl->fin_ready[d], 0));
      }
    };
    // statistics record of one pair from its summed pass-B partials and the two models' (m2, l2s)
    auto make_stats = [&](float js, float big, float differ, float m2s, float l2ss, float m2l, float l2sl) {
      RowStats st{};
      int flags = 0;
      if (!(fabsf(m2s + l2ss) < INFINITY)) flags |= kFlagSmallNonfinite;   // NaN, +inf, or no finite logit
      if (!(fabsf(m2l + l2sl) < INFINITY)) flags |= kFlagLargeNonfinite;
      if (flags) {
        st.m2_small = st.l2s_small = st.m2_large = st.l2s_large = st.div = st.resid = __int_as_float(0x7fc00000);
      } else {
        float D;
        const float res = big - 1.f;   // sum max(p,q) - sum q = sum max(0, p - q)
        if (DIV == kDivJS) D = (0.5f * kLn2) * js;   // bits -> nats, and the 1/2 of the definition
        else if (DIV == kDivKL) D = kLn2 * js;
        else D = res;
        st.m2_small = m2s; st.l2s_small = l2ss; st.m2_large = m2l; st.l2s_large = l2sl;
        st.div = fmaxf(D, 0.f);
        st.resid = fmaxf(res, 0.f);
        if (differ == 0.f) { st.div = 0.f; st.resid = 0.f; }   // bitwise identical rows: exactly zero
      }
      st.flags = flags;
      return st;
    };
    auto event_f = [&](int n, const RowWalk& w) {   // rank 0 only
      const int d = n % kClDepth;
      wait_phase(&ctl->fin_ready[d], (n / kClDepth) & 1u);
      if (lane == 0) {
        float js = 0.f, big = 0.f, differ = 0.f;
        for (int j = 0; j < G.cs; ++j) {   // rank order
          const float4 v = ctl->fin_in[d][j];
          js += v.x; big += v.y; differ += v.z;
        }
        const float4 lse = ctl->row_lse[d];
        const RowStats st = make_stats(js, big, differ, lse.x, lse.y, lse.z, lse.w);
        if (w.r < rows1) P.stats[w.r] = st;
        else P.stats2[w.r - rows1] = st;
        if (TRI && w.tri) {
          float js2 = 0.f, big2 = 0.f, differ2 = 0.f;
          for (int j = 0; j < G.cs; ++j) {
            const float4 v = ctl->fin_in2[d][j];
            js2 += v.x; big2 += v.y; differ2 += v.z;
          }
          const float4 lse3 = ctl->row_lse3[d];
          P.stats2[w.r2] = make_stats(js2, big2, differ2, lse.z, lse.w, lse3.x, lse3.y);
        }
      }
    };

    RowWalk w;
    w.init(P, cluster_id, G.n_clusters, TRI);
    if (warp == kClConsumerWarps + 1) {
      // first agent: a(n), g(n) -- the path that releases pass B
      while (w.advance()) {
        // row n reuses the buffers of row n - kClDepth: the second agent must be through with that row
        unsigned spins = 0;
        while (!dead && *reinterpret_cast<volatile int*>(&ctl->rows_closed) < w.n - (kClDepth - 2))
          if (++spins > kClSpinLimit) give_up();
        event_a(w.n, w.tri);
        event_g(w.n, w.tri);
      }
    } else {
      // second agent: b(n), f(n) -- off the critical path
      while (w.advance()) {
        event_b(w.n, w.tri);
        if (rank == 0) event_f(w.n, w);
        __syncwarp();
        if (lane == 0) *reinterpret_cast<volatile int*>(&ctl->rows_closed) = w.n + 1;
      }
    }
  }
  // no CTA may leave while a peer can still write into its shared memory
  __syncthreads();
  cluster_sync_all();
}

// ---- self-test of the give-up path --------------------------------------------------------------------
// One warp waits on a barrier of its own that expects an arrival nobody makes. The wait is the kernels' bounded
// wait with a limit of a few thousand polls; when it runs out the lane records the fact in the status word the
// way give_up() does, and the kernel ends normally.
constexpr unsigned kSelfTestPolls = 2048;
__global__ void wait_timeout_selftest_kernel(int* status) {
  __shared__ unsigned long long bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  unsigned spins = 0;
  bool done = mbar_test(&bar, 0u);
  while (!done && ++spins <= kSelfTestPolls) done = mbar_try(&bar, 0u);
  if (!done) atomicExch(status, 1);
}

// ---- host side --------------------------------------------------------------------------------------
template <typename T, int DIV, bool RS, bool TRI>
inline cudaError_t cluster_prepare_one() {
  cudaError_t e = cudaFuncSetAttribute(rowstats_cluster_kernel<T, DIV, RS, TRI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(kClSmemBytes));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(rowstats_cluster_kernel<T, DIV, RS, TRI>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
}
template <typename T, int DIV>
inline cudaError_t cluster_prepare() {
  cudaError_t e = cluster_prepare_one<T, DIV, false, false>();
  if (e == cudaSuccess) e = cluster_prepare_one<T, DIV, true, false>();
  if (e == cudaSuccess) e = cluster_prepare_one<T, DIV, true, true>();
  return e;
}

// Co-resident clusters of this size. The variants of the kernel have the same shared memory and nearly the
// same block size; the smallest answer is taken so that one cached figure serves all of them.
template <typename T, int DIV, bool RS, bool TRI>
inline int cluster_max_active_one(int cs) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(cs));
  cfg.blockDim = dim3(RS ? kClThreadsRS : kClThreads);
  cfg.dynamicSmemBytes = kClSmemBytes;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = static_cast<unsigned>(cs);
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, rowstats_cluster_kernel<T, DIV, RS, TRI>, &cfg) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return n;
}
template <typename T, int DIV>
inline int cluster_max_active(int cs) {
  return min(min(cluster_max_active_one<T, DIV, false, false>(cs), cluster_max_active_one<T, DIV, true, false>(cs)),
             cluster_max_active_one<T, DIV, true, true>(cs));
}

// Per-device cache of the function attributes and of the number of co-resident clusters the device
// grants per (dtype, divergence kind, cluster size).
constexpr int kClMaxDevices = 64;
struct ClusterDeviceCache {
  bool prepared[2][3];
  int max_active[2][3][kClMaxRanks + 1];   // by cluster size; 0 = not queried yet, -1 = none fit
  int sm_count;
};
inline ClusterDeviceCache* cluster_cache() {
  static ClusterDeviceCache cache[kClMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kClMaxDevices) return nullptr;
  return &cache[dev];
}

template <typename T, int DIV>
inline int cluster_max_active_cached(int dtype, int cs) {
  ClusterDeviceCache* cc = cluster_cache();
  if (cc == nullptr) return 0;
  if (!cc->prepared[dtype][DIV]) {
    if (cluster_prepare<T, DIV>() != cudaSuccess) { cudaGetLastError(); return 0; }
    cc->prepared[dtype][DIV] = true;
  }
  int& slot = cc->max_active[dtype][DIV][cs];
  if (slot == 0) {
    const int n = cluster_max_active<T, DIV>(cs);
    slot = n > 0 ? n : -1;
  }
  return slot > 0 ? slot : 0;
}

inline int cluster_max_active_any(int dtype, int div_kind, int cs) {
  if (dtype == 0) {
    if (div_kind == kDivJS) return cluster_max_active_cached<float, kDivJS>(0, cs);
    if (div_kind == kDivTV) return cluster_max_active_cached<float, kDivTV>(0, cs);
    return cluster_max_active_cached<float, kDivKL>(0, cs);
  }
  if (div_kind == kDivJS) return cluster_max_active_cached<__nv_bfloat16, kDivJS>(1, cs);
  if (div_kind == kDivTV) return cluster_max_active_cached<__nv_bfloat16, kDivTV>(1, cs);
  return cluster_max_active_cached<__nv_bfloat16, kDivKL>(1, cs);
}

inline int cluster_sm_count() {
  ClusterDeviceCache* cc = cluster_cache();
  if (cc == nullptr) return 0;
  if (cc->sm_count == 0) {
    int dev = 0, n = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n = 0;
    cc->sm_count = n;
  }
  return cc->sm_count;
}

// Slice / chunk arithmetic for a vocabulary of V logits split over cs CTAs (pure host arithmetic).
inline void cluster_slices(int V, int elem_bytes, int cs, int* slice, int* chunks) {
  const int vec = 16 / elem_bytes, ch = kClHalfBytes / elem_bytes;
  const int per = (V + cs - 1) / cs;
  *slice = (per + vec - 1) / vec * vec;
  *chunks = (*slice + ch - 1) / ch;
}

// The cluster kernel takes rows that can be copied in 16-byte units: V a multiple of the vector length,
// 16-byte aligned bases and sequence strides, and at least one full vector per row.
inline bool cluster_shape_ok(const StageParams& P, int dtype) {
  const int es = dtype == 0 ? 4 : 2, vec = 16 / es;
  if (P.V < 2048 || (P.V % vec) != 0) return false;
  if ((P.seq_stride_small % vec) != 0 || (P.seq_stride_large % vec) != 0) return false;
  if (((reinterpret_cast<uintptr_t>(P.small) | reinterpret_cast<uintptr_t>(P.large)) & 15u) != 0) return false;
  if (P.K2 > 0) {
    if ((P.seq_stride_small2 % vec) != 0 || (P.seq_stride_large2 % vec) != 0) return false;
    if (((reinterpret_cast<uintptr_t>(P.small2) | reinterpret_cast<uintptr_t>(P.large2)) & 15u) != 0) return false;
  }
  return true;
}

// Picks the cluster size (or takes `forced_cs`; a forced size whose slice exceeds the ring is streamed
// twice), and sizes the grid to the clusters that can be co-resident. Returns false when the shape does not
// fit the kernel.
inline bool cluster_geometry(const StageParams& P, int dtype, int forced_cs, bool force_streamed, bool allow_triples, ClusterGeom* g) {
  if (!cluster_shape_ok(P, dtype)) return false;
  const int es = dtype == 0 ? 4 : 2;
  const long long rows = static_cast<long long>(P.B) * (P.K + P.K2);
  int cs = 0, slice = 0, chunks = 0;
  bool restream = false;
  if (forced_cs > 0) {
    if (forced_cs > kClMaxRanks) return false;
    cs = forced_cs;
    cluster_slices(P.V, es, cs, &slice, &chunks);
    restream = chunks > kClSlots - 1 || force_streamed;   // a slice the ring cannot hold is streamed twice
  } else {
    // the smallest cluster whose slice leaves at least five ring slots beyond a row (measured: 4 CTAs for
    // V = 128256 bf16, 5 for V = 152064 bf16); failing that, three slots
    const int wanted[2] = {kClSlots - 5, kClSlots - 3};
    bool found = false;
    for (int pass = 0; pass < 2 && !found; ++pass)
      for (cs = 1; cs <= (pass == 0 ? 8 : kClMaxRanks); ++cs) {   // sizes above 8 place few clusters: last resort
        cluster_slices(P.V, es, cs, &slice, &chunks);
        if (chunks <= wanted[pass] && cluster_max_active_any(dtype, P.div_kind, cs) > 0) { found = true; break; }
      }
    // few rows: spread each row over more CTAs so that more SMs pull on HBM
    const int sms = cluster_sm_count();
    while (found && cs < 8 && chunks >= 2 && rows * cs * 2 <= sms) {
      cs *= 2;
      cluster_slices(P.V, es, cs, &slice, &chunks);
    }
    // Small clusters fill more SMs (148 with one or two CTAs, 135 with three, 132 with four on B200; eight
    // CTAs place only 120), but for a large vocabulary their slice exceeds the ring and has to be streamed
    // twice. Estimated time = rounds of co-resident clusters / CTAs per row, times a factor fitted to sweeps
    // over the cluster size (V = 128256 and 152064, bf16 and fp32, 1536 to 3072 rows):
    //   resident: 1 + 0.049 per CTA of the cluster (the per-row exchange, and a pipeline that is one row deep);
    //   streamed twice: 1 + 0.056 per CTA; and once the bytes between a slice's first and second copy -- one row
    //   per co-resident cluster -- pass 60 MB, L2 no longer serves the second copy: x 1.5 with fp32 logits, which
    //   then wait for DRAM twice, x 1.08 with bf16 logits, whose arithmetic hides most of it.
    auto rounds_per_cta = [&](int c, int n_active) {
      return static_cast<double>((rows + n_active - 1) / n_active) / c;
    };
    double best = found ? (1.0 + 0.049 * cs) * rounds_per_cta(cs, cluster_max_active_any(dtype, P.div_kind, cs)) : 1e300;
    for (int c2 = 8; c2 >= 1; --c2) {
      int sl2 = 0, ch2 = 0;
      cluster_slices(P.V, es, c2, &sl2, &ch2);
      if (ch2 <= wanted[0]) continue;   // fits the ring with room to spare: the rule above has seen it
      const int na = cluster_max_active_any(dtype, P.div_kind, c2);
      if (na <= 0) continue;
      const double in_flight_mb = 2.0 * sl2 * es * static_cast<double>(na < rows ? na : rows) * c2 / 1048576.0;
      double factor = 1.0 + 0.056 * c2;
      if (in_flight_mb > 60.0) factor *= (es == 4 ? 1.5 : 1.08);
      const double t = factor * rounds_per_cta(c2, na);
      if (t < best) { best = t; cs = c2; slice = sl2; chunks = ch2; restream = true; found = true; }
    }
    if (!found) return false;
  }
  const int max_active = cluster_max_active_any(dtype, P.div_kind, cs);
  if (max_active <= 0) return false;
  g->cs = cs;
  g->slice = slice;
  g->chunks = chunks;
  g->ring = max(chunks + 1, min(kClSlots, 3 * chunks - 1));
  g->ra = 0;
  g->lead = kClDepth;
  if (restream) {
    // slots of two chunks each (32 KB): six of them, `ra` for pass A and the rest for pass B
    g->ring = kClSlots / kClSubRS;
    g->ra = (kClSlots / kClSubRS) / 2;   // measured: 3 + 3 beats 2 + 4 and 4 + 2
    g->lead = kClDepth;                  // measured: a shorter lead changes neither the time nor the DRAM traffic
  }
  // A wrapper launch whose second row set pairs the first set's large rows (the qualifier's, in place) with a
  // third tensor can be walked as row triples where it is streamed twice anyway.
  g->tri = (allow_triples && restream && P.K2 > 0 && P.K2 <= P.K && P.n_valid == nullptr && P.small2 == P.large &&
            P.seq_stride_small2 == P.seq_stride_large) ? 1 : 0;
  const long long items = g->tri ? static_cast<long long>(P.B) * P.K : rows;
  g->n_clusters = static_cast<int>(items < max_active ? items : max_active);
  return g->n_clusters > 0;
}

template <typename T, int DIV>
inline cudaError_t cluster_launch_typed(const StageParams& P, const ClusterGeom& g, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(g.n_clusters * g.cs));
  cfg.blockDim = dim3(g.ra > 0 ? kClThreadsRS : kClThreads);
  cfg.dynamicSmemBytes = kClSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = static_cast<unsigned>(g.cs);
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  if (g.ra > 0 && g.tri) return cudaLaunchKernelEx(&cfg, rowstats_cluster_kernel<T, DIV, true, true>, P, g);
  if (g.ra > 0) return cudaLaunchKernelEx(&cfg, rowstats_cluster_kernel<T, DIV, true, false>, P, g);
  return cudaLaunchKernelEx(&cfg, rowstats_cluster_kernel<T, DIV, false, false>, P, g);
}

// Launches the statistics pass with the cluster kernel. Returns 0, or -2 when the launch was refused.
inline int launch_rowstats_cluster(const StageParams& P, int dtype, const ClusterGeom& g, cudaStream_t stream) {
  cudaError_t e;
  if (dtype == 0) {
    if (P.div_kind == kDivJS) e = cluster_launch_typed<float, kDivJS>(P, g, stream);
    else if (P.div_kind == kDivTV) e = cluster_launch_typed<float, kDivTV>(P, g, stream);
    else e = cluster_launch_typed<float, kDivKL>(P, g, stream);
  } else {
    if (P.div_kind == kDivJS) e = cluster_launch_typed<__nv_bfloat16, kDivJS>(P, g, stream);
    else if (P.div_kind == kDivTV) e = cluster_launch_typed<__nv_bfloat16, kDivTV>(P, g, stream);
    else e = cluster_launch_typed<__nv_bfloat16, kDivKL>(P, g, stream);
  }
  return e == cudaSuccess ? 0 : -2;
}

}  // namespace psd
