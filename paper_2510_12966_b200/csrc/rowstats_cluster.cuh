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
// the ring holds more than one row slice, each warp runs pass A ahead of pass B for as long as loaded
// chunks are available, and an agent warp carries partials between CTAs. Warps are independent of each
// other; they meet only on mbarriers (chunk landed / chunk free / row partials complete).
//
// Roles: warps 0..15 consumers (each owns 32 consecutive 16-byte vectors of every chunk), warp 16 lane 0
// issues the bulk copies, warp 17 is the agent (reduces the warps' partials, talks to the peers; on
// rank 0 it also writes the row's RowStats). Every wait is bounded: on giving up a thread records
// PSD_ERR_TIMEOUT in the status word and stops waiting, so the kernel always terminates.
#pragma once

#include "common.cuh"

namespace psd {

constexpr int kClConsumerWarps = 16;
constexpr int kClConsumers = kClConsumerWarps * 32;
constexpr int kClThreads = kClConsumers + 64;      // + loader warp + agent warp
constexpr int kClHalfBytes = 8192;                 // one model's part of a chunk: 512 threads x 16 bytes
constexpr int kClSlotBytes = 2 * kClHalfBytes;
constexpr int kClSlots = 13;                       // ring slots
constexpr int kClDepth = 4;                        // rows of exchange buffers in flight
constexpr int kClMaxRanks = 16;
constexpr unsigned kClSpinLimit = 1u << 22;        // polls before a wait gives up (a fraction of a second at the least)

struct ClusterGeom {
  int cs;        // CTAs per cluster
  int slice;     // vocabulary indices per CTA (multiple of the 16-byte vector)
  int chunks;    // chunks per slice
  int ring;      // ring slots in use: min(kClSlots, 3 * chunks - 1), at least chunks + 1
  int n_clusters;
};

// Shared-memory control block behind the ring.
struct __align__(16) ClusterCtl {
  unsigned long long full[kClSlots];
  unsigned long long empty[kClSlots];
  unsigned long long a_done[kClDepth], b_done[kClDepth], lse_ready[kClDepth], fin_ready[kClDepth];
  float4 a_part[kClDepth][kClConsumerWarps];       // (ref_small, sum_small, ref_large, sum_large) per warp
  double b_part[kClDepth][kClConsumerWarps][4];    // (sum p*a + q*b, sum s*lg s, sum max(p,q), differ bits)
  float4 row_lse[kClDepth];                        // (m2_small, l2s_small, m2_large, l2s_large) of the row
  float4 lse_in[kClDepth][kClMaxRanks];            // partials received from every rank of the cluster
  double fin_in[kClDepth][kClMaxRanks][4];         // pass-B partials received (rank 0 only)
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
__device__ __forceinline__ bool mbar_test(unsigned long long* bar, unsigned parity) {
  unsigned ok;
  asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// same, observing writes made by other CTAs of the cluster before their arrive
__device__ __forceinline__ bool mbar_test_cluster(unsigned long long* bar, unsigned parity) {
  unsigned ok;
  asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned map_to_rank(const void* local, unsigned rank) {
  unsigned r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(local)), "r"(rank));
  return r;
}
__device__ __forceinline__ void remote_arrive(unsigned cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void remote_store_f4(unsigned cluster_addr, float4 v) {
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ void remote_store_d2(unsigned cluster_addr, double a, double b) {
  asm volatile("st.shared::cluster.v2.f64 [%0], {%1, %2};" ::"r"(cluster_addr), "d"(a), "d"(b) : "memory");
}
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, unsigned bytes, unsigned long long* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)) : "memory");
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
struct RowWalk {
  int next_r, stride, rows, K;
  const int32_t* n_valid;
  int n;     // ordinal of the current row among the rows this cluster takes
  int r;     // current row index (valid after advance() returned true)
  __device__ void init(const StageParams& P, int cluster_id, int n_clusters) {
    next_r = cluster_id; stride = n_clusters; rows = P.B * P.K; K = P.K; n_valid = P.n_valid; n = -1; r = -1;
  }
  __device__ bool advance() {
    while (next_r < rows) {
      const int cand = next_r;
      next_r += stride;
      if (n_valid != nullptr) {
        const int b = cand / K, k = cand - b * K;
        if (k >= n_valid[b]) continue;
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

// ---- pass A: streaming log-sum-exp -------------------------------------------------------------------
// State per thread and model: a reference `ref` (in the scaled base-2 domain), the sum S of 2^(x*c - ref)
// and `thr`, the largest logit that may still be added without moving the reference (ref + 64 in the
// scaled domain). The reference starts at a finite floor so that -inf logits give exactly 0.
struct LseState {
  float ref, thr, s0, s1;
  __device__ __forceinline__ void reset(float inv_c) { ref = -1e30f; thr = (-1e30f + 64.f) * inv_c; s0 = 0.f; s1 = 0.f; }
};

template <int E>
__device__ __forceinline__ void lse_accumulate(const float (&x)[E], float c, float inv_c, LseState& st) {
  float gm = x[0];
#pragma unroll
  for (int j = 1; j < E; ++j) gm = fmaxf(gm, x[j]);
  if (gm > st.thr) {  // rare: the group holds a logit far above the reference (always true for the first finite group)
    const float nr = gm * c;
    const float sc = ex2_approx(st.ref - nr);
    st.s0 *= sc; st.s1 *= sc;
    st.ref = nr;
    st.thr = gm + 64.f * inv_c;
  }
#pragma unroll
  for (int j = 0; j < E; j += 2) {
    st.s0 += ex2_approx(fmaf(x[j], c, -st.ref));
    st.s1 += ex2_approx(fmaf(x[j + 1], c, -st.ref));
  }
}

// Combine (ref, S) partials: returns the pair for the union. Fixed order, NaN-preserving in S.
__device__ __forceinline__ void lse_merge(float& ref, float& s, float oref, float os) {
  const float m = fmaxf(ref, oref);
  s = s * ex2_approx(ref - m) + os * ex2_approx(oref - m);
  ref = m;
}

// ---- pass B accumulators ----------------------------------------------------------------------------
struct DivAcc {
  float pa, qb, sl, big;
  unsigned differ;
  __device__ __forceinline__ void reset() { pa = qb = sl = big = 0.f; differ = 0u; }
};

template <int DIV, int E>
__device__ __forceinline__ void div_accumulate(const float (&xl_in)[E], const float (&xs_in)[E], float c, float off_l,
                                               float off_s, DivAcc& acc) {
#pragma unroll
  for (int j = 0; j < E; ++j) {
    // -inf (masked vocabulary) and huge negative logits: clamp so that 0 * log 0 stays 0
    const float xl = fmaxf(xl_in[j], -1e30f), xs = fmaxf(xs_in[j], -1e30f);
    const float a = fmaf(xl, c, -off_l), b = fmaf(xs, c, -off_s);   // log2 p, log2 q
    const float p = ex2_approx(a), q = ex2_approx(b);
    acc.big += fmaxf(p, q);
    if (DIV == kDivJS) {
      const float s = p + q;
      const float l = lg2_approx(s + 1e-36f);
      acc.pa = fmaf(p, a, acc.pa);
      acc.qb = fmaf(q, b, acc.qb);
      acc.sl = fmaf(s, l, acc.sl);
    } else if (DIV == kDivKL) {
      // p * (log2 p - log2 q); q == 0 with p > 0 gives +inf, as it should
      if (p > 0.f) acc.pa = (q > 0.f) ? fmaf(p, a - b, acc.pa) : INFINITY;
    }
  }
}

template <typename V>
__device__ __forceinline__ V warp_sum(V v) { return warp_reduce<OpSum>(v); }

// ---- the kernel -------------------------------------------------------------------------------------
template <typename T, int DIV>
__global__ void __launch_bounds__(kClThreads, 1) rowstats_cluster_kernel(const StageParams P, const ClusterGeom G) {
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

  if (tid == 0) {
    for (int s = 0; s < kClSlots; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], kClConsumerWarps); }
    for (int d = 0; d < kClDepth; ++d) {
      mbar_init(&ctl->a_done[d], kClConsumerWarps);
      mbar_init(&ctl->b_done[d], kClConsumerWarps);
      mbar_init(&ctl->lse_ready[d], G.cs);
      mbar_init(&ctl->fin_ready[d], G.cs);
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

  if (warp < kClConsumerWarps) {
    // ================================ consumers ================================
    const float c = P.c, inv_c = 1.f / P.c;
    RowWalk wa, wb;
    wa.init(P, cluster_id, G.n_clusters);
    wb.init(P, cluster_id, G.n_clusters);
    bool a_row = wa.advance(), b_row = wb.advance();
    int ca = 0, cb = 0;          // chunk inside the current row of each pass
    unsigned ga = 0, gb = 0;     // chunks finished by each pass since kernel start
    bool b_ready = false;        // normalisers of pass B's current row are in registers
    float off_l = 0.f, off_s = 0.f;
    LseState ls, ll;
    ls.reset(inv_c); ll.reset(inv_c);
    DivAcc acc;
    acc.reset();
    const int vec_in_chunk = warp * 32 + lane;
    unsigned idle = 0;

    while (b_row) {
      bool progressed = false;
      // ---- pass A on the next chunk, if it has landed ----
      if (a_row) {
        const unsigned slot = ga % R;
        if (dead || mbar_test(&ctl->full[slot], (ga / R) & 1u)) {
          const int e0 = ca * CH + vec_in_chunk * E;
          if (e0 < slice_len) {
            const unsigned char* base = ring + static_cast<size_t>(slot) * kClSlotBytes + vec_in_chunk * 16;
            float xs[E], xl[E];
            Elem<T>::unpack(lds128(base), xs);
            Elem<T>::unpack(lds128(base + kClHalfBytes), xl);
            lse_accumulate<E>(xs, c, inv_c, ls);
            lse_accumulate<E>(xl, c, inv_c, ll);
          }
          ++ga;
          if (++ca == C) {
            // row finished: warp partial -> a_part, then tell the agent
            float rs = ls.ref, ss = ls.s0 + ls.s1, rl = ll.ref, sl = ll.s0 + ll.s1;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
              lse_merge(rs, ss, __shfl_xor_sync(0xffffffffu, rs, o), __shfl_xor_sync(0xffffffffu, ss, o));
              lse_merge(rl, sl, __shfl_xor_sync(0xffffffffu, rl, o), __shfl_xor_sync(0xffffffffu, sl, o));
            }
            const int d = wa.n % kClDepth;
            if (lane == 0) {
              ctl->a_part[d][warp] = make_float4(rs, ss, rl, sl);
              mbar_arrive(&ctl->a_done[d]);
            }
            ls.reset(inv_c); ll.reset(inv_c);
            ca = 0;
            a_row = wa.advance();
          }
          progressed = true;
        }
      }
      // ---- pass B on its next chunk, if pass A has been there and the row's normalisers are known ----
      if (gb < ga) {
        const int d = wb.n % kClDepth;
        if (!b_ready && (dead || mbar_test_cluster(&ctl->lse_ready[d], (wb.n / kClDepth) & 1u))) {
          float ms = -INFINITY, ml = -INFINITY;
          for (int j = 0; j < G.cs; ++j) { ms = fmaxf(ms, ctl->lse_in[d][j].x); ml = fmaxf(ml, ctl->lse_in[d][j].z); }
          float ss = 0.f, sl = 0.f;
          for (int j = 0; j < G.cs; ++j) {
            const float4 v = ctl->lse_in[d][j];
            ss += v.y * ex2_approx(v.x - ms);
            sl += v.w * ex2_approx(v.z - ml);
          }
          const float l2ss = lg2_approx(ss), l2sl = lg2_approx(sl);
          off_s = ms + l2ss;
          off_l = ml + l2sl;
          if (warp == 0 && lane == 0) ctl->row_lse[d] = make_float4(ms, l2ss, ml, l2sl);
          b_ready = true;
        }
        if (b_ready) {
          const unsigned slot = gb % R;
          const int e0 = cb * CH + vec_in_chunk * E;
          if (e0 < slice_len) {
            const unsigned char* base = ring + static_cast<size_t>(slot) * kClSlotBytes + vec_in_chunk * 16;
            const uint4 us = lds128(base), ul = lds128(base + kClHalfBytes);
            acc.differ |= (us.x ^ ul.x) | (us.y ^ ul.y) | (us.z ^ ul.z) | (us.w ^ ul.w);
            float xs[E], xl[E];
            Elem<T>::unpack(us, xs);
            Elem<T>::unpack(ul, xl);
            div_accumulate<DIV, E>(xl, xs, c, off_l, off_s, acc);
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(&ctl->empty[slot]);   // this warp is done with the slot
          ++gb;
          if (++cb == C) {
            const double pab = warp_sum(static_cast<double>(acc.pa) + static_cast<double>(acc.qb));
            const double sl = warp_sum(static_cast<double>(acc.sl));
            const double big = warp_sum(static_cast<double>(acc.big));
            const unsigned differ = __reduce_or_sync(0xffffffffu, acc.differ);
            if (lane == 0) {
              ctl->b_part[d][warp][0] = pab;
              ctl->b_part[d][warp][1] = sl;
              ctl->b_part[d][warp][2] = big;
              ctl->b_part[d][warp][3] = differ ? 1.0 : 0.0;
              mbar_arrive(&ctl->b_done[d]);
            }
            acc.reset();
            cb = 0;
            b_ready = false;
            b_row = wb.advance();
          }
          progressed = true;
        }
      }
      if (progressed) idle = 0;
      else if (!dead && ++idle > kClSpinLimit) give_up();
    }
  } else if (warp == kClConsumerWarps) {
    // ================================ loader ================================
    if (lane == 0) {
      RowWalk w;
      w.init(P, cluster_id, G.n_clusters);
      unsigned g = 0;
      while (w.advance()) {
        const T* rs = row_ptr<T>(P.small, P.seq_stride_small, w.r, K, V) + slice_begin;
        const T* rl = row_ptr<T>(P.large, P.seq_stride_large, w.r, K, V) + slice_begin;
        for (int cidx = 0; cidx < C; ++cidx, ++g) {
          const unsigned slot = g % R;
          if (g >= static_cast<unsigned>(R)) {
            const unsigned parity = ((g / R) - 1u) & 1u;
            unsigned spins = 0;
            while (!dead && !mbar_test(&ctl->empty[slot], parity))
              if (++spins > kClSpinLimit) give_up();
          }
          const int e0 = cidx * CH;
          const int n = min(CH, slice_len - e0);
          if (n > 0) {
            const unsigned bytes = static_cast<unsigned>(n) * sizeof(T);
            unsigned char* dst = ring + static_cast<size_t>(slot) * kClSlotBytes;
            mbar_arrive_expect_tx(&ctl->full[slot], 2u * bytes);
            bulk_load(dst, rs + e0, bytes, &ctl->full[slot]);
            bulk_load(dst + kClHalfBytes, rl + e0, bytes, &ctl->full[slot]);
          } else {
            mbar_arrive(&ctl->full[slot]);   // nothing of this chunk falls into this CTA's slice
          }
        }
      }
      // every copy issued above is waited for by pass A of the consumers before they leave
    }
  } else {
    // ================================ agent ================================
    RowWalk wa, wb, wf;
    wa.init(P, cluster_id, G.n_clusters);
    wb.init(P, cluster_id, G.n_clusters);
    wf.init(P, cluster_id, G.n_clusters);
    bool a_row = wa.advance(), b_row = wb.advance();
    bool f_row = (rank == 0) ? wf.advance() : false;
    unsigned idle = 0;
    // Events are taken in row order within each kind. A row's exchange buffers are reused kClDepth rows
    // later, and nothing of row m + kClDepth can be produced anywhere in the cluster before this agent has
    // sent the pass-A partial of that row; so that partial is held back until the pass-B partial of row m
    // has been forwarded (and, on rank 0, row m's statistics written).
    int na = 0, nb = 0, nf = 0;
    while (a_row || b_row || f_row) {
      bool progressed = false;
      if (a_row && na - nb < kClDepth - 1 && (rank != 0 || na - nf < kClDepth - 1)) {
        const int d = wa.n % kClDepth;
        if (dead || mbar_test(&ctl->a_done[d], (wa.n / kClDepth) & 1u)) {
          // reduce the 16 warp partials (fixed tree) and hand the CTA's partial to every rank
          float4 v = (lane < kClConsumerWarps) ? ctl->a_part[d][lane] : make_float4(-1e30f, 0.f, -1e30f, 0.f);
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            lse_merge(v.x, v.y, __shfl_xor_sync(0xffffffffu, v.x, o), __shfl_xor_sync(0xffffffffu, v.y, o));
            lse_merge(v.z, v.w, __shfl_xor_sync(0xffffffffu, v.z, o), __shfl_xor_sync(0xffffffffu, v.w, o));
          }
          if (lane < G.cs) {
            remote_store_f4(map_to_rank(&ctl->lse_in[d][rank], lane), v);
            remote_arrive(map_to_rank(&ctl->lse_ready[d], lane));
          }
          a_row = wa.advance();
          ++na;
          progressed = true;
        }
      }
      if (b_row && nb < na) {
        const int d = wb.n % kClDepth;
        if (dead || mbar_test(&ctl->b_done[d], (wb.n / kClDepth) & 1u)) {
          double v0 = 0.0, v1 = 0.0, v2 = 0.0, v3 = 0.0;
          if (lane < kClConsumerWarps) {
            v0 = ctl->b_part[d][lane][0]; v1 = ctl->b_part[d][lane][1];
            v2 = ctl->b_part[d][lane][2]; v3 = ctl->b_part[d][lane][3];
          }
          v0 = warp_sum(v0); v1 = warp_sum(v1); v2 = warp_sum(v2); v3 = warp_sum(v3);
          if (lane == 0) {
            const unsigned dst = map_to_rank(&ctl->fin_in[d][rank][0], 0);
            remote_store_d2(dst, v0, v1);
            remote_store_d2(dst + 16, v2, v3);
            remote_arrive(map_to_rank(&ctl->fin_ready[d], 0));
          }
          b_row = wb.advance();
          ++nb;
          progressed = true;
        }
      }
      if (f_row && nf < nb) {
        const int d = wf.n % kClDepth;
        if (dead || mbar_test_cluster(&ctl->fin_ready[d], (wf.n / kClDepth) & 1u)) {
          if (lane == 0) {
            double pab = 0.0, sl = 0.0, big = 0.0, differ = 0.0;
            for (int j = 0; j < G.cs; ++j) {
              pab += ctl->fin_in[d][j][0]; sl += ctl->fin_in[d][j][1];
              big += ctl->fin_in[d][j][2]; differ += ctl->fin_in[d][j][3];
            }
            const float4 lse = ctl->row_lse[d];
            RowStats st{};
            int flags = 0;
            if (!(fabsf(lse.x + lse.y) < INFINITY)) flags |= kFlagSmallNonfinite;   // NaN, +inf, or no finite logit
            if (!(fabsf(lse.z + lse.w) < INFINITY)) flags |= kFlagLargeNonfinite;
            if (flags) {
              st.m2_small = st.l2s_small = st.m2_large = st.l2s_large = st.div = st.resid = __int_as_float(0x7fc00000);
            } else {
              double D;
              const double res = big - 1.0;   // sum max(p,q) - sum q = sum max(0, p - q)
              if (DIV == kDivJS) D = 0.5 * 0.6931471805599453 * (pab - sl + 2.0);   // sum s*(lg s - 1) = sl - 2
              else if (DIV == kDivKL) D = 0.6931471805599453 * pab;
              else D = res;
              st.m2_small = lse.x; st.l2s_small = lse.y; st.m2_large = lse.z; st.l2s_large = lse.w;
              st.div = fmaxf(static_cast<float>(D), 0.f);
              st.resid = fmaxf(static_cast<float>(res), 0.f);
              if (differ == 0.0) { st.div = 0.f; st.resid = 0.f; }   // bitwise identical rows: exactly zero
            }
            st.flags = flags;
            P.stats[wf.r] = st;
          }
          f_row = wf.advance();
          ++nf;
          progressed = true;
        }
      }
      if (progressed) idle = 0;
      else if (!dead && ++idle > kClSpinLimit) give_up();
    }
  }
  // no CTA may leave while a peer can still write into its shared memory
  __syncthreads();
  cluster_sync_all();
}

// ---- host side --------------------------------------------------------------------------------------
template <typename T, int DIV>
inline cudaError_t cluster_prepare() {
  cudaError_t e = cudaFuncSetAttribute(rowstats_cluster_kernel<T, DIV>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(kClSmemBytes));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(rowstats_cluster_kernel<T, DIV>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
}

template <typename T, int DIV>
inline int cluster_max_active(int cs) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(cs));
  cfg.blockDim = dim3(kClThreads);
  cfg.dynamicSmemBytes = kClSmemBytes;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = static_cast<unsigned>(cs);
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, rowstats_cluster_kernel<T, DIV>, &cfg) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return n;
}

// Per-device cache of the function attributes and of the number of co-resident clusters the device
// grants per (dtype, divergence kind, cluster size).
constexpr int kClMaxDevices = 64;
struct ClusterDeviceCache {
  bool prepared[2][3];
  int max_active[2][3][5];   // 0 = not queried yet, -1 = none fit
  int sm_count;
};
inline ClusterDeviceCache* cluster_cache() {
  static ClusterDeviceCache cache[kClMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kClMaxDevices) return nullptr;
  return &cache[dev];
}

template <typename T, int DIV>
inline int cluster_max_active_cached(int dtype, int log2cs) {
  ClusterDeviceCache* cc = cluster_cache();
  if (cc == nullptr) return 0;
  if (!cc->prepared[dtype][DIV]) {
    if (cluster_prepare<T, DIV>() != cudaSuccess) { cudaGetLastError(); return 0; }
    cc->prepared[dtype][DIV] = true;
  }
  int& slot = cc->max_active[dtype][DIV][log2cs];
  if (slot == 0) {
    const int n = cluster_max_active<T, DIV>(1 << log2cs);
    slot = n > 0 ? n : -1;
  }
  return slot > 0 ? slot : 0;
}

inline int cluster_max_active_any(int dtype, int div_kind, int log2cs) {
  if (dtype == 0) {
    if (div_kind == kDivJS) return cluster_max_active_cached<float, kDivJS>(0, log2cs);
    if (div_kind == kDivTV) return cluster_max_active_cached<float, kDivTV>(0, log2cs);
    return cluster_max_active_cached<float, kDivKL>(0, log2cs);
  }
  if (div_kind == kDivJS) return cluster_max_active_cached<__nv_bfloat16, kDivJS>(1, log2cs);
  if (div_kind == kDivTV) return cluster_max_active_cached<__nv_bfloat16, kDivTV>(1, log2cs);
  return cluster_max_active_cached<__nv_bfloat16, kDivKL>(1, log2cs);
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
  return true;
}

// Picks the cluster size (or takes `forced_cs`), and sizes the grid to the clusters that can be
// co-resident. Returns false when the shape does not fit the kernel.
inline bool cluster_geometry(const StageParams& P, int dtype, int forced_cs, ClusterGeom* g) {
  if (!cluster_shape_ok(P, dtype)) return false;
  const int es = dtype == 0 ? 4 : 2;
  const long long rows = static_cast<long long>(P.B) * P.K;
  int cs = 0, slice = 0, chunks = 0;
  if (forced_cs > 0) {
    if (forced_cs > kClMaxRanks || (forced_cs & (forced_cs - 1)) != 0) return false;
    cs = forced_cs;
    cluster_slices(P.V, es, cs, &slice, &chunks);
    if (chunks > kClSlots - 1) return false;
  } else {
    for (cs = 1; cs <= kClMaxRanks; cs *= 2) {
      cluster_slices(P.V, es, cs, &slice, &chunks);
      if (chunks <= kClSlots - 3) break;
    }
    if (cs > kClMaxRanks) return false;
    // few rows: spread each row over more CTAs so that more SMs pull on HBM
    const int sms = cluster_sm_count();
    while (cs < 8 && chunks >= 2 && rows * cs * 2 <= sms) {
      cs *= 2;
      cluster_slices(P.V, es, cs, &slice, &chunks);
    }
  }
  int log2cs = 0;
  while ((1 << log2cs) < cs) ++log2cs;
  const int max_active = cluster_max_active_any(dtype, P.div_kind, log2cs);
  if (max_active <= 0) return false;
  g->cs = cs;
  g->slice = slice;
  g->chunks = chunks;
  g->ring = max(chunks + 1, min(kClSlots, 3 * chunks - 1));
  g->n_clusters = static_cast<int>(rows < max_active ? rows : max_active);
  return g->n_clusters > 0;
}

template <typename T, int DIV>
inline cudaError_t cluster_launch_typed(const StageParams& P, const ClusterGeom& g, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(g.n_clusters * g.cs));
  cfg.blockDim = dim3(kClThreads);
  cfg.dynamicSmemBytes = kClSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = static_cast<unsigned>(g.cs);
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, rowstats_cluster_kernel<T, DIV>, P, g);
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
