// Row statistics in ONE pass over the logits, for the divergence whose terms separate: KL(P_large || P_small)
// (one of the selectable divergences of Sec. 3.1's `Div`). With a = log2 p_i and b = log2 q_i linear in the
// logits once the two normalisers L_l, L_s (base-2 log-sum-exps) are known,
//     sum_i p_i (a_i - b_i)  =  c * T / S_l - (L_l - L_s),   T = sum_i e_i (z_l,i - z_s,i),   e_i = 2^(z_l,i c - ref_l),
//     S_l = sum_i e_i,
// so T and both log-sum-exps are gathered in the same sweep: two ex2 per vocabulary index instead of the four of
// the two-pass kernel, and every logit read once. One persistent CTA per SM takes whole rows (no cluster: there is
// no second pass whose copy would have to come out of L2), bulk copies feed a shared-memory ring, sixteen warps
// consume it, one warp loads, one merges the warps' partials of a row and writes its statistics. The residual
// mass sum max(0, p - q) does not separate; a caller that wants it per row gets the two-pass kernel. The
// finalisation needs it only to tell an exactly zero residual from a positive one, which its draw finds out by
// itself, so the record carries a positive stand-in.
#pragma once

#include "rowstats_cluster.cuh"

namespace psd {

constexpr int kOpWarps = 16;                                    // consumer warps
constexpr int kOpThreads = (kOpWarps + 2) * 32;                 // + loader warp + finisher warp
constexpr int kOpVec = 2;                                       // 16-byte vectors per lane, step and model
constexpr int kOpHalfBytes = kOpWarps * 32 * 16 * kOpVec;       // one model's part of a step: 16 KB
constexpr int kOpRingBytes = 12 * kOpHalfBytes;                 // 192 KB: six slots of a pair, four of a triple
constexpr float kOpResidUnknown = 1.0f;                         // RowStats.resid of this kernel: "positive unless the draw finds otherwise"

struct __align__(16) OpCtl {
  unsigned long long full[6], empty[6];
  unsigned long long part_done[2], part_free[2];   // the warps' partials of a row are in / have been read (rows alternate)
  float4 part[2][kOpWarps];                        // (ref_0, S_0, ref_1, S_1) per warp: the pair's small and large model
  float4 part_x[2][kOpWarps];                      // (T_10, T_21, ref_2, S_2): the cross sums, and a triple's third model
};
constexpr size_t kOpSmemBytes = static_cast<size_t>(kOpRingBytes) + sizeof(OpCtl) + 128;

// TRI: the launch is a two-stage wrapper's, walked as row triples (draft, qualifier, target) for the positions both
// stages verify and as pairs (draft, qualifier) beyond them: the qualifier's row, stage 1's large model and stage
// 2's small one (Fig. 1), is read and exponentiated once. A model's share of a step, and with it the order of every
// sum, is the same in both forms, so they return the same bits.
template <typename T, bool TRI>
__global__ void __launch_bounds__(kOpThreads, 1) rowstats_kl_onepass_kernel(const StageParams P) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  OpCtl* ctl = reinterpret_cast<OpCtl*>(ring + static_cast<size_t>(kOpRingBytes));

  constexpr int E = Elem<T>::kPerVec;
  constexpr int CH = kOpHalfBytes / sizeof(T);   // logits per step and model
  constexpr int kMaxModels = TRI ? 3 : 2;
  constexpr int kSlotBytes = kMaxModels * kOpHalfBytes;
  constexpr int kSlots = kOpRingBytes / kSlotBytes;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int V = P.V, K = P.K;
  const int rows1 = P.B * K;
  const int steps = (V + CH - 1) / CH;

  if (tid == 0) {
    for (int s = 0; s < kSlots; ++s) {
      mbar_init(&ctl->full[s], 1);
      mbar_init(&ctl->empty[s], kOpWarps);
    }
    for (int d = 0; d < 2; ++d) {
      mbar_init(&ctl->part_done[d], kOpWarps);
      mbar_init(&ctl->part_free[d], 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  release_dependent_launch();

  bool dead = false;    // this thread gave up on a wait: stop waiting, just run to the end
  auto give_up = [&]() {
    dead = true;
    atomicExch(P.status, 1);
  };
  auto wait_phase = [&](unsigned long long* bar, unsigned parity) {
    if (mbar_test(bar, parity)) return;
    unsigned spins = 0;
    while (!dead && !mbar_try(bar, parity))
      if (++spins > kClSpinLimit) give_up();
  };
  // model m of the walk's current item: 0 the pair's small model, 1 its large one, 2 (triples) the target
  auto model_row = [&](const RowWalk& w, int m) -> const T* {
    if (TRI) {
      if (m == 0) return row_ptr<T>(P.small, P.seq_stride_small, w.r, K, V);
      if (m == 1) return row_ptr<T>(P.large, P.seq_stride_large, w.r, K, V);
      return row_ptr<T>(P.large2, P.seq_stride_large2, w.r2, P.K2, V);
    }
    const bool second = w.r >= rows1;   // second row set: stage 2 of the wrapper
    if (m == 0) return second ? row_ptr<T>(P.small2, P.seq_stride_small2, w.r - rows1, P.K2, V)
                              : row_ptr<T>(P.small, P.seq_stride_small, w.r, K, V);
    return second ? row_ptr<T>(P.large2, P.seq_stride_large2, w.r - rows1, P.K2, V)
                  : row_ptr<T>(P.large, P.seq_stride_large, w.r, K, V);
  };
  RowWalk w;
  w.init(P, blockIdx.x, gridDim.x, TRI);

  if (warp < kOpWarps) {
    // ================================ consumers ================================
    const float c = P.c;
    const unsigned char* my = ring + (warp * 32 + lane) * 16;
    constexpr int kVecStride = kOpWarps * 32 * 16;   // bytes between a lane's vectors
    int len[kOpVec];   // > step offset while vector i of this lane lies inside the row
#pragma unroll
    for (int i = 0; i < kOpVec; ++i) len[i] = V - (warp * 32 + lane + i * kOpWarps * 32) * E;
    unsigned slot = 0, par = 0;
    // One row of NM models. Per model m a reference per warp and S_m = sum 2^(z_m c - ref_m); per neighbouring pair
    // T_(m+1,m) = sum 2^(z_(m+1) c - ref_(m+1)) (z_(m+1) - z_m), the cross sum of KL(model m+1 || model m).
    auto row = [&](auto nm_c) {
      constexpr int NM = decltype(nm_c)::value;
      float ref[NM], ss[NM], tt[NM - 1];
#pragma unroll
      for (int m = 0; m < NM; ++m) { ref[m] = -1e30f; ss[m] = 0.f; }
#pragma unroll
      for (int m = 0; m < NM - 1; ++m) tt[m] = 0.f;
      // one vector of every model into the sums
      auto add_vectors = [&](const uint4 (&u)[NM], bool live) {
        float x[NM][E];
#pragma unroll
        for (int m = 0; m < NM; ++m) Elem<T>::unpack(u[m], x[m]);
        float a[NM], t[NM - 1];
#pragma unroll
        for (int m = 0; m < NM; ++m) a[m] = 0.f;
#pragma unroll
        for (int m = 0; m < NM - 1; ++m) t[m] = 0.f;
#pragma unroll
        for (int j = 0; j < E; ++j) {
          float e[NM];
#pragma unroll
          for (int m = 0; m < NM; ++m) {
            e[m] = ex2_approx(fmaf(x[m][j], c, -ref[m]));
            a[m] += e[m];
          }
#pragma unroll
          for (int m = 0; m < NM - 1; ++m)   // q_i = 0 under p_i > 0 gives +inf, as it should; p_i = 0 adds nothing
            if (e[m + 1] > 0.f) t[m] = fmaf(e[m + 1], x[m + 1][j] - x[m][j], t[m]);
        }
        if (live) {
#pragma unroll
          for (int m = 0; m < NM; ++m) ss[m] += a[m];
#pragma unroll
          for (int m = 0; m < NM - 1; ++m) tt[m] += t[m];
        }
      };
      // the warp's references from the maxima of the vectors `first` (the floor keeps rows that start with -inf at 0)
      auto take_refs = [&](float (&g)[NM]) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
#pragma unroll
          for (int m = 0; m < NM; ++m) g[m] = fmaxf(g[m], __shfl_xor_sync(0xffffffffu, g[m], o));
#pragma unroll
        for (int m = 0; m < NM; ++m) ref[m] = fmaxf(g[m] * c, -1e30f);
      };
      int off = 0;
      for (int step = 0; step < steps; ++step, off += CH) {
        wait_phase(&ctl->full[slot], par);
        const unsigned char* base = my + slot * kSlotBytes;
        uint4 u[kOpVec][NM];
#pragma unroll
        for (int i = 0; i < kOpVec; ++i)
#pragma unroll
          for (int m = 0; m < NM; ++m) u[i][m] = lds128(base + m * kOpHalfBytes + i * kVecStride);
        if (step == 0) {
          float g[NM];
#pragma unroll
          for (int m = 0; m < NM; ++m) g[m] = vector_max<T>(u[0][m], len[0] > 0);
          take_refs(g);
        }
#pragma unroll
        for (int i = 0; i < kOpVec; ++i) add_vectors(u[i], len[i] > off);
        __syncwarp();
        if (lane == 0) mbar_arrive(&ctl->empty[slot]);
        if (++slot == kSlots) { slot = 0; par ^= 1u; }
      }
      float tot = 0.f;
#pragma unroll
      for (int m = 0; m < NM; ++m) tot += ss[m];
      if (__any_sync(0xffffffffu, !(tot < INFINITY))) {
        // A sum left the range of a float (a logit far above the warp's first vectors), or the row holds a NaN or
        // +inf: the warp takes its share of the row again from global memory, against its true maxima.
        const T* src[NM];
#pragma unroll
        for (int m = 0; m < NM; ++m) src[m] = model_row(w, m);
        float g[NM];
#pragma unroll
        for (int m = 0; m < NM; ++m) g[m] = -INFINITY;
        for (int e0 = 0; e0 < V; e0 += CH)
          for (int i = 0; i < kOpVec; ++i) {
            const int e = e0 + (warp * 32 + lane + i * kOpWarps * 32) * E;
            if (e < V) {
#pragma unroll
              for (int m = 0; m < NM; ++m) g[m] = fmaxf(g[m], vector_max<T>(*reinterpret_cast<const uint4*>(src[m] + e), true));
            }
          }
        take_refs(g);
#pragma unroll
        for (int m = 0; m < NM; ++m) ss[m] = 0.f;
#pragma unroll
        for (int m = 0; m < NM - 1; ++m) tt[m] = 0.f;
        for (int e0 = 0; e0 < V; e0 += CH)
          for (int i = 0; i < kOpVec; ++i) {
            const int e = e0 + (warp * 32 + lane + i * kOpWarps * 32) * E;
            if (e < V) {
              uint4 v[NM];
#pragma unroll
              for (int m = 0; m < NM; ++m) v[m] = *reinterpret_cast<const uint4*>(src[m] + e);
              add_vectors(v, true);
            }
          }
      }
      float S[NM], Tw[NM - 1];
#pragma unroll
      for (int m = 0; m < NM; ++m) S[m] = warp_reduce<OpSum>(ss[m]);
#pragma unroll
      for (int m = 0; m < NM - 1; ++m) Tw[m] = warp_reduce<OpSum>(tt[m]);
      const int d = w.n & 1;
      if (w.n >= 2) wait_phase(&ctl->part_free[d], ((w.n >> 1) - 1) & 1u);   // the finisher has read row n - 2
      if (lane == 0) {
        ctl->part[d][warp] = make_float4(ref[0], S[0], ref[1], S[1]);
        ctl->part_x[d][warp] = make_float4(Tw[0], NM == 3 ? Tw[NM - 2] : 0.f, NM == 3 ? ref[NM - 1] : -1e30f, NM == 3 ? S[NM - 1] : 0.f);
        mbar_arrive(&ctl->part_done[d]);
      }
    };
    while (w.advance()) {
      if (TRI && w.tri) row(std::integral_constant<int, 3>{});
      else row(std::integral_constant<int, 2>{});
    }
  } else if (warp == kOpWarps) {
    // ================================ loader ================================
    if (lane == 0) {
      const unsigned long long policy = l2_policy_drop();   // every byte is read once
      unsigned slot = 0, fills = 0;
      while (!dead && w.advance()) {
        const int nm = (TRI && w.tri) ? 3 : 2;
        const T* src[3] = {model_row(w, 0), model_row(w, 1), nm == 3 ? model_row(w, 2) : nullptr};
        for (int step = 0; step < steps; ++step) {
          if (fills > 0) wait_phase(&ctl->empty[slot], (fills - 1u) & 1u);
          if (dead) break;   // the slot was never handed back: nothing more is copied into the ring
          const int e0 = step * CH;
          const unsigned bytes = static_cast<unsigned>(min(CH, V - e0)) * sizeof(T);
          unsigned char* dst = ring + static_cast<size_t>(slot) * kSlotBytes;
          mbar_arrive_expect_tx(&ctl->full[slot], static_cast<unsigned>(nm) * bytes);
          for (int m = 0; m < nm; ++m) bulk_load_hint(dst + m * kOpHalfBytes, src[m] + e0, bytes, &ctl->full[slot], policy);
          if (++slot == kSlots) { slot = 0; ++fills; }
        }
      }
      // Every copy issued above is waited for by its consumers before they leave -- unless a wait gave up somewhere
      // in the CTA. Then this thread has stopped issuing, and it sees every copy it did issue land before the CTA's
      // shared memory goes away: each slot's barrier is polled (bounded) for its latest phase.
      if (dead || *reinterpret_cast<volatile int*>(P.status) != 0) {
        for (unsigned s = 0; s < static_cast<unsigned>(kSlots); ++s) {
          const unsigned turns = fills + (s < slot ? 1u : 0u);
          if (turns == 0) continue;
          unsigned spins = 0;
          while (!mbar_try(&ctl->full[s], (turns - 1u) & 1u) && ++spins <= kClSpinLimit) {}
        }
      }
    }
  } else {
    // ================================ finisher ================================
    const float c = P.c;
    // the record of one pair from the merged sums: (m2, l2s) of its small and large model, T against the large
    // model's reference, S of the large model
    auto make_stats = [&](float ms, float l2ss, float ml, float l2sl, float T_r, float S_l) {
      RowStats st{};
      int flags = 0;
      if (!(fabsf(ms + l2ss) < INFINITY)) flags |= kFlagSmallNonfinite;   // NaN, +inf, or no finite logit
      if (!(fabsf(ml + l2sl) < INFINITY)) flags |= kFlagLargeNonfinite;
      if (flags) {
        st.m2_small = st.l2s_small = st.m2_large = st.l2s_large = st.div = st.resid = __int_as_float(0x7fc00000);
      } else {
        const float bits = c * __fdiv_rn(T_r, S_l) - ((ml + l2sl) - (ms + l2ss));
        st.m2_small = ms; st.l2s_small = l2ss; st.m2_large = ml; st.l2s_large = l2sl;
        st.div = fmaxf(kLn2 * bits, 0.f);
        st.resid = kOpResidUnknown;
      }
      st.flags = flags;
      return st;
    };
    while (w.advance()) {
      const bool tri = TRI && w.tri;
      const int d = w.n & 1;
      wait_phase(&ctl->part_done[d], (w.n >> 1) & 1u);
      const float4 a = lane < kOpWarps ? ctl->part[d][lane] : make_float4(-1e30f, 0.f, -1e30f, 0.f);
      const float4 x = lane < kOpWarps ? ctl->part_x[d][lane] : make_float4(0.f, 0.f, -1e30f, 0.f);
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctl->part_free[d]);
      float m0 = a.x, m1 = a.z, m2 = x.z;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, o));
        m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, o));
        m2 = fmaxf(m2, __shfl_xor_sync(0xffffffffu, m2, o));
      }
      const float f1 = ex2_approx(a.z - m1);
      const float S0 = warp_reduce<OpSum>(a.y * ex2_approx(a.x - m0));
      const float S1 = warp_reduce<OpSum>(a.w * f1);
      // a warp's T may be +inf (q = 0 under p > 0): it stays +inf whatever the warp's scale
      const float T10 = warp_reduce<OpSum>(x.x == INFINITY ? INFINITY : x.x * f1);
      const float l0 = lg2_approx(S0), l1 = lg2_approx(S1);
      float S2 = 0.f, T21 = 0.f, l2 = 0.f;
      if (tri) {
        const float f2 = ex2_approx(x.z - m2);
        S2 = warp_reduce<OpSum>(x.w * f2);
        T21 = warp_reduce<OpSum>(x.y == INFINITY ? INFINITY : x.y * f2);
        l2 = lg2_approx(S2);
      }
      if (lane == 0) {
        const RowStats st = make_stats(m0, l0, m1, l1, T10, S1);
        if (TRI || w.r < rows1) P.stats[w.r] = st;
        else P.stats2[w.r - rows1] = st;
        if (tri) P.stats2[w.r2] = make_stats(m1, l1, m2, l2, T21, S2);
      }
    }
  }
}

// ---- host side --------------------------------------------------------------------------------------
// Whether a launch may take the one-pass kernel: the KL divergence, no caller waiting for residual masses, rows
// that bulk copies can take (the shape test of the cluster kernel) and enough of them to give every SM a row.
inline bool onepass_applies(const StageParams& P, int dtype, bool resid_wanted) {
  if (P.div_kind != kDivKL || resid_wanted) return false;
  if (!cluster_shape_ok(P, dtype)) return false;
  const long long rows = static_cast<long long>(P.B) * (P.K + P.K2);
  const int sms = cluster_sm_count();
  return sms > 0 && rows >= sms;
}

template <typename T, bool TRI>
inline cudaError_t onepass_launch_typed(const StageParams& P, int sms, cudaStream_t stream) {
  static bool prepared[kClMaxDevices] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kClMaxDevices) return cudaErrorInvalidDevice;
  if (!prepared[dev]) {
    e = cudaFuncSetAttribute(rowstats_kl_onepass_kernel<T, TRI>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kOpSmemBytes));
    if (e != cudaSuccess) return e;
    prepared[dev] = true;
  }
  rowstats_kl_onepass_kernel<T, TRI><<<sms, kOpThreads, kOpSmemBytes, stream>>>(P);
  return cudaGetLastError();
}

// Whether a wrapper launch can be walked as row triples: its second row set pairs the first set's large rows (the
// qualifier's, in place) with a third tensor.
inline bool onepass_triples(const StageParams& P) {
  return P.K2 > 0 && P.K2 <= P.K && P.n_valid == nullptr && P.small2 == P.large && P.seq_stride_small2 == P.seq_stride_large;
}

inline int launch_rowstats_onepass(const StageParams& P, int dtype, cudaStream_t stream, bool triples) {
  const int sms = cluster_sm_count();
  cudaError_t e;
  if (triples && onepass_triples(P))
    e = (dtype == 0) ? onepass_launch_typed<float, true>(P, sms, stream) : onepass_launch_typed<__nv_bfloat16, true>(P, sms, stream);
  else
    e = (dtype == 0) ? onepass_launch_typed<float, false>(P, sms, stream) : onepass_launch_typed<__nv_bfloat16, false>(P, sms, stream);
  return e == cudaSuccess ? 0 : 1;
}

}  // namespace psd
