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
constexpr int kOpSlotBytes = 2 * kOpHalfBytes;                  // both models
constexpr int kOpSlots = 6;                                     // ring slots: 192 KB in flight
constexpr float kOpResidUnknown = 1.0f;                         // RowStats.resid of this kernel: "positive unless the draw finds otherwise"

struct __align__(16) OpCtl {
  unsigned long long full[kOpSlots], empty[kOpSlots];
  unsigned long long part_done[2], part_free[2];   // the warps' partials of a row are in / have been read (rows alternate)
  float4 part[2][kOpWarps];                        // (ref_s, S_s, ref_l, S_l) per warp
  float part_t[2][kOpWarps];                       // T per warp, against ref_l
};
constexpr size_t kOpSmemBytes = static_cast<size_t>(kOpSlots) * kOpSlotBytes + sizeof(OpCtl) + 128;

template <typename T>
__global__ void __launch_bounds__(kOpThreads, 1) rowstats_kl_onepass_kernel(const StageParams P) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  OpCtl* ctl = reinterpret_cast<OpCtl*>(ring + static_cast<size_t>(kOpSlots) * kOpSlotBytes);

  constexpr int E = Elem<T>::kPerVec;
  constexpr int CH = kOpHalfBytes / sizeof(T);   // logits per step and model
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int V = P.V, K = P.K;
  const int rows1 = P.B * K;
  const int steps = (V + CH - 1) / CH;

  if (tid == 0) {
    for (int s = 0; s < kOpSlots; ++s) {
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
  auto model_row = [&](const RowWalk& w, int m) -> const T* {
    const bool second = w.r >= rows1;   // second row set: stage 2 of the wrapper
    if (m == 0) return second ? row_ptr<T>(P.small2, P.seq_stride_small2, w.r - rows1, P.K2, V)
                              : row_ptr<T>(P.small, P.seq_stride_small, w.r, K, V);
    return second ? row_ptr<T>(P.large2, P.seq_stride_large2, w.r - rows1, P.K2, V)
                  : row_ptr<T>(P.large, P.seq_stride_large, w.r, K, V);
  };
  RowWalk w;
  w.init(P, blockIdx.x, gridDim.x, false);

  if (warp < kOpWarps) {
    // ================================ consumers ================================
    const float c = P.c;
    const unsigned char* my = ring + (warp * 32 + lane) * 16;
    constexpr int kVecStride = kOpWarps * 32 * 16;   // bytes between a lane's vectors
    int len[kOpVec];   // > step offset while vector i of this lane lies inside the row
#pragma unroll
    for (int i = 0; i < kOpVec; ++i) len[i] = V - (warp * 32 + lane + i * kOpWarps * 32) * E;
    unsigned slot = 0, par = 0;
    // one vector pair into the sums: S_s, S_l and T against the warp's two references
    auto add_vectors = [&](const uint4& us, const uint4& ul, bool live, float ref_s, float ref_l, float& ss, float& sl, float& tt) {
      float xs[E], xl[E];
      Elem<T>::unpack(us, xs);
      Elem<T>::unpack(ul, xl);
      float a = 0.f, b = 0.f, t = 0.f;
#pragma unroll
      for (int j = 0; j < E; ++j) {
        const float es = ex2_approx(fmaf(xs[j], c, -ref_s)), el = ex2_approx(fmaf(xl[j], c, -ref_l));
        a += es;
        b += el;
        if (el > 0.f) t = fmaf(el, xl[j] - xs[j], t);   // q_i = 0 under p_i > 0 gives +inf, as it should; p_i = 0 adds nothing
      }
      if (live) { ss += a; sl += b; tt += t; }
    };
    while (w.advance()) {
      float ref_s = -1e30f, ref_l = -1e30f;   // one reference per warp and model, from the warp's first vectors
      float ss = 0.f, sl = 0.f, tt = 0.f;
      int off = 0;
      for (int step = 0; step < steps; ++step, off += CH) {
        wait_phase(&ctl->full[slot], par);
        const unsigned char* base = my + slot * kOpSlotBytes;
        uint4 u[2][kOpVec];
#pragma unroll
        for (int i = 0; i < kOpVec; ++i)
#pragma unroll
          for (int m = 0; m < 2; ++m) u[m][i] = lds128(base + m * kOpHalfBytes + i * kVecStride);
        if (step == 0) {
          float gs = vector_max<T>(u[0][0], len[0] > 0), gl = vector_max<T>(u[1][0], len[0] > 0);
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            gs = fmaxf(gs, __shfl_xor_sync(0xffffffffu, gs, o));
            gl = fmaxf(gl, __shfl_xor_sync(0xffffffffu, gl, o));
          }
          ref_s = fmaxf(gs * c, -1e30f);   // the floor keeps rows that start with -inf at 0
          ref_l = fmaxf(gl * c, -1e30f);
        }
#pragma unroll
        for (int i = 0; i < kOpVec; ++i) add_vectors(u[0][i], u[1][i], len[i] > off, ref_s, ref_l, ss, sl, tt);
        __syncwarp();
        if (lane == 0) mbar_arrive(&ctl->empty[slot]);
        if (++slot == kOpSlots) { slot = 0; par ^= 1u; }
      }
      if (__any_sync(0xffffffffu, !(ss + sl < INFINITY))) {
        // A sum left the range of a float (a logit far above the warp's first vectors), or the row holds a NaN or
        // +inf: the warp takes its share of the row again from global memory, against its true maxima.
        const T* gs_row = model_row(w, 0);
        const T* gl_row = model_row(w, 1);
        float gs = -INFINITY, gl = -INFINITY;
        for (int e0 = 0; e0 < V; e0 += CH)
          for (int i = 0; i < kOpVec; ++i) {
            const int e = e0 + (warp * 32 + lane + i * kOpWarps * 32) * E;
            if (e < V) {
              gs = fmaxf(gs, vector_max<T>(*reinterpret_cast<const uint4*>(gs_row + e), true));
              gl = fmaxf(gl, vector_max<T>(*reinterpret_cast<const uint4*>(gl_row + e), true));
            }
          }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          gs = fmaxf(gs, __shfl_xor_sync(0xffffffffu, gs, o));
          gl = fmaxf(gl, __shfl_xor_sync(0xffffffffu, gl, o));
        }
        ref_s = fmaxf(gs * c, -1e30f);
        ref_l = fmaxf(gl * c, -1e30f);
        ss = sl = tt = 0.f;
        for (int e0 = 0; e0 < V; e0 += CH)
          for (int i = 0; i < kOpVec; ++i) {
            const int e = e0 + (warp * 32 + lane + i * kOpWarps * 32) * E;
            if (e < V)
              add_vectors(*reinterpret_cast<const uint4*>(gs_row + e), *reinterpret_cast<const uint4*>(gl_row + e), true,
                          ref_s, ref_l, ss, sl, tt);
          }
      }
      const float S_s = warp_reduce<OpSum>(ss), S_l = warp_reduce<OpSum>(sl), T_w = warp_reduce<OpSum>(tt);
      const int d = w.n & 1;
      if (w.n >= 2) wait_phase(&ctl->part_free[d], ((w.n >> 1) - 1) & 1u);   // the finisher has read row n - 2
      if (lane == 0) {
        ctl->part[d][warp] = make_float4(ref_s, S_s, ref_l, S_l);
        ctl->part_t[d][warp] = T_w;
        mbar_arrive(&ctl->part_done[d]);
      }
    }
  } else if (warp == kOpWarps) {
    // ================================ loader ================================
    if (lane == 0) {
      const unsigned long long policy = l2_policy_drop();   // every byte is read once
      unsigned slot = 0, fills = 0;
      while (!dead && w.advance()) {
        const T* src_s = model_row(w, 0);
        const T* src_l = model_row(w, 1);
        for (int step = 0; step < steps; ++step) {
          if (fills > 0) wait_phase(&ctl->empty[slot], (fills - 1u) & 1u);
          if (dead) break;   // the slot was never handed back: nothing more is copied into the ring
          const int e0 = step * CH;
          const unsigned bytes = static_cast<unsigned>(min(CH, V - e0)) * sizeof(T);
          unsigned char* dst = ring + static_cast<size_t>(slot) * kOpSlotBytes;
          mbar_arrive_expect_tx(&ctl->full[slot], 2u * bytes);
          bulk_load_hint(dst, src_s + e0, bytes, &ctl->full[slot], policy);
          bulk_load_hint(dst + kOpHalfBytes, src_l + e0, bytes, &ctl->full[slot], policy);
          if (++slot == kOpSlots) { slot = 0; ++fills; }
        }
      }
      // Every copy issued above is waited for by its consumers before they leave -- unless a wait gave up somewhere
      // in the CTA. Then this thread has stopped issuing, and it sees every copy it did issue land before the CTA's
      // shared memory goes away: each slot's barrier is polled (bounded) for its latest phase.
      if (dead || *reinterpret_cast<volatile int*>(P.status) != 0) {
        for (unsigned s = 0; s < kOpSlots; ++s) {
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
    while (w.advance()) {
      const int d = w.n & 1;
      wait_phase(&ctl->part_done[d], (w.n >> 1) & 1u);
      const float4 a = lane < kOpWarps ? ctl->part[d][lane] : make_float4(-1e30f, 0.f, -1e30f, 0.f);
      const float t = lane < kOpWarps ? ctl->part_t[d][lane] : 0.f;
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctl->part_free[d]);
      float ms = a.x, ml = a.z;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        ms = fmaxf(ms, __shfl_xor_sync(0xffffffffu, ms, o));
        ml = fmaxf(ml, __shfl_xor_sync(0xffffffffu, ml, o));
      }
      const float fl = ex2_approx(a.z - ml);
      const float S_s = warp_reduce<OpSum>(a.y * ex2_approx(a.x - ms));
      const float S_l = warp_reduce<OpSum>(a.w * fl);
      // a warp's T may be +inf (q = 0 under p > 0): it stays +inf whatever the warp's scale
      const float T_r = warp_reduce<OpSum>(t == INFINITY ? INFINITY : t * fl);
      const float l2ss = lg2_approx(S_s), l2sl = lg2_approx(S_l);
      if (lane == 0) {
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
        if (w.r < rows1) P.stats[w.r] = st;
        else P.stats2[w.r - rows1] = st;
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

template <typename T>
inline cudaError_t onepass_launch_typed(const StageParams& P, int sms, cudaStream_t stream) {
  static bool prepared[kClMaxDevices] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kClMaxDevices) return cudaErrorInvalidDevice;
  if (!prepared[dev]) {
    e = cudaFuncSetAttribute(rowstats_kl_onepass_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kOpSmemBytes));
    if (e != cudaSuccess) return e;
    prepared[dev] = true;
  }
  rowstats_kl_onepass_kernel<T><<<sms, kOpThreads, kOpSmemBytes, stream>>>(P);
  return cudaGetLastError();
}

inline int launch_rowstats_onepass(const StageParams& P, int dtype, cudaStream_t stream) {
  const int sms = cluster_sm_count();
  const cudaError_t e = (dtype == 0) ? onepass_launch_typed<float>(P, sms, stream)
                                     : onepass_launch_typed<__nv_bfloat16>(P, sms, stream);
  return e == cudaSuccess ? 0 : 1;
}

}  // namespace psd
