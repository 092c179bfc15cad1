// Baseline row-statistics kernel: one CTA per (sequence, position) row, three passes over global
// memory (row maxima; sum-exps; divergence and residual mass). Works for any V, alignment and dtype;
// the optimised cluster kernel falls back to it for shapes it does not take, and tests use it as a
// second opinion on the GPU. Passes two and three mostly hit L2, but the row pair still crosses the
// SM's load path three times.
#pragma once

#include "common.cuh"

namespace psd {

// Calls f(x_large, x_small, i) for every vocabulary index i of the row pair, 16-byte vector loads when
// `vec_ok`, scalar loads otherwise. Thread t of the CTA sees vectors t, t + blockDim, ...
template <typename T, typename F>
__device__ __forceinline__ void for_each_pair(const T* __restrict__ large, const T* __restrict__ small, int V,
                                              bool vec_ok, F&& f) {
  constexpr int E = Elem<T>::kPerVec;
  if (vec_ok) {
    const int nvec = V / E;
    for (int v = threadIdx.x; v < nvec; v += blockDim.x) {
      const uint4 ul = ldg_vec(large, v), us = ldg_vec(small, v);
      float xl[E], xs[E];
      Elem<T>::unpack(ul, xl);
      Elem<T>::unpack(us, xs);
#pragma unroll
      for (int j = 0; j < E; ++j) f(xl[j], xs[j], v * E + j);
    }
  } else {
    for (int i = threadIdx.x; i < V; i += blockDim.x) f(Elem<T>::load(large, i), Elem<T>::load(small, i), i);
  }
}

template <typename T>
__global__ void __launch_bounds__(1024) rowstats_baseline_kernel(const StageParams P) {
  __shared__ float scratch[32];
  const int r = blockIdx.x;
  const int b = r / P.K, k = r - b * P.K;
  if (P.n_valid != nullptr && k >= P.n_valid[b]) return;  // position outside this sequence's window

  const T* large = static_cast<const T*>(P.large) + b * P.seq_stride_large + static_cast<long long>(k) * P.V;
  const T* small = static_cast<const T*>(P.small) + b * P.seq_stride_small + static_cast<long long>(k) * P.V;
  const int V = P.V;
  const bool vec_ok = ((reinterpret_cast<uintptr_t>(large) | reinterpret_cast<uintptr_t>(small)) & 15u) == 0 &&
                      (V % Elem<T>::kPerVec) == 0;
  const float c = P.c;

  // pass 1: row maxima (NaN-propagating) and a bitwise "rows identical" test
  float ml = -INFINITY, ms = -INFINITY;
  unsigned differ = 0u;
  for_each_pair<T>(large, small, V, vec_ok, [&](float xl, float xs, int) {
    ml = max_nan(ml, xl);
    ms = max_nan(ms, xs);
    differ |= (__float_as_uint(xl) ^ __float_as_uint(xs));
  });
  ml = block_reduce<OpMaxNan>(ml, scratch, -INFINITY);
  ms = block_reduce<OpMaxNan>(ms, scratch, -INFINITY);
  differ = block_reduce_or(differ, reinterpret_cast<unsigned*>(scratch));

  int flags = 0;
  if (!(fabsf(ml) < INFINITY)) flags |= kFlagLargeNonfinite;  // NaN, +inf, or every entry -inf
  if (!(fabsf(ms) < INFINITY)) flags |= kFlagSmallNonfinite;
  if (flags) {
    if (threadIdx.x == 0) {
      RowStats st{};
      st.m2_small = st.l2s_small = st.m2_large = st.l2s_large = st.div = st.resid = __int_as_float(0x7fc00000);
      st.flags = flags;
      P.stats[r] = st;
    }
    return;
  }

  // pass 2: sum of 2^(z*c - max*c) for both models
  const float m2l = ml * c, m2s = ms * c;
  float sl = 0.f, ss = 0.f;
  for_each_pair<T>(large, small, V, vec_ok, [&](float xl, float xs, int) {
    sl += ex2_approx(fmaf(xl, c, -m2l));
    ss += ex2_approx(fmaf(xs, c, -m2s));
  });
  sl = block_reduce<OpSum>(sl, scratch, 0.f);
  ss = block_reduce<OpSum>(ss, scratch, 0.f);
  const float l2sl = lg2_approx(sl), l2ss = lg2_approx(ss);

  // pass 3: divergence and residual mass from the normalised probabilities p = 2^((z*c - m2) - l2s)
  float acc = 0.f, res = 0.f;
  const int kind = P.div_kind;
  for_each_pair<T>(large, small, V, vec_ok, [&](float xl, float xs, int) {
    const float a2 = fmaf(xl, c, -m2l) - l2sl, b2 = fmaf(xs, c, -m2s) - l2ss;  // log2 p, log2 q
    const float p = ex2_approx(a2), q = ex2_approx(b2);
    res += fmaxf(p - q, 0.f);
    if (kind == kDivJS) {
      // JS = 1/2 sum p ln(p/m) + 1/2 sum q ln(q/m), m = (p+q)/2, accumulated in bits: log2 m = log2(p+q) - 1
      const float lm = lg2_approx(p + q) - 1.f;
      if (p > 0.f) acc = fmaf(p, a2 - lm, acc);
      if (q > 0.f) acc = fmaf(q, b2 - lm, acc);
    } else if (kind == kDivKL) {
      if (p > 0.f) acc = fmaf(p, a2 - b2, acc);  // q == 0 with p > 0 gives +inf, as it should
    }
  });
  acc = block_reduce<OpSum>(acc, scratch, 0.f);
  res = block_reduce<OpSum>(res, scratch, 0.f);

  if (threadIdx.x == 0) {
    float D;
    if (kind == kDivJS) D = 0.5f * kLn2 * acc;
    else if (kind == kDivKL) D = kLn2 * acc;
    else D = res;  // total variation equals the residual mass
    D = fmaxf(D, 0.f);
    if (differ == 0u) { D = 0.f; res = 0.f; }  // bitwise identical rows: exactly zero
    RowStats st{};
    st.m2_small = m2s; st.l2s_small = l2ss;
    st.m2_large = m2l; st.l2s_large = l2sl;
    st.div = D;
    st.resid = res;
    st.flags = 0;
    P.stats[r] = st;
  }
}

}  // namespace psd
