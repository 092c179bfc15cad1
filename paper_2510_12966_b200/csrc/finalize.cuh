// Finalisation: a warp turns a sequence's per-row statistics into accept bits (fuzzy threshold test of
// Sec. 3.1/3.2, or the standard-SD coin flip), a ballot gives the accepted prefix length (Sec. 1), and, when a
// position was rejected, the correction token is drawn from the residual max(0, p_large - p_small) (Sec. 3.4) --
// or from p_large in the assisted variant -- by a hierarchical inverse CDF in vocabulary order: tiles of 8192
// indices, then warps, then lanes, then elements, each level picking the first child whose inclusive cumulative
// weight exceeds the remaining target. Two forms share this code and return the same bits: one launch with a CTA
// (or a cluster of CTAs) per sequence, and, for batches that fill the GPU, three small launches that spread the
// tile totals of all draws over all SMs (second half of this file).
#pragma once

#include "common.cuh"

namespace psd {

constexpr int kFinThreads = 1024;
constexpr int kFinElemsPerThread = 8;                      // consecutive vocabulary indices per thread and tile
constexpr int kFinTile = kFinThreads * kFinElemsPerThread;  // 8192 indices per tile
constexpr int kFinMaxTiles = 1024;                          // V <= 8,388,608
constexpr int kFinBatch = 32;

__device__ __forceinline__ unsigned fin_cluster_rank() {
  unsigned r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void fin_cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// one double into the same shared-memory variable of another CTA of the cluster
__device__ __forceinline__ void fin_remote_store(double* local, unsigned rank, double v) {
  unsigned addr;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(addr) : "r"(static_cast<unsigned>(__cvta_generic_to_shared(local))), "r"(rank));
  asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(addr), "d"(v) : "memory");
}                               // tiles summed between two CTA-wide barriers

// A finalisation launch may start while the launch before it drains; it reads nothing of that launch before this.
__device__ __forceinline__ void wait_for_previous_launch() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next launch on the stream, if it was launched as a dependent, be scheduled from here on.
__device__ __forceinline__ void release_next_launch() { asm volatile("griddepcontrol.launch_dependents;"); }

template <typename T>
struct RowView {
  const T* large;
  const T* small;
  int V;
  bool vec_ok;
  float c, m2l, l2sl, m2s, l2ss;
  bool from_large;  // weights are p_large itself (assisted variant, or an all-zero residual)

  static constexpr int kVecs = kFinElemsPerThread / Elem<T>::kPerVec;   // 16-byte vectors per thread, tile and model

  // whether the thread's indices starting at i0 can be taken as whole vectors
  __device__ __forceinline__ bool whole(int i0) const { return vec_ok && i0 + kFinElemsPerThread <= V; }
  // the raw vectors of those indices: loads only, so that a caller can have several tiles' loads in flight
  __device__ __forceinline__ void fetch(int i0, uint4* rl, uint4* rs) const {
    constexpr int E = Elem<T>::kPerVec;
#pragma unroll
    for (int h = 0; h < kVecs; ++h) {
      rl[h] = ldg_vec(large, i0 / E + h);
      rs[h] = ldg_vec(small, i0 / E + h);
    }
  }
  __device__ __forceinline__ void weights_of(const float* xl, const float* xs, float* w) const {
#pragma unroll
    for (int j = 0; j < kFinElemsPerThread; ++j) {
      const float p = ex2_approx(fmaf(xl[j], c, -m2l) - l2sl);
      const float q = ex2_approx(fmaf(xs[j], c, -m2s) - l2ss);
      w[j] = from_large ? p : fmaxf(p - q, 0.f);
    }
  }
  // weights from vectors fetched earlier
  __device__ __forceinline__ void weights_fetched(const uint4* rl, const uint4* rs, float* w) const {
    constexpr int E = Elem<T>::kPerVec;
    float xl[kFinElemsPerThread], xs[kFinElemsPerThread];
#pragma unroll
    for (int h = 0; h < kVecs; ++h) {
      Elem<T>::unpack(rl[h], xl + h * E);
      Elem<T>::unpack(rs[h], xs + h * E);
    }
    weights_of(xl, xs, w);
  }
  // weights of the kFinElemsPerThread consecutive indices starting at i0 (0 beyond V)
  __device__ __forceinline__ void weights(int i0, float* w) const {
    if (whole(i0)) {
      uint4 rl[kVecs], rs[kVecs];
      fetch(i0, rl, rs);
      weights_fetched(rl, rs, w);
    } else {
      float xl[kFinElemsPerThread], xs[kFinElemsPerThread];
#pragma unroll
      for (int j = 0; j < kFinElemsPerThread; ++j) {
        const bool in = i0 + j < V;
        xl[j] = in ? Elem<T>::load(large, i0 + j) : -INFINITY;
        xs[j] = in ? Elem<T>::load(small, i0 + j) : -INFINITY;
      }
      weights_of(xl, xs, w);
    }
  }
};

struct FinShared {
  double tile_total[kFinMaxTiles];
  float warp_total[32];
  float warp_tile[kFinBatch][32];   // per-warp sums of a batch of tiles
  int sh_L, sh_nv, sh_flags, sh_tile, sh_warp, sh_token;
  float sh_u2, sh_m2l, sh_l2sl, sh_m2s, sh_l2ss, sh_resid, sh_target;
};

// What the accept scan of one sequence hands to the draw: the first rejected position (or the number of valid
// positions when all were accepted) and the statistics of that position's row.
struct ScanOut {
  int L, nv, flags;
  float u2, m2l, l2sl, m2s, l2ss, resid;
};

// Accept bits and prefix length of sequence b, by one full warp: lane k owns position k (K <= 32). Every lane
// returns the same values. `write_rows`: this warp also writes the per-row outputs. `nv_given` >= 0 replaces
// P.n_valid[b], and `tokens_given` (with `n_given` entries; positions beyond it count as token 0) replaces
// P.tokens for this sequence.
template <typename T>
__device__ __forceinline__ ScanOut scan_unit(const StageParams& P, const int b, const int lane, const bool write_rows,
                                             const int nv_given, const int32_t* tokens_given, const int n_given) {
  const int K = P.K, V = P.V;
  const T* large_seq = static_cast<const T*>(P.large) + b * P.seq_stride_large;
  const T* small_seq = static_cast<const T*>(P.small) + b * P.seq_stride_small;
  int nv = K;
  if (nv_given >= 0) nv = min(nv_given, K);
  else if (P.n_valid != nullptr) nv = min(max(P.n_valid[b], 0), K);

  bool acc = true;  // lanes beyond nv never end the prefix
  RowStats st{};
  float u = 0.f, u2 = 0.f;
  int flags = 0;
  if (lane < nv) {
    const int r = b * K + lane;
    st = P.stats[r];
    const int x = (tokens_given != nullptr) ? (lane < n_given ? tokens_given[lane] : 0) : P.tokens[r];
    flags = st.flags | ((x < 0 || x >= V) ? kFlagTokenRange : 0);
    row_uniforms(P.seed, P.offset, static_cast<unsigned>((P.seq_base + b) * K + lane), &u, &u2);
    const float nanf_ = __int_as_float(0x7fc00000);
    float px = nanf_, qx = nanf_;
    bool coin_ok = false;
    // the token's two probabilities decide the coin flip; the threshold rule needs them only as outputs
    const bool want_p = P.mode != kModeFuzzy || P.out_p_small_tok != nullptr || P.out_p_large_tok != nullptr;
    if (!flags && want_p) {
      const long long off = static_cast<long long>(lane) * V + x;
      px = ex2_approx(fmaf(Elem<T>::load(large_seq, off), P.c, -st.m2_large) - st.l2s_large);
      qx = ex2_approx(fmaf(Elem<T>::load(small_seq, off), P.c, -st.m2_small) - st.l2s_small);
      // standard SD: accept with probability min(1, p_large(x) / p_small(x))
      const float rho = (qx > 0.f) ? __fdiv_rn(px, qx) : (px > 0.f ? INFINITY : 0.f);
      coin_ok = u < fminf(1.f, rho);
    }
    const bool fuzzy_ok = st.div <= P.threshold;
    if (P.mode == kModeFuzzy) acc = fuzzy_ok;
    else if (P.mode == kModeStrict || P.mode == kModeAssisted) acc = coin_ok;
    else acc = fuzzy_ok || coin_ok;
    if (flags) acc = false;
    if (write_rows) {
      if (P.out_div) P.out_div[r] = st.div;
      if (P.out_resid_mass) P.out_resid_mass[r] = st.resid;
      if (P.out_p_small_tok) P.out_p_small_tok[r] = qx;
      if (P.out_p_large_tok) P.out_p_large_tok[r] = px;
      if (P.out_row_flags) P.out_row_flags[r] = flags;
    }
  } else if (lane < K && write_rows) {
    const int r = b * K + lane;
    if (P.out_div) P.out_div[r] = 0.f;
    if (P.out_resid_mass) P.out_resid_mass[r] = 0.f;
    if (P.out_p_small_tok) P.out_p_small_tok[r] = 0.f;
    if (P.out_p_large_tok) P.out_p_large_tok[r] = 0.f;
    if (P.out_row_flags) P.out_row_flags[r] = 0;
  }
  const unsigned rejected = ~__ballot_sync(0xffffffffu, acc);
  const int L = rejected ? (__ffs(rejected) - 1) : nv;  // first rejected position, or all accepted
  const int src = min(L, 31);   // L < nv <= 32 when a rejection exists; otherwise the row data go unused
  ScanOut o;
  o.L = L;
  o.nv = nv;
  o.flags = __shfl_sync(0xffffffffu, flags, src);
  o.u2 = __shfl_sync(0xffffffffu, u2, src);
  o.m2l = __shfl_sync(0xffffffffu, st.m2_large, src);
  o.l2sl = __shfl_sync(0xffffffffu, st.l2s_large, src);
  o.m2s = __shfl_sync(0xffffffffu, st.m2_small, src);
  o.l2ss = __shfl_sync(0xffffffffu, st.l2s_small, src);
  o.resid = __shfl_sync(0xffffffffu, st.resid, src);
  return o;
}

// The results of one sequence, by one thread: prefix length, next token, and in the two-stage wrapper the stage-2
// window (Fig. 1): accepted draft tokens, then the correction token.
__device__ __forceinline__ void write_results(const StageParams& P, const int b, const int L, const int next) {
  P.out_accept_len[b] = L;
  P.out_next_token[b] = next;
  if (P.window != nullptr) {
    const int have = L + (next >= 0 ? 1 : 0);
    const int n2 = min(have, P.K_window);
    P.n_window[b] = n2;
    if (P.fill_out != nullptr && b < P.fill_cap) P.fill_out[b] = n2;
    for (int j = 0; j < P.K_window; ++j)
      P.window[b * P.K_window + j] = (j < n2) ? ((j < L) ? P.tokens[b * P.K + j] : next) : 0;
  }
}

// Level 0 of the draw, by one thread, once every tile's total is in S.tile_total: the first tile whose inclusive
// cumulative weight exceeds the target, else the last non-empty tile. Leaves the tile in S.sh_tile (-1: no
// positive weight at all; -2: the residual weights all came out zero, take the totals again over p_large) and
// the target that remains inside it in S.sh_target.
__device__ __forceinline__ void pick_tile(FinShared& S, const int n_tiles, const bool from_large) {
  const double* tile_total = S.tile_total;
  double total = 0.0;
  for (int j = 0; j < n_tiles; ++j) total += tile_total[j];
  const double target = static_cast<double>(S.sh_u2) * total;
  const bool redo = !(total > 0.0) && !from_large;
  int pick = -1, last_pos = -1;
  double cum = 0.0, cum_before_pick = 0.0, cum_before_last = 0.0;
  for (int j = 0; j < n_tiles; ++j) {
    const double nxt = cum + tile_total[j];
    if (tile_total[j] > 0.0) { last_pos = j; cum_before_last = cum; }
    if (pick < 0 && nxt > target && tile_total[j] > 0.0) { pick = j; cum_before_pick = cum; }
    cum = nxt;
  }
  if (pick < 0) { pick = last_pos; cum_before_pick = cum_before_last; }
  S.sh_tile = redo ? -2 : pick;
  S.sh_token = -1;
  S.sh_target = static_cast<float>(target - cum_before_pick);
}

// Levels 1 to 3 of the draw inside the chosen tile, by the whole CTA: warps, lanes, the thread's own elements.
// Leaves the token in S.sh_token (valid after the closing barrier).
template <typename T>
__device__ __forceinline__ void descend_tile(const RowView<T>& row, FinShared& S, const int tile) {
  float (&warp_total)[32] = S.warp_total;
  int &sh_warp = S.sh_warp, &sh_token = S.sh_token;
  float &sh_target = S.sh_target;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float w[kFinElemsPerThread];
  {
    // level 1: warps of the chosen tile
    const int i0 = tile * kFinTile + tid * kFinElemsPerThread;
    row.weights(i0, w);
    float ts = 0.f;
#pragma unroll
    for (int e = 0; e < kFinElemsPerThread; ++e) ts += w[e];
    // inclusive scan of thread sums across the warp (fixed shuffle tree)
    float incl = ts;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const float up = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += up;
    }
    if (lane == 31) warp_total[warp] = incl;
    __syncthreads();
    if (tid == 0) {
      const float target = sh_target;
      int pick = -1, last_pos = -1;
      float cum = 0.f, before_pick = 0.f, before_last = 0.f;
      for (int j = 0; j < kFinThreads / 32; ++j) {
        const float nxt = cum + warp_total[j];
        if (warp_total[j] > 0.f) { last_pos = j; before_last = cum; }
        if (pick < 0 && nxt > target && warp_total[j] > 0.f) { pick = j; before_pick = cum; }
        cum = nxt;
      }
      if (pick < 0) { pick = last_pos; before_pick = before_last; }
      sh_warp = pick;
      sh_target = target - before_pick;
    }
    __syncthreads();
    if (warp == sh_warp) {
      // level 2: lanes of the chosen warp
      const float target = sh_target;
      const float excl = incl - ts;  // only used as the offset handed to the next level
      const unsigned hit = __ballot_sync(0xffffffffu, incl > target && ts > 0.f);
      const unsigned pos = __ballot_sync(0xffffffffu, ts > 0.f);
      const int pick_lane = hit ? (__ffs(hit) - 1) : (pos ? 31 - __clz(pos) : -1);
      if (lane == pick_lane) {
        // level 3: the thread's own consecutive elements
        const float t3 = target - excl;
        float run = 0.f;
        int choice = -1, last_pos = -1;
#pragma unroll
        for (int e = 0; e < kFinElemsPerThread; ++e) {
          run += w[e];
          if (w[e] > 0.f) {
            last_pos = e;
            if (choice < 0 && run > t3) choice = e;
          }
        }
        if (choice < 0) choice = last_pos;
        sh_token = (choice >= 0) ? i0 + choice : -1;
      }
    }
    __syncthreads();
  }
}

// One stage's finalisation of sequence b; every thread of the CTA calls it. With CL > 1 the CTAs of a
// cluster all call it for the same sequence: each repeats the (cheap) accept scan, the tile sums of the draw
// are split between them and exchanged through distributed shared memory, and the CTA that owns the chosen
// tile finishes the draw and writes the results. `nv_given` >= 0 replaces P.n_valid[b], and `tokens_given`
// (with `n_given` entries; positions beyond it count as token 0) replaces P.tokens for this sequence: that
// is how a stage 2 that accepts by the threshold rule runs without waiting for stage 1's draw.
template <typename T, int CL>
__device__ __forceinline__ void finalize_sequence(const StageParams& P, const int b, FinShared& S, const int nv_given = -1,
                                                  const int32_t* tokens_given = nullptr, const int n_given = 0) {
  const unsigned cl_rank = (CL > 1) ? fin_cluster_rank() : 0u;
  double (&tile_total)[kFinMaxTiles] = S.tile_total;
  float (&warp_total)[32] = S.warp_total;
  float (&warp_tile)[kFinBatch][32] = S.warp_tile;
  int &sh_L = S.sh_L, &sh_nv = S.sh_nv, &sh_flags = S.sh_flags, &sh_tile = S.sh_tile, &sh_warp = S.sh_warp, &sh_token = S.sh_token;
  float &sh_u2 = S.sh_u2, &sh_m2l = S.sh_m2l, &sh_l2sl = S.sh_l2sl, &sh_m2s = S.sh_m2s, &sh_l2ss = S.sh_l2ss,
        &sh_resid = S.sh_resid, &sh_target = S.sh_target;

  const int K = P.K, V = P.V;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const T* large_seq = static_cast<const T*>(P.large) + b * P.seq_stride_large;
  const T* small_seq = static_cast<const T*>(P.small) + b * P.seq_stride_small;

  // ---- accept bits and prefix length: lane k of warp 0 owns position k (K <= 32) ----
  if (warp == 0) {
    const ScanOut o = scan_unit<T>(P, b, lane, cl_rank == 0, nv_given, tokens_given, n_given);
    if (lane == 0) {
      sh_L = o.L;
      sh_nv = o.nv;
      sh_flags = o.flags;
      sh_u2 = o.u2;
      sh_m2l = o.m2l; sh_l2sl = o.l2sl;
      sh_m2s = o.m2s; sh_l2ss = o.l2ss;
      sh_resid = o.resid;
    }
  }
  __syncthreads();
  const int L = sh_L;
  int next = -1;
  unsigned writer = 0;   // the CTA of the cluster that writes the sequence's results
  bool need_draw = false;
  if (L < sh_nv) {
    if (sh_flags & (kFlagSmallNonfinite | kFlagLargeNonfinite)) next = -2;  // no distribution to draw from
    else need_draw = true;
  }
  const bool bonus = P.bonus && L == sh_nv;   // everything accepted: the larger model's next token comes for free
  if (bonus) {
    // The row after the window was not part of the statistics pass: every CTA takes its normaliser here, with
    // the same two passes and reduction trees (so all CTAs of a cluster hold the same bits).
    const T* brow = large_seq + static_cast<long long>(L) * V;
    const bool vec_ok = (reinterpret_cast<uintptr_t>(brow) & 15u) == 0 && (V % Elem<T>::kPerVec) == 0;
    constexpr int E = Elem<T>::kPerVec;
    float mx = -INFINITY;
    if (vec_ok) {
      for (int v = tid; v < V / E; v += kFinThreads) {
        float x[E];
        Elem<T>::unpack(ldg_vec(brow, v), x);
#pragma unroll
        for (int j = 0; j < E; ++j) mx = max_nan(mx, x[j]);
      }
    } else {
      for (int i = tid; i < V; i += kFinThreads) mx = max_nan(mx, Elem<T>::load(brow, i));
    }
    mx = block_reduce<OpMaxNan>(mx, warp_total, -INFINITY);
    if (!(fabsf(mx) < INFINITY)) {
      next = -2;   // NaN, +inf or no finite logit: no distribution to draw from
    } else {
      const float m2 = mx * P.c;
      float sum = 0.f;
      if (vec_ok) {
        for (int v = tid; v < V / E; v += kFinThreads) {
          float x[E];
          Elem<T>::unpack(ldg_vec(brow, v), x);
#pragma unroll
          for (int j = 0; j < E; ++j) sum += ex2_approx(fmaf(x[j], P.c, -m2));
        }
      } else {
        for (int i = tid; i < V; i += kFinThreads) sum += ex2_approx(fmaf(Elem<T>::load(brow, i), P.c, -m2));
      }
      sum = block_reduce<OpSum>(sum, warp_total, 0.f);
      if (tid == 0) {
        sh_m2l = m2; sh_l2sl = lg2_approx(sum);
        sh_m2s = m2; sh_l2ss = sh_l2sl;
        sh_resid = 0.f;   // weights are p_large itself
        sh_u2 = bonus_uniform(P.seed, P.offset, static_cast<unsigned>(P.seq_base + b));
      }
      __syncthreads();
      need_draw = true;
    }
  }

  if (need_draw) {  // uniform across the CTA
    RowView<T> row;
    row.large = large_seq + static_cast<long long>(L) * V;
    row.small = bonus ? row.large : small_seq + static_cast<long long>(L) * V;   // the bonus row has no small partner
    row.V = V;
    row.vec_ok = ((reinterpret_cast<uintptr_t>(row.large) | reinterpret_cast<uintptr_t>(row.small)) & 15u) == 0 &&
                 (V % Elem<T>::kPerVec) == 0;
    row.c = P.c;
    row.m2l = sh_m2l; row.l2sl = sh_l2sl;
    row.m2s = sh_m2s; row.l2ss = sh_l2ss;
    row.from_large = (P.mode == kModeAssisted) || !(sh_resid > 0.f);

    const int n_tiles = (V + kFinTile - 1) / kFinTile;
    float w[kFinElemsPerThread];
    // level 0: total weight of every tile. CTA `cl_rank` of the cluster takes tiles cl_rank, cl_rank + CL, ...;
    // the tiles of a batch are independent (their loads overlap); each warp leaves its sum per tile, then one
    // thread per tile adds the 32 warp sums in warp order and hands the total to every CTA of the cluster.
    const int my_tiles = (n_tiles - static_cast<int>(cl_rank) + CL - 1) / CL;
    // A second go happens only when the residual weights, taken again here in single precision, all come out
    // zero although the row's residual mass did not (two rows that differ only where both probabilities
    // underflow): the draw then comes from p_large, as for a zero residual, so a rejected row with a
    // distribution always yields a token.
    for (int attempt = 0; attempt < 2; ++attempt) {
    for (int m0 = 0; m0 < my_tiles; m0 += kFinBatch) {
      const int nb = min(kFinBatch, my_tiles - m0);
#pragma unroll 4
      for (int m = 0; m < nb; ++m) {
        const int j = (m0 + m) * CL + static_cast<int>(cl_rank);
        row.weights(j * kFinTile + tid * kFinElemsPerThread, w);
        float ts = 0.f;
#pragma unroll
        for (int e = 0; e < kFinElemsPerThread; ++e) ts += w[e];
        ts = warp_reduce<OpSum>(ts);
        if (lane == 0) warp_tile[m][warp] = ts;
      }
      __syncthreads();
      if (tid < nb) {
        double tt = 0.0;
        for (int k = 0; k < 32; ++k) tt += static_cast<double>(warp_tile[tid][k]);
        const int j = (m0 + tid) * CL + static_cast<int>(cl_rank);
        tile_total[j] = tt;
        if (CL > 1) {
#pragma unroll
          for (int p = 0; p < CL; ++p)
            if (p != static_cast<int>(cl_rank)) fin_remote_store(&tile_total[j], static_cast<unsigned>(p), tt);
        }
      }
      __syncthreads();
    }
    if (CL > 1) fin_cluster_sync();   // every CTA now holds every tile's total
    if (tid == 0) pick_tile(S, n_tiles, row.from_large);
    __syncthreads();
    if (sh_tile != -2) break;
    row.from_large = true;            // every CTA of the cluster holds the same totals and takes the same turn
    if (CL > 1) fin_cluster_sync();   // nobody posts new totals while a peer still reads the old ones
    __syncthreads();
    }
    const int tile = sh_tile;
    writer = (CL > 1 && tile >= 0) ? static_cast<unsigned>(tile % CL) : 0u;   // the CTA that summed the chosen tile goes on
    if (tile >= 0 && cl_rank == writer) {
      descend_tile<T>(row, S, tile);
      next = sh_token;
    }
  }

  if (tid == 0 && cl_rank == writer) write_results(P, b, L, next);
}

template <typename T, int CL>
__global__ void __launch_bounds__(kFinThreads, 1) finalize_kernel(const StageParams P) {
  __shared__ FinShared S;
  wait_for_previous_launch();
  finalize_sequence<T, CL>(P, blockIdx.x / CL, S);
  if (CL > 1) fin_cluster_sync();   // nobody leaves while a peer may still post tile sums into its shared memory
}

// Both stages of the two-stage wrapper for one sequence: stage 1 (draft against qualifier) writes the
// window and its length, stage 2 (window against target) reads them back. The statistics of every
// stage-2 row were computed beforehand, whatever the window turned out to be.
template <typename T, int CL>
__global__ void __launch_bounds__(kFinThreads) finalize_pyramid_kernel(const StageParams P1, const StageParams P2) {
  __shared__ FinShared S;
  wait_for_previous_launch();
  finalize_sequence<T, CL>(P1, blockIdx.x / CL, S);
  __threadfence();
  __syncthreads();
  if (CL > 1) fin_cluster_sync();   // the window and its length, written by one thread of the cluster, are visible to all of it
  finalize_sequence<T, CL>(P2, blockIdx.x / CL, S);
  if (CL > 1) fin_cluster_sync();
}

// The window of the stage-2 half of a pyramid whose stage 2 uses the threshold rule, by one full warp: stage 1's
// accept scan again (whatever its rule: the coin flips are functions of the row index), without its outputs. The
// window holds the accepted prefix and, unless everything was accepted or the rejected row has no distribution, the
// correction token; which token that is does not matter to a threshold test.
template <typename T>
__device__ __forceinline__ void stage1_prefix(const StageParams& P1, const int K2, const int b, const int lane, int* L1, int* n2) {
  const ScanOut o = scan_unit<T>(P1, b, lane, false, -1, nullptr, 0);
  const int has_next = (o.L < o.nv && !(o.flags & (kFlagSmallNonfinite | kFlagLargeNonfinite))) ? 1 : 0;
  *L1 = o.L;
  *n2 = min(o.L + has_next, K2);
}

// Stage 2 by the threshold rule (stage 1 by any rule, the assisted variant of Sec. 3.4 among them): the stage-2
// half of the pyramid does not need stage 1's drawn token -- its accept bits depend on the divergences alone, and
// the window length follows from stage 1's accept scan -- so the two stages of a sequence run side by side, one
// cluster each. Cluster 2b is stage 1 (it also writes the window); cluster 2b+1 repeats stage 1's cheap scan to
// get the window length, then runs stage 2 on the accepted draft prefix.
template <typename T, int CL>
__global__ void __launch_bounds__(kFinThreads) finalize_pyramid_split_kernel(const StageParams P1, const StageParams P2) {
  __shared__ FinShared S;
  wait_for_previous_launch();
  __shared__ int sh_L1, sh_n2;
  const int unit = blockIdx.x / CL, b = unit >> 1;
  if ((unit & 1) == 0) {
    finalize_sequence<T, CL>(P1, b, S);
  } else {
    if (threadIdx.x < 32) {
      int L1, n2;
      stage1_prefix<T>(P1, P2.K, b, threadIdx.x, &L1, &n2);
      if (threadIdx.x == 0) { sh_L1 = L1; sh_n2 = n2; }
    }
    __syncthreads();
    finalize_sequence<T, CL>(P2, b, S, sh_n2, P1.tokens + b * P1.K, sh_L1);
  }
  if (CL > 1) fin_cluster_sync();
}

// ---- finalisation of a large batch in three launches -------------------------------------------------------
// With one CTA (or pair) per sequence a draw is a chain of dependent steps on one SM -- the tile totals alone take
// a microsecond per tile -- while the SMs whose sequences accepted everything idle; and when every sequence
// draws, the CTAs come in waves. For batches that fill the GPU the work is cut differently. A scan launch (one
// warp per sequence and stage) takes the accept bits, finishes the sequences that need no draw and leaves a record
// for each one that does. A tile launch of one CTA per SM spreads level 0 of all draws, the (record, tile) pairs,
// over all CTAs. A pick launch then gives each draw a CTA for the pick and levels 1 to 3. Launch boundaries order
// the three; no CTA waits for another and nothing is counted atomically. Each tile total, the pick and the descent
// are the code of the one-launch form, so both forms return the same bits.
constexpr int kDrawMaxTiles = 32;      // V <= 262144
constexpr int kDrawMaxUnits = 4096;    // sequences x stages of one call
constexpr int kScanWarps = 4;

struct DrawRecord {
  int L;
  float u2, m2l, l2sl, m2s, l2ss, resid;
  int unit;
};

struct DrawScratch {
  int* need;            // [units] 1: the unit draws
  int* count;           // [0]: number of drawing units
  DrawRecord* record;   // [units] by unit, written by the scan
  DrawRecord* drawn;    // [d]: the record of the d-th drawing unit (in unit order), gathered by the tile launch so
                        // that the pick launch finds all it needs at addresses it knows from its block index
  double* tile_total;   // [d][kDrawMaxTiles]
};

__host__ __device__ inline size_t draw_scratch_bytes(long long units) {
  return static_cast<size_t>(units) * (sizeof(int) + 2 * sizeof(DrawRecord) + kDrawMaxTiles * sizeof(double)) + 256;
}

// Scan launch: unit = sequence (n_stages == 1) or 2 * sequence + stage (the side-by-side form of a pyramid).
template <typename T>
__global__ void __launch_bounds__(kScanWarps * 32) finalize_scan_kernel(const StageParams P1, const StageParams P2, const int n_stages,
                                                                        const DrawScratch ds) {
  wait_for_previous_launch();
  release_next_launch();
  const int lane = threadIdx.x & 31;
  const int unit = blockIdx.x * kScanWarps + (threadIdx.x >> 5);
  if (unit >= n_stages * P1.B) return;   // whole warps leave
  const int b = (n_stages == 2) ? unit >> 1 : unit;
  const bool second = (n_stages == 2) && (unit & 1);
  ScanOut o;
  if (!second) {
    o = scan_unit<T>(P1, b, lane, true, -1, nullptr, 0);
  } else {
    int L1, n2;
    stage1_prefix<T>(P1, P2.K, b, lane, &L1, &n2);
    o = scan_unit<T>(P2, b, lane, true, n2, P1.tokens + b * P1.K, L1);
  }
  if (lane == 0) {
    int next = -1;
    bool draw = false;
    if (o.L < o.nv) {
      if (o.flags & (kFlagSmallNonfinite | kFlagLargeNonfinite)) next = -2;   // no distribution to draw from
      else draw = true;
    }
    ds.need[unit] = draw ? 1 : 0;
    if (draw) {
      DrawRecord r;
      r.L = o.L; r.u2 = o.u2; r.m2l = o.m2l; r.l2sl = o.l2sl; r.m2s = o.m2s; r.l2ss = o.l2ss; r.resid = o.resid; r.unit = unit;
      ds.record[unit] = r;
    } else {
      write_results(second ? P2 : P1, b, o.L, next);
    }
  }
}

template <typename T>
__device__ __forceinline__ RowView<T> draw_row(const StageParams& P, const int b, const DrawRecord& r) {
  RowView<T> row;
  row.large = static_cast<const T*>(P.large) + b * P.seq_stride_large + static_cast<long long>(r.L) * P.V;
  row.small = static_cast<const T*>(P.small) + b * P.seq_stride_small + static_cast<long long>(r.L) * P.V;
  row.V = P.V;
  row.vec_ok = ((reinterpret_cast<uintptr_t>(row.large) | reinterpret_cast<uintptr_t>(row.small)) & 15u) == 0 &&
               (P.V % Elem<T>::kPerVec) == 0;
  row.c = P.c;
  row.m2l = r.m2l; row.l2sl = r.l2sl;
  row.m2s = r.m2s; row.l2ss = r.l2ss;
  row.from_large = (P.mode == kModeAssisted) || !(r.resid > 0.f);
  return row;
}

template <typename T>
struct TileShared {
  RowView<T> row[kFinBatch];            // the rows of a batch of (record, tile) pairs
  double* out[kFinBatch];               // where each pair's total goes
  int i_base[kFinBatch];                // first vocabulary index of each pair's tile
  float warp_tile[kFinBatch][32];
  unsigned short list[kDrawMaxUnits];   // the units that draw, in unit order
  int warp_count[32];
  int n_list;
};

// Tile launch: level 0 of every draw. One CTA per SM; any grid size gives the same totals.
template <typename T>
__global__ void __launch_bounds__(kFinThreads) finalize_tiles_kernel(const StageParams P1, const StageParams P2, const int n_stages,
                                                                     const DrawScratch ds) {
  __shared__ TileShared<T> S;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int units = n_stages * P1.B;
  // every CTA builds the same list of drawing units, in unit order
  if (tid == 0) S.n_list = 0;
  wait_for_previous_launch();
  release_next_launch();
  __syncthreads();
  for (int base = 0; base < units; base += kFinThreads) {
    const int unit = base + tid;
    const bool need = unit < units && ds.need[unit] != 0;
    const unsigned m = __ballot_sync(0xffffffffu, need);
    if (lane == 0) S.warp_count[warp] = __popc(m);
    __syncthreads();
    int before = S.n_list;
    for (int k = 0; k < warp; ++k) before += S.warp_count[k];
    if (need) {
      const int pos = before + __popc(m & ((1u << lane) - 1u));
      S.list[pos] = static_cast<unsigned short>(unit);
      if (pos % static_cast<int>(gridDim.x) == static_cast<int>(blockIdx.x)) ds.drawn[pos] = ds.record[unit];   // for the pick launch
    }
    __syncthreads();
    if (tid == 0) {
      int total = S.n_list;
      for (int k = 0; k < kFinThreads / 32; ++k) total += S.warp_count[k];
      S.n_list = total;
    }
    __syncthreads();
  }
  const int n_list = S.n_list;
  if (blockIdx.x == 0 && tid == 0) ds.count[0] = n_list;
  if (n_list == 0) return;
  const int n_tiles = (P1.V + kFinTile - 1) / kFinTile;
  const int items = n_list * n_tiles;   // <= kDrawMaxUnits * kDrawMaxTiles

  for (int first = blockIdx.x; first < items; first += static_cast<int>(gridDim.x) * kFinBatch) {
    const int nb = min(kFinBatch, (items - first + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x));
    if (tid < nb) {
      const int item = first + tid * static_cast<int>(gridDim.x);
      const int d = item / n_tiles, j = item % n_tiles;
      const int unit = S.list[d];
      const bool second = (n_stages == 2) && (unit & 1);
      S.row[tid] = draw_row<T>(second ? P2 : P1, (n_stages == 2) ? unit >> 1 : unit, ds.record[unit]);
      S.out[tid] = ds.tile_total + d * kDrawMaxTiles + j;
      S.i_base[tid] = j * kFinTile;
    }
    __syncthreads();
    // the loads of kTileDepth pairs (32 registers of vectors) are issued before the first of them is used
    constexpr int kTileDepth = 4 / RowView<T>::kVecs;
    for (int m = 0; m < nb; m += kTileDepth) {
      uint4 rl[kTileDepth][RowView<T>::kVecs], rs[kTileDepth][RowView<T>::kVecs];
      bool fetched[kTileDepth];
#pragma unroll
      for (int d = 0; d < kTileDepth; ++d) {
        fetched[d] = false;
        if (m + d < nb) {
          const int i0 = S.i_base[m + d] + tid * kFinElemsPerThread;
          fetched[d] = S.row[m + d].whole(i0);
          if (fetched[d]) S.row[m + d].fetch(i0, rl[d], rs[d]);
        }
      }
#pragma unroll
      for (int d = 0; d < kTileDepth; ++d) {
        if (m + d < nb) {   // uniform across the CTA
          float w[kFinElemsPerThread];
          if (fetched[d]) S.row[m + d].weights_fetched(rl[d], rs[d], w);
          else S.row[m + d].weights(S.i_base[m + d] + tid * kFinElemsPerThread, w);
          float ts = 0.f;
#pragma unroll
          for (int e = 0; e < kFinElemsPerThread; ++e) ts += w[e];
          ts = warp_reduce<OpSum>(ts);
          if (lane == 0) S.warp_tile[m + d][warp] = ts;
        }
      }
    }
    __syncthreads();
    if (tid < nb) {
      double tt = 0.0;
      for (int k = 0; k < 32; ++k) tt += static_cast<double>(S.warp_tile[tid][k]);
      *S.out[tid] = tt;
    }
    __syncthreads();   // the batch's shared memory is free again
  }
}

// Pick launch: the pick among the tile totals and levels 1 to 3, one draw per CTA at a time.
template <typename T>
__global__ void __launch_bounds__(kFinThreads) finalize_pick_kernel(const StageParams P1, const StageParams P2, const int n_stages,
                                                                    const DrawScratch ds) {
  __shared__ FinShared S;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  wait_for_previous_launch();
  const int n_tiles = (P1.V + kFinTile - 1) / kFinTile;
  // the first draw's record and totals are asked for together with the count (stale but allocated memory if this
  // CTA has no draw)
  const bool may = static_cast<int>(blockIdx.x) < n_stages * P1.B;
  DrawRecord rec = may ? ds.drawn[blockIdx.x] : DrawRecord{};
  double tt = (may && tid < n_tiles) ? ds.tile_total[blockIdx.x * kDrawMaxTiles + tid] : 0.0;
  const int n_list = ds.count[0];
  for (int d = blockIdx.x; d < n_list; d += gridDim.x) {
    if (d != static_cast<int>(blockIdx.x)) {
      rec = ds.drawn[d];
      if (tid < n_tiles) tt = ds.tile_total[d * kDrawMaxTiles + tid];
    }
    const int unit = rec.unit;
    const bool second = (n_stages == 2) && (unit & 1);
    const StageParams& P = second ? P2 : P1;
    const int b = (n_stages == 2) ? unit >> 1 : unit;
    RowView<T> row = draw_row<T>(P, b, rec);
    if (tid < n_tiles) S.tile_total[tid] = tt;
    if (tid == 0) S.sh_u2 = rec.u2;
    __syncthreads();
    if (tid == 0) pick_tile(S, n_tiles, row.from_large);
    __syncthreads();
    if (S.sh_tile == -2) {
      // the residual weights all came out zero although the row's residual mass did not: the totals again, over p_large
      row.from_large = true;
      for (int j = 0; j < n_tiles; ++j) {
        float w[kFinElemsPerThread];
        row.weights(j * kFinTile + tid * kFinElemsPerThread, w);
        float ts = 0.f;
#pragma unroll
        for (int e = 0; e < kFinElemsPerThread; ++e) ts += w[e];
        ts = warp_reduce<OpSum>(ts);
        if (lane == 0) S.warp_tile[0][warp] = ts;
        __syncthreads();
        if (tid == 0) {
          double tt = 0.0;
          for (int k = 0; k < 32; ++k) tt += static_cast<double>(S.warp_tile[0][k]);
          S.tile_total[j] = tt;
        }
        __syncthreads();
      }
      if (tid == 0) pick_tile(S, n_tiles, true);
      __syncthreads();
    }
    const int tile = S.sh_tile;
    int next = -1;
    if (tile >= 0) {
      descend_tile<T>(row, S, tile);
      next = S.sh_token;
    }
    if (tid == 0) write_results(P, b, rec.L, next);
    __syncthreads();   // S is free for the next draw
  }
}

}  // namespace psd
