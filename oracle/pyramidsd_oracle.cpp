// PyramidSD verification oracle — TEST INFRASTRUCTURE, not the product.
//
// A plain, slow, double-precision CPU statement of the two-stage hierarchical verification of
// Pyramid Speculative Decoding ("3-Model Speculative Decoding", Sec. 3.1-3.4 and Fig. 1). It exists so
// that the CUDA library can be checked against something written independently from the paper. It
// shares no code, header, table or helper with the CUDA path, and only tests, the smoke check and the
// bench's CPU-baseline leg may call it.
//
// The paper fixes the structure (per-position divergence test Div(P_large, P_small) <= tau in Sec. 3.1
// and the two-stage criterion in Sec. 3.2; prefix acceptance with fall-back to the larger model in
// Sec. 1; the "standard SD probability rule" on rejection and the assisted variant in Sec. 3.4; the
// draft->qualifier->target chaining in Fig. 1). It does not print the divergence, the residual formula
// or a random-number convention. The readings taken here:
//   * Div = Jensen-Shannon divergence in nats of the two full-vocabulary softmax distributions
//     (total variation and KL(large||small) are selectable extras);
//   * strict mode = standard speculative sampling: accept with probability min(1, p_large(x)/p_small(x));
//   * rejection = draw from max(0, p_large - p_small), normalised, by inverse CDF in index order;
//   * random numbers = Philox4x32-10 (Salmon et al., SC'11), one call per row.
// Parity status: the arithmetic below is pinned by tests against hand-computed values, closed forms,
// invariants, a chi-square Monte Carlo and published Philox known-answer vectors. The *choice* of
// Jensen-Shannon and of threshold-only fuzzy acceptance cannot be pinned by anything the paper prints:
// for those two choices "parity unpinned" against the authors' own code.
//
// No blocking, fusion or reordering: every sum runs over the vocabulary in index order.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

namespace {

enum { DT_F32 = 0, DT_BF16 = 1, DT_F64 = 2 };
enum { MODE_FUZZY = 0, MODE_STRICT = 1, MODE_FUZZY_SD_FALLBACK = 2, MODE_ASSISTED = 3 };
enum { DIV_JS = 0, DIV_TV = 1, DIV_KL = 2 };
enum { FLAG_SMALL_NONFINITE = 1, FLAG_LARGE_NONFINITE = 2, FLAG_TOKEN_RANGE = 4 };

// ---- Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3") ----
void philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4]) {
  const uint64_t M0 = 0xD2511F53ull, M1 = 0xCD9E8D57ull;
  const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
  uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
  uint32_t k0 = key_in[0], k1 = key_in[1];
  for (int round = 0; round < 10; ++round) {
    if (round > 0) { k0 += W0; k1 += W1; }
    const uint64_t prod0 = M0 * (uint64_t)c0;
    const uint64_t prod1 = M1 * (uint64_t)c2;
    const uint32_t hi0 = (uint32_t)(prod0 >> 32), lo0 = (uint32_t)prod0;
    const uint32_t hi1 = (uint32_t)(prod1 >> 32), lo1 = (uint32_t)prod1;
    const uint32_t n0 = hi1 ^ c1 ^ k0;
    const uint32_t n1 = lo1;
    const uint32_t n2 = hi0 ^ c3 ^ k1;
    const uint32_t n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// The two uniforms of row r: u decides the strict coin flip, u2 drives the inverse CDF.
// Counter = (r, 0, offset_lo, offset_hi), key = (seed_lo, seed_hi); 24-bit mantissas in [0, 1).
void row_uniforms(uint64_t seed, uint64_t offset, uint32_t r, double* u, double* u2) {
  const uint32_t ctr[4] = {r, 0u, (uint32_t)offset, (uint32_t)(offset >> 32)};
  const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t w[4];
  philox4x32_10(ctr, key, w);
  *u = (double)(w[0] >> 8) * (1.0 / 16777216.0);
  *u2 = (double)(w[1] >> 8) * (1.0 / 16777216.0);
}

// The uniform that drives a sequence's bonus draw (all positions accepted, Sec. 1: the larger model's next
// token comes for free). Counter = (b, 1, offset_lo, offset_hi): word 1 = 1 keeps it apart from every row's
// counter (b*K + k, 0, ...). Same 24-bit mantissa rule, taken from output word 1 like the other draws.
double bonus_uniform(uint64_t seed, uint64_t offset, uint32_t b) {
  const uint32_t ctr[4] = {b, 1u, (uint32_t)offset, (uint32_t)(offset >> 32)};
  const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t w[4];
  philox4x32_10(ctr, key, w);
  return (double)(w[1] >> 8) * (1.0 / 16777216.0);
}

// ---- logits -> double -------------------------------------------------------------------------------
double logit_at(const void* base, int dtype, size_t idx) {
  if (dtype == DT_F32) return (double)((const float*)base)[idx];
  if (dtype == DT_F64) return ((const double*)base)[idx];
  // bf16 = the upper 16 bits of an IEEE binary32
  const uint32_t bits = (uint32_t)((const uint16_t*)base)[idx] << 16;
  float f;
  std::memcpy(&f, &bits, 4);
  return (double)f;
}

// Softmax of one row (Sec. 3.1: P_M is the distribution over the next token). Returns false when the
// row holds a NaN or +inf, or no finite entry at all; -inf entries are legal and get probability 0.
bool softmax_row(const void* base, int dtype, size_t row_off, int V, double inv_temperature,
                 std::vector<double>& p) {
  p.resize(V);
  double m = -std::numeric_limits<double>::infinity();
  bool bad = false;
  for (int i = 0; i < V; ++i) {
    const double z = logit_at(base, dtype, row_off + i) * inv_temperature;
    if (std::isnan(z) || z == std::numeric_limits<double>::infinity()) bad = true;
    p[i] = z;
    if (z > m) m = z;
  }
  if (bad || m == -std::numeric_limits<double>::infinity()) return false;
  double S = 0.0;
  for (int i = 0; i < V; ++i) { p[i] = std::exp(p[i] - m); S += p[i]; }
  for (int i = 0; i < V; ++i) p[i] /= S;
  return true;
}

// Div(P_large, P_small) of Sec. 3.1, p = large, q = small. 0*ln(0) = 0.
double divergence(const std::vector<double>& p, const std::vector<double>& q, int kind) {
  const int V = (int)p.size();
  double D = 0.0;
  if (kind == DIV_JS) {
    for (int i = 0; i < V; ++i) {
      const double mix = 0.5 * (p[i] + q[i]);
      if (p[i] > 0.0) D += 0.5 * p[i] * std::log(p[i] / mix);
      if (q[i] > 0.0) D += 0.5 * q[i] * std::log(q[i] / mix);
    }
  } else if (kind == DIV_TV) {
    for (int i = 0; i < V; ++i) D += 0.5 * std::fabs(p[i] - q[i]);
  } else {  // KL(large || small)
    for (int i = 0; i < V; ++i) {
      if (p[i] > 0.0) {
        if (q[i] > 0.0) D += p[i] * std::log(p[i] / q[i]);
        else D = std::numeric_limits<double>::infinity();
      }
    }
  }
  return D;
}

// Mass of the residual distribution max(0, p_large - p_small) (the standard SD rule, Sec. 3.4).
double residual_mass(const std::vector<double>& p, const std::vector<double>& q) {
  double R = 0.0;
  for (size_t i = 0; i < p.size(); ++i) R += std::fmax(0.0, p[i] - q[i]);
  return R;
}

// Inverse CDF in index order: the smallest i whose inclusive prefix sum of w exceeds u2 * sum(w);
// if rounding leaves none, the last i with positive weight. -1 when all weights are zero.
int inverse_cdf(const std::vector<double>& w, double u2) {
  double total = 0.0;
  for (double x : w) total += x;
  const double target = u2 * total;
  double c = 0.0;
  int last_positive = -1;
  for (size_t i = 0; i < w.size(); ++i) {
    if (w[i] > 0.0) last_positive = (int)i;
    c += w[i];
    if (c > target && w[i] > 0.0) return (int)i;
  }
  return last_positive;
}

struct RowResult {
  double D, R, p_small_tok, p_large_tok, u, u2;
  int flags;
  int accept;
  int resample;  // token this row would emit if it were the first rejection
};

struct StageArgs {
  const void* small; const void* large; const int32_t* tokens;
  int B, K, V, dtype;
  int64_t stride_small, stride_large;  // elements between consecutive rows
  double tau; int mode; uint64_t seed, offset;
  const int32_t* n_valid; double inv_temperature; int div_kind;
  const int32_t* seq_ids;  // optional: global sequence index of each local sequence (for the Philox counter)
};

// Steps for one (sequence, position) row: softmaxes, divergence, residual mass, token probabilities,
// Philox uniforms, accept bit, and the token the row would emit on rejection.
void verify_row(const StageArgs& a, int r, RowResult& out) {
  std::vector<double> p, q;
  const bool ok_q = softmax_row(a.small, a.dtype, (size_t)r * (size_t)a.stride_small, a.V, a.inv_temperature, q);
  const bool ok_p = softmax_row(a.large, a.dtype, (size_t)r * (size_t)a.stride_large, a.V, a.inv_temperature, p);
  const int x = a.tokens[r];
  out.flags = (ok_q ? 0 : FLAG_SMALL_NONFINITE) | (ok_p ? 0 : FLAG_LARGE_NONFINITE) |
              ((x < 0 || x >= a.V) ? FLAG_TOKEN_RANGE : 0);
  // Philox counter word 0 is the row index b*K + k of the sequence's position in the full batch
  const int b_local = r / a.K, k_local = r % a.K;
  const uint32_t r_global = (uint32_t)((a.seq_ids ? a.seq_ids[b_local] : b_local) * a.K + k_local);
  row_uniforms(a.seed, a.offset, r_global, &out.u, &out.u2);
  const double nan = std::numeric_limits<double>::quiet_NaN();
  out.D = nan; out.R = nan; out.p_small_tok = nan; out.p_large_tok = nan;
  out.accept = 0; out.resample = -2;
  if (!ok_p || !ok_q) return;  // no distribution to verify against: reject, emit the invalid marker

  out.D = divergence(p, q, a.div_kind);
  out.R = residual_mass(p, q);
  double rho = 0.0;
  if (!(out.flags & FLAG_TOKEN_RANGE)) {
    out.p_large_tok = p[x];
    out.p_small_tok = q[x];
    if (q[x] > 0.0) rho = p[x] / q[x];
    else rho = (p[x] > 0.0) ? std::numeric_limits<double>::infinity() : 0.0;
  }
  const bool fuzzy_ok = out.D <= a.tau;                 // Sec. 3.1 / 3.2: Div <= tau
  const bool coin_ok = out.u < std::fmin(1.0, rho);     // standard SD acceptance
  bool acc = false;
  if (a.mode == MODE_FUZZY) acc = fuzzy_ok;
  else if (a.mode == MODE_STRICT || a.mode == MODE_ASSISTED) acc = coin_ok;
  else if (a.mode == MODE_FUZZY_SD_FALLBACK) acc = fuzzy_ok || coin_ok;
  if (out.flags) acc = false;
  out.accept = acc ? 1 : 0;

  // Token emitted if this row is the first rejection: residual rule, or (assisted variant, Sec. 3.4,
  // or a zero residual) a draw from the larger model's own distribution.
  std::vector<double> w(a.V);
  if (a.mode != MODE_ASSISTED && out.R > 0.0) {
    for (int i = 0; i < a.V; ++i) w[i] = std::fmax(0.0, p[i] - q[i]);
  } else {
    w = p;
  }
  out.resample = inverse_cdf(w, out.u2);
}

void run_rows(const StageArgs& a, std::vector<RowResult>& rows, int n_threads) {
  const int n_rows = a.B * a.K;
  rows.resize(n_rows);
  if (n_threads < 1) n_threads = 1;
  if (n_threads > n_rows) n_threads = n_rows > 0 ? n_rows : 1;
  auto work = [&](int t) {
    for (int r = t; r < n_rows; r += n_threads) {
      const int b = r / a.K, k = r % a.K;
      const int nv = a.n_valid ? a.n_valid[b] : a.K;
      if (k < nv) verify_row(a, r, rows[r]);
      else { RowResult z{}; z.resample = -1; rows[r] = z; }
    }
  };
  if (n_threads == 1) { work(0); return; }
  std::vector<std::thread> pool;
  for (int t = 0; t < n_threads; ++t) pool.emplace_back(work, t);
  for (auto& th : pool) th.join();
}

// Accepted-prefix length: number of leading accepted positions among the first n_valid (Sec. 1: on the
// first disagreement decoding falls back to the larger model).
int prefix_length(const int* accept, int n_valid) {
  int L = 0;
  while (L < n_valid && accept[L]) ++L;
  return L;
}

int verify_stage_impl(const StageArgs& a, int32_t* out_accept_len, int32_t* out_next_token,
                      double* out_div, double* out_p_small_tok, double* out_p_large_tok,
                      double* out_resid_mass, int32_t* out_row_flags, int32_t* out_accept_bits,
                      int n_threads) {
  if (a.B < 0 || a.K < 0 || a.V < 1) return -1;
  std::vector<RowResult> rows;
  run_rows(a, rows, n_threads);
  for (int b = 0; b < a.B; ++b) {
    int nv = a.n_valid ? a.n_valid[b] : a.K;
    if (nv < 0) nv = 0;
    if (nv > a.K) nv = a.K;
    std::vector<int> acc(a.K, 0);
    for (int k = 0; k < nv; ++k) acc[k] = rows[(size_t)b * a.K + k].accept;
    const int L = prefix_length(acc.data(), nv);
    out_accept_len[b] = L;
    out_next_token[b] = (L < nv) ? rows[(size_t)b * a.K + L].resample : -1;
  }
  for (int r = 0; r < a.B * a.K; ++r) {
    if (out_div) out_div[r] = rows[r].D;
    if (out_p_small_tok) out_p_small_tok[r] = rows[r].p_small_tok;
    if (out_p_large_tok) out_p_large_tok[r] = rows[r].p_large_tok;
    if (out_resid_mass) out_resid_mass[r] = rows[r].R;
    if (out_row_flags) out_row_flags[r] = rows[r].flags;
    if (out_accept_bits) out_accept_bits[r] = rows[r].accept;
  }
  return 0;
}

}  // namespace

extern "C" {

void psd_oracle_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
  philox4x32_10(ctr, key, out);
}

void psd_oracle_row_uniforms(uint64_t seed, uint64_t offset, uint32_t row, double* u, double* u2) {
  row_uniforms(seed, offset, row, u, u2);
}

// Softmax of one row of V logits into p (double[V]); returns 1 if the row was valid.
int psd_oracle_softmax(const void* logits, int dtype, int V, double inv_temperature, double* p) {
  std::vector<double> v;
  const bool ok = softmax_row(logits, dtype, 0, V, inv_temperature, v);
  for (int i = 0; i < V; ++i) p[i] = v[i];
  return ok ? 1 : 0;
}

double psd_oracle_divergence(const double* p_large, const double* p_small, int V, int kind) {
  return divergence(std::vector<double>(p_large, p_large + V), std::vector<double>(p_small, p_small + V), kind);
}

double psd_oracle_residual_mass(const double* p_large, const double* p_small, int V) {
  return residual_mass(std::vector<double>(p_large, p_large + V), std::vector<double>(p_small, p_small + V));
}

int psd_oracle_inverse_cdf(const double* w, int V, double u2) {
  return inverse_cdf(std::vector<double>(w, w + V), u2);
}

int psd_oracle_prefix_length(const int32_t* accept, int n_valid) { return prefix_length(accept, n_valid); }

// One verification stage (Sec. 3.1-3.2 for one model pair). Host pointers. Optional outputs may be null.
int psd_oracle_verify_stage(const void* logits_small, const void* logits_large, const int32_t* tokens,
                            int B, int K, int V, int dtype, int64_t stride_small, int64_t stride_large,
                            double tau, int mode, uint64_t seed, uint64_t offset,
                            const int32_t* n_valid, double inv_temperature, int div_kind,
                            const int32_t* seq_ids,
                            int32_t* out_accept_len, int32_t* out_next_token,
                            double* out_div, double* out_p_small_tok, double* out_p_large_tok,
                            double* out_resid_mass, int32_t* out_row_flags, int32_t* out_accept_bits,
                            int n_threads) {
  StageArgs a{logits_small, logits_large, tokens, B, K, V, dtype,
              stride_small ? stride_small : V, stride_large ? stride_large : V,
              tau, mode, seed, offset, n_valid, inv_temperature, div_kind, seq_ids};
  return verify_stage_impl(a, out_accept_len, out_next_token, out_div, out_p_small_tok, out_p_large_tok,
                           out_resid_mass, out_row_flags, out_accept_bits, n_threads);
}

// One stage where the larger model supplies K+1 rows per sequence ([B, K+1, V]): row k < K scores the
// token at position k, and the row after the last valid position is the distribution of the token that
// follows a fully accepted window (Sec. 1: every accepted run ends with a token of the larger model, the
// correction on a rejection or this bonus token otherwise). When all n_valid[b] positions are accepted,
// next_token[b] is drawn from softmax(large[b, n_valid[b], :]) by inverse CDF with the bonus uniform; a
// bonus row with no distribution (NaN, +inf, no finite entry) gives -2. Everything else is the plain stage.
int psd_oracle_verify_stage_bonus(const void* logits_small, const void* logits_large_k1, const int32_t* tokens,
                                  int B, int K, int V, int dtype, double tau, int mode, uint64_t seed,
                                  uint64_t offset, const int32_t* n_valid, double inv_temperature, int div_kind,
                                  const int32_t* seq_ids, int32_t* out_accept_len, int32_t* out_next_token,
                                  double* out_div, int n_threads) {
  const size_t es = dtype == DT_F32 ? 4 : dtype == DT_BF16 ? 2 : 8;
  // rows 0..K-1 of every sequence, made dense, are the ordinary stage's large logits
  std::vector<unsigned char> dense((size_t)B * K * V * es);
  for (int b = 0; b < B; ++b)
    std::memcpy(dense.data() + (size_t)b * K * V * es,
                (const unsigned char*)logits_large_k1 + (size_t)b * (K + 1) * V * es, (size_t)K * V * es);
  StageArgs a{logits_small, dense.data(), tokens, B, K, V, dtype, V, V,
              tau, mode, seed, offset, n_valid, inv_temperature, div_kind, seq_ids};
  const int rc = verify_stage_impl(a, out_accept_len, out_next_token, out_div, nullptr, nullptr, nullptr,
                                   nullptr, nullptr, n_threads);
  if (rc) return rc;
  for (int b = 0; b < B; ++b) {
    int nv = n_valid ? n_valid[b] : K;
    if (nv < 0) nv = 0;
    if (nv > K) nv = K;
    if (out_accept_len[b] != nv) continue;   // a rejection: the correction token stands
    std::vector<double> p;
    const bool ok = softmax_row(logits_large_k1, dtype, ((size_t)b * (K + 1) + nv) * (size_t)V, V, inv_temperature, p);
    if (!ok) { out_next_token[b] = -2; continue; }
    const uint32_t b_global = (uint32_t)(seq_ids ? seq_ids[b] : b);
    out_next_token[b] = inverse_cdf(p, bonus_uniform(seed, offset, b_global));
  }
  return 0;
}

double psd_oracle_bonus_uniform(uint64_t seed, uint64_t offset, uint32_t b) { return bonus_uniform(seed, offset, b); }

// Two-stage pyramid (Fig. 1): stage 1 verifies the K_d draft tokens against the qualifier with tau_q;
// the accepted prefix plus the qualifier's correction token form the window, cut to K_q; stage 2
// verifies the window against the target with tau_t, the qualifier's distribution standing in for the
// draft's. Stage 1 draws with `offset`, stage 2 with `offset + 1`. Each stage has its own acceptance mode:
// the assisted variant of Sec. 3.4 (PSD_A) replaces only the qualifier stage by assisted decoding -- strict
// acceptance, and on rejection a draw from the qualifier's own distribution -- while the target stage keeps
// its threshold tau_t; the fuzzy variant (PSD_F) uses the threshold rule in both.
int psd_oracle_verify(const void* logits_draft, const void* logits_qual, const void* logits_target,
                      const int32_t* draft_tokens, int B, int K_d, int K_q, int V, int dtype,
                      double tau_q, double tau_t, int mode_q, int mode_t, uint64_t seed, uint64_t offset,
                      double inv_temperature, int div_kind, const int32_t* seq_ids,
                      int32_t* out_accept_len_q, int32_t* out_next_token_q,
                      int32_t* out_accept_len, int32_t* out_next_token,
                      int32_t* out_window /* [B,K_q] or null */, int32_t* out_n_window /* [B] or null */,
                      double* out_div_q /* [B,K_d] or null */, double* out_div_t /* [B,K_q] or null */,
                      int n_threads) {
  if (K_q > K_d || K_q < 0) return -1;
  StageArgs s1{logits_draft, logits_qual, draft_tokens, B, K_d, V, dtype, V, V,
               tau_q, mode_q, seed, offset, nullptr, inv_temperature, div_kind, seq_ids};
  int rc = verify_stage_impl(s1, out_accept_len_q, out_next_token_q, out_div_q, nullptr, nullptr, nullptr,
                             nullptr, nullptr, n_threads);
  if (rc) return rc;
  std::vector<int32_t> window((size_t)B * K_q, 0), n2(B, 0);
  for (int b = 0; b < B; ++b) {
    const int L1 = out_accept_len_q[b];
    const int t1 = out_next_token_q[b];
    const int have = L1 + (t1 >= 0 ? 1 : 0);
    n2[b] = have < K_q ? have : K_q;
    for (int j = 0; j < n2[b]; ++j)
      window[(size_t)b * K_q + j] = (j < L1) ? draft_tokens[(size_t)b * K_d + j] : t1;
  }
  // The qualifier's rows 0..K_q-1 of each sequence are the small model of stage 2: row stride K_d*V
  // between sequences is expressed by handing the stage a [B,K_q] view with per-row stride V inside a
  // sequence; since rows are addressed as r*stride, copy the view into a dense buffer first.
  const size_t es = dtype == DT_F32 ? 4 : dtype == DT_BF16 ? 2 : 8;
  std::vector<unsigned char> qual_view((size_t)B * K_q * V * es);
  for (int b = 0; b < B; ++b)
    std::memcpy(qual_view.data() + (size_t)b * K_q * V * es,
                (const unsigned char*)logits_qual + (size_t)b * K_d * V * es, (size_t)K_q * V * es);
  StageArgs s2{qual_view.data(), logits_target, window.data(), B, K_q, V, dtype, V, V,
               tau_t, mode_t, seed, offset + 1, n2.data(), inv_temperature, div_kind, seq_ids};
  rc = verify_stage_impl(s2, out_accept_len, out_next_token, out_div_t, nullptr, nullptr, nullptr,
                         nullptr, nullptr, n_threads);
  if (out_window) std::memcpy(out_window, window.data(), window.size() * sizeof(int32_t));
  if (out_n_window) std::memcpy(out_n_window, n2.data(), n2.size() * sizeof(int32_t));
  return rc;
}

// Fused-LM-head variant: the large model's logits are hidden x W, taken in double from the bf16
// operands and NOT rounded back to bf16. hidden [M,d] and W [d,V] are bf16, row-major; out [M,V] double.
void psd_oracle_lmhead_logits(const void* hidden, const void* W, int M, int d, int V, double* out,
                              int n_threads) {
  if (n_threads < 1) n_threads = 1;
  auto work = [&](int t) {
    for (int r = t; r < M; r += n_threads) {
      double* z = out + (size_t)r * V;
      for (int v = 0; v < V; ++v) z[v] = 0.0;
      for (int j = 0; j < d; ++j) {
        const double hj = logit_at(hidden, DT_BF16, (size_t)r * d + j);
        for (int v = 0; v < V; ++v) z[v] += hj * logit_at(W, DT_BF16, (size_t)j * V + v);
      }
    }
  };
  if (n_threads == 1) { work(0); return; }
  std::vector<std::thread> pool;
  for (int t = 0; t < n_threads; ++t) pool.emplace_back(work, t);
  for (auto& th : pool) th.join();
}

// Single stage where the two models' logits may have different element types (fused variant: small
// logits bf16, large logits double).
int psd_oracle_verify_stage_mixed(const void* logits_small, int dtype_small, const void* logits_large,
                                  int dtype_large, const int32_t* tokens, int B, int K, int V,
                                  double tau, int mode, uint64_t seed, uint64_t offset, int div_kind,
                                  int32_t* out_accept_len, int32_t* out_next_token, double* out_div,
                                  double* out_resid_mass, int n_threads) {
  // Bring both to double, exactly, then run the ordinary stage.
  const size_t n = (size_t)B * K * V;
  std::vector<double> s(n), l(n);
  for (size_t i = 0; i < n; ++i) { s[i] = logit_at(logits_small, dtype_small, i); l[i] = logit_at(logits_large, dtype_large, i); }
  StageArgs a{s.data(), l.data(), tokens, B, K, V, DT_F64, V, V, tau, mode, seed, offset, nullptr, 1.0, div_kind, nullptr};
  return verify_stage_impl(a, out_accept_len, out_next_token, out_div, nullptr, nullptr, out_resid_mass,
                           nullptr, nullptr, n_threads);
}

}  // extern "C"
