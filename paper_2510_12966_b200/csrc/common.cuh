// Shared device helpers of the verification kernels: row-statistics record, vector unpacking,
// special-function wrappers, warp/block reductions and the Philox4x32-10 generator.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace psd {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

enum : int { kFlagSmallNonfinite = 1, kFlagLargeNonfinite = 2, kFlagTokenRange = 4 };
enum : int { kModeFuzzy = 0, kModeStrict = 1, kModeFuzzyFallback = 2, kModeAssisted = 3 };
enum : int { kDivJS = 0, kDivTV = 1, kDivKL = 2 };

// What the statistics pass leaves per (sequence, position) row for the finalisation kernel.
// The log-sum-exp of the temperature-scaled logits is kept in the base-2 domain as two floats,
// log2(sum_i exp(z_i / T)) = m2 + l2s with m2 = max_i(z_i * c), l2s = log2(sum_i 2^(z_i * c - m2)),
// c = log2(e) / T, so that p_i = 2^((z_i * c - m2) - l2s). One float would quantise the sum of the two
// (magnitude ~20) to 2^-19 and shift every probability of the row by up to 7e-7 relative.
struct __align__(32) RowStats {
  float m2_small, l2s_small;
  float m2_large, l2s_large;
  float div;        // Div(P_large, P_small) of Sec. 3.1 in nats (JS), or TV / KL when selected
  float resid;      // R = sum_i max(0, p_large_i - p_small_i)
  int flags;        // kFlag* bits for non-finite rows
  int pad;
};

struct StageParams {
  const void* small;
  const void* large;
  const int32_t* tokens;
  const int32_t* n_valid;
  int B, K, V;
  long long seq_stride_small, seq_stride_large;  // elements
  float c;            // log2(e) * inv_temperature
  float threshold;
  int mode, div_kind;
  unsigned long long seed, offset;
  RowStats* stats;
  int32_t* out_accept_len;
  int32_t* out_next_token;
  float* out_div;
  float* out_p_small_tok;
  float* out_p_large_tok;
  float* out_resid_mass;
  int32_t* out_row_flags;
  // two-stage wrapper: when window != nullptr the finalisation of stage 1 also writes the stage-2
  // window [B, K_window] (accepted draft tokens followed by the correction token) and its length.
  int32_t* window;
  int32_t* n_window;
  int K_window;
  int* status;        // device status word (bounded-wait timeouts)
  // Second row set of the statistics pass (two-stage wrapper): rows [B*K, B*K + B*K2) of the launch are
  // the stage-2 pairs (qualifier as the small model, target as the large one). K2 == 0: none.
  const void* small2;
  const void* large2;
  long long seq_stride_small2, seq_stride_large2;
  int K2;
  RowStats* stats2;
  // 1: the large tensor holds K + 1 rows per sequence; a sequence whose valid positions were all accepted
  // gets its next token from the row after the last valid one (the larger model's bonus token, Sec. 1).
  int bonus;
  // Two-stage wrapper, optional: the window lengths of the first fill_cap sequences are also stored here (host
  // memory mapped into the device), where the host reads them to choose its schedule for later calls.
  int32_t* fill_out;
  int fill_cap;
  // Index of this call's sequence 0 in the whole batch: row (b, k) draws with Philox counter word 0 =
  // (seq_base + b) * K + k and sequence b's bonus draw with seq_base + b, so a slice of a batch draws what the
  // whole batch draws.
  long long seq_base;
};

// ---- special functions (single MUFU instruction each) -------------------------------------------------
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2_approx(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// max that returns NaN when either operand is NaN, so a poisoned row shows in its row maximum
__device__ __forceinline__ float max_nan(float a, float b) {
  float y;
  asm("max.NaN.f32 %0, %1, %2;" : "=f"(y) : "f"(a), "f"(b));
  return y;
}

// ---- element access ---------------------------------------------------------------------------------
template <typename T> struct Elem;
template <> struct Elem<float> {
  static constexpr int kPerVec = 4;  // elements per 16-byte vector
  __device__ static __forceinline__ float load(const float* p, long long i) { return __ldg(p + i); }
  __device__ static __forceinline__ void unpack(const uint4& u, float* x) {
    x[0] = __uint_as_float(u.x); x[1] = __uint_as_float(u.y);
    x[2] = __uint_as_float(u.z); x[3] = __uint_as_float(u.w);
  }
};
template <> struct Elem<__nv_bfloat16> {
  static constexpr int kPerVec = 8;
  __device__ static __forceinline__ float load(const __nv_bfloat16* p, long long i) {
    const unsigned short b = __ldg(reinterpret_cast<const unsigned short*>(p) + i);
    return __uint_as_float(static_cast<unsigned>(b) << 16);
  }
  // bf16 is the upper half of a binary32: widen by shifting / masking
  __device__ static __forceinline__ void unpack(const uint4& u, float* x) {
    x[0] = __uint_as_float(u.x << 16); x[1] = __uint_as_float(u.x & 0xffff0000u);
    x[2] = __uint_as_float(u.y << 16); x[3] = __uint_as_float(u.y & 0xffff0000u);
    x[4] = __uint_as_float(u.z << 16); x[5] = __uint_as_float(u.z & 0xffff0000u);
    x[6] = __uint_as_float(u.w << 16); x[7] = __uint_as_float(u.w & 0xffff0000u);
  }
};

__device__ __forceinline__ uint4 ldg_vec(const void* base, long long vec_index) {
  return __ldg(reinterpret_cast<const uint4*>(base) + vec_index);
}

// ---- reductions -------------------------------------------------------------------------------------
struct OpSum {
  template <typename V> __device__ static V apply(V a, V b) { return a + b; }
};
struct OpMaxNan { __device__ static float apply(float a, float b) { return max_nan(a, b); } };

template <typename Op, typename V>
__device__ __forceinline__ V warp_reduce(V v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = Op::apply(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Reduce over the whole CTA; every thread gets the result. `scratch` holds >= 32 values. Fixed tree, so
// results are bit-identical from run to run.
template <typename Op, typename V>
__device__ __forceinline__ V block_reduce(V v, V* scratch, V identity) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
  v = warp_reduce<Op>(v);
  __syncthreads();  // scratch may still be read from a previous reduction
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  V r = (lane < nwarps) ? scratch[lane] : identity;
  r = warp_reduce<Op>(r);
  return r;
}

__device__ __forceinline__ unsigned block_reduce_or(unsigned v, unsigned* scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
  v = __reduce_or_sync(0xffffffffu, v);
  __syncthreads();
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  unsigned r = (lane < nwarps) ? scratch[lane] : 0u;
  return __reduce_or_sync(0xffffffffu, r);
}

// ---- Philox4x32-10 (Salmon et al., SC'11): 10 rounds, key bumped by the Weyl constants between rounds --
__device__ __forceinline__ uint4 philox4x32_10(uint4 ctr, uint2 key) {
  constexpr unsigned kM0 = 0xD2511F53u, kM1 = 0xCD9E8D57u, kW0 = 0x9E3779B9u, kW1 = 0xBB67AE85u;
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    const unsigned hi0 = __umulhi(kM0, ctr.x), lo0 = kM0 * ctr.x;
    const unsigned hi1 = __umulhi(kM1, ctr.z), lo1 = kM1 * ctr.z;
    ctr = make_uint4(hi1 ^ ctr.y ^ key.x, lo1, hi0 ^ ctr.w ^ key.y, lo0);
    key.x += kW0;
    key.y += kW1;
  }
  return ctr;
}

// The two uniforms of row r in [0, 1) with 24-bit mantissas: u for the strict coin flip, u2 for the
// inverse CDF. Counter (r, 0, offset_lo, offset_hi), key (seed_lo, seed_hi).
__device__ __forceinline__ void row_uniforms(unsigned long long seed, unsigned long long offset, unsigned r,
                                             float* u, float* u2) {
  const uint4 w = philox4x32_10(make_uint4(r, 0u, static_cast<unsigned>(offset), static_cast<unsigned>(offset >> 32)),
                                make_uint2(static_cast<unsigned>(seed), static_cast<unsigned>(seed >> 32)));
  *u = static_cast<float>(w.x >> 8) * (1.0f / 16777216.0f);
  *u2 = static_cast<float>(w.y >> 8) * (1.0f / 16777216.0f);
}

// The uniform behind a sequence's bonus draw: counter (b, 1, offset_lo, offset_hi), output word 1; word 1 of
// the counter keeps it apart from every row's (r, 0, ...).
__device__ __forceinline__ float bonus_uniform(unsigned long long seed, unsigned long long offset, unsigned b) {
  const uint4 w = philox4x32_10(make_uint4(b, 1u, static_cast<unsigned>(offset), static_cast<unsigned>(offset >> 32)),
                                make_uint2(static_cast<unsigned>(seed), static_cast<unsigned>(seed >> 32)));
  return static_cast<float>(w.y >> 8) * (1.0f / 16777216.0f);
}

}  // namespace psd
