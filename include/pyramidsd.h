/* pyramidsd.h — C ABI of the B200 (sm_100a) two-stage verification library for Pyramid Speculative
 * Decoding ("3-Model Speculative Decoding").
 *
 * What the calls compute, per (sequence b, speculative position k) row r = b*K + k, for a "small" and a
 * "large" model (draft/qualifier in stage 1, qualifier/target in stage 2 — Fig. 1 and Sec. 3.2):
 *   1. softmax of both models' full-vocabulary logits (Sec. 3.1: P_M is the next-token distribution);
 *   2. the divergence Div(P_large, P_small) of Sec. 3.1 — Jensen-Shannon in nats by default;
 *   3. acceptance: fuzzy mode accepts when Div <= threshold (Sec. 3.1, two-stage criterion of Sec. 3.2);
 *      strict mode is standard speculative sampling, u < min(1, p_large(x)/p_small(x)) (Sec. 3.1-3.2);
 *   4. per sequence, the length of the accepted prefix (Sec. 1: fall back to the larger model at the
 *      first disagreement);
 *   5. at the first rejection, a token drawn from the normalised residual max(0, p_large - p_small)
 *      ("standard SD probability rule", Sec. 3.4) by inverse CDF in vocabulary order, or from p_large
 *      itself in the assisted variant (Sec. 3.4).
 * Random numbers: one Philox4x32-10 block per row, counter (r, 0, offset_lo, offset_hi), key
 * (seed_lo, seed_hi); u = (word0 >> 8) * 2^-24 decides the strict coin flip, u' = (word1 >> 8) * 2^-24
 * drives the inverse CDF. The two-stage wrapper uses `offset` for stage 1 and `offset + 1` for stage 2.
 * r is the row's index in the WHOLE batch: r = (seq_index_base + b) * K + k (low 32 bits), so that a call on a
 * slice of a batch -- a shard on another GPU, a micro-batch -- draws what the call on the whole batch draws.
 *
 * Conventions shared by every entry point unless stated otherwise:
 *   - All data pointers are DEVICE pointers owned by the caller; the library never frees or keeps them.
 *   - Logits are row-major [B, K, V], dtype float32 or bfloat16. Rows whose base address is 16-byte
 *     aligned with V * sizeof(element) a multiple of 16 take the vector path; other shapes take a
 *     scalar path — never an error. -inf logits are legal (probability 0). A row holding NaN or +inf,
 *     or no finite entry, or a token outside [0, V), is flagged and rejected; a flagged non-finite row
 *     at the first rejection emits token -2. Finite logits are meant to be of ordinary size: beyond about
 *     1e9 in magnitude the product with log2(e)/T is rounded by more than the exponent range of a float and
 *     the row may be flagged as if it were not finite.
 *   - out_accept_len[b] in [0, n_valid[b]]; out_next_token[b] = resampled token at the first rejection,
 *     or -1 when every valid position was accepted.
 *   - Work is enqueued on the stream set by pyramidsd_set_stream (default: the legacy default stream)
 *     or given in the argument struct; calls return without synchronising. Scratch memory comes from
 *     the caller's workspace when one is supplied (pyramidsd_workspace_bytes /
 *     pyramidsd_pyramid_workspace_bytes), otherwise from library-owned buffers kept per (device, stream):
 *     a call only ever touches the buffers of the stream it runs on, so calls on different streams, from
 *     one host thread or several, do not share scratch. Such a buffer is created with cudaMalloc the
 *     first time a stream is used and grown when a larger call arrives (growing waits for that stream's
 *     earlier work, frees, allocates). At most PSD_MAX_STREAMS streams per device get buffers; a call on
 *     yet another stream without a workspace returns PSD_ERR_WORKSPACE (see pyramidsd_release_stream). Two host
 *     threads that share one stream are serialised for the duration of the enqueue. A stage or pyramid call
 *     that brings its workspace uses no library buffer at all (its status word sits in the workspace's last
 *     256 bytes and is cleared on the stream): it allocates nothing and synchronises nothing.
 *   - Return value: PSD_OK or a negative psd_status. Arguments are validated on the host before any
 *     launch; nothing is launched on error. Device-side bounded waits that give up report
 *     PSD_ERR_TIMEOUT through pyramidsd_last_status().
 */
#define PSD_MAX_STREAMS 16
#ifndef PYRAMIDSD_H_
#define PYRAMIDSD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { PSD_F32 = 0, PSD_BF16 = 1 } psd_dtype;

typedef enum {
  PSD_FUZZY = 0,             /* accept iff Div <= threshold (Sec. 3.1, 3.2) */
  PSD_STRICT = 1,            /* standard speculative sampling (Sec. 3.1 "standard SD", tau = 0 end) */
  PSD_FUZZY_SD_FALLBACK = 2, /* Div <= threshold OR the strict coin flip succeeds */
  PSD_ASSISTED = 3           /* strict acceptance; on rejection draw from p_large itself (Sec. 3.4) */
} psd_mode;

/* The divergence `Div` of Sec. 3.1, which the paper leaves open ("a divergence measure"): Jensen-Shannon in nats
 * (the default: bounded by ln 2, so the paper's thresholds 0.2 .. 0.5 mean something), total variation, or
 * KL(large || small). The terms of KL separate -- sum_i p_i (log p_i - log q_i) needs the normalisers only as two
 * numbers at the end -- so a call with PSD_DIV_KL that asks for no per-row residual masses (out_resid_mass, or
 * out_resid_q / out_resid_t, NULL) and has at least one row per SM takes both softmaxes and the divergence in ONE
 * pass over the logits: half the exponentials of the other kinds and every byte read once, which on bf16 logits
 * is the difference between the special-function unit and HBM as the bound. */
typedef enum { PSD_DIV_JS = 0, PSD_DIV_TV = 1, PSD_DIV_KL = 2 } psd_div_kind;

typedef enum {
  PSD_OK = 0,
  PSD_ERR_INVALID_ARG = -1,
  PSD_ERR_UNSUPPORTED = -2,
  PSD_ERR_WORKSPACE = -3,
  PSD_ERR_CUDA = -4,
  PSD_ERR_TIMEOUT = -5
} psd_status;

/* Per-row flag bits written to out_row_flags. */
#define PSD_FLAG_SMALL_NONFINITE 1
#define PSD_FLAG_LARGE_NONFINITE 2
#define PSD_FLAG_TOKEN_RANGE 4

/* Kernel selection for the per-row statistics pass. AUTO picks the fastest variant the shape allows. */
typedef enum {
  PSD_KERNEL_AUTO = 0,
  PSD_KERNEL_BASELINE = 1, /* one CTA per row, three passes over global memory */
  PSD_KERNEL_CLUSTER = 2,  /* one thread-block cluster per row pair; its slices sit in the CTAs' shared memory for both passes, or,
                            * for clusters of 1 or 2 CTAs on a large vocabulary, are copied in once per pass (second copy from L2) */
  PSD_KERNEL_CLUSTER_STREAMED = 3 /* the cluster kernel in its copied-in-once-per-pass form whatever the slice size (needs cluster_size);
                                   * same arithmetic, same bits as PSD_KERNEL_CLUSTER with that cluster size */
} psd_kernel_variant;

/* Extended single-stage arguments. Zero-initialise, set struct_size = sizeof(psd_stage_args), fill what
 * you need; every optional field left zero means "off"/default. */
typedef struct psd_stage_args {
  uint32_t struct_size;
  int32_t dtype;                 /* psd_dtype */
  const void* logits_small;      /* [B, K, V] device */
  const void* logits_large;      /* [B, K, V] device */
  const int32_t* tokens;         /* [B, K] device, each in [0, V) */
  int32_t B, K, V;
  int32_t mode;                  /* psd_mode */
  int32_t div_kind;              /* psd_div_kind */
  float threshold;
  float inv_temperature;         /* logits are multiplied by this before the softmax; 0 means 1 (Sec. 4.1 uses T = 0.7) */
  int64_t seq_stride_small;      /* elements between sequences; 0 means K * V. Rows inside a sequence are V apart. */
  int64_t seq_stride_large;
  uint64_t philox_seed, philox_offset;
  const int32_t* n_valid;        /* [B] device or NULL: only positions k < n_valid[b] take part */
  int32_t* out_accept_len;       /* [B] device, required */
  int32_t* out_next_token;       /* [B] device, required */
  float* out_div;                /* [B, K] device or NULL */
  float* out_p_small_tok;        /* [B, K] device or NULL */
  float* out_p_large_tok;        /* [B, K] device or NULL */
  float* out_resid_mass;         /* [B, K] device or NULL (NULL lets PSD_DIV_KL take one pass: see psd_div_kind) */
  int32_t* out_row_flags;        /* [B, K] device or NULL */
  void* workspace;               /* device, >= pyramidsd_workspace_bytes(B, K, V, dtype), 256-byte aligned; NULL = library-owned */
  size_t workspace_bytes;
  void* stream;                  /* cudaStream_t, or NULL for the stream set by pyramidsd_set_stream */
  int32_t use_stream_field;      /* non-zero: take `stream` even when it is NULL (the legacy default stream) */
  int32_t kernel_variant;        /* psd_kernel_variant */
  int32_t cluster_size;          /* CTAs per cluster for the cluster kernel (1..16); 0 = chosen by the library. Results are
                                  * bit-identical run to run for a given size; different sizes differ in the last bits */
  int32_t large_has_bonus_row;   /* 1: logits_large is [B, K + 1, V] (seq_stride_large 0 then means (K + 1) * V). Row k < K scores
                                  * position k as usual. A sequence whose valid positions were ALL accepted gets, instead of -1,
                                  * a next token drawn from the softmax of the row after its last valid position (row
                                  * n_valid[b], or K) -- the larger model's own next token, which ends every accepted run
                                  * (Sec. 1) -- by inverse CDF with the uniform of Philox counter (b, 1, offset_lo, offset_hi),
                                  * word 1; -2 if that row holds NaN, +inf or no finite logit. */
  int32_t reserved0;
  int64_t seq_index_base;        /* index of this call's sequence 0 in the whole batch (see the Philox counter above and the
                                  * bonus counter): 0 for an unsharded call; >= 0 */
} psd_stage_args;

/* One verification stage (Sec. 3.1 for one model pair; Sec. 3.2 applies it twice). Jensen-Shannon
 * divergence, temperature 1, all K positions valid. Device pointers. Asynchronous on the library stream. */
int pyramidsd_verify_stage(const void* logits_small, const void* logits_large, const int32_t* draft_tokens,
                           int B, int K, int V, psd_dtype dtype, float threshold, psd_mode mode,
                           uint64_t philox_seed, uint64_t offset,
                           int32_t* out_accept_len, int32_t* out_next_token);

/* Same stage with every option exposed (strides, n_valid, temperature, divergence kind, per-row outputs,
 * caller workspace, stream, kernel variant). Returns PSD_ERR_INVALID_ARG on a NULL required pointer,
 * non-positive V, negative B/K, K > 32, an unknown enum value or a wrong struct_size; PSD_ERR_WORKSPACE
 * when a supplied workspace is too small or misaligned. B == 0 or K == 0 is a valid empty call. */
int pyramidsd_verify_stage_ex(const psd_stage_args* args);

/* Two-stage pyramid (Fig. 1, Sec. 3.2): stage 1 verifies the K_d draft tokens against the qualifier
 * with tau_q; the accepted prefix followed by the qualifier's correction token forms the window, cut to
 * K_q tokens; stage 2 verifies the window against the target with tau_t, with the qualifier's
 * distribution (rows 0..K_q-1 of each sequence of logits_qual) as the small model. Requires
 * 1 <= K_q <= K_d <= 32. logits_draft and logits_qual are [B, K_d, V], logits_target is [B, K_q, V].
 * Stage-1 results go to out_accept_len_q / out_next_token_q, final results to out_accept_len /
 * out_next_token (all [B], device). Consumes Philox offsets `offset` and `offset + 1`. */
int pyramidsd_verify(const void* logits_draft, const void* logits_qual, const void* logits_target,
                     const int32_t* draft_tokens, int B, int K_d, int K_q, int V, psd_dtype dtype,
                     float tau_q, float tau_t, psd_mode mode, uint64_t philox_seed, uint64_t offset,
                     int32_t* out_accept_len_q, int32_t* out_next_token_q,
                     int32_t* out_accept_len, int32_t* out_next_token);

/* The two-stage pyramid with every option exposed. Zero-initialise, set struct_size, fill what you need.
 *   mode_q / mode_t   acceptance mode of the qualifier stage and of the target stage. PSD_F of the paper is
 *                     (PSD_FUZZY, PSD_FUZZY); PSD_A (Sec. 3.4: assisted decoding in place of tau_Q, on rejection
 *                     a draw from the qualifier's own distribution, the target stage unchanged) is
 *                     (PSD_ASSISTED, PSD_FUZZY), and tau_q is then unused.
 *   seq_index_base    as in psd_stage_args: a call on sequences [base, base + B) of a batch returns, bit for
 *                     bit, what the call on the whole batch returns for them.
 *   target_has_bonus_row  logits_target is [B, K_q + 1, V] (see pyramidsd_verify_bonus).
 *   out_div_q [B, K_d], out_resid_q [B, K_d], out_div_t [B, K_q], out_resid_t [B, K_q]: per-row divergence and
 *                     residual mass of the two stages, or NULL. Stage-2 rows at or beyond the window hold 0.
 *   out_window [B, K_q], out_n_window [B]: the stage-2 window and its length, or NULL.
 *   schedule          PSD_TWO_STAGE_DEFAULT (the thread's policy) or one of the schedules below.
 *   workspace         >= pyramidsd_pyramid_workspace_bytes(B, K_d, K_q, V, dtype) bytes, 256-byte aligned; NULL =
 *                     library-owned. */
typedef struct psd_pyramid_args {
  uint32_t struct_size;
  int32_t dtype;                 /* psd_dtype */
  const void* logits_draft;      /* [B, K_d, V] device */
  const void* logits_qual;       /* [B, K_d, V] device */
  const void* logits_target;     /* [B, K_q (+ 1), V] device */
  const int32_t* draft_tokens;   /* [B, K_d] device */
  int32_t B, K_d, K_q, V;
  int32_t mode_q, mode_t;        /* psd_mode */
  float tau_q, tau_t;
  float inv_temperature;         /* 0 means 1 */
  int32_t div_kind;              /* psd_div_kind */
  uint64_t philox_seed, philox_offset;
  int64_t seq_index_base;
  int32_t target_has_bonus_row;
  int32_t schedule;
  int32_t* out_accept_len_q;     /* [B] device, required */
  int32_t* out_next_token_q;     /* [B] device, required */
  int32_t* out_accept_len;       /* [B] device, required */
  int32_t* out_next_token;       /* [B] device, required */
  float* out_div_q;
  float* out_resid_q;
  float* out_div_t;
  float* out_resid_t;
  int32_t* out_window;
  int32_t* out_n_window;
  void* workspace;
  size_t workspace_bytes;
  void* stream;                  /* cudaStream_t, or NULL for the stream set by pyramidsd_set_stream */
  int32_t use_stream_field;      /* non-zero: take `stream` even when it is NULL */
  int32_t kernel_variant;        /* PSD_KERNEL_AUTO or PSD_KERNEL_BASELINE */
} psd_pyramid_args;
int pyramidsd_verify_ex(const psd_pyramid_args* args);
size_t pyramidsd_pyramid_workspace_bytes(int B, int K_d, int K_q, int V, psd_dtype dtype);

/* pyramidsd_verify for a target that supplies one more row: logits_target is [B, K_q + 1, V]. Stage 1, the
 * window and the accept lengths are those of pyramidsd_verify; a window whose tokens were all accepted by
 * the target gets its next token from the target's row after the window (see large_has_bonus_row above)
 * instead of -1, so the caller needs no sampler of its own (Sec. 1, Sec. 3.4). */
int pyramidsd_verify_bonus(const void* logits_draft, const void* logits_qual, const void* logits_target,
                           const int32_t* draft_tokens, int B, int K_d, int K_q, int V, psd_dtype dtype,
                           float tau_q, float tau_t, psd_mode mode, uint64_t philox_seed, uint64_t offset,
                           int32_t* out_accept_len_q, int32_t* out_next_token_q,
                           int32_t* out_accept_len, int32_t* out_next_token);

/* pyramidsd_verify with HOST pointers for every array: copies the three logits tensors and the tokens
 * to library-owned device staging buffers, runs both stages, copies the four [B] results back and
 * synchronises the stream before returning. For callers whose logits live in host memory; the copies
 * are part of the call. Pinned host memory makes the copies asynchronous up to the final sync. */
int pyramidsd_verify_host(const void* logits_draft, const void* logits_qual, const void* logits_target,
                          const int32_t* draft_tokens, int B, int K_d, int K_q, int V, psd_dtype dtype,
                          float tau_q, float tau_t, psd_mode mode, uint64_t philox_seed, uint64_t offset,
                          int32_t* out_accept_len_q, int32_t* out_next_token_q,
                          int32_t* out_accept_len, int32_t* out_next_token);

/* (No counterpart in the paper: a packaging variant of pyramidsd_verify_stage.)
 * The same single stage for callers that must not allocate device memory: a component running inside
 * somebody else's memory plan (an inference server that hands every byte out at start-up and treats a
 * later cudaMalloc as a bug, a plug-in loaded into a process whose allocator it may not touch, code
 * running where an allocation would stall the whole device). The other entry points keep their per-row
 * statistics in a workspace the caller supplies or the library cudaMallocs on first use; this one keeps
 * them in an array built into the library image: PSD_NOALLOC_MAX_ROWS rows of 32 bytes plus one 256-byte
 * line, 256.25 KiB on every device that loads the library, until the process ends. It calls no
 * cudaMalloc / cudaFree and no allocating library routine.
 *   - Same arguments, results, Jensen-Shannon divergence and kernels as pyramidsd_verify_stage; the work
 *     is enqueued on `cuda_stream` (a cudaStream_t; NULL = the legacy default stream) and the call returns
 *     without synchronising.
 *   - B * K must not exceed PSD_NOALLOC_MAX_ROWS: a larger stage returns PSD_ERR_UNSUPPORTED (with a line on
 *     stderr) and launches nothing. Split such a batch over several calls, one after the other.
 *   - out_wait_timeout: device pointer to one int32, or NULL. It receives 0, or 1 if a bounded wait inside
 *     the kernels gave up (results are then invalid); pyramidsd_last_status() does not cover this call.
 *   - The first call on each device looks up the built-in array's device address
 *     (cudaGetSymbolAddress, with that device current). Make that first call outside any stream capture.
 *   - Every call on a device shares the one array, and the array keeps what the last call left in it.
 *     The call clears the only word that must start at zero. Two calls whose kernels overlap on the GPU
 *     (different streams, or several host threads) race on it: keep calls on one device in stream order. */
#define PSD_NOALLOC_MAX_ROWS 8192
int pyramidsd_verify_stage_noalloc(const void* logits_small, const void* logits_large, const int32_t* draft_tokens,
                                   int B, int K, int V, psd_dtype dtype, float threshold, psd_mode mode,
                                   uint64_t philox_seed, uint64_t offset,
                                   int32_t* out_accept_len, int32_t* out_next_token,
                                   int32_t* out_wait_timeout, void* cuda_stream);

/* One verification stage whose LARGE-model logits are produced inside the call: z_large = hidden x W^T
 * (the model's LM head), by a tensor-core GEMM whose epilogue does the softmax / divergence / residual
 * arithmetic of Sec. 3.1-3.2, so the large model's logits are never written to memory. Not in the paper
 * (it verifies logits the models have already produced); the rest of the stage is pyramidsd_verify_stage.
 *   hidden        [B*K, d_model] bf16, row-major (the large model's final hidden states), device
 *   w_t           [V, d_model]  bf16, row-major: the LM-head weight as checkpoints store it (out x in), device
 *   logits_small  [B, K, V] bf16, device; tokens [B, K] int32
 *   out_div, out_resid_mass  [B, K] float32 or NULL
 * Requires d_model a multiple of 64 (else PSD_ERR_UNSUPPORTED); hidden and w_t 16-byte aligned. Rows are
 * processed in blocks of 256 (B*K <= 256 is the intended case: one block, the weight streamed twice).
 * Jensen-Shannon divergence, temperature 1. Runs the GEMM twice (the divergence needs the large model's
 * normaliser first). Scratch (partial sums per row and 128-column tile) is library-owned, grown with
 * cudaMalloc on first use. Asynchronous on `cuda_stream`; device-side timeouts via pyramidsd_last_status(). */
int pyramidsd_verify_fused_lmhead(const void* hidden, const void* w_t, const void* logits_small,
                                  const int32_t* tokens, int B, int K, int d_model, int V, float threshold,
                                  psd_mode mode, uint64_t philox_seed, uint64_t offset,
                                  int32_t* out_accept_len, int32_t* out_next_token,
                                  float* out_div, float* out_resid_mass, void* cuda_stream);

/* The same call with every option exposed. Zero-initialise, set struct_size, fill what you need.
 *   seq_index_base  as in psd_stage_args.
 *   tile_variant    PSD_LMHEAD_TILES_AUTO (pairs of CTAs on 256 x 256 tiles, tcgen05 cta_group::2) or
 *                   PSD_LMHEAD_TILES_ONE_SM (one CTA per 256 x 128 tile); same results within rounding.
 *   div_kind        PSD_DIV_KL: KL(large || small), whose terms separate -- sum_i p_i (log p_i - log q_i) needs the
 *                   normalisers only at the end -- so the divergences are known after ONE sweep of the GEMM. The second
 *                   sweep then only serves the residual masses: it is launched, and returns at once unless some rejected
 *                   row draws from the residual (any mode but the assisted one) or out_resid_mass is wanted. With
 *                   PSD_ASSISTED, or when every position is accepted, the weight is streamed once per call. */
#define PSD_LMHEAD_TILES_AUTO 0
#define PSD_LMHEAD_TILES_ONE_SM 1
typedef struct psd_lmhead_args {
  uint32_t struct_size;
  int32_t mode;                  /* psd_mode */
  const void* hidden;            /* [B*K, d_model] bf16 device */
  const void* w_t;               /* [V, d_model] bf16 device */
  const void* logits_small;      /* [B, K, V] bf16 device */
  const int32_t* tokens;         /* [B, K] device */
  int32_t B, K, d_model, V;
  float threshold;
  int32_t tile_variant;
  int32_t div_kind;              /* PSD_DIV_JS or PSD_DIV_KL (PSD_DIV_TV: PSD_ERR_UNSUPPORTED) */
  int32_t reserved0;
  uint64_t philox_seed, philox_offset;
  int64_t seq_index_base;
  int32_t* out_accept_len;       /* [B] device, required */
  int32_t* out_next_token;       /* [B] device, required */
  float* out_div;                /* [B, K] or NULL */
  float* out_resid_mass;         /* [B, K] or NULL */
  void* stream;                  /* cudaStream_t; NULL = the legacy default stream */
} psd_lmhead_args;
int pyramidsd_verify_fused_lmhead_ex(const psd_lmhead_args* args);

/* Analytic throughput model of Sec. 3.3 (host arithmetic, no GPU): tokens per second of standard or
 * fuzzy speculative decoding with speculative length ell and acceptance rate beta between a small model
 * of speed v_small and a large one of speed v_large (tokens/s each),
 *     V = beta * (ell + 1) / (ell / v_small + 1 / v_large),
 * and of the pyramid: the draft/qualifier pair first (beta_qd, ell_d, v_draft, v_qual), whose result takes
 * the place of the small model's speed against the target (beta_tq, ell_q, v_target).
 * Return NaN on non-positive speeds or lengths, or acceptance rates outside [0, 1]. */
double pyramidsd_model_sd_throughput(double beta, double ell, double v_small, double v_large);
double pyramidsd_model_psd_throughput(double beta_qd, double ell_d, double v_draft, double v_qual,
                                      double beta_tq, double ell_q, double v_target);

/* The Philox uniforms the verification draws for rows 0..n_rows-1 with this seed and offset (see the
 * header comment for the counter layout): out_u[r] decides the strict coin flip of row r, out_u2[r]
 * drives its inverse CDF. Device pointers, float32 [n_rows]; either may be NULL. Lets a caller replay
 * or audit the random choices of a call. */
int pyramidsd_row_uniforms(uint64_t philox_seed, uint64_t offset, int n_rows, float* out_u, float* out_u2);

/* Scratch bytes one stage call of this shape needs (per-row statistics and the stage-2 window of the
 * wrapper). Pure host arithmetic; 0 on invalid arguments. */
size_t pyramidsd_workspace_bytes(int B, int K, int V, psd_dtype dtype);

/* How the two-stage calls schedule their launches (per host thread; every schedule returns the same results, bit
 * for bit: all of them cut a row over the CTAs of a cluster the same way). A "finalisation" below is one launch (a
 * cluster of CTAs per sequence), or, for batches that fill the GPU on calls that use the library's own scratch,
 * three small launches that hand over to one another (accept scan; the tile totals of every draw, spread over all
 * SMs; pick and descent) -- again with the same bits.
 *   PSD_TWO_STAGE_FUSED     two steps: one statistics launch over the B*K_d stage-1 row pairs and all B*K_q
 *                           stage-2 row pairs, one finalisation for both stages. Best when windows are
 *                           (nearly) full, as in the paper's pipeline, which keeps drafting until the window holds
 *                           K_q tokens (Fig. 1).
 *   PSD_TWO_STAGE_SEPARATE  four steps, stage by stage; stage 2 then skips the rows beyond each window, which
 *                           wins when acceptance is low and windows are short.
 *   PSD_TWO_STAGE_AUTO      (the default) the library chooses between the two per call. Stage 1 also leaves each
 *                           sequence's window length in a small host-mapped buffer (no copy, no synchronisation);
 *                           a later call with the same B and K_q on this device reads whatever lengths are there
 *                           -- those of a recent call -- and runs stage by stage when the unfilled part of the
 *                           windows is more than a tenth of all rows and the batch has at least 1024 rows, else
 *                           in two steps, over row triples where they apply (FUSED_ROWS below). The first call
 *                           of a shape runs in two steps.
 *   PSD_TWO_STAGE_FUSED_ROWS two steps like FUSED, but positions k < K_q are walked as row triples (draft,
 *                           qualifier, target): the qualifier row, which stage 1 uses as its large model and
 *                           stage 2 as its small one (Fig. 1), is read, widened and normalised once --
 *                           (2 K_d + K_q) V s bytes instead of 2 (K_d + K_q) V s. Applies where the statistics
 *                           kernel streams its rows twice (large batches); elsewhere it is FUSED. */
#define PSD_TWO_STAGE_DEFAULT 0
#define PSD_TWO_STAGE_FUSED 1
#define PSD_TWO_STAGE_SEPARATE 2
#define PSD_TWO_STAGE_AUTO 3
#define PSD_TWO_STAGE_FUSED_ROWS 4
/* PSD_TWO_STAGE_DEFAULT restores the library default. */
int pyramidsd_set_two_stage_policy(int policy);

/* Stream used by the entry points that carry no stream argument (a cudaStream_t; NULL = legacy default
 * stream). Per host thread. */
int pyramidsd_set_stream(void* cuda_stream);

/* Gives back the library-owned buffers of `cuda_stream` on the current device (after waiting for the stream's work)
 * and frees its place among the PSD_MAX_STREAMS streams; call it before destroying a stream the library has been
 * used on. PSD_OK also when the stream owns nothing. */
int pyramidsd_release_stream(void* cuda_stream);

/* Synchronises the stream of this host thread's most recent call (the library stream if there was none) and
 * returns PSD_OK, PSD_ERR_TIMEOUT if a device-side bounded wait gave up on that stream since its status was last
 * read, or PSD_ERR_CUDA if the stream reports an error. Clears that stream's status word. */
int pyramidsd_last_status(void);

const char* pyramidsd_version(void);
const char* pyramidsd_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* PYRAMIDSD_H_ */
