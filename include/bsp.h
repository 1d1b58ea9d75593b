/*
 * bsp.h -- C ABI of the backward-state-policy operator library for NVIDIA B200 (sm_100a).
 *
 * The paper ("Backward-State Policy Is Part of the Learning Algorithm") studies what each
 * backward *use* of a saved, rounded tensor reads: U the original, R the forward's rounding, N a
 * new stochastic rounding from a separate generator stream (Introduction; Section "One tensor,
 * two uses").  This library evaluates single operators under such a per-use policy and checks
 * each use against the paper's reference -- the gradient of the forward as it ran, rounding
 * passed straight through -- with a K-draw Monte-Carlo reduction, without any training.
 *
 * Conventions (all entry points):
 *   - plain C, every function returns a bsp_status_t as int;
 *   - every pointer is a CALLER-OWNED DEVICE pointer unless its comment says "host"; tensors are
 *     row-major and contiguous, base addresses 16-byte aligned;
 *   - the library allocates no device memory: scratch comes from the caller's workspace `ws` of
 *     `ws_bytes` bytes (256-byte aligned); the needed size is returned by the matching
 *     *_workspace_bytes() query; a too-small workspace returns BSP_ERR_WORKSPACE before launch;
 *   - calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = default stream)
 *     unless stated; outputs are valid after the caller synchronises that stream;
 *   - argument errors are detected on the host and returned before anything is launched;
 *   - device-detected conditions (non-finite inputs, saturated roundings, a bounded wait that
 *     ran out) are accumulated into the caller's device-resident bsp_diag_t, never trapped; the
 *     caller clears it (bsp_diag_clear) and reads it back after synchronising;
 *   - the same inputs give byte-identical outputs.  State the library keeps per process, none of
 *     which influences a result: the counters behind bsp_launch_count() and bsp_d2h_byte_count(), the record of which
 *     kernels already have their shared-memory limit raised on which device, and the fixed scratch
 *     array of bsp_norm_bwd_noalloc (a 20 MiB device array every GPU that loads the library holds).
 *     No stream, event or allocation outlives a call.
 *
 * FP8 codes are raw bit patterns (uint8): E4M3 = 1-4-3 bits, bias 7, no infinity, max 448; E5M2 =
 * 1-5-2, bias 15, max 57344.  Encoding maps every NaN input to the single code 0x7F (the sign of a
 * NaN is not kept); decoding reads 0x7F / 0xFF (E4M3) and 0x7D..0x7F / 0xFD..0xFF (E5M2) as NaN.
 * A code stands for decode(code) / scale.
 *
 * Shape limits (BSP_ERR_UNSUPPORTED beyond them): normalisation width C a multiple of 4 and at
 * most 8192; the per-use check of a normalisation -> linear workload needs C and O multiples of
 * 16; attention needs head dimension 64 and bf16 inputs (FP8-operand mode: uint8 codes).
 */
#ifndef BSP_H_
#define BSP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  BSP_OK = 0,
  BSP_ERR_ARG = 1,          /* NULL / negative / inconsistent argument                    */
  BSP_ERR_ALIGN = 2,        /* pointer or leading dimension not 16-byte aligned           */
  BSP_ERR_UNSUPPORTED = 3,  /* valid request this build does not implement                */
  BSP_ERR_WORKSPACE = 4,    /* workspace missing or too small                             */
  BSP_ERR_NONFINITE = 5,    /* (diag.status) NaN or infinity met in an input              */
  BSP_ERR_TIMEOUT = 6,      /* (diag.status) a bounded device-side wait ran out           */
  BSP_ERR_CUDA = 7,         /* a CUDA runtime or driver call failed                       */
  BSP_ERR_TOO_LARGE = 8     /* problem exceeds the fixed capacity of a no-allocation entry */
} bsp_status_t;

typedef enum { BSP_E4M3 = 0, BSP_E5M2 = 1 } bsp_format_t;
typedef enum { BSP_ROUND_NEAREST = 0, BSP_ROUND_STOCHASTIC = 1 } bsp_round_mode_t;
/* What a backward use reads (Section "One tensor, two uses"; Appendix table "Store policies"). */
typedef enum { BSP_READ_ORIGINAL = 0 /* U */, BSP_READ_FORWARD = 1 /* R */, BSP_READ_FRESH = 2 /* N */,
               /* the forward's rounding plus the error of a new one, u_q + (u_f - u): the weight-use
                  read of the table's last policy, U/R+eps (b-bit store only) */
               BSP_READ_FORWARD_PLUS_FRESH_ERROR = 3 } bsp_policy_t;
typedef enum { BSP_F32 = 0, BSP_BF16 = 1 } bsp_dtype_t;
typedef enum { BSP_RMSNORM = 0, BSP_LAYERNORM = 1 } bsp_norm_t;
typedef enum { BSP_HOLDS = 0, BSP_FAILS = 1, BSP_UNDECIDED = 2 } bsp_verdict_t;

/* Generator streams: the `stream` field of bsp_key_t.  "The new rounding uses a separate stream
 * of the same law" (Appendix "The forks"). */
enum { BSP_STREAM_FORWARD = 0, BSP_STREAM_GAIN = 1, BSP_STREAM_WGRAD = 2, BSP_STREAM_DX = 3,
       BSP_STREAM_ATTN_D = 4, BSP_STREAM_SHARED = 255 };

/* Key of the counter-based generator (Philox4x32-10).  Element with row-major logical index e of
 * tensor `tensor_id` uses word (e & 3) of
 *   philox(counter = (lo32(e>>2), hi32(e>>2), draw, (tensor_id << 8) | stream),
 *          key     = (lo32(seed), hi32(seed))).
 * One 32-bit word per element, independent of layout, tiling and launch shape. */
typedef struct {
  uint64_t seed;
  uint32_t tensor_id;   /* < 2^24 */
  uint32_t stream;      /* < 256  */
  uint32_t draw;
  uint32_t reserved;    /* must be 0 */
} bsp_key_t;

/* How a tensor is rounded: code = round(fl32(x * scale)).  If scale_dev is not NULL the kernels
 * read the scale from that device float (scale_dev[0]) and ignore `scale`; this lets a scale
 * computed on the device (bsp_scale_from_amax) be used without a host round trip. */
typedef struct {
  int32_t fmt;              /* bsp_format_t     */
  int32_t mode;             /* bsp_round_mode_t */
  float scale;
  const float* scale_dev;
} bsp_quant_t;

/* Device-resident diagnostics, accumulated with atomics by every kernel that is handed one. */
typedef struct {
  unsigned long long n_saturated;   /* finite magnitudes above the format's maximum          */
  unsigned long long n_nonfinite;   /* NaN or infinite inputs                                 */
  uint32_t amax_bits;               /* bit pattern of the largest finite |value| seen (float) */
  int32_t status;                   /* BSP_OK, BSP_ERR_NONFINITE or BSP_ERR_TIMEOUT           */
} bsp_diag_t;

/* Result of one (use, output tensor) evaluation of the check; lives in HOST memory.
 * Statistics: standard error over draws and z = (m - g*) / se (Appendix "Checkpointing");
 * R = ||m - g*||^2 / sum_j se_j^2 (Appendix "The normalization store"); Q' = mean z^2 (K-3)/(K-1);
 * rel = ||m - g*||_2 / ||g*||_2.  An element whose draws all coincide (se = 0) is judged as a
 * deterministic read: z = 0 if its error is within the deterministic tolerance of |g*|, else
 * +-infinity.  Verdict: see bsp_verdict_rule_t. */
typedef struct {
  int32_t use_id;            /* BSP_STREAM_* of the use                         */
  int32_t output_id;         /* bsp_output_t                                    */
  int32_t policy;            /* bsp_policy_t                                    */
  int32_t K;                 /* draws (1 for U and R)                           */
  int64_t n_elements;
  double rel_l2_mean_err;
  double R;
  double Qprime;
  double mean_z;
  double rms_z;
  double max_abs_z;
  double frac_abs_z_gt3;
  int32_t verdict;           /* bsp_verdict_t                                   */
  int32_t informational;     /* 1: statistics reported for information; the use's verdict is the row
                                of its own output (FP8-operand attention: dQ and dK pass through a
                                nearest rounding of dS, which is not linear in D)  */
} bsp_use_result_t;

/* The decision rule of the check.  The paper registers a reading rule per test before measuring
 * (Appendix "How the three tests were registered": nulls as "z < 2 and under x %", detections as
 * "z > 5"); this is that template on the pooled statistics.  Deterministic read: HOLDS iff
 * rel <= rel_tol_deterministic.  Fresh read: FAILS if Q' >= qprime_fail or R >= r_fail; HOLDS if
 * Q' <= qprime_hold and R <= r_hold and (rel_hold == 0 or rel <= rel_hold); UNDECIDED otherwise.
 * Passing NULL where a rule is expected selects {1e-4, 2, 3, 4, 6, 0}.  A rule with a hold
 * threshold above its fail threshold, or a negative entry, is BSP_ERR_ARG. */
typedef struct {
  double rel_tol_deterministic;
  double qprime_hold, r_hold;
  double qprime_fail, r_fail;
  double rel_hold;
} bsp_verdict_rule_t;

typedef enum { BSP_OUT_DGAMMA = 0, BSP_OUT_DBETA = 1, BSP_OUT_DW = 2, BSP_OUT_DX = 3,
               BSP_OUT_D = 4, BSP_OUT_DQ = 5, BSP_OUT_DK = 6, BSP_OUT_DV = 7 } bsp_output_t;

const char* bsp_status_string(int status);

/* Number of kernels this library has launched in this process so far (a monotone counter kept for
 * accounting; it influences no result). */
unsigned long long bsp_launch_count(void);

/* Bytes this library has itself copied from the device to the host in this process so far (the
 * block partials of the statistics passes: the only results a check brings back).  Accounting only. */
unsigned long long bsp_d2h_byte_count(void);

/* Clears a device bsp_diag_t (asynchronous memset). */
int bsp_diag_clear(bsp_diag_t* diag, void* stream);

/* ------------------------------------------------------------------------------------------
 * Rounding (Section "Same rounding distribution, opposite outcomes": stochastic rounding sends
 * a bracketed value to one of its two neighbours with a zero-mean error; Appendix "The forks":
 * entries at the top of the range round to nearest and are counted, generator keyed on seed and
 * stream).
 * ------------------------------------------------------------------------------------------ */

/* out[i] = the 32-bit generator word of element i, i in [0, n).  For the bit-exact stream test. */
int bsp_philox_fill(bsp_key_t key, size_t n, uint32_t* out, void* stream);

/* amax[g] = max |x| over group g (n_groups contiguous groups of group_size elements); NaN and
 * infinities are skipped and counted in diag (may be NULL).  Overwrites amax. */
int bsp_amax(const void* x, int dt, size_t n_groups, size_t group_size, float* amax,
             bsp_diag_t* diag, void* stream);

/* scale[g] = fl32(fmax / amax[g]); 1 when amax is 0, non-finite, or the quotient overflows. */
int bsp_scale_from_amax(const float* amax, size_t n, int fmt, float* scale, void* stream);

/* codes[i] = round(fl32(x[i] * scale)), nearest-even saturating, or stochastic with the word of
 * element `elem_offset + i` under `key`.  x: dt[n]; codes: uint8[n]. */
int bsp_round(const void* x, int dt, size_t n, bsp_quant_t q, bsp_key_t key, uint64_t elem_offset,
              uint8_t* codes, bsp_diag_t* diag, void* stream);

/* Same with one scale per contiguous group: scales[n_groups] (device).  Element index is the
 * position in the whole tensor. */
int bsp_round_grouped(const void* x, int dt, size_t n_groups, size_t group_size, int fmt, int mode,
                      const float* scales, bsp_key_t key, uint8_t* codes, bsp_diag_t* diag,
                      void* stream);

/* 2-D variant that can also write the transposed code matrix used by the weight-gradient
 * contraction: codes[r*cols + c] (may be NULL) and codes_t[c*ld_t + r] (may be NULL), ld_t >= rows
 * and a multiple of 16. */
int bsp_round_2d(const void* x, int dt, int64_t rows, int64_t cols, bsp_quant_t q, bsp_key_t key,
                 uint8_t* codes, uint8_t* codes_t, int64_t ld_t, bsp_diag_t* diag, void* stream);

/* ------------------------------------------------------------------------------------------
 * Normalisation store (Appendix "The normalization store"; Eq. norm-uses): z, u = gamma o z
 * (+ beta), u_q = round(u).  RMSNorm: rstd = 1/sqrt(mean x^2 + eps); LayerNorm: mean, biased
 * variance.  The value handed to the rounding is a fixed chain of FP32 operations without FMA:
 *   RMS  fl(fl(fl(x*rstd)*gamma)*scale);  LN  fl(fl(fl(fl(fl(x-mean)*rstd)*gamma)+beta)*scale).
 * ------------------------------------------------------------------------------------------ */

/* Row statistics and the largest |u| (for a current-amax scale).  rstd[T], mean[T] (LayerNorm
 * only; may be NULL for RMSNorm), amax: one device float, overwritten (may be NULL). */
int bsp_norm_stats(int kind, const void* x, int dt, int64_t T, int64_t C, const float* gamma,
                   const float* beta, float eps, float* rstd, float* mean, float* amax,
                   bsp_diag_t* diag, void* stream);

/* Rounds u from saved statistics.  Any of the outputs may be NULL:
 *   u_codes[T*C], u_codes_t[C*ld_t] (transposed), u_f32[T*C] (the FP32 u before scaling),
 *   u_bf16_t[C*ld_t] (u rounded to bf16, transposed: the U operand of the weight gradient).
 * With key.stream = BSP_STREAM_FORWARD this is the forward's store; with another stream and
 * mode stochastic it is the re-rounding pass that feeds a fresh read (policy N). */
int bsp_norm_fwd(int kind, const void* x, int dt, int64_t T, int64_t C, const float* gamma,
                 const float* beta, const float* rstd, const float* mean, bsp_quant_t q,
                 bsp_key_t key, uint8_t* u_codes, uint8_t* u_codes_t, int64_t ld_t, float* u_f32,
                 void* u_bf16_t, bsp_diag_t* diag, void* stream);

/* The re-rounding pass for n_draws consecutive draws [draw0, draw0 + n_draws) of a fresh read
 * (policy N; "a new rounding draws separate random numbers the same way", Section "Same rounding
 * distribution, opposite outcomes"): the FP32 value of each element is formed once and rounded
 * stochastically once per draw (key.draw is ignored).  Writes only the transposed code matrices,
 * draw d at u_codes_t_draws + d * C * ld_t, each [C * ld_t]. */
int bsp_norm_fwd_draws(int kind, const void* x, int dt, int64_t T, int64_t C, const float* gamma,
                       const float* beta, const float* rstd, const float* mean, bsp_quant_t q,
                       bsp_key_t key, int draw0, int n_draws, uint8_t* u_codes_t_draws, int64_t ld_t,
                       void* stream);

/* Backward of the normalisation with du passed through the rounding unchanged:
 *   dgamma[C] = sum_t z_g o du, z_g = z (U) | (decode(u_codes)/scale - beta)/gamma (R) |
 *               the same from a fresh rounding under `key` (N, one draw);
 *   dbeta[C] = sum_t du (may be NULL);  dx[T*C] (may be NULL):
 *   RMS dx = rstd (dz - z mean_j(dz o z)), LN dx = rstd (dz - mean_j dz - z mean_j(dz o z)),
 *   dz = gamma o du, with z read under `dx_read`.  The paper's input gradient "uses unrounded
 *   values" (Appendix "The normalization store"): that is dx_read = BSP_READ_ORIGINAL, the
 *   reference and what every configuration uses; R and N read z as the gain use does, N under
 *   generator stream BSP_STREAM_DX of the same key (dx is quadratic in z, so a fresh read leaves a
 *   small bias: no verdict is put on it).  du: du_dt[T*C].  Outputs FP32. */
size_t bsp_norm_bwd_workspace_bytes(int64_t T, int64_t C);
int bsp_norm_bwd(int kind, const void* x, int dt, int64_t T, int64_t C, const float* gamma,
                 const float* beta, const float* rstd, const float* mean, const void* du, int du_dt,
                 int gain_read, int dx_read, const uint8_t* u_codes, bsp_quant_t q, bsp_key_t key,
                 float* dgamma, float* dbeta, float* dx, void* ws, size_t ws_bytes,
                 bsp_diag_t* diag, void* stream);

/* bsp_norm_bwd for callers that cannot hand over a workspace.  (The paper has no counterpart: this
 * is a packaging variant of the entry point above, same arithmetic, same results.)
 *
 * Who needs it: code that runs where device allocation is off the table -- a plug-in inside a host
 * application that reserved the whole GPU for its own pool at start-up and gives extensions no
 * allocator; a latency-critical loop where cudaMalloc's implicit device-wide synchronisation and
 * unbounded duration are not acceptable; a process running under a hard device-memory quota fixed
 * at launch.  Such callers still own their inputs and outputs, but have nowhere to get scratch.
 *
 * What it does instead: the column partials that bsp_norm_bwd keeps in `ws` go to a fixed 20 MiB
 * array inside the library's device image (BSP_NORM_BWD_NOALLOC_CAPACITY_BYTES).  Every GPU on
 * which the library is loaded holds that array until the process exits, used or not.  The call
 * never calls cudaMalloc, cudaFree or any allocating routine.
 *
 * Limits and rules:
 *  - the problem must satisfy bsp_norm_bwd_workspace_bytes(T, C) <= the capacity (true for every
 *    T when C <= 4096, and for T <= 320 when C = 8192); otherwise BSP_ERR_TOO_LARGE is returned
 *    before anything is launched and no output is touched;
 *  - the first call on each device looks up the array's device address (one
 *    cudaGetSymbolAddress, with that device current) and caches it; make that first call during
 *    set-up, before any stream capture is begun;
 *  - the array is shared by all calls and keeps whatever the last call wrote.  This pass writes
 *    every partial it later reads, so nothing needs clearing between calls (a block whose bounded
 *    wait ran out writes NaN partials and raises BSP_ERR_TIMEOUT in `diag`, so a failed call
 *    cannot pass off the previous call's sums as its own) -- but two calls that overlap on the
 *    GPU (different streams, or threads issuing concurrently) race on it and corrupt each
 *    other's sums.  Serialise them, or use bsp_norm_bwd with separate workspaces.
 * Arguments, outputs and error behaviour are otherwise those of bsp_norm_bwd. */
#define BSP_NORM_BWD_NOALLOC_CAPACITY_BYTES ((size_t)20 << 20)
int bsp_norm_bwd_noalloc(int kind, const void* x, int dt, int64_t T, int64_t C, const float* gamma,
                         const float* beta, const float* rstd, const float* mean, const void* du,
                         int du_dt, int gain_read, int dx_read, const uint8_t* u_codes, bsp_quant_t q,
                         bsp_key_t key, float* dgamma, float* dbeta, float* dx, bsp_diag_t* diag,
                         void* stream);

/* K fresh draws of the gain use in one pass over x and du: for draw k in [draw0, draw0+K) the
 * gain gradient g_k is formed as in bsp_norm_bwd (policy N, key.draw = k) and the shifted sums
 * S1[c] += sum_k (g_k[c] - g_ref[c]), S2[c] += sum_k (g_k[c] - g_ref[c])^2 are accumulated, so
 * draw ranges can be split and merged by addition.  Never materialises the K gradients. */
size_t bsp_norm_gain_mc_workspace_bytes(int64_t T, int64_t C, int K);
int bsp_norm_gain_mc(int kind, const void* x, int dt, int64_t T, int64_t C, const float* gamma,
                     const float* beta, const float* rstd, const float* mean, const void* du,
                     int du_dt, bsp_quant_t q, bsp_key_t key, int draw0, int K, const float* g_ref,
                     float* S1, float* S2, void* ws, size_t ws_bytes, bsp_diag_t* diag, void* stream);

/* ------------------------------------------------------------------------------------------
 * Linear layer after the store (Eq. norm-uses: dW = u_q^T dy; reading the original adds
 * -r^T dy).  W is stored [O, C]; dW[O, C] = dY^T X with X the copy the weight use reads.
 * Operands are "token-minor" (transposed) matrices: dy_t[O*ld_t], x_t[C*ld_t], entry (row, t) at
 * row*ld_t + t, ld_t a multiple of 16 -- as written by bsp_round_2d / bsp_norm_fwd.
 *   x_read = U: x_t is bf16 (u rounded to bf16), dy is decoded to bf16 in `ws`; BF16 tensor cores.
 *   x_read = R or N: x_t is uint8 codes in q_x.fmt; FP8 tensor cores (E5M2 x E4M3).
 * FP32 accumulation; dW = acc / (scale_dy * scale_x).
 * If mc_ref is not NULL the epilogue does not store dW but accumulates the shifted sums
 *   S1 += dW - mc_ref, S2 += (dW - mc_ref)^2          (all [O*C] FP32).
 * ------------------------------------------------------------------------------------------ */
size_t bsp_linear_wgrad_workspace_bytes(int64_t T, int64_t O, int64_t C, int x_read);
int bsp_linear_wgrad(int64_t T, int64_t O, int64_t C, const uint8_t* dy_codes_t, bsp_quant_t q_dy,
                     int x_read, const void* x_t, bsp_quant_t q_x, int64_t ld_t, float* dW,
                     const float* mc_ref, float* mc_S1, float* mc_S2, void* ws, size_t ws_bytes,
                     bsp_diag_t* diag, void* stream);

/* The contraction primitive behind the weight gradient, the input gradient and the attention
 * products (helper, not an operator of the paper): C[M,N] (FP32, pitch ldc) = alpha * A * B^T on
 * the tensor cores with FP32 accumulation.  elem = 1: FP8 codes (a_fmt / b_fmt = bsp_format_t,
 * any combination), elem = 2: bf16.  An operand is either K-major -- stored [rows][K], pitch ld --
 * or, with its *_mn flag set, MN-major -- stored [K][rows], pitch ld -- so a product over the
 * leading dimension of two row-major matrices (dW = dY^T X) needs no transposed copy.  Pitches are
 * in elements; pitch * elem must be a multiple of 16 bytes; ldc a multiple of 4. */
int bsp_gemm(int64_t M, int64_t N, int64_t K, int elem, const void* A, int64_t lda, int a_mn, int a_fmt,
             const void* B, int64_t ldb, int b_mn, int b_fmt, float alpha, float* C, int64_t ldc,
             bsp_diag_t* diag, void* stream);

/* The weight use under n_draws fresh roundings in one launch (Section "Each use has a checkable
 * requirement": the substitute's own draw is averaged with the forward and the incoming gradient
 * held fixed).  x_t_draws holds n_draws code matrices [C * ld_t] back to back (as written by
 * bsp_norm_fwd_draws).  For every draw d: dW_d = dY^T X_d, and
 *   S1 += dW_d - g_ref,  S2 += (dW_d - g_ref)^2      (all [O*C] FP32; S1, S2 are read, updated,
 * written back, so draw ranges can be chained).  The per-draw gradients are never written: the
 * running sums of an output tile stay in tensor memory while the kernel walks the draws.
 * C must be a multiple of 16. */
int bsp_linear_wgrad_mc(int64_t T, int64_t O, int64_t C, const uint8_t* dy_codes_t, bsp_quant_t q_dy,
                        const uint8_t* x_t_draws, bsp_quant_t q_x, int64_t ld_t, int n_draws,
                        const float* g_ref, float* S1, float* S2, bsp_diag_t* diag, void* stream);

/* du[T*C] (du_dt) = dY W with dY = decode(dy_codes[T*O]) / scale and W w_dt[O*C]: the incoming
 * gradient passed through the rounding unchanged.  BF16 tensor cores (W rounded to bf16). */
size_t bsp_linear_dgrad_workspace_bytes(int64_t T, int64_t O, int64_t C);
int bsp_linear_dgrad(int64_t T, int64_t O, int64_t C, const uint8_t* dy_codes, bsp_quant_t q_dy,
                     const void* W, int w_dt, void* du, int du_dt, void* ws, size_t ws_bytes,
                     bsp_diag_t* diag, void* stream);

/* ------------------------------------------------------------------------------------------
 * Causal softmax attention (Section "Same rounding distribution, opposite outcomes"):
 * P = softmax(c Q K^T), O = P V; dV = P^T dO, dP = dO V^T, dS = P o (dP - D),
 * D = rowsum(P o dP) = rowsum(dO o O); dQ = c dS K, dK = c dS^T Q.  The forward rounds O before the
 * next layer consumes it; the correction term D is the one use of the saved output, and reading a
 * copy O + E adds rowsum(dO o E) (Eq. dterm).  Tensors are [B, H, S, Dh] row-major, bf16
 * (dt = BSP_BF16), Dh = 64, FP32 outputs; lse, D are [B, H, S].
 *
 * Two operand modes.  BF16 operands (fp8 = NULL): the three products that consume a computed
 * operand take P and dS rounded to bf16; against the plain definition that rounding alone is a
 * relative distance of about 1.7e-3 per output tensor on the benchmark's inputs.  FP8 operands
 * (fp8 != NULL), after the emulated FP8 attention backward of Appendix "The forks": Q, K, V are
 * rounded to nearest onto E4M3 and dO onto E5M2, each at the per-(b,h) amax scale of its slice; P is
 * recomputed (unrounded) from the dequantised Q and K; dV = P_q^T dO with P_q = RN_E4M3(P p_scale)
 * / p_scale; dP = dO V^T; D from the assigned output copy; dS = P o (dP - D); dS_q = RN_E5M2(dS
 * ds_scale) / ds_scale feeds dQ and dK (ds_scale supplied by the caller, like a delayed scale).
 * In that mode q, k, v, dO are bf16 tensors holding the DECODED codes as written by
 * bsp_attn_quantize (every FP8 value is a bf16 value): the forward helper reads those (its P V
 * product has an unrounded P).  The backward reads the codes themselves (bsp_attn_fp8_t: q_codes,
 * k_codes, v_codes E4M3, do_codes E5M2, uint8 [B, H, S, Dh], all four required) and issues its
 * seven products as FP8 tensor-core products, P and dS entering as E4M3 / E5M2 codes; the scales are
 * folded back in the kernel.  The final E5M2 cast of the returned gradients is not applied (outputs
 * FP32).  Quantisation points and the two scales are this library's reading of that appendix.
 * ------------------------------------------------------------------------------------------ */

typedef struct {
  const float* q_scale;      /* [B*H] device: scale of each slice of q (code = round(x * scale)) */
  const float* k_scale;
  const float* v_scale;
  const float* do_scale;
  float p_scale;             /* power of two; 256 keeps P * p_scale <= 256 < 448 */
  float ds_scale;
  const uint8_t* q_codes;    /* the codes themselves, [B, H, S, Dh]: read by the backward (NULL for the forward helper) */
  const uint8_t* k_codes;
  const uint8_t* v_codes;
  const uint8_t* do_codes;
} bsp_attn_fp8_t;

/* For each of n_groups contiguous groups of group_size bf16 elements, scale_g = fmax / amax_g:
 * xq (bf16, same shape, may be NULL) = decode(RN_fmt(x * scale_g)), codes (uint8, same shape, may be
 * NULL) = RN_fmt(x * scale_g); amax[n_groups] and scales[n_groups] are written too.  group_size a
 * multiple of 8; x, xq 16-byte and codes 8-byte aligned. */
int bsp_attn_quantize(const void* x, int n_groups, size_t group_size, int fmt, void* xq, uint8_t* codes,
                      float* amax, float* scales, bsp_diag_t* diag, void* stream);

/* Forward statistics from the operands exactly as the backward will see them: o = P V (FP32, the
 * "original" output the store rounds; P unrounded) and lse = log sum_j exp(c q.k_j). */
int bsp_attn_fwd_stats(int B, int H, int S, int Dh, int causal, float softmax_scale, const void* q,
                       const void* k, const void* v, int dt, const bsp_attn_fp8_t* fp8, float* o,
                       float* lse, bsp_diag_t* diag, void* stream);

/* The D use: d_out[d][b,h,i] = sum_j dO[b,h,i,j] * O_copy[b,h,i,j] for n_draws draws, with
 * O_copy = o_orig (U), decode(o_codes)/o_scales[b,h] (R), or a fresh stochastic rounding of
 * fl32(o_orig * o_scales[b,h]) in o_fmt under (key, draw0 + d) (N).  U and R write one draw.
 * dO: dt[B,H,S,Dh]; do_scales: NULL, or (FP8-operand mode) the per-(b,h) scales of a dO that holds
 * decoded codes; o_scales: one scale per (b,h) slice.  dO and o_orig 16-byte aligned, o_codes
 * 8-byte aligned (BSP_ERR_ALIGN otherwise). */
int bsp_attn_dterm(int B, int H, int S, int Dh, const void* dO, int dt, const float* do_scales,
                   const float* o_orig, const uint8_t* o_codes, const float* o_scales, int o_fmt,
                   int d_read, bsp_key_t key, int draw0, int n_draws, float* d_out, bsp_diag_t* diag,
                   void* stream);

/* Backward given D (dterm[B,H,S]).  dq may be NULL; dk and dv may both be NULL; dv may be NULL
 * alone (dK only: dV does not read D); dv without dk is BSP_ERR_ARG. */
int bsp_attn_bwd_dterm(int B, int H, int S, int Dh, int causal, float softmax_scale, const void* q,
                       const void* k, const void* v, const void* dO, int dt, const bsp_attn_fp8_t* fp8,
                       const float* lse, const float* dterm, float* dq, float* dk, float* dv,
                       bsp_diag_t* diag, void* stream);

/* The same backward (BF16 operands, all three gradients required) in one kernel: every score tile's
 * S, dP and exponentials are formed once and serve dV, dK and dQ; the tile's share of dQ is added to
 * dq in device memory, which this call clears first.  dk and dv are bit-reproducible; dq is up to the
 * order of its FP32 additions (S/128 shares per element).  Arguments as bsp_attn_bwd_dterm. */
int bsp_attn_bwd_dterm_fused(int B, int H, int S, int Dh, int causal, float softmax_scale, const void* q,
                             const void* k, const void* v, const void* dO, int dt, const float* lse,
                             const float* dterm, float* dq, float* dk, float* dv, bsp_diag_t* diag,
                             void* stream);

/* Backward under a read policy at the D use: bsp_attn_dterm (draw key.draw) into d_out[B,H,S]
 * (required), then bsp_attn_bwd_dterm.  fp8_operands = 0: fp8 must be NULL; fp8_operands = 1: fp8
 * gives the operand scales (BSP_ERR_ARG when the flag and the pointer disagree). */
int bsp_attn_bwd(int B, int H, int S, int Dh, int causal, float softmax_scale, int fp8_operands,
                 const void* q, const void* k, const void* v, const void* dO, int dt,
                 const bsp_attn_fp8_t* fp8, const float* lse, const float* o_orig, const uint8_t* o_codes,
                 const float* o_scales, int o_fmt, int d_read, bsp_key_t key, float* dq, float* dk,
                 float* dv, float* d_out, bsp_diag_t* diag, void* stream);

/* ------------------------------------------------------------------------------------------
 * Monte-Carlo reduction (Section "Each use has a checkable requirement").
 * ------------------------------------------------------------------------------------------ */

/* One draw's contribution to the shifted sums, elementwise: S1 += g - g_ref, S2 += (g - g_ref)^2
 * (n a multiple of 4).  Used where the producing kernel has no fused accumulation. */
int bsp_mc_accumulate(const float* g, const float* g_ref, float* S1, float* S2, size_t n, void* stream);

/* Per-element moments from the shifted sums of K draws (K >= 2): mean = g_ref + S1/K,
 * var = (S2 - S1^2/K) / (K - 1) (clamped at 0), z = (S1/K) / sqrt(var/K) (0 when numerator and
 * denominator both vanish, +-infinity when only the denominator does).  Any output may be NULL. */
int bsp_mc_moments(const float* g_ref, const float* S1, const float* S2, size_t n, int K, float* mean,
                   float* var, float* z, void* stream);

/* Reduces per-element shifted sums to the statistics of bsp_use_result_t and the verdict.
 * fresh = 0: deterministic read, `g` holds the gradient itself (S2 ignored, K = 1).
 * fresh = 1: g = S1, with S2, over K >= 4 draws.  ws: >= bsp_mc_stats_workspace_bytes(n).
 * Synchronises `stream`; `result` is HOST memory; use_id/output_id/policy are left untouched. */
size_t bsp_mc_stats_workspace_bytes(int64_t n);
int bsp_mc_stats(const float* g_ref, const float* g, const float* S2, int64_t n, int K, int fresh,
                 const bsp_verdict_rule_t* rule, bsp_use_result_t* result, void* ws, size_t ws_bytes,
                 void* stream);

/* The whole per-use check of a normalisation -> linear workload, device-resident inputs.
 * Once per call: statistics, current-amax scale, forward store (stream 0, `forward_mode`),
 * incoming gradient dY -> E5M2 nearest at its own amax, du = dY W.  Then per use and policy:
 *   gain use  (dgamma, reference read U):  U, R, N (K draws); each is followed by the result for
 *   dbeta, which reads no saved tensor and so equals its reference under every read;
 *   weight use (dW,    reference read R):  U, R, N (K draws: re-round + FP8 contraction + fused
 *   shifted-sum epilogue).
 * `policy_mask` bit (use*3 + policy) selects evaluations, use 0 = gain, 1 = weight.
 * K >= 4 (the factor (K-3)/(K-1) of Q' must be positive).
 * results: HOST array of at least 9 entries, filled in order gain U (dgamma, dbeta), R, N, then
 * weight U, R, N (selected ones only); *n_results returns the count.  Synchronises before
 * returning.  The per-element results stay in `ws` at the offsets bsp_mc_check_layout gives.
 * `side_stream` (a cudaStream_t, or NULL): when both uses ask for N, the K-draw gain kernel runs
 * beside the first K-draw contraction on that stream, forked from and joined back into `stream`
 * inside the call; with NULL the two run one after the other.  `draw_buffer_bytes` bounds the
 * buffer of fresh code matrices (0 = 1 GiB): K draws are taken in chunks of as many draws as fit.
 * Calls on one device may overlap in time only if they use different workspaces. */
typedef struct {
  int32_t norm_kind;         /* bsp_norm_t  */
  int32_t dtype;             /* bsp_dtype_t of x, W, dY (and of du) */
  int64_t T, C, O;
  const void* x;             /* [T, C] */
  const float* gamma;        /* [C]    */
  const float* beta;         /* [C] or NULL */
  const void* W;             /* [O, C] */
  const void* dY;            /* [T, O] */
  float eps;
  int32_t store_fmt;         /* bsp_format_t of the store (E4M3)      */
  int32_t grad_fmt;          /* bsp_format_t of dY (E5M2)             */
  int32_t forward_mode;      /* bsp_round_mode_t of the forward store */
  uint64_t seed;
  uint32_t tensor_id;
  uint32_t policy_mask;
  void* side_stream;
  size_t draw_buffer_bytes;
} bsp_norm_linear_desc_t;

/* Byte offsets into the workspace of bsp_mc_check, of the FP32 arrays it leaves there.  With
 * bsp_mc_moments they give the per-element mean, variance and z-score of every gradient
 * (dgamma and dbeta: [C]; dW: [O*C]; under N: sums over K draws; dbeta has no sums, it equals its
 * reference in every draw). */
typedef struct {
  size_t dgamma_ref, dbeta_ref;      /* [C]: the reference gradients (gain use reads U)          */
  size_t dgamma_forward;             /* [C]: dgamma under read R                                 */
  size_t dgamma_S1, dgamma_S2;       /* [C]: shifted sums of dgamma over the K draws of read N   */
  size_t dW_ref;                     /* [O*C]: the reference (weight use reads R)                */
  size_t dW_S1, dW_S2;               /* [O*C]: shifted sums of dW over the K draws of read N     */
  size_t dx;                         /* [T*C]: the input gradient from unrounded values          */
  size_t rstd, mean;                 /* [T]: saved statistics                                    */
  size_t u_codes;                    /* [T*C] uint8: the forward's store                         */
  size_t scale_u, scale_dy;          /* one float each                                           */
  size_t du;                         /* [T*C] in the workload's dtype                            */
} bsp_mc_layout_t;

size_t bsp_mc_check_workspace_bytes(const bsp_norm_linear_desc_t* op, int K);
int bsp_mc_check_layout(const bsp_norm_linear_desc_t* op, int K, bsp_mc_layout_t* layout);
int bsp_mc_check(const bsp_norm_linear_desc_t* op, int K, const bsp_verdict_rule_t* rule,
                 bsp_use_result_t* results, int* n_results, void* ws, size_t ws_bytes, bsp_diag_t* diag,
                 void* stream);

/* The per-use check of the attention D use (Section "Same rounding distribution, opposite
 * outcomes"; Eq. dterm), device-resident inputs.  Once per call: (FP8-operand mode: the operands
 * rounded per (b,h) slice), O = P V and LSE, the output store (per-(b,h) amax scale,
 * `forward_mode`, stream 0).  Reference: D reads the original output.  Then for each selected
 * policy (policy_mask bit p = bsp_policy_t p) the backward is evaluated with D read under that
 * policy -- U and R once, N for K >= 4 draws -- and four results are written per policy in the
 * order D, dQ, dK, dV.  `results` is a HOST array (up to 12 entries).  Synchronises.
 *
 * BF16-operand mode evaluates the fresh read through Eq. dterm itself: dS, dQ and dK are affine in
 * D, so draw k differs from the reference by  dQ_k - dQ* = -c diag(D_k - D*) (P K)  and
 * dK_k - dK* = -c P^T diag(D_k - D*) Q.  The kernels form these differences directly (the K draws
 * of dQ collapse to one pass for P K and the sums of D_k - D*; dK takes one contraction per draw,
 * four draws per pass of the probabilities), so the statistics are not blurred by the rounding of
 * a full dS to the operand type, and no per-draw gradient is written.  dV does not read D: its
 * difference is exactly zero in every draw.
 * FP8-operand mode (fp8_operands = 1; p_scale, ds_scale as in bsp_attn_fp8_t) runs the rounded
 * backward once per draw: there dQ and dK pass through the nearest rounding of dS, which is not
 * linear in D, so their rows are marked `informational` and the verdict of the use is the row of D. */
typedef struct {
  int32_t B, H, S, Dh;
  int32_t causal;
  float softmax_scale;
  int32_t dtype;             /* bsp_dtype_t of q, k, v, dO (BSP_BF16) */
  const void* q;             /* [B, H, S, Dh] */
  const void* k;
  const void* v;
  const void* dO;
  int32_t store_fmt;         /* bsp_format_t of the output store (E4M3) */
  int32_t forward_mode;      /* bsp_round_mode_t of the forward's store   */
  uint64_t seed;
  uint32_t tensor_id;
  uint32_t policy_mask;
  int32_t fp8_operands;      /* 0: BF16 operands; 1: the FP8-operand mode */
  float p_scale, ds_scale;   /* FP8-operand mode only */
} bsp_attn_desc_t;

size_t bsp_mc_check_attn_workspace_bytes(const bsp_attn_desc_t* op, int K);
int bsp_mc_check_attn(const bsp_attn_desc_t* op, int K, const bsp_verdict_rule_t* rule,
                      bsp_use_result_t* results, int* n_results, void* ws, size_t ws_bytes,
                      bsp_diag_t* diag, void* stream);

/* ------------------------------------------------------------------------------------------
 * The paper's own store (Appendix "The normalization store"; table "Store policies"): for each
 * token a b-bit uniform grid of step s = max_j |u_j| / (2^(b-1) - 1), u_q = s floor(u / s + xi)
 * with an independent uniform xi per entry, so that u_q averages to u without clipping; the new
 * rounding u_f uses a separate generator stream.  Reads: gain use z | u_q / gamma | u_f / gamma;
 * weight use u | u_q | u_f | u_q + (u_f - u).  Reference: gain use z, weight use u_q.
 * Arithmetic: u is the FP32 chain value of the normalisation; s = fl32(amax / M), M = 2^(b-1) - 1
 * (1 for an all-zero token); t = fl32(u / s); n = floor(t) + [W < P] with W the element's generator
 * word and P = min(floor(fl32(t - floor(t)) 2^32), 2^32 - 1) -- the same law as floor(t + xi).
 * Codes are int8 (b = 2 .. 7; the paper ran 6 and 5), a code stands for s * code.
 * ------------------------------------------------------------------------------------------ */

/* codes[T*C], steps[T] from the saved statistics (rstd, mean as for bsp_norm_fwd) under `key`
 * (stream BSP_STREAM_FORWARD: the forward's store). */
int bsp_store_fwd(int kind, const void* x, int dt, int64_t T, int64_t C, const float* gamma,
                  const float* beta, const float* rstd, const float* mean, int bits, bsp_key_t key,
                  int8_t* codes, float* steps, void* stream);

/* The copy of u a use reads: read = BSP_READ_ORIGINAL (u), BSP_READ_FORWARD (s * code),
 * BSP_READ_FRESH (a new rounding under `key`) or BSP_READ_FORWARD_PLUS_FRESH_ERROR.  Outputs, each
 * may be NULL: copy_f32[T*C], and copy_split_t[C][2*ld_t] bf16, the operand of bsp_store_wgrad:
 * the copy split into two bf16 terms hi + lo (16 significant bits), token-minor, hi in columns
 * [0, ld_t), lo in [ld_t, 2 ld_t); ld_t >= T, a multiple of 16, padding zeroed.
 * C a multiple of 16 (BSP_ERR_UNSUPPORTED otherwise); x, codes and the outputs 16-byte aligned. */
int bsp_store_read(int kind, const void* x, int dt, int64_t T, int64_t C, const float* gamma,
                   const float* beta, const float* rstd, const float* mean, const int8_t* codes,
                   const float* steps, int read, bsp_key_t key, float* copy_f32, void* copy_split_t,
                   int64_t ld_t, void* stream);

/* dW[O, C] = dY^T X for a copy X given as the split operand of bsp_store_read: BF16 tensor cores,
 * dW = [dY | dY] [X_hi | X_lo]^T with dY's codes decoded to bf16 (exact), FP32 accumulation.  The
 * per-token step is part of X, so no operand is rounded below 16 bits. */
size_t bsp_store_wgrad_workspace_bytes(int64_t T, int64_t O);
int bsp_store_wgrad(int64_t T, int64_t O, int64_t C, const uint8_t* dy_codes_t, bsp_quant_t q_dy,
                    const void* copy_split_t, int64_t ld_t, float* dW, void* ws, size_t ws_bytes,
                    bsp_diag_t* diag, void* stream);

/* The per-use check with the b-bit store in place of the FP8 store: as bsp_mc_check, with
 * policy_mask bits 0..2 = gain use U, R, N and bits 3..6 = weight use U, R, N, U/R+eps (K >= 4 draws
 * for each fresh read).  results: HOST array of at least 7 entries in that order (dgamma, dW). */
typedef struct {
  int32_t norm_kind;         /* bsp_norm_t  */
  int32_t dtype;             /* bsp_dtype_t of x, W, dY (and of du) */
  int64_t T, C, O;
  const void* x;             /* [T, C] */
  const float* gamma;        /* [C]    */
  const float* beta;         /* [C] or NULL */
  const void* W;             /* [O, C] */
  const void* dY;            /* [T, O] */
  float eps;
  int32_t bits;              /* width of the store: 2 .. 7 */
  int32_t grad_fmt;          /* bsp_format_t of dY (E5M2) */
  uint64_t seed;
  uint32_t tensor_id;
  uint32_t policy_mask;
} bsp_store_desc_t;

size_t bsp_mc_check_store_workspace_bytes(const bsp_store_desc_t* op, int K);
int bsp_mc_check_store(const bsp_store_desc_t* op, int K, const bsp_verdict_rule_t* rule,
                       bsp_use_result_t* results, int* n_results, void* ws, size_t ws_bytes,
                       bsp_diag_t* diag, void* stream);

/* ------------------------------------------------------------------------------------------
 * Log-softmax backward with a +-eps error in its saved output (Appendix "Log-softmax").  The
 * operator's backward returns h - exp(S) (1^T h) from the incoming gradient h and the saved output
 * S = l + r, r_j = +-eps independently with equal probability (+eps when the top bit of the
 * element's generator word is set; element = row * classes + class; draw = trial; the consumed
 * error on stream 0 of (seed, tensor_id), the independent copy r' on stream 1).  With p = exp(l), g
 * the returned gradient and g* the one from l itself with the same h, a trial's statistic is the
 * mean over rows and classes of (g_j - g*_j) / p_j.  Statistics, in order:
 *   0 likelihood (h = -e_target), S read under reuse (l + r)        -> mean cosh(eps) - 1
 *   1 likelihood, independent copy (l + r')                         -> mean cosh(eps) - 1
 *   2 constructed loss (h = r), reuse                               -> mean -eps sinh(eps)
 *   3 constructed loss, independent copy                            -> mean 0
 *   4 as 0 with the reconstruction exp(S) divided by cosh(eps)      -> mean 0
 *   5 as 2 with that division                                       -> mean -eps sinh(eps) / cosh(eps)
 *   6, 7 the paired contrasts 0 - 1 and 2 - 3 (reuse minus independent copy), trial by trial
 * stats: HOST array of 8 {mean over trials, standard error over trials, z = |mean| / se}.
 * per_trial: device [trials * 6] (the six statistics of every trial) or NULL.  logits FP32
 * [rows * classes], classes a multiple of 4 and at most 8192; trials >= 2.  Synchronises.
 * ------------------------------------------------------------------------------------------ */
typedef struct { double mean, se, z; } bsp_lsm_stat_t;
size_t bsp_lsm_check_workspace_bytes(int rows, int classes, int trials);
int bsp_lsm_check(const float* logits, const int32_t* target, int rows, int classes, float eps, int trials,
                  uint64_t seed, uint32_t tensor_id, float* per_trial, bsp_lsm_stat_t* stats, void* ws,
                  size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------------------------
 * Rounded attention probabilities as the saved tensor (Appendix "Theory": the theorem "No shared
 * substitute serves both uses of attention probabilities", the table of average errors, and "One
 * new rounding suffices at the softmax's backward").  A row has probabilities p[n] and values
 * V[n, d] (shared by all rows); the forward rounds p to p_q and outputs o = V^T p_q; with the loss
 * ||o||^2 / 2 the incoming gradient is h = o and dp = V h.  Reference: dV = p_q h^T, ds = J(p) dp,
 * J(x) = diag(x) - x x^T.  For draws draw0 .. draw0 + K - 1 (the forward's rounding on generator
 * stream 0, new roundings a and b on streams 1 and 2 of (seed, tensor_id); element = row * n +
 * entry) the kernel sums the errors of
 *   ds_sum[5][rows][n]:  (J_hat - J(p)) dp for J_hat = J(p_q) | J(a) | K(a) | J2(a, b) | J2(p_q, b),
 *     K(a) = diag(a 1^T a) - a a^T,  J2(a, b) = diag((a + b)/2) - (a b^T + b a^T)/2;
 *   ds_sq (same shape, may be NULL): the sums of their squares;
 *   dV_sum[2][rows][n][d]:  (p_hat - p_q) h^T for p_hat = p | a.
 * Averages over the draws estimate the table's entries: delta, -Sigma_r G p, 0, 0,
 * (g o sigma^2 - tau p - Sigma_r G p)/2, and rows -sigma_j^2 v_j^T for both reads.
 * law 0: stochastic rounding to a uniform grid of spacing `param` (t = fl32(p / param), up iff
 * W < floor(frac(t) 2^32)); law 1: r = +param when the top bit of W is set, else -param.
 * n <= 256, d <= 64, d <= n.  Outputs are overwritten.
 * ------------------------------------------------------------------------------------------ */
int bsp_probs_mc(const float* p, const float* V, int64_t rows, int n, int d, int law, float param,
                 uint64_t seed, uint32_t tensor_id, int draw0, int K, float* ds_sum, float* ds_sq,
                 float* dV_sum, void* stream);

/* ------------------------------------------------------------------------------------------
 * Averages over the forward's rounding (Appendix "What the checker reads and reports": the split
 * E[Delta h] = E[Delta] E[h] + E[(Delta - E Delta)(h - E h)]; Appendix "The same dependence in a
 * normalization backward": the paired statistic T and its control; Appendix "The normalization
 * store", continuation probes: the estimator X).  Setting: normalisation -> FP8 store u_q = u + r
 * (per-tensor amax scale, `forward_mode`) -> y = u_q W^T under the loss ||y||^2 / 2, so dy = y and
 * du = dy W depend on the rounding the forward consumed.  2 * pairs forwards are drawn (generator
 * stream 0 of (seed, tensor_id), draws 0, 1, ...; pair k = draws 2k and 2k + 1) and the call leaves
 * in `ws`, at the offsets bsp_coupling_layout gives, the FP32 averages
 *   gain_total[C]      the gain-use error under read R, sum_t (r / gamma) o du
 *   gain_mean_part[C]  sum_t (E r / gamma) o E du; the coupling is gain_total - gain_mean_part
 *   gain_fresh[C]      the same error under a fresh read (stream 1, the draw of its forward)
 *   X[C*O], X_sq[C*O]  the mean over pairs of X_k = -(r_a - r_b)^T (dy_a - dy_b) / 2 and of X_k^2;
 *                      X averages to the weight-use error -r^T dy
 * and returns in HOST arrays of `pairs` doubles T_k = <r_a - r_b, du_a - du_b> / 2 and the control
 * <du_a, r_b>.  Under stochastic rounding with per-entry variance sigma^2 and A = W^T W the averages
 * tend to: gain_total_c -> sum_t sigma^2[t, c] A[c, c] / gamma_c (all of it coupling), T -> sum_{t, c}
 * sigma^2 A[c, c], control -> 0, X -> -diag(sum_t sigma^2) W^T; with round-to-nearest the forwards
 * coincide and T and X are exactly zero.  W is rounded to bf16 for the tensor cores (exact for
 * bf16 workloads); r = u_q - u with u the FP32 chain value.  C, O multiples of 16.  Synchronises.
 * ------------------------------------------------------------------------------------------ */
typedef struct {
  int32_t norm_kind;         /* bsp_norm_t  */
  int32_t dtype;             /* bsp_dtype_t of x and W */
  int64_t T, C, O;
  const void* x;             /* [T, C] */
  const float* gamma;        /* [C]    */
  const float* beta;         /* [C] or NULL */
  const void* W;             /* [O, C] */
  float eps;
  int32_t store_fmt;         /* bsp_format_t of the store */
  int32_t forward_mode;      /* bsp_round_mode_t of the store */
  uint64_t seed;
  uint32_t tensor_id;
  uint32_t reserved;
} bsp_coupling_desc_t;
typedef struct { size_t gain_total, gain_mean_part, gain_fresh, X, X_sq; } bsp_coupling_layout_t;
size_t bsp_coupling_check_workspace_bytes(const bsp_coupling_desc_t* op, int pairs);
int bsp_coupling_layout(const bsp_coupling_desc_t* op, int pairs, bsp_coupling_layout_t* layout);
int bsp_coupling_check(const bsp_coupling_desc_t* op, int pairs, double* T, double* control, void* ws,
                       size_t ws_bytes, bsp_diag_t* diag, void* stream);

/* ------------------------------------------------------------------------------------------
 * Self-test of the bounded device-side wait (no counterpart in the paper).  Every wait a kernel of
 * this library performs on a barrier gives up after a time limit, raises BSP_ERR_TIMEOUT in `diag`
 * and lets the kernel return normally.  This entry launches one small block whose wait is on a
 * barrier that nothing ever completes, with the limit set to `limit_ns` nanoseconds (1 .. 10^8);
 * after synchronising, diag.status == BSP_ERR_TIMEOUT and the context is intact.
 * ------------------------------------------------------------------------------------------ */
int bsp_selftest_bounded_wait(uint64_t limit_ns, bsp_diag_t* diag, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* BSP_H_ */
