/*
 * ciar.h -- C ABI of the B200 (sm_100a) CIAR hot path.
 *
 * Per image token the library computes, on the GPU, what the paper's device and cloud sides
 * compute over the visual-vocabulary logits: the row softmax, the InterFuse probability
 * interval and its Omega * Sigma uncertainty score, the threshold test that decides whether
 * the token is sent to the cloud, and for the tokens that are, the speculative-decoding
 * accept / reject test with residual resampling and the accepted prefix length per draft
 * window; ciar_decode_step strings these together for a batch of concurrent requests.
 *
 * Conventions that hold for every entry point
 *   - All data pointers are DEVICE pointers owned by the caller (unless a comment says host);
 *     they must stay valid until the stream has passed the call.  The library allocates and
 *     frees nothing, never synchronises, and issues all work on the given stream (a
 *     cudaStream_t passed as void*; NULL is the legacy default stream).
 *   - Every function returns a ciar_status (0 = OK).  Bad arguments are rejected on the host
 *     before anything is launched.  Nothing throws across the ABI and no kernel traps: a row
 *     holding a NaN or +inf logit, no finite logit, or a token id outside [0, vocab) gets a bit
 *     in row_status and conservative results (flag = 1, accept = 0, scores NaN).
 *   - Logits are row-major, [rows, row_stride] elements of float32 or bfloat16; the base
 *     address must be 16-byte aligned and row_stride * element size a multiple of 16 bytes.
 *     Only codes valid_begin .. valid_begin + valid_count - 1 of a row belong to the
 *     vocabulary V of that row (n = |V| = valid_count); the others are never read.  A -inf
 *     logit inside the slice is legal (probability 0, interval width 0, still counted in n).
 *   - Token ids are global code indices in [0, vocab).  Uniforms are float32 in [0, 1).
 *   - Optional outputs may be NULL.
 */
#ifndef CIAR_H
#define CIAR_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CIAR_VERSION 100

typedef enum {
    CIAR_OK = 0,
    CIAR_ERR_INVALID_ARG = 1,
    CIAR_ERR_UNSUPPORTED = 2,
    CIAR_ERR_ALIGNMENT = 3,
    CIAR_ERR_WORKSPACE_TOO_SMALL = 4,
    CIAR_ERR_CUDA = 5,
    CIAR_ERR_TIMEOUT = 6
} ciar_status;

enum { CIAR_F32 = 0, CIAR_BF16 = 1 };
/* Radius of the logit interval [c - r, c + r] (Inter-Head equation): one value for all rows,
   one per row, or one per code. */
enum { CIAR_RADIUS_SCALAR = 0, CIAR_RADIUS_PER_ROW = 1, CIAR_RADIUS_PER_CODE = 2 };
/* Which scalar decides the cloud flag.  INTERVAL is the paper's rule (Algorithm 1: the token is
   kept on the device iff U <= tau); ENTROPY, MAXPROB and RANDOM are the baselines it is compared
   with (uncertainty-method ablation table); ALL flags every token (verify-everything baseline). */
enum { CIAR_POLICY_INTERVAL = 0, CIAR_POLICY_ENTROPY = 1, CIAR_POLICY_MAXPROB = 2, CIAR_POLICY_RANDOM = 3,
       CIAR_POLICY_ALL = 4 };
/* Which rows of a draft window the cloud tests.  ANCHORED is Algorithm 1: the buffer starts at
   the first flagged token and runs to the end of the window.  PER_TOKEN tests flagged rows only.
   ALL tests every row. */
enum { CIAR_VERIFY_ANCHORED = 0, CIAR_VERIFY_PER_TOKEN = 1, CIAR_VERIFY_ALL = 2 };
/* row_status bits.  TIMEOUT: the device gave up waiting for the row's data to arrive on chip (a
   bounded wait ran out; never expected in normal operation); the row's results are unusable. */
enum { CIAR_ROW_NAN = 1, CIAR_ROW_NO_FINITE = 2, CIAR_ROW_BAD_TOKEN = 4, CIAR_ROW_TIMEOUT = 8 };

#define CIAR_MAX_WINDOW 64

typedef struct {
    int64_t rows;        /* number of token rows */
    int64_t row_stride;  /* elements between consecutive rows, >= vocab */
    int32_t vocab;       /* codes per row */
    int32_t valid_begin; /* first code of the valid slice */
    int32_t valid_count; /* n = |V|, >= 1, valid_begin + valid_count <= vocab */
    int32_t dtype;       /* CIAR_F32 | CIAR_BF16 */
} ciar_logits_desc;

/*
 * Interval and threshold parameters.
 *   radius: SCALAR -> unused (r_scalar is the radius); PER_ROW -> device float32[rows];
 *           PER_CODE -> device tensor with the logits' dtype, stride and alignment.
 *   radius_is_raw != 0: the stored value is the pre-activation rho and r = Softplus(rho)
 *           (Inter-Head equation); otherwise the stored value is r >= 0 itself.
 *   r_max:  the radius is clamped to r_max (interval appendix, closing remark); must be in (0, 80].
 *   lo_cap, hi_cap: the 0.99 / 1.01 of the normalisation step (interval appendix).
 *   tau:    threshold of the chosen policy; u_flag: device float32[rows], RANDOM policy only.
 */
typedef struct {
    int32_t radius_mode;
    int32_t radius_is_raw;
    const void *radius;
    float r_scalar;
    float r_max;
    float lo_cap;
    float hi_cap;
    int32_t policy;
    float tau;
    const float *u_flag;
} ciar_interval_params;

/*
 * Per-row results of the quantifier, each float32[rows] unless noted.
 *   row_max m = max_i c_i; sum_exp Z' = sum_i exp(c_i - m); lse = m + ln Z'; p_max = 1 / Z';
 *   entropy: Shannon entropy of softmax(c) in nats;
 *   S_lo, S_up: sums of the raw InterFuse bounds before the rescale;
 *   omega, sigma, score: Omega = sum of widths, Sigma = population std of widths, U = Omega*Sigma
 *   (uncertainty-score equation), widths taken after the rescale;
 *   argmax int32: lowest code index attaining the maximum; flag uint8: 1 = send to the cloud;
 *   row_status uint8: CIAR_ROW_* bits.
 *   dense_p, dense_lo, dense_up: float32[rows, valid_count], the softmax and the rescaled
 *   bounds of every valid code -- test / inspection output, costs 3 extra row writes.
 */
typedef struct {
    float *row_max, *sum_exp, *lse, *p_max, *entropy;
    float *S_lo, *S_up, *omega, *sigma, *score;
    int32_t *argmax;
    uint8_t *flag;
    uint8_t *row_status;
    float *dense_p, *dense_lo, *dense_up;
} ciar_quantify_out;

/*
 * Device-side uncertainty quantification of every row (method section "Device-Side Uncertainty
 * Quantification"; InterFuse and its normalisation: appendix "Proof of Interval Validity";
 * score: the uncertainty-score equation; decision: Algorithm 1, the U <= tau test).
 * Each logit row is read from HBM once.  Needs no workspace.
 * Errors: INVALID_ARG (NULL desc/logits/params/out, rows < 0, bad slice, bad enum, r_max out of
 * range, missing radius / u_flag), UNSUPPORTED (dtype), ALIGNMENT, CUDA (launch failed).
 * rows == 0 is OK and launches nothing.
 */
ciar_status ciar_quantify(const ciar_logits_desc *desc, const void *draft_logits,
                          const ciar_interval_params *params, const ciar_quantify_out *out, void *stream);

typedef struct {
    int32_t window; /* W >= 1, <= CIAR_MAX_WINDOW; rows must be a multiple of it */
    int32_t mode;   /* CIAR_VERIFY_* */
} ciar_verify_params;

/*
 * Results of the cloud-side test.
 *   per row [rows]: accept uint8 (1 = kept; rows that are not tested report 1),
 *     p_draft_tok / p_target_tok float32: probability of the drafted token under softmax(draft
 *     row) / softmax(target row) (0 for rows that are not tested), row_status uint8.
 *   per window [rows / W]: first_flag int32 f (first flagged row, W if none; 0 in mode ALL),
 *     accepted_len int32 a (rows 0..a-1 of the window are kept), resampled_token int32 (token
 *     drawn from the residual distribution on row a, -1 when a == W), cloud_call uint8 (f < W).
 */
typedef struct {
    uint8_t *accept;
    float *p_draft_tok, *p_target_tok;
    uint8_t *row_status;
    int32_t *first_flag, *accepted_len, *resampled_token;
    uint8_t *cloud_call;
} ciar_verify_out;

/* Bytes of scratch ciar_verify / ciar_decode_step need for `rows` rows in windows of `window`. */
size_t ciar_workspace_bytes(int64_t rows, int32_t window);

/*
 * Cloud-side verification of draft windows (Algorithm 1, else-branch: buffer, cloud
 * verification, resampling; the rule itself is the speculative-decoding test the method
 * section refers to: keep token x iff u < min(1, q_x / p_x), written as u * p_x < q_x, else draw
 * from norm(max(0, q - p)) by inverse CDF with u_resample of that row: smallest k whose
 * cumulative residual exceeds u * total).  p = softmax(draft row), q = softmax(target row).
 *   flag: uint8[rows] from ciar_quantify; may be NULL only in mode ALL.
 *   draft_row_max, draft_sum_exp: float32[rows] from ciar_quantify (m and Z' of the draft row);
 *     both NULL -> recomputed here at the price of one more read of each tested draft row.
 *   u_accept, u_resample: float32[rows].
 *   ws: scratch of at least ciar_workspace_bytes(rows, window) bytes, 16-byte aligned; contents
 *     need not be preserved between calls; two calls that overlap on the GPU must not share it.
 * Target rows are read only for tested rows; draft and target are read once more for rejected rows.
 * Errors: as ciar_quantify, plus INVALID_ARG for rows % window != 0 and WORKSPACE_TOO_SMALL.
 */
ciar_status ciar_verify(const ciar_logits_desc *desc, const void *draft_logits, const void *target_logits,
                        const int32_t *draft_tokens, const uint8_t *flag,
                        const float *draft_row_max, const float *draft_sum_exp,
                        const float *u_accept, const float *u_resample,
                        const ciar_verify_params *params, const ciar_verify_out *out,
                        void *ws, size_t ws_bytes, void *stream);

/*
 * ciar_verify without a workspace argument -- the paper has no counterpart; this entry point exists
 * for integration reasons only.
 *
 * Some hosts of this library cannot give ciar_verify a workspace: a plug-in that runs inside another
 * engine's pre-sized memory arena, a latency-critical serving loop, or code running between the
 * begin and end of a stream capture must not call cudaMalloc (it may fail against the arena's
 * budget, it synchronises the device, and it is illegal during capture), and some of them have no
 * allocator of their own to carve a buffer from.  Here the scratch is a fixed array of
 * CIAR_STATIC_SCRATCH_BYTES inside the library image: every GPU that loads the library holds that
 * much memory until the process ends, whether or not this function is ever called.
 *
 * Same arguments, results and errors as ciar_verify, minus ws / ws_bytes, plus:
 *   - WORKSPACE_TOO_SMALL when ciar_workspace_bytes(desc->rows, params->window) exceeds
 *     CIAR_STATIC_SCRATCH_BYTES (2 MiB: enough for 72 000 rows at window 8); nothing is launched then.
 *   - The first call on each device looks up the array's device address (once, with that device
 *     current).  Make that first call outside any stream capture.
 *   - No cudaMalloc, cudaFree or other allocating call is made, on any call.
 *   - All calls on a device share the one array, which keeps whatever the previous call left in
 *     it; the part that must start at zero is cleared on the given stream at the start of every
 *     call.  Two calls that may overlap on the GPU (different streams without an ordering between
 *     them) race on it: order them, or use ciar_verify with separate workspaces.
 */
#define CIAR_STATIC_SCRATCH_BYTES (2 * 1024 * 1024)
ciar_status ciar_verify_static(const ciar_logits_desc *desc, const void *draft_logits, const void *target_logits,
                               const int32_t *draft_tokens, const uint8_t *flag,
                               const float *draft_row_max, const float *draft_sum_exp,
                               const float *u_accept, const float *u_resample,
                               const ciar_verify_params *params, const ciar_verify_out *out, void *stream);

/*
 * State of a batch of concurrent requests, all arrays device memory owned by the caller.
 *   pos int32[requests]: next position to generate; tokens_out int32[requests, seq_len];
 *   counters int64[8], accumulated over steps: 0 windows processed, 1 windows with a cloud call,
 *   2 rows sent to the cloud, 3 rows flagged, 4 drafted tokens kept, 5 tokens resampled,
 *   6 rows quantified, 7 requests that finished.
 */
typedef struct {
    int32_t requests;
    int32_t seq_len;
    int32_t *pos;
    int32_t *tokens_out;
    int64_t *counters;
} ciar_decode_state;

/* Set pos[q] = pos0 for every request, tokens_out to -1 and the counters to 0 (Algorithm 1,
   initialisation; pos0 > 0 stands for a prefix the cloud has already generated). */
ciar_status ciar_decode_init(const ciar_decode_state *state, int32_t pos0, void *stream);

/*
 * One trip of Algorithm 1's device loop for every unfinished request, in draft windows of
 * `window` tokens: quantify rows pos .. pos + wlen - 1 (wlen = min(window, seq_len - pos): the
 * buffer stops at the end of the sequence), verify the window, write the kept draft tokens and
 * the resampled token into tokens_out, and advance pos by a + (a < wlen) (position update of
 * Algorithm 1's last line).  Everything runs on the device; the host reads nothing.
 *   desc->rows must equal requests * seq_len: the pools hold, for request q and position s, row
 *   q * seq_len + s of the draft / target logits, the drafted token and the two uniforms
 *   (params->radius PER_ROW / PER_CODE and u_flag are pools with the same indexing).
 *   ws: at least ciar_workspace_bytes(requests * window, window) bytes.
 */
ciar_status ciar_decode_step(const ciar_decode_state *state, const ciar_logits_desc *desc,
                             const void *draft_pool, const void *target_pool, const int32_t *draft_token_pool,
                             const float *u_accept_pool, const float *u_resample_pool,
                             const ciar_interval_params *params, const ciar_verify_params *vparams,
                             void *ws, size_t ws_bytes, void *stream);

/*
 * Test hook for the bounded device-side waits (the paper has no counterpart; not for production use).
 * The streaming kernels wait for a row's bytes to land on chip with a bound of about a second of SM
 * clocks; a wait that runs out ends the CTA's walk, and the rows it had not finished get
 * CIAR_ROW_TIMEOUT in row_status (flag 1, scores NaN) while the call itself still returns CIAR_OK --
 * no entry point returns CIAR_ERR_TIMEOUT; that code is reserved.  This hook makes such a wait run out
 * without any fault: in every later ciar_quantify launch of the streaming quantifier, CTA `cta` never
 * asks for the `row_in_walk`-th row of its walk (nothing is left in flight), and every wait is bounded
 * by `wait_cycles` SM clocks.  cta < 0 switches the hook off; wait_cycles <= 0 restores the default bound.
 * Host-side state, process-wide; returns CIAR_OK.
 */
ciar_status ciar_test_stall(int32_t cta, int32_t row_in_walk, int64_t wait_cycles);

/*
 * Discrete top-k quantifier: the "Discrete" side of the paper's discrete-vs-continuous comparison
 * (ablation section and its table, k = 100 .. 400).  The paper prints no formula; the reading
 * built here: the solution set of a row is its k most probable codes (largest logits, equal logits
 * by lowest index) and the row's discrete uncertainty is the interval score of ciar_quantify
 * applied to those k codes alone (softmax renormalised over the set, n = k).  The set is found by
 * a radix select over the logits' bit patterns with a shared-memory histogram, not by a sort.
 * Outputs, each [rows], all device pointers, all nullable:
 *   kth_logit float32: k-th largest logit; n_above int32: codes strictly above it (the set is
 *   these plus the k - n_above lowest-index codes equal to kth_logit);
 *   mass float32: probability of the set under the full-row softmax; entropy float32: Shannon
 *   entropy (nats) of the renormalised distribution; S_lo, S_up, omega, sigma, score: as in
 *   ciar_quantify_out but over the set; flag uint8 = score > tau; row_status uint8;
 *   indices int32[rows, k]: the set's global code ids in ascending order (-1 for an unusable row).
 * params: radius SCALAR or PER_ROW (PER_CODE: UNSUPPORTED); policy is ignored.
 * Errors as ciar_quantify, plus INVALID_ARG for k < 1 or k > valid_count.  Needs no workspace.
 */
typedef struct {
    float *kth_logit;
    int32_t *n_above;
    float *mass, *entropy, *S_lo, *S_up, *omega, *sigma, *score;
    uint8_t *flag;
    uint8_t *row_status;
    int32_t *indices;
} ciar_topk_out;

ciar_status ciar_quantify_topk(const ciar_logits_desc *desc, const void *draft_logits, int32_t k,
                               const ciar_interval_params *params, const ciar_topk_out *out, void *stream);

/*
 * Score variants (uncertainty appendix, "Practical Remarks for Thresholding and Normalization"),
 * formed from the omega and sigma arrays ciar_quantify wrote (device float32[rows]):
 *   PRODUCT Omega*Sigma; PER_N Omega*Sigma/n; PER_OMEGA2 Sigma/Omega; SMOOTHED
 *   Omega*sqrt(Sigma^2 + eps); ADDITIVE lambda1*Omega + lambda2*Omega*Sigma.
 * score_out float32[rows] and flag_out uint8[rows] (= value > tau; 1 for a NaN input) are nullable.
 * Errors: INVALID_ARG (NULL omega / sigma with rows > 0, n < 1, bad variant, NaN tau).
 */
enum { CIAR_SCORE_PRODUCT = 0, CIAR_SCORE_PER_N = 1, CIAR_SCORE_PER_OMEGA2 = 2, CIAR_SCORE_SMOOTHED = 3, CIAR_SCORE_ADDITIVE = 4 };
typedef struct {
    int32_t variant;
    float eps, lambda1, lambda2, tau;
} ciar_score_params;

ciar_status ciar_rescore(int64_t rows, int32_t n, const float *omega, const float *sigma,
                         const ciar_score_params *params, float *score_out, uint8_t *flag_out, void *stream);

/*
 * Several Inter-Heads (appendix "Impact of Inter-Head Capacity").
 * ciar_quantify_ensemble -- soft voting: the heads' softmax distributions are averaged code by
 * code and the interval (InterFuse, normalisation, Omega, Sigma, U) is formed around the averaged
 * distribution with the mean of the heads' clamped radii.  head_logits: device tensor
 * [n_heads, rows, row_stride] (head h starts head_stride elements after head h - 1; each head
 * follows desc).  params: radius SCALAR, or PER_ROW with radius = device float32[n_heads, rows];
 * PER_CODE: UNSUPPORTED; policy is ignored (flag = U > tau).  1 <= n_heads <= CIAR_MAX_HEADS.
 * Outputs taken from ciar_quantify_out: p_max (largest averaged probability), entropy (of the
 * averaged distribution), S_lo, S_up, omega, sigma, score, flag, row_status, and dense_p (the
 * averaged distribution, float32[rows, valid_count]); the other members must be NULL.
 * ciar_vote -- hard voting: flags uint8[n_heads, rows] (one ciar_quantify per head wrote them);
 * flag_out[row] = 1 when more than half of the heads flagged the row; votes_out int32[rows] nullable.
 */
#define CIAR_MAX_HEADS 8
ciar_status ciar_quantify_ensemble(const ciar_logits_desc *desc, const void *head_logits, int32_t n_heads,
                                   int64_t head_stride, const ciar_interval_params *params,
                                   const ciar_quantify_out *out, void *stream);
ciar_status ciar_vote(int32_t n_heads, int64_t rows, const uint8_t *flags, uint8_t *flag_out,
                      int32_t *votes_out, void *stream);

/*
 * Forward value of the Inter-DRO loss over a batch of rows (method section, "Inter-DRO Loss": the
 * anchor-loss, DRO re-weighting, alignment and complete-loss equations).  center, radius, cloud:
 * device tensors that follow desc (radius = one value per code, raw rho when radius_is_raw).
 * Per row: p_x = softmax(c), softmax(c + r), softmax(c - r) for x = mid, up, lo; p_cloud =
 * softmax(cloud); L1_x = sum |p_x - p_cloud|; CE_x = -sum p_cloud ln p_x; KL = KL(p_cloud || p_mid).
 * Over the batch: anchor(x) = lambda_v mean L1_x + lambda_p mean CE_x; align = lambda_beta mean KL;
 * w = softmax(alpha CE_lo) over the rows, dro = sum w CE_lo; total = anchor(mid) + align +
 * anchor(up) + anchor(lo) + dro.
 * Outputs (device, nullable): l1, ce float32[3, rows] (mid, up, lo); kl, weights float32[rows];
 * loss float32[6] = total, centre, upper, lower, dro, align.
 * workspace: device scratch of ciar_interdro_workspace_bytes(rows) bytes, 16-byte aligned.
 * Errors: as ciar_quantify, plus WORKSPACE_TOO_SMALL; rows must be >= 1.
 */
typedef struct {
    int32_t radius_is_raw;
    float r_max;
    float lambda_v, lambda_p, lambda_beta, alpha;
} ciar_interdro_params;
typedef struct {
    float *l1, *ce, *kl, *weights, *loss;
} ciar_interdro_out;
size_t ciar_interdro_workspace_bytes(int64_t rows);
ciar_status ciar_interdro_forward(const ciar_logits_desc *desc, const void *center, const void *radius,
                                  const void *cloud, const ciar_interdro_params *params,
                                  const ciar_interdro_out *out, void *workspace, size_t workspace_bytes,
                                  void *stream);

/* Human-readable name of a status code (host pointer to a static string). */
const char *ciar_status_string(ciar_status s);

/* CIAR_VERSION of the built library. */
int ciar_version(void);

/* Number of kernels the library has launched in this process so far (host counter; used by the
   benchmark to report its launch count). */
int64_t ciar_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* CIAR_H */
