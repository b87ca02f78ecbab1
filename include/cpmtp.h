/*
 * cpmtp — fused log-likelihood of a rank-r canonical-polyadic (CP) multi-token
 * prediction head, for NVIDIA B200 (sm_100a).
 *
 * The joint distribution of the next n tokens is modelled as a mixture of r
 * experts, each a product of n per-token softmax factors (Eq. 2, Eq. 3), with
 * mixture weights from a gate (Eq. 7) and factors from per-(token, expert)
 * head projections followed by a shared unembedding (Eq. 6 in its reduced,
 * shared-head form from the fine-tuning section):
 *
 *   w[i, :]        = softmax(W_g h[i])                                   (Eq. 7)
 *   S[i, s, a, :]  = E (W_head[s*r + a] h[i])                            (Eq. 6, shared head)
 *   C[i, s, a]     = S[i, s, a, x[i, s]] - logsumexp_v S[i, s, a, v]     (Eq. 8)
 *   logp[i]        = logsumexp_a( log w[i, a] + sum_s C[i, s, a] )       (Eq. 9)
 *
 * Conventions for every entry point
 *  - All tensor pointers are DEVICE pointers owned by the caller unless a
 *    parameter is documented as a host pointer.  Row-major, densely packed.
 *    bf16 tensors are passed as `const void*` / `void*` (2 bytes per element)
 *    and must be 16-byte aligned; fp32 / int32 tensors 4-byte aligned.
 *  - The library allocates and frees no device memory; scratch space is the
 *    caller's `workspace`, sized by cpmtp_workspace_bytes(), 256-byte aligned.
 *    Work is enqueued on `stream` and is asynchronous with respect to the host.
 *  - Return value: CPMTP_OK or a negative error code; on a validation error
 *    nothing was enqueued.  `dev_status` (device int32, may be NULL; the caller
 *    zeroes it) is raised by kernels to 1 if a target token was outside [0, V)
 *    (the token is clamped, the run continues), 2 if an internal bounded wait
 *    expired (results invalid), or 3 in the checked build when an index check failed
 *    (see cpmtp_debug_status).
 *  - Limits: d % 64 == 0, 1 <= r <= 32, 1 <= n <= 8, N >= 1, V >= 2,
 *    N*n*r*d < 2^40.
 *  - CUDA graphs: the entry points only enqueue kernels and copies, so they may be recorded by stream
 *    capture and replayed (same pointers, new contents); call each once outside capture first, since the
 *    first launch of a kernel sets its shared-memory attribute.  Environment knobs are read at capture time.
 *  - Threads: calls may be made from several host threads as long as each uses
 *    its own stream, workspace and outputs (the library's few host-side caches --
 *    device properties, kernel attributes, tensor maps -- are guarded by a lock); the
 *    per-stage profiling calls and cpmtp_reload_knobs are the exception (one thread,
 *    no other call in flight).
 *  - Environment knobs, for testing and tuning only.  They are read ONCE, at the first call
 *    into the library; cpmtp_reload_knobs() reads them again.
 *    CPMTP_BWD_CHUNK_ROWS / CPMTP_BWD_CHUNK_HEADS (rows / heads of logit gradients
 *    recomputed at a time in the backward passes; also changes the workspace the
 *    backward needs, so set it before querying cpmtp_workspace_bytes),
 *    CPMTP_LSE_GROUP_MB, CPMTP_LSE_SPLITS and CPMTP_LSE_GROUP_TILES (schedule of the
 *    fused unembedding),
 *    CPMTP_GEMM_GROUP_ROWS (rows swept together by the other GEMMs), CPMTP_WIDE_MIN_K
 *    and CPMTP_WIDE_MIN_ROWS (shortest contraction / fewest rows that get 256-row tiles), CPMTP_KL_GROUP_TILES and CPMTP_KL_SPLITS
 *    (schedule of the KL sweep of cpmtp_distill_forward; the latter also sizes its workspace),
 *    CPMTP_PROJ_TILE_ROWS (128 or 256: run the head projection on the plain 128- or 256-row tiles with four
 *    epilogue warps per row block instead of its own configuration),
 *    CPMTP_WAIT_LIMIT_US (how long a wait inside a kernel may last before the kernel gives up with
 *    device status 2; default 4 s) and CPMTP_TEST_SKIP_LOAD (test hook: every CTA of the tensor-core
 *    kernels leaves out that one operand load, so the give-up path runs; results are invalid).
 *  - Accuracy: log-probabilities are within 2e-3 of the exact definition and gradients within 1e-2
 *    relative L2 at the weight scales of trained heads (logit standard deviation of a few units) when
 *    V is in the thousands or more.  The projected hidden state z is held in bf16 between the two
 *    products; a vocabulary-wide logsumexp averages that rounding out, but with d >= 4096 and only a few
 *    hundred vocabulary entries it does not: there logsumexp_v can be off by up to 2e-3 and the KL terms
 *    of cpmtp_distill_forward by up to 2e-2.  The target logits are taken from the unrounded z and the
 *    full-head entry points have no bf16 intermediate.
 */
#ifndef CPMTP_H
#define CPMTP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CPMTP_MAX_R 32
#define CPMTP_MAX_N 8

enum {
  CPMTP_OK = 0,
  CPMTP_ERR_NULL = -1,      /* a required pointer is NULL */
  CPMTP_ERR_SHAPE = -2,     /* sizes outside the limits above */
  CPMTP_ERR_ALIGN = -3,     /* a pointer is not aligned as required */
  CPMTP_ERR_WORKSPACE = -4, /* workspace_bytes too small */
  CPMTP_ERR_ARCH = -5,      /* current device is not compute capability 10.x */
  CPMTP_ERR_LAUNCH = -6,    /* a CUDA call failed; see cudaGetLastError */
  CPMTP_ERR_LIMIT = -7      /* size beyond a fixed built-in capacity */
};

enum {
  CPMTP_OP_FORWARD = 0,
  CPMTP_OP_BACKWARD = 1,
  CPMTP_OP_SCORE = 2,
  CPMTP_OP_SAMPLE = 3,
  CPMTP_OP_FORWARD_FULL = 4,
  CPMTP_OP_BACKWARD_FULL = 5,
  CPMTP_OP_DISTILL_FORWARD = 6,
  CPMTP_OP_DISTILL_BACKWARD = 7
};

/* flags */
#define CPMTP_FLAG_AUX 1u /* add aux_coef * sum_a wbar_a^2 to the loss (soft form of Eq. 10) */
/* Backward only: `dloss_dlogp` is [N, n] and weighs the PREFIX log-probabilities, the objective being
 * sum_i sum_s dloss_dlogp[i, s] * log P(x[i, 0..s]).  The discounted per-token cross-entropy of the
 * fine-tuning loss (Eq. 14 and the sum after it, CE_k = log P(x[0..k-1]) - log P(x[0..k])) is of this form. */
#define CPMTP_FLAG_PER_TOKEN 2u
/* Do not keep the projected hidden states between the passes: cpmtp_forward leaves saved->z
 * untouched (it may be NULL) and cpmtp_backward recomputes z in its workspace (which grows by
 * N*n*r*d*2 bytes while the saved state shrinks by as much; +2*N*n*r*d*d flop).  Set the flag in
 * both calls and in the workspace query. */
#define CPMTP_FLAG_RECOMPUTE_Z 4u
/* Backward entry points: add the gradients to what dh / dW_head (dW_full) / dE / dW_g already hold instead
 * of overwriting them (gradient accumulation over micro-batches, the usual way the training objective of
 * Eq. 9 is run at more positions than one call holds).  The sum is formed in fp32 from the stored bf16
 * value and this call's fp32 accumulator and rounded to bf16 once per call; the caller zeroes the buffers
 * before the first micro-batch. */
#define CPMTP_FLAG_ACCUM_GRADS 8u

typedef struct cpmtp_shape {
  int32_t N;        /* positions */
  int32_t d;        /* embedding size (the paper's E) */
  int32_t V;        /* vocabulary size */
  int32_t n;        /* tokens predicted per position */
  int32_t r;        /* CP rank = number of experts */
  uint32_t flags;   /* CPMTP_FLAG_* */
  float aux_coef;   /* weight of the balance term, used when CPMTP_FLAG_AUX is set */
} cpmtp_shape;

/* Forward results kept for the backward pass; every pointer is a caller-owned
 * device buffer of the stated size. */
typedef struct cpmtp_saved {
  float* lse;   /* [N, n*r]  logsumexp_v S                       */
  float* tgt;   /* [N, n*r]  S at the target token               */
  float* logw;  /* [N, r]    log gate weights (Eq. 7)            */
  float* q;     /* [N, r]    expert posterior exp(a - logp)      */
  float* wbar;  /* [r]       mean gate weight over positions     */
  void* z;      /* [N, n*r, d] bf16 projected hidden states      */
} cpmtp_saved;

typedef struct CUstream_st* cpmtp_stream;

/* Checked build only (libcpmtp_debug.so, compiled with -DCPMTP_DEBUG; there is no counterpart in the paper).
 * In that build every store and gather of the tensor-core kernels' epilogues, and the candidate gather of
 * draft generation, first compares the elements it is about to touch with the extent of the buffer; an access
 * that does not fit is skipped and raises status 3, in `dev_status` and in a per-device word that stays
 * raised until the library is unloaded.  This call synchronizes the current device and returns that word:
 * 0 = every index check since the library was loaded has passed, 3 = one failed.  The release library
 * compiles the checks out and returns -1 here. */
int cpmtp_debug_status(void);

int cpmtp_version(void);   /* major * 100 + minor * 10; 110 added the distillation entry points, 120 CPMTP_FLAG_ACCUM_GRADS */
const char* cpmtp_status_string(int status);

/* Read the environment knobs listed above again (they are otherwise read once per process).  For tests
 * and tuning runs that change a knob between calls; not to be called while another call is in flight.
 * The paper has no counterpart for this call. */
int cpmtp_reload_knobs(void);

/* Scratch bytes needed by `op` (CPMTP_OP_*) for this shape; 0 if the shape is invalid. */
size_t cpmtp_workspace_bytes(const cpmtp_shape* shape, int op);

/*
 * Joint log-likelihood per position, logp[i] of Eq. 9, with the vocabulary
 * reduction of Eq. 8 fused into the unembedding so that the logits are never
 * written to memory.
 *   h [N,d] bf16, W_head [n*r,d,d] bf16 (k = s*r + a, [out][in]), E [V,d] bf16,
 *   W_g [r,d] bf16, x [N,n] int32 targets.
 *   logp [N] fp32 out.
 *   loss [1] fp32 out or NULL: -(1/N) sum_i logp[i] (+ aux_coef * sum_a wbar_a^2 with CPMTP_FLAG_AUX).
 *   saved: NULL for inference, else filled for cpmtp_backward.
 *   expert_counts [r] int32 out or NULL: n_a of Eq. 10, the number of positions
 *     whose largest gate weight is expert a (ties to the lowest a).
 */
int cpmtp_forward(const cpmtp_shape* shape, const void* h, const void* W_head, const void* E,
                  const void* W_g, const int32_t* x, float* logp, float* loss,
                  const cpmtp_saved* saved, int32_t* expert_counts, void* workspace,
                  size_t workspace_bytes, int32_t* dev_status, cpmtp_stream stream);

/*
 * Gradient of  sum_i u[i] * logp[i] (+ the balance term with CPMTP_FLAG_AUX)
 * with respect to h, W_head, E and W_g (chain rule through Eq. 9, Eq. 8, Eq. 7);
 * u = dloss_dlogp [N] fp32, or NULL for u[i] = -1/N (the mean negative
 * log-likelihood that training minimises).  The logits are recomputed tile by
 * tile from `saved` (as filled by cpmtp_forward on the same inputs).  Outputs are
 * bf16, rounded once from fp32 accumulators:
 *   dh [N,d], dW_head [n*r,d,d], dE [V,d], dW_g [r,d].
 * Any of the four may be NULL and is then not computed (at least one must be
 * given): with the shared unembedding frozen, as in the paper's fine-tuning
 * set-up, dE = NULL skips a quarter of the backward work; with a frozen trunk
 * dh = NULL skips its GEMM.
 */
int cpmtp_backward(const cpmtp_shape* shape, const void* h, const void* W_head, const void* E,
                   const void* W_g, const int32_t* x, const cpmtp_saved* saved,
                   const float* dloss_dlogp, void* dh, void* dW_head, void* dE, void* dW_g,
                   void* workspace, size_t workspace_bytes, int32_t* dev_status,
                   cpmtp_stream stream);

/*
 * Score a given draft for verification (speculative-decoding section): the same
 * quantity as cpmtp_forward for a small number of positions, tuned for the
 * memory-bound regime where E and W_head are each streamed once.
 *   draft [N,n] int32.  logp_joint [N] fp32 out.
 *   logp_prefix [N,n] fp32 out or NULL: log P(draft[i, 0..s]) for s = 0..n-1,
 *   the mixture with only the first s+1 factors folded into the expert weights
 *   (sampling section; s = 0 is Eq. 11).
 */
int cpmtp_score_draft(const cpmtp_shape* shape, const void* h, const void* W_head, const void* E,
                      const void* W_g, const int32_t* draft, float* logp_joint, float* logp_prefix,
                      void* workspace, size_t workspace_bytes, int32_t* dev_status,
                      cpmtp_stream stream);

/*
 * Generate a draft of n tokens per position from the factors (sampling section).
 * Token s is drawn from  sum_a b_a P^(s)(v | a) / sum_a b_a  with
 * b_a = w_a * prod_{t<s} P^(t)(x_t | a): Eq. 11 for the first token, and for the
 * later ones the expert weights updated with the factors of the tokens already
 * drawn, as the text under Eq. 12 describes (the printed Eq. 12 / Eq. 13 lack the
 * s-th factor and the normaliser).  E and W_head are streamed once; the logits of
 * the N*n*r rows are kept in the workspace (fp32) for the n sequential steps, so
 * this entry point is meant for decode-sized N (N <= 65535, else CPMTP_ERR_LIMIT).
 *   uniform [N,n,V] fp32, every value strictly inside (0,1), or NULL.  NULL: the
 *     most likely token is taken (temperature 0; ties go to the lowest id).
 *     Otherwise the token is argmax_v( log p(v) / temperature - log(-log uniform[v]) ),
 *     an exact draw from the conditional sharpened by 1/temperature (> 0).
 *   topk in [1, 8]: how many most-likely tokens of every conditional to report.
 *   forced [N,n] int32 or NULL: an entry >= 0 is taken as the token of that step instead of the
 *     selection (the candidates reported for the step are still those of the conditional); -1 leaves
 *     the step to the sampler.  A caller walks a draft tree this way: the conditionals of a node are
 *     those given its path.  Entries >= V are clamped to V-1 and raise dev_status 1.
 *   draft [N,n] int32 out.  logp_joint [N] fp32 out or NULL: Eq. 9 at the draft.
 *   topk_tokens [N,n,topk] int32 / topk_logp [N,n,topk] fp32 out or NULL: the
 *     candidates, best first, with their conditional log-probabilities (for a
 *     static draft tree as in the speculative-decoding section).
 * Precision: the SELECTION of a token (and of the candidate set) works on logits computed from the
 * bf16-rounded projected hidden state, both for the step's own factors and for the factors of the tokens
 * already drawn, so among tokens whose probabilities differ by less than about 1 % the choice may differ from
 * exact arithmetic; every VALUE returned (logp_joint, topk_logp) is recomputed from the unrounded state and is
 * within 2e-3 of the definition for the tokens that were chosen.
 */
int cpmtp_sample_draft(const cpmtp_shape* shape, const void* h, const void* W_head, const void* E,
                       const void* W_g, const float* uniform, float temperature, int32_t topk,
                       const int32_t* forced, int32_t* draft, float* logp_joint, int32_t* topk_tokens,
                       float* topk_logp,
                       void* workspace, size_t workspace_bytes, int32_t* dev_status,
                       cpmtp_stream stream);

/*
 * The same log-likelihood with the FULL head of Eq. 6 as printed: one unembedding
 * W^(s)_a in R^{V x d} per (token, expert) instead of E . W_head[s, a],
 *   S[i, s, a, :] = W_full[s*r + a] h[i],     W_full [n*r, V, d] bf16,
 * the parametrisation used when the model is trained from scratch.  All n*r heads
 * run as one GEMM over h; Eq. 8's vocabulary reduction is fused as above and the
 * target logit is read from the fp32 accumulator.  Other arguments as for
 * cpmtp_forward; `saved->z` is not used and may be NULL; logp_prefix [N,n] (or NULL)
 * as for cpmtp_score_draft.  Workspace: CPMTP_OP_FORWARD_FULL.
 */
int cpmtp_forward_full(const cpmtp_shape* shape, const void* h, const void* W_full, const void* W_g,
                       const int32_t* x, float* logp, float* loss, float* logp_prefix,
                       const cpmtp_saved* saved, int32_t* expert_counts, void* workspace,
                       size_t workspace_bytes, int32_t* dev_status, cpmtp_stream stream);

/*
 * Gradients for the full head (same objective and conventions as cpmtp_backward):
 *   dh [N,d], dW_full [n*r,V,d], dW_g [r,d], bf16, all required.
 * The logits are recomputed a few heads at a time.  Workspace: CPMTP_OP_BACKWARD_FULL.
 */
int cpmtp_backward_full(const cpmtp_shape* shape, const void* h, const void* W_full, const void* W_g,
                        const int32_t* x, const cpmtp_saved* saved, const float* dloss_dlogp,
                        void* dh, void* dW_full, void* dW_g, void* workspace,
                        size_t workspace_bytes, int32_t* dev_status, cpmtp_stream stream);

/*
 * Fine-tuning objective with distillation (fine-tuning section, Eq. 14 and the sum after it).
 * For every position i and predicted token k the head's distribution of that token given the
 * tokens before it (taken from the sequence),
 *   p^d[i,k,:] = sum_a pi[i,k,a] P^(k)(. | a),   pi[i,k,a] ~ w_a prod_{t<k} P^(t)(x[i,t] | a)
 * (the conditional of the sampling section), is compared with a frozen model's p^c[i,k,:] =
 * softmax(teacher[i,k,:]):
 *   kl[i,k] = sum_v p^d(v) log(p^d(v) / p^c(v))                 (head first, as printed)
 *   ce[i,k] = -log p^d[i,k,x[i,k]] = logp_prefix[i,k-1] - logp_prefix[i,k]
 *   loss    = (1/N) sum_i sum_k gamma^k (beta kl[i,k] + (1 - beta) ce[i,k])   (k = 0..n-1)
 *             (+ aux_coef * sum_a wbar_a^2 with CPMTP_FLAG_AUX).
 * The printed conditioning of p^d is garbled and the printed sum runs over "0..d"; the reading
 * above is the one the surrounding text supports.  The paper sets beta = 0.9.
 *   teacher [N,n,V] bf16 logits (a constant added to a row changes nothing), 16-byte aligned.
 *   logp [N], logp_prefix [N,n], dsaved->kl [N,n] fp32 out; loss [1] fp32 out or NULL.
 *   saved and dsaved are required and are filled for cpmtp_distill_backward.
 * The vocabulary is swept twice: the fused log-sum-exp pass of cpmtp_forward, then a pass in which
 * the r experts of a (position, token) pair occupy adjacent accumulator rows (padded to a power of
 * two) and are mixed across lanes, so p^d and the logits are never written to memory either.  The teacher
 * logits are read once, in that second pass, which also accumulates their logsumexp (dsaved->lse_t).
 * Workspace: CPMTP_OP_DISTILL_FORWARD.  CPMTP_FLAG_RECOMPUTE_Z is honoured as in cpmtp_forward.
 */
typedef struct cpmtp_distill_saved {
  float* lse_t;  /* [N, n]    logsumexp_v teacher                                  */
  float* logpi;  /* [N, n*r]  log pi                                               */
  float* pm;     /* [N, n*r]  sum_v pi P^(k)(v | a) log(p^d(v) / p^c(v))           */
  float* kl;     /* [N, n]    the KL terms (sum_a pm)                              */
} cpmtp_distill_saved;

int cpmtp_distill_forward(const cpmtp_shape* shape, const void* h, const void* W_head, const void* E,
                          const void* W_g, const int32_t* x, const void* teacher, float beta, float gamma,
                          float* logp, float* logp_prefix, float* loss, const cpmtp_saved* saved,
                          const cpmtp_distill_saved* dsaved, void* workspace, size_t workspace_bytes,
                          int32_t* dev_status, cpmtp_stream stream);

/*
 * Gradient of  sum_i sum_k ( dloss_dprefix[i,k] * logp_prefix[i,k] + dloss_dkl[i,k] * kl[i,k] )
 * (+ the balance term with CPMTP_FLAG_AUX) with respect to h, W_head, E and W_g.  Either weight
 * array may be NULL and then takes the values that make the sum equal the loss of
 * cpmtp_distill_forward for (beta, gamma): dloss_dkl = beta gamma^k / N and
 * dloss_dprefix = (1 - beta)(gamma^(k+1) [k+1 < n] - gamma^k) / N.
 * The KL term reaches the logits directly and, through the expert weights pi, the target terms of
 * the earlier tokens and the gate.  Outputs and the NULL-able gradient pointers as for
 * cpmtp_backward.  Workspace: CPMTP_OP_DISTILL_BACKWARD.
 */
int cpmtp_distill_backward(const cpmtp_shape* shape, const void* h, const void* W_head, const void* E,
                           const void* W_g, const int32_t* x, const void* teacher, const cpmtp_saved* saved,
                           const cpmtp_distill_saved* dsaved, float beta, float gamma, const float* dloss_dprefix,
                           const float* dloss_dkl, void* dh, void* dW_head, void* dE, void* dW_g, void* workspace,
                           size_t workspace_bytes, int32_t* dev_status, cpmtp_stream stream);

/*
 * Verify drafts (draft-then-verify of the Preliminaries; speculative-decoding section).
 * accepted [N] int32 out: how many leading tokens of each draft are kept.
 *  - Greedy (base_tokens != NULL): the longest common prefix of draft [N,n] and the
 *    base model's tokens base_tokens [N,n].
 *  - Probabilistic (base_tokens == NULL): token s of a draft is kept with probability
 *    min(1, p_s / q_s), where q_s = exp(logp_prefix[i,s] - logp_prefix[i,s-1]) is the
 *    probability the CP head gave it (logp_prefix [N,n] as returned by
 *    cpmtp_score_draft) and p_s = exp(logp_base[i,s]) the base model's; uniform [N,n]
 *    in [0,1) decides; counting stops at the first rejection.
 * All pointers are device pointers; no workspace is needed.
 */
int cpmtp_verify_draft(int32_t N, int32_t n, const int32_t* draft, const int32_t* base_tokens,
                       const float* logp_prefix, const float* logp_base, const float* uniform,
                       int32_t* accepted, cpmtp_stream stream);

/*
 * cpmtp_score_draft for callers that cannot hand over scratch memory.  Code that
 * runs where device allocation is off-limits -- inside a serving loop that has
 * frozen its memory pool, in a plugin that is given tensors but no allocator, or
 * after the process has handed all free memory to another component -- has no way
 * to obtain the `workspace` the other entry points ask for.  This variant takes
 * none: its scratch is a fixed array of CPMTP_STATIC_SCRATCH_BYTES that is part of
 * the library image, so every GPU that loads the library holds that much memory
 * until the process exits.  Inputs and outputs are the caller's, exactly as for
 * cpmtp_score_draft, and the results are identical to it.
 *
 *  - Shapes whose scratch need (cpmtp_workspace_bytes(shape, CPMTP_OP_SCORE))
 *    exceeds CPMTP_STATIC_SCRATCH_BYTES are refused with CPMTP_ERR_LIMIT and
 *    nothing is enqueued.  At d = 4096, n*r = 32 that allows up to 8 positions.
 *  - No cudaMalloc / cudaFree or other allocating call is made, on any call.
 *  - The first call on each device looks up the array's device address (a
 *    one-time host-side query, made with that device current, guarded by the
 *    library's cache lock).  Make that first call outside any stream capture.
 *    The address is kept for the life of the process: do not call
 *    cudaDeviceReset() between calls.
 *  - All calls on a device share the one array, which keeps whatever the
 *    previous call left in it.  Every location is written before it is read
 *    within a call, so nothing needs clearing; but two calls that overlap on the
 *    GPU (different streams, no ordering between them) race on it.  Serialise them.
 *  The paper has no counterpart for this entry point.
 */
#define CPMTP_STATIC_SCRATCH_BYTES (4u << 20)
int cpmtp_score_draft_static(const cpmtp_shape* shape, const void* h, const void* W_head, const void* E,
                             const void* W_g, const int32_t* draft, float* logp_joint,
                             float* logp_prefix, int32_t* dev_status, cpmtp_stream stream);

/*
 * cpmtp_forward with the per-step operands in HOST memory: h_host [N,d] bf16 and
 * x_host [N,n] int32 (pinned memory recommended) are copied to the device, the
 * forward pass of Eq. 9 runs, and logp_host [N] / loss_host [1] (either may be
 * NULL) are copied back, all on `stream`.  Weights stay device-resident.  The
 * workspace must hold cpmtp_workspace_bytes(shape, CPMTP_OP_FORWARD) plus
 * cpmtp_host_staging_bytes(shape) bytes.  Returns after enqueueing: synchronise
 * the stream before reading the host outputs.
 */
size_t cpmtp_host_staging_bytes(const cpmtp_shape* shape);
int cpmtp_forward_host(const cpmtp_shape* shape, const void* h_host, const void* W_head,
                       const void* E, const void* W_g, const int32_t* x_host, float* logp_host,
                       float* loss_host, const cpmtp_saved* saved, void* workspace,
                       size_t workspace_bytes, int32_t* dev_status, cpmtp_stream stream);

/*
 * Per-stage device timing, for benchmarks.  Between cpmtp_profile_begin() and
 * cpmtp_profile_end() every kernel launch of the entry points above is bracketed
 * by a pair of CUDA events on the launching stream (host-side bookkeeping only:
 * the numerical path is unchanged).  cpmtp_profile_end() synchronises the device,
 * writes the summed kernel time in milliseconds and the launch count of each
 * stage into stage_ms[count] / stage_launches[count] (count <= CPMTP_STAGE_COUNT;
 * either array may be NULL), releases the events and returns the total number of
 * launches recorded, or a negative error code.  Not thread-safe; one device at a
 * time.  The paper has no counterpart for these two calls.
 */
enum {
  CPMTP_STAGE_GATE = 0,      /* unused: the gate of Eq. 7 runs inside the mixture launch */
  CPMTP_STAGE_PROJ,          /* head projection + target-logit partials */
  CPMTP_STAGE_LSE,           /* unembedding fused with logsumexp_V (Eq. 6, Eq. 8) */
  CPMTP_STAGE_MIXTURE,       /* Eq. 7 + Eq. 9 */
  CPMTP_STAGE_FINALIZE,      /* loss, wbar, counts */
  CPMTP_STAGE_COEFF,         /* backward coefficients */
  CPMTP_STAGE_LOGIT_GRAD,    /* logits recompute -> dloss/dS */
  CPMTP_STAGE_DZ,
  CPMTP_STAGE_DE,
  CPMTP_STAGE_DE_CONVERT,
  CPMTP_STAGE_DW_HEAD,
  CPMTP_STAGE_DH,
  CPMTP_STAGE_DW_G,
  CPMTP_STAGE_DRAFT_STEP,    /* per-token selection passes of cpmtp_sample_draft */
  CPMTP_STAGE_TEACHER_LSE,   /* expert weights per token (Eq. 14); the teacher's logsumexp_V is part of the KL pass */
  CPMTP_STAGE_KL,            /* second unembedding pass: KL term of Eq. 14 */
  CPMTP_STAGE_COUNT
};
int cpmtp_profile_begin(void);
int cpmtp_profile_end(float* stage_ms, int32_t* stage_launches, int count);

#ifdef __cplusplus
}
#endif
#endif /* CPMTP_H */
