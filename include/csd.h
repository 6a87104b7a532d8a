/*
 * csd.h -- C ABI of libcsd: the batched verify-and-resample round of Cool-SD
 * (annealed relaxation of speculative decoding) on one NVIDIA B200 (sm_100a).
 *
 * What one call computes, for B independent sequences with gamma drafted
 * tokens each (Algorithm 1, verification stage):
 *   1. softmax statistics of every target and drafter logit row (Algorithm 1,
 *      "calculate P(x~_i | ...) in parallel");
 *   2. the relaxed acceptance probability f_i = min{1, omega_i P(x~_i)/Q(x~_i)}
 *      (Eq. relax; 0/0 := 1 per the Notations appendix) and the accept test
 *      r_i <= f_i for every position;
 *   3. tau = number of leading accepted positions (the for/break of Algorithm 1);
 *   4. at the first rejected position j = tau + 1 the bound-minimising
 *      resampling distribution G*_j = Norm([P_j - Q_j f_j(.)]_+) (Eq. opt_G,
 *      Theorem 2) and one inverse-CDF draw from it; if every position was
 *      accepted, the bonus token from P_{gamma+1} (Algorithm 1, last step);
 *   5. the emitted block x_{1:tau+1}.
 * The schedule omega_1..omega_gamma is an input (csd_make_schedule builds the
 * paper's: UniformRSD, Eq. sdar, and the linear variant of the ablation).
 *
 * Conventions
 *   - All data pointers are DEVICE pointers owned by the caller unless a
 *     parameter says HOST.  The library reads inputs, writes outputs and the
 *     caller's workspace, and nothing else.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is the
 *     legacy default stream) of the CURRENT device; calls return without
 *     synchronising.  Outputs are valid once the stream has reached that point.
 *   - Return value: CSD_OK (0) or a negative csd_error.  Errors found on the
 *     host are reported before anything is enqueued.  Problems in the DATA
 *     never trap or hang: they set bits in out_status[b] and give a defined
 *     result (see csd_status_bits).
 *   - Layout: row-major, V contiguous.  Row (b, i) of target_logits starts at
 *     element b*target_batch_stride + i*V, of draft_logits at
 *     b*draft_batch_stride + i*V.  The fast path needs 16-byte aligned base
 *     pointers and V*sizeof(element) and the batch strides in bytes to be
 *     multiples of 16; anything else takes a slower scalar path with the same
 *     results.
 *   - Inverse-CDF convention: token = smallest x with C(x) > u*Z in token-id
 *     order (C the running sum of the unnormalised weights, Z their total); if
 *     rounding leaves none, the last x with positive weight.  One uniform per
 *     sequence (uniforms[b][gamma]) serves the resample or the bonus draw.
 *   - If the positive part in Eq. opt_G is empty (P == Q, omega >= 1; reachable
 *     only through rounding) the draw falls back to G := P_j.
 */
#ifndef CSD_H_
#define CSD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { CSD_F32 = 0, CSD_BF16 = 1 } csd_dtype;

typedef enum {
  CSD_OK = 0,
  CSD_ERR_NULL = -1,      /* a required pointer is NULL */
  CSD_ERR_SHAPE = -2,     /* B < 1, gamma outside [1,32], V outside [2, 2^20], bad target_rows/stride */
  CSD_ERR_DTYPE = -3,     /* unknown csd_dtype */
  CSD_ERR_WORKSPACE = -4, /* workspace NULL, misaligned (256 B) or smaller than csd_workspace_size */
  CSD_ERR_ARG = -5,       /* inconsistent options (one unconditional array without the other, top_k < 0, ...) */
  CSD_ERR_LAUNCH = -6,    /* the CUDA runtime refused a launch or copy; see cudaGetLastError */
  CSD_ERR_ALIGN = -7,     /* csd_verify only: the inputs need the scalar path, which needs a workspace
                             (logits not 16-byte aligned, V not a multiple of 4, or V < 128) */
  CSD_ERR_STATIC_LIMIT = -8 /* csd_verify_static only: the problem needs more scratch than the
                               built-in CSD_STATIC_SCRATCH_BYTES */
} csd_error;

/* Bits of out_status[b]; they refer only to positions the algorithm looked at
 * (1..tau+1 and the bonus row), like the sequential loop of Algorithm 1. */
/* Finite logits are expected within +-1e37: the exponent arithmetic multiplies them by log2(e). */
typedef enum {
  CSD_STATUS_BADROW = 1,   /* a row held NaN or +inf, or no finite entry: that position
                              rejects (f := 0).  An unusable drafter row resamples from
                              P_j (Eq. opt_G at f = 0); an unusable target row emits -1. */
  CSD_STATUS_BADTOKEN = 2, /* draft token outside [0, V): that position rejects */
  CSD_STATUS_ZFALLBACK = 4, /* empty positive part of Eq. opt_G (its sum is zero, or below the 1e-38
                               that the fp32 weights can hold): drew from P_j instead.  A valid
                               draft token is rejected at such a position with that probability,
                               so in practice only a CSD_STATUS_BADTOKEN rejection gets here. */
  CSD_STATUS_TIMEOUT = 8    /* a bounded wait inside the kernel gave up (a copy into shared memory did
                               not arrive within about a second): results of this call are unreliable.
                               The condition stays set in the workspace until csd_workspace_init. */
} csd_status_bits;

/*
 * Simple form (Algorithm 1, verification stage; Eq. relax; Eq. opt_G):
 * fp32 logits, contiguous [B, gamma, V] arrays, no bonus row (slot gamma of a
 * fully accepted sequence is -1), no guidance mix, no top-k.
 *
 *   target_logits  [B, gamma, V]  device, read
 *   draft_logits   [B, gamma, V]  device, read
 *   draft_tokens   [B, gamma]     device, read; each in [0, V)
 *   uniforms       [B, gamma+1]   device, read; in (0,1); columns 0..gamma-1 are the
 *                                 accept draws r_i, column gamma the resample draw u
 *   relax_schedule [gamma]        device, read; omega_i >= 0 (all 1.0 = vanilla
 *                                 speculative decoding); negative or NaN counts as 0
 *   out_tokens     [B, gamma+1]   device, written; x_{1:tau+1}, then -1
 *   out_accept_len [B]            device, written; tau in [0, gamma]
 *
 * Scratch: none.  This form never allocates, frees or synchronises and keeps no
 * state between calls, so it may be called from any number of streams at once.
 * It serves only inputs the single-launch path can take -- 16-byte aligned logit
 * pointers, V a multiple of 4, V >= 128 -- and returns CSD_ERR_ALIGN otherwise
 * (csd_verify_ex with a workspace takes any layout).  It has no status output:
 * unusable rows or tokens still give the defined results, silently.
 */
int csd_verify(const float* target_logits, const float* draft_logits, const int32_t* draft_tokens,
               const float* uniforms, const float* relax_schedule, int B, int gamma, int V,
               int32_t* out_tokens, int32_t* out_accept_len, void* stream);

/*
 * Allocation-free form of csd_verify.  (The paper has no counterpart: this entry
 * point exists for the sake of callers, not of the method.)
 *
 * Some callers must not trigger a device allocation when they call into the
 * library: code running between cudaStreamBeginCapture and EndCapture, a
 * serving loop whose memory pool owns every byte of the device and treats a
 * stray cudaMalloc as a bug, a real-time thread that cannot afford the implicit
 * device synchronisation cudaMalloc/cudaFree may bring, or a process that is
 * simply not allowed to grow.  csd_verify allocates (and may re-allocate) its
 * scratch internally and csd_verify_ex wants the caller to provide it; this form
 * does neither.  Its scratch is a fixed array of CSD_STATIC_SCRATCH_BYTES that is
 * part of the library's device image, so every GPU on which the library is
 * loaded holds those bytes from load until the process exits, whether or not
 * this function is ever called.
 *
 * Arguments, results and conventions are exactly those of csd_verify (fp32
 * logits, contiguous [B, gamma, V], no bonus row).  Differences:
 *   - No cudaMalloc, cudaFree or other allocating call is made, ever.
 *   - Problems whose csd_workspace_size(B, gamma, V, CSD_F32) exceeds
 *     CSD_STATIC_SCRATCH_BYTES are refused with CSD_ERR_STATIC_LIMIT before
 *     anything is enqueued (for scale: B=256, gamma=16, V=16384 needs about
 *     1.1 MB and fits; B=512, gamma=16, V=16384 needs 2.2 MB and does not).
 *   - The first call on each device looks up the device address of the array
 *     (a cudaGetSymbolAddress call, made with that device current) and keeps
 *     it; make that first call outside any stream capture.
 *   - All calls on one device share the one array.  Nothing in it has to start
 *     at a value the caller provides -- each call overwrites what it later reads -- so no
 *     clearing is needed between calls, and what a call leaves behind is otherwise
 *     meaningless.  One word is an exception: if a bounded wait inside a kernel ever
 *     gives up (CSD_STATUS_TIMEOUT), that is recorded in the array and stays there
 *     for the life of the process -- the caller cannot run csd_workspace_init on it.
 *     This form has no status output, so nothing reads that word and later calls
 *     are unaffected; a caller that must learn of timeouts uses csd_verify_ex.
 *     Two calls that may run on the GPU at the same time (different
 *     streams, no ordering between them) would overwrite each other's scratch:
 *     keep calls on one device ordered, or use csd_verify_ex with separate
 *     workspaces for the concurrent ones.
 */
#define CSD_STATIC_SCRATCH_BYTES (2u * 1024u * 1024u)
int csd_verify_static(const float* target_logits, const float* draft_logits, const int32_t* draft_tokens,
                      const float* uniforms, const float* relax_schedule, int B, int gamma, int V,
                      int32_t* out_tokens, int32_t* out_accept_len, void* stream);

/*
 * Full form.  Adds: bf16 logits; an optional (gamma+1)-th target row for the
 * bonus token (Algorithm 1, last step); batch strides; guidance mixing fused
 * into the load, z = fmaf(cfg_scale, cond - uncond, uncond) evaluated in fp32
 * with the difference rounded to fp32 first (the drafter-side classifier-free
 * guidance of the paper's Additional Implementation Details, applied here to
 * both models' rows when the unconditional arrays are given); top-k filtering
 * before the softmax (keep every logit >= the k-th largest of its row, ties
 * kept; not in the paper, part of the benchmark definition); per-sequence
 * status; optional diagnostic outputs.
 */
typedef struct csd_params {
  const void* target_logits; /* [B, target_rows, V] conditional (or only) rows     */
  const void* draft_logits;  /* [B, gamma, V]                                      */
  const void* target_uncond; /* same layout as target_logits, or NULL               */
  const void* draft_uncond;  /* same layout as draft_logits; NULL iff target_uncond */
  float cfg_scale;           /* s in uncond + s*(cond - uncond); unused without uncond */
  int32_t top_k;             /* 0 or >= V: off.  Any k gives the exact filter (every logit >= the k-th
                                largest of its row is kept); k up to about 2400 runs at streaming speed,
                                larger k selects every row by radix, several times slower */
  int32_t dtype;             /* csd_dtype of all four logit arrays                  */
  int32_t B, gamma, V;
  int32_t target_rows;         /* gamma or gamma + 1                                */
  int64_t target_batch_stride; /* elements; 0 means target_rows * V                 */
  int64_t draft_batch_stride;  /* elements; 0 means gamma * V                       */
  const int32_t* draft_tokens; /* [B, gamma]                                        */
  const float* uniforms;       /* [B, gamma+1]                                      */
  const float* relax_schedule; /* [gamma]                                           */
  int32_t* out_tokens;         /* [B, gamma+1]                                      */
  int32_t* out_accept_len;     /* [B]                                               */
  int32_t* out_status;         /* [B] or NULL; csd_status_bits                      */
  float* dbg_p;                /* [B, gamma] or NULL: P_i(x~_i)                     */
  float* dbg_q;                /* [B, gamma] or NULL: Q_i(x~_i)                     */
  float* dbg_f;                /* [B, gamma] or NULL: f_i (0 where the row or token is unusable) */
  float* dbg_G;                /* [B, V] or NULL: the distribution the emitted token was drawn
                                  from (G*_j, or P for the bonus draw / fallbacks); zeros if none */
  void* workspace;             /* >= csd_workspace_size(...) bytes, 256-byte aligned, zero-filled
                                  once before its first use (csd_workspace_init or any memset);
                                  every call leaves it ready for the next.  Two calls that may
                                  overlap on the GPU need different workspaces.             */
  size_t workspace_bytes;
  void* stream;
  int back_to_back;            /* 0 (default): ordinary stream order.  The call starts when everything
                                  enqueued before it on the stream has completed, and its work is
                                  spread over the whole GPU (each sequence over up to 8 thread
                                  blocks): the shortest time for one call, and safe after any
                                  producer of its inputs.
                                  1: for many calls enqueued back to back.  The call may START while
                                  the operation before it on the stream is still running
                                  (programmatic dependent launch) and uses one thread block per
                                  sequence once B >= 16, so that the blocks of several consecutive
                                  calls share the GPU; its outputs still become visible in call
                                  order.  The caller guarantees that the inputs of such a call are
                                  NOT produced by the operation that immediately precedes it on
                                  the stream (another call of this library is fine: it writes only
                                  its outputs and its workspace).  Results are identical either
                                  way.                                                           */
  float* diag_accept_mass;     /* [B, gamma] or NULL.  Fidelity/efficiency monitors of Theorem 2, for every   */
  float* diag_bound_term;      /* [B, gamma] or NULL.  position i given its drafted prefix, with
                                  f_i(x) = min{1, omega_i P_i(x)/Q_i(x)}:
                                    accept_mass = sum_x Q_i(x) f_i(x)   (inner sum of Eq. token_exp: the
                                      probability that position i accepts; their running products along
                                      the draft add up to E[tau]);
                                    bound_term  = sum_x |P_i(x) - Q_i(x) f_i(x)| - sum_x (1 - f_i(x)) Q_i(x)
                                      (the bracket of Eq. bd2, i.e. position i's contribution to the
                                      total-variation bound at G*; 0 whenever omega_i <= 1).
                                  NaN where a row of the position is unusable.  Either pointer may be
                                  NULL.  Asking for them costs a second pass over every row.       */
} csd_params;

int csd_verify_ex(const csd_params* p);

/* Bytes of workspace that csd_verify_ex needs for any call with these sizes
 * (any target_rows, guidance and top-k setting).  0 if the sizes are invalid. */
size_t csd_workspace_size(int B, int gamma, int V, int dtype);

/* Number of kernels csd_verify_ex(p) would enqueue (1 on the fused path; 2, or 3 with
 * top-k, on the path for unaligned or very small rows), or a negative csd_error.
 * Validates like csd_verify_ex and enqueues nothing. */
int csd_launch_count(const csd_params* p);

/* Zero-fills a workspace on `stream` (needed once, before its first use; also the
 * way to clear the sticky CSD_STATUS_TIMEOUT condition). */
int csd_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/*
 * Host-buffer form: the same round for a caller whose logits, tokens, uniforms
 * and schedule sit in HOST memory (pinned memory makes the copies asynchronous).
 * Every data pointer of `host` (inputs, outputs, optional diagnostics) is a
 * HOST pointer; host->workspace / workspace_bytes, back_to_back and the two
 * diag_ pointers are ignored (the kernel follows its own input copies in
 * ordinary stream order; the Theorem 2 monitors are outputs of the device form).  `staging` is a
 * DEVICE buffer of at least csd_host_staging_size(host) bytes, 256-byte
 * aligned, that the library uses for the device copies of inputs and outputs
 * and for its workspace.  The call enqueues host->device copies, the kernels and
 * device->host copies of out_tokens / out_accept_len / out_status (and any
 * diagnostics requested) on host->stream and returns; results are in the host
 * arrays once the stream has been synchronised.
 */
int csd_verify_host(const csd_params* host, void* staging, size_t staging_bytes);
size_t csd_host_staging_size(const csd_params* host);

/*
 * Drafting stage (Algorithm 1, "x~_i ~ Q(. | prefix)"): one token per row of logits, drawn from the
 * row's softmax with the same input preparation as the verification (guidance mix fused into the
 * load -- the paper runs the drafter under classifier-free guidance, Additional Implementation
 * Details -- and top-k) and the same inverse-CDF convention.
 *   logits      DEVICE, R rows of V elements (fp32 or bf16), row r at element r*row_stride
 *               (row_stride 0 means V); 16-byte alignment as for csd_verify_ex's fast path
 *   uncond      DEVICE, same layout, or NULL (no guidance mix)
 *   uniforms    DEVICE [R] in (0, 1): token r = smallest x with C_r(x) > uniforms[r] * Z_r
 *   out_tokens  DEVICE [R]; -1 for a row that holds NaN or +inf or no finite entry
 *   out_status  DEVICE [R] or NULL: CSD_STATUS_BADROW / CSD_STATUS_TIMEOUT
 *   workspace   DEVICE, >= csd_sample_workspace_size(R, V, dtype) bytes, 256-byte aligned, zero-filled
 *               once before its first use
 *   back_to_back  as in csd_params
 * Returns CSD_OK or a negative csd_error; nothing is enqueued on an error.
 */
size_t csd_sample_workspace_size(int R, int V, int dtype);
int csd_sample_rows(const void* logits, const void* uncond, float cfg_scale, int top_k, int dtype, int R, int V,
                    int64_t row_stride, const float* uniforms, int32_t* out_tokens, int32_t* out_status,
                    void* workspace, size_t workspace_bytes, int back_to_back, void* stream);

/*
 * Similarity relaxation with the paper's resampling distribution (Ablation Study, "Principled
 * Resampling Strategy": LANTERN++'s acceptance f^{k,lambda} of the Speculative Decoding section with
 * G* of Eq. opt_G in place of LANTERN++'s own G^{k,lambda}).  The round of csd_verify_ex in which the
 * target mass of a candidate x is aggregated over a selected subset of its k nearest tokens:
 *   A(x) = P(x) + sum of P(y) over the selected y,
 *   f_i  = min{1, omega_i A(x~_i) / Q(x~_i)},      G*_j = Norm([P_j - Q_j min{1, omega_j A(.)/Q_j(.)}]_+)
 * (for omega_j >= 1 this G* is the vanilla Norm([P_j - Q_j]_+), Proposition 2).  The paper says only
 * that the subset is "selected" with sum_{y} P(y) < lambda P(x); here neighbours are taken in table
 * order (nearest first) while the running sum stays strictly below lambda P(x), and the first one that
 * would break it ends the selection.
 *   neighbours  DEVICE [V, k] int32: row x lists the nearest tokens of x; entries that are -1, out of
 *               range or x itself are skipped.  1 <= k <= 64.  (The paper's tables come from the image
 *               tokenizer's codebook, which the caller supplies.)
 *   lambda      >= 0; 0 selects nothing: the call then equals csd_verify_ex
 * dbg_p reports A(x~_i).  The Theorem 2 monitors are not available in this form (CSD_ERR_ARG).  The
 * call enqueues two kernels (statistics of every row, then one block per sequence for the tests and the
 * draw), three for rows that are unaligned or shorter than 512 bytes; csd_launch_count does not apply.
 */
int csd_verify_similar(const csd_params* p, const int32_t* neighbours, int k, float lambda);

/*
 * Tree-structured verification: the same round over a static TREE of drafted candidates, the draft
 * structure of the paper's experiments (Experiments, "Implementation Details": the Eagle-1 static
 * tree); Algorithm 1 states the chain, which is the tree in which every node has one child.
 * The paper gives no rule for several candidates of one node under the relaxed test; the rule here:
 *   - the candidates of a node are independent draws from the drafter's distribution Q in that
 *     node's context, and are tried in increasing node index;
 *   - with R the target's distribution in that context, a candidate x at level i is accepted with
 *     probability min{1, omega_i R(x)/Q(x)} (Eq. relax on the current residual); a rejection replaces
 *     R by Norm([R - Q f(.)]_+) (Eq. opt_G applied to R; the recursive rejection sampling of
 *     multi-candidate speculative decoding when omega_i = 1, which keeps Theorem 1), and the next
 *     sibling is tried against that with the same Q;
 *   - an accepted candidate becomes the context of the next level; a node without children ends the
 *     walk with a bonus token from the target's distribution there (Algorithm 1, last step);
 *   - when every candidate of a node is rejected, the emitted token is drawn from the last residual
 *     by inverse CDF with the sequence's one extra uniform.
 * Contexts are numbered 0 (the root: the prefix alone) and n + 1 (after node n); row c of
 * target_logits and of draft_logits is that model's output in context c (the drafter's rows of
 * contexts without children are read for their statistics but never used).
 *   parent         HOST [N]: -1 for a child of the root, else the index of an EARLIER node;
 *                  1 <= N <= 63, at most 8 children per node, at most 32 levels
 *   draft_tokens   DEVICE [B, N]
 *   uniforms       DEVICE [B, N + 1] in (0, 1): the accept draw of every node, then the resample /
 *                  bonus draw
 *   relax_schedule DEVICE [D], D = csd_tree_depth(parent, N): omega of levels 1..D
 *   out_tokens     DEVICE [B, D + 1]: the accepted path's tokens, the drawn token, then -1
 *   out_accept_len DEVICE [B]: number of accepted levels
 *   out_nodes      DEVICE [B, D] or NULL: the node accepted at each level, then -1
 *   out_status     DEVICE [B] or NULL: csd_status_bits (over the contexts the walk visited)
 *   dbg_G          DEVICE [B, V] or NULL: the distribution the emitted token was drawn from
 *   workspace      DEVICE, >= csd_tree_workspace_size(B, N, V, dtype) bytes, 256-byte aligned
 * Other fields as in csd_params.  Every rejection costs one more pass over the two rows of the
 * current context.  Returns CSD_OK or a negative csd_error (CSD_ERR_ARG for a malformed tree);
 * nothing is enqueued on an error.
 */
typedef struct csd_tree_params {
  const void* target_logits; /* [B, N + 1, V]                                        */
  const void* draft_logits;  /* [B, N + 1, V]                                        */
  const void* target_uncond; /* same layouts, or both NULL                           */
  const void* draft_uncond;
  float cfg_scale;
  int32_t top_k;
  int32_t dtype;
  int32_t B, N, V;
  const int32_t* parent;
  const int32_t* draft_tokens;
  const float* uniforms;
  const float* relax_schedule;
  int32_t* out_tokens;
  int32_t* out_accept_len;
  int32_t* out_nodes;
  int32_t* out_status;
  float* dbg_G;
  void* workspace;
  size_t workspace_bytes;
  void* stream;
} csd_tree_params;

int csd_verify_tree(const csd_tree_params* p);
size_t csd_tree_workspace_size(int B, int N, int V, int dtype);
/* Deepest level of the tree (the root's children are level 1), or a negative csd_error. */
int csd_tree_depth(const int32_t* parent_host, int N);

/*
 * Vocabulary-sharded verification: the round for a tensor-parallel LM head, where each of n ranks
 * holds a contiguous slice [v_offset, v_offset + Vs) of every logit row (Algorithm 1's steps are the
 * same; only the three reductions over the vocabulary cross the ranks).  A rank calls, in order and on
 * one stream,
 *   csd_shard_stats    its slice's softmax statistics per row (Algorithm 1, "calculate P ... in
 *                      parallel") and the logits of the drafted tokens that lie in the slice: one
 *                      16-byte record per row, [B * (target_rows + gamma)] of them
 *        -- all-gather the records, rank-major: records_all [n][rows] --
 *   csd_shard_partial  the rows' global statistics, the accept tests and tau (Eq. relax; identical on
 *                      every rank), then the slice's total of Eq. opt_G's weights at position tau + 1
 *                      (and its share of P_j, which the fall-back of an empty positive part uses):
 *                      out_totals [B][2] doubles; dbg_p / dbg_q / dbg_f [B, gamma] or NULL (written by
 *                      the rank with shard == 0)
 *        -- all-gather the totals: totals_all [n][B][2] --
 *   csd_shard_pick     the slice holding the crossing C(x) > u Z picks the token (global id), the
 *                      others report -1: out_candidates [B][2] int32 (token, status bits)
 *        -- all-gather the candidates: candidates_all [n][B][2] --
 *   csd_shard_emit     x_{1:tau+1}, tau and the status on every rank.
 * The exchanges are the caller's (NCCL all-gather of a few KB each); the library never touches a
 * peer's memory.  Slices must be numbered in vocabulary order (the inverse CDF runs in token-id
 * order); they may have different sizes.  The workspace carries state from one of the four calls to
 * the next.  Top-k filtering (its threshold is a k-th largest value over ALL slices) is not available
 * in this form; the guidance mix is.  All pointers are DEVICE pointers.
 */
typedef struct csd_shard_params {
  const void* target_logits; /* [B, target_rows, Vs]: this rank's slice */
  const void* draft_logits;  /* [B, gamma, Vs]                          */
  const void* target_uncond; /* same layouts, or both NULL              */
  const void* draft_uncond;
  float cfg_scale;
  int32_t dtype;
  int32_t B, gamma, target_rows;
  int32_t Vs;                /* tokens in this slice                    */
  int32_t V_total;           /* tokens in all slices                    */
  int32_t v_offset;          /* global id of this slice's first token   */
  int32_t n_shards, shard;   /* ranks, and this rank's index in vocabulary order */
  const int32_t* draft_tokens;
  const float* uniforms;
  const float* relax_schedule;
  void* workspace;           /* >= csd_shard_workspace_size(...) bytes, 256-byte aligned */
  size_t workspace_bytes;
  void* stream;
} csd_shard_params;

size_t csd_shard_workspace_size(int B, int gamma, int target_rows, int Vs, int dtype);
int csd_shard_stats(const csd_shard_params* p, void* out_records);
int csd_shard_partial(const csd_shard_params* p, const void* records_all, double* out_totals, float* dbg_p, float* dbg_q,
                      float* dbg_f);
int csd_shard_pick(const csd_shard_params* p, const void* records_all, const double* totals_all, int32_t* out_candidates);
int csd_shard_emit(const csd_shard_params* p, const int32_t* candidates_all, int32_t* out_tokens, int32_t* out_accept_len,
                   int32_t* out_status);

/*
 * Relaxation schedules, written to HOST memory out_host[0..L-1] = omega_1..omega_L.
 *   kind 0  UniformRSD: omega_i = delta.
 *   kind 1  Cool-SD, Eq. sdar: omega_i = delta * exp(-nu*i - mu) with mu fixed by
 *           sum_{i=1..L} exp(-nu*i - mu) = L  (nu_or_ell = nu >= 0).
 *   kind 2  linear variant of the schedule ablation: omega_i = delta * L * w_i / sum_j w_j,
 *           w_i = (ell - i) / (ell (ell + 1)), clamped at 0 for i >= ell (nu_or_ell = ell > 1).
 * Returns CSD_OK, CSD_ERR_NULL or CSD_ERR_ARG.
 */
int csd_make_schedule(int kind, double delta, double nu_or_ell, int L, float* out_host);

/*
 * Testing aid for the bounded waits (every wait of a kernel on a copy into shared memory gives up
 * after a limit and reports CSD_STATUS_TIMEOUT instead of hanging).  Process-wide, applies to calls
 * made afterwards:
 *   wait_limit_log2_cycles  0: the normal limit (2^31 SM cycles, about a second); 10..40: 2^n cycles
 *   drop_first_copy         non-zero: in every following call, the first copy of thread block 0 is
 *                           announced to its barrier but never issued, so the wait on it runs out
 *                           (nothing is left in flight; the block finishes and the call reports
 *                           CSD_STATUS_TIMEOUT for every sequence)
 * csd_test_hooks(0, 0) restores normal operation.  Returns CSD_OK or CSD_ERR_ARG.  Not for production use.
 */
int csd_test_hooks(int wait_limit_log2_cycles, int drop_first_copy);

/*
 * Testing aid: the library can be built with -DCSD_CHECKED (paper_2601_09212_b200/_build.py,
 * build_checked_library), in which every element access of a logit row whose index comes from the
 * data -- a drafted token, a neighbour id -- or from the row length is tested against the row's
 * length first; a bad index is recorded and the access skipped, so nothing can fault.  This call
 * synchronises the device and copies the record to HOST out_host[4]: number of bad indices seen since
 * the library was loaded, the first one, the length it was tested against, and a site tag (1 vector
 * load, 2 scalar load, 3 bulk copy into shared memory).  Returns 1 from a checked build, 0 from the normal build (whose record stays
 * zero), or a negative csd_error.
 */
int csd_checked_report(int32_t* out_host);

/* Static, NUL-terminated description of a csd_error value. */
const char* csd_error_string(int code);

/* Version of this ABI: major*10000 + minor*100 + patch. */
int csd_version(void);

#ifdef __cplusplus
}
#endif
#endif /* CSD_H_ */
