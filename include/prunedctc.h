/*
 * prunedctc.h -- C ABI of the Pruned-CTC head-and-loss library for NVIDIA B200 (sm_100a).
 *
 * One call evaluates Algorithm 1 of the paper ("Pruned CTC"): the CTC loss of a
 * batch under a full-vocabulary softmax head, and the gradients of the sum of
 * the utterance losses with respect to the head input and the head, without
 * ever holding a frames-by-vocabulary array.
 *
 * All device work is ordered after what the caller enqueued on its stream, and
 * the stream waits for all of it (the alignment DP runs on one auxiliary stream
 * per device that the library creates at its first call and joins back before
 * the call's later steps).  Every buffer is owned by the caller; the library
 * keeps no pointers between calls and, except where an entry point says
 * otherwise, allocates no device memory.  Calls on one device must not be issued
 * from several host threads at once; several devices may be driven from one process.
 * No call waits for the stream or for the device: the host length arrays travel as kernel
 * parameters and every table derived from them is built on the device.
 * pruned_ctc_fwd_bwd, its traced and host-buffer forms and pctc_greedy_decode fork onto
 * the library's auxiliary streams, which has not been arranged for stream capture: on a
 * stream that is being captured they return PCTC_ERR_UNSUPPORTED before enqueuing anything.
 * Functions return a status code and never throw or abort.
 */
#ifndef PRUNEDCTC_H_
#define PRUNEDCTC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  PCTC_OK = 0,
  PCTC_ERR_INVALID_ARG = 1,         /* null pointer, non-positive size, length out of range      */
  PCTC_ERR_WORKSPACE_TOO_SMALL = 2, /* workspace_bytes below pctc_workspace_bytes()              */
  PCTC_ERR_UNSUPPORTED = 3,         /* dtype/shape the kernels do not cover (see each function)  */
  PCTC_ERR_CUDA = 4,                /* a CUDA runtime or driver call failed (launch errors)      */
  PCTC_ERR_BAD_TARGET = 5,          /* reserved: bad targets are reported per utterance instead  */
  PCTC_ERR_TIMEOUT = 6              /* a bounded device-side wait gave up (see pctc_workspace_status) */
} pctc_status_t;

typedef enum { PCTC_BF16 = 0, PCTC_FP32 = 1 } pctc_dtype_t;

/* Which contraction kernels run.  AUTO: tcgen05 tensor-core kernels for bf16,
 * fp32 FMA kernels for fp32.  SIMT: the FMA kernels for either dtype (bf16
 * operands are widened to fp32; used to cross-check the tensor-core path). */
typedef enum { PCTC_GEMM_AUTO = 0, PCTC_GEMM_SIMT = 1 } pctc_gemm_path_t;

/* Per-utterance flags written to `utt_flags` (Appendix B.1, "Loss aggregation"). */
#define PCTC_UTT_INFEASIBLE 1 /* T_n < |y_n| + (adjacent equal pairs): no alignment exists  */
#define PCTC_UTT_NONFINITE 2  /* loss not finite (NaN/Inf input, or empty retained lattice)  */
#define PCTC_UTT_BAD_TARGET 4 /* a token equals blank_id or lies outside [0, V)              */
#define PCTC_UTT_SUBSET_OVERFLOW 8 /* the batch has more selected classes than problem.max_K  */

/*
 * The problem of Section 3.1 / Algorithm 1, line 1.
 *   hidden  [N, T, D]  padded head-input states; utterance n has T_n valid frames
 *   W       [V, D]     head weight, bias [V] optional; logits Z = X W^T + 1 b^T
 *   targets [N, target_stride] blank-free token ids, first U_n entries of row n count
 */
typedef struct {
  int32_t N;             /* utterances                                                        */
  int32_t T;             /* padded frames per utterance (row count of hidden[n])              */
  int32_t D;             /* head input width; bf16 tensor-core path needs D % 8 == 0          */
  int64_t V;             /* classes, blank included (any value >= 1)                          */
  int32_t dtype;         /* pctc_dtype_t of hidden, W, bias, dH, dW, dbias; loss is fp32      */
  int32_t blank_id;      /* in [0, V)                                                         */
  float   beam;          /* alignment beam in nats (Section 3.3); <= 0 or +inf: no pruning    */
  int32_t chunk;         /* vocabulary chunk width C (Algorithm 1); 0: library default        */
  int32_t target_stride; /* row pitch of targets and relabeled_out                            */
  int32_t gemm_path;     /* pctc_gemm_path_t                                                  */
  int32_t skip_dW;       /* 1: frozen head (the LLM-CTC setting, Section 4.2): dW is neither
                            computed nor touched (dW may be NULL); dH and dbias still are        */
  int32_t accumulate_dW; /* 1: dW and dbias are added to (gradient accumulation over
                            micro-batches) instead of overwritten                              */
  int32_t forward_only;  /* 1: losses only (validation): lines 11-17 are skipped, dH, dW and dbias
                            are neither computed nor touched and may be NULL                    */
  int32_t max_K;         /* 0, or a promise K <= max_K (K = |U| is only known on the device; a
                            data loader that holds the targets on the host knows it).  Sizes the
                            [M, K] buffers by max_K instead of the bound 1 + sum U_n.  If the
                            batch breaks the promise, nothing faults: every utterance is flagged
                            PCTC_UTT_SUBSET_OVERFLOW, losses and gradients are zero, and the
                            status word reads non-zero                                          */
  const float* utt_weights; /* device [N] or NULL: upstream gradient c_n of each utterance loss
                            (loss scaling, token-count normalisation; Appendix B.1, "row sums of
                            G"): gradients are those of sum_n c_n L_n; the returned losses stay
                            unweighted.  NULL means c_n = 1                                    */
} pctc_problem_t;

/*
 * Workspace size for a problem (host-only; touches no device).
 * input_lengths_host [N]: 1 <= T_n <= T.  target_lengths_host [N]: 0 <= U_n <= target_stride.
 * The size depends on M = sum T_n, D, sum U_n and the chunk width, and on V only
 * through O(V) index tables: there is no M*V term (Section 3.4, activation storage).
 */
pctc_status_t pctc_workspace_bytes(const pctc_problem_t* problem,
                                   const int32_t* input_lengths_host,
                                   const int32_t* target_lengths_host,
                                   size_t* bytes_out);

/*
 * The vocabulary chunk width C a call on this problem will use, and the number of
 * chunks ceil(V / C) (host-only; touches no device).  With problem->chunk > 0 it
 * is that value rounded up to the tile width of the path that runs; with 0 it is
 * the library's choice: 4,096 for fp32; for bf16 and D <= 1,024 the largest of 56,832,
 * 37,888 and 18,944 columns (multiples of 74 x 256: whole waves of the 74 CTA pairs of a
 * B200) whose [M, C] chunk temporary of Algorithm 1 (lines 12-13) stays within 512 MiB;
 * otherwise 16,384 columns, halved down to no less than 8,192 while that temporary would
 * exceed 512 MiB.  The
 * chunk width changes the order of summation only, never what is computed.
 * nchunks_out may be NULL.  Same argument checks as pctc_workspace_bytes.
 */
pctc_status_t pctc_chunk_width(const pctc_problem_t* problem,
                               const int32_t* input_lengths_host,
                               const int32_t* target_lengths_host,
                               int32_t* chunk_out, int32_t* nchunks_out);

/*
 * Algorithm 1, forward and backward in one call.
 *
 * Steps, all on `stream`:
 *   line 2-3  U = blank followed by the ascending distinct target labels; K = |U|;
 *             targets relabelled by their index in U               -> subset_out, K_out, relabeled_out
 *   line 4    the M = sum T_n valid frames are stacked             (workspace)
 *   line 5    lambda_m = log sum_v exp Z[m,v], online over vocabulary chunks (Eq. "lognorm")
 *   line 6    Z_U = X W_U^T + 1 b_U^T  (workspace, fp32); the shift by lambda is applied to
 *             the loss instead of to every entry (Eq. "ctc-factorization"): occupancies do
 *             not depend on it, and the DP can run while line 5 is still computing
 *   line 7-9  per utterance: loss = sum_t lambda_t - log sum over (retained) alignments of
 *             exp(sum_t Z_U); loss of an infeasible, bad-target or non-finite utterance
 *             is 0                                                  -> loss, utt_flags
 *   line 10   occupancies gamma (G = -gamma)                       (workspace, fp32)
 *   line 11-17 per vocabulary chunk: recompute Z, dZ = w_m (exp(Z - lambda) - scatter_U(gamma))
 *             (Eq. "vjp"; w_m = c_n on frames of utterance n, 0 on frames of excluded utterances),
 *             dH += dZ W_c, dW_c = dZ^T X, db_c = dZ^T 1           -> dH, dW, dbias
 *
 * Pointers (device unless marked HOST; all contiguous, row-major):
 *   hidden [N,T,D], W [V,D], bias [V] or NULL, targets [N,target_stride] int32,
 *   input_lengths HOST [N], target_lengths HOST [N],
 *   loss [N] fp32 (per-utterance, not normalised),
 *   dH [N,T,D] (padded frames are written as zero), dW [V,D] (overwritten),
 *   dbias [V] or NULL (ignored when bias is NULL),
 *   subset_out [1 + sum U_n] or NULL, K_out [1] or NULL,
 *   relabeled_out [N,target_stride] or NULL (entries past U_n and bad tokens: -1),
 *   utt_flags [N] or NULL,
 *   workspace: >= pctc_workspace_bytes(), 256-byte aligned.
 * hidden, W, dH, dW must be 16-byte aligned.
 *
 * Gradients are those of the plain sum of the utterance losses (no division by
 * token or frame counts).  With a finite beam the retained lattice is treated
 * as fixed (Section 3.3).
 *
 * Errors: host-detectable problems return before anything is launched and leave
 * the outputs untouched.  Bad targets and non-finite losses never fault; they are
 * reported in utt_flags.  The return value covers launch errors only: the call
 * does not synchronise.
 */
pctc_status_t pruned_ctc_fwd_bwd(const pctc_problem_t* problem,
                                 const void* hidden, const void* W, const void* bias,
                                 const int32_t* targets,
                                 const int32_t* input_lengths, const int32_t* target_lengths,
                                 float* loss, void* dH, void* dW, void* dbias,
                                 int32_t* subset_out, int32_t* K_out, int32_t* relabeled_out,
                                 int32_t* utt_flags,
                                 void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same call with a per-phase timeline, for measurement.  The caller creates
 * `capacity` CUDA events (timing enabled); the call records one at the start of
 * every phase and one at the end, on `stream`, without synchronising:
 * events[i], events[i+1] bracket a span of phase kinds[i], for i < used-1;
 * spans with a negative kind are gaps between streams and carry no meaning (the
 * alignment DP runs on an auxiliary stream, concurrently with line 5).
 * capacity must be at least 12 + 4 * (number of vocabulary chunks), i.e.
 * 12 + 4 * ceil(V / chunk); otherwise PCTC_ERR_INVALID_ARG and nothing is launched.
 * trace == NULL makes the call identical to pruned_ctc_fwd_bwd.  No counterpart
 * in the paper (its Appendix C times whole steps with a device synchronise).
 */
#define PCTC_PHASE_PREP 0        /* Algorithm 1 lines 2-4: subset, relabel, frame stacking       */
#define PCTC_PHASE_LSE 1         /* line 5: chunked projection with online log-sum-exp            */
#define PCTC_PHASE_SUBSET_LOGP 2 /* line 6: gather W_U, S = X W_U^T + b_U - lambda                */
#define PCTC_PHASE_DP 3          /* lines 7-10: alignment DP, losses, occupancies                 */
#define PCTC_PHASE_DLOGITS 4     /* lines 13-14: recompute Z_c and form Eq. "vjp"                 */
#define PCTC_PHASE_DH 5          /* line 15: dX += dZ_c W_c                                       */
#define PCTC_PHASE_DW 6          /* line 16: dW_c = dZ_c^T X                                      */
#define PCTC_PHASE_DBIAS 7       /* line 16: db_c = dZ_c^T 1                                      */
#define PCTC_PHASE_FINISH 8      /* un-stacking dX into [N,T,D], integer outputs                  */

typedef struct {
  void** events;    /* HOST array of cudaEvent_t handles, [capacity]                    */
  int32_t capacity;
  int32_t used;     /* out: number of events recorded                                   */
  int32_t* kinds;   /* HOST [capacity], out: kinds[i] = phase of span (events[i], events[i+1]) */
} pctc_trace_t;

pctc_status_t pruned_ctc_fwd_bwd_traced(const pctc_problem_t* problem,
                                        const void* hidden, const void* W, const void* bias,
                                        const int32_t* targets,
                                        const int32_t* input_lengths, const int32_t* target_lengths,
                                        float* loss, void* dH, void* dW, void* dbias,
                                        int32_t* subset_out, int32_t* K_out, int32_t* relabeled_out,
                                        int32_t* utt_flags,
                                        void* workspace, size_t workspace_bytes, void* stream,
                                        pctc_trace_t* trace);

/*
 * The same computation for callers whose tensors live in HOST memory (pinned
 * memory makes the copies asynchronous).  Every data pointer of
 * pruned_ctc_fwd_bwd is a host pointer here; `device_scratch` is one device
 * buffer of at least pctc_host_call_scratch_bytes() bytes, 256-byte aligned,
 * that the call carves into input staging, output staging and the workspace.
 * Order: host-to-device copies of hidden, bias, targets on `stream`; W follows on a
 * copy stream of the library in four row segments, and the normaliser kernel of a
 * segment starts as soon as that segment has landed (for V >= 16,384; the summation
 * order of lambda then differs from the device entry point in the last bits);
 * Algorithm 1; the rows of dW go back to the host chunk by chunk while later
 * chunks are still being computed (with problem->chunk == 0 a bf16 call uses
 * 8,192-column chunks here, so that the first rows leave early); loss, dH, dbias and the optional integer
 * outputs at the end.  `stream` waits for all of it.  The call does not synchronise: the host outputs are valid once
 * `stream` has been synchronised, and the host inputs must stay unchanged until
 * then.  Same return codes as pruned_ctc_fwd_bwd.  skip_dW, accumulate_dW and utt_weights
 * belong to the device entry point only: here they return PCTC_ERR_UNSUPPORTED.
 */
pctc_status_t pctc_host_call_scratch_bytes(const pctc_problem_t* problem,
                                           const int32_t* input_lengths_host,
                                           const int32_t* target_lengths_host,
                                           int32_t has_bias, size_t* bytes_out);

pctc_status_t pruned_ctc_fwd_bwd_host(const pctc_problem_t* problem,
                                      const void* hidden, const void* W, const void* bias,
                                      const int32_t* targets,
                                      const int32_t* input_lengths, const int32_t* target_lengths,
                                      float* loss, void* dH, void* dW, void* dbias,
                                      int32_t* subset_out, int32_t* K_out, int32_t* relabeled_out,
                                      int32_t* utt_flags,
                                      void* device_scratch, size_t scratch_bytes, void* stream);

/*
 * Greedy CTC recognition with the same head (the paper's recognition path for
 * LLM-CTC, Section 5.1 / Appendix D: the head is applied in vocabulary chunks, the
 * frame-wise arg-max is taken and the CTC collapse map B of Section 3.1 -- merge
 * repeats, then drop blanks -- gives the hypothesis).  The logits are never
 * stored: the projection kernel keeps a running (max, arg-max) per frame.
 *
 * Uses N, T, D, V, dtype, blank_id, gemm_path of `problem`.  hidden [N,T,D], W [V,D],
 * bias [V] or NULL (device); input_lengths HOST [N].  Outputs (device):
 *   frame_labels [N,T] or NULL: arg-max class of every valid frame, -1 on padded frames
 *                 (the smallest index wins among equal logits);
 *   tokens [N,T]: the collapsed hypothesis of each utterance, padded with -1;
 *   token_lengths [N].
 * workspace: at least pctc_greedy_workspace_bytes(), 256-byte aligned.
 */
pctc_status_t pctc_greedy_workspace_bytes(const pctc_problem_t* problem, const int32_t* input_lengths_host,
                                          size_t* bytes_out);
pctc_status_t pctc_greedy_decode(const pctc_problem_t* problem,
                                 const void* hidden, const void* W, const void* bias,
                                 const int32_t* input_lengths,
                                 int32_t* frame_labels, int32_t* tokens, int32_t* token_lengths,
                                 void* workspace, size_t workspace_bytes, void* stream);

/*
 * The k best classes of every frame with their log-probabilities under the full-vocabulary
 * softmax: what a CTC prefix beam search (the paper's decoder, Section 5.1: beam 4; the search
 * itself is not part of this library) consumes per frame.  The head is applied in vocabulary
 * chunks of problem->chunk columns (0: 4,096) as in the paper's recognition path (Appendix D);
 * a chunk's logits live in the workspace only until the frame's running k best and its running
 * log-sum-exp (Eq. "lognorm") have been updated, so no frames-by-vocabulary array exists.
 *
 * Uses N, T, D, V, dtype, chunk, gemm_path of `problem`.  hidden [N,T,D], W [V,D], bias [V] or
 * NULL (device); input_lengths HOST [N]; k is 1, 2, 4 or 8.  Outputs (device):
 *   topk_classes  [N,T,k] int32: classes by descending logit, the smaller class first among
 *                 equal logits; -1 on padded frames and for ranks beyond V;
 *   topk_logprobs [N,T,k] fp32 or NULL: log p of those classes; -inf where the class is -1.
 * workspace: at least pctc_topk_workspace_bytes(), 256-byte aligned.
 */
pctc_status_t pctc_topk_workspace_bytes(const pctc_problem_t* problem, const int32_t* input_lengths_host,
                                        int32_t k, size_t* bytes_out);
pctc_status_t pctc_topk_decode(const pctc_problem_t* problem,
                               const void* hidden, const void* W, const void* bias,
                               const int32_t* input_lengths, int32_t k,
                               int32_t* topk_classes, float* topk_logprobs,
                               void* workspace, size_t workspace_bytes, void* stream);

/*
 * Contraction kernel on its own, for validation of the tensor-core path:
 *   C[i,j] = sum_k A(i,k) B(j,k),  i < m, j < n, k < k,  C fp32 [m, n] row-major.
 * a_mn_major == 0: A is stored [m, k] (k contiguous); else A is stored [k, m].
 * b_mn_major == 0: B is stored [n, k] (k contiguous); else B is stored [k, n].
 * Operands are bf16 device arrays, 16-byte aligned, with the contiguous extent a
 * multiple of 8.  gemm_path as in pctc_problem_t.  Not part of Algorithm 1: it is
 * the building block of lines 5, 6 and 13-16.
 */
pctc_status_t pctc_gemm_bf16(const void* A, const void* B, float* C,
                             int32_t m, int32_t n, int32_t k,
                             int32_t a_mn_major, int32_t b_mn_major,
                             int32_t gemm_path,
                             int32_t* device_status, /* device [1] or NULL; see below */
                             void* stream);

/*
 * Algorithm 1 lines 2-3 on their own, for callers that cannot allocate device
 * memory.  (The paper has no counterpart: this is a packaging of the subset and
 * relabelling step, not another method.)
 *
 * Who needs it: code that runs where cudaMalloc is off the table -- inside a
 * framework's memory-pool callback, in a process whose device memory was handed
 * out in full at start-up, or in a latency-critical loop that must not touch the
 * allocator -- and that only wants U, K and the relabelled targets, e.g. to size
 * its own buffers before the main call.  pruned_ctc_fwd_bwd takes its scratch
 * from a caller-provided workspace; this entry point needs no workspace at all:
 * its scratch (a V-bit set, its rank table and a class-to-index map) lives in a
 * fixed device array inside the library, PCTC_NOALLOC_MAX_V classes large
 * (about 1.1 MB, resident on every GPU that loads the library until exit).
 *
 *   targets [N, target_stride] int32 (device), target_lengths [N] int32 (DEVICE
 *   here, unlike pruned_ctc_fwd_bwd), outputs as in pruned_ctc_fwd_bwd, all
 *   device and all required: subset_out [1 + sum U_n] (entries past K are left
 *   untouched), K_out [1], relabeled_out [N, target_stride], utt_flags [N]
 *   (only PCTC_UTT_BAD_TARGET can be set).
 *
 * V > PCTC_NOALLOC_MAX_V returns PCTC_ERR_UNSUPPORTED and launches nothing.
 * The call makes no cudaMalloc/cudaFree and uses no allocating library routine.
 * The first call on each device looks up the address of the scratch array
 * (with that device current); make that first call before any stream capture.
 * All calls share the one array: calls whose kernels overlap on the GPU (two
 * streams, two threads) race on it.  The array keeps the previous call's
 * contents; each call clears what it reads before use.
 */
#define PCTC_NOALLOC_MAX_V 262144
pctc_status_t pctc_subset_relabel_noalloc(const int32_t* targets, const int32_t* target_lengths,
                                          int32_t N, int32_t target_stride, int64_t V, int32_t blank_id,
                                          int32_t* subset_out, int32_t* K_out, int32_t* relabeled_out,
                                          int32_t* utt_flags, void* stream);

/*
 * Device-side status word.  Every wait inside a kernel (on an mbarrier) is
 * bounded; a wait that gives up stores a non-zero code and the kernel returns
 * cleanly instead of hanging: it waits (again bounded) for the copies and tensor-core
 * operations it has in flight, frees its tensor memory and leaves.  pruned_ctc_fwd_bwd
 * keeps the word at the start of its workspace (zeroed by each call); this function
 * copies it to the host after synchronising `stream`.  Codes (the first event wins):
 *   0            nothing to report                                     -> PCTC_OK
 *   1 .. 4       a bounded wait gave up (1 producer waiting for a free stage, 2 MMA issuer
 *                waiting for a drained accumulator, 3 MMA issuer waiting for operands,
 *                4 epilogue waiting for an accumulator)                 -> PCTC_ERR_TIMEOUT
 *   0x100        the batch has more selected classes than problem.max_K -> PCTC_ERR_INVALID_ARG
 *   0x201 ..     only in a library built with -DPCTC_DEBUG_BOUNDS: an index that a kernel was
 *                about to gather or scatter through was out of range (0x200 + checking site);
 *                the access was skipped                                 -> PCTC_ERR_INVALID_ARG
 * `workspace` may be any device word that received a status, e.g. the device_status of
 * pctc_gemm_bf16.
 */
pctc_status_t pctc_workspace_status(const void* workspace, void* stream, int32_t* status_host);

const char* pctc_status_string(pctc_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* PRUNEDCTC_H_ */
