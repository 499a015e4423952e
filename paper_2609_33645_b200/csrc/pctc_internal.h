// Internal declarations shared by the translation units of libprunedctc.
// Host-callable launch wrappers only; every wrapper enqueues on `stream` and
// returns the cudaError_t of its launch.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace pctc {

// ---------------------------------------------------------------------------
// Index checks of the debug build (-DPCTC_DEBUG_BOUNDS): every index a kernel gathers or scatters
// through (row tables, selected classes, relabelled targets, label chains) is range-checked before
// use.  A bad index stores 0x200 + the number of the checking site in the status word (the first
// one wins) and the access is skipped; nothing faults.  In the regular build the check is compiled
// out.  Status word codes: 1-4 a bounded wait gave up (which wait), 0x100 more selected classes than
// problem.max_K, 0x201.. an index out of range.
// ---------------------------------------------------------------------------
#ifdef PCTC_DEBUG_BOUNDS
constexpr bool kCheckBounds = true;
#else
constexpr bool kCheckBounds = false;
#endif
#ifdef __CUDACC__
__device__ __forceinline__ bool index_ok(long long idx, long long lo, long long hi, int* status, int site) {
  if (!kCheckBounds) return true;
  if (idx >= lo && idx < hi) return true;
  if (status) atomicCAS(status, 0, 0x200 + site);
  return false;
}
#endif

// ---------------------------------------------------------------------------
// Contractions:  acc(i,j) = sum_k A(i,k) * B(j,k),  then an epilogue.
// ---------------------------------------------------------------------------

enum EpiKind : int {
  EPI_STORE_F32 = 0,    // C[i*ld + j] = acc                                  (validation GEMM)
  EPI_LSE_PARTIAL = 1,  // running (max, sum exp) of z = acc + bias[j] over a column range
  EPI_SUBSET_LOGP = 2,  // S[i*ld + j] = acc + bias[U[j]] - lambda[i],  j < K  (Algorithm 1 line 6); lambda null: no shift
  EPI_DLOGITS = 3,      // chunk[i*ld + j] = w_i (exp(acc + bias[v0+j] - lambda[i]) - gamma[i, vmap[v0+j]])
  EPI_ACCUM_F32 = 4,    // acc_out[i*ld + j] (+)= acc                          (dH across chunks)
  EPI_STORE_OUT = 5,    // out[i*ld + j] = T(acc)                              (rows of dW)
  EPI_ARGMAX_PARTIAL = 6  // running (max, argmax) of z = acc + bias[j] over a column range (recognition)
};

struct Epilogue {
  int kind = EPI_STORE_F32;
  void* out = nullptr;          // destination (type depends on kind)
  long long ld = 0;             // its row pitch in elements
  const float* lambda = nullptr;
  const void* bias = nullptr;   // [V] in the operand dtype, or null
  long long v0 = 0;             // vocabulary index of column 0 (EPI_DLOGITS / EPI_LSE_PARTIAL)
  const int* vmap = nullptr;    // [V] class -> index in U, or -1
  const float* gamma = nullptr; // [M, ld_gamma]
  long long ld_gamma = 0;
  const float* roww = nullptr;  // [M] 1 for frames of utterances in N+, else 0
  const int* U = nullptr;       // [K] selected classes
  const int* Kdev = nullptr;    // device scalar K
  float2* partial = nullptr;    // [M, partial_stride] (max, sum) or (max, arg-max)
  int nsplit = 1;               // column splits of this launch
  int partial_stride = 0;       // split slots per row in `partial` (0: nsplit); a launch over a row
  int partial_offset = 0;       // segment of B writes its splits at partial_offset .. +nsplit-1
  int accumulate = 0;           // EPI_ACCUM_F32 / EPI_STORE_OUT: add to the destination instead of overwriting
  int out_is_bf16 = 0;          // EPI_DLOGITS / EPI_STORE_OUT destination type
  float* colpart = nullptr;     // EPI_DLOGITS on the tensor-core path: [ceil(m/32), ld_colpart] column sums of
  long long ld_colpart = 0;     //   each block of 32 rows of the rounded output (db_c = dZ_c^T 1), or null
  int ksplit = 1;               // EPI_ACCUM_F32 on the tensor-core path: the contraction is cut into this many
  int ksplit_rows = 0;          //   ranges of k; range s accumulates into rows [s * ksplit_rows, ...) of `out`
  long long vocab = 0;          // V, for the index checks of the debug build
  int* status = nullptr;        //   ... and the status word they report to
};

struct GemmShape {
  int m = 0, n = 0, k = 0;      // extents of i, j, k
  // element strides: A(i,k) at A[i*a_i + k*a_k], B(j,k) at B[j*b_j + k*b_k]
  long long a_i = 0, a_k = 0, b_j = 0, b_k = 0;
};

// fp32-FMA contraction (operands fp32 or bf16 widened to fp32).
cudaError_t simt_gemm(const void* A, const void* B, bool operands_bf16, const GemmShape& g,
                      const Epilogue& e, cudaStream_t stream);

// tcgen05 tensor-core contraction, bf16 operands.  A is [m,k] (a_mn_major=0) or [k,m];
// B is [n,k] (b_mn_major=0) or [k,n]; row pitches lda/ldb in elements (multiples of 8).
// status: device word receiving a non-zero code if a bounded wait gives up.
cudaError_t umma_gemm(const __nv_bfloat16* A, long long lda, bool a_mn_major,
                      const __nv_bfloat16* B, long long ldb, bool b_mn_major,
                      int m, int n, int k, const Epilogue& e, int* status, cudaStream_t stream);
bool umma_available();   // the driver entry point for tensor maps could be resolved
int umma_lse_splits(int m, int n);   // column splits (<= 32) for EPI_LSE_PARTIAL on this device
// EPI_ACCUM_F32 with few output tiles (small m x n): how many k-ranges per tile fill the device, given
// that every range beyond the first costs another [slab_rows, n] fp32 accumulator (at most max_extra_bytes
// in total); and the slab height (m rounded up to whole row tiles) that goes with it.
int umma_accum_splits(int m, int n, int k, size_t max_extra_bytes);
int umma_accum_slab_rows(int m);
int umma_lse_partials_per_split(int k);   // the kernel writes this many partials per split (1 or 2):
                                          // partial[(i*nsplit + sp)*pps + h]

// Combine argmax partials (value, column index as int bits): labels[i] = argmax, smallest index on ties.
cudaError_t argmax_combine(const float2* partial, int nparts, int M, int* labels, cudaStream_t stream);

// Greedy CTC hypothesis per utterance: merge repeated frame labels, drop blanks.  frame_labels (may be
// null) and tokens are [N, T] padded with -1; token_lengths [N].
cudaError_t greedy_collapse(const int* labels, const int* row0, const int* T_n, int N, int T, int blank,
                            int* frame_labels, int* tokens, int* token_lengths, cudaStream_t stream);

// The k best classes per stacked frame (k in {1, 2, 4, 8}), chunk by chunk: `logits` is an fp32
// [M, ld] block holding columns v0 .. v0+cols-1 of X W^T (bias, if any, is added here); run_val/run_idx
// [M, k] and run_ms [M] (max, sum of exponentials) carry the state between chunks (first: start afresh).
// Order: larger logit first, smaller class index among equals.
cudaError_t topk_update(int k, const float* logits, long long ld, int M, int cols, long long v0, const void* bias,
                        bool bias_bf16, float* run_val, int* run_idx, float2* run_ms, bool first, cudaStream_t stream);
// classes [N,T,k] (-1 on padded frames) and log-probabilities [N,T,k] (may be null) from that state
cudaError_t topk_finish(int k, const float* run_val, const int* run_idx, const float2* run_ms, const int* row0,
                        const int* T_n, int N, int T, int* classes, float* logprobs, cudaStream_t stream);

// Combine LSE partials: lambda[i] = log sum over splits.
cudaError_t lse_combine(const float2* partial, int nsplit, int M, float* lambda, cudaStream_t stream);

// ---------------------------------------------------------------------------
// Integer / copy steps
// ---------------------------------------------------------------------------

struct BatchMeta {              // device arrays describing the batch
  const int* T_n;               // [N]
  const int* U_n;               // [N]
  const int* row0;              // [N+1] first stacked row of each utterance
  const long long* cell0;       // [N] first trellis cell of each utterance
  const int* row_utt;           // [M] utterance of each stacked row
  int N = 0, M = 0;             // extents, for the index checks of the debug build
  int* status = nullptr;        // status word
};

// Batch description from the host length arrays (U_host may be null: no targets).  The lengths
// travel as kernel parameters, so nothing is copied from pageable host memory and the host does
// not wait for the stream.  Writes T_n [N], U_n [N], row0 [N+1], cell0 [N] and mcell0 [N] (either
// may be null), row_utt [M].
cudaError_t batch_meta(const int* T_host, const int* U_host, int N, int* T_n, int* U_n, int* row0,
                       long long* cell0, long long* mcell0, int* row_utt, cudaStream_t stream);

// Algorithm 1 lines 2-3.  bitmap: ceil(V/32) words (zeroed here), vmap: [V].
cudaError_t subset_and_relabel(const int* targets, int target_stride, const int* U_n_dev, int N,
                               long long V, int blank, unsigned* bitmap, int* word_rank,
                               int* vmap, int* U_out, int* K_out, int* relabeled, int* utt_flags,
                               int cap, int* status, cudaStream_t stream);   // cap: capacity of U_out

// Algorithm 1 line 4: X[row0[n] + t] = hidden[n, t], t < T_n.
cudaError_t stack_frames(const void* hidden, void* X, int N, int T, int D, int elem_bytes,
                         const int* row_utt, const int* row0, int M, int* status, cudaStream_t stream);

// Zero the stacked frames of utterances flagged non-finite (flag 2), before the backward pass.
cudaError_t zero_nonfinite_rows(void* X, int M, int D, int elem_bytes, const int* row_utt, const int* utt_flags,
                                int N, int* status, cudaStream_t stream);

// dH[n,t,:] = T(sum over slabs s < nslab, in ascending s, of acc[s*slab_stride + (row0[n]+t)*D + :]) for
// t < T_n, zero for padded frames.
// db[v0 + j] (+)= sum over the nblocks row blocks, in ascending order, of colpart[b * ld + j], j < cols.
cudaError_t colpart_sums(const float* colpart, long long ld, int nblocks, int cols, void* db, bool db_bf16,
                         long long v0, bool accumulate, cudaStream_t stream);

cudaError_t unstack_cast(const float* acc, int nslab, size_t slab_stride, void* dH, int N, int T, int D,
                         bool out_bf16, const int* T_n, const int* row0, int M, int* status, cudaStream_t stream);

// W_U[j,:] = W[U[j],:] for j < K (rows K.. of the [Kcap, D] buffer are zeroed).
cudaError_t gather_rows(const void* W, void* W_U, const int* U, const int* Kdev, int Kcap, int D,
                        int elem_bytes, long long V, int* status, cudaStream_t stream);

// db[v0 + j] = sum_i chunk[i*ld + j]
cudaError_t column_sums(const void* chunk, bool chunk_bf16, long long ld, int M, int cols,
                        void* db, bool db_bf16, long long v0, bool accumulate, cudaStream_t stream);

// ---------------------------------------------------------------------------
// Alignment dynamic program (Algorithm 1 lines 7-10; Section 3.3 for the beam)
// ---------------------------------------------------------------------------

struct DpBuffers {
  float* alpha;        // [cells]  forward scores, per-frame normalised
  float* beta;         // [cells]
  float* va;           // [cells]  best-alignment forward scores (beam only)
  float* vb;           // [cells]
  double* off_a;       // [M] per-frame offsets of va   (beam only)
  double* off_b;       // [M]
  double* best;        // [N] best alignment score (beam only)
  unsigned char* mask_f;      // [sum T_n * roundup4(L_n)] arc flags, forward sweep coordinates (beam only)
  unsigned char* mask_b;      // same, backward sweep coordinates
  const long long* mcell0;    // [N] first flag byte of each utterance
  float* roww;         // [M]
  const float* utt_weights;   // [N] upstream gradient of each utterance loss, or null (all 1)
  int* links;          // [N, target_stride] chains of label positions with equal labels (see k_repeat_links)
};

// Largest trellis width the DP kernels cover.
int dp_max_states();

cudaError_t alignment_dp(const float* S, long long ldS, const int* relabeled, int target_stride,
                         const BatchMeta& meta, int N, int M, int Lmax, float beam,
                         const DpBuffers& buf, float* gamma, long long ld_gamma, const int* Kdev,
                         float* loss, int* utt_flags, cudaStream_t stream);

// loss[n] += sum of lambda over the frames of utterance n (Eq. "ctc-factorization"): the DP ran on
// unnormalised selected logits.  Utterances already excluded keep loss 0; a non-finite result
// flags the utterance, zeroes its loss and its row weights.
cudaError_t finalize_loss(const float* lambda, const BatchMeta& meta, int N, float* loss, int* utt_flags,
                          float* roww, cudaStream_t stream);

}  // namespace pctc
