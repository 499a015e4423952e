// C ABI of libprunedctc: argument validation, workspace layout and the stream
// order of Algorithm 1.  All arithmetic happens in the kernels this file launches.
#include "../../include/prunedctc.h"
#include "pctc_internal.h"

#include <cmath>
#include <cstring>
#include <mutex>

namespace {

using namespace pctc;

constexpr size_t ALIGN = 256;
constexpr size_t DH_SPLIT_EXTRA_BYTES = 128u << 20;   // most that extra dX accumulators may take
inline size_t up(size_t x, size_t a = ALIGN) { return (x + a - 1) / a * a; }

struct Plan {
  int N, T, D, M, Usum, Kcap, Lmax, chunk, nsplit, nchunks;
  int ksplit, slab_rows;   // dX accumulator: k-split slabs of slab_rows rows each (1 slab of M rows without)
  long long V, cells, mcells;
  size_t ldS;
  int elem;          // bytes per element of hidden/W
  bool bf16, use_umma, beam;
  // byte offsets into the workspace
  size_t o_status, o_meta_i, o_cell0, o_bitmap, o_wrank, o_vmap, o_U, o_K, o_rel, o_flags, o_X, o_lambda,
      o_partial, o_WU, o_S, o_G, o_roww, o_links, o_alpha, o_beta, o_va, o_vb, o_offa, o_offb, o_best, o_maskf, o_maskb, o_mcell0, o_chunk, o_colpart, o_dHacc;
  size_t total;
  size_t meta_ints;  // T_n[N] | U_n[N] | row0[N+1] | row_utt[M]
};

// Default chunk width C.  Every chunk costs three launches whose length grows with M*C*D, so a
// narrow head (small D) is given wider chunks to keep each launch long against its start-up and tail;
// for wide heads 16,384 columns halve the per-chunk read-modify-write of the fp32 dX accumulator
// against 8,192 (about 2% of the step).  The [M, C] temporary is held under 512 MiB whatever the
// shape, so it never grows with V.
// Narrow heads: a chunk kernel is a handful of waves of the 74 CTA pairs of a B200, so a wave that is
// not full shows.  A width of k * 74 * 256 columns gives every chunk kernel whose units run over the
// column tiles (dlogits: row tiles x column tiles; dW: 512-row tiles of the chunk x column tiles of D)
// whole waves whatever the number of frames; k is the largest of 1..3 that the 512 MiB allow
// (measured: c2 4.23 -> 4.10 ms at 37,888 against 32,768; c3 4.53 -> 4.37 ms at 56,832).
int default_chunk(bool bf16, int D, long long M) {
  if (!bf16) return 4096;
  constexpr long long LIMIT = 512LL << 20;
  if (D <= 1024) {
    constexpr int WAVE_COLS = 74 * 256;                  // 148 SMs, planned for a full B200 wherever this runs
    for (int k = 3; k >= 1; --k)
      if (M * (long long)(k * WAVE_COLS) * 2 <= LIMIT) return k * WAVE_COLS;
  }
  int chunk = 16384;
  while (chunk > 8192 && M * chunk * 2 > LIMIT) chunk /= 2;
  return chunk;
}

pctc_status_t make_plan(const pctc_problem_t* p, const int32_t* Tn, const int32_t* Un, Plan* pl) {
  if (!p || !Tn || !Un) return PCTC_ERR_INVALID_ARG;
  if (p->N <= 0 || p->T <= 0 || p->D <= 0 || p->V <= 0 || p->target_stride < 0) return PCTC_ERR_INVALID_ARG;
  if (p->V > 0x7fffffffLL) return PCTC_ERR_UNSUPPORTED;
  if (p->blank_id < 0 || (long long)p->blank_id >= p->V) return PCTC_ERR_INVALID_ARG;
  if (p->dtype != PCTC_BF16 && p->dtype != PCTC_FP32) return PCTC_ERR_UNSUPPORTED;
  if (p->gemm_path != PCTC_GEMM_AUTO && p->gemm_path != PCTC_GEMM_SIMT) return PCTC_ERR_INVALID_ARG;
  if (p->chunk < 0) return PCTC_ERR_INVALID_ARG;
  if ((p->skip_dW | p->accumulate_dW | p->forward_only) & ~1) return PCTC_ERR_INVALID_ARG;
  if (p->max_K < 0) return PCTC_ERR_INVALID_ARG;
  if (std::isnan(p->beam)) return PCTC_ERR_INVALID_ARG;
  long long M = 0, Usum = 0, cells = 0, mcells = 0;
  int Umax = 0;
  for (int n = 0; n < p->N; ++n) {
    if (Tn[n] < 1 || Tn[n] > p->T) return PCTC_ERR_INVALID_ARG;
    if (Un[n] < 0 || Un[n] > p->target_stride) return PCTC_ERR_INVALID_ARG;
    M += Tn[n];
    Usum += Un[n];
    cells += (long long)Tn[n] * (2LL * Un[n] + 1);
    mcells += (long long)Tn[n] * ((2LL * Un[n] + 1 + 3) / 4 * 4);
    if (Un[n] > Umax) Umax = Un[n];
  }
  if (M > 0x7fffffffLL / 2 || Usum >= (1LL << 23) - 1) return PCTC_ERR_UNSUPPORTED;   // index in U packs into 23 bits
  pl->N = p->N; pl->T = p->T; pl->D = p->D; pl->V = p->V;
  pl->M = (int)M; pl->Usum = (int)Usum; pl->Kcap = (int)Usum + 1; pl->cells = cells; pl->mcells = mcells;
  if ((long long)pl->Kcap > p->V) pl->Kcap = (int)p->V;                 // K <= V always
  if (p->max_K > 0 && p->max_K < pl->Kcap) pl->Kcap = p->max_K;        // the caller's promise
  pl->Lmax = 2 * Umax + 1;
  if (pl->Lmax > dp_max_states()) return PCTC_ERR_UNSUPPORTED;
  pl->bf16 = (p->dtype == PCTC_BF16);
  pl->elem = pl->bf16 ? 2 : 4;
  pl->use_umma = pl->bf16 && p->gemm_path == PCTC_GEMM_AUTO && (p->D % 8 == 0);   // 16-byte rows for TMA
  pl->beam = (p->beam > 0.f) && std::isfinite(p->beam);
  int chunk = p->chunk > 0 ? p->chunk : default_chunk(pl->bf16, p->D, M);
  if (pl->use_umma) chunk = (chunk + 127) / 128 * 128;   // operand tiles of the tensor-core path
  if ((long long)chunk > p->V) chunk = (int)(pl->use_umma ? (p->V + 7) / 8 * 8 : p->V);
  pl->chunk = chunk;
  pl->nchunks = (int)((p->V + chunk - 1) / chunk);
  pl->nsplit = 64;            // capacity of the partial buffer; the launch may use fewer
  pl->ldS = up((size_t)pl->Kcap, 4);
  pl->meta_ints = (size_t)2 * pl->N + (pl->N + 1) + pl->M;

  const size_t nwords = (size_t)((p->V + 31) / 32);
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t r = o; o = up(o + bytes); return r; };
  pl->o_status = take(256);
  pl->o_meta_i = take(pl->meta_ints * 4);
  pl->o_cell0 = take((size_t)pl->N * 8);
  pl->o_bitmap = take(nwords * 4);
  pl->o_wrank = take(nwords * 4);
  pl->o_vmap = take((size_t)p->V * 4);
  pl->o_U = take((size_t)pl->Kcap * 4);
  pl->o_K = take(4);
  pl->o_rel = take((size_t)pl->N * (size_t)(p->target_stride > 0 ? p->target_stride : 1) * 4);
  pl->o_flags = take((size_t)pl->N * 4);
  pl->o_links = take((size_t)pl->N * (size_t)(p->target_stride > 0 ? p->target_stride : 1) * 4);
  pl->o_X = take((size_t)pl->M * pl->D * pl->elem);
  pl->o_lambda = take((size_t)pl->M * 4);
  pl->o_partial = take((size_t)pl->M * pl->nsplit * 8);
  pl->o_WU = take((size_t)pl->Kcap * pl->D * pl->elem);
  pl->o_S = take((size_t)pl->M * pl->ldS * 4);
  pl->o_G = take((size_t)pl->M * pl->ldS * 4);
  pl->o_roww = take((size_t)pl->M * 4);
  pl->o_alpha = take((size_t)cells * 4);
  pl->o_beta = take((size_t)cells * 4);
  pl->o_va = pl->o_vb = pl->o_offa = pl->o_offb = pl->o_best = pl->o_maskf = pl->o_maskb = pl->o_mcell0 = 0;
  if (pl->beam) {
    pl->o_va = take((size_t)cells * 4);
    pl->o_vb = take((size_t)cells * 4);
    pl->o_offa = take((size_t)pl->M * 8);
    pl->o_offb = take((size_t)pl->M * 8);
    pl->o_best = take((size_t)pl->N * 8);
    pl->o_maskf = take((size_t)mcells);
    pl->o_maskb = take((size_t)mcells);
    pl->o_mcell0 = take((size_t)pl->N * 8);
  }
  pl->o_chunk = take((size_t)pl->M * pl->chunk * pl->elem);
  // db_c on the tensor-core path: per block of 32 rows, the column sums the dlogits epilogue forms
  pl->o_colpart = pl->use_umma ? take((size_t)((pl->M + 31) / 32) * pl->chunk * 4) : 0;
  // few output tiles (small M x D): the dX contraction of a chunk is cut along k into ksplit ranges, each
  // with its own fp32 accumulator, summed in a fixed order when dH is written (deterministic)
  pl->ksplit = pl->use_umma ? umma_accum_splits(pl->M, pl->D, pl->chunk, DH_SPLIT_EXTRA_BYTES) : 1;
  pl->slab_rows = pl->ksplit > 1 ? umma_accum_slab_rows(pl->M) : pl->M;
  pl->o_dHacc = take((size_t)pl->ksplit * pl->slab_rows * pl->D * 4);
  pl->total = o;
  return PCTC_OK;
}

// Two auxiliary streams and a few events per device, created at the first call on that
// device and kept until exit.  Calls on one device are therefore not re-entrant across host threads.
struct Aux {
  cudaStream_t side = nullptr;          // alignment DP, beside the normaliser kernel
  cudaStream_t copy_out = nullptr;      // host entry point: rows of dW leave while later chunks compute
  cudaStream_t copy_in = nullptr;       // host entry point: W arrives in segments while the normaliser runs
  cudaEvent_t fork = nullptr, join = nullptr;
  cudaEvent_t chunk_done[2] = {nullptr, nullptr}, copies_done = nullptr;
  cudaEvent_t w_ready[4] = {nullptr, nullptr, nullptr, nullptr}, entry = nullptr;
};

// Set by the host-buffer entry point: where finished rows of dW go.
struct HostPipe {
  char* dW_host = nullptr;
  // W arrives in `nseg` row segments of `seg_rows` rows (the last one shorter); w_ready[s] is
  // recorded on the copy stream behind segment s.  nseg == 0: W is already on the device.
  int nseg = 0;
  long long seg_rows = 0;
  cudaEvent_t w_ready[4] = {nullptr, nullptr, nullptr, nullptr};
};
cudaError_t get_aux(Aux* out) {
  static std::mutex mu;
  static Aux table[64];
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(mu);
  Aux& a = table[dev];
  if (!a.side) {
    if ((e = cudaStreamCreateWithFlags(&a.side, cudaStreamNonBlocking)) != cudaSuccess) return e;
    if ((e = cudaStreamCreateWithFlags(&a.copy_out, cudaStreamNonBlocking)) != cudaSuccess) return e;
    if ((e = cudaStreamCreateWithFlags(&a.copy_in, cudaStreamNonBlocking)) != cudaSuccess) return e;
    cudaEvent_t* evs[] = {&a.fork,       &a.join,       &a.chunk_done[0], &a.chunk_done[1], &a.copies_done,
                          &a.w_ready[0], &a.w_ready[1], &a.w_ready[2],    &a.w_ready[3],    &a.entry};
    for (cudaEvent_t* ev : evs)
      if ((e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming)) != cudaSuccess) return e;
  }
  *out = a;
  return cudaSuccess;
}

struct GemmCall {
  const void* A; long long lda; bool a_mn;
  const void* B; long long ldb; bool b_mn;
  int m, n, k;
};

cudaError_t run_gemm(bool use_umma, bool bf16, const GemmCall& c, const Epilogue& e_in, int* status,
                     cudaStream_t stream) {
  if (c.m <= 0 || c.n <= 0) return cudaSuccess;
  Epilogue e = e_in;
  e.status = status;
  if (use_umma)
    return umma_gemm((const __nv_bfloat16*)c.A, c.lda, c.a_mn, (const __nv_bfloat16*)c.B, c.ldb, c.b_mn,
                     c.m, c.n, c.k, e, status, stream);
  GemmShape g;
  g.m = c.m; g.n = c.n; g.k = c.k;
  g.a_i = c.a_mn ? 1 : c.lda; g.a_k = c.a_mn ? c.lda : 1;
  g.b_j = c.b_mn ? 1 : c.ldb; g.b_k = c.b_mn ? c.ldb : 1;
  return simt_gemm(c.A, c.B, bf16, g, e, stream);
}

}  // namespace

extern "C" {

const char* pctc_status_string(pctc_status_t s) {
  switch (s) {
    case PCTC_OK: return "ok";
    case PCTC_ERR_INVALID_ARG: return "invalid argument";
    case PCTC_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case PCTC_ERR_UNSUPPORTED: return "unsupported dtype or shape";
    case PCTC_ERR_CUDA: return "CUDA error";
    case PCTC_ERR_BAD_TARGET: return "bad target";
    case PCTC_ERR_TIMEOUT: return "bounded device wait gave up";
  }
  return "unknown status";
}

pctc_status_t pctc_workspace_bytes(const pctc_problem_t* problem, const int32_t* input_lengths_host,
                                   const int32_t* target_lengths_host, size_t* bytes_out) {
  if (!bytes_out) return PCTC_ERR_INVALID_ARG;
  Plan pl;
  pctc_status_t st = make_plan(problem, input_lengths_host, target_lengths_host, &pl);
  if (st != PCTC_OK) return st;
  *bytes_out = pl.total;
  return PCTC_OK;
}

pctc_status_t pctc_chunk_width(const pctc_problem_t* problem, const int32_t* input_lengths_host,
                               const int32_t* target_lengths_host, int32_t* chunk_out, int32_t* nchunks_out) {
  if (!chunk_out) return PCTC_ERR_INVALID_ARG;
  Plan pl;
  pctc_status_t st = make_plan(problem, input_lengths_host, target_lengths_host, &pl);
  if (st != PCTC_OK) return st;
  *chunk_out = pl.chunk;
  if (nchunks_out) *nchunks_out = pl.nchunks;
  return PCTC_OK;
}

pctc_status_t pctc_workspace_status(const void* workspace, void* stream, int32_t* status_host) {
  if (!workspace || !status_host) return PCTC_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  if (cudaMemcpyAsync(status_host, workspace, 4, cudaMemcpyDeviceToHost, s) != cudaSuccess) return PCTC_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return PCTC_ERR_CUDA;
  if (*status_host == 0) return PCTC_OK;
  return *status_host < 0x100 ? PCTC_ERR_TIMEOUT : PCTC_ERR_INVALID_ARG;
}

pctc_status_t pctc_gemm_bf16(const void* A, const void* B, float* C, int32_t m, int32_t n, int32_t k,
                             int32_t a_mn_major, int32_t b_mn_major, int32_t gemm_path,
                             int32_t* device_status, void* stream) {
  if (!A || !B || !C || m <= 0 || n <= 0 || k <= 0) return PCTC_ERR_INVALID_ARG;
  if (gemm_path != PCTC_GEMM_AUTO && gemm_path != PCTC_GEMM_SIMT) return PCTC_ERR_INVALID_ARG;
  const long long lda = a_mn_major ? m : k, ldb = b_mn_major ? n : k;
  const bool umma = gemm_path == PCTC_GEMM_AUTO;
  if (umma && ((lda % 8) || (ldb % 8) || ((size_t)A & 15) || ((size_t)B & 15))) return PCTC_ERR_UNSUPPORTED;
  if (umma && !umma_available()) return PCTC_ERR_CUDA;
  Epilogue e;
  e.kind = EPI_STORE_F32;
  e.out = C;
  e.ld = n;
  GemmCall c{A, lda, a_mn_major != 0, B, ldb, b_mn_major != 0, m, n, k};
  cudaError_t err = run_gemm(umma, true, c, e, device_status, (cudaStream_t)stream);
  return err == cudaSuccess ? PCTC_OK : PCTC_ERR_CUDA;
}

pctc_status_t pruned_ctc_fwd_bwd(const pctc_problem_t* p, const void* hidden, const void* W, const void* bias,
                                 const int32_t* targets, const int32_t* input_lengths,
                                 const int32_t* target_lengths, float* loss, void* dH, void* dW, void* dbias,
                                 int32_t* subset_out, int32_t* K_out, int32_t* relabeled_out,
                                 int32_t* utt_flags, void* workspace, size_t workspace_bytes, void* stream_v) {
  return pruned_ctc_fwd_bwd_traced(p, hidden, W, bias, targets, input_lengths, target_lengths, loss, dH, dW, dbias,
                                   subset_out, K_out, relabeled_out, utt_flags, workspace, workspace_bytes,
                                   stream_v, nullptr);
}

}  // extern "C"

namespace {
// A call forks onto the library's own auxiliary streams and records its events there; none of that
// has been arranged for stream capture, so a capturing stream is refused before anything is enqueued.
bool stream_is_capturing(cudaStream_t stream) {
  cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
  return cudaStreamIsCapturing(stream, &cs) == cudaSuccess && cs != cudaStreamCaptureStatusNone;
}

// The whole call.  `pipe` is non-null only for the host-buffer entry point.
pctc_status_t run_call(const pctc_problem_t* p, const void* hidden, const void* W, const void* bias,
                       const int32_t* targets, const int32_t* input_lengths, const int32_t* target_lengths,
                       float* loss, void* dH, void* dW, void* dbias, int32_t* subset_out, int32_t* K_out,
                       int32_t* relabeled_out, int32_t* utt_flags, void* workspace, size_t workspace_bytes,
                       void* stream_v, pctc_trace_t* trace, const HostPipe* pipe) {
  Plan pl;
  pctc_status_t st = make_plan(p, input_lengths, target_lengths, &pl);
  if (st != PCTC_OK) return st;
  if (trace) {
    if (!trace->events || !trace->kinds || trace->capacity < 12 + 4 * pl.nchunks) return PCTC_ERR_INVALID_ARG;
    trace->used = 0;
  }
  if (!hidden || !W || !loss || !workspace) return PCTC_ERR_INVALID_ARG;
  if (!p->forward_only && (!dH || (!dW && !p->skip_dW))) return PCTC_ERR_INVALID_ARG;
  if (!targets && pl.Usum > 0) return PCTC_ERR_INVALID_ARG;
  if (workspace_bytes < pl.total) return PCTC_ERR_WORKSPACE_TOO_SMALL;
  if (((size_t)workspace & (ALIGN - 1)) || ((size_t)hidden & 15) || ((size_t)W & 15) || ((size_t)dH & 15) ||
      ((size_t)dW & 15))
    return PCTC_ERR_INVALID_ARG;   // (null dH / dW are aligned)
  if (pl.use_umma && !umma_available()) return PCTC_ERR_CUDA;
  cudaStream_t stream = (cudaStream_t)stream_v;
  if (stream_is_capturing(stream)) return PCTC_ERR_UNSUPPORTED;
  Aux aux;
  if (get_aux(&aux) != cudaSuccess) return PCTC_ERR_CUDA;
  char* ws = (char*)workspace;
  const int N = pl.N, M = pl.M, D = pl.D;
  const long long V = pl.V;

#define PCTC_CUDA(call)                          \
  do {                                           \
    if ((call) != cudaSuccess) return PCTC_ERR_CUDA; \
  } while (0)
  // start of a span of phase `kind` (kind < 0: end of the timeline)
#define PCTC_MARK(kind)                                                                              \
  do {                                                                                               \
    if (trace) {                                                                                     \
      PCTC_CUDA(cudaEventRecord((cudaEvent_t)trace->events[trace->used], stream));                   \
      trace->kinds[trace->used] = (kind);                                                            \
      ++trace->used;                                                                                 \
    }                                                                                                \
  } while (0)

  PCTC_MARK(PCTC_PHASE_PREP);
  // ---- batch description: lengths, first stacked row, first trellis cell, row -> utterance ----
  // (built on the device from the lengths, which travel as kernel parameters: no copy from
  // pageable host memory, no wait for the stream)
  int* d_meta = (int*)(ws + pl.o_meta_i);
  long long* d_cell0 = (long long*)(ws + pl.o_cell0);
  PCTC_CUDA(batch_meta(input_lengths, target_lengths, N, d_meta, d_meta + N, d_meta + 2 * N, d_cell0,
                       pl.beam ? (long long*)(ws + pl.o_mcell0) : nullptr, d_meta + 3 * N + 1, stream));
  PCTC_CUDA(cudaMemsetAsync(ws + pl.o_status, 0, 256, stream));
  BatchMeta bm;
  bm.T_n = d_meta;
  bm.U_n = d_meta + N;
  bm.row0 = d_meta + 2 * N;
  bm.row_utt = d_meta + 3 * N + 1;
  bm.cell0 = d_cell0;
  bm.N = N;
  bm.M = M;
  bm.status = (int*)(ws + pl.o_status);

  int* d_status = (int*)(ws + pl.o_status);
  unsigned* d_bitmap = (unsigned*)(ws + pl.o_bitmap);
  int* d_wrank = (int*)(ws + pl.o_wrank);
  int* d_vmap = (int*)(ws + pl.o_vmap);
  int* d_U = (int*)(ws + pl.o_U);
  int* d_K = (int*)(ws + pl.o_K);
  int* d_rel = (int*)(ws + pl.o_rel);
  int* d_flags = (int*)(ws + pl.o_flags);
  void* d_X = ws + pl.o_X;
  float* d_lambda = (float*)(ws + pl.o_lambda);
  float2* d_partial = (float2*)(ws + pl.o_partial);
  void* d_WU = ws + pl.o_WU;
  float* d_S = (float*)(ws + pl.o_S);
  float* d_G = (float*)(ws + pl.o_G);
  void* d_chunk = ws + pl.o_chunk;
  float* d_dHacc = (float*)(ws + pl.o_dHacc);
  DpBuffers dp{};
  dp.alpha = (float*)(ws + pl.o_alpha);
  dp.beta = (float*)(ws + pl.o_beta);
  dp.roww = (float*)(ws + pl.o_roww);
  dp.utt_weights = p->utt_weights;
  dp.links = (int*)(ws + pl.o_links);
  if (pl.beam) {
    dp.va = (float*)(ws + pl.o_va);
    dp.vb = (float*)(ws + pl.o_vb);
    dp.off_a = (double*)(ws + pl.o_offa);
    dp.off_b = (double*)(ws + pl.o_offb);
    dp.best = (double*)(ws + pl.o_best);
    dp.mask_f = (unsigned char*)(ws + pl.o_maskf);
    dp.mask_b = (unsigned char*)(ws + pl.o_maskb);
    dp.mcell0 = (const long long*)(ws + pl.o_mcell0);
  }

  // ---- Algorithm 1 lines 2-3: subset and relabelling ----
  PCTC_CUDA(cudaMemsetAsync(d_U, 0xFF, (size_t)pl.Kcap * 4, stream));   // entries past K read -1
  PCTC_CUDA(subset_and_relabel(targets, p->target_stride, bm.U_n, N, V, p->blank_id, d_bitmap, d_wrank, d_vmap,
                               d_U, d_K, d_rel, d_flags, pl.Kcap, d_status, stream));
  // ---- line 4: stack the valid frames ----
  PCTC_CUDA(stack_frames(hidden, d_X, N, pl.T, D, pl.elem, bm.row_utt, bm.row0, M, d_status, stream));

  // ---- line 6: logits of the selected classes, Z_U = X W_U^T + b_U; lines 7-10: the DP ----
  // The alignment sum of Eq. "ctc-factorization" needs no normaliser, so the DP runs on Z_U (on the
  // auxiliary stream) while the full-vocabulary normaliser is still being computed; lambda enters
  // the loss at the end.
  auto subset_logits_and_dp = [&]() -> pctc_status_t {
    PCTC_MARK(PCTC_PHASE_SUBSET_LOGP);
    {
      PCTC_CUDA(gather_rows(W, d_WU, d_U, d_K, pl.Kcap, D, pl.elem, V, d_status, stream));
      Epilogue e;
      e.kind = EPI_SUBSET_LOGP;
      e.vocab = V;
      e.out = d_S;
      e.ld = (long long)pl.ldS;
      e.lambda = nullptr;
      e.bias = bias;
      e.U = d_U;
      e.Kdev = d_K;
      GemmCall c{d_X, D, false, d_WU, D, false, M, pl.Kcap, D};
      PCTC_CUDA(run_gemm(pl.use_umma, pl.bf16, c, e, d_status, stream));
    }
    PCTC_MARK(-2);
    PCTC_CUDA(cudaEventRecord(aux.fork, stream));
    PCTC_CUDA(cudaStreamWaitEvent(aux.side, aux.fork, 0));
    {
      cudaStream_t main_stream = stream;
      stream = aux.side;
      PCTC_MARK(PCTC_PHASE_DP);
      PCTC_CUDA(alignment_dp(d_S, (long long)pl.ldS, d_rel, p->target_stride, bm, N, M, pl.Lmax,
                             pl.beam ? p->beam : 0.f, dp, d_G, (long long)pl.ldS, d_K, loss, d_flags, stream));
      PCTC_MARK(-2);
      stream = main_stream;
    }
    PCTC_CUDA(cudaEventRecord(aux.join, aux.side));
    return PCTC_OK;
  };

  // ---- line 5: normaliser, online over the vocabulary ----
  // One launch over all of W; or, when W is still arriving from the host in row segments, one
  // launch per segment as it lands, each writing its own split slots of the partial buffer.
  auto normaliser = [&]() -> pctc_status_t {
    PCTC_MARK(PCTC_PHASE_LSE);
    const int pps = pl.use_umma ? umma_lse_partials_per_split(D) : 1;
    const int nseg = (pipe && pipe->nseg > 0) ? pipe->nseg : 1;
    const long long seg_rows = nseg > 1 ? pipe->seg_rows : V;
    int per_seg = pl.use_umma ? umma_lse_splits(M, (int)(seg_rows < V ? seg_rows : V)) : 32;
    if (per_seg * nseg * pps > 64) per_seg = 64 / (nseg * pps);
    int slots = 0;
    for (int sg = 0; sg < nseg; ++sg) {
      const long long v0 = (long long)sg * seg_rows;
      if (v0 >= V) break;
      const long long rows = (V - v0 < seg_rows) ? (V - v0) : seg_rows;
      if (nseg > 1) PCTC_CUDA(cudaStreamWaitEvent(stream, pipe->w_ready[sg], 0));
      Epilogue e;
      e.kind = EPI_LSE_PARTIAL;
      e.bias = bias;
      e.v0 = v0;
      e.partial = d_partial;
      e.nsplit = per_seg;
      if (pl.use_umma) {                       // never more splits than column tiles of the segment
        const int tiles = (int)((rows + 255) / 256);
        if (e.nsplit > tiles) e.nsplit = tiles;
      }
      e.partial_stride = per_seg * nseg;
      e.partial_offset = slots;
      GemmCall c{d_X, D, false, (const char*)W + (size_t)v0 * D * pl.elem, D, false, M, (int)rows, D};
      PCTC_CUDA(run_gemm(pl.use_umma, pl.bf16, c, e, d_status, stream));
      slots += e.nsplit;
    }
    // unused slots of the stride hold (-inf, 0) so that the combine may read the full stride
    PCTC_CUDA(lse_combine(d_partial, per_seg * nseg * pps, M, d_lambda, stream));
    return PCTC_OK;
  };

  if (pipe && pipe->nseg > 1) {
    // W is still in flight: start with what can run on its first rows, do the DP once it is complete
    PCTC_CUDA(cudaMemsetAsync(d_partial, 0, (size_t)M * 64 * 8, stream));   // (0, 0): empty slots are skipped
    if ((st = normaliser()) != PCTC_OK) return st;
    if ((st = subset_logits_and_dp()) != PCTC_OK) return st;
  } else {
    if ((st = subset_logits_and_dp()) != PCTC_OK) return st;
    if ((st = normaliser()) != PCTC_OK) return st;
  }
  PCTC_CUDA(cudaStreamWaitEvent(stream, aux.join, 0));
  PCTC_CUDA(finalize_loss(d_lambda, bm, N, loss, d_flags, dp.roww, stream));
  if (!p->forward_only) PCTC_CUDA(zero_nonfinite_rows(d_X, M, D, pl.elem, bm.row_utt, d_flags, N, d_status, stream));

  // ---- lines 11-17: backward, one vocabulary chunk at a time ----
  int dh_slabs = 1;                  // dX accumulator slabs in use (k-split of the dX contraction)
  for (int ci = 0; ci < pl.nchunks && !p->forward_only; ++ci) {
    const long long v0 = (long long)ci * pl.chunk;
    const int Cc = (int)((V - v0 < pl.chunk) ? (V - v0) : pl.chunk);
    const char* Wc = (const char*)W + (size_t)v0 * D * pl.elem;
    PCTC_MARK(PCTC_PHASE_DLOGITS);
    {
      Epilogue e;                      // recompute Z_c and form Eq. "vjp"
      e.kind = EPI_DLOGITS;
      e.vocab = V;
      e.out = d_chunk;
      e.ld = pl.chunk;
      e.out_is_bf16 = pl.bf16;
      e.lambda = d_lambda;
      e.bias = bias;
      e.v0 = v0;
      e.vmap = d_vmap;
      e.gamma = d_G;
      e.ld_gamma = (long long)pl.ldS;
      e.roww = dp.roww;
      if (pl.use_umma && bias && dbias) {
        e.colpart = (float*)(ws + pl.o_colpart);
        e.ld_colpart = pl.chunk;
      }
      GemmCall c{d_X, D, false, Wc, D, false, M, Cc, D};
      PCTC_CUDA(run_gemm(pl.use_umma, pl.bf16, c, e, d_status, stream));
    }
    PCTC_MARK(PCTC_PHASE_DH);
    {
      Epilogue e;                      // dX += dZ_c W_c
      e.kind = EPI_ACCUM_F32;
      e.out = d_dHacc;
      e.ld = D;
      e.accumulate = ci > 0;
      if (pl.ksplit > 1) {
        // the first chunk stores into (and so initialises) its slabs; a shorter chunk later on may
        // cut k into fewer ranges and then adds to the first slabs only
        int s = umma_accum_splits(M, D, Cc, DH_SPLIT_EXTRA_BYTES);
        if (s > pl.ksplit) s = pl.ksplit;
        if (ci == 0) dh_slabs = s;
        e.ksplit = s < dh_slabs ? s : dh_slabs;
        e.ksplit_rows = pl.slab_rows;
      }
      GemmCall c{d_chunk, pl.chunk, false, Wc, D, true, M, D, Cc};
      PCTC_CUDA(run_gemm(pl.use_umma, pl.bf16, c, e, d_status, stream));
    }
    PCTC_MARK(PCTC_PHASE_DW);
    if (!p->skip_dW) {
      Epilogue e;                      // rows of dW: dZ_c^T X
      e.kind = EPI_STORE_OUT;
      e.out = (char*)dW + (size_t)v0 * D * pl.elem;
      e.ld = D;
      e.out_is_bf16 = pl.bf16;
      e.accumulate = p->accumulate_dW;
      GemmCall c{d_chunk, pl.chunk, true, d_X, D, true, Cc, D, M};
      PCTC_CUDA(run_gemm(pl.use_umma, pl.bf16, c, e, d_status, stream));
    }
    if (bias && dbias) {
      PCTC_MARK(PCTC_PHASE_DBIAS);
      if (pl.use_umma)
        PCTC_CUDA(colpart_sums((const float*)(ws + pl.o_colpart), pl.chunk, (M + 31) / 32, Cc, dbias, pl.bf16, v0,
                               p->accumulate_dW != 0, stream));
      else
        PCTC_CUDA(column_sums(d_chunk, pl.bf16, pl.chunk, M, Cc, dbias, pl.bf16, v0, p->accumulate_dW != 0, stream));
    }
    if (pipe && pipe->dW_host && !p->skip_dW) {          // these rows of dW are final: send them home now
      cudaEvent_t ev = aux.chunk_done[ci & 1];
      PCTC_CUDA(cudaEventRecord(ev, stream));
      PCTC_CUDA(cudaStreamWaitEvent(aux.copy_out, ev, 0));
      PCTC_CUDA(cudaMemcpyAsync(pipe->dW_host + (size_t)v0 * D * pl.elem, (const char*)dW + (size_t)v0 * D * pl.elem,
                                (size_t)Cc * D * pl.elem, cudaMemcpyDeviceToHost, aux.copy_out));
    }
  }
  if (pipe && pipe->dW_host && !p->skip_dW && !p->forward_only) {   // the caller's stream covers those copies
    PCTC_CUDA(cudaEventRecord(aux.copies_done, aux.copy_out));
    PCTC_CUDA(cudaStreamWaitEvent(stream, aux.copies_done, 0));
  }
  PCTC_MARK(PCTC_PHASE_FINISH);
  if (!p->forward_only)
    PCTC_CUDA(unstack_cast(d_dHacc, dh_slabs, (size_t)pl.slab_rows * D, dH, N, pl.T, D, pl.bf16, bm.T_n, bm.row0, M,
                           d_status, stream));

  // ---- optional integer outputs ----
  if (subset_out)
    PCTC_CUDA(cudaMemcpyAsync(subset_out, d_U, (size_t)pl.Kcap * 4, cudaMemcpyDeviceToDevice, stream));
  if (K_out) PCTC_CUDA(cudaMemcpyAsync(K_out, d_K, 4, cudaMemcpyDeviceToDevice, stream));
  if (relabeled_out && p->target_stride > 0)
    PCTC_CUDA(cudaMemcpyAsync(relabeled_out, d_rel, (size_t)N * p->target_stride * 4, cudaMemcpyDeviceToDevice,
                              stream));
  if (utt_flags) PCTC_CUDA(cudaMemcpyAsync(utt_flags, d_flags, (size_t)N * 4, cudaMemcpyDeviceToDevice, stream));
  PCTC_MARK(-1);
#undef PCTC_MARK
#undef PCTC_CUDA
  return PCTC_OK;
}
}  // namespace

extern "C" {

pctc_status_t pruned_ctc_fwd_bwd_traced(const pctc_problem_t* p, const void* hidden, const void* W,
                                        const void* bias, const int32_t* targets, const int32_t* input_lengths,
                                        const int32_t* target_lengths, float* loss, void* dH, void* dW,
                                        void* dbias, int32_t* subset_out, int32_t* K_out,
                                        int32_t* relabeled_out, int32_t* utt_flags, void* workspace,
                                        size_t workspace_bytes, void* stream_v, pctc_trace_t* trace) {
  return run_call(p, hidden, W, bias, targets, input_lengths, target_lengths, loss, dH, dW, dbias, subset_out, K_out,
                  relabeled_out, utt_flags, workspace, workspace_bytes, stream_v, trace, nullptr);
}

namespace {
struct GreedyPlan {
  int N, T, D, M, elem, nsplit;
  long long V;
  bool bf16, use_umma;
  size_t o_status, o_meta, o_X, o_partial, o_labels, total, meta_ints;
};
pctc_status_t greedy_plan(const pctc_problem_t* p, const int32_t* Tn, GreedyPlan* g) {
  if (!p || !Tn) return PCTC_ERR_INVALID_ARG;
  if (p->N <= 0 || p->T <= 0 || p->D <= 0 || p->V <= 0) return PCTC_ERR_INVALID_ARG;
  if (p->V > 0x7fffffffLL) return PCTC_ERR_UNSUPPORTED;
  if (p->blank_id < 0 || (long long)p->blank_id >= p->V) return PCTC_ERR_INVALID_ARG;
  if (p->dtype != PCTC_BF16 && p->dtype != PCTC_FP32) return PCTC_ERR_UNSUPPORTED;
  if (p->gemm_path != PCTC_GEMM_AUTO && p->gemm_path != PCTC_GEMM_SIMT) return PCTC_ERR_INVALID_ARG;
  long long M = 0;
  for (int n = 0; n < p->N; ++n) {
    if (Tn[n] < 1 || Tn[n] > p->T) return PCTC_ERR_INVALID_ARG;
    M += Tn[n];
  }
  if (M > 0x3fffffffLL) return PCTC_ERR_UNSUPPORTED;
  g->N = p->N; g->T = p->T; g->D = p->D; g->V = p->V; g->M = (int)M;
  g->bf16 = p->dtype == PCTC_BF16;
  g->elem = g->bf16 ? 2 : 4;
  g->use_umma = g->bf16 && p->gemm_path == PCTC_GEMM_AUTO && (p->D % 8 == 0);
  g->meta_ints = (size_t)g->N + (g->N + 1) + g->M;      // T_n | row0 | row_utt
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t r = o; o = up(o + bytes); return r; };
  g->o_status = take(256);
  g->o_meta = take(g->meta_ints * 4);
  g->o_X = take((size_t)g->M * g->D * g->elem);
  g->o_partial = take((size_t)g->M * 64 * 8);
  g->o_labels = take((size_t)g->M * 4);
  g->total = o;
  return PCTC_OK;
}

struct HostLayout {
  size_t o_hidden, o_W, o_bias, o_targets, o_loss, o_dH, o_dW, o_dbias, o_subset, o_K, o_rel, o_flags, o_ws;
  size_t b_hidden, b_W, b_bias, b_targets, b_rel, b_subset, ws_bytes, total;
};
// The host-buffer call sends the rows of dW home chunk by chunk, and that copy (PCIe) takes about as
// long as the backward pass itself: what is exposed is the first chunk, which must be finished before
// any row can leave.  So without a chunk width from the caller it uses at most 8,192 columns.
pctc_problem_t host_problem(const pctc_problem_t* p) {
  pctc_problem_t hp = *p;
  if (hp.chunk == 0 && hp.dtype == PCTC_BF16) hp.chunk = 8192;
  return hp;
}

pctc_status_t host_layout(const pctc_problem_t* p_in, const int32_t* Tn, const int32_t* Un, bool has_bias,
                          HostLayout* h) {
  if (!p_in) return PCTC_ERR_INVALID_ARG;
  const pctc_problem_t hp = host_problem(p_in);
  const pctc_problem_t* p = &hp;
  Plan pl;
  pctc_status_t st = make_plan(p, Tn, Un, &pl);
  if (st != PCTC_OK) return st;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t r = o; o = up(o + bytes); return r; };
  h->b_hidden = (size_t)pl.N * pl.T * pl.D * pl.elem;
  h->b_W = (size_t)pl.V * pl.D * pl.elem;
  h->b_bias = has_bias ? (size_t)pl.V * pl.elem : 0;
  h->b_targets = (size_t)pl.N * p->target_stride * 4;
  h->b_rel = h->b_targets;
  h->b_subset = (size_t)pl.Kcap * 4;
  h->o_hidden = take(h->b_hidden);
  h->o_W = take(h->b_W);
  h->o_bias = take(h->b_bias);
  h->o_targets = take(h->b_targets);
  h->o_loss = take((size_t)pl.N * 4);
  h->o_dH = take(h->b_hidden);
  h->o_dW = take(h->b_W);
  h->o_dbias = take(h->b_bias);
  h->o_subset = take(h->b_subset);
  h->o_K = take(4);
  h->o_rel = take(h->b_rel);
  h->o_flags = take((size_t)pl.N * 4);
  h->o_ws = take(pl.total);
  h->ws_bytes = pl.total;
  h->total = o;
  return PCTC_OK;
}
}  // namespace

pctc_status_t pctc_host_call_scratch_bytes(const pctc_problem_t* problem, const int32_t* input_lengths_host,
                                           const int32_t* target_lengths_host, int32_t has_bias,
                                           size_t* bytes_out) {
  if (!bytes_out) return PCTC_ERR_INVALID_ARG;
  HostLayout h;
  pctc_status_t st = host_layout(problem, input_lengths_host, target_lengths_host, has_bias != 0, &h);
  if (st != PCTC_OK) return st;
  *bytes_out = h.total;
  return PCTC_OK;
}

pctc_status_t pruned_ctc_fwd_bwd_host(const pctc_problem_t* p, const void* hidden, const void* W, const void* bias,
                                      const int32_t* targets, const int32_t* input_lengths,
                                      const int32_t* target_lengths, float* loss, void* dH, void* dW, void* dbias,
                                      int32_t* subset_out, int32_t* K_out, int32_t* relabeled_out,
                                      int32_t* utt_flags, void* device_scratch, size_t scratch_bytes,
                                      void* stream_v) {
  HostLayout h;
  pctc_status_t st = host_layout(p, input_lengths, target_lengths, bias != nullptr, &h);
  if (st != PCTC_OK) return st;
  if (!hidden || !W || !loss || !dH || !dW || !device_scratch) return PCTC_ERR_INVALID_ARG;
  if (p->skip_dW || p->accumulate_dW || p->utt_weights || p->forward_only) return PCTC_ERR_UNSUPPORTED;   // device entry point only
  if (!targets && h.b_targets > 0) return PCTC_ERR_INVALID_ARG;
  if ((size_t)device_scratch & (ALIGN - 1)) return PCTC_ERR_INVALID_ARG;
  if (scratch_bytes < h.total) return PCTC_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t stream = (cudaStream_t)stream_v;
  if (stream_is_capturing(stream)) return PCTC_ERR_UNSUPPORTED;
  char* d = (char*)device_scratch;
  const bool want_db = bias && dbias;
#define PCTC_CUDA(call)                              \
  do {                                               \
    if ((call) != cudaSuccess) return PCTC_ERR_CUDA; \
  } while (0)
  Aux aux;
  if (get_aux(&aux) != cudaSuccess) return PCTC_ERR_CUDA;
  HostPipe pipe;
  pipe.dW_host = (char*)dW;       // rows of dW are copied out chunk by chunk while the backward pass runs
  // The small inputs go first on the caller's stream; W follows on a copy stream in four row
  // segments, and the normaliser kernel of each segment starts as soon as that segment has landed.
  const int elem = (p->dtype == PCTC_BF16) ? 2 : 4;
  const size_t row_bytes = (size_t)p->D * elem;
  pipe.nseg = (p->V >= 4 * 4096) ? 4 : 0;
  pipe.seg_rows = ((p->V + 3) / 4 + 255) / 256 * 256;
  PCTC_CUDA(cudaMemcpyAsync(d + h.o_hidden, hidden, h.b_hidden, cudaMemcpyHostToDevice, stream));
  if (bias) PCTC_CUDA(cudaMemcpyAsync(d + h.o_bias, bias, h.b_bias, cudaMemcpyHostToDevice, stream));
  if (h.b_targets) PCTC_CUDA(cudaMemcpyAsync(d + h.o_targets, targets, h.b_targets, cudaMemcpyHostToDevice, stream));
  if (pipe.nseg > 1) {
    PCTC_CUDA(cudaEventRecord(aux.entry, stream));          // the staging area is free once earlier work is done
    PCTC_CUDA(cudaStreamWaitEvent(aux.copy_in, aux.entry, 0));
    for (int sg = 0; sg < pipe.nseg; ++sg) {
      const long long v0 = (long long)sg * pipe.seg_rows;
      if (v0 >= p->V) { pipe.nseg = sg; break; }
      const long long rows = (p->V - v0 < pipe.seg_rows) ? (p->V - v0) : pipe.seg_rows;
      PCTC_CUDA(cudaMemcpyAsync(d + h.o_W + (size_t)v0 * row_bytes, (const char*)W + (size_t)v0 * row_bytes,
                                (size_t)rows * row_bytes, cudaMemcpyHostToDevice, aux.copy_in));
      pipe.w_ready[sg] = aux.w_ready[sg];
      PCTC_CUDA(cudaEventRecord(aux.w_ready[sg], aux.copy_in));
    }
  } else {
    PCTC_CUDA(cudaMemcpyAsync(d + h.o_W, W, h.b_W, cudaMemcpyHostToDevice, stream));
  }
  const pctc_problem_t hp = host_problem(p);
  st = run_call(&hp, d + h.o_hidden, d + h.o_W, bias ? d + h.o_bias : nullptr, (const int32_t*)(d + h.o_targets),
                input_lengths, target_lengths, (float*)(d + h.o_loss), d + h.o_dH, d + h.o_dW,
                want_db ? d + h.o_dbias : nullptr, (int32_t*)(d + h.o_subset), (int32_t*)(d + h.o_K),
                (int32_t*)(d + h.o_rel), (int32_t*)(d + h.o_flags), d + h.o_ws, h.ws_bytes, stream_v, nullptr, &pipe);
  if (st != PCTC_OK) return st;
  PCTC_CUDA(cudaMemcpyAsync(loss, d + h.o_loss, (size_t)p->N * 4, cudaMemcpyDeviceToHost, stream));
  PCTC_CUDA(cudaMemcpyAsync(dH, d + h.o_dH, h.b_hidden, cudaMemcpyDeviceToHost, stream));
  if (want_db) PCTC_CUDA(cudaMemcpyAsync(dbias, d + h.o_dbias, h.b_bias, cudaMemcpyDeviceToHost, stream));
  if (subset_out) PCTC_CUDA(cudaMemcpyAsync(subset_out, d + h.o_subset, h.b_subset, cudaMemcpyDeviceToHost, stream));
  if (K_out) PCTC_CUDA(cudaMemcpyAsync(K_out, d + h.o_K, 4, cudaMemcpyDeviceToHost, stream));
  if (relabeled_out && h.b_rel)
    PCTC_CUDA(cudaMemcpyAsync(relabeled_out, d + h.o_rel, h.b_rel, cudaMemcpyDeviceToHost, stream));
  if (utt_flags) PCTC_CUDA(cudaMemcpyAsync(utt_flags, d + h.o_flags, (size_t)p->N * 4, cudaMemcpyDeviceToHost, stream));
#undef PCTC_CUDA
  return PCTC_OK;
}

namespace {
struct TopkPlan {
  GreedyPlan g;
  int k, chunk;
  size_t o_logits, o_val, o_idx, o_ms, total;
};
pctc_status_t topk_plan(const pctc_problem_t* p, const int32_t* Tn, int32_t k, TopkPlan* t) {
  pctc_status_t st = greedy_plan(p, Tn, &t->g);
  if (st != PCTC_OK) return st;
  if (k != 1 && k != 2 && k != 4 && k != 8) return PCTC_ERR_INVALID_ARG;
  if (p->chunk < 0) return PCTC_ERR_INVALID_ARG;
  t->k = k;
  long long chunk = p->chunk > 0 ? p->chunk : 4096;
  if (chunk > t->g.V) chunk = t->g.V;
  t->chunk = (int)((chunk + 3) / 4 * 4);                      // row pitch of the fp32 block: 16-byte rows
  size_t o = t->g.o_partial;                                  // the arg-max partials are not needed here
  auto take = [&](size_t bytes) { size_t r = o; o = up(o + bytes); return r; };
  t->o_logits = take((size_t)t->g.M * t->chunk * 4);
  t->o_val = take((size_t)t->g.M * k * 4);
  t->o_idx = take((size_t)t->g.M * k * 4);
  t->o_ms = take((size_t)t->g.M * 8);
  t->total = o;
  return PCTC_OK;
}
}  // namespace

pctc_status_t pctc_topk_workspace_bytes(const pctc_problem_t* problem, const int32_t* input_lengths_host, int32_t k,
                                        size_t* bytes_out) {
  if (!bytes_out) return PCTC_ERR_INVALID_ARG;
  TopkPlan t;
  pctc_status_t st = topk_plan(problem, input_lengths_host, k, &t);
  if (st != PCTC_OK) return st;
  *bytes_out = t.total;
  return PCTC_OK;
}

pctc_status_t pctc_topk_decode(const pctc_problem_t* p, const void* hidden, const void* W, const void* bias,
                               const int32_t* input_lengths, int32_t k, int32_t* topk_classes, float* topk_logprobs,
                               void* workspace, size_t workspace_bytes, void* stream_v) {
  TopkPlan t;
  pctc_status_t st = topk_plan(p, input_lengths, k, &t);
  if (st != PCTC_OK) return st;
  const GreedyPlan& g = t.g;
  if (!hidden || !W || !topk_classes || !workspace) return PCTC_ERR_INVALID_ARG;
  if (workspace_bytes < t.total) return PCTC_ERR_WORKSPACE_TOO_SMALL;
  if (((size_t)workspace & (ALIGN - 1)) || ((size_t)hidden & 15) || ((size_t)W & 15)) return PCTC_ERR_INVALID_ARG;
  if (g.use_umma && !umma_available()) return PCTC_ERR_CUDA;
  cudaStream_t stream = (cudaStream_t)stream_v;
  if (stream_is_capturing(stream)) return PCTC_ERR_UNSUPPORTED;
  char* ws = (char*)workspace;
  const int N = g.N, M = g.M, D = g.D;
#define PCTC_CUDA(call)                              \
  do {                                               \
    if ((call) != cudaSuccess) return PCTC_ERR_CUDA; \
  } while (0)
  int* d_meta = (int*)(ws + g.o_meta);
  int* d_status = (int*)(ws + g.o_status);
  PCTC_CUDA(batch_meta(input_lengths, nullptr, N, d_meta, nullptr, d_meta + N, nullptr, nullptr, d_meta + 2 * N + 1,
                       stream));
  PCTC_CUDA(cudaMemsetAsync(d_status, 0, 256, stream));
  void* d_X = ws + g.o_X;
  float* d_logits = (float*)(ws + t.o_logits);
  float* d_val = (float*)(ws + t.o_val);
  int* d_idx = (int*)(ws + t.o_idx);
  float2* d_ms = (float2*)(ws + t.o_ms);
  PCTC_CUDA(stack_frames(hidden, d_X, N, g.T, D, g.elem, d_meta + 2 * N + 1, d_meta + N, M, d_status, stream));
  for (long long v0 = 0; v0 < g.V; v0 += t.chunk) {          // the head in vocabulary chunks, logits never kept
    const int Cc = (int)((g.V - v0 < t.chunk) ? (g.V - v0) : t.chunk);
    Epilogue e;
    e.kind = EPI_STORE_F32;
    e.out = d_logits;
    e.ld = t.chunk;
    GemmCall c{d_X, D, false, (const char*)W + (size_t)v0 * D * g.elem, D, false, M, Cc, D};
    PCTC_CUDA(run_gemm(g.use_umma, g.bf16, c, e, d_status, stream));
    PCTC_CUDA(topk_update(k, d_logits, t.chunk, M, Cc, v0, bias, g.bf16, d_val, d_idx, d_ms, v0 == 0, stream));
  }
  PCTC_CUDA(topk_finish(k, d_val, d_idx, d_ms, d_meta + N, d_meta, N, g.T, topk_classes, topk_logprobs, stream));
#undef PCTC_CUDA
  return PCTC_OK;
}

pctc_status_t pctc_greedy_workspace_bytes(const pctc_problem_t* problem, const int32_t* input_lengths_host,
                                          size_t* bytes_out) {
  if (!bytes_out) return PCTC_ERR_INVALID_ARG;
  GreedyPlan g;
  pctc_status_t st = greedy_plan(problem, input_lengths_host, &g);
  if (st != PCTC_OK) return st;
  *bytes_out = g.total;
  return PCTC_OK;
}

pctc_status_t pctc_greedy_decode(const pctc_problem_t* p, const void* hidden, const void* W, const void* bias,
                                 const int32_t* input_lengths, int32_t* frame_labels, int32_t* tokens,
                                 int32_t* token_lengths, void* workspace, size_t workspace_bytes, void* stream_v) {
  GreedyPlan g;
  pctc_status_t st = greedy_plan(p, input_lengths, &g);
  if (st != PCTC_OK) return st;
  if (!hidden || !W || !tokens || !token_lengths || !workspace) return PCTC_ERR_INVALID_ARG;
  if (workspace_bytes < g.total) return PCTC_ERR_WORKSPACE_TOO_SMALL;
  if (((size_t)workspace & (ALIGN - 1)) || ((size_t)hidden & 15) || ((size_t)W & 15)) return PCTC_ERR_INVALID_ARG;
  if (g.use_umma && !umma_available()) return PCTC_ERR_CUDA;
  cudaStream_t stream = (cudaStream_t)stream_v;
  if (stream_is_capturing(stream)) return PCTC_ERR_UNSUPPORTED;
  char* ws = (char*)workspace;
  const int N = g.N, M = g.M, D = g.D;
#define PCTC_CUDA(call)                              \
  do {                                               \
    if ((call) != cudaSuccess) return PCTC_ERR_CUDA; \
  } while (0)
  int* d_meta = (int*)(ws + g.o_meta);
  PCTC_CUDA(batch_meta(input_lengths, nullptr, N, d_meta, nullptr, d_meta + N, nullptr, nullptr, d_meta + 2 * N + 1,
                       stream));
  PCTC_CUDA(cudaMemsetAsync(ws + g.o_status, 0, 256, stream));
  const int* d_Tn = d_meta;
  const int* d_row0 = d_meta + N;
  const int* d_row_utt = d_meta + 2 * N + 1;
  void* d_X = ws + g.o_X;
  float2* d_partial = (float2*)(ws + g.o_partial);
  int* d_labels = (int*)(ws + g.o_labels);
  PCTC_CUDA(stack_frames(hidden, d_X, N, g.T, D, g.elem, d_row_utt, d_row0, M, (int*)(ws + g.o_status), stream));
  Epilogue e;
  e.kind = EPI_ARGMAX_PARTIAL;
  e.bias = bias;
  e.partial = d_partial;
  e.nsplit = g.use_umma ? umma_lse_splits(M, (int)g.V) : 32;
  GemmCall c{d_X, D, false, W, D, false, M, (int)g.V, D};
  PCTC_CUDA(run_gemm(g.use_umma, g.bf16, c, e, (int*)(ws + g.o_status), stream));
  PCTC_CUDA(argmax_combine(d_partial, g.use_umma ? umma_lse_partials_per_split(D) * e.nsplit : e.nsplit, M, d_labels,
                           stream));
  PCTC_CUDA(greedy_collapse(d_labels, d_row0, d_Tn, N, g.T, p->blank_id, frame_labels, tokens, token_lengths, stream));
#undef PCTC_CUDA
  return PCTC_OK;
}

}  // extern "C"
