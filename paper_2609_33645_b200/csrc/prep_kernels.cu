// Integer and copy steps of Algorithm 1: batch-union subset and relabelling
// (lines 2-3), stacking of the valid frames (line 4), the gather of the selected
// head rows (line 6), and the small reductions around the contractions.
#include "../../include/prunedctc.h"
#include "pctc_internal.h"

#include <math_constants.h>

#include <mutex>

namespace pctc {

namespace {

// --- Algorithm 1 line 2: mark every target token in a V-bit set -------------------------------
__global__ void k_mark_targets(const int* __restrict__ targets, int stride, const int* __restrict__ U_n,
                               int N, long long V, int blank, unsigned* bitmap, int* utt_flags) {
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= N * stride) return;
  int n = idx / stride, i = idx - n * stride;
  if (i >= U_n[n]) return;
  int tok = targets[idx];
  if (tok == blank || tok < 0 || (long long)tok >= V) {
    atomicOr(&utt_flags[n], 4);      // bad target: never enters U
  } else {
    atomicOr(&bitmap[tok >> 5], 1u << (tok & 31));
  }
}

// --- rank the set bits: U = blank, then ascending ids; vmap[id] = position in U ----------------
// One CTA: each thread owns a contiguous run of bitmap words, a block-wide exclusive scan of the
// per-thread popcounts gives every run its first rank.
// Ranks past `cap` are dropped (their classes stay unmapped): the caller then flags the batch.
__global__ void k_rank_subset(const unsigned* __restrict__ bitmap, int nwords, int blank, int* word_rank,
                              int* vmap, int* U_out, int* K_out, int cap, int* utt_flags, int N, int* status) {
  __shared__ int s_scan[1024];
  const int tid = threadIdx.x, nt = blockDim.x;
  const int per = (nwords + nt - 1) / nt;
  const int w0 = min(nwords, tid * per), w1 = min(nwords, w0 + per);
  int cnt = 0;
  for (int w = w0; w < w1; ++w) cnt += __popc(bitmap[w]);
  s_scan[tid] = cnt;
  __syncthreads();
  for (int off = 1; off < nt; off <<= 1) {       // inclusive Hillis-Steele scan
    int v = (tid >= off) ? s_scan[tid - off] : 0;
    __syncthreads();
    s_scan[tid] += v;
    __syncthreads();
  }
  int rank = s_scan[tid] - cnt;                  // exclusive prefix
  for (int w = w0; w < w1; ++w) {
    unsigned bits = bitmap[w];
    word_rank[w] = rank;
    while (bits) {
      int b = __ffs(bits) - 1;
      bits &= bits - 1;
      int id = (w << 5) + b;
      if (1 + rank < cap) {
        U_out[1 + rank] = id;
        vmap[id] = 1 + rank;
      }
      ++rank;
    }
  }
  const int K = 1 + s_scan[nt - 1];
  if (tid == nt - 1) {
    *K_out = min(K, cap);
    U_out[0] = blank;
    vmap[blank] = 0;
    if (K > cap && status) atomicCAS(status, 0, 0x100);
  }
  if (K > cap)                                   // more selected classes than the buffers hold
    for (int n = tid; n < N; n += nt) atomicOr(&utt_flags[n], 8);
}

// --- Algorithm 1 line 3: relabel ----------------------------------------------------------------
__global__ void k_relabel(const int* __restrict__ targets, int stride, const int* __restrict__ U_n, int N,
                          long long V, int blank, const int* __restrict__ vmap, int* relabeled) {
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= N * stride) return;
  int n = idx / stride, i = idx - n * stride;
  int out = -1;
  if (i < U_n[n]) {
    int tok = targets[idx];
    if (tok != blank && tok >= 0 && (long long)tok < V) out = vmap[tok];
  }
  relabeled[idx] = out;
}

// --- batch description (Algorithm 1 line 4: which stacked row belongs to which frame) ------------
// The lengths reach the device as kernel parameters, up to LEN_SLICE utterances per launch, so the
// host never copies from pageable memory and never waits for the stream; everything derived from
// them (first stacked row, first trellis cell, first arc-flag byte, row -> utterance) is computed
// on the device.
constexpr int LEN_SLICE = 1024;
struct LengthSlice {
  int T[LEN_SLICE];
  int U[LEN_SLICE];
};

__global__ void k_put_lengths(const __grid_constant__ LengthSlice s, int n0, int cnt, int* __restrict__ T_n,
                              int* __restrict__ U_n) {
  for (int i = threadIdx.x; i < cnt; i += blockDim.x) {
    T_n[n0 + i] = s.T[i];
    if (U_n) U_n[n0 + i] = s.U[i];
  }
}

// One CTA: exclusive prefix sums over the utterances of T_n (rows), T_n (2 U_n + 1) (trellis cells)
// and T_n roundup4(2 U_n + 1) (arc-flag bytes).  Each thread owns a contiguous run of utterances.
__global__ void k_batch_offsets(const int* __restrict__ T_n, const int* __restrict__ U_n, int N, int* __restrict__ row0,
                                long long* __restrict__ cell0, long long* __restrict__ mcell0) {
  __shared__ long long s_rows[1024], s_cells[1024], s_mcells[1024];
  const int tid = threadIdx.x, nt = blockDim.x;
  const int per = (N + nt - 1) / nt;
  const int n0 = min(N, tid * per), n1 = min(N, n0 + per);
  long long rows = 0, cells = 0, mcells = 0;
  for (int n = n0; n < n1; ++n) {
    const long long T = T_n[n], L = U_n ? 2LL * U_n[n] + 1 : 1;
    rows += T;
    cells += T * L;
    mcells += T * ((L + 3) / 4 * 4);
  }
  s_rows[tid] = rows; s_cells[tid] = cells; s_mcells[tid] = mcells;
  __syncthreads();
  for (int off = 1; off < nt; off <<= 1) {       // inclusive Hillis-Steele scan of the three sums
    long long a = 0, b = 0, c = 0;
    if (tid >= off) { a = s_rows[tid - off]; b = s_cells[tid - off]; c = s_mcells[tid - off]; }
    __syncthreads();
    s_rows[tid] += a; s_cells[tid] += b; s_mcells[tid] += c;
    __syncthreads();
  }
  long long r = s_rows[tid] - rows, c = s_cells[tid] - cells, mc = s_mcells[tid] - mcells;
  for (int n = n0; n < n1; ++n) {
    const long long T = T_n[n], L = U_n ? 2LL * U_n[n] + 1 : 1;
    row0[n] = (int)r;
    if (cell0) cell0[n] = c;
    if (mcell0) mcell0[n] = mc;
    r += T;
    c += T * L;
    mc += T * ((L + 3) / 4 * 4);
  }
  if (tid == nt - 1) row0[N] = (int)s_rows[nt - 1];
}

__global__ void k_row_utt(const int* __restrict__ T_n, const int* __restrict__ row0, int N, int* __restrict__ row_utt) {
  for (int n = blockIdx.x; n < N; n += gridDim.x) {
    const int r0 = row0[n], T = T_n[n];
    for (int t = threadIdx.x; t < T; t += blockDim.x) row_utt[r0 + t] = n;
  }
}

// --- row copies ---------------------------------------------------------------------------------
__device__ __forceinline__ void copy_row(const char* __restrict__ src, char* __restrict__ dst, size_t bytes) {
  if ((((size_t)src | (size_t)dst | bytes) & 15) == 0) {
    const uint4* s = reinterpret_cast<const uint4*>(src);
    uint4* d = reinterpret_cast<uint4*>(dst);
    for (size_t i = threadIdx.x; i < bytes / 16; i += blockDim.x) d[i] = s[i];
  } else {
    for (size_t i = threadIdx.x; i < bytes; i += blockDim.x) dst[i] = src[i];
  }
}

__device__ __forceinline__ void zero_row(char* __restrict__ dst, size_t bytes) {
  if ((((size_t)dst | bytes) & 15) == 0) {
    uint4* d = reinterpret_cast<uint4*>(dst);
    for (size_t i = threadIdx.x; i < bytes / 16; i += blockDim.x) d[i] = make_uint4(0, 0, 0, 0);
  } else {
    for (size_t i = threadIdx.x; i < bytes; i += blockDim.x) dst[i] = 0;
  }
}

__global__ void k_stack_frames(const char* __restrict__ hidden, char* __restrict__ X, int T, size_t row_bytes,
                               const int* __restrict__ row_utt, const int* __restrict__ row0, int N, int* status) {
  const int m = blockIdx.x;
  const int n = row_utt[m];
  if (!index_ok(n, 0, N, status, 1)) return;
  const int t = m - row0[n];
  if (!index_ok(t, 0, T, status, 1)) return;
  copy_row(hidden + ((size_t)n * T + t) * row_bytes, X + (size_t)m * row_bytes, row_bytes);
}

__device__ __forceinline__ void store4(float* dst, float4 v) { *reinterpret_cast<float4*>(dst) = v; }
__device__ __forceinline__ void store4(__nv_bfloat16* dst, float4 v) {
  const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 o;
  o.x = *reinterpret_cast<const unsigned*>(&lo);
  o.y = *reinterpret_cast<const unsigned*>(&hi);
  *reinterpret_cast<uint2*>(dst) = o;
}

template <typename TOut>
__global__ void k_unstack_cast(const float* __restrict__ acc, int nslab, size_t slab_stride, TOut* __restrict__ dH,
                               int T, int D, const int* __restrict__ T_n, const int* __restrict__ row0, int M,
                               int* status) {
  const int n = blockIdx.x / T, t = blockIdx.x - n * T;
  TOut* dst = dH + ((size_t)n * T + t) * D;
  if (t >= T_n[n]) {
    zero_row(reinterpret_cast<char*>(dst), (size_t)D * sizeof(TOut));
    return;
  }
  if (!index_ok((long long)row0[n] + t, 0, M, status, 3)) return;
  const float* src = acc + ((size_t)row0[n] + t) * D;
  if ((D & 3) == 0) {                          // four columns per thread: 16-byte loads, 8- or 16-byte stores
    for (int d = threadIdx.x * 4; d < D; d += blockDim.x * 4) {
      float4 v = *reinterpret_cast<const float4*>(src + d);
      for (int s = 1; s < nslab; ++s) {        // k-split partial sums, fixed order
        const float4 u = *reinterpret_cast<const float4*>(src + s * slab_stride + d);
        v.x += u.x; v.y += u.y; v.z += u.z; v.w += u.w;
      }
      store4(dst + d, v);
    }
    return;
  }
  for (int d = threadIdx.x; d < D; d += blockDim.x) {
    float v = src[d];
    for (int s = 1; s < nslab; ++s) v += src[s * slab_stride + d];     // k-split partial sums, fixed order
    dst[d] = TOut(v);
  }
}

__global__ void k_gather_rows(const char* __restrict__ W, char* __restrict__ W_U, const int* __restrict__ U,
                              const int* __restrict__ Kdev, size_t row_bytes, long long V, int* status) {
  const int j = blockIdx.x;
  char* dst = W_U + (size_t)j * row_bytes;
  if (j < *Kdev && index_ok(U[j], 0, V, status, 4)) copy_row(W + (size_t)U[j] * row_bytes, dst, row_bytes);
  else zero_row(dst, row_bytes);
}

// --- frames of an utterance with a non-finite loss (NaN/Inf in its states): the stacked copy is
// zeroed before the backward pass, so that 0 * NaN cannot leak into dW through dZ^T X ---
__global__ void k_zero_nonfinite_rows(char* __restrict__ X, size_t row_bytes, const int* __restrict__ row_utt,
                                      const int* __restrict__ flags, int N, int* status) {
  const int m = blockIdx.x;
  if (!index_ok(row_utt[m], 0, N, status, 2)) return;
  if (flags[row_utt[m]] & 2) zero_row(X + (size_t)m * row_bytes, row_bytes);
}

// --- db_c = dZ_c^T 1 (Algorithm 1 line 16): fixed summation order, no atomics -------------------
template <typename TIn, typename TOut>
__global__ void k_column_sums(const TIn* __restrict__ chunk, long long ld, int M, int cols,
                              TOut* __restrict__ db, long long v0, bool accumulate) {
  __shared__ float s_part[32][33];
  const int cx = threadIdx.x, ry = threadIdx.y;
  const int j = blockIdx.x * 32 + cx;
  float acc = 0.f;
  if (j < cols)
    for (int i = ry; i < M; i += 32) acc += float(chunk[(size_t)i * ld + j]);
  s_part[ry][cx] = acc;
  __syncthreads();
  if (ry == 0 && j < cols) {
    float tot = 0.f;
    for (int r = 0; r < 32; ++r) tot += s_part[r][cx];
    if (accumulate) tot += float(db[v0 + j]);
    db[v0 + j] = TOut(tot);
  }
}

// --- second stage of db_c when the dlogits epilogue has already summed blocks of 32 rows: a fixed-order
// sum over the row blocks (reads 1/16 of the bytes of the chunk itself) ---
template <typename TOut>
__global__ void k_colpart_sums(const float* __restrict__ colpart, long long ld, int nblocks, int cols,
                               TOut* __restrict__ db, long long v0, bool accumulate) {
  __shared__ float s_part[8][33];
  const int cx = threadIdx.x, ry = threadIdx.y;          // 32 columns x 8 interleaved row-block lanes
  const int j = blockIdx.x * 32 + cx;
  float acc = 0.f;
  if (j < cols)
    for (int b = ry; b < nblocks; b += 8) acc += colpart[(size_t)b * ld + j];
  s_part[ry][cx] = acc;
  __syncthreads();
  if (ry == 0 && j < cols) {
    float tot = 0.f;
    for (int r = 0; r < 8; ++r) tot += s_part[r][cx];
    if (accumulate) tot += float(db[v0 + j]);
    db[v0 + j] = TOut(tot);
  }
}

__global__ void k_lse_combine(const float2* __restrict__ partial, int nsplit, int M, float* __restrict__ lambda) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= M) return;
  // a slot nothing was written to holds (anything, 0): it must not take part in the maximum either,
  // or a frame whose every logit lies far below the empty slot's value would lose its whole sum
  float mx = -CUDART_INF_F;
  for (int s = 0; s < nsplit; ++s) {
    const float2 p = partial[(size_t)i * nsplit + s];
    if (!(p.y <= 0.f)) mx = fmaxf(mx, p.x);
  }
  float sum = 0.f;
  for (int s = 0; s < nsplit; ++s) {
    float2 p = partial[(size_t)i * nsplit + s];
    if (!(p.y <= 0.f)) sum += p.y * __expf(p.x - mx);
  }
  lambda[i] = mx + logf(sum);
}

// --- recognition: frame arg-max from per-split partials, then the collapse map B of Section 3.1 ---
__global__ void k_argmax_combine(const float2* __restrict__ partial, int nparts, int M, int* __restrict__ labels) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= M) return;
  float best = -CUDART_INF_F;
  int idx = 0x7fffffff;
  for (int s = 0; s < nparts; ++s) {
    const float2 p = partial[(size_t)i * nparts + s];
    const int j = __float_as_int(p.y);
    if (j < 0) continue;                                   // empty split
    if (p.x > best || (p.x == best && j < idx)) { best = p.x; idx = j; }
  }
  labels[i] = (idx == 0x7fffffff) ? 0 : idx;
}

// --- recognition: the k best classes of every frame with their log-probabilities ------------------
// One warp per stacked frame and vocabulary chunk.  Every lane scans its share of the chunk's logits
// keeping its own k best (sorted, in registers) and a running (max, sum of exponentials); the lanes'
// lists, seeded with the frame's k best of the earlier chunks, are then merged by k rounds of a warp-wide
// arg-max.  Order: larger logit first, among equal logits the smaller class index (the rule of the
// frame arg-max above), so the result does not depend on the chunk width.
__device__ __forceinline__ bool topk_before(float av, int ai, float bv, int bi) {
  return av > bv || (av == bv && ai < bi);
}

template <int K, typename TB>
__global__ void k_topk_update(const float* __restrict__ logits, long long ld, int M, int cols, long long v0,
                              const TB* __restrict__ bias, float* __restrict__ run_val, int* __restrict__ run_idx,
                              float2* __restrict__ run_ms, int first) {
  const int m = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (m >= M) return;
  float val[K];
  int idx[K];
#pragma unroll
  for (int r = 0; r < K; ++r) { val[r] = -CUDART_INF_F; idx[r] = 0x7fffffff; }
  auto insert = [&](float z, int j) {
    if (!topk_before(z, j, val[K - 1], idx[K - 1])) return;
    val[K - 1] = z; idx[K - 1] = j;
#pragma unroll
    for (int r = K - 1; r > 0; --r) {
      if (topk_before(val[r], idx[r], val[r - 1], idx[r - 1])) {
        const float tv = val[r]; val[r] = val[r - 1]; val[r - 1] = tv;
        const int ti = idx[r]; idx[r] = idx[r - 1]; idx[r - 1] = ti;
      }
    }
  };
  if (!first && lane < K) insert(run_val[(size_t)m * K + lane], run_idx[(size_t)m * K + lane]);
  float mx = -CUDART_INF_F, sum = 0.f;
  const float* row = logits + (size_t)m * ld;
  for (int j = lane; j < cols; j += 32) {
    float z = row[j];
    if (bias) z += float(bias[v0 + j]);
    if (z > mx) { sum = sum * __expf(mx - z) + 1.f; mx = z; }      // exp(-inf) = 0 at the first logit
    else sum += __expf(z - mx);                                   // a NaN logit makes the sum NaN
    insert(z, (int)(v0 + j));
  }
  // merge the 32 sorted lists: K rounds, each takes the best head and pops it in the lane that held it
  float out_v = -CUDART_INF_F;
  int out_i = 0x7fffffff;
#pragma unroll
  for (int r = 0; r < K; ++r) {
    float bv = val[0];
    int bi = idx[0];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (topk_before(ov, oi, bv, bi)) { bv = ov; bi = oi; }
    }
    if (lane == r) { out_v = bv; out_i = bi; }
    if (idx[0] == bi && bi != 0x7fffffff) {        // class indices are distinct across lanes: one lane pops
#pragma unroll
      for (int q = 0; q + 1 < K; ++q) { val[q] = val[q + 1]; idx[q] = idx[q + 1]; }
      val[K - 1] = -CUDART_INF_F; idx[K - 1] = 0x7fffffff;
    }
  }
  if (lane < K) { run_val[(size_t)m * K + lane] = out_v; run_idx[(size_t)m * K + lane] = out_i; }
  // running normaliser: combine the lanes' (max, sum) pairs, then the earlier chunks'
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, mx, o), os = __shfl_xor_sync(0xffffffffu, sum, o);
    const float nm = fmaxf(mx, om);
    if (nm == -CUDART_INF_F) { sum = sum + os; }                   // both empty (or NaN sums pass through)
    else { sum = sum * __expf(mx - nm) + os * __expf(om - nm); }
    mx = nm;
  }
  if (lane == 0) {
    if (!first) {
      const float2 p = run_ms[m];
      const float nm = fmaxf(mx, p.x);
      if (nm != -CUDART_INF_F) sum = sum * __expf(mx - nm) + p.y * __expf(p.x - nm);
      else sum += p.y;
      mx = nm;
    }
    run_ms[m] = make_float2(mx, sum);
  }
}

// classes [N,T,K] and log-probabilities [N,T,K] of the padded layout; padded frames and ranks beyond V
// read class -1 and log-probability -inf
template <int K>
__global__ void k_topk_finish(const float* __restrict__ run_val, const int* __restrict__ run_idx,
                              const float2* __restrict__ run_ms, const int* __restrict__ row0,
                              const int* __restrict__ T_n, int N, int T, int* __restrict__ classes,
                              float* __restrict__ logprobs) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;          // (n, t, r)
  if (i >= N * T * K) return;
  const int r = i % K, nt = i / K, t = nt % T, n = nt / T;
  int cls = -1;
  float lp = -CUDART_INF_F;
  if (t < T_n[n]) {
    const size_t m = (size_t)row0[n] + t;
    const int j = run_idx[m * K + r];
    if (j != 0x7fffffff) {
      const float2 p = run_ms[m];
      cls = j;
      lp = run_val[m * K + r] - (p.x + logf(p.y));
    }
  }
  classes[i] = cls;
  if (logprobs) logprobs[i] = lp;
}

// One warp per utterance, 32 frames at a time: a frame emits its label iff the label is not blank
// and differs from the previous frame's label.
__global__ void k_greedy_collapse(const int* __restrict__ labels, const int* __restrict__ row0,
                                  const int* __restrict__ T_n, int T, int blank, int* frame_labels,
                                  int* tokens, int* token_lengths) {
  const int n = blockIdx.x, lane = threadIdx.x;
  const int Tn = T_n[n], r0 = row0[n];
  int count = 0, prev_last = -1;
  for (int t0 = 0; t0 < T; t0 += 32) {
    const int t = t0 + lane;
    const int lab = (t < Tn) ? labels[r0 + t] : -1;
    if (frame_labels && t < T) frame_labels[(size_t)n * T + t] = lab;
    int prev = __shfl_up_sync(0xffffffffu, lab, 1);
    if (lane == 0) prev = prev_last;
    const bool emit = (t < Tn) && lab != blank && lab != prev;
    const unsigned mask = __ballot_sync(0xffffffffu, emit);
    if (emit) tokens[(size_t)n * T + count + __popc(mask & ((1u << lane) - 1u))] = lab;
    count += __popc(mask);
    prev_last = __shfl_sync(0xffffffffu, lab, 31);
  }
  for (int t = count + lane; t < T; t += 32) tokens[(size_t)n * T + t] = -1;
  if (lane == 0) token_lengths[n] = count;
}

}  // namespace

cudaError_t argmax_combine(const float2* partial, int nparts, int M, int* labels, cudaStream_t stream) {
  k_argmax_combine<<<(M + 127) / 128, 128, 0, stream>>>(partial, nparts, M, labels);
  return cudaGetLastError();
}

namespace {
template <int K>
cudaError_t topk_update_k(const float* logits, long long ld, int M, int cols, long long v0, const void* bias,
                          bool bias_bf16, float* run_val, int* run_idx, float2* run_ms, bool first, cudaStream_t stream) {
  const int warps = 8;
  const dim3 grid((M + warps - 1) / warps), block(warps * 32);
  if (bias_bf16)
    k_topk_update<K, __nv_bfloat16><<<grid, block, 0, stream>>>(logits, ld, M, cols, v0, (const __nv_bfloat16*)bias,
                                                               run_val, run_idx, run_ms, first ? 1 : 0);
  else
    k_topk_update<K, float><<<grid, block, 0, stream>>>(logits, ld, M, cols, v0, (const float*)bias, run_val, run_idx,
                                                       run_ms, first ? 1 : 0);
  return cudaGetLastError();
}
}  // namespace

cudaError_t topk_update(int k, const float* logits, long long ld, int M, int cols, long long v0, const void* bias,
                        bool bias_bf16, float* run_val, int* run_idx, float2* run_ms, bool first, cudaStream_t stream) {
  switch (k) {
    case 1: return topk_update_k<1>(logits, ld, M, cols, v0, bias, bias_bf16, run_val, run_idx, run_ms, first, stream);
    case 2: return topk_update_k<2>(logits, ld, M, cols, v0, bias, bias_bf16, run_val, run_idx, run_ms, first, stream);
    case 4: return topk_update_k<4>(logits, ld, M, cols, v0, bias, bias_bf16, run_val, run_idx, run_ms, first, stream);
    case 8: return topk_update_k<8>(logits, ld, M, cols, v0, bias, bias_bf16, run_val, run_idx, run_ms, first, stream);
  }
  return cudaErrorInvalidValue;
}

cudaError_t topk_finish(int k, const float* run_val, const int* run_idx, const float2* run_ms, const int* row0,
                        const int* T_n, int N, int T, int* classes, float* logprobs, cudaStream_t stream) {
  const long long total = (long long)N * T * k;
  const int blocks = (int)((total + 255) / 256);
  switch (k) {
    case 1: k_topk_finish<1><<<blocks, 256, 0, stream>>>(run_val, run_idx, run_ms, row0, T_n, N, T, classes, logprobs); break;
    case 2: k_topk_finish<2><<<blocks, 256, 0, stream>>>(run_val, run_idx, run_ms, row0, T_n, N, T, classes, logprobs); break;
    case 4: k_topk_finish<4><<<blocks, 256, 0, stream>>>(run_val, run_idx, run_ms, row0, T_n, N, T, classes, logprobs); break;
    case 8: k_topk_finish<8><<<blocks, 256, 0, stream>>>(run_val, run_idx, run_ms, row0, T_n, N, T, classes, logprobs); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

cudaError_t greedy_collapse(const int* labels, const int* row0, const int* T_n, int N, int T, int blank,
                            int* frame_labels, int* tokens, int* token_lengths, cudaStream_t stream) {
  k_greedy_collapse<<<N, 32, 0, stream>>>(labels, row0, T_n, T, blank, frame_labels, tokens, token_lengths);
  return cudaGetLastError();
}

cudaError_t subset_and_relabel(const int* targets, int target_stride, const int* U_n_dev, int N,
                               long long V, int blank, unsigned* bitmap, int* word_rank,
                               int* vmap, int* U_out, int* K_out, int* relabeled, int* utt_flags,
                               int cap, int* status, cudaStream_t stream) {
  const int nwords = (int)((V + 31) / 32);
  cudaError_t e;
  if ((e = cudaMemsetAsync(bitmap, 0, (size_t)nwords * 4, stream)) != cudaSuccess) return e;
  if ((e = cudaMemsetAsync(vmap, 0xFF, (size_t)V * 4, stream)) != cudaSuccess) return e;
  if ((e = cudaMemsetAsync(utt_flags, 0, (size_t)N * 4, stream)) != cudaSuccess) return e;
  const int total = N * target_stride;
  const int blocks = (total + 255) / 256;
  if (total > 0)
    k_mark_targets<<<blocks, 256, 0, stream>>>(targets, target_stride, U_n_dev, N, V, blank, bitmap, utt_flags);
  k_rank_subset<<<1, 1024, 0, stream>>>(bitmap, nwords, blank, word_rank, vmap, U_out, K_out, cap, utt_flags, N,
                                        status);
  if (total > 0)
    k_relabel<<<blocks, 256, 0, stream>>>(targets, target_stride, U_n_dev, N, V, blank, vmap, relabeled);
  return cudaGetLastError();
}

cudaError_t batch_meta(const int* T_host, const int* U_host, int N, int* T_n, int* U_n, int* row0,
                       long long* cell0, long long* mcell0, int* row_utt, cudaStream_t stream) {
  LengthSlice s;
  for (int n0 = 0; n0 < N; n0 += LEN_SLICE) {
    const int cnt = (N - n0 < LEN_SLICE) ? (N - n0) : LEN_SLICE;
    for (int i = 0; i < cnt; ++i) {
      s.T[i] = T_host[n0 + i];
      s.U[i] = U_host ? U_host[n0 + i] : 0;
    }
    k_put_lengths<<<1, 256, 0, stream>>>(s, n0, cnt, T_n, U_host ? U_n : nullptr);
  }
  k_batch_offsets<<<1, 1024, 0, stream>>>(T_n, U_host ? U_n : nullptr, N, row0, cell0, mcell0);
  k_row_utt<<<(N < 1024 ? N : 1024), 256, 0, stream>>>(T_n, row0, N, row_utt);
  return cudaGetLastError();
}

cudaError_t stack_frames(const void* hidden, void* X, int N, int T, int D, int elem_bytes,
                         const int* row_utt, const int* row0, int M, int* status, cudaStream_t stream) {
  k_stack_frames<<<M, 128, 0, stream>>>((const char*)hidden, (char*)X, T, (size_t)D * elem_bytes, row_utt, row0, N,
                                        status);
  return cudaGetLastError();
}

cudaError_t zero_nonfinite_rows(void* X, int M, int D, int elem_bytes, const int* row_utt, const int* utt_flags,
                                int N, int* status, cudaStream_t stream) {
  k_zero_nonfinite_rows<<<M, 64, 0, stream>>>((char*)X, (size_t)D * elem_bytes, row_utt, utt_flags, N, status);
  return cudaGetLastError();
}

cudaError_t unstack_cast(const float* acc, int nslab, size_t slab_stride, void* dH, int N, int T, int D,
                         bool out_bf16, const int* T_n, const int* row0, int M, int* status, cudaStream_t stream) {
  if (out_bf16)
    k_unstack_cast<__nv_bfloat16><<<N * T, 128, 0, stream>>>(acc, nslab, slab_stride, (__nv_bfloat16*)dH, T, D, T_n,
                                                             row0, M, status);
  else
    k_unstack_cast<float><<<N * T, 128, 0, stream>>>(acc, nslab, slab_stride, (float*)dH, T, D, T_n, row0, M, status);
  return cudaGetLastError();
}

cudaError_t gather_rows(const void* W, void* W_U, const int* U, const int* Kdev, int Kcap, int D,
                        int elem_bytes, long long V, int* status, cudaStream_t stream) {
  k_gather_rows<<<Kcap, 128, 0, stream>>>((const char*)W, (char*)W_U, U, Kdev, (size_t)D * elem_bytes, V, status);
  return cudaGetLastError();
}

cudaError_t column_sums(const void* chunk, bool chunk_bf16, long long ld, int M, int cols,
                        void* db, bool db_bf16, long long v0, bool accumulate, cudaStream_t stream) {
  dim3 block(32, 32), grid((cols + 31) / 32);
  if (chunk_bf16 && db_bf16)
    k_column_sums<<<grid, block, 0, stream>>>((const __nv_bfloat16*)chunk, ld, M, cols, (__nv_bfloat16*)db, v0, accumulate);
  else if (!chunk_bf16 && !db_bf16)
    k_column_sums<<<grid, block, 0, stream>>>((const float*)chunk, ld, M, cols, (float*)db, v0, accumulate);
  else
    return cudaErrorInvalidValue;
  return cudaGetLastError();
}

cudaError_t colpart_sums(const float* colpart, long long ld, int nblocks, int cols, void* db, bool db_bf16,
                         long long v0, bool accumulate, cudaStream_t stream) {
  dim3 block(32, 8), grid((cols + 31) / 32);
  if (db_bf16)
    k_colpart_sums<<<grid, block, 0, stream>>>(colpart, ld, nblocks, cols, (__nv_bfloat16*)db, v0, accumulate);
  else
    k_colpart_sums<<<grid, block, 0, stream>>>(colpart, ld, nblocks, cols, (float*)db, v0, accumulate);
  return cudaGetLastError();
}

cudaError_t lse_combine(const float2* partial, int nsplit, int M, float* lambda, cudaStream_t stream) {
  k_lse_combine<<<(M + 127) / 128, 128, 0, stream>>>(partial, nsplit, M, lambda);
  return cudaGetLastError();
}

}  // namespace pctc

// ---------------------------------------------------------------------------------------------
// Subset and relabelling without any allocation: the scratch of the kernels above lives in a
// file-scope device array instead of a caller-provided workspace.
// ---------------------------------------------------------------------------------------------
namespace pctc {
namespace {

constexpr long long NOALLOC_MAX_V = PCTC_NOALLOC_MAX_V;
constexpr size_t NOALLOC_WORDS = (size_t)(NOALLOC_MAX_V / 32);
// layout: bitmap [words] | word_rank [words] | vmap [MAX_V]
constexpr size_t NOALLOC_BYTES = NOALLOC_WORDS * 4 * 2 + (size_t)NOALLOC_MAX_V * 4;

static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_BYTES];

constexpr int MAX_DEVICES = 64;
std::mutex g_noalloc_mutex;
unsigned char* g_noalloc_ptr[MAX_DEVICES] = {};

// The array's name is only a host-side handle; the device address has to be asked for, once per
// device, while that device is current.
cudaError_t noalloc_scratch(unsigned char** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (!g_noalloc_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    g_noalloc_ptr[dev] = (unsigned char*)p;
  }
  *out = g_noalloc_ptr[dev];
  return cudaSuccess;
}

}  // namespace
}  // namespace pctc

extern "C" pctc_status_t pctc_subset_relabel_noalloc(const int32_t* targets, const int32_t* target_lengths,
                                                     int32_t N, int32_t target_stride, int64_t V,
                                                     int32_t blank_id, int32_t* subset_out, int32_t* K_out,
                                                     int32_t* relabeled_out, int32_t* utt_flags, void* stream) {
  using namespace pctc;
  if (N <= 0 || target_stride < 0 || V <= 0 || blank_id < 0 || (long long)blank_id >= V) return PCTC_ERR_INVALID_ARG;
  if (!target_lengths || !subset_out || !K_out || !utt_flags) return PCTC_ERR_INVALID_ARG;
  if (target_stride > 0 && (!targets || !relabeled_out)) return PCTC_ERR_INVALID_ARG;
  if (V > NOALLOC_MAX_V) return PCTC_ERR_UNSUPPORTED;      // the fixed scratch holds PCTC_NOALLOC_MAX_V classes
  unsigned char* base = nullptr;
  if (noalloc_scratch(&base) != cudaSuccess) return PCTC_ERR_CUDA;
  unsigned* bitmap = (unsigned*)base;
  int* word_rank = (int*)(base + NOALLOC_WORDS * 4);
  int* vmap = (int*)(base + NOALLOC_WORDS * 8);
  // subset_and_relabel clears the bitmap, the class map and the flags itself: nothing of an
  // earlier call survives into this one.
  cudaError_t e = subset_and_relabel(targets, target_stride, target_lengths, N, V, blank_id, bitmap, word_rank, vmap,
                                     subset_out, K_out, relabeled_out, utt_flags, 0x7fffffff, nullptr,
                                     (cudaStream_t)stream);
  return e == cudaSuccess ? PCTC_OK : PCTC_ERR_CUDA;
}
