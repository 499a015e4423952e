// Alignment dynamic program on the subset log-probabilities S (Algorithm 1,
// lines 7-10), with the finite-beam arc pruning of Section 3.3 / Appendix B.3 as
// an option.
//
// The CTC graph of utterance n is the trellis over l' = (blank, y_1, blank, ...,
// y_U, blank): L = 2U+1 positions, T_n frames.  One CTA handles one (utterance,
// direction) pair; the backward recursion is the forward recursion on the
// time- and label-reversed problem, so one kernel serves both.  A CTA of a
// single warp exchanges the two boundary states between lanes by shuffle; wider
// trellises use several warps and one barrier per frame.  Each thread keeps SPL
// consecutive positions in registers; the emission scores it needs, gathered
// from the row of S, are staged DEPTH frames ahead in shared memory with
// cp.async so that the serial chain never waits on memory.
//
// Scores are kept per-frame normalised (the row maximum of the previous frame is
// subtracted, its running sum carried in double) so that fp32 magnitudes stay
// O(100) for any T.  Occupancies are then formed per frame as a softmax over
// positions of alpha + beta - emission, which needs no global constant.
#include "pctc_internal.h"

#include <math_constants.h>

namespace pctc {

namespace {

#define NEG_INF (-CUDART_INF_F)

enum SweepMode : int { MODE_LOG = 0, MODE_MAX = 1, MODE_MASKED = 2 };

struct SweepArgs {
  const float* S; long long ldS;
  const int* rel; int stride;
  const int* T_n; const int* U_n; const int* row0; const long long* cell0;
  float beam;
  float* out_f; float* out_b;        // rows written by the forward / backward sweep
  const float* va; const float* vb;  // MODE_MASKED: best-alignment scores
  double* off_a; double* off_b;      // per-frame offsets of va / vb (written by MODE_MAX)
  double* best;                      // [N] best alignment score
  float* loss; int* flags;
};

__device__ __forceinline__ void cp_async4(float* smem_dst, const float* gsrc) {
  unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(d), "l"(gsrc));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

__device__ __forceinline__ float lse3(float a, float b, float c) {
  const float mx = fmaxf(a, fmaxf(b, c));
  const float sh = (mx == NEG_INF) ? 0.f : mx;
  return sh + __logf(__expf(a - sh) + __expf(b - sh) + __expf(c - sh));
}

template <int W, int SPL, int DEPTH, int MODE>
__global__ void __launch_bounds__(W * 32) k_ctc_sweep(SweepArgs a) {
  constexpr int NTH = W * 32;
  constexpr int NE = (SPL == 1) ? 1 : 1 + SPL / 2;                 // emission slots per thread
  constexpr int NX = (MODE == MODE_MASKED) ? (2 * SPL + 2) : 0;    // beam: cur[SPL], prev[SPL+2]
  constexpr int NSLOT = NE + NX;
  extern __shared__ float s_ring[];                                // [DEPTH][NSLOT][NTH]
  __shared__ float s_wmax[2][W];
  __shared__ float s_tail[2][W][2];
  __shared__ float s_fin[2];
  __shared__ int s_rep;

  const int n = blockIdx.x, dir = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int T = a.T_n[n], U = a.U_n[n], L = 2 * U + 1;
  const int* rel = a.rel + (long long)n * a.stride;

  if (tid == 0) { s_rep = 0; s_fin[0] = NEG_INF; s_fin[1] = NEG_INF; }
  __syncthreads();
  if (a.flags[n] & 4) {                                            // bad target: excluded
    if (dir == 0 && tid == 0 && MODE != MODE_MAX) a.loss[n] = 0.f;
    return;
  }
  {
    int cnt = 0;
    for (int i = tid + 1; i < U; i += NTH) cnt += (rel[i] == rel[i - 1]);
    if (cnt) atomicAdd(&s_rep, cnt);
  }
  __syncthreads();
  if (T < U + s_rep) {                                             // no alignment exists (Appendix B.1)
    if (dir == 0 && tid == 0 && MODE != MODE_MAX) { atomicOr(&a.flags[n], 1); a.loss[n] = 0.f; }
    return;
  }

  // ---- static per-thread description of its positions, in sweep coordinates ----
  const int s_first = tid * SPL;
  int col[NE];                 // column of S per emission slot
  bool skip[SPL];              // transition s-2 -> s exists
#pragma unroll
  for (int k = 0; k < SPL; ++k) skip[k] = false;
  auto label_of = [&](int s) -> int {          // s odd, in sweep coordinates
    const int i = (s - 1) >> 1;
    return rel[dir ? (U - 1 - i) : i];
  };
  if (SPL == 1) {
    const int s = s_first;
    col[0] = (s < L && (s & 1)) ? label_of(s) : 0;
    skip[0] = (s < L) && (s & 1) && s >= 3 && label_of(s) != label_of(s - 2);
  } else {
    col[0] = 0;
#pragma unroll
    for (int q = 1; q < NE; ++q) {
      const int s = s_first + 2 * q - 1;
      col[q] = (s < L) ? label_of(s) : 0;
      skip[2 * q - 1] = (s < L) && s >= 3 && label_of(s) != label_of(s - 2);
    }
  }

  const long long cell0 = a.cell0[n];
  const int row0 = a.row0[n];
  auto real_t = [&](int tau) { return dir ? (T - 1 - tau) : tau; };
  auto real_s = [&](int s) { return dir ? (L - 1 - s) : s; };
  const float* Pm = nullptr;   // beam: the array read at the previous sweep frame
  const float* Cm = nullptr;   // beam: the array read at the current sweep frame
  if (MODE == MODE_MASKED) { Pm = dir ? a.vb : a.va; Cm = dir ? a.va : a.vb; }

  auto ring = [&](int tau, int slot) -> float* {
    return s_ring + ((size_t)(tau % DEPTH) * NSLOT + slot) * NTH + tid;
  };
  auto issue = [&](int tau) {
    if (tau < T) {
      const int t = real_t(tau);
      const float* Srow = a.S + (long long)(row0 + t) * a.ldS;
#pragma unroll
      for (int q = 0; q < NE; ++q) cp_async4(ring(tau, q), Srow + col[q]);
      if (MODE == MODE_MASKED) {
        const float* crow = Cm + cell0 + (long long)t * L;
#pragma unroll
        for (int k = 0; k < SPL; ++k) {
          const int s = s_first + k;
          if (s < L) cp_async4(ring(tau, NE + k), crow + real_s(s));
        }
        if (tau >= 1) {
          const float* prow = Pm + cell0 + (long long)real_t(tau - 1) * L;
#pragma unroll
          for (int k = 0; k < SPL + 2; ++k) {
            const int s = s_first + k - 2;
            if (s >= 0 && s < L) cp_async4(ring(tau, NE + SPL + k), prow + real_s(s));
          }
        }
      }
    }
    cp_async_commit();
  };

  for (int tau = 0; tau < DEPTH - 1; ++tau) issue(tau);

  float prev[SPL];
#pragma unroll
  for (int k = 0; k < SPL; ++k) prev[k] = NEG_INF;
  float m_prev = 0.f;          // row maximum of the previous frame (already folded into offsets)
  double C = 0.0;              // sum of the row maxima subtracted so far (thread 0)
  double best = 0.0;
  if (MODE == MODE_MASKED) best = a.best[n];
  float* out = dir ? a.out_b : a.out_f;
  double* off_out = dir ? a.off_b : a.off_a;

  for (int tau = 0; tau < T; ++tau) {
    issue(tau + DEPTH - 1);
    cp_async_wait<DEPTH - 1>();
    const int t = real_t(tau);

    // neighbour positions s_first-1 and s_first-2 of the previous frame
    float n1, n2;
    if (SPL == 1) {
      n1 = __shfl_up_sync(0xffffffffu, prev[0], 1);
      n2 = __shfl_up_sync(0xffffffffu, prev[0], 2);
      if (lane < 1) n1 = NEG_INF;
      if (lane < 2) n2 = NEG_INF;
    } else {
      n1 = __shfl_up_sync(0xffffffffu, prev[SPL - 1], 1);
      n2 = __shfl_up_sync(0xffffffffu, prev[SPL >= 2 ? SPL - 2 : 0], 1);
      if (lane == 0) {
        if (warp == 0) { n1 = NEG_INF; n2 = NEG_INF; }
        else { n1 = s_tail[(tau + 1) & 1][warp - 1][0]; n2 = s_tail[(tau + 1) & 1][warp - 1][1]; }
      }
    }
    if (W > 1 && tau > 0) {
      float mx = s_wmax[(tau + 1) & 1][0];
#pragma unroll
      for (int w = 1; w < W; ++w) mx = fmaxf(mx, s_wmax[(tau + 1) & 1][w]);
      m_prev = (mx == NEG_INF) ? 0.f : mx;
    }
    if (tid == 0 && tau > 0) C += (double)m_prev;

    float cst = 0.f;           // beam: offsets of the two frames minus the best score
    if (MODE == MODE_MASKED) {
      if (tau == 0) {
        cst = (float)((dir ? a.off_a[row0 + t] : a.off_b[row0 + t]) - best);
      } else {
        const int ta = dir ? t : t - 1;      // the earlier of the two real frames
        cst = (float)(a.off_a[row0 + ta] + a.off_b[row0 + ta + 1] - best);
      }
    }

    float cur[SPL];
    float local_max = NEG_INF;
#pragma unroll
    for (int k = 0; k < SPL; ++k) {
      const int s = s_first + k;
      float e;
      if (SPL == 1) e = *ring(tau, 0);
      else e = (k & 1) ? *ring(tau, (k + 1) / 2) : *ring(tau, 0);
      float p0 = prev[k];
      float p1 = (k >= 1) ? prev[k >= 1 ? k - 1 : 0] : n1;
      float p2 = (k >= 2) ? prev[k >= 2 ? k - 2 : 0] : (k == 1 ? n1 : n2);
      if (SPL == 1) { p1 = n1; p2 = n2; }
      if (!skip[k]) p2 = NEG_INF;
      float v;
      if (tau == 0) {
        v = (s <= 1) ? e : NEG_INF;
        if (MODE == MODE_MASKED && s <= 1 && s < L) {
          const float c = *ring(tau, NE + k);
          if (!(c + cst >= -a.beam)) v = NEG_INF;
        }
      } else {
        if (MODE == MODE_MASKED) {
          const float c = (s < L) ? *ring(tau, NE + k) : 0.f;
          // arcs (tau-1, s-j) -> (tau, s), j = 0, 1, 2: prev-slot index k+2-j
          if (p0 != NEG_INF && !(*ring(tau, NE + SPL + k + 2) + c + cst >= -a.beam)) p0 = NEG_INF;
          if (p1 != NEG_INF && !(*ring(tau, NE + SPL + k + 1) + c + cst >= -a.beam)) p1 = NEG_INF;
          if (p2 != NEG_INF && !(*ring(tau, NE + SPL + k + 0) + c + cst >= -a.beam)) p2 = NEG_INF;
        }
        if (MODE == MODE_MAX) v = e + fmaxf(p0, fmaxf(p1, p2)) - m_prev;
        else v = e + lse3(p0, p1, p2) - m_prev;
      }
      if (s >= L) v = NEG_INF;
      cur[k] = v;
      local_max = fmaxf(local_max, v);
    }

    // store the row at its natural (frame, position) location
    {
      float* orow = out + cell0 + (long long)t * L;
#pragma unroll
      for (int k = 0; k < SPL; ++k) {
        const int s = s_first + k;
        if (s < L) orow[real_s(s)] = cur[k];
      }
    }
    if (MODE == MODE_MAX && tid == 0) off_out[row0 + t] = C;

#pragma unroll
    for (int k = 0; k < SPL; ++k) prev[k] = cur[k];

    // row maximum and boundary exchange for the next frame
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) local_max = fmaxf(local_max, __shfl_xor_sync(0xffffffffu, local_max, o));
    if (W == 1) {
      m_prev = (local_max == NEG_INF) ? 0.f : local_max;
    } else {
      if (lane == 31) {
        s_tail[tau & 1][warp][0] = cur[SPL - 1];
        s_tail[tau & 1][warp][1] = cur[SPL >= 2 ? SPL - 2 : 0];
      }
      if (lane == 0) s_wmax[tau & 1][warp] = local_max;
      __syncthreads();
    }
  }
  cp_async_wait<0>();

  // ---- total score: positions L-1 and L-2 of the last sweep frame ----
#pragma unroll
  for (int k = 0; k < SPL; ++k) {
    const int s = s_first + k;
    if (s == L - 1 || (s == L - 2 && L >= 2)) {
      float v = prev[k];
      if (MODE == MODE_MASKED) {
        // exit arc (forward) / entry arc (backward): best alignment through this position
        const int t = real_t(T - 1);
        const float p = Pm[cell0 + (long long)t * L + real_s(s)];
        const float c = (float)((dir ? a.off_b[row0 + t] : a.off_a[row0 + t]) - best);
        if (!(p + c >= -a.beam)) v = NEG_INF;
      }
      s_fin[s == L - 1 ? 0 : 1] = v;
    }
  }
  __syncthreads();
  if (tid == 0 && dir == 0) {
    const float f0 = s_fin[0], f1 = s_fin[1];
    if (MODE == MODE_MAX) {
      a.best[n] = C + (double)fmaxf(f0, f1);
    } else {
      const float mx = fmaxf(f0, f1);
      const double ll = C + (double)(mx + __logf(__expf(f0 - mx) + __expf(f1 - mx)));
      const float lossv = (float)(-ll);
      if (isfinite(lossv)) {
        a.loss[n] = lossv;
      } else {
        a.loss[n] = 0.f;
        atomicOr(&a.flags[n], 2);
      }
    }
  }
}

// ---- occupancies (Algorithm 1 line 10, G = -gamma): one warp per stacked frame ----
__global__ void k_gamma(const float* __restrict__ alpha, const float* __restrict__ beta,
                        const float* __restrict__ S, long long ldS, const int* __restrict__ rel_all, int stride,
                        BatchMeta meta, int M, const int* __restrict__ flags,
                        float* __restrict__ gamma, long long ldg, float* __restrict__ roww) {
  const int m = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (m >= M) return;
  const int n = meta.row_utt[m];
  if (flags[n] != 0) { if (lane == 0) roww[m] = 0.f; return; }
  const int t = m - meta.row0[n];
  const int U = meta.U_n[n], L = 2 * U + 1;
  const int* rel = rel_all + (long long)n * stride;
  const float* a = alpha + meta.cell0[n] + (long long)t * L;
  const float* b = beta + meta.cell0[n] + (long long)t * L;
  const float* Srow = S + (long long)m * ldS;
  const float e_blank = Srow[0];

  float mx = NEG_INF;
  for (int s = lane; s < L; s += 32) {
    const float e = (s & 1) ? Srow[rel[(s - 1) >> 1]] : e_blank;
    mx = fmaxf(mx, a[s] + b[s] - e);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float sum = 0.f;
  for (int s = lane; s < L; s += 32) {
    const float e = (s & 1) ? Srow[rel[(s - 1) >> 1]] : e_blank;
    sum += __expf(a[s] + b[s] - e - mx);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if (!(sum > 0.f) || !isfinite(mx)) { if (lane == 0) roww[m] = 0.f; return; }
  const float inv = 1.f / sum;
  float gb = 0.f;
  float* grow = gamma + (long long)m * ldg;
  for (int s = lane; s < L; s += 32) {
    const int c = (s & 1) ? rel[(s - 1) >> 1] : 0;
    const float e = (s & 1) ? Srow[c] : e_blank;
    const float g = __expf(a[s] + b[s] - e - mx) * inv;
    if (s & 1) { if (g != 0.f) atomicAdd(grow + c, g); }
    else gb += g;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) gb += __shfl_xor_sync(0xffffffffu, gb, o);
  if (lane == 0) { grow[0] = gb; roww[m] = 1.f; }
}

// loss_n = sum_t lambda_t - log sum over alignments of exp(sum_t Z[t, pi_t])  (Eq. "ctc-factorization")
__global__ void k_finalize_loss(const float* __restrict__ lambda, BatchMeta meta, float* loss, int* flags,
                                float* roww) {
  __shared__ double s_part[8];
  __shared__ int s_bad;
  const int n = blockIdx.x, tid = threadIdx.x;
  const int r0 = meta.row0[n], T = meta.T_n[n];
  if (flags[n] != 0) return;                 // excluded: loss is already 0, row weights already 0
  double acc = 0.0;
  for (int t = tid; t < T; t += blockDim.x) acc += (double)lambda[r0 + t];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((tid & 31) == 0) s_part[tid >> 5] = acc;
  __syncthreads();
  if (tid == 0) {
    double tot = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot += s_part[w];
    const float l = (float)((double)loss[n] + tot);
    const bool ok = isfinite(l);
    loss[n] = ok ? l : 0.f;
    if (!ok) atomicOr(&flags[n], 2);
    s_bad = ok ? 0 : 1;
  }
  __syncthreads();
  if (s_bad)
    for (int t = tid; t < T; t += blockDim.x) roww[r0 + t] = 0.f;
}

template <int W, int SPL, int MODE>
cudaError_t launch_sweep(const SweepArgs& a, int N, cudaStream_t stream) {
  constexpr int DEPTH = (MODE == MODE_MASKED) ? (SPL >= 8 ? 3 : 4) : 4;   // small enough to share an SM with a GEMM CTA
  constexpr int NE = (SPL == 1) ? 1 : 1 + SPL / 2;
  constexpr int NX = (MODE == MODE_MASKED) ? (2 * SPL + 2) : 0;
  const size_t smem = (size_t)DEPTH * (NE + NX) * W * 32 * sizeof(float);
  auto kern = k_ctc_sweep<W, SPL, DEPTH, MODE>;
  if (smem + 2048 > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  kern<<<dim3(N, 2), W * 32, smem, stream>>>(a);
  return cudaGetLastError();
}

template <int MODE>
cudaError_t dispatch_sweep(const SweepArgs& a, int N, int Lmax, cudaStream_t s) {
  if (Lmax <= 32) return launch_sweep<1, 1, MODE>(a, N, s);
  if (Lmax <= 64) return launch_sweep<1, 2, MODE>(a, N, s);
  if (Lmax <= 128) return launch_sweep<1, 4, MODE>(a, N, s);
  if (Lmax <= 256) return launch_sweep<2, 4, MODE>(a, N, s);
  if (Lmax <= 512) return launch_sweep<4, 4, MODE>(a, N, s);
  if (Lmax <= 1024) return launch_sweep<8, 4, MODE>(a, N, s);
  if (Lmax <= 2048) return launch_sweep<16, 4, MODE>(a, N, s);
  if (Lmax <= 4096) return launch_sweep<16, 8, MODE>(a, N, s);
  return cudaErrorInvalidValue;
}

}  // namespace

int dp_max_states() { return 4096; }

cudaError_t finalize_loss(const float* lambda, const BatchMeta& meta, int N, float* loss, int* utt_flags,
                          float* roww, cudaStream_t stream) {
  k_finalize_loss<<<N, 256, 0, stream>>>(lambda, meta, loss, utt_flags, roww);
  return cudaGetLastError();
}

cudaError_t alignment_dp(const float* S, long long ldS, const int* relabeled, int target_stride,
                         const BatchMeta& meta, int N, int M, int Lmax, float beam,
                         const DpBuffers& buf, float* gamma, long long ld_gamma, const int* Kdev,
                         float* loss, int* utt_flags, cudaStream_t stream) {
  (void)Kdev;
  SweepArgs a{};
  a.S = S; a.ldS = ldS; a.rel = relabeled; a.stride = target_stride;
  a.T_n = meta.T_n; a.U_n = meta.U_n; a.row0 = meta.row0; a.cell0 = meta.cell0;
  a.beam = beam; a.loss = loss; a.flags = utt_flags;
  a.off_a = buf.off_a; a.off_b = buf.off_b; a.best = buf.best;
  const bool use_beam = (beam > 0.f) && isfinite(beam);
  cudaError_t e;
  if (use_beam) {
    a.out_f = buf.va; a.out_b = buf.vb;
    if ((e = dispatch_sweep<MODE_MAX>(a, N, Lmax, stream)) != cudaSuccess) return e;
    a.va = buf.va; a.vb = buf.vb;
    a.out_f = buf.alpha; a.out_b = buf.beta;
    if ((e = dispatch_sweep<MODE_MASKED>(a, N, Lmax, stream)) != cudaSuccess) return e;
  } else {
    a.out_f = buf.alpha; a.out_b = buf.beta;
    if ((e = dispatch_sweep<MODE_LOG>(a, N, Lmax, stream)) != cudaSuccess) return e;
  }
  if ((e = cudaMemsetAsync(gamma, 0, (size_t)M * ld_gamma * sizeof(float), stream)) != cudaSuccess) return e;
  const int warps = 8;
  k_gamma<<<(M + warps - 1) / warps, warps * 32, 0, stream>>>(buf.alpha, buf.beta, S, ldS, relabeled,
                                                                target_stride, meta, M, utt_flags, gamma,
                                                                ld_gamma, buf.roww);
  return cudaGetLastError();
}

}  // namespace pctc
