// Alignment dynamic program on the selected-class logits Z_U (Algorithm 1, lines
// 7-10), with the finite-beam arc pruning of Section 3.3 / Appendix B.3 as an
// option.
//
// The CTC graph of utterance n is the trellis over l' = (blank, y_1, blank, ...,
// y_U, blank): L = 2U+1 positions, T_n frames.  One CTA handles one (utterance,
// direction) pair; the backward recursion is the forward recursion on the
// time- and label-reversed problem, so one kernel serves both.  A CTA of a
// single warp exchanges the two boundary positions between lanes by shuffle;
// wider trellises use several warps and one barrier per frame.  Each thread
// keeps SPL consecutive positions in registers; the emission scores it needs,
// gathered from the row of Z_U, are staged DEPTH frames ahead in shared memory
// with cp.async so that the serial chain never waits on memory.
//
// Scores are base-2 logarithms.  Every NORM frames the row maximum is subtracted
// (its running sum carried in double), so fp32 magnitudes stay O(100) for any T.
// The recursion needs no normaliser: adding a per-frame constant to all
// emissions shifts every alignment equally (Eq. "ctc-factorization"), so the
// caller adds sum_t lambda_t to the loss afterwards.  Occupancies are formed per
// frame as a softmax over positions of alpha + beta - emission, which needs no
// global constant either.
//
// Finite beam: best-alignment (max-semiring) sweeps give a[t,s], b[t,s]; a fully
// parallel kernel turns them into one byte of arc flags per trellis cell, laid out
// in the sweep coordinates of its consumer; the arc-masked sum sweeps then read
// one 32-bit word per four positions and frame.
#include "pctc_internal.h"

#include <math_constants.h>

namespace pctc {

namespace {

#define NEG_INF (-CUDART_INF_F)

constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;
constexpr int DEPTH = 4;      // frames staged ahead
constexpr int NORM = 8;       // renormalise every NORM frames

enum SweepMode : int { MODE_LOG = 0, MODE_MAX = 1, MODE_MASKED = 2 };

struct SweepArgs {
  const float* S; long long ldS;
  const int* rel; int stride;
  const int* T_n; const int* U_n; const int* row0; const long long* cell0; const long long* mcell0;
  float* out_f; float* out_b;              // rows written by the forward / backward sweep
  const unsigned char* mask_f;             // MODE_MASKED: arc flags in forward sweep coordinates
  const unsigned char* mask_b;             //              and in backward sweep coordinates
  double* off_a; double* off_b;            // MODE_MAX: per-frame offsets of the rows written
  double* best;                            // [N] best alignment score (base 2)
  float* loss; int* flags;
  int* status;                             // status word (index checks of the debug build)
};

__device__ __forceinline__ void cp_async4(void* smem_dst, const void* gsrc) {
  unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}
__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2f(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <int W, int SPL, int MODE>
__global__ void __launch_bounds__(W * 32) k_ctc_sweep(SweepArgs a) {
  constexpr int NTH = W * 32;
  constexpr int NE = (SPL == 1) ? 1 : 1 + SPL / 2;                 // emission slots per thread
  constexpr int NM = (MODE == MODE_MASKED) ? SPL / 4 : 0;          // arc-flag words per thread
  constexpr int NSLOT = NE + NM;
  static_assert(MODE != MODE_MASKED || SPL % 4 == 0, "masked sweeps read four positions per word");
  extern __shared__ float s_ring[];                                // [DEPTH][NSLOT][NTH]
  __shared__ __align__(16) float s_wmax[2][W < 4 ? 4 : W];
  __shared__ float s_tail[2][W][2];
  __shared__ float s_fin[2];
  __shared__ int s_rep;

  const int n = blockIdx.x, dir = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int T = a.T_n[n], U = a.U_n[n], L = 2 * U + 1;
  const int* rel = a.rel + (long long)n * a.stride;

  if (tid == 0) { s_rep = 0; s_fin[0] = NEG_INF; s_fin[1] = NEG_INF; }
  if (tid < 2 * (W < 4 ? 4 : W)) (&s_wmax[0][0])[tid] = NEG_INF;
  __syncthreads();
  if (a.flags[n] & (4 | 8)) {                                      // bad target or subset overflow: excluded
    if (dir == 0 && tid == 0 && MODE != MODE_MAX) a.loss[n] = 0.f;
    return;
  }
  {
    int cnt = 0;
    for (int i = tid + 1; i < U; i += NTH) cnt += (rel[i] == rel[i - 1]);
    if (cnt) atomicAdd(&s_rep, cnt);
  }
  __syncthreads();
  if (kCheckBounds) {                                              // every label indexes a column of Z_U
    __shared__ int s_badidx;
    if (tid == 0) s_badidx = 0;
    __syncthreads();
    for (int i = tid; i < U; i += NTH)
      if (!index_ok(rel[i], 0, a.ldS, a.status, 5)) s_badidx = 1;
    __syncthreads();
    if (s_badidx) return;
  }
  if (T < U + s_rep) {                                             // no alignment exists (Appendix B.1)
    if (dir == 0 && tid == 0 && MODE != MODE_MAX) { atomicOr(&a.flags[n], 1); a.loss[n] = 0.f; }
    return;
  }

  // ---- static per-thread description of its positions, in sweep coordinates ----
  const int s_first = tid * SPL;
  auto label_of = [&](int s) -> int {          // s odd, in sweep coordinates
    const int i = (s - 1) >> 1;
    return rel[dir ? (U - 1 - i) : i];
  };
  float skipadd[SPL], validadd[SPL];           // 0 where the s-2 -> s arc / the position exists, else -inf
  int col[NE];
#pragma unroll
  for (int k = 0; k < SPL; ++k) {
    const int s = s_first + k;
    validadd[k] = (s < L) ? 0.f : NEG_INF;
    const bool sk = (s < L) && (s & 1) && s >= 3 && label_of(s) != label_of(s - 2);
    skipadd[k] = sk ? 0.f : NEG_INF;
  }
  if (SPL == 1) {
    col[0] = (s_first < L && (s_first & 1)) ? label_of(s_first) : 0;
  } else {
    col[0] = 0;
#pragma unroll
    for (int q = 1; q < NE; ++q) {
      const int s = s_first + 2 * q - 1;
      col[q] = (s < L) ? label_of(s) : 0;
    }
  }
  const float edgeadd = (tid == 0) ? NEG_INF : 0.f;

  const long long cell0 = a.cell0[n];
  const int row0 = a.row0[n];
  const int t_first = dir ? (T - 1) : 0;
  const long long tstep = dir ? -1 : 1;

  // running source pointers of the staged loads (advance one frame per issue)
  const float* esrc[NE];
#pragma unroll
  for (int q = 0; q < NE; ++q) esrc[q] = a.S + (long long)(row0 + t_first) * a.ldS + col[q];
  const long long estep = tstep * a.ldS;
  const unsigned* msrc = nullptr;
  int mstep = 0;
  if (MODE == MODE_MASKED) {
    const int Lp4 = (L + 3) & ~3;
    const unsigned char* mb = (dir ? a.mask_b : a.mask_f) + a.mcell0[n];
    msrc = reinterpret_cast<const unsigned*>(mb) + (s_first >> 2);
    mstep = Lp4 >> 2;
  }
  float* ring_base = s_ring + tid;
  int issued = 0;
  auto issue = [&]() {
    if (issued < T) {
      float* dst = ring_base + (size_t)(issued & (DEPTH - 1)) * NSLOT * NTH;
#pragma unroll
      for (int q = 0; q < NE; ++q) { cp_async4(dst + q * NTH, esrc[q]); esrc[q] += estep; }
      if (MODE == MODE_MASKED) {
#pragma unroll
        for (int q = 0; q < NM; ++q)
          if (s_first + 4 * q < L) cp_async4(dst + (NE + q) * NTH, msrc + q);
        msrc += mstep;
      }
    }
    ++issued;
    cp_async_commit();
  };
#pragma unroll
  for (int i = 0; i < DEPTH - 1; ++i) issue();

  float prev[SPL];
#pragma unroll
  for (int k = 0; k < SPL; ++k) prev[k] = NEG_INF;
  double C = 0.0;              // sum of the row maxima subtracted so far (thread 0)
  float* out = (dir ? a.out_b : a.out_f) + cell0 + (long long)t_first * L + (dir ? (L - 1 - s_first) : s_first);
  const long long ostep = tstep * L;
  double* off_out = nullptr;
  if (MODE == MODE_MAX) off_out = (dir ? a.off_b : a.off_a) + row0 + t_first;

  for (int tau = 0; tau < T; ++tau) {
    issue();
    cp_async_wait<DEPTH - 1>();
    const float* slot = ring_base + (size_t)(tau & (DEPTH - 1)) * NSLOT * NTH;

    // positions s_first-1 and s_first-2 of the previous frame
    float n1 = NEG_INF, n2 = NEG_INF, msub = 0.f;
    if (tau > 0) {
      if (SPL == 1) {
        n1 = __shfl_up_sync(0xffffffffu, prev[0], 1);
        n2 = __shfl_up_sync(0xffffffffu, prev[0], 2);
        if (lane < 1) n1 = NEG_INF;
        if (lane < 2) n2 = NEG_INF;
      } else {
        n1 = __shfl_up_sync(0xffffffffu, prev[SPL - 1], 1);
        n2 = __shfl_up_sync(0xffffffffu, prev[SPL >= 2 ? SPL - 2 : 0], 1);
        if (W > 1 && lane == 0 && warp > 0) {
          n1 = s_tail[(tau + 1) & 1][warp - 1][0];
          n2 = s_tail[(tau + 1) & 1][warp - 1][1];
        }
        n1 += edgeadd;
        n2 += edgeadd;
      }
      if ((tau & (NORM - 1)) == 0) {           // the previous frame published its row maximum
        const float4* wm = reinterpret_cast<const float4*>(s_wmax[(tau / NORM) & 1]);
        float4 v4 = wm[0];
        float mx = fmaxf(fmaxf(v4.x, v4.y), fmaxf(v4.z, v4.w));
#pragma unroll
        for (int w4 = 1; w4 < (W + 3) / 4; ++w4) {
          v4 = wm[w4];
          mx = fmaxf(mx, fmaxf(fmaxf(v4.x, v4.y), fmaxf(v4.z, v4.w)));
        }
        msub = (mx == NEG_INF) ? 0.f : mx;
        if (tid == 0) C += (double)msub;
      }
    }

    unsigned mword[NM > 0 ? NM : 1];
    if (MODE == MODE_MASKED) {
#pragma unroll
      for (int q = 0; q < NM; ++q) mword[q] = __float_as_uint(slot[(NE + q) * NTH]);
    }
    const float e_blank = slot[0] * LOG2E;
    float cur[SPL];
    float local_max = NEG_INF;
#pragma unroll
    for (int k = 0; k < SPL; ++k) {
      float e2;
      if (SPL == 1) e2 = e_blank;
      else e2 = (k & 1) ? slot[((k + 1) / 2) * NTH] * LOG2E : e_blank;
      unsigned bits = 0x1f;
      if (MODE == MODE_MASKED) bits = (mword[k >> 2] >> (8 * (k & 3))) & 0xffu;
      float v;
      if (tau == 0) {
        const int s = s_first + k;
        v = (s <= 1 && (bits & 8u)) ? e2 : NEG_INF;
      } else {
        float p0 = prev[k];
        float p1 = (SPL == 1) ? n1 : ((k >= 1) ? prev[k >= 1 ? k - 1 : 0] : n1);
        float p2 = (SPL == 1) ? n2 : ((k >= 2) ? prev[k >= 2 ? k - 2 : 0] : (k == 1 ? n1 : n2));
        p2 += skipadd[k];
        if (MODE == MODE_MASKED) {
          if (!(bits & 1u)) p0 = NEG_INF;
          if (!(bits & 2u)) p1 = NEG_INF;
          if (!(bits & 4u)) p2 = NEG_INF;
        }
        const float mx = fmaxf(p0, fmaxf(p1, p2));
        if (MODE == MODE_MAX) {
          v = e2 + mx - msub;
        } else {
          const float sh = fmaxf(mx, -1e30f);      // keeps (-inf) - (-inf) out of the exponentials
          v = (e2 - msub) + sh + lg2f(ex2f(p0 - sh) + ex2f(p1 - sh) + ex2f(p2 - sh));
        }
      }
      v += validadd[k];
      cur[k] = v;
      local_max = fmaxf(local_max, v);
    }

    // store the row at its natural (frame, position) location
#pragma unroll
    for (int k = 0; k < SPL; ++k)
      if (s_first + k < L) out[dir ? -k : k] = cur[k];
    out += ostep;
    if (MODE == MODE_MAX) {
      if (tid == 0) *off_out = C;
      off_out += tstep;
    }
#pragma unroll
    for (int k = 0; k < SPL; ++k) prev[k] = cur[k];

    // publish the row maximum (every NORM frames) and the boundary positions for the next frame
    if ((tau & (NORM - 1)) == NORM - 1) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) local_max = fmaxf(local_max, __shfl_xor_sync(0xffffffffu, local_max, o));
      if (lane == 0) s_wmax[((tau + 1) / NORM) & 1][warp] = local_max;
    }
    if (W == 1) {
      __syncwarp();
    } else {
      if (lane == 31) {
        s_tail[tau & 1][warp][0] = cur[SPL - 1];
        s_tail[tau & 1][warp][1] = cur[SPL >= 2 ? SPL - 2 : 0];
      }
      __syncthreads();
    }
  }
  cp_async_wait<0>();

  // ---- total score: positions L-1 and L-2 of the last sweep frame ----
  unsigned last_bits[SPL];
#pragma unroll
  for (int k = 0; k < SPL; ++k) last_bits[k] = 0x1f;
  if (MODE == MODE_MASKED) {
    const float* slot = ring_base + (size_t)((T - 1) & (DEPTH - 1)) * NSLOT * NTH;
#pragma unroll
    for (int k = 0; k < SPL; ++k)
      last_bits[k] = (s_first + k < L) ? ((__float_as_uint(slot[(NE + (k >> 2)) * NTH]) >> (8 * (k & 3))) & 0xffu) : 0u;
  }
#pragma unroll
  for (int k = 0; k < SPL; ++k) {
    const int s = s_first + k;
    if (s == L - 1 || (s == L - 2 && L >= 2)) {
      float v = prev[k];
      if (MODE == MODE_MASKED && !(last_bits[k] & 16u)) v = NEG_INF;   // exit arc dropped
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
      const float sh = fmaxf(mx, -1e30f);
      const double ll2 = C + (double)(sh + lg2f(ex2f(f0 - sh) + ex2f(f1 - sh)));
      const float lossv = (float)(-ll2 * (double)LN2);      // minus the log-sum over alignments of exp(sum Z_U)
      if (isfinite(lossv)) {
        a.loss[n] = lossv;
      } else {
        a.loss[n] = 0.f;
        atomicOr(&a.flags[n], 2);
      }
    }
  }
}

// ---- finite beam: arc flags from the best-alignment scores (Appendix B.3) ----------------------
// One CTA per stacked frame.  Flags of cell (t,s), bit j (j = 0,1,2): the arc into the cell from
// position s-j of the previous sweep frame is kept; bit 3: the sweep may start here; bit 4: the
// sweep may end here.  An arc (t-1,s') -> (t,s) is kept iff a[t-1,s'] + b[t,s] >= best - beam.
// The same expression, in the same operand order, feeds both layouts, so the forward and the
// backward sweep see one lattice.
__global__ void k_arc_flags(const float* __restrict__ va, const float* __restrict__ vb,
                            const double* __restrict__ off_a, const double* __restrict__ off_b,
                            const double* __restrict__ best_all, BatchMeta meta, const long long* __restrict__ mcell0,
                            const int* __restrict__ flags, float beam2, unsigned char* __restrict__ mask_f,
                            unsigned char* __restrict__ mask_b) {
  const int m = blockIdx.x;
  const int n = meta.row_utt[m];
  if (!index_ok(n, 0, meta.N, meta.status, 6)) return;
  if (flags[n] != 0) return;
  const int r0 = meta.row0[n], t = m - r0, T = meta.T_n[n];
  if (!index_ok(t, 0, T, meta.status, 6)) return;
  const int L = 2 * meta.U_n[n] + 1, Lp4 = (L + 3) & ~3;
  const double best = best_all[n];
  const float* a_prev = va + meta.cell0[n] + (long long)(t - 1) * L;   // read for t >= 1 only
  const float* a_cur = va + meta.cell0[n] + (long long)t * L;
  const float* b_cur = vb + meta.cell0[n] + (long long)t * L;
  const float* b_next = vb + meta.cell0[n] + (long long)(t + 1) * L;    // read for t <= T-2 only
  const float cst_in = (t >= 1) ? (float)(off_a[m - 1] + off_b[m] - best) : 0.f;
  const float cst_out = (t <= T - 2) ? (float)(off_a[m] + off_b[m + 1] - best) : 0.f;
  const float cst_entry = (float)(off_b[m] - best);   // used at t == 0
  const float cst_exit = (float)(off_a[m] - best);    // used at t == T-1
  unsigned char* mf = mask_f + mcell0[n] + (long long)t * Lp4;
  unsigned char* mb = mask_b + mcell0[n] + (long long)(T - 1 - t) * Lp4;
  for (int s = threadIdx.x; s < Lp4; s += blockDim.x) {
    unsigned f = 0, b = 0;
    if (s < L) {
      const float bc = b_cur[s], ac = a_cur[s];
      const bool entry = (t == 0) && (bc + cst_entry >= -beam2);
      const bool exit_ = (t == T - 1) && (ac + cst_exit >= -beam2);
      if (t >= 1) {
#pragma unroll
        for (int j = 0; j < 3; ++j)
          if (s - j >= 0 && (a_prev[s - j] + bc) + cst_in >= -beam2) f |= 1u << j;
      }
      if (t <= T - 2) {
#pragma unroll
        for (int j = 0; j < 3; ++j)
          if (s + j < L && (ac + b_next[s + j]) + cst_out >= -beam2) b |= 1u << j;
      }
      if (entry) { f |= 8u; b |= 16u; }
      if (exit_) { f |= 16u; b |= 8u; }
      mb[L - 1 - s] = (unsigned char)b;
    }
    mf[s] = (unsigned char)f;
    if (s >= L) mb[s] = 0;
  }
}

// ---- positions that carry the same label ---------------------------------------------------------
// The occupancy of a class is the sum over the positions that carry it (Section 3.2).  To add them
// in a fixed order without atomics, every label position i of an utterance gets a link word: the low
// 16 bits hold 1 + the next position with the same label (0: none), bit 16 says that an earlier
// position carries the label too.  The first position of a label then sums its chain in ascending
// order.  One CTA per utterance; depends on the relabelled targets only.
constexpr int LINK_HAS_PREV = 1 << 16;
constexpr int LINK_MAX_U = 2048;               // >= (dp_max_states() - 1) / 2

__global__ void k_repeat_links(const int* __restrict__ rel_all, int stride, const int* __restrict__ U_n,
                               const int* __restrict__ flags, int* __restrict__ links_all) {
  __shared__ int s_rel[LINK_MAX_U];
  __shared__ int s_prev[LINK_MAX_U];
  const int n = blockIdx.x;
  if (flags[n] & (4 | 8)) return;              // excluded utterance: its labels may be -1, nobody reads its links
  const int U = min(U_n[n], LINK_MAX_U);
  const int* rel = rel_all + (long long)n * stride;
  int* links = links_all + (long long)n * stride;
  for (int i = threadIdx.x; i < U; i += blockDim.x) { s_rel[i] = rel[i]; s_prev[i] = 0; }
  __syncthreads();
  for (int i = threadIdx.x; i < U; i += blockDim.x) {
    const int c = s_rel[i];
    int nxt = 0;
    for (int j = i + 1; j < U; ++j)
      if (s_rel[j] == c) { nxt = j + 1; break; }
    links[i] = nxt;
    if (nxt) s_prev[nxt - 1] = 1;              // a position has at most one predecessor in its chain
  }
  __syncthreads();
  for (int i = threadIdx.x; i < U; i += blockDim.x)
    if (s_prev[i]) links[i] |= LINK_HAS_PREV;
}

// ---- occupancies (Algorithm 1 line 10, G = -gamma): one warp per stacked frame ----
__global__ void k_gamma(const float* __restrict__ alpha, const float* __restrict__ beta,
                        const float* __restrict__ S, long long ldS, const int* __restrict__ rel_all, int stride,
                        BatchMeta meta, int M, const int* __restrict__ flags,
                        float* __restrict__ gamma, long long ldg, float* __restrict__ roww,
                        const float* __restrict__ utt_weights, const int* __restrict__ links_all) {
  const int m = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (m >= M) return;
  const int n = meta.row_utt[m];
  if (!index_ok(n, 0, meta.N, meta.status, 7)) return;
  if (flags[n] != 0) { if (lane == 0) roww[m] = 0.f; return; }
  const int t = m - meta.row0[n];
  const int U = meta.U_n[n], L = 2 * U + 1;
  if (!index_ok(t, 0, meta.T_n[n], meta.status, 7)) return;
  if (kCheckBounds) {                          // labels index the row of Z_U and of gamma; links stay inside the utterance
    bool bad = false;
    for (int i = lane; i < U; i += 32) {
      const int nxt = (links_all[(long long)n * stride + i] & 0xffff) - 1;
      if (!index_ok(rel_all[(long long)n * stride + i], 0, ldg < ldS ? ldg : ldS, meta.status, 7) ||
          !index_ok(nxt, -1, U, meta.status, 7) || (nxt >= 0 && nxt <= i && !index_ok(-1, 0, 1, meta.status, 7)))
        bad = true;
    }
    if (__any_sync(0xffffffffu, bad)) return;
  }
  const int* rel = rel_all + (long long)n * stride;
  const float* a = alpha + meta.cell0[n] + (long long)t * L;
  const float* b = beta + meta.cell0[n] + (long long)t * L;
  const float* Srow = S + (long long)m * ldS;
  const float e_blank = Srow[0] * LOG2E;

  float mx = NEG_INF;
  for (int s = lane; s < L; s += 32) {
    const float e = (s & 1) ? Srow[rel[(s - 1) >> 1]] * LOG2E : e_blank;
    mx = fmaxf(mx, a[s] + b[s] - e);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float sum = 0.f;
  for (int s = lane; s < L; s += 32) {
    const float e = (s & 1) ? Srow[rel[(s - 1) >> 1]] * LOG2E : e_blank;
    sum += ex2f(a[s] + b[s] - e - mx);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if (!(sum > 0.f) || !isfinite(mx)) { if (lane == 0) roww[m] = 0.f; return; }
  const float inv = 1.f / sum;
  float gb = 0.f;
  float* grow = gamma + (long long)m * ldg;
  const int* links = links_all + (long long)n * stride;
  for (int s = lane; s < L; s += 32) {
    if (s & 1) {
      // label position i: the first position of a label adds up the positions that carry it, in
      // ascending order (a fixed order: repeated calls give the same bits), and stores the sum
      const int i = (s - 1) >> 1;
      int link = links[i];
      if (link & LINK_HAS_PREV) continue;
      const int c = rel[i];
      const float e = Srow[c] * LOG2E;
      float g = ex2f(a[s] + b[s] - e - mx);
      for (int j = (link & 0xffff) - 1; j >= 0; j = (links[j] & 0xffff) - 1) {
        const int s2 = 2 * j + 1;
        g += ex2f(a[s2] + b[s2] - e - mx);
      }
      grow[c] = g * inv;
    } else {
      gb += ex2f(a[s] + b[s] - e_blank - mx) * inv;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) gb += __shfl_xor_sync(0xffffffffu, gb, o);
  if (lane == 0) { grow[0] = gb; roww[m] = utt_weights ? utt_weights[n] : 1.f; }
}

// loss_n = sum_t lambda_t - log sum over alignments of exp(sum_t Z[t, pi_t])  (Eq. "ctc-factorization")
__global__ void k_finalize_loss(const float* __restrict__ lambda, BatchMeta meta, float* loss, int* flags,
                                float* roww) {
  __shared__ double s_part[8];
  __shared__ int s_bad;
  const int n = blockIdx.x, tid = threadIdx.x;
  const int r0 = meta.row0[n], T = meta.T_n[n];
  if (!index_ok((long long)r0 + T, 1, (long long)meta.M + 1, meta.status, 8)) return;
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
  constexpr int NE = (SPL == 1) ? 1 : 1 + SPL / 2;
  constexpr int NM = (MODE == MODE_MASKED) ? SPL / 4 : 0;
  const size_t smem = (size_t)DEPTH * (NE + NM) * W * 32 * sizeof(float);   // <= 56 KB
  auto kern = k_ctc_sweep<W, SPL, MODE>;
  if (smem + 2048 > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  kern<<<dim3(N, 2), W * 32, smem, stream>>>(a);
  return cudaGetLastError();
}

template <int MODE>
cudaError_t dispatch_sweep(const SweepArgs& a, int N, int Lmax, cudaStream_t s) {
  if (MODE != MODE_MASKED) {
    constexpr int M2 = (MODE == MODE_MASKED) ? MODE_LOG : MODE;   // narrow trellises: one position per lane
    if (Lmax <= 32) return launch_sweep<1, 1, M2>(a, N, s);
    if (Lmax <= 64) return launch_sweep<1, 2, M2>(a, N, s);
  }
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
  a.T_n = meta.T_n; a.U_n = meta.U_n; a.row0 = meta.row0; a.cell0 = meta.cell0; a.mcell0 = buf.mcell0;
  a.loss = loss; a.flags = utt_flags; a.status = meta.status;
  a.off_a = buf.off_a; a.off_b = buf.off_b; a.best = buf.best;
  const bool use_beam = (beam > 0.f) && isfinite(beam);
  cudaError_t e;
  if (use_beam) {
    a.out_f = buf.va; a.out_b = buf.vb;
    if ((e = dispatch_sweep<MODE_MAX>(a, N, Lmax, stream)) != cudaSuccess) return e;
    k_arc_flags<<<M, 256, 0, stream>>>(buf.va, buf.vb, buf.off_a, buf.off_b, buf.best, meta, buf.mcell0, utt_flags,
                                       beam * LOG2E, buf.mask_f, buf.mask_b);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    a.mask_f = buf.mask_f; a.mask_b = buf.mask_b;
    a.out_f = buf.alpha; a.out_b = buf.beta;
    if ((e = dispatch_sweep<MODE_MASKED>(a, N, Lmax, stream)) != cudaSuccess) return e;
  } else {
    a.out_f = buf.alpha; a.out_b = buf.beta;
    if ((e = dispatch_sweep<MODE_LOG>(a, N, Lmax, stream)) != cudaSuccess) return e;
  }
  if ((e = cudaMemsetAsync(gamma, 0, (size_t)M * ld_gamma * sizeof(float), stream)) != cudaSuccess) return e;
  k_repeat_links<<<N, 256, 0, stream>>>(relabeled, target_stride, meta.U_n, utt_flags, buf.links);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  const int warps = 8;
  k_gamma<<<(M + warps - 1) / warps, warps * 32, 0, stream>>>(buf.alpha, buf.beta, S, ldS, relabeled,
                                                                target_stride, meta, M, utt_flags, gamma,
                                                                ld_gamma, buf.roww, buf.utt_weights, buf.links);
  return cudaGetLastError();
}

}  // namespace pctc
