// fp32-FMA contraction with the fused epilogues of Algorithm 1.
//
// This is the arithmetic path of fp32 problems (tensor-core bf16/tf32 products
// cannot meet the fp32 tolerances), and, with bf16 operands widened to fp32, the
// on-device cross-check of the tcgen05 path.  acc(i,j) = sum_k A(i,k) B(j,k) over
// 128x128 output tiles (64x64 when the problem has too few of those to fill the
// device), 16-wide k steps staged through shared memory (the next step's operands
// are fetched into registers while the current one is multiplied), 8x8 (4x4)
// accumulators per thread read from shared memory as float4.
#include "pctc_internal.h"

#include <math_constants.h>

namespace pctc {

namespace {

#ifndef PCTC_TUNE_SIMT_CTAS
#define PCTC_TUNE_SIMT_CTAS 1      // resident CTAs per SM the register budget is set for (2 spills, no faster)
#endif

constexpr int TK = 16, NT = 256;

template <typename T> __device__ __forceinline__ float ldf(const T* p) { return float(*p); }

template <typename T>
__device__ __forceinline__ float bias_at(const void* bias, long long v) {
  return bias ? float(reinterpret_cast<const T*>(bias)[v]) : 0.f;
}

// The thread's r-th row (or column) inside the tile: two groups of four, 64 apart, so that a
// quarter warp reads 128 contiguous bytes of a staged k-row with one 16-byte load per thread.
__device__ __forceinline__ int micro(int t, int r) { return (r >> 2) * 64 + t * 4 + (r & 3); }

// One CTA computes column tiles jt_begin..jt_end-1 of row tile blockIdx.y; only the LSE and arg-max
// epilogues walk more than one column tile (they keep their running state across them).
template <typename T, int EPI, int TS>
__global__ void __launch_bounds__(NT, TS == 64 ? 3 : PCTC_TUNE_SIMT_CTAS) k_simt_gemm(const T* __restrict__ A, const T* __restrict__ B,
                                                  GemmShape g, Epilogue e, int tiles_per_cta) {
  constexpr int TM = TS, TN = TS;                 // tile: 64 or 128 square
  constexpr int RM = TS / 16, RN = TS / 16;       // accumulators per thread: rows x columns
  constexpr int LDT = TS + 4;                     // padded pitch of a staged k-row
  constexpr int PER_THREAD = (TS * TK) / NT;      // operand elements each thread stages per k step
  __shared__ __align__(16) float As[TK][LDT];
  __shared__ __align__(16) float Bs[TK][LDT];
  __shared__ float s_red[2][TM][17];

  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const int i0 = blockIdx.y * TM;
  const int ntiles = (g.n + TN - 1) / TN;
  const int jt_begin = blockIdx.x * tiles_per_cta;
  const int jt_end = min(ntiles, jt_begin + tiles_per_cta);
  const int Kdev = (EPI == EPI_SUBSET_LOGP) ? *e.Kdev : 0;

  // where this thread's staged elements sit in a tile: k fastest for a k-contiguous operand, the
  // row (column) index fastest otherwise, so that neighbouring threads read neighbouring addresses.
  // Element q of the thread is (base + q * step) in the slower index; the faster one is fixed.
  const bool a_kc = g.a_k == 1, b_kc = g.b_k == 1;
  const int a_k0 = a_kc ? tid % TK : tid / TM, a_i0 = a_kc ? tid / TK : tid % TM;
  const int b_k0 = b_kc ? tid % TK : tid / TN, b_j0 = b_kc ? tid / TK : tid % TN;
  const int a_dk = a_kc ? 0 : NT / TM, a_di = a_kc ? NT / TK : 0;
  const int b_dk = b_kc ? 0 : NT / TN, b_dj = b_kc ? NT / TK : 0;

  float run_max[RM], run_sum[RM];
  int run_idx[RM];
#pragma unroll
  for (int r = 0; r < RM; ++r) { run_max[r] = -CUDART_INF_F; run_sum[r] = 0.f; run_idx[r] = -1; }

  for (int jt = jt_begin; jt < jt_end; ++jt) {
    const int j0 = jt * TN;
    if (EPI == EPI_SUBSET_LOGP && j0 >= Kdev) break;
    float acc[RM][RN];
#pragma unroll
    for (int r = 0; r < RM; ++r)
#pragma unroll
      for (int c = 0; c < RN; ++c) acc[r][c] = 0.f;

    float pa[PER_THREAD], pb[PER_THREAD];
    auto fetch = [&](int k0) {
#pragma unroll
      for (int q = 0; q < PER_THREAD; ++q) {
        const int gi = i0 + a_i0 + q * a_di, gk = k0 + a_k0 + q * a_dk;
        pa[q] = (gi < g.m && gk < g.k) ? ldf(A + (long long)gi * g.a_i + (long long)gk * g.a_k) : 0.f;
        const int gj = j0 + b_j0 + q * b_dj, gk2 = k0 + b_k0 + q * b_dk;
        pb[q] = (gj < g.n && gk2 < g.k) ? ldf(B + (long long)gj * g.b_j + (long long)gk2 * g.b_k) : 0.f;
      }
    };
    fetch(0);
    for (int k0 = 0; k0 < g.k; k0 += TK) {
#pragma unroll
      for (int q = 0; q < PER_THREAD; ++q) {
        As[a_k0 + q * a_dk][a_i0 + q * a_di] = pa[q];
        Bs[b_k0 + q * b_dk][b_j0 + q * b_dj] = pb[q];
      }
      __syncthreads();
      if (k0 + TK < g.k) fetch(k0 + TK);          // in flight while this step is multiplied
#pragma unroll
      for (int kk = 0; kk < TK; ++kk) {
        float a[RM], b[RN];
#pragma unroll
        for (int h = 0; h < RM / 4; ++h) {
          const float4 av = *reinterpret_cast<const float4*>(&As[kk][h * 64 + ty * 4]);
          const float4 bv = *reinterpret_cast<const float4*>(&Bs[kk][h * 64 + tx * 4]);
          a[h * 4 + 0] = av.x; a[h * 4 + 1] = av.y; a[h * 4 + 2] = av.z; a[h * 4 + 3] = av.w;
          b[h * 4 + 0] = bv.x; b[h * 4 + 1] = bv.y; b[h * 4 + 2] = bv.z; b[h * 4 + 3] = bv.w;
        }
#pragma unroll
        for (int r = 0; r < RM; ++r)
#pragma unroll
          for (int c = 0; c < RN; ++c) acc[r][c] = fmaf(a[r], b[c], acc[r][c]);
      }
      __syncthreads();
    }

    // ---- epilogue for this tile ----
#pragma unroll
    for (int r = 0; r < RM; ++r) {
      const int i = i0 + micro(ty, r);
      if (i >= g.m) continue;
      float lam = 0.f, w = 0.f;
      if (EPI == EPI_DLOGITS || (EPI == EPI_SUBSET_LOGP && e.lambda)) lam = e.lambda[i];
      if (EPI == EPI_DLOGITS) w = e.roww[i];
#pragma unroll
      for (int c = 0; c < RN; ++c) {
        const int j = j0 + micro(tx, c);
        if (j >= g.n) continue;
        const float a = acc[r][c];
        if (EPI == EPI_STORE_F32) {
          reinterpret_cast<float*>(e.out)[(long long)i * e.ld + j] = a;
        } else if (EPI == EPI_LSE_PARTIAL) {
          const float z = a + bias_at<T>(e.bias, e.v0 + j);
          if (z > run_max[r]) {
            run_sum[r] = run_sum[r] * __expf(run_max[r] - z) + 1.f;
            run_max[r] = z;
          } else {
            run_sum[r] += __expf(z - run_max[r]);
          }
        } else if (EPI == EPI_ARGMAX_PARTIAL) {
          const float z = a + bias_at<T>(e.bias, e.v0 + j);
          if (z > run_max[r]) { run_max[r] = z; run_idx[r] = j; }     // ascending j: first maximum wins
        } else if (EPI == EPI_SUBSET_LOGP) {
          if (j < Kdev && index_ok(e.U[j], 0, e.vocab, e.status, 10))
            reinterpret_cast<float*>(e.out)[(long long)i * e.ld + j] = a + bias_at<T>(e.bias, e.U[j]) - lam;
        } else if (EPI == EPI_DLOGITS) {
          const long long v = e.v0 + j;
          const float p = __expf(a + bias_at<T>(e.bias, v) - lam);
          int jj = e.vmap[v];
          if (!index_ok(jj, -1, e.ld_gamma, e.status, 9)) jj = -1;
          const float gam = (jj >= 0) ? e.gamma[(long long)i * e.ld_gamma + jj] : 0.f;
          reinterpret_cast<T*>(e.out)[(long long)i * e.ld + j] = T(w == 0.f ? 0.f : w * (p - gam));
        } else if (EPI == EPI_ACCUM_F32) {
          float* dst = reinterpret_cast<float*>(e.out) + (long long)i * e.ld + j;
          *dst = e.accumulate ? (*dst + a) : a;
        } else if (EPI == EPI_STORE_OUT) {
          T* dst = reinterpret_cast<T*>(e.out) + (long long)i * e.ld + j;
          *dst = e.accumulate ? T(float(*dst) + a) : T(a);
        }
      }
    }
  }

  if (EPI == EPI_ARGMAX_PARTIAL) {
    __shared__ int s_idx[TM][17];
#pragma unroll
    for (int r = 0; r < RM; ++r) { s_red[0][micro(ty, r)][tx] = run_max[r]; s_idx[micro(ty, r)][tx] = run_idx[r]; }
    __syncthreads();
    if (tid < TM) {
      const int i = i0 + tid;
      if (i < g.m) {
        float best = -CUDART_INF_F;
        int idx = -1;
        for (int q = 0; q < 16; ++q) {
          const float v = s_red[0][tid][q];
          const int j = s_idx[tid][q];
          if (j >= 0 && (v > best || (v == best && j < idx) || idx < 0)) { best = v; idx = j; }
        }
        e.partial[(long long)i * (e.partial_stride ? e.partial_stride : e.nsplit) + e.partial_offset + blockIdx.x] =
            make_float2(best, __int_as_float(idx));
      }
    }
  }
  if (EPI == EPI_LSE_PARTIAL) {
    // merge the 16 threads that share a row, in a fixed order
#pragma unroll
    for (int r = 0; r < RM; ++r) {
      s_red[0][micro(ty, r)][tx] = run_max[r];
      s_red[1][micro(ty, r)][tx] = run_sum[r];
    }
    __syncthreads();
    if (tid < TM) {
      const int i = i0 + tid;
      if (i < g.m) {
        float mx = -CUDART_INF_F;
        for (int q = 0; q < 16; ++q) mx = fmaxf(mx, s_red[0][tid][q]);
        float sum = 0.f;
        for (int q = 0; q < 16; ++q)
          if (!(s_red[1][tid][q] <= 0.f)) sum += s_red[1][tid][q] * __expf(s_red[0][tid][q] - mx);
        e.partial[(long long)i * (e.partial_stride ? e.partial_stride : e.nsplit) + e.partial_offset + blockIdx.x] =
            make_float2(mx, sum);
      }
    }
  }
}

template <typename T, int EPI, int TS>
cudaError_t launch_ts(const void* A, const void* B, const GemmShape& g, const Epilogue& e, cudaStream_t stream) {
  const int ntiles = (g.n + TS - 1) / TS;
  int tiles_per_cta = 1, gx = ntiles;
  if (EPI == EPI_LSE_PARTIAL || EPI == EPI_ARGMAX_PARTIAL) {
    tiles_per_cta = (ntiles + e.nsplit - 1) / e.nsplit;
    gx = e.nsplit;
  }
  dim3 grid(gx, (g.m + TS - 1) / TS);
  if (grid.x == 0 || grid.y == 0) return cudaSuccess;
  k_simt_gemm<T, EPI, TS><<<grid, NT, 0, stream>>>((const T*)A, (const T*)B, g, e, tiles_per_cta);
  return cudaGetLastError();
}

// Large tiles once there are enough of them for every SM to hold two; small ones below that.
template <typename T, int EPI>
cudaError_t launch(const void* A, const void* B, const GemmShape& g, const Epilogue& e, cudaStream_t stream) {
  const long long big_tiles = (long long)((g.m + 127) / 128) * ((g.n + 127) / 128);
  if (big_tiles >= 296) return launch_ts<T, EPI, 128>(A, B, g, e, stream);
  return launch_ts<T, EPI, 64>(A, B, g, e, stream);
}

template <typename T>
cudaError_t dispatch(const void* A, const void* B, const GemmShape& g, const Epilogue& e, cudaStream_t s) {
  switch (e.kind) {
    case EPI_STORE_F32: return launch<T, EPI_STORE_F32>(A, B, g, e, s);
    case EPI_LSE_PARTIAL: return launch<T, EPI_LSE_PARTIAL>(A, B, g, e, s);
    case EPI_SUBSET_LOGP: return launch<T, EPI_SUBSET_LOGP>(A, B, g, e, s);
    case EPI_DLOGITS: return launch<T, EPI_DLOGITS>(A, B, g, e, s);
    case EPI_ACCUM_F32: return launch<T, EPI_ACCUM_F32>(A, B, g, e, s);
    case EPI_STORE_OUT: return launch<T, EPI_STORE_OUT>(A, B, g, e, s);
    case EPI_ARGMAX_PARTIAL: return launch<T, EPI_ARGMAX_PARTIAL>(A, B, g, e, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t simt_gemm(const void* A, const void* B, bool operands_bf16, const GemmShape& g,
                      const Epilogue& e, cudaStream_t stream) {
  return operands_bf16 ? dispatch<__nv_bfloat16>(A, B, g, e, stream) : dispatch<float>(A, B, g, e, stream);
}

}  // namespace pctc
