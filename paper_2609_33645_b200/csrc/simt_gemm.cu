// fp32-FMA contraction with the fused epilogues of Algorithm 1.
//
// This is the arithmetic path of fp32 problems (tensor-core bf16/tf32 products
// cannot meet the fp32 tolerances), and, with bf16 operands widened to fp32, the
// on-device cross-check of the tcgen05 path.  acc(i,j) = sum_k A(i,k) B(j,k) over
// 64x64 output tiles, 16-wide k steps staged through shared memory, 4x4
// accumulators per thread.
#include "pctc_internal.h"

#include <math_constants.h>

namespace pctc {

namespace {

constexpr int TM = 64, TN = 64, TK = 16, NT = 256;

template <typename T> __device__ __forceinline__ float ldf(const T* p) { return float(*p); }

template <typename T>
__device__ __forceinline__ float bias_at(const void* bias, long long v) {
  return bias ? float(reinterpret_cast<const T*>(bias)[v]) : 0.f;
}

// One CTA computes column tiles jt_begin..jt_end-1 of row tile blockIdx.y; only the LSE epilogue
// walks more than one column tile (it keeps its running (max, sum) across them).
template <typename T, int EPI>
__global__ void __launch_bounds__(NT) k_simt_gemm(const T* __restrict__ A, const T* __restrict__ B,
                                                  GemmShape g, Epilogue e, int tiles_per_cta) {
  __shared__ float As[TK][TM + 4];
  __shared__ float Bs[TK][TN + 4];
  __shared__ float s_red[2][TM][17];

  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const int i0 = blockIdx.y * TM;
  const int ntiles = (g.n + TN - 1) / TN;
  const int jt_begin = blockIdx.x * tiles_per_cta;
  const int jt_end = min(ntiles, jt_begin + tiles_per_cta);
  const int Kdev = (EPI == EPI_SUBSET_LOGP) ? *e.Kdev : 0;

  float run_max[4], run_sum[4];
  int run_idx[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) { run_max[r] = -CUDART_INF_F; run_sum[r] = 0.f; run_idx[r] = -1; }

  for (int jt = jt_begin; jt < jt_end; ++jt) {
    const int j0 = jt * TN;
    if (EPI == EPI_SUBSET_LOGP && j0 >= Kdev) break;
    float acc[4][4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[r][c] = 0.f;

    for (int k0 = 0; k0 < g.k; k0 += TK) {
#pragma unroll
      for (int q = 0; q < (TM * TK) / NT; ++q) {
        const int el = tid + q * NT;
        int ii, kk;
        if (g.a_k == 1) { kk = el % TK; ii = el / TK; } else { ii = el % TM; kk = el / TM; }
        const int gi = i0 + ii, gk = k0 + kk;
        As[kk][ii] = (gi < g.m && gk < g.k) ? ldf(A + (long long)gi * g.a_i + (long long)gk * g.a_k) : 0.f;
        int jj;
        if (g.b_k == 1) { kk = el % TK; jj = el / TK; } else { jj = el % TN; kk = el / TN; }
        const int gj = j0 + jj;
        const int gk2 = k0 + kk;
        Bs[kk][jj] = (gj < g.n && gk2 < g.k) ? ldf(B + (long long)gj * g.b_j + (long long)gk2 * g.b_k) : 0.f;
      }
      __syncthreads();
#pragma unroll
      for (int kk = 0; kk < TK; ++kk) {
        float a[4], b[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) a[r] = As[kk][ty * 4 + r];
#pragma unroll
        for (int c = 0; c < 4; ++c) b[c] = Bs[kk][tx * 4 + c];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
          for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(a[r], b[c], acc[r][c]);
      }
      __syncthreads();
    }

    // ---- epilogue for this tile ----
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int i = i0 + ty * 4 + r;
      if (i >= g.m) continue;
      float lam = 0.f, w = 0.f;
      if (EPI == EPI_DLOGITS || (EPI == EPI_SUBSET_LOGP && e.lambda)) lam = e.lambda[i];
      if (EPI == EPI_DLOGITS) w = e.roww[i];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int j = j0 + tx * 4 + c;
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
          if (j < Kdev)
            reinterpret_cast<float*>(e.out)[(long long)i * e.ld + j] = a + bias_at<T>(e.bias, e.U[j]) - lam;
        } else if (EPI == EPI_DLOGITS) {
          const long long v = e.v0 + j;
          const float p = __expf(a + bias_at<T>(e.bias, v) - lam);
          const int jj = e.vmap[v];
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
    for (int r = 0; r < 4; ++r) { s_red[0][ty * 4 + r][tx] = run_max[r]; s_idx[ty * 4 + r][tx] = run_idx[r]; }
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
    for (int r = 0; r < 4; ++r) {
      s_red[0][ty * 4 + r][tx] = run_max[r];
      s_red[1][ty * 4 + r][tx] = run_sum[r];
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

template <typename T, int EPI>
cudaError_t launch(const void* A, const void* B, const GemmShape& g, const Epilogue& e, cudaStream_t stream) {
  const int ntiles = (g.n + TN - 1) / TN;
  int tiles_per_cta = 1, gx = ntiles;
  if (EPI == EPI_LSE_PARTIAL || EPI == EPI_ARGMAX_PARTIAL) {
    tiles_per_cta = (ntiles + e.nsplit - 1) / e.nsplit;
    gx = e.nsplit;
  }
  dim3 grid(gx, (g.m + TM - 1) / TM);
  if (grid.x == 0 || grid.y == 0) return cudaSuccess;
  k_simt_gemm<T, EPI><<<grid, NT, 0, stream>>>((const T*)A, (const T*)B, g, e, tiles_per_cta);
  return cudaGetLastError();
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
