#include "pctc_internal.h"
namespace pctc {
bool umma_available() { return false; }
cudaError_t umma_gemm(const __nv_bfloat16*, long long, bool, const __nv_bfloat16*, long long, bool, int, int, int,
                      const Epilogue&, int*, cudaStream_t) {
  return cudaErrorNotSupported;
}
}  // namespace pctc
