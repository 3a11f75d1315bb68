// Tensor-core NS5 products (placeholder until the tcgen05 kernel lands).
#include "epilogue.cuh"

namespace prm {

struct TcContext { int unused; };

TcContext* tc_create(std::string* err) { (void)err; return new TcContext(); }
void tc_destroy(TcContext* tc) { delete tc; }

cudaError_t launch_gemm_tc(TcContext*, const GemmProblem&, const Epilogue&, int*, cudaStream_t, int64_t*) {
  return cudaErrorNotSupported;
}

}  // namespace prm
