// The tensor-core-product kernel (chunk-16 order, fast floor quantiser) and its device error word.
#include "lba_kernel_umma.cuh"

namespace lba {

cudaError_t launch_umma_family(int load, const Problem& p, cudaStream_t stream) {
  switch (load) {
    case LD_GEMM_VEC: return launch_umma<LD_GEMM_VEC>(p, stream);
    case LD_CONV_VEC: return launch_umma<LD_CONV_VEC>(p, stream);
    case LD_ANY: return launch_umma<LD_ANY>(p, stream);
    default: return cudaErrorInvalidValue;
  }
}

// reads (and clears) the error word the kernel sets when one of its bounded waits runs out; synchronises
cudaError_t read_umma_error(int* code) {
  int zero = 0;
  cudaError_t e = cudaMemcpyFromSymbol(code, g_umma_error, sizeof(int));
  if (e != cudaSuccess) return e;
  return cudaMemcpyToSymbol(g_umma_error, &zero, sizeof(int));
}

}  // namespace lba
