// Fixed-point accumulators (Eq. 1): instantiations of the integer kernel.
#include "lba_kernel_fixed.cuh"

namespace lba {
namespace {

template <int ORD, int LD, bool WP, bool WA>
cudaError_t launch(const Problem& p, cudaStream_t stream) {
  const dim3 grid((unsigned)((p.M + 63) / 64), (unsigned)((p.N + 63) / 64), (unsigned)p.batch);
  lba_fixed_kernel<ORD, LD, WP, WA><<<grid, 256, 0, stream>>>(p);
  return cudaGetLastError();
}

template <int ORD, int LD>
cudaError_t by_wrap(const Problem& p, cudaStream_t stream) {
  if (p.fx_wrap_p) return p.fx_wrap_a ? launch<ORD, LD, true, true>(p, stream) : launch<ORD, LD, true, false>(p, stream);
  return p.fx_wrap_a ? launch<ORD, LD, false, true>(p, stream) : launch<ORD, LD, false, false>(p, stream);
}

template <int ORD>
cudaError_t by_loader(int load, const Problem& p, cudaStream_t stream) {
  switch (load) {
    case LD_GEMM_VEC: return by_wrap<ORD, LD_GEMM_VEC>(p, stream);
    case LD_CONV_VEC: return by_wrap<ORD, LD_CONV_VEC>(p, stream);
    default: return by_wrap<ORD, LD_ANY>(p, stream);
  }
}

}  // namespace

cudaError_t launch_fixed(int ord, int load, const Problem& p, cudaStream_t stream) {
  switch (ord) {
    case ORD_SEQ: return by_loader<ORD_SEQ>(load, p, stream);
    case ORD_CHUNK_SLAB: return by_loader<ORD_CHUNK_SLAB>(load, p, stream);
    case ORD_CHUNK_ANY: return by_loader<ORD_CHUNK_ANY>(load, p, stream);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace lba
