// Fixed-point accumulators (Eq. 1): instantiations of the integer kernel.
#include "lba_kernel_fixed.cuh"

namespace lba {
namespace {

template <int ORD, int LD, int HP, bool WA>
cudaError_t launch(const Problem& p, cudaStream_t stream) {
  const dim3 grid((unsigned)((p.M + 63) / 64), (unsigned)((p.N + 63) / 64), (unsigned)p.batch);
  lba_fixed_kernel<ORD, LD, HP, WA><<<grid, 256, 0, stream>>>(p);
  return cudaGetLastError();
}

template <int ORD, int LD>
cudaError_t by_wrap(const Problem& p, cudaStream_t stream) {
  // fx_hold_p: 0 = products provably inside the product format's range, 1 = saturate, 2 = wrap around
  switch (p.fx_hold_p) {
    case 0: return p.fx_wrap_a ? launch<ORD, LD, 0, true>(p, stream) : launch<ORD, LD, 0, false>(p, stream);
    case 1: return p.fx_wrap_a ? launch<ORD, LD, 1, true>(p, stream) : launch<ORD, LD, 1, false>(p, stream);
    default: return p.fx_wrap_a ? launch<ORD, LD, 2, true>(p, stream) : launch<ORD, LD, 2, false>(p, stream);
  }
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
