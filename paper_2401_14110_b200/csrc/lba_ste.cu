// Re-computation passes for the fine-grained straight-through estimators (Sec. 4, App. D of the paper): the
// forward chain of every output is replayed with the tracking variants of the scalar kernel, which report
// the last overflow (recursive estimator) or one bit per FMAq step (overflow and difference estimators).
#include "lba_kernel.cuh"

namespace lba {

namespace {

constexpr int BM = 64, BN = 64, TM = 4, TN = 4;

template <int ORD, int LD, int TRACK>
cudaError_t launch(const Problem& p, cudaStream_t stream) {
  const dim3 grid((unsigned)((p.M + BM - 1) / BM), (unsigned)((p.N + BN - 1) / BN), 1);
  lba_contract_kernel<BM, BN, TM, TN, QM_FLOOR_FULL, ORD, LD, TRACK><<<grid, (BM / TM) * (BN / TN), 0, stream>>>(p);
  return cudaGetLastError();
}

template <int ORD, int TRACK>
cudaError_t by_loader(int load, const Problem& p, cudaStream_t stream) {
  return load == LD_GEMM_VEC ? launch<ORD, LD_GEMM_VEC, TRACK>(p, stream) : launch<ORD, LD_ANY, TRACK>(p, stream);
}

template <int TRACK>
cudaError_t by_order(int ord, int load, const Problem& p, cudaStream_t stream) {
  switch (ord) {
    case ORD_SEQ: return by_loader<ORD_SEQ, TRACK>(load, p, stream);
    case ORD_CHUNK_SLAB: return by_loader<ORD_CHUNK_SLAB, TRACK>(load, p, stream);
    case ORD_CHUNK_ANY: return by_loader<ORD_CHUNK_ANY, TRACK>(load, p, stream);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

cudaError_t launch_last_overflow(int load, const Problem& p, cudaStream_t stream) {
  return by_loader<ORD_SEQ, TRACK_LAST_OF>(load, p, stream);
}

// ord: ORD_SEQ, ORD_CHUNK_SLAB (chunk a multiple of the slab length) or ORD_CHUNK_ANY; diff: 0 = STE^OF, 1 = STE^DIFF
cudaError_t launch_ste_mask(int ord, int diff, int load, const Problem& p, cudaStream_t stream) {
  return diff ? by_order<TRACK_MASK_DIFF>(ord, load, p, stream) : by_order<TRACK_MASK_OF>(ord, load, p, stream);
}

}  // namespace lba
