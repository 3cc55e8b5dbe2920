// Re-computation passes for the fine-grained straight-through estimators (Sec. 4, App. D of the paper): the
// forward chain of every output is replayed with the tracking variants of the scalar kernel, which report
// the last overflow (recursive estimator) or one bit per FMAq step (overflow and difference estimators).
#include "lba_kernel.cuh"

namespace lba {

namespace {

constexpr int BM = 64, BN = 64, TM = 4, TN = 4;

template <int QM, int ORD, int LD, int TRACK>
cudaError_t launch(const Problem& p, cudaStream_t stream) {
  const dim3 grid((unsigned)((p.M + BM - 1) / BM), (unsigned)((p.N + BN - 1) / BN), 1);
  lba_contract_kernel<BM, BN, TM, TN, QM, ORD, LD, TRACK><<<grid, (BM / TM) * (BN / TN), 0, stream>>>(p);
  return cudaGetLastError();
}

template <int QM, int ORD, int TRACK>
cudaError_t by_loader(int load, const Problem& p, cudaStream_t stream) {
  return load == LD_GEMM_VEC ? launch<QM, ORD, LD_GEMM_VEC, TRACK>(p, stream) : launch<QM, ORD, LD_ANY, TRACK>(p, stream);
}

template <int QM, int TRACK>
cudaError_t by_order(int ord, int load, const Problem& p, cudaStream_t stream) {
  switch (ord) {
    case ORD_SEQ: return by_loader<QM, ORD_SEQ, TRACK>(load, p, stream);
    case ORD_CHUNK_SLAB: return by_loader<QM, ORD_CHUNK_SLAB, TRACK>(load, p, stream);
    case ORD_CHUNK_ANY: return by_loader<QM, ORD_CHUNK_ANY, TRACK>(load, p, stream);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

// qm: QM_FLOOR_FAST (Q_prod is the flush alone) or QM_FLOOR_FULL
cudaError_t launch_last_overflow(int qm, int load, const Problem& p, cudaStream_t stream) {
  return qm == QM_FLOOR_FAST ? by_loader<QM_FLOOR_FAST, ORD_SEQ, TRACK_LAST_OF>(load, p, stream)
                             : by_loader<QM_FLOOR_FULL, ORD_SEQ, TRACK_LAST_OF>(load, p, stream);
}

// ord: ORD_SEQ, ORD_CHUNK_SLAB (chunk a multiple of the slab length) or ORD_CHUNK_ANY; diff: 0 = STE^OF, 1 = STE^DIFF
cudaError_t launch_ste_mask(int qm, int ord, int diff, int load, const Problem& p, cudaStream_t stream) {
  if (qm == QM_FLOOR_FAST)
    return diff ? by_order<QM_FLOOR_FAST, TRACK_MASK_DIFF>(ord, load, p, stream)
                : by_order<QM_FLOOR_FAST, TRACK_MASK_OF>(ord, load, p, stream);
  return diff ? by_order<QM_FLOOR_FULL, TRACK_MASK_DIFF>(ord, load, p, stream)
              : by_order<QM_FLOOR_FULL, TRACK_MASK_OF>(ord, load, p, stream);
}

}  // namespace lba
