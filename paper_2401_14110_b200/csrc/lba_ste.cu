// Re-computation helper for the recursive overflow straight-through estimator (App. D of the paper): replays
// the sequential FMAq chain of every output and reports the last step at which Q_acc overflowed.
#include "lba_kernel.cuh"

namespace lba {

cudaError_t launch_last_overflow(int load, const Problem& p, cudaStream_t stream) {
  constexpr int BM = 64, BN = 64, TM = 4, TN = 4;
  const dim3 grid((unsigned)((p.M + BM - 1) / BM), (unsigned)((p.N + BN - 1) / BN), 1);
  const int threads = (BM / TM) * (BN / TN);
  if (load == LD_GEMM_VEC)
    lba_contract_kernel<BM, BN, TM, TN, QM_FLOOR_FULL, ORD_SEQ, LD_GEMM_VEC, true><<<grid, threads, 0, stream>>>(p);
  else
    lba_contract_kernel<BM, BN, TM, TN, QM_FLOOR_FULL, ORD_SEQ, LD_ANY, true><<<grid, threads, 0, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace lba
