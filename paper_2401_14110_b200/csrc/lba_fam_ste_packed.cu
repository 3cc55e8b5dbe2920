// Overflow masks of the straight-through estimator STE^OF (App. D of the paper) from the packed kernel:
// 64x64 tile, 4x8 outputs per thread, floor quantisers, sequential or chunk-16 order.
#include "lba_kernel.cuh"

namespace lba {
namespace {

constexpr int BM = 64, BN = 64, TM = 4, TN = 8;

template <int PQ, int ORD, int LD>
cudaError_t launch(const Problem& p, cudaStream_t stream) {
  const dim3 grid((unsigned)((p.M + BM - 1) / BM), (unsigned)((p.N + BN - 1) / BN), 1);
  auto kernel = lba_contract_packed_kernel<BM, BN, TM, TN, PQ, false, ORD, LD, 1>;
  constexpr size_t smem = packed_ste_smem_bytes<BM, BN, TM, TN>();
  static_assert(smem > 48 * 1024, "opt-in below assumes the large shared-memory carve-out is needed");
  static bool done[64] = {};  // opt in to large dynamic shared memory, once per device and kernel
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!done[dev]) {
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    done[dev] = true;
  }
  kernel<<<grid, (BM / TM) * (BN / TN), smem, stream>>>(p);
  return cudaGetLastError();
}

template <int PQ, int ORD>
cudaError_t by_loader(int load, const Problem& p, cudaStream_t stream) {
  return load == LD_GEMM_VEC ? launch<PQ, ORD, LD_GEMM_VEC>(p, stream) : launch<PQ, ORD, LD_ANY>(p, stream);
}

template <int ORD>
cudaError_t by_product(int pq, int load, const Problem& p, cudaStream_t stream) {
  switch (pq) {
    case PQ_NONE: return by_loader<PQ_NONE, ORD>(load, p, stream);
    case PQ_MASK: return by_loader<PQ_MASK, ORD>(load, p, stream);
    default: return by_loader<PQ_MASK_SAT, ORD>(load, p, stream);
  }
}

}  // namespace

// pq: PackedProd; chunk16: 0 = sequential order, 1 = chunks of 16
cudaError_t launch_ste_packed(int pq, int chunk16, int load, const Problem& p, cudaStream_t stream) {
  return chunk16 ? by_product<ORD_CHUNK16>(pq, load, p, stream) : by_product<ORD_SEQ>(pq, load, p, stream);
}

}  // namespace lba
