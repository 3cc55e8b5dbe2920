// Chunk-16 order with two CTAs of a thread-block cluster per output tile (see lba_contract_packed_kernel, CL = 2):
// 64x64 tile, 4x8 outputs per thread, floor quantisers.
#include "lba_kernel.cuh"

namespace lba {
namespace {

constexpr int BM = 64, BN = 64, TM = 4, TN = 8, CL = 2;

template <int PQ, int LD, bool H16>
cudaError_t launch(const Problem& p, cudaStream_t stream) {
  auto kernel = lba_contract_packed_kernel<BM, BN, TM, TN, PQ, false, ORD_CHUNK16, LD, 0, CL, H16>;
  constexpr size_t smem = packed_cluster_smem_bytes<BM, BN, TM, TN>();
  static_assert(smem <= 48 * 1024, "no opt-in needed");
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((p.M + BM - 1) / BM) * CL, (unsigned)((p.N + BN - 1) / BN), (unsigned)p.batch);
  cfg.blockDim = dim3((BM / TM) * (BN / TN), 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CL;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, p);
}

template <int PQ>
cudaError_t by_loader(int load, const Problem& p, cudaStream_t stream) {
  // an accumulator value with at most 7 mantissa bits (low 16 bits of the binary32 pattern clear) is a bfloat16
  const bool h16 = (p.qa.mask & 0xFFFFu) == 0u;
  switch (load) {
    case LD_GEMM_VEC: return h16 ? launch<PQ, LD_GEMM_VEC, true>(p, stream) : launch<PQ, LD_GEMM_VEC, false>(p, stream);
    case LD_CONV_VEC: return h16 ? launch<PQ, LD_CONV_VEC, true>(p, stream) : launch<PQ, LD_CONV_VEC, false>(p, stream);
    default: return cudaErrorInvalidValue;  // the byte-wise loader keeps the single-CTA tiles
  }
}

}  // namespace

// pq: PackedProd.  The caller has checked: floor rounding, chunk-16 order, 16-byte loader.
cudaError_t launch_cluster_pair(int pq, int load, const Problem& p, cudaStream_t stream) {
  switch (pq) {
    case PQ_NONE: return by_loader<PQ_NONE>(load, p, stream);
    case PQ_MASK: return by_loader<PQ_MASK>(load, p, stream);
    default: return by_loader<PQ_MASK_SAT>(load, p, stream);
  }
}

}  // namespace lba
