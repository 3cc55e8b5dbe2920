// LBA contraction with the products formed by the 5th-generation tensor cores (tcgen05.mma), sm_100a.
//
// The method rounds after every single addition (Eq. 4 of the paper), so the tensor cores may not add two
// products together.  They may still *multiply*: for one k-step the 128 x BN outer product a[:, k] b[:, k]^T
// is an MMA whose K extent holds a single non-zero term,
//     D[m][n] = sum_j A[m][j] * Bk[n][j],   Bk[n][j] = b[n][k] if j == k else 0   (j over the 16 k of a slab)
// = a[m][k] * b[n][k] exactly (bf16 operands carry the 4-bit E4M3 significands and the power-of-two carrier
// scale exactly; the fp32 accumulator holds the 8-bit product exactly; the other 15 terms are exact zeros).
// The CUDA cores then only do what the definition forces on them: per product one half of a packed
// fma.rz.ftz.f32x2 (exact sum, one rounding toward zero, flush of sums below R_UF; a product below R_UF_prod
// arrives as a binary32 subnormal or zero and is flushed on input) and one LOP3 (the mantissa mask).  Compared
// with the all-CUDA-core kernel this removes the packed multiply and every shared-memory operand load from the
// issue stream; the logic pipe (one mask per MAC) is what remains.
//
// Layout of one CTA (160 threads, 128 output rows x BN output columns):
//   warps 0-3   decode the next slab into shared memory (A: one bf16 [128][16] K-major tile; B: sixteen
//               [BN][16] tiles, tile k holding column k of the slab and zeros elsewhere - the zeros are written
//               once), and consume the products: thread t owns output row t and its BN running sums
//   warp 4      one lane issues the MMAs (tile k -> tensor-memory buffer k % 3) and commits each to an mbarrier
//   tensor memory: 3 product buffers of BN columns + BN columns for the second-level sums of the chunked order
// Every wait on an mbarrier is bounded; a wait that runs out records an error code, and the CTA still frees
// its tensor memory and exits.
#pragma once
#include "lba_kernel.cuh"

namespace lba {

constexpr int UMMA_BM = 128;
constexpr int UMMA_NBUF = 3;
constexpr long long UMMA_WAIT_CYCLES = 1ll << 31;  // about one second of SM clock: a wait that long has failed

__device__ int g_umma_error = 0;  // 0 ok; 1 consumer wait, 2 issuer wait on a stage, 3 issuer wait on a buffer

template <int BN>
struct UmmaSmem {
  static constexpr int A_STAGE = UMMA_BM * 32;          // bf16 [128][16]
  static constexpr int B_TILE = BN * 32;                // bf16 [BN][16]
  static constexpr int B_STAGE = 16 * B_TILE;
  static constexpr int OFF_A = 0;
  static constexpr int OFF_B = 2 * A_STAGE;
  static constexpr int OFF_BAR = OFF_B + 2 * B_STAGE;   // 2 + 3 + 3 mbarriers
  static constexpr int OFF_NRM = OFF_BAR + 8 * 8;
  static constexpr int OFF_SLOT = OFF_NRM + 6 * 4;
  static constexpr int BYTES = OFF_SLOT + 8;
};

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// bounded wait for the completion of the phase with the given parity; false if it ran out
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  const long long t0 = clock64();
  for (uint32_t tries = 0;; ++tries) {
    if ((tries & 255u) == 255u && clock64() - t0 > UMMA_WAIT_CYCLES) return false;
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
  }
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// shared-memory matrix descriptor: K-major, no swizzle, 8-row x 16-byte core matrices; the two K halves of a
// row group are 128 bytes apart (leading offset), row groups 256 bytes apart (stride offset)
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
  return (uint64_t)((smem_addr >> 4) & 0x3FFFu) | ((uint64_t)(128u >> 4) << 16) | ((uint64_t)(256u >> 4) << 32) |
         ((uint64_t)1 << 46);
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}

template <int BN, int LD>
__global__ void __launch_bounds__(160, 2) lba_contract_umma_kernel(const Problem p) {
  static_assert(BN == 64, "one tensor-memory budget: 3 x BN product columns + BN sum columns = 256");
  typedef UmmaSmem<BN> S;
  constexpr int NT = 128;  // consumer / decoder threads
  constexpr int PN = BN / 2;
  constexpr int TMEM_COLS = 256;
  constexpr int T_COL = UMMA_NBUF * BN;
  constexpr int LPT = (UMMA_BM + BN + NT - 1) / NT;

  extern __shared__ __align__(16) unsigned char smem_raw[];
  const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem_raw);
  const uint32_t bar_stage = smem_base + S::OFF_BAR;             // [2] operands of a slab are in shared memory
  const uint32_t bar_full = bar_stage + 16;                      // [3] products of a k-step are in tensor memory
  const uint32_t bar_empty = bar_full + 24;                      // [3] all four warps have read a product buffer
  unsigned (*nrm)[2] = reinterpret_cast<unsigned (*)[2]>(smem_raw + S::OFF_NRM);
  unsigned* tmem_slot = reinterpret_cast<unsigned*>(smem_raw + S::OFF_SLOT);

  // once any CTA has reported a failed wait, later CTAs of the grid (and later launches, until the host reads
  // the error word) do nothing: a fault must not be paid for once per CTA
  if (*reinterpret_cast<volatile int*>(&g_umma_error) != 0) return;

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int64_t m0 = (int64_t)blockIdx.x * UMMA_BM;
  const int64_t n0 = (int64_t)blockIdx.y * BN;
  const int nslab = (int)((p.K + BK - 1) / BK);

  // ---- set-up: zero the B tiles (only their diagonals are ever rewritten), barriers, tensor memory
  for (int i = tid; i < 2 * S::B_STAGE / 16; i += blockDim.x)
    reinterpret_cast<uint4*>(smem_raw + S::OFF_B)[i] = make_uint4(0u, 0u, 0u, 0u);
  if (tid == 0) {
    mbar_init(bar_stage, NT);
    mbar_init(bar_stage + 8, NT);
    for (int i = 0; i < UMMA_NBUF; ++i) {
      mbar_init(bar_full + 8 * i, 1);
      mbar_init(bar_empty + 8 * i, 4);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < 6) nrm[tid >> 1][tid & 1] = 0u;
  if (warp == 0) {
    const uint32_t slot = (uint32_t)__cvta_generic_to_shared(tmem_slot);
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the zeros must be visible to the tensor core
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  bool dead = false;  // a bounded wait ran out: stop waiting, finish, free tensor memory

  if (warp == 4) {
    // =========================================================== MMA issuer (one lane)
    if ((tid & 31) == 0) {
      // instruction descriptor: fp32 accumulate, bf16 x bf16, both K-major, N = BN, M = 128
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(UMMA_BM >> 4) << 24);
      int g = 0;  // global k-step
      int buf = 0;
      uint32_t empty_parity = 0;  // bit i: parity to wait for on bar_empty[i]
      for (int s = 0; s < nslab && !dead; ++s) {
        const int st = s & 1;
        if (!mbar_wait(bar_stage + 8 * st, (uint32_t)(s >> 1) & 1u)) {
          atomicExch(&g_umma_error, 2);
          dead = true;
          break;
        }
        tc_fence_after();
        const uint64_t desc_a = umma_desc(smem_base + S::OFF_A + st * S::A_STAGE);
        for (int kk = 0; kk < BK; ++kk, ++g) {
          if (g >= UMMA_NBUF) {
            if (!mbar_wait(bar_empty + 8 * buf, (empty_parity >> buf) & 1u)) {
              atomicExch(&g_umma_error, 3);
              dead = true;
              break;
            }
            empty_parity ^= 1u << buf;
            tc_fence_after();
          }
          const uint64_t desc_b = umma_desc(smem_base + S::OFF_B + st * S::B_STAGE + kk * S::B_TILE);
          const uint32_t d_addr = tmem_base + (uint32_t)(buf * BN);
          asm volatile(
              "{\n\t.reg .pred p;\n\t"
              "setp.ne.b32 p, %4, 0;\n\t"
              "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
              :
              : "r"(d_addr), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(0u), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
              : "memory");
          asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_full + 8 * buf)
                       : "memory");
          buf = buf == UMMA_NBUF - 1 ? 0 : buf + 1;
        }
      }
    }
  } else {
    // =========================================================== decoders / consumers
    RowLoader<UMMA_BM, BN, NT, LD> loader;
    loader.init(p, tid, m0, n0);

    auto decode_store = [&](const uint4 (&raw)[LPT], int st, int cell) {
#pragma unroll
      for (int l = 0; l < LPT; ++l) {
        const int r = tid + l * NT;
        if (r < UMMA_BM + BN) {  // uniform per warp
          const bool is_a = r < UMMA_BM;
          const float mul = is_a ? p.pk_a : p.pk_b;
          const uint32_t w4[4] = {raw[l].x, raw[l].y, raw[l].z, raw[l].w};
          float n2 = 0.0f;
          uint32_t packed[8];  // bf16 pairs (k even in the low half)
#pragma unroll
          for (int q = 0; q < 4; ++q) {
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
              float v0, v1;
              e4m3x2_to_f32(hh == 0 ? w4[q] : (w4[q] >> 16), v0, v1);
              n2 = fma_rn(v0, v0, n2);
              n2 = fma_rn(v1, v1, n2);
              const float s0 = mul_ieee(v0, mul), s1 = mul_ieee(v1, mul);
              asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(packed[q * 2 + hh]) : "f"(s1), "f"(s0));  // exact: 4 significant bits
            }
          }
          if (is_a) {
            unsigned char* dst = smem_raw + S::OFF_A + st * S::A_STAGE + (r >> 3) * 256 + (r & 7) * 16;
            *reinterpret_cast<uint4*>(dst) = make_uint4(packed[0], packed[1], packed[2], packed[3]);        // k 0..7
            *reinterpret_cast<uint4*>(dst + 128) = make_uint4(packed[4], packed[5], packed[6], packed[7]);  // k 8..15
          } else {
            const int n = r - UMMA_BM;
            unsigned char* row = smem_raw + S::OFF_B + st * S::B_STAGE + (n >> 3) * 256 + (n & 7) * 16;
#pragma unroll
            for (int kk = 0; kk < BK; ++kk) {
              const uint32_t pair = packed[kk >> 1];
              const unsigned short h = (unsigned short)((kk & 1) ? (pair >> 16) : (pair & 0xFFFFu));
              *reinterpret_cast<unsigned short*>(row + kk * S::B_TILE + (kk >> 3) * 128 + (kk & 7) * 2) = h;
            }
          }
          const unsigned m = __reduce_max_sync(0xFFFFFFFFu, __float_as_uint(n2 * p.nrm_scale));
          if ((tid & 31) == 0) atomicMax(&nrm[cell][is_a ? 0 : 1], m);
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(bar_stage + 8 * st);
    };

    const uint32_t t_lane = tmem_base + ((uint32_t)(warp * 32) << 16);  // this thread's row of tensor memory
    u64 acc1[PN];
#pragma unroll
    for (int j = 0; j < PN; ++j) acc1[j] = 0ull;
    {  // second-level sums start at zero
      uint32_t zero[16];
#pragma unroll
      for (int c = 0; c < 16; ++c) zero[c] = 0u;
#pragma unroll
      for (int gq = 0; gq < BN / 16; ++gq) tmem_st16(t_lane + T_COL + 16 * gq, zero);
      tmem_wait_st();
    }
    const u64 cc2 = pack2(p.c, p.c);
    const uint32_t mask = p.qa.mask;
    const float sat = p.qa.sat;

    uint4 raw[LPT];
    if (nslab > 0) {
      loader.fetch(p, tid, 0, raw);
      decode_store(raw, 0, 0);
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");  // the first slab's norms are complete

    // One slab = 16 k-steps, each read from tensor memory in two halves of 32 columns.  The load of the next
    // half is in flight while the current half is accumulated (tcgen05.wait::ld comes after the arithmetic), and a
    // product buffer is handed back to the issuer as soon as its second half is in registers.
    int buf = 0;                 // product buffer of the next k-step (g % 3)
    uint32_t full_parity = 0;    // bit i: parity to wait for on bar_full[i]
    auto wait_products = [&](int b) {
      if (!dead && !mbar_wait(bar_full + 8 * b, (full_parity >> b) & 1u)) {
        atomicExch(&g_umma_error, 1);
        dead = true;
      }
      full_parity ^= 1u << b;
      tc_fence_after();
    };
    auto accumulate = [&](const uint32_t (&pr)[32], int half, auto clamp_tag) {
      constexpr bool CLAMP = decltype(clamp_tag)::value;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const u64 t = fma2_rz_ftz(pack2u(pr[2 * j], pr[2 * j + 1]), cc2, acc1[half * 16 + j]);
        float lo, hi;
        unpack2(t, lo, hi);
        lo = and_bits(lo, mask);
        hi = and_bits(hi, mask);
        if (CLAMP) {
          lo = clamp_mag(lo, sat);
          hi = clamp_mag(hi, sat);
        }
        acc1[half * 16 + j] = pack2(lo, hi);
      }
    };
    auto slab = [&](auto clamp_tag) {
      uint32_t pa[32], pb[32];
      wait_products(buf);
      tmem_ld32(t_lane + (uint32_t)(buf * BN), pa);
      tmem_wait_ld();
#pragma unroll 1
      for (int kk = 0; kk < BK; ++kk) {
        tmem_ld32(t_lane + (uint32_t)(buf * BN + 32), pb);  // second half of this k-step, in flight
        accumulate(pa, 0, clamp_tag);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if ((tid & 31) == 0) mbar_arrive(bar_empty + 8 * buf);  // this warp has read the whole buffer
        buf = buf == UMMA_NBUF - 1 ? 0 : buf + 1;
        if (kk + 1 < BK) {
          wait_products(buf);
          tmem_ld32(t_lane + (uint32_t)(buf * BN), pa);      // first half of the next k-step, in flight
        }
        accumulate(pb, 1, clamp_tag);
        if (kk + 1 < BK) tmem_wait_ld();
      }
    };

    // second hierarchy on this thread's row: T <- Q_acc(C + T), C <- 0; FINAL keeps T in acc1 for the epilogue
    auto close_chunk = [&](auto clamp_tag, bool final) -> float {
      constexpr bool CLAMP = decltype(clamp_tag)::value;
      float mx = 0.0f;
#pragma unroll
      for (int gq = 0; gq < BN / 16; ++gq) {
        uint32_t cur[16];
        tmem_ld16(t_lane + T_COL + 16 * gq, cur);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          float lo, hi;
          unpack2(add2_rz_ftz(acc1[gq * 8 + j], pack2u(cur[2 * j], cur[2 * j + 1])), lo, hi);
          lo = and_bits(lo, mask);
          hi = and_bits(hi, mask);
          if (CLAMP) {
            lo = clamp_mag(lo, sat);
            hi = clamp_mag(hi, sat);
            mx = fmaxf(mx, fmaxf(fabsf(lo), fabsf(hi)));
          }
          cur[2 * j] = __float_as_uint(lo);
          cur[2 * j + 1] = __float_as_uint(hi);
          acc1[gq * 8 + j] = final ? pack2(lo, hi) : 0ull;
        }
        if (!final) tmem_st16(t_lane + T_COL + 16 * gq, cur);
      }
      if (!final) tmem_wait_st();
      return mx;
    };

    float u2 = 0.0f;
    int cell = 0;
    for (int s = 0; s < nslab; ++s) {
      const int cell_next = cell == 2 ? 0 : cell + 1;
      const int cell_clear = cell_next == 2 ? 0 : cell_next + 1;
      if (s + 1 < nslab) loader.fetch(p, tid, s + 1, raw);
      const float na = __uint_as_float(nrm[cell][0]), nb = __uint_as_float(nrm[cell][1]);
      if (tid < 2) nrm[cell_clear][tid] = 0u;
      const float grow = sqrtf(na * nb) * 1.01f;
      if (grow < 0.999f) slab(std::false_type());
      else slab(std::true_type());
      const bool last = s + 1 == nslab;
      if (__all_sync(0xFFFFFFFFu, u2 + grow < 0.999f)) {
        close_chunk(std::false_type(), last);
        u2 += grow;
      } else {
        u2 = close_chunk(std::true_type(), last) * p.inv_top;
      }
      if (s + 1 < nslab) decode_store(raw, (s + 1) & 1, cell_next);
      asm volatile("bar.sync 1, 128;" ::: "memory");  // norms of the next slab complete, cleared cell not yet reused
      cell = cell_next;
    }

    // ---- epilogue: thread = output row, BN consecutive columns
    const int64_t m = m0 + tid;
    if (m < p.M) {
      const float sa = p.sa[p.sa_per_row ? m : 0];
      float* orow = p.out + (int64_t)blockIdx.z * p.batch_out + m * p.N;
      const bool vec_store = (p.N % 4 == 0) && ((reinterpret_cast<uintptr_t>(p.out) & 15) == 0) && (p.batch_out % 4 == 0);
#pragma unroll
      for (int q = 0; q < BN / 4; ++q) {
        const int64_t n = n0 + q * 4;
        float o[4];
        unpack2(acc1[q * 2], o[0], o[1]);
        unpack2(acc1[q * 2 + 1], o[2], o[3]);
        float rr[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float y = __fmul_rn(__fmul_rn(o[j], p.un1), p.un2);
          y = (y == 0.0f) ? 0.0f : y;
          if (n + j < p.N) {
            const float sb = p.sb[p.sb_per_col ? n + j : 0];
            float r = __fmul_rn(__fmul_rn(y, sa), sb);
            if (p.bias) r = __fadd_rn(r, p.bias[n + j]);
            rr[j] = r;
          } else {
            rr[j] = 0.0f;
          }
        }
        if (n + 3 < p.N && vec_store) {
          *reinterpret_cast<float4*>(orow + n) = make_float4(rr[0], rr[1], rr[2], rr[3]);
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (n + j < p.N) orow[n + j] = rr[j];
        }
      }
    }
  }

  // ---- every thread is done with tensor memory
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

template <int LD>
cudaError_t launch_umma(const Problem& p, cudaStream_t stream) {
  constexpr int BN = 64;
  auto kernel = lba_contract_umma_kernel<BN, LD>;
  constexpr int smem = UmmaSmem<BN>::BYTES + 64;
  static bool done[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!done[dev]) {
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    done[dev] = true;
  }
  const dim3 grid((unsigned)((p.M + UMMA_BM - 1) / UMMA_BM), (unsigned)((p.N + BN - 1) / BN), (unsigned)p.batch);
  kernel<<<grid, 160, smem, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace lba
