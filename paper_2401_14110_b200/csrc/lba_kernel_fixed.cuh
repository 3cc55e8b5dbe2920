// Fixed-point accumulation (Eq. 1 of the paper, Sec. 2.1) on the integer pipe.
//
//   FMAq(x, w, S) = Q_acc( Q_prod(x * w) + S ),   Q_{B,b}(v) = 2^-b * hold( floor(v * 2^b) )
//
// where hold() keeps the integer in [-2^(B-1), 2^(B-1) - 1] by saturation (Eq. 1) or by two's-complement
// wrap-around (the integer accumulators of the WrapNet comparison, Sec. 2.2).  An E4M3 value is s * 2^q with an
// integer |s| <= 15, so a product is P * 2^(qx + qw) with |P| <= 225, and floor(P * 2^t) for any integer t is one
// arithmetic right shift of P << 22 by 22 - t (exact: for t <= -9 the value lies in (-1, 1) and a shift by 31 or
// more leaves 0 or -1).  The running sums are plain 32-bit integers in units of 2^-b_acc.
// The host checks that none of the left shifts can leave 32 bits.
//
// Layout: 64 x 64 outputs per CTA, 4 x 4 per thread, 256 threads, K in slabs of 16, operands decoded once per
// CTA into shared memory, mantissas and shift contributions in arrays of their own (a thread's four neighbouring
// values are then one 16-byte load from consecutive addresses: as {mantissa, shift} pairs the 32-byte stride between
// lanes put two lanes of every quarter-warp on the same banks); orders and loaders as in the scalar kernel.
#pragma once
#include "lba_kernel.cuh"

namespace lba {

// hold() of the header comment
template <bool WRAP>
__device__ __forceinline__ int fx_hold(int v, int lo, int hi, int sh) {
  if (WRAP) return (v << sh) >> sh;  // sign-extend the low B bits (sh = 32 - B)
  return min(max(v, lo), hi);
}
// arithmetic right shift whose count may exceed 31: the PTX instruction clamps the count at 32 (all sign bits),
// where the C++ operator would be undefined
__device__ __forceinline__ int fx_sar(int v, int count) {
  int d;
  asm("shr.s32 %0, %1, %2;" : "=r"(d) : "r"(v), "r"(count));
  return d;
}

// HOLD_P: 0 = the host proved that no product leaves the product format's range (Q_prod is the floor alone),
// 1 = saturate, 2 = wrap around.
template <int ORD, int LD, int HOLD_P, bool WRAP_A>
__global__ void __launch_bounds__(256) lba_fixed_kernel(const Problem p) {
  constexpr int BM = 64, BN = 64, TM = 4, TN = 4, NT = 256, TX = BN / TN;
  constexpr int ROWS = BM + BN;
  constexpr int LPT = (ROWS + NT - 1) / NT;
  constexpr bool CHUNKED = ORD != ORD_SEQ;
  static_assert(ORD == ORD_SEQ || ORD == ORD_CHUNK_SLAB || ORD == ORD_CHUNK_ANY, "order");

  // m: mantissa (A: shifted left by 22), q: contribution to the right-shift count
  __shared__ __align__(16) int Am[2][BK][BM];
  __shared__ __align__(16) int Aq[2][BK][BM];
  __shared__ __align__(16) int Bm[2][BK][BN];
  __shared__ __align__(16) int Bq[2][BK][BN];

  const int tid = threadIdx.x;
  const int tx = tid % TX, ty = tid / TX;
  const int64_t m0 = (int64_t)blockIdx.x * BM;
  const int64_t n0 = (int64_t)blockIdx.y * BN;
  const int64_t K = p.K;
  const int nslab = (int)((K + BK - 1) / BK);

  RowLoader<BM, BN, NT, LD> loader;
  loader.init(p, tid, m0, n0);

  auto decode_store = [&](const uint4 (&raw)[LPT], int buf) {
#pragma unroll
    for (int l = 0; l < LPT; ++l) {
      const int r = tid + l * NT;
      if (r < ROWS) {
        const bool is_a = r < BM;
        int* dm = is_a ? &Am[buf][0][r] : &Bm[buf][0][r - BM];
        int* dq = is_a ? &Aq[buf][0][r] : &Bq[buf][0][r - BM];
        const int stride = is_a ? BM : BN;
        const uint32_t w4[4] = {raw[l].x, raw[l].y, raw[l].z, raw[l].w};
#pragma unroll
        for (int j = 0; j < BK; ++j) {
          const uint32_t c = (w4[j >> 2] >> (8 * (j & 3))) & 0xFFu;
          const int e = (int)((c >> 3) & 15u), f = (int)(c & 7u);
          int s = e ? 8 + f : f;            // value = s * 2^q
          const int q = e ? e - 10 : -9;
          if (c & 0x80u) s = -s;
          // right-shift count of the product = (22 - b_prod - qx) + (-qw)
          dm[j * stride] = is_a ? s << 22 : s;
          dq[j * stride] = is_a ? p.fx_shift0 - q : -q;
        }
      }
    }
  };

  int acc1[TM][TN];
  int acc2[CHUNKED ? TM : 1][CHUNKED ? TN : 1];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      acc1[i][j] = 0;
      if (CHUNKED) acc2[CHUNKED ? i : 0][CHUNKED ? j : 0] = 0;
    }

  const int lo_p = p.fx_lo_p, hi_p = p.fx_hi_p, sh_p = p.fx_sh_p;
  const int lo_a = p.fx_lo_a, hi_a = p.fx_hi_a, sh_a = p.fx_sh_a;
  const int dl = p.fx_dl, dr = p.fx_dr;  // product units -> accumulator units: << dl, then >> dr (one of them is 0)

  auto close_chunk = [&]() {  // second hierarchy: T <- Q_acc(C + T), C <- 0 (both already on the accumulator's grid)
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
      for (int j = 0; j < TN; ++j) {
        int& t2 = acc2[CHUNKED ? i : 0][CHUNKED ? j : 0];
        t2 = fx_hold<WRAP_A>(acc1[i][j] + t2, lo_a, hi_a, sh_a);
        acc1[i][j] = 0;
      }
  };

  // UP: the accumulator's grid is finer than the product's (shift left); else equal or coarser (shift right)
  auto mac_step = [&](int buf, int kk, auto up_tag) {
    constexpr bool UP = decltype(up_tag)::value;
    int2 a[TM], b[TN];
    {
      const int4 vm = *reinterpret_cast<const int4*>(&Am[buf][kk][ty * 4]);
      const int4 vq = *reinterpret_cast<const int4*>(&Aq[buf][kk][ty * 4]);
      a[0] = make_int2(vm.x, vq.x); a[1] = make_int2(vm.y, vq.y);
      a[2] = make_int2(vm.z, vq.z); a[3] = make_int2(vm.w, vq.w);
    }
    {
      const int4 vm = *reinterpret_cast<const int4*>(&Bm[buf][kk][tx * 4]);
      const int4 vq = *reinterpret_cast<const int4*>(&Bq[buf][kk][tx * 4]);
      b[0] = make_int2(vm.x, vq.x); b[1] = make_int2(vm.y, vq.y);
      b[2] = make_int2(vm.z, vq.z); b[3] = make_int2(vm.w, vq.w);
    }
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
      for (int j = 0; j < TN; ++j) {
        // Q_prod: floor(x w 2^b_prod), held to B_prod bits
        int np = fx_sar(a[i].x * b[j].x, a[i].y + b[j].y);
        if (HOLD_P == 1) np = fx_hold<false>(np, lo_p, hi_p, sh_p);
        if (HOLD_P == 2) np = fx_hold<true>(np, lo_p, hi_p, sh_p);
        // Q_acc: the sum on the accumulator's grid (S already lies on it, so only the product is re-cut), held
        acc1[i][j] = fx_hold<WRAP_A>(acc1[i][j] + (UP ? (np << dl) : (np >> dr)), lo_a, hi_a, sh_a);
      }
  };

  uint4 raw[LPT];
  int slabs_in_chunk = 0;
  int k_in_chunk = 0;
  if (nslab > 0) {
    loader.fetch(p, tid, 0, raw);
    decode_store(raw, 0);
  }
  __syncthreads();
  for (int s = 0; s < nslab; ++s) {
    const int buf = s & 1;
    if (s + 1 < nslab) loader.fetch(p, tid, s + 1, raw);
    if (ORD == ORD_CHUNK_ANY) {
      const int kmax = (int)((K - (int64_t)s * BK) < BK ? (K - (int64_t)s * BK) : BK);
#pragma unroll 1
      for (int kk = 0; kk < kmax; ++kk) {
        if (dl) mac_step(buf, kk, std::true_type());
        else mac_step(buf, kk, std::false_type());
        if (++k_in_chunk == p.chunk) {
          close_chunk();
          k_in_chunk = 0;
        }
      }
    } else {
      // zero-padded steps past K add floor(0) = 0 to a sum that is already held: no change
      if (dl) {
#pragma unroll 4
        for (int kk = 0; kk < BK; ++kk) mac_step(buf, kk, std::true_type());
      } else {
#pragma unroll 4
        for (int kk = 0; kk < BK; ++kk) mac_step(buf, kk, std::false_type());
      }
      if (ORD == ORD_CHUNK_SLAB) {
        if (++slabs_in_chunk == p.chunk_slabs) {
          close_chunk();
          slabs_in_chunk = 0;
        }
      }
    }
    if (s + 1 < nslab) decode_store(raw, buf ^ 1);
    __syncthreads();
  }
  if (ORD == ORD_CHUNK_SLAB && slabs_in_chunk > 0) close_chunk();
  if (ORD == ORD_CHUNK_ANY && k_in_chunk > 0) close_chunk();

  // ---- epilogue: integer -> binary32 (exact, B <= 24), * 2^-b_acc, scales and bias in binary32
  float* const outz = p.out + (int64_t)blockIdx.z * p.batch_out;
#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const int64_t m = m0 + ty * 4 + i;
    if (m >= p.M) continue;
    const float sa = p.sa[p.sa_per_row ? m : 0];
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      const int64_t n = n0 + tx * 4 + j;
      if (n >= p.N) continue;
      const int t = CHUNKED ? acc2[CHUNKED ? i : 0][CHUNKED ? j : 0] : acc1[i][j];
      const float y = __fmul_rn(__int2float_rn(t), p.fx_unit);
      const float sb = p.sb[p.sb_per_col ? n : 0];
      float r = __fmul_rn(__fmul_rn(y, sa), sb);
      if (p.bias) r = __fadd_rn(r, p.bias[n]);
      outz[m * p.N + n] = r;
    }
  }
}

}  // namespace lba
