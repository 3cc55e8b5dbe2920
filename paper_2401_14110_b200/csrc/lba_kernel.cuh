// LBA contraction kernels for sm_100a: out[m][n] = epilogue(chain_k FMAq(A[m][k], B[n][k], .)).
//
// The method rounds after every single addition (Eq. 4 of the paper), so no group of products may be summed
// exactly first: tensor-core MMA is excluded by definition and the kernels are bound by CUDA-core issue slots
// and pipes.  Everything below exists to keep the per-MAC instruction count low.
//
// Carrier arithmetic.  Values are carried in binary32 registers, scaled by a power of two so that the
// format's underflow threshold R_UF sits at binary32's smallest normal 2^-126:
//   * product:   p' = x' * w' with x' = x * 2^sx, w' = w * 2^sw, sx + sw = b_prod - 126.  The product of two
//     E4M3 values has at most 8 significant bits, so it is exact; `mul.ftz` then flushes exactly the products
//     with |x*w| < R_UF_prod (Eq. 2, second case).
//   * sum:       t = fma.rz.ftz(p', 2^(b_acc-b_prod), S').  The FMA forms p'*c + S' exactly and rounds once
//     toward zero to 24 bits; cutting a toward-zero result to M < 24 bits again toward zero equals cutting the
//     exact sum (truncations compose), so `t & mask` is the floor of Eq. 2 on the exact sum.  `.ftz` flushes
//     exactly the sums below R_UF_acc, because a toward-zero rounding never moves a value across 2^-126.
//   * saturation: min.xorsign.abs(t, R_OF') = sign(t) * min(|t|, R_OF'), one instruction.
// Nearest-even does not compose with a binary32 rounding, so that mode first builds the round-to-odd image of
// the exact sum (from directed roundings of the FMA) and rounds that.
// The host proves per call which branches of Eq. 2 E4M3 inputs can reach and picks the cheapest exact variant.
//
// Two kernels share the operand loaders:
//   lba_contract_packed_kernel  packed f32x2 arithmetic (two outputs per instruction), the magnitude clamp
//                               skipped per slab under a norm bound; floor and nearest-even; the fast path
//   lba_contract_kernel         scalar arithmetic, always clamped; any chunk length, 24-bit accumulator
// Data path of both: a CTA owns a BM x BN output tile and walks K in slabs of 16 bytes per row; each thread
// fetches 16-byte row pieces (one 128-bit load), decodes the 16 E4M3 bytes to scaled binary32 once, and stores
// them k-major into shared memory (double buffered, one barrier per slab).  Each thread keeps a TM x TN
// register micro-tile of running sums and walks k in order; K is never split across threads, so the paper's
// accumulation order is kept by construction.
#pragma once
#include <cstdint>
#include <type_traits>
#include <cuda_runtime.h>

namespace lba {

enum QMode { QM_FLOOR_FAST = 0, QM_FLOOR_FULL = 1, QM_RNE_FULL = 2, QM_RNE_WIDE = 3, QM_COUNT = 4 };
// ORD_CHUNK16: chunk == BK, the paper's chunk size; only the packed floor kernel specialises it
enum OrdMode { ORD_SEQ = 0, ORD_CHUNK_SLAB = 1, ORD_CHUNK_ANY = 2, ORD_CHUNK16 = 3, ORD_COUNT = 4 };
enum LoadMode { LD_GEMM_VEC = 0, LD_CONV_VEC = 1, LD_ANY = 2, LD_COUNT = 3 };

constexpr int BK = 16;  // bytes of K per row per slab = one 128-bit load = one paper-sized chunk

struct QConst {
  uint32_t mask;     // keeps sign, exponent and the top M mantissa bits
  uint32_t rne_add;  // nearest-even: 2^(22-M) - 1
  uint32_t rne_lsb;  // nearest-even: 1, or 0 when M = 23
  int32_t rne_shift; // nearest-even: 23 - M
  float sat;         // R_OF in carrier scaling, or FLT_MAX when saturation is unreachable
};

struct Problem {
  const uint8_t* A;   // GEMM: [M][K]; conv: x, NHWC
  const uint8_t* B;   // [N][K]
  const float* sa;
  const float* sb;
  const float* bias;
  float* out;
  int64_t M, N, K;
  // batched GEMM: problem z = blockIdx.z reads A + z*batch_a, B + z*batch_b (bytes) and writes out + z*batch_out
  // (floats); a plain call has batch = 1
  int64_t batch, batch_a, batch_b, batch_out;
  int sa_per_row, sb_per_col;
  int is_conv, H, W, Cin, KH, KW, sh, sw, ph, pw, Hout, Wout;
  float dec_a, dec_b;  // decode multipliers 2^(120+sx), 2^(120+sw)
  float c;             // 2^(b_acc' - b_prod'): product carrier -> accumulator carrier
  float un1, un2;      // un1*un2 = accumulator carrier -> real value
  QConst qp, qa;
  int chunk_slabs;     // ORD_CHUNK_SLAB: chunk / BK
  int chunk;           // ORD_CHUNK_ANY
  // packed floor kernel only
  float pk_a, pk_b;    // 2^sx, 2^sw: decoded value -> product-carrier operand
  float nrm_scale;     // 2^-(e_max_acc + 1), or 0 when the accumulator cannot saturate
  float inv_top;       // accumulator carrier -> fraction of 2^(e_max_acc + 1)
  int pq;              // PackedProd: what Q_prod does beyond the flush
  int rne_packed;      // nearest-even: 1 if the packed kernel's conditions hold (see the host plan)
  int in_m4e3;         // operands are bytes of the paper's M4E3 W/A format (Sec. 3.1) instead of OCP E4M3
  float rne_k_acc, rne_k_prod;  // 2^(23 - M) for the accumulator and the product format
  // clamp elision: a slab or fold runs without the magnitude clamp while (bound + growth) * factor < clamp_lim.
  // Floor never raises a magnitude: factors 1, limit just under 1 (of 2^(e_max+1)).  Nearest-even can raise one by
  // half a grid step per rounding: slab_factor bounds sixteen such steps (and the product's own rounding),
  // fold_factor one, and the limit keeps every sum at or below R_OF, which then rounds to at most R_OF.
  float clamp_lim, slab_factor, fold_factor;
  // straight-through-estimator masks (tracking variants of the scalar kernel only)
  uint32_t *mask1, *mask2;
  int64_t mask2_words;  // ceil(chunks / 32)
  // DIFF comparison: carried in "accumulator carrier * diff_scale" so that differences of neighbouring
  // accumulator values stay normal numbers
  float diff_scale;    // accumulator carrier -> comparison scaling (2^32)
  float diff_a_scale;  // product-carrier A operand -> operand whose product with B is |x w| in comparison scaling
  float diff_eps1;     // eps1 in comparison scaling
  float diff_eps2;     // eps2 (a pure ratio)
  float ste_limit;     // packed mask variant: 0.999 * R_OF / 2^(e_max + 1) = 0.999 * (1 - 2^-(M_acc + 1))
  // fixed-point accumulation (Eq. 1; the integer kernel only)
  int fx_shift0;               // 22 - b_prod
  int fx_lo_p, fx_hi_p, fx_sh_p, fx_hold_p;  // product: range of the integer, 32 - B, 0 = never out of range / 1 = saturate / 2 = wrap
  int fx_lo_a, fx_hi_a, fx_sh_a, fx_wrap_a;  // accumulator
  int fx_dl, fx_dr;            // product units -> accumulator units: << dl then >> dr
  float fx_unit;               // 2^-b_acc
};

// ------------------------------------------------------------------ scalar building blocks
__device__ __forceinline__ float mul_ftz(float a, float b) {
  float d;
  asm("mul.rn.ftz.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
  return d;
}
__device__ __forceinline__ float mul_ieee(float a, float b) {  // subnormal operands honoured
  float d;
  asm("mul.rn.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
  return d;
}
__device__ __forceinline__ float add_ieee(float a, float b) {
  float d;
  asm("add.rn.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
  return d;
}
__device__ __forceinline__ float fma_rz_ftz(float a, float b, float c) {
  float d;
  asm("fma.rz.ftz.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float fma_rm(float a, float b, float c) {
  float d;
  asm("fma.rm.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float fma_rp(float a, float b, float c) {
  float d;
  asm("fma.rp.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float fma_rn(float a, float b, float c) {
  float d;
  asm("fma.rn.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// sign(t) * min(|t|, r) for r > 0
__device__ __forceinline__ float clamp_mag(float t, float r) {
  float d;
  asm("min.xorsign.abs.f32 %0, %1, %2;" : "=f"(d) : "f"(t), "f"(r));
  return d;
}
__device__ __forceinline__ float and_bits(float t, uint32_t m) { return __uint_as_float(__float_as_uint(t) & m); }

// nearest-even cut of a binary32 pattern to M mantissa bits (carry into the exponent is the
// wanted behaviour); exact when t itself is exact or is the round-to-odd image of the exact value
__device__ __forceinline__ float rne_bits(float t, const QConst& q) {
  uint32_t u = __float_as_uint(t);
  u = u + q.rne_add + ((u >> q.rne_shift) & q.rne_lsb);
  return __uint_as_float(u & q.mask);
}

// Q_prod(x*w) in product-carrier scaling.
template <int QM>
__device__ __forceinline__ float q_prod(float a, float b, const QConst& qp) {
  float p = mul_ftz(a, b);  // exact; flushes |x*w| < R_UF_prod
  if (QM == QM_FLOOR_FULL) {
    p = clamp_mag(and_bits(p, qp.mask), qp.sat);
  } else if (QM == QM_RNE_FULL) {
    p = clamp_mag(rne_bits(p, qp), qp.sat);
  }
  return p;
}

// S <- Q_acc(P*c + S) in accumulator-carrier scaling (c = 1 and P = chunk sum at the second level).
template <int QM>
__device__ __forceinline__ float q_acc_fma(float p, float c, float s, const QConst& qa) {
  if (QM == QM_FLOOR_FAST || QM == QM_FLOOR_FULL) {
    float t = fma_rz_ftz(p, c, s);
    return clamp_mag(and_bits(t, qa.mask), qa.sat);
  } else if (QM == QM_RNE_FULL) {
    float tz = fma_rz_ftz(p, c, s);   // zero exactly when the exact sum is below R_UF_acc (or is 0)
    float tm = fma_rm(p, c, s);       // neighbours of the exact sum in binary32
    float tp = fma_rp(p, c, s);
    // round-to-odd: if the sum is inexact tm and tp are adjacent and exactly one is odd
    float ro = (__float_as_uint(tm) & 1u) ? tm : tp;
    float r = clamp_mag(rne_bits(ro, qa), qa.sat);
    return tz == 0.0f ? 0.0f : r;
  } else {  // QM_RNE_WIDE: 24-bit accumulator, nothing of Eq. 2 reachable: one IEEE addition
    return fma_rn(p, c, s);
  }
}

// E4M3 byte (held in the top byte of `top`, lower bytes zero) -> value * mul.
// (byte & 0x7F) << 20 read as binary32 is value * 2^-120 for normal and subnormal codes alike
// (E4M3 subnormals land on binary32 subnormals), so one IEEE multiply finishes the decode.
__device__ __forceinline__ float decode_e4m3_top(uint32_t top, float mul) {
  float mag = __uint_as_float((top >> 4) & 0x07F00000u);
  float v = mul_ieee(mag, mul);
  return __uint_as_float(__float_as_uint(v) | (top & 0x80000000u));
}

// Byte of the paper's W/A format (Sec. 3.1; s eee mmmm, held in the top byte of `top`) -> its value
// (-1)^s 2^e (1 + m/16): the seven magnitude bits, moved to the low exponent and high mantissa bits of a binary32
// pattern and added to the pattern of 1.0, are that number; the code e = m = 0 is zero.
__device__ __forceinline__ float decode_m4e3_top(uint32_t top) {
  const uint32_t mag = (top >> 5) & 0x03F80000u;
  const uint32_t bits = mag ? mag + 0x3F800000u : 0u;
  return __uint_as_float(bits | (top & 0x80000000u));
}

__device__ __forceinline__ uint32_t byte_to_top(uint32_t word, int j) {  // j in 0..3
  return __byte_perm(word, 0u, (uint32_t)(j << 12) | 0x0444u);
}

// ------------------------------------------------------------------ packed building blocks
// Two binary32 values in one 64-bit register pair and the f32x2 instructions of sm_100 on them.
typedef unsigned long long u64;

__device__ __forceinline__ u64 pack2(float lo, float hi) {
  u64 d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
  return d;
}
__device__ __forceinline__ void unpack2(u64 v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ u64 mul2_ftz(u64 a, u64 b) {
  u64 d;
  asm("mul.rn.ftz.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ u64 fma2_rz_ftz(u64 a, u64 b, u64 c) {
  u64 d;
  asm("fma.rz.ftz.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ u64 fma2_rn(u64 a, u64 b, u64 c) {
  u64 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ u64 fma2_rn_ftz(u64 a, u64 b, u64 c) {
  u64 d;
  asm("fma.rn.ftz.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
// Nearest-even cut of a pair of binary32 values to M mantissa bits on the FP32 pipe.  With e the value's own
// exponent, K = 1.5 * 2^(23-M) * 2^e (same sign) moves the value into a binade whose unit in the last place is the
// target grid step, so the addition v + K itself rounds to nearest-even on that grid (K/ulp is even, so ties carry
// over); subtracting K again is exact.  k0 = +-1.5 * 2^e is one logic operation per value (sign and exponent
// kept, mantissa set to 1.5), and both steps are one packed FMA each: r = k0 * ks + v, result = k0 * (-ks) + r
// with ks = 2^(23-M).  A zero stays zero (k0 is then a subnormal; r = k0 * ks is cancelled exactly).  Needs M <= 21
// and exponent headroom for K, which the host checks.  `v` must be exact (or the correctly rounded binary32 image
// of a sum whose rounding cannot decide an M-bit tie; see the host's conditions for the packed nearest-even path).
__device__ __forceinline__ u64 rne2_fp(u64 v, u64 ks, u64 nks) {
  uint32_t lo, hi;
  asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v));
  u64 k0;
  asm("mov.b64 %0, {%1, %2};" : "=l"(k0) : "r"((lo & 0xFF800000u) | 0x00400000u), "r"((hi & 0xFF800000u) | 0x00400000u));
  const u64 r = fma2_rn(k0, ks, v);
  return fma2_rn(k0, nks, r);
}
__device__ __forceinline__ u64 mul2_rn_ftz(u64 a, u64 b) {
  u64 d;
  asm("mul.rn.ftz.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ u64 add2_rn_ftz(u64 a, u64 b) {
  u64 d;
  asm("add.rn.ftz.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ u64 mul2_rz_ftz(u64 a, u64 b) {
  u64 d;
  asm("mul.rz.ftz.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ u64 add2_rz_ftz(u64 a, u64 b) {
  u64 d;
  asm("add.rz.ftz.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ u64 mul2_rn(u64 a, u64 b) {  // subnormal operands and results honoured
  u64 d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// ------------------------------------------------------------------ operand fetch
// Each thread fetches, per slab, 16-byte pieces of the rows r = tid + l*NT of the CTA's A tile
// (r < BM) and B tile (BM <= r < BM + BN).  Rows past the matrix edge and padded convolution taps
// read as zero bytes, i.e. the value 0.
template <int BM, int BN, int NT, int LD>
struct RowLoader {
  static constexpr int ROWS = BM + BN;
  static constexpr int LPT = (ROWS + NT - 1) / NT;
  const uint8_t* row_ptr[LPT];
  bool row_ok[LPT];
  int ih0[LPT], iw0[LPT];               // conv: top-left input coordinate of the receptive field
  int ld_kh = 0, ld_kw = 0, ld_c0 = 0;  // conv vector path: position of the next slab inside (kh, kw, c_in)
  // conv byte-wise path: for one output position and one kh, the taps (kw, c_in) are KW*C_in contiguous
  // bytes of the input row ih0 + kh; the cursor is (kh, offset inside that run) of the next slab's first k
  int any_kh = 0, any_off = 0;

  __device__ __forceinline__ void init(const Problem& p, int tid, int64_t m0, int64_t n0) {
    const uint8_t* const baseA = p.A + (int64_t)blockIdx.z * p.batch_a;
    const uint8_t* const baseB = p.B + (int64_t)blockIdx.z * p.batch_b;
#pragma unroll
    for (int l = 0; l < LPT; ++l) {
      const int r = tid + l * NT;
      row_ptr[l] = nullptr;
      row_ok[l] = false;
      ih0[l] = 0;
      iw0[l] = 0;
      if (r < BM) {
        const int64_t m = m0 + r;
        if (m < p.M) {
          row_ok[l] = true;
          if (LD == LD_GEMM_VEC || (LD == LD_ANY && !p.is_conv)) {
            row_ptr[l] = baseA + m * p.K;
          } else {
            const int ow = (int)(m % p.Wout);
            const int64_t t = m / p.Wout;
            const int oh = (int)(t % p.Hout);
            const int64_t b = t / p.Hout;
            ih0[l] = oh * p.sh - p.ph;
            iw0[l] = ow * p.sw - p.pw;
            row_ptr[l] = baseA + b * ((int64_t)p.H * p.W * p.Cin);
          }
        }
      } else if (r < ROWS) {
        const int64_t n = n0 + (r - BM);
        if (n < p.N) {
          row_ok[l] = true;
          row_ptr[l] = baseB + n * p.K;
        }
      }
    }
  }

  // slabs must be requested in increasing order, each once (the conv vector path keeps a cursor)
  __device__ __forceinline__ void fetch(const Problem& p, int tid, int slab, uint4 (&raw)[LPT]) {
    const int64_t K = p.K;
    const int64_t k0 = (int64_t)slab * BK;
#pragma unroll
    for (int l = 0; l < LPT; ++l) {
      const int r = tid + l * NT;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (row_ok[l]) {
        const bool is_a = r < BM;
        if (LD == LD_GEMM_VEC || (LD == LD_CONV_VEC && !is_a)) {
          v = __ldg(reinterpret_cast<const uint4*>(row_ptr[l] + k0));
        } else if (LD == LD_CONV_VEC) {
          const int ih = ih0[l] + ld_kh, iw = iw0[l] + ld_kw;
          if (ih >= 0 && ih < p.H && iw >= 0 && iw < p.W)
            v = __ldg(reinterpret_cast<const uint4*>(row_ptr[l] + ((int64_t)ih * p.W + iw) * p.Cin + ld_c0));
        } else {  // LD_ANY: byte-wise, any K, any alignment, GEMM or conv
          uint32_t w4[4] = {0u, 0u, 0u, 0u};
          if (!is_a || !p.is_conv) {
#pragma unroll
            for (int j = 0; j < BK; ++j) {
              const int64_t k = k0 + j;
              const uint32_t byte = k < K ? (uint32_t)__ldg(row_ptr[l] + k) : 0u;
              w4[j >> 2] |= byte << (8 * (j & 3));
            }
          } else {
            // walk the runs: no division per byte.  Bytes of a run are valid where the tap column
            // iw0 + kw lies inside the image, i.e. for run offsets in [lo, lo + span)
            const int run = p.KW * p.Cin;
            const int kw_lo = iw0[l] < 0 ? -iw0[l] : 0;
            const int kw_hi = p.W - iw0[l] < p.KW ? p.W - iw0[l] : p.KW;
            const int lo = kw_lo * p.Cin;
            const unsigned span = kw_hi > kw_lo ? (unsigned)((kw_hi - kw_lo) * p.Cin) : 0u;
            const int64_t row_pitch = (int64_t)p.W * p.Cin;
            int off = any_off;
            int ih = ih0[l] + any_kh;
            // address of run offset 0 of input row ih (left of the image when iw0 < 0; only valid bytes are read)
            int64_t pos = (int64_t)ih * row_pitch + (int64_t)iw0[l] * p.Cin + off;
#pragma unroll
            for (int j = 0; j < BK; ++j) {
              const bool ok = (k0 + j < K) && ((unsigned)ih < (unsigned)p.H) && ((unsigned)(off - lo) < span);
              const uint32_t byte = ok ? (uint32_t)__ldg(row_ptr[l] + pos) : 0u;
              w4[j >> 2] |= byte << (8 * (j & 3));
              ++off;
              ++pos;
              if (off == run) {
                off = 0;
                ++ih;
                pos += row_pitch - run;
              }
            }
          }
          v = make_uint4(w4[0], w4[1], w4[2], w4[3]);
        }
      }
      raw[l] = v;
    }
    skip_slab(p);
  }

  // move the convolution cursors past one slab without fetching it (fetch does this itself; a CTA that
  // handles every second slab calls it once more)
  __device__ __forceinline__ void skip_slab(const Problem& p) {
    if (LD == LD_ANY && p.is_conv) {  // advance the run cursor by one slab
      const int run = p.KW * p.Cin;
      any_off += BK;
      while (any_off >= run) {
        any_off -= run;
        ++any_kh;
      }
    }
    if (LD == LD_CONV_VEC) {  // advance (kh, kw, c0) to the next slab
      ld_c0 += BK;
      if (ld_c0 >= p.Cin) {
        ld_c0 = 0;
        if (++ld_kw == p.KW) {
          ld_kw = 0;
          ++ld_kh;
        }
      }
    }
  }
};

// ------------------------------------------------------------------ the kernel
// TRACK selects the re-computation passes of the straight-through estimators (Sec. 4, App. D; floor quantisers
// only).  Instead of the sums the kernel then writes what the backward pass needs:
//   TRACK_LAST_OF  sequential order; `out` is read as int32 [M][N]: index of the last step whose exact sum
//                  Q_prod(x_i w_i) + S_i reached R_OF, or -1 (all the recursive overflow estimator needs);
//   TRACK_MASK_OF  one bit per FMAq step, 1 iff |Q_prod(x_i w_i) + S_i| < R_OF (STE^OF);
//   TRACK_MASK_DIFF one bit per FMAq step, 1 iff |z - S| > eps2 * (|x_i w_i| + eps1) (STE^DIFF), each of the three
//                  operations rounded to binary32.
// Masks: mask1 uint32 [M][ceil(K/32)][N], bit i%32 of word i/32 for step i; in chunked order mask2
// [M][ceil(chunks/32)][N] holds the bits of the folds T <- Q_acc(C + T), the chunk sum C in the product's place.
enum { TRACK_NONE = 0, TRACK_LAST_OF = 1, TRACK_MASK_OF = 2, TRACK_MASK_DIFF = 3 };

template <int BM, int BN, int TM, int TN, int QM, int ORD, int LD, int TRACK = TRACK_NONE>
__global__ void __launch_bounds__((BM / TM) * (BN / TN), TRACK == TRACK_MASK_DIFF ? 2 : 1) lba_contract_kernel(const Problem p) {
  static_assert(TRACK == TRACK_NONE || QM == QM_FLOOR_FULL || QM == QM_FLOOR_FAST, "tracking variants use the floor quantisers");
  static_assert(TRACK != TRACK_LAST_OF || ORD == ORD_SEQ, "last-overflow index: sequential order");
  static_assert(TRACK == TRACK_NONE || ORD != ORD_CHUNK16, "tracking variants: generic orders");
  constexpr bool MASKS = TRACK == TRACK_MASK_OF || TRACK == TRACK_MASK_DIFF;
  constexpr bool DIFF = TRACK == TRACK_MASK_DIFF;
  constexpr int NT = (BM / TM) * (BN / TN);
  constexpr int TX = BN / TN;
  constexpr int ROWS = BM + BN;
  constexpr int LPT = (ROWS + NT - 1) / NT;  // 16-byte row pieces fetched per thread per slab
  constexpr bool CHUNKED = ORD != ORD_SEQ;
  static_assert(TM == 4 || TM == 8, "micro-tile rows");
  static_assert(TN == 4 || TN == 8, "micro-tile cols");

  __shared__ __align__(16) float As[2][BK][BM];
  __shared__ __align__(16) float Bs[2][BK][BN];

  const int tid = threadIdx.x;
  const int tx = tid % TX, ty = tid / TX;
  const int64_t m0 = (int64_t)blockIdx.x * BM;
  const int64_t n0 = (int64_t)blockIdx.y * BN;
  const int64_t K = p.K;
  const int nslab = (int)((K + BK - 1) / BK);

  RowLoader<BM, BN, NT, LD> loader;
  loader.init(p, tid, m0, n0);
  auto fetch = [&](int slab, uint4 (&raw)[LPT]) { loader.fetch(p, tid, slab, raw); };

  auto decode_store = [&](const uint4 (&raw)[LPT], int buf) {
#pragma unroll
    for (int l = 0; l < LPT; ++l) {
      const int r = tid + l * NT;
      if (r < ROWS) {
        const bool is_a = r < BM;
        const float mul = is_a ? p.dec_a : p.dec_b;
        float* dst = is_a ? &As[buf][0][r] : &Bs[buf][0][r - BM];
        const int stride = is_a ? BM : BN;
        const uint32_t w4[4] = {raw[l].x, raw[l].y, raw[l].z, raw[l].w};
#pragma unroll
        for (int j = 0; j < BK; ++j) {
          const uint32_t top = byte_to_top(w4[j >> 2], j & 3);
          dst[j * stride] = p.in_m4e3 ? mul_ieee(decode_m4e3_top(top), mul) : decode_e4m3_top(top, mul);
        }
      }
    }
  };

  // ---- running sums: first hierarchy (or the sequential S) and, in chunked order, the second
  float acc1[TM][TN];
  float acc2[CHUNKED ? TM : 1][CHUNKED ? TN : 1];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc1[i][j] = 0.0f;
  if (CHUNKED) {
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
      for (int j = 0; j < TN; ++j) acc2[CHUNKED ? i : 0][CHUNKED ? j : 0] = 0.0f;
  }

  const float cc = p.c;
  const QConst qp = p.qp, qa = p.qa;

  // ---- tracking state
  constexpr bool LAST = TRACK == TRACK_LAST_OF;
  int last[LAST ? TM : 1][LAST ? TN : 1];                       // TRACK_LAST_OF
  uint32_t bits1[MASKS ? TM : 1][MASKS ? TN : 1];               // current word of mask1
  uint32_t half1[MASKS ? TM : 1][MASKS ? TN : 1];               // the 16 bits of the current slab
  uint32_t bits2[MASKS && CHUNKED ? TM : 1][MASKS && CHUNKED ? TN : 1];
  float prev1[DIFF ? TM : 1][DIFF ? TN : 1];                    // S and T in the comparison's scaling
  float prev2[DIFF && CHUNKED ? TM : 1][DIFF && CHUNKED ? TN : 1];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      if (LAST) last[LAST ? i : 0][LAST ? j : 0] = -1;
      if (MASKS) bits1[MASKS ? i : 0][MASKS ? j : 0] = half1[MASKS ? i : 0][MASKS ? j : 0] = 0u;
      if (MASKS && CHUNKED) bits2[MASKS && CHUNKED ? i : 0][MASKS && CHUNKED ? j : 0] = 0u;
      if (DIFF) prev1[DIFF ? i : 0][DIFF ? j : 0] = 0.0f;
      if (DIFF && CHUNKED) prev2[DIFF && CHUNKED ? i : 0][DIFF && CHUNKED ? j : 0] = 0.0f;
    }
  int kbase = 0;     // global index of the slab's first step
  int chunk_id = 0;  // index of the chunk being accumulated
  uint32_t* const mask1z = MASKS ? p.mask1 : nullptr;
  uint32_t* const mask2z = MASKS ? p.mask2 : nullptr;
  const int64_t W1 = MASKS ? (K + 31) / 32 : 0;
  const int64_t W2 = MASKS ? p.mask2_words : 0;
  const float dscale = p.diff_scale, deps1 = p.diff_eps1, deps2 = p.diff_eps2;

  // one word of a mask for every output of the thread: word w of output (m, n) is base[(m * words + w) * N + n],
  // so the four neighbouring outputs of a micro-tile row go out as one 16-byte store where alignment allows
  auto flush_words = [&](uint32_t* base, int64_t words, int64_t w, auto& bits) {
    const bool vec = (p.N % 4 == 0) && ((reinterpret_cast<uintptr_t>(base) & 15) == 0);
#pragma unroll
    for (int i = 0; i < TM; ++i) {
      const int64_t m = m0 + (i / 4) * (BM / 2) + ty * 4 + (i % 4);
#pragma unroll
      for (int h = 0; h < TN / 4; ++h) {
        const int64_t n = n0 + h * (BN / 2) + tx * 4;
        uint32_t* dst = base + (m * words + w) * p.N + n;
        if (m < p.M) {
          if (vec && n + 3 < p.N) {
            *reinterpret_cast<uint4*>(dst) = make_uint4(bits[i][h * 4], bits[i][h * 4 + 1], bits[i][h * 4 + 2], bits[i][h * 4 + 3]);
          } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (n + j < p.N) dst[j] = bits[i][h * 4 + j];
          }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) bits[i][h * 4 + j] = 0u;
      }
    }
  };

  // STE bit of one step: t = the exact sum cut toward zero to M bits (|t| >= R_OF exactly when the exact
  // sum is), z = Q_acc of it, u = the unquantised product or the chunk sum (DIFF scaling), s_prev = S before
  auto ste_bit = [&](float t, float z, float u, float& s_prev) -> bool {
    if (DIFF) {
      const float zd = mul_ieee(z, dscale);                       // exact: z is a normal number
      const float d = fabsf(__fadd_rn(zd, -s_prev));              // one rounding, as the definition says
      s_prev = zd;
      const float thr = __fmul_rn(deps2, __fadd_rn(fabsf(u), deps1));
      return d > thr;
    }
    (void)z; (void)u; (void)s_prev;
    return fabsf(t) < qa.sat;
  };

  auto close_chunk = [&]() {  // second hierarchy: T <- Q_acc(C + T), C <- 0
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
      for (int j = 0; j < TN; ++j) {
        float& t2 = acc2[CHUNKED ? i : 0][CHUNKED ? j : 0];
        if (MASKS && CHUNKED) {
          const float t = and_bits(fma_rz_ftz(acc1[i][j], 1.0f, t2), qa.mask);
          const float z = clamp_mag(t, qa.sat);
          const float u = DIFF ? mul_ieee(acc1[i][j], dscale) : 0.0f;
          if (ste_bit(t, z, u, prev2[DIFF && CHUNKED ? i : 0][DIFF && CHUNKED ? j : 0]))
            bits2[MASKS && CHUNKED ? i : 0][MASKS && CHUNKED ? j : 0] |= 1u << (chunk_id & 31);
          t2 = z;
          if (DIFF) prev1[DIFF ? i : 0][DIFF ? j : 0] = 0.0f;
        } else {
          t2 = q_acc_fma<QM>(acc1[i][j], 1.0f, t2, qa);
        }
        acc1[i][j] = 0.0f;
      }
    if constexpr (MASKS && CHUNKED) {
      if ((chunk_id & 31) == 31) flush_words(mask2z, W2, (int64_t)(chunk_id >> 5), bits2);
      ++chunk_id;
    }
  };

  auto mac_step = [&](int buf, int kk) {
    float a[TM], b[TN];
#pragma unroll
    for (int h = 0; h < TM / 4; ++h) {
      const float4 v = *reinterpret_cast<const float4*>(&As[buf][kk][h * (BM / 2) + ty * 4]);
      a[h * 4 + 0] = v.x; a[h * 4 + 1] = v.y; a[h * 4 + 2] = v.z; a[h * 4 + 3] = v.w;
    }
#pragma unroll
    for (int h = 0; h < TN / 4; ++h) {
      const float4 v = *reinterpret_cast<const float4*>(&Bs[buf][kk][h * (BN / 2) + tx * 4]);
      b[h * 4 + 0] = v.x; b[h * 4 + 1] = v.y; b[h * 4 + 2] = v.z; b[h * 4 + 3] = v.w;
    }
    if constexpr (DIFF) {
      // STE^DIFF: two neighbouring columns share the packed instructions.  Per pair and step: product, sum, the sum
      // in the comparison's scaling, its distance from the previous one, |x w| + eps1 and the threshold are one f32x2
      // instruction each; every rounding is the scalar definition's (the products and rescalings are exact; the previous
      // sum of the first hierarchy is the accumulator itself before the step, so only the folds keep a copy).  The bit
      // is the sign of thr - |d| (negative exactly when |d| > thr: a difference of two binary32 numbers never rounds
      // to zero), shifted into the slab's halfword from below, so the halfword holds the steps in reverse until the
      // slab ends.
      u64 b2[TN / 2], babs2[TN / 2];
#pragma unroll
      for (int jp = 0; jp < TN / 2; ++jp) {
        b2[jp] = pack2(b[2 * jp], b[2 * jp + 1]);
        babs2[jp] = pack2(fabsf(b[2 * jp]), fabsf(b[2 * jp + 1]));
      }
      const u64 cc2 = pack2(cc, cc), ds2 = pack2(dscale, dscale), nds2 = pack2(-dscale, -dscale);
      const u64 e1 = pack2(deps1, deps1), e2 = pack2(deps2, deps2);
#pragma unroll
      for (int i = 0; i < TM; ++i) {
        const u64 a2 = pack2(a[i], a[i]);
        const float ada = fabsf(mul_ieee(a[i], p.diff_a_scale));
        const u64 ada2 = pack2(ada, ada);
#pragma unroll
        for (int jp = 0; jp < TN / 2; ++jp) {
          u64 pr = mul2_ftz(a2, b2[jp]);  // exact; flushes |x w| < R_UF_prod
          if (QM == QM_FLOOR_FULL) {
            float plo, phi;
            unpack2(pr, plo, phi);
            pr = pack2(clamp_mag(and_bits(plo, qp.mask), qp.sat), clamp_mag(and_bits(phi, qp.mask), qp.sat));
          }
          float lo, hi;
          const u64 s_old = pack2(acc1[i][2 * jp], acc1[i][2 * jp + 1]);
          unpack2(fma2_rz_ftz(pr, cc2, s_old), lo, hi);
          lo = clamp_mag(and_bits(lo, qa.mask), qa.sat);
          hi = clamp_mag(and_bits(hi, qa.mask), qa.sat);
          acc1[i][2 * jp] = lo;
          acc1[i][2 * jp + 1] = hi;
          const u64 zd = mul2_rn(pack2(lo, hi), ds2);                                   // exact: the sums are normal numbers
          float dlo, dhi, tlo, thi;
          unpack2(fma2_rn(s_old, nds2, zd), dlo, dhi);          // zd - S_prev * dscale (exact product), one rounding
          unpack2(mul2_rn(fma2_rn(ada2, babs2[jp], e1), e2), tlo, thi);                 // eps2 * (|x w| + eps1)
          uint32_t& h0 = half1[MASKS ? i : 0][MASKS ? 2 * jp : 0];
          uint32_t& h1 = half1[MASKS ? i : 0][MASKS ? 2 * jp + 1 : 0];
          h0 = __funnelshift_l(__float_as_uint(add_ieee(tlo, -fabsf(dlo))), h0, 1);
          h1 = __funnelshift_l(__float_as_uint(add_ieee(thi, -fabsf(dhi))), h1, 1);
        }
      }
      (void)kk;
      return;
    }
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
      for (int j = 0; j < TN; ++j) {
        if (TRACK != TRACK_NONE) {
          // the exact sum reaches R_OF exactly when its toward-zero image cut to M bits does (R_OF is on that
          // grid); zero-padded steps past K are not steps of the chain: no index, bit 0
          const float t = and_bits(fma_rz_ftz(q_prod<QM>(a[i], b[j], qp), cc, acc1[i][j]), qa.mask);
          const float z = clamp_mag(t, qa.sat);
          const bool real_step = kbase + kk < (int)K;
          if (LAST) {
            if (fabsf(t) >= qa.sat && real_step) last[LAST ? i : 0][LAST ? j : 0] = kbase + kk;
          } else {
            const float u = 0.0f;
            // bit kk of the slab's halfword; steps past K are cleared when the halfword joins its word
            if (ste_bit(t, z, u, prev1[DIFF ? i : 0][DIFF ? j : 0])) half1[MASKS ? i : 0][MASKS ? j : 0] |= 1u << kk;
          }
          acc1[i][j] = z;
        } else {
          acc1[i][j] = q_acc_fma<QM>(q_prod<QM>(a[i], b[j], qp), cc, acc1[i][j], qa);
        }
      }
  };

  // ---- main loop
  uint4 raw[LPT];
  int slabs_in_chunk = 0;  // ORD_CHUNK_SLAB
  int k_in_chunk = 0;      // ORD_CHUNK_ANY
  if (nslab > 0) {
    fetch(0, raw);
    decode_store(raw, 0);
  }
  __syncthreads();
  for (int s = 0; s < nslab; ++s) {
    const int buf = s & 1;
    if (s + 1 < nslab) fetch(s + 1, raw);
    int steps_run = BK;  // mac_step calls of this slab
    if (ORD == ORD_CHUNK_ANY) {
      const int kmax = (int)((K - (int64_t)s * BK) < BK ? (K - (int64_t)s * BK) : BK);
      steps_run = kmax;
#pragma unroll 1
      for (int kk = 0; kk < kmax; ++kk) {
        mac_step(buf, kk);
        if (++k_in_chunk == p.chunk) {
          close_chunk();
          k_in_chunk = 0;
        }
      }
    } else {
#pragma unroll
      for (int kk = 0; kk < BK; ++kk) mac_step(buf, kk);
      if (ORD == ORD_CHUNK_SLAB) {
        if (++slabs_in_chunk == p.chunk_slabs) {
          close_chunk();
          slabs_in_chunk = 0;
        }
      }
    }
    if constexpr (MASKS) {  // the slab's 16 bits join their word; a word is complete after every second slab
      const int valid = (int)((K - kbase) < BK ? (K - kbase) : BK);
      const uint32_t keep = valid >= 16 ? 0xFFFFu : ((1u << valid) - 1u);
      const int sh = (s & 1) * 16;
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) {
          // STE^DIFF shifted its bits in from below: step 0 of the slab's `steps_run` steps sits highest
          if (DIFF) half1[i][j] = steps_run > 0 ? (__brev(half1[i][j]) >> (32 - steps_run)) : 0u;
          bits1[i][j] |= (half1[i][j] & keep) << sh;
          half1[i][j] = 0u;
        }
      if ((s & 1) || s + 1 == nslab) flush_words(mask1z, W1, (int64_t)(s >> 1), bits1);
    }
    if (s + 1 < nslab) decode_store(raw, buf ^ 1);
    __syncthreads();
    kbase += BK;
  }
  if (ORD == ORD_CHUNK_SLAB && slabs_in_chunk > 0) close_chunk();
  if (ORD == ORD_CHUNK_ANY && k_in_chunk > 0) close_chunk();

  if constexpr (MASKS) {
    if constexpr (CHUNKED) {
      if ((chunk_id & 31) != 0) flush_words(mask2z, W2, (int64_t)(chunk_id >> 5), bits2);
    }
    return;
  }
  if (LAST) {
    int* const lastz = reinterpret_cast<int*>(p.out) + (int64_t)blockIdx.z * p.batch_out;
#pragma unroll
    for (int i = 0; i < TM; ++i) {
      const int64_t m = m0 + (i / 4) * (BM / 2) + ty * 4 + (i % 4);
      if (m >= p.M) continue;
#pragma unroll
      for (int j = 0; j < TN; ++j) {
        const int64_t n = n0 + (j / 4) * (BN / 2) + tx * 4 + (j % 4);
        if (n < p.N) lastz[m * p.N + n] = last[LAST ? i : 0][LAST ? j : 0];
      }
    }
    return;
  }

  // ---- epilogue: back to real values, +0 for every zero, scales and bias in binary32
  float* const outz = p.out + (int64_t)blockIdx.z * p.batch_out;
  const bool vec_store = (p.N % 4 == 0) && ((reinterpret_cast<uintptr_t>(outz) & 15) == 0);
#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const int64_t m = m0 + (i / 4) * (BM / 2) + ty * 4 + (i % 4);
    if (m >= p.M) continue;
    const float sa = p.sa[p.sa_per_row ? m : 0];
#pragma unroll
    for (int h = 0; h < TN / 4; ++h) {
      const int64_t n = n0 + h * (BN / 2) + tx * 4;
      float o[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float s = CHUNKED ? acc2[CHUNKED ? i : 0][CHUNKED ? h * 4 + j : 0] : acc1[i][h * 4 + j];
        float y = __fmul_rn(__fmul_rn(s, p.un1), p.un2);
        y = (y == 0.0f) ? 0.0f : y;
        o[j] = y;
      }
      if (n + 3 < p.N && vec_store) {
        float4 v;
        float* ov = &v.x;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float sb = p.sb[p.sb_per_col ? n + j : 0];
          float r = __fmul_rn(__fmul_rn(o[j], sa), sb);
          if (p.bias) r = __fadd_rn(r, p.bias[n + j]);
          ov[j] = r;
        }
        *reinterpret_cast<float4*>(outz + m * p.N + n) = v;
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (n + j < p.N) {
            const float sb = p.sb[p.sb_per_col ? n + j : 0];
            float r = __fmul_rn(__fmul_rn(o[j], sa), sb);
            if (p.bias) r = __fadd_rn(r, p.bias[n + j]);
            outz[m * p.N + n + j] = r;
          }
        }
      }
    }
  }
}

// ------------------------------------------------------------------ packed floor kernel
// The fast floor quantiser (Q_prod reduced to its flush, floor rounding) on the packed binary32
// instructions of sm_100: two neighbouring outputs of a row share one 64-bit register pair, so
// the product and the sum of two emulated MACs cost one `mul.ftz.f32x2` and one `fma.rz.ftz.f32x2`,
// followed by one mantissa mask per output.  The magnitude clamp of Eq. 2 is left out of a slab
// whenever it provably cannot act there:
//   |S_i| <= |S_start| + sum_k |x_k w_k| <= |S_start| + ||x||_2 ||w||_2        (floor never grows |.|)
// so if that bound stays below 2^(e_max+1) every masked sum is already <= R_OF.  The loader
// computes the squared 2-norm of every 16-byte row piece while decoding it; the largest A-row and
// B-row norms of the slab give one bound per CTA, and each thread carries an upper bound `u` of
// its own |S| (as a fraction of 2^(e_max+1)), refreshed from the registers when it gets too loose.
// A warp whose bound fails runs the same slab with the clamp.  Results are identical either way.
constexpr int KUNROLL = 16;  // k-steps unrolled in the packed slab body (the whole slab: measured fastest)

// two E4M3 bytes (low 16 bits of `pair`) -> their exact values, by the hardware converter
__device__ __forceinline__ void e4m3x2_to_f32(uint32_t pair, float& v0, float& v1) {
  asm("{\n\t.reg .b16 c, lo, hi;\n\t.reg .b32 h;\n\t"
      "cvt.u16.u32 c, %2;\n\t"
      "cvt.rn.f16x2.e4m3x2 h, c;\n\t"
      "mov.b32 {lo, hi}, h;\n\t"
      "cvt.f32.f16 %0, lo;\n\t"
      "cvt.f32.f16 %1, hi;\n\t}"
      : "=f"(v0), "=f"(v1)
      : "r"(pair));
}

// ---- tensor memory as a second register file.  In chunk-16 order the second-level sums T are touched
// once per 16 k-steps; keeping them in TMEM (each thread owns TM*TN 32-bit columns of its own lane)
// frees TM*TN registers, which doubles the CTAs an SM can hold for the 8-row micro-tiles.  No MMA is
// involved: tcgen05.ld / tcgen05.st move 16 columns of a lane to and from registers.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]) : "r"(taddr));
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" :: "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ u64 pack2u(uint32_t lo, uint32_t hi) {
  u64 d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
  return d;
}

// columns of tensor memory a CTA of the packed kernel allocates (0: second-level sums stay in registers)
template <int BM, int BN, int TM, int TN, bool RNE, int ORD>
__host__ __device__ constexpr int packed_tmem_cols() {
  constexpr int warps = (BM / TM) * (BN / TN) / 32;
  constexpr int cols = ((warps + 3) / 4) * TM * TN;
  return (ORD == ORD_CHUNK16 && TM == 8 && !RNE) ? (cols < 32 ? 32 : cols) : 0;
}

// the 8x8 micro-tile is held to 128 registers (two CTAs of 256 threads per SM) wherever the second-level
// sums are not in registers; so is the byte-wise loader, whose sixteen loads in flight would otherwise
// cost fifty registers and half the resident CTAs
// PQ: what Q_prod has to do beyond the flush (the host proves which cases are reachable): nothing, cut the
// mantissa (M_prod < 7), or cut and saturate (448^2 >= R_OF_prod)
// PQ_FUSED: Q_prod is the identity on every reachable product (no cut, no saturation, and no product can fall under
// R_UF_prod), so FMAq(x, w, S) = Q_acc(x w + S) and the product needs no instruction of its own: one packed FMA forms the
// exact product and the sum; the B operand then carries the accumulator's scaling.
enum PackedProd { PQ_NONE = 0, PQ_MASK = 1, PQ_MASK_SAT = 2, PQ_FUSED = 3 };

// RNE: nearest-even instead of floor (then PQ_MASK means "round the product to M_prod bits").  Nearest-even
// can raise a magnitude by half a grid step per rounding, so the slab-level proof that the clamp is idle carries a
// growth factor for the roundings of a slab and a limit that keeps every sum at or below R_OF.
//
// STE = 1 (floor, sequential or chunk-16 order): instead of the sums the kernel writes the overflow masks of the
// straight-through estimator STE^OF (App. D; layout as in the scalar tracking kernel).  The proof that lets a
// slab run without the clamp is the proof that none of its steps overflows, so such a slab contributes sixteen
// 1-bits per output without looking at them; only clamped slabs and clamped folds record bits step by step.
// Bits that must outlive a slab wait in shared memory (per thread: 16 words for the low half of a mask1
// word, 32 words for the mask2 word in progress), so the common path keeps the forward kernel's registers.
//
// CL = 2 (floor, chunk-16 order): two CTAs of a thread-block cluster share
// one output tile.  The chunk sums C_j of the first hierarchy do not depend on each other; only the folds
// T <- Q_acc(C_j + T), one addition in sixteen, are sequential.  CTA r forms the chunk sums of the chunks j = r, r + 2,
// ... for the whole tile and folds, in chunk order, all chunks for the column half r of every thread's micro-tile;
// the chunk sums of the other half cross to the other CTA through distributed shared memory, double buffered, with
// one cluster barrier per pair of chunks.  H16: the chunk sums travel as bfloat16 pairs, which a value with at most 7
// mantissa bits is exactly (half the traffic, 2 % faster); otherwise as binary32 words.
// This doubles the CTAs of a small problem without splitting any sequential chain, and both CTAs do the same work.
template <int BM, int BN, int TM, int TN, int PQ, bool RNE, int ORD, int LD, int STE = 0, int CL = 1, bool H16 = false>
__global__ void __launch_bounds__((BM / TM) * (BN / TN),
                                  ((TM * TN == 64 && ORD != ORD_CHUNK_SLAB && !RNE) ||
                                   ((LD == LD_ANY || STE != 0) && !RNE && ORD != ORD_CHUNK_SLAB))
                                      ? 512 / ((BM / TM) * (BN / TN)) : 1)
    lba_contract_packed_kernel(const Problem p) {
  static_assert(STE == 0 || (!RNE && TM == 4 && TN == 8 && (ORD == ORD_SEQ || ORD == ORD_CHUNK16)), "mask variant");
  static_assert(CL == 1 || (CL == 2 && !RNE && STE == 0 && ORD == ORD_CHUNK16 && TM == 4), "cluster variant");
  constexpr int NT = (BM / TM) * (BN / TN);
  constexpr int TX = BN / TN;
  constexpr int ROWS = BM + BN;
  constexpr int LPT = (ROWS + NT - 1) / NT;
  constexpr int PN = TN / 2;  // register pairs per micro-tile row
  constexpr bool CH16 = ORD == ORD_CHUNK16;  // every slab is exactly one chunk
  constexpr bool CHUNKED = ORD == ORD_CHUNK_SLAB || CH16;
  constexpr int TMEM_COLS = packed_tmem_cols<BM, BN, TM, TN, RNE, ORD>();
  constexpr bool T_IN_TMEM = TMEM_COLS > 0;   // second-level sums in tensor memory
  constexpr bool T_IN_REGS = CHUNKED && !T_IN_TMEM;
  static_assert(!T_IN_TMEM || (TM * TN) % 16 == 0, "tensor-memory groups of 16 columns");
  static_assert(ORD == ORD_SEQ || ORD == ORD_CHUNK_SLAB || ORD == ORD_CHUNK16, "order");
  static_assert(TM == 4 || TM == 8, "micro-tile rows");
  static_assert(TN == 4 || TN == 8, "micro-tile cols");
  static_assert(BM % 32 == 0 && BN % 32 == 0, "a warp loads rows of one operand only");

  // A is stored twice, {a, a}, so that a 64-bit shared load yields the packed multiplier directly
  extern __shared__ __align__(16) unsigned char smem_raw[];
  typedef float2 (*AsT)[BK][BM];
  typedef float (*BsT)[BK][BN];
  AsT As = reinterpret_cast<AsT>(smem_raw);
  BsT Bs = reinterpret_cast<BsT>(smem_raw + sizeof(float2) * 2 * BK * BM);
  // largest normalised squared row norm of the slab, as binary32 bits (non-negative, so they order
  // like integers): [slab % 3][0 = A, 1 = B]; three cells so that one can be cleared while the
  // neighbours are read and filled
  unsigned (*nrm)[2] = reinterpret_cast<unsigned (*)[2]>(smem_raw + sizeof(float2) * 2 * BK * BM + sizeof(float) * 2 * BK * BN);
  unsigned* tmem_slot = reinterpret_cast<unsigned*>(nrm) + 6;  // base address written by tcgen05.alloc
  // STE: [q][tid] words, q = i * PN + j: bits of the pair's low output in the low half, of its high output above
  uint32_t* const stash1 = reinterpret_cast<uint32_t*>(nrm) + 8;
  uint32_t* const stash2 = stash1 + (STE ? TM * PN * NT : 0);   // [o][tid], o = i * TN + 2 * j + half

  const int tid = threadIdx.x;
  const int tx = tid % TX, ty = tid / TX;
  unsigned crank = 0;  // rank of this CTA in its cluster (CL = 2: 0 folds, 1 hands its chunk sums over)
  if (CL > 1) asm("mov.u32 %0, %%cluster_ctarank;" : "=r"(crank));
  const int64_t m0 = (int64_t)(blockIdx.x / CL) * BM;
  const int64_t n0 = (int64_t)blockIdx.y * BN;
  const int nslab = (int)((p.K + BK - 1) / BK);
  // CL = 2: chunk sums in flight between the two CTAs, [buffer][group of 2 pairs][thread] as uint4
  uint4* const hand = reinterpret_cast<uint4*>(reinterpret_cast<uint32_t*>(nrm) + 8);

  RowLoader<BM, BN, NT, LD> loader;
  loader.init(p, tid, m0, n0);

  auto decode_store = [&](const uint4 (&raw)[LPT], int buf, int cell) {
#pragma unroll
    for (int l = 0; l < LPT; ++l) {
      const int r = tid + l * NT;
      if (r < ROWS) {  // uniform per warp: BM, BN and NT are multiples of 32
        const bool is_a = r < BM;
        const float mul = is_a ? p.pk_a : p.pk_b;
        const uint32_t w4[4] = {raw[l].x, raw[l].y, raw[l].z, raw[l].w};
        float n2 = 0.0f;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          float v[4];
          if (p.in_m4e3) {
#pragma unroll
            for (int j = 0; j < 4; ++j) v[j] = decode_m4e3_top(byte_to_top(w4[q], j));
          } else {
            e4m3x2_to_f32(w4[q], v[0], v[1]);
            e4m3x2_to_f32(w4[q] >> 16, v[2], v[3]);
          }
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            n2 = fma_rn(v[j], v[j], n2);
            const float s = mul_ieee(v[j], mul);
            if (is_a) As[buf][q * 4 + j][r] = make_float2(s, s);
            else Bs[buf][q * 4 + j][r - BM] = s;
          }
        }
        {
          const unsigned m = __reduce_max_sync(0xFFFFFFFFu, __float_as_uint(n2 * p.nrm_scale));
          if ((tid & 31) == 0) atomicMax(&nrm[cell][is_a ? 0 : 1], m);
        }
      }
    }
  };

  u64 acc1[TM][PN];
  u64 acc2[T_IN_REGS ? TM : 1][T_IN_REGS ? PN : 1];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < PN; ++j) acc1[i][j] = 0ull;
  if (T_IN_REGS) {
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
      for (int j = 0; j < PN; ++j) acc2[T_IN_REGS ? i : 0][T_IN_REGS ? j : 0] = 0ull;
  }

  const u64 cc2 = pack2(p.c, p.c);
  const uint32_t mask = p.qa.mask;
  const float sat = p.qa.sat;
  const uint32_t pmask = p.qp.mask;
  const float psat = p.qp.sat;
  const u64 ks_acc = pack2(p.rne_k_acc, p.rne_k_acc), nks_acc = pack2(-p.rne_k_acc, -p.rne_k_acc);
  const u64 ks_prod = pack2(p.rne_k_prod, p.rne_k_prod), nks_prod = pack2(-p.rne_k_prod, -p.rne_k_prod);

  // one slab of 16 k-steps; CLAMP selects whether the magnitude clamp of Eq. 2 is applied.  The clamped
  // variant is the rare one and stays a rolled loop.  In chunk-16 order the slab starts a chunk: its first
  // step adds to zero, which is a plain (exact) scaling of the product, so the sums need no clearing.
  uint32_t hb[STE ? TM : 1][STE ? PN : 1];  // STE: the slab's bits of a clamped slab (pair layout as stash1)
  auto slab_body = [&](int buf, auto clamp_tag) {
    constexpr bool CLAMP = decltype(clamp_tag)::value;
    constexpr bool REC = CLAMP && STE != 0;
    constexpr int UNR = CLAMP ? 1 : (RNE ? 4 : KUNROLL);  // nearest-even: a four-step body keeps the loop in the instruction cache
    if constexpr (REC) {
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < PN; ++j) hb[i][j] = 0u;
    }
#pragma unroll UNR
    for (int kk = 0; kk < BK; ++kk) {
      u64 a2[TM], b2[PN];
#pragma unroll
      for (int h = 0; h < TM / 4; ++h) {
        const ulonglong2* src = reinterpret_cast<const ulonglong2*>(&As[buf][kk][h * (BM / 2) + ty * 4]);
        const ulonglong2 v0 = src[0], v1 = src[1];
        a2[h * 4 + 0] = v0.x; a2[h * 4 + 1] = v0.y; a2[h * 4 + 2] = v1.x; a2[h * 4 + 3] = v1.y;
      }
#pragma unroll
      for (int h = 0; h < TN / 4; ++h) {
        const ulonglong2 v = *reinterpret_cast<const ulonglong2*>(&Bs[buf][kk][h * (BN / 2) + tx * 4]);
        b2[h * 2 + 0] = v.x; b2[h * 2 + 1] = v.y;
      }
      if constexpr (!RNE) {
        // floor: the products of micro-tile row i + 1 are formed while row i is added and masked, so that
        // multiplies (FP32 pipe) and masks (logic pipe) of independent outputs sit side by side in the stream
        auto product = [&](u64 av, u64 bv) -> u64 {
          u64 pr = mul2_ftz(bv, av);
          if (PQ == PQ_MASK || PQ == PQ_MASK_SAT) {  // floor of Eq. 2 on the exact product, then its saturation
            float plo, phi;
            unpack2(pr, plo, phi);
            plo = and_bits(plo, pmask);
            phi = and_bits(phi, pmask);
            if (PQ == PQ_MASK_SAT) {
              plo = clamp_mag(plo, psat);
              phi = clamp_mag(phi, psat);
            }
            pr = pack2(plo, phi);
          }
          return pr;
        };
        if constexpr (PQ == PQ_FUSED) {
#pragma unroll
          for (int i = 0; i < TM; ++i)
#pragma unroll
            for (int j = 0; j < PN; ++j) {
              const u64 t = (CH16 && kk == 0) ? mul2_rz_ftz(b2[j], a2[i]) : fma2_rz_ftz(b2[j], a2[i], acc1[i][j]);
              float lo, hi;
              unpack2(t, lo, hi);
              lo = and_bits(lo, mask);
              hi = and_bits(hi, mask);
              if constexpr (REC) {
                if (fabsf(lo) < sat) hb[i][j] |= 1u << kk;
                if (fabsf(hi) < sat) hb[i][j] |= 0x10000u << kk;
              }
              if (CLAMP) {
                lo = clamp_mag(lo, sat);
                hi = clamp_mag(hi, sat);
              }
              acc1[i][j] = pack2(lo, hi);
            }
          continue;
        }
        u64 pr[PN], nx[PN];
#pragma unroll
        for (int j = 0; j < PN; ++j) pr[j] = product(a2[0], b2[j]);
#pragma unroll
        for (int i = 0; i < TM; ++i) {
          if (i + 1 < TM) {
#pragma unroll
            for (int j = 0; j < PN; ++j) nx[j] = product(a2[i + 1], b2[j]);
          }
#pragma unroll
          for (int j = 0; j < PN; ++j) {
            const u64 t = (CH16 && kk == 0) ? mul2_rz_ftz(cc2, pr[j]) : fma2_rz_ftz(cc2, pr[j], acc1[i][j]);
            float lo, hi;
            unpack2(t, lo, hi);
            lo = and_bits(lo, mask);
            hi = and_bits(hi, mask);
            if constexpr (REC) {  // 1 where the exact sum stayed below R_OF (its cut image decides: R_OF is on the grid)
              if (fabsf(lo) < sat) hb[i][j] |= 1u << kk;
              if (fabsf(hi) < sat) hb[i][j] |= 0x10000u << kk;
            }
            if (CLAMP) {
              lo = clamp_mag(lo, sat);
              hi = clamp_mag(hi, sat);
            }
            acc1[i][j] = pack2(lo, hi);
          }
          if (i + 1 < TM) {
#pragma unroll
            for (int j = 0; j < PN; ++j) pr[j] = nx[j];
          }
        }
        continue;
      }
      if constexpr (RNE) {
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < PN; ++j) {
          // nearest-even (the floor path has left the loop body above).  The sum is formed by one packed FMA rounded to
          // nearest: whenever that rounding is inexact the smaller operand lies so far below the larger one (which is
          // on the accumulator's grid) that neither the exact sum nor its binary32 image can reach a tie of the M-bit
          // grid, so rounding the image equals rounding the exact sum (the host admits only formats for which this holds).
          // `.ftz` flushes exactly the sums below R_UF_acc: such a sum is a short dyadic number and survives as a subnormal.
          u64 v;
          if constexpr (PQ == PQ_FUSED) {  // Q_prod is the identity: product and sum in one FMA
            v = (CH16 && kk == 0) ? mul2_rn_ftz(b2[j], a2[i]) : fma2_rn_ftz(b2[j], a2[i], acc1[i][j]);
          } else {
            u64 pr = mul2_ftz(b2[j], a2[i]);
            if (PQ == PQ_MASK || PQ == PQ_MASK_SAT) {  // nearest-even on the exact product, then its saturation
              pr = rne2_fp(pr, ks_prod, nks_prod);
              if (PQ == PQ_MASK_SAT) {
                float plo, phi;
                unpack2(pr, plo, phi);
                pr = pack2(clamp_mag(plo, psat), clamp_mag(phi, psat));
              }
            }
            v = (CH16 && kk == 0) ? mul2_rn_ftz(cc2, pr) : fma2_rn_ftz(cc2, pr, acc1[i][j]);
          }
          float lo, hi;
          const u64 q = rne2_fp(v, ks_acc, nks_acc);
          if (CLAMP) {
            unpack2(q, lo, hi);
            acc1[i][j] = pack2(clamp_mag(lo, sat), clamp_mag(hi, sat));
          } else {
            acc1[i][j] = q;
          }
        }
      }
    }
  };

  // second hierarchy: T <- Q_acc(C + T), C <- 0.  With CLAMP the largest |T| is returned as well.
  uint32_t cb = 0xFFFFFFFFu;  // STE: bit o = 1 where the fold just done stayed below R_OF, o = i * TN + 2 * j + half
  auto close_chunk = [&](auto clamp_tag) -> float {
    constexpr bool CLAMP = decltype(clamp_tag)::value;
    float mx = 0.0f;
    if constexpr (STE != 0) cb = CLAMP ? 0u : 0xFFFFFFFFu;
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
      for (int j = 0; j < PN; ++j) {
        u64& t2 = acc2[T_IN_REGS ? i : 0][T_IN_REGS ? j : 0];
        float lo, hi;
        if (RNE) {  // both operands lie on the accumulator's grid: see the note at the first hierarchy
          unpack2(rne2_fp(add2_rn_ftz(acc1[i][j], t2), ks_acc, nks_acc), lo, hi);
        } else {
          unpack2(add2_rz_ftz(acc1[i][j], t2), lo, hi);
          lo = and_bits(lo, mask);
          hi = and_bits(hi, mask);
        }
        if constexpr (CLAMP && STE != 0) {
          if (fabsf(lo) < sat) cb |= 1u << (i * TN + 2 * j);
          if (fabsf(hi) < sat) cb |= 2u << (i * TN + 2 * j);
        }
        if (CLAMP) {
          lo = clamp_mag(lo, sat);
          hi = clamp_mag(hi, sat);
          mx = fmaxf(mx, fmaxf(fabsf(lo), fabsf(hi)));
        }
        t2 = pack2(lo, hi);
        if (!CH16) acc1[i][j] = 0ull;
      }
    return mx;
  };

  // the same with T in tensor memory: 16 columns (16 / TN micro-tile rows) at a time, the next group's
  // load in flight while the current one is processed.  FINAL leaves the new T in acc1 for the epilogue
  // instead of storing it back.
  uint32_t taddr = 0;
  auto close_chunk_tmem = [&](auto clamp_tag, auto final_tag) -> float {
    constexpr bool CLAMP = decltype(clamp_tag)::value;
    constexpr bool FINAL = decltype(final_tag)::value;
    constexpr int GROUPS = TM * TN / 16;
    constexpr int ROWS_PER_GROUP = 16 / TN;
    float mx = 0.0f;
    uint32_t cur[16], nxt[16];
    tmem_ld16(taddr, cur);
#pragma unroll
    for (int g = 0; g < GROUPS; ++g) {
      tmem_wait_ld();
      if (g + 1 < GROUPS) tmem_ld16(taddr + 16 * (g + 1), nxt);
#pragma unroll
      for (int r = 0; r < ROWS_PER_GROUP; ++r)
#pragma unroll
        for (int j = 0; j < PN; ++j) {
          const int i = g * ROWS_PER_GROUP + r;
          const int c = r * TN + 2 * j;
          float lo, hi;
          unpack2(add2_rz_ftz(acc1[i][j], pack2u(cur[c], cur[c + 1])), lo, hi);
          lo = and_bits(lo, mask);
          hi = and_bits(hi, mask);
          if (CLAMP) {
            lo = clamp_mag(lo, sat);
            hi = clamp_mag(hi, sat);
            mx = fmaxf(mx, fmaxf(fabsf(lo), fabsf(hi)));
          }
          if (FINAL) {
            acc1[i][j] = pack2(lo, hi);
          } else {
            cur[c] = __float_as_uint(lo);
            cur[c + 1] = __float_as_uint(hi);
          }
        }
      if (!FINAL) tmem_st16(taddr + 16 * g, cur);
      if (g + 1 < GROUPS) {
#pragma unroll
        for (int c = 0; c < 16; ++c) cur[c] = nxt[c];
      }
    }
    if (!FINAL) tmem_wait_st();  // the next close reads these columns again
    return mx;
  };

  if (tid < 6) nrm[tid >> 1][tid & 1] = 0u;
  if (T_IN_TMEM) {
    // one warp allocates for the CTA; tcgen05.alloc returns once the SM has the columns free (CTAs
    // that hold columns never wait for anything before they release them at the end of the kernel)
    if (tid < 32) {
      const uint32_t slot = (uint32_t)__cvta_generic_to_shared(tmem_slot);
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(TMEM_COLS) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  }
  __syncthreads();
  if (T_IN_TMEM) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const int warp = tid >> 5;
    // lanes: a warp may touch only the quadrant (warp % 4); warps of the same quadrant take different columns
    taddr = *tmem_slot + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * TM * TN);
    uint32_t zero[16];
#pragma unroll
    for (int c = 0; c < 16; ++c) zero[c] = 0u;
#pragma unroll
    for (int g = 0; g < TM * TN / 16; ++g) tmem_st16(taddr + 16 * g, zero);
    tmem_wait_st();
  }
  uint4 raw[LPT];
  const int s_first = CL > 1 ? (int)crank : 0;  // first slab of this CTA
  if (CL > 1 && crank != 0) loader.skip_slab(p);
  if (s_first < nslab) {
    loader.fetch(p, tid, s_first, raw);
    decode_store(raw, 0, 0);
  }
  __syncthreads();

  // ---- STE bookkeeping (see the kernel's header comment)
  bool low_fast = true;    // the even slab of the mask1 word in progress ran without the clamp
  bool s2_active = false;  // the mask2 word in progress lives in stash2 (one of its folds was clamped)
  const int64_t W1 = (p.K + 31) / 32;
  const int64_t W2 = p.mask2_words;
  // one 32-bit word for every output of the thread; word_of(i, c): micro-tile row i, column c = 2 * pair + half
  auto emit_words = [&](uint32_t* base, int64_t words, int64_t w, auto word_of) {
    const bool vec = (p.N % 4 == 0) && ((reinterpret_cast<uintptr_t>(base) & 15) == 0);
#pragma unroll
    for (int i = 0; i < TM; ++i) {
      const int64_t m = m0 + (i / 4) * (BM / 2) + ty * 4 + (i % 4);
      if (m >= p.M) continue;
#pragma unroll
      for (int h = 0; h < TN / 4; ++h) {
        const int64_t n = n0 + h * (BN / 2) + tx * 4;
        uint32_t* const dst = base + (m * words + w) * p.N + n;
        uint32_t v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) v[q] = word_of(i, h * 4 + q);
        if (vec && n + 3 < p.N) {
          *reinterpret_cast<uint4*>(dst) = make_uint4(v[0], v[1], v[2], v[3]);
        } else {
#pragma unroll
          for (int q = 0; q < 4; ++q)
            if (n + q < p.N) dst[q] = v[q];
        }
      }
    }
  };
  // the same word for every output of the thread (the common case: nothing overflowed); a rolled loop, to keep
  // the hot path short
  auto emit_const = [&](uint32_t* base, int64_t words, int64_t w, uint32_t value) {
    const bool vec = (p.N % 4 == 0) && ((reinterpret_cast<uintptr_t>(base) & 15) == 0);
    const uint4 v4 = make_uint4(value, value, value, value);
    uint32_t* row = base + ((m0 + ty * 4) * words + w) * p.N + n0 + tx * 4;
    const int64_t pitch = words * p.N;
#pragma unroll 1
    for (int i = 0; i < TM; ++i, row += pitch) {
      if (m0 + ty * 4 + i >= p.M) break;
#pragma unroll
      for (int h = 0; h < TN / 4; ++h) {
        const int64_t n = n0 + h * (BN / 2) + tx * 4;
        uint32_t* const dst = row + h * (BN / 2);
        if (vec && n + 3 < p.N) {
          *reinterpret_cast<uint4*>(dst) = v4;
        } else {
#pragma unroll
          for (int q = 0; q < 4; ++q)
            if (n + q < p.N) dst[q] = value;
        }
      }
    }
  };
  // after slab s: its sixteen bits per output (all ones below `keep` if it ran without the clamp, else hb)
  // complete or start a word of mask1
  auto ste_after_slab = [&](int s, bool cur_fast) {
    const int64_t left = p.K - (int64_t)s * BK;
    const uint32_t keep = left >= BK ? 0xFFFFu : ((1u << (int)left) - 1u);
    if ((s & 1) == 0) {
      if (s + 1 == nslab) {  // the last word has a low half only
        if (cur_fast) emit_const(p.mask1, W1, s >> 1, keep);
        else emit_words(p.mask1, W1, s >> 1, [&](int i, int c) { return (hb[i][c >> 1] >> (16 * (c & 1))) & keep; });
      } else {
        low_fast = cur_fast;
        if (!cur_fast) {
#pragma unroll
          for (int i = 0; i < TM; ++i)
#pragma unroll
            for (int j = 0; j < PN; ++j) stash1[(i * PN + j) * NT + tid] = hb[i][j];
        }
      }
    } else {
      const bool lf = low_fast;
      auto low_of = [&](int i, int c) -> uint32_t {
        return lf ? 0xFFFFu : ((stash1[(i * PN + (c >> 1)) * NT + tid] >> (16 * (c & 1))) & 0xFFFFu);
      };
      if (cur_fast && lf) emit_const(p.mask1, W1, s >> 1, 0xFFFFu | (keep << 16));
      else if (cur_fast) emit_words(p.mask1, W1, s >> 1, [&](int i, int c) { return low_of(i, c) | (keep << 16); });
      else emit_words(p.mask1, W1, s >> 1, [&](int i, int c) {
        return low_of(i, c) | (((hb[i][c >> 1] >> (16 * (c & 1))) & keep) << 16);
      });
    }
  };
  // after the fold of chunk s (chunk-16 order): cb holds its bit for every output of the thread
  auto ste_after_fold = [&](int s) {
    const int pos = s & 31;
    if (!s2_active && cb != 0xFFFFFFFFu) {  // first clamped fold of this word: the earlier folds all passed
      s2_active = true;
      const uint32_t prev = (1u << pos) - 1u;
#pragma unroll
      for (int o = 0; o < TM * TN; ++o) stash2[o * NT + tid] = prev;
    }
    if (s2_active) {
#pragma unroll
      for (int o = 0; o < TM * TN; ++o)
        if ((cb >> o) & 1u) stash2[o * NT + tid] |= 1u << pos;
    }
    if (pos == 31 || s + 1 == nslab) {
      const uint32_t ones = pos == 31 ? 0xFFFFFFFFu : ((2u << pos) - 1u);
      if (s2_active) emit_words(p.mask2, W2, s >> 5, [&](int i, int c) { return stash2[(i * TN + c) * NT + tid]; });
      else emit_const(p.mask2, W2, s >> 5, ones);
      s2_active = false;
    }
  };

  // a slab (or fold) whose sums provably stay below `lim` * 2^(e_max + 1) runs without the clamp: below 2^(e_max + 1)
  // the mantissa mask alone respects R_OF.  The mask variant needs more, namely that no sum reaches R_OF itself
  // (a sum in [R_OF, 2^(e_max + 1)) needs no clamp but is an overflow), so its limit is R_OF / 2^(e_max + 1)
  const float lim = STE != 0 ? p.ste_limit : p.clamp_lim;
  const float gs = p.slab_factor, gf = p.fold_factor;
  float u = 0.0f;   // upper bound of max |acc1| of this thread, as a fraction of 2^(e_max + 1)
  float u2 = 0.0f;  // chunk-16 order: the same for the second-level sums
  int slabs_in_chunk = 0;
  int cell = 0;     // s % 3
  if constexpr (CL > 1) {
    // ---- two CTAs per output tile (see the kernel's header comment).  Both run the same number of rounds and
    // meet at one cluster barrier per round; nothing leaves the loop early.  CTA r forms the chunk sums of the
    // chunks 2q + r for the whole tile, but keeps and folds the second-level sums T only for the column half r of
    // every thread's micro-tile; the chunk sums of the other half go to the other CTA.  The work is the same on
    // both sides: one slab and two folds of half a micro-tile per round.
    static_assert(PN == 4, "column halves of the 4x8 micro-tile");
    constexpr int HP = PN / 2;  // pairs per row in a column half
    const int rounds = (nslab + CL - 1) / CL;
    uint32_t hand_remote;  // the other CTA's hand buffer as seen from this CTA
    asm("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(hand_remote) : "r"((uint32_t)__cvta_generic_to_shared(hand)), "r"(crank ^ 1u));
    u64 T[TM][HP];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
      for (int j = 0; j < HP; ++j) T[i][j] = 0ull;

    // T <- Q_acc(C + T) for this CTA's column half H; C from the own chunk sums (acc1) or from the words received
    auto fold = [&](auto half_tag, auto clamp_tag, const uint32_t* recv) -> float {
      constexpr int H = decltype(half_tag)::value;
      constexpr bool CLAMP = decltype(clamp_tag)::value;
      float mx = 0.0f;
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < HP; ++j) {
          u64 c = acc1[i][H * HP + j];
          if (recv) {
            c = H16 ? pack2u(recv[i * HP + j] << 16, recv[i * HP + j] & 0xFFFF0000u)
                    : pack2u(recv[2 * (i * HP + j)], recv[2 * (i * HP + j) + 1]);
          }
          float lo, hi;
          unpack2(add2_rz_ftz(c, T[i][j]), lo, hi);
          lo = and_bits(lo, mask);
          hi = and_bits(hi, mask);
          if (CLAMP) {
            lo = clamp_mag(lo, sat);
            hi = clamp_mag(hi, sat);
            mx = fmaxf(mx, fmaxf(fabsf(lo), fabsf(hi)));
          }
          T[i][j] = pack2(lo, hi);
        }
      return mx;
    };
    // the own chunk may skip the clamp under the running bound; a received chunk is always clamped and
    // refreshes the bound
    auto fold_own = [&](auto half_tag, float grow) {
      if (__all_sync(0xFFFFFFFFu, u2 + grow < lim)) {
        fold(half_tag, std::false_type(), nullptr);
        u2 += grow;
      } else {
        u2 = fold(half_tag, std::true_type(), nullptr) * p.inv_top;
      }
    };
    auto fold_received = [&](auto half_tag, int q) {
      constexpr int NG = H16 ? TM * HP / 4 : TM * HP / 2;  // 16-byte groups per thread and chunk
      uint32_t w[4 * NG];
#pragma unroll
      for (int g = 0; g < NG; ++g) {
        const uint4 v = hand[((q & 1) * NG + g) * NT + tid];
        w[g * 4 + 0] = v.x; w[g * 4 + 1] = v.y; w[g * 4 + 2] = v.z; w[g * 4 + 3] = v.w;
      }
      u2 = fold(half_tag, std::true_type(), w) * p.inv_top;
    };
    // chunk sums of the column half `other` into the other CTA's buffer, 16 bytes per store
    auto send = [&](auto other_tag, int q) {
      constexpr int O = decltype(other_tag)::value;
      if constexpr (H16) {
#pragma unroll
        for (int g = 0; g < TM * HP / 4; ++g) {
          uint32_t w[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int idx = g * 4 + e;
            float lo, hi;
            unpack2(acc1[idx / HP][O * HP + idx % HP], lo, hi);
            w[e] = (__float_as_uint(lo) >> 16) | (__float_as_uint(hi) & 0xFFFF0000u);
          }
          const uint32_t dst = hand_remote + (uint32_t)(((q & 1) * (TM * HP / 4) + g) * NT + tid) * 16u;
          asm volatile("st.shared::cluster.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]),
                       "r"(w[3]) : "memory");
        }
      } else {
#pragma unroll
        for (int g = 0; g < TM * HP / 2; ++g) {
          const u64 c0 = acc1[(2 * g) / HP][O * HP + (2 * g) % HP], c1 = acc1[(2 * g + 1) / HP][O * HP + (2 * g + 1) % HP];
          const uint32_t dst = hand_remote + (uint32_t)(((q & 1) * (TM * HP / 2) + g) * NT + tid) * 16u;
          asm volatile("st.shared::cluster.v2.u64 [%0], {%1, %2};" ::"r"(dst), "l"(c0), "l"(c1) : "memory");
        }
      }
    };

    for (int q = 0; q < rounds; ++q) {
      const int s = q * CL + (int)crank;
      const bool have = s < nslab;          // only CTA 1 can run out, in the last round of an odd slab count
      const bool more = s + CL < nslab;
      const int buf = q & 1;
      const int cell_next = cell == 2 ? 0 : cell + 1;
      const int cell_clear = cell_next == 2 ? 0 : cell_next + 1;
      if (more) {
        loader.skip_slab(p);
        loader.fetch(p, tid, s + CL, raw);
      }
      float grow = 0.0f;
      if (have) {
        const float na = __uint_as_float(nrm[cell][0]), nb = __uint_as_float(nrm[cell][1]);
        if (tid < 2) nrm[cell_clear][tid] = 0u;
        grow = sqrtf(na * nb) * 1.01f;
        if (grow < lim) slab_body(buf, std::false_type());
        else slab_body(buf, std::true_type());
        if (crank == 0) send(std::integral_constant<int, 1>(), q);
        else send(std::integral_constant<int, 0>(), q);
      }
      asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
      asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
      // chunk 2q (formed by CTA 0) is folded before chunk 2q + 1 (formed by CTA 1), on both sides
      if (crank == 0) {
        fold_own(std::integral_constant<int, 0>(), grow);
        if (s + 1 < nslab) fold_received(std::integral_constant<int, 0>(), q);
      } else {
        fold_received(std::integral_constant<int, 1>(), q);
        if (have) fold_own(std::integral_constant<int, 1>(), grow);
      }
      if (more) decode_store(raw, buf ^ 1, cell_next);
      __syncthreads();
      cell = cell_next;
    }

    // ---- epilogue of the pair: this CTA's column half
    float* const outz = p.out + (int64_t)blockIdx.z * p.batch_out;
    const bool vec_store = (p.N % 4 == 0) && ((reinterpret_cast<uintptr_t>(outz) & 15) == 0);
    const int64_t n = n0 + (int64_t)crank * (BN / 2) + tx * 4;
#pragma unroll
    for (int i = 0; i < TM; ++i) {
      const int64_t m = m0 + ty * 4 + i;
      if (m >= p.M) continue;
      const float sa = p.sa[p.sa_per_row ? m : 0];
      float o[4];
#pragma unroll
      for (int jp = 0; jp < HP; ++jp) unpack2(T[i][jp], o[jp * 2], o[jp * 2 + 1]);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float y = __fmul_rn(__fmul_rn(o[j], p.un1), p.un2);
        o[j] = (y == 0.0f) ? 0.0f : y;
        if (n + j < p.N) {
          const float sb = p.sb[p.sb_per_col ? n + j : 0];
          float r = __fmul_rn(__fmul_rn(o[j], sa), sb);
          if (p.bias) r = __fadd_rn(r, p.bias[n + j]);
          o[j] = r;
        }
      }
      if (n + 3 < p.N && vec_store) {
        *reinterpret_cast<float4*>(outz + m * p.N + n) = make_float4(o[0], o[1], o[2], o[3]);
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (n + j < p.N) outz[m * p.N + n + j] = o[j];
      }
    }
    return;
  } else
  for (int s = 0; s < nslab; ++s) {
    const int buf = s & 1;
    const int cell_next = cell == 2 ? 0 : cell + 1;
    const int cell_clear = cell_next == 2 ? 0 : cell_next + 1;
    if (s + 1 < nslab) loader.fetch(p, tid, s + 1, raw);
    const float na = __uint_as_float(nrm[cell][0]), nb = __uint_as_float(nrm[cell][1]);
    if (tid < 2) nrm[cell_clear][tid] = 0u;  // read during the previous slab, filled during the next
    // ||x|| ||w|| / 2^(e_max+1), rounded up generously (the norms carry rounding errors near 2^-20)
    const float grow = sqrtf(na * nb) * 1.01f;
    if (CH16) {
      // the chunk starts from zero, so the CTA-wide bound alone decides (same value in every thread)
      const float gw = grow * gs;
      if (gw < lim) slab_body(buf, std::false_type());
      else slab_body(buf, std::true_type());
      if constexpr (STE != 0) ste_after_slab(s, gw < lim);
      // |T + C| <= |T| + |C| <= u2 + gw: below the limit the rounding alone already respects R_OF
      const bool last = T_IN_TMEM && s + 1 == nslab;  // the final T goes to registers for the epilogue
      if (__all_sync(0xFFFFFFFFu, u2 + gw < lim)) {
        if (!T_IN_TMEM) close_chunk(std::false_type());
        else if (!last) close_chunk_tmem(std::false_type(), std::false_type());
        else close_chunk_tmem(std::false_type(), std::true_type());
        u2 = (u2 + gw) * gf;
      } else {  // clamped, and the bound is refreshed from the sums
        float mx;
        if (!T_IN_TMEM) mx = close_chunk(std::true_type());
        else if (!last) mx = close_chunk_tmem(std::true_type(), std::false_type());
        else mx = close_chunk_tmem(std::true_type(), std::true_type());
        u2 = mx * p.inv_top;
      }
      if constexpr (STE != 0) ste_after_fold(s);
    } else {
      bool fast = __all_sync(0xFFFFFFFFu, (u + grow) * gs < lim);
      // the carried bound may just be loose: measure |acc1|.  The test must be the same in every lane of the warp (the
      // vote inside is a warp-wide operation): a lane whose outputs are all zero carries u = 0 while its neighbours do not
      if (!fast && __any_sync(0xFFFFFFFFu, u > 0.0f)) {
        float mx = 0.0f;
#pragma unroll
        for (int i = 0; i < TM; ++i)
#pragma unroll
          for (int j = 0; j < PN; ++j) {
            float lo, hi;
            unpack2(acc1[i][j], lo, hi);
            mx = fmaxf(mx, fmaxf(fabsf(lo), fabsf(hi)));
          }
        u = mx * p.inv_top;
        fast = __all_sync(0xFFFFFFFFu, (u + grow) * gs < lim);
      }
      if (fast) slab_body(buf, std::false_type());
      else slab_body(buf, std::true_type());
      if constexpr (STE != 0) ste_after_slab(s, fast);
      u = fminf((u + grow) * gs, 1.0f);
      if (CHUNKED) {
        if (++slabs_in_chunk == p.chunk_slabs) {
          close_chunk(std::true_type());
          slabs_in_chunk = 0;
          u = 0.0f;
        }
      }
    }
    if (s + 1 < nslab) decode_store(raw, buf ^ 1, cell_next);
    __syncthreads();
    cell = cell_next;
  }
  if (CHUNKED && !CH16 && slabs_in_chunk > 0) close_chunk(std::true_type());
  if (T_IN_TMEM) {  // every thread is done with its columns (with K = 0 nothing was ever closed and acc1 is 0)
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (tid < 32) {
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(*tmem_slot), "r"(TMEM_COLS) : "memory");
    }
  }

  if constexpr (STE != 0) return;  // the masks are the output

  // ---- epilogue: back to real values, +0 for every zero, scales and bias in binary32
  float* const outz = p.out + (int64_t)blockIdx.z * p.batch_out;
  const bool vec_store = (p.N % 4 == 0) && ((reinterpret_cast<uintptr_t>(outz) & 15) == 0);
#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const int64_t m = m0 + (i / 4) * (BM / 2) + ty * 4 + (i % 4);
    if (m >= p.M) continue;
    const float sa = p.sa[p.sa_per_row ? m : 0];
#pragma unroll
    for (int h = 0; h < TN / 4; ++h) {
      const int64_t n = n0 + h * (BN / 2) + tx * 4;
      float o[4];
#pragma unroll
      for (int jp = 0; jp < 2; ++jp) {
        const u64 sv = T_IN_REGS ? acc2[T_IN_REGS ? i : 0][T_IN_REGS ? h * 2 + jp : 0] : acc1[i][h * 2 + jp];
        unpack2(sv, o[jp * 2], o[jp * 2 + 1]);
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float y = __fmul_rn(__fmul_rn(o[j], p.un1), p.un2);
        o[j] = (y == 0.0f) ? 0.0f : y;
      }
      if (n + 3 < p.N && vec_store) {
        float4 v;
        float* ov = &v.x;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float sb = p.sb[p.sb_per_col ? n + j : 0];
          float r = __fmul_rn(__fmul_rn(o[j], sa), sb);
          if (p.bias) r = __fadd_rn(r, p.bias[n + j]);
          ov[j] = r;
        }
        *reinterpret_cast<float4*>(outz + m * p.N + n) = v;
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (n + j < p.N) {
            const float sb = p.sb[p.sb_per_col ? n + j : 0];
            float r = __fmul_rn(__fmul_rn(o[j], sa), sb);
            if (p.bias) r = __fadd_rn(r, p.bias[n + j]);
            outz[m * p.N + n + j] = r;
          }
        }
      }
    }
  }
}

template <int BM, int BN>
constexpr size_t packed_smem_bytes() {
  return sizeof(float2) * 2 * BK * BM + sizeof(float) * 2 * BK * BN + sizeof(unsigned) * 8;
}
// the cluster variant adds the double-buffered hand-over of chunk sums (one word per output of a column half and buffer)
template <int BM, int BN, int TM, int TN>
constexpr size_t packed_cluster_smem_bytes() {
  return packed_smem_bytes<BM, BN>() + sizeof(uint32_t) * 2 * (BM / TM) * (BN / TN) * (TM * (TN / 2));
}
// the mask variant adds its two per-thread stashes (16 + 32 words for the 4x8 micro-tile)
template <int BM, int BN, int TM, int TN>
constexpr size_t packed_ste_smem_bytes() {
  return packed_smem_bytes<BM, BN>() + sizeof(uint32_t) * (BM / TM) * (BN / TN) * (TM * (TN / 2) + TM * TN);
}

// Launch entry of one (quantiser mode, order mode) family; defined once per translation unit.
// tile: 0 = 128x128 (8x8 per thread, 256 threads), 1 = 128x64 (4x8, 256 threads), 2 = 64x64 (4x8, 128 threads),
// 3 = 32x32 (4x4, 64 threads).  Micro-tiles are wider than tall because only the A operand is stored twice:
// a 4x8 micro-tile needs 2 + 2 shared loads per k-step, an 8x4 one 4 + 1.  Measured and dropped: 8x8 in CTAs of
// 64 or 128 threads, 4x8 in 32x64, 32x128, 64x128, 128x128, 64x256 tiles, a one-warp 32x32 tile.
struct TileInfo { int bm, bn, tm, tn; };
constexpr int TILE_COUNT = 4;
constexpr int TILE_PAIR = 5;  // 64x64 tile shared by a cluster of two CTAs (chunk-16 order, floor rounding)
__host__ inline TileInfo tile_info(int t) {
  const TileInfo tab[TILE_COUNT] = {{128, 128, 8, 8}, {128, 64, 4, 8}, {64, 64, 4, 8}, {32, 32, 4, 4}};
  return tab[t];
}

typedef cudaError_t (*LaunchFn)(int tile, int load, const Problem& p, cudaStream_t stream);

template <int QM, int ORD>
cudaError_t launch_family(int tile, int load, const Problem& p, cudaStream_t stream);

}  // namespace lba
