// CPU oracle for the LBA (low bit-width accumulator) contraction.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, exact statement of what
// the method computes.  It is used by the tests, by the smoke check and by the
// benchmark's CPU-baseline leg.  The CUDA library never links, includes or calls
// anything here, and nothing here includes anything from the CUDA library.
//
// What is computed (paper sections in brackets):
//   * Q^FLOAT_{M,E,b}: the floating-point quantiser                         [Eq. 2]
//   * rounding of the mantissa: floor on the magnitude (the paper's choice,
//     Sec. 3 "floor ... via bit-mask"), or round-to-nearest-even (a parameter)
//   * FMAq(x, w, s) = Q_acc(Q_prod(x*w) + s)                                 [Eq. 4]
//   * the sequential recursion S_0 = 0, S_{i+1} = FMAq(x_i, w_i, S_i)       [Eq. 8-9]
//   * chunk-based accumulation in two hierarchies, chunk size 16 by default
//     [Sec. 3, Fig. 1 (right), App. D last paragraph]
//   * Y = X W^T with x_i = X_ki, w_i = W_li                                 [App. A]
//   * convolution as the same dot product per output scalar                 [Eq. 3, App. A]
//   * Q^FIXED_{B,b}: the fixed-point quantiser, floor, saturating or wrapping  [Eq. 1]
//   * the straight-through estimators STE^OF and STE^DIFF of every FMAq step, as bit
//     masks, and the last overflowing step of a sequential chain           [Sec. 4, App. D]
//
// Exactness: every intermediate value is a dyadic rational (sign, 128-bit integer
// magnitude, power-of-two exponent).  Products and sums are formed exactly and
// rounded once, by Q, as Eq. 2 and Eq. 4 are written.  No float or double
// arithmetic takes part in the chain; floats appear only in the final scaling
// epilogue, where each operation is a single IEEE binary32 operation.
//
// Readings taken where the paper is silent (each is listed in the design notes):
//   * floor acts on the magnitude (Eq. 2 is written on |x|), i.e. toward zero
//   * the range tests of Eq. 2 use the unrounded |x|; after rounding the magnitude
//     is clamped to R_OF (matters only for nearest-even just below R_OF)
//   * all 2^E exponent codes are ordinary binades [-b, 2^E-b-1]; no subnormals
//   * every zero is +0
//   * Eq. 8-9 end at y = S_N (all N products), not S_{N-1}
//   * second hierarchy of chunking: chunk results are added sequentially, in
//     chunk order, starting from 0, with Q_acc after every addition; Q_prod is
//     not applied there; a short last chunk is allowed
//   * inputs are OCP E4M3 bytes (4 exponent bits, bias 7, 3 mantissa bits,
//     subnormals, max 448, codes 0x7F/0xFF are NaN and are rejected), or, when the product
//     format carries flag bit2, bytes of the paper's own W/A format "M4E3" (Sec. 3.1): sign,
//     3 exponent bits, 4 mantissa bits, value (-1)^s 2^e (1 + m/16) as Eq. 2 gives for
//     (M, E, b) = (4, 3, 0); Eq. 2 has no code for zero, so the code with e = m = 0 is read as
//     zero (the magnitude 2^0 is given up); the per-tensor flex-bias 2^-b of Sec. 3.1 is the
//     power-of-two scale the caller applies to the finished sum
//   * convolution walks k = (kh, kw, c_in) with c_in fastest; padded taps are x = 0
//     and still count toward the chunk position
//   * output scaling: out = fl32(fl32(y*sa)*sb) (+ bias), outside the FMAq unit
//
// Parity status: every function here is pinned by the CPU tests (closed forms of
// Eq. 1 and Eq. 2, hand-derived values and chains, invariants, reduction to IEEE binary32
// summation and to integer arithmetic, hand-worked estimator masks, an independent
// exact-rational coding, brute force).  The paper's accuracy tables
// need datasets and weights and are "parity unpinned".

#include <cstdint>
#include <cstring>
#include <cmath>
#include <vector>
#include <thread>
#include <atomic>
#include <algorithm>

typedef unsigned __int128 u128;

extern "C" {

struct lbo_fmt {
  int32_t man_bits;  // M of Eq. 2
  int32_t exp_bits;  // E of Eq. 2
  int32_t bias;      // b of Eq. 2
  int32_t rounding;  // 0 = floor on magnitude, 1 = nearest, ties to even
  int32_t flags;     // bit0: 1 = underflow flush on (Eq. 2), 0 = "excluding underflow";
                     // bit2 (product format only): the input bytes are M4E3 codes, not OCP E4M3
};
// exp_bits = 0 selects the fixed-point quantiser of Eq. 1 instead: man_bits = B (all bits, sign included),
// bias = b, rounding 0 = floor (toward minus infinity, the plain reading of "Floor" for a two's-complement
// number), flags bit1: 1 = wrap around modulo 2^B (the integer accumulators of the WrapNet comparison, Sec. 2.2)
// instead of saturating at R_min / R_max.

enum {
  LBO_OK = 0,
  LBO_ERR_ARG = -1,       // null pointer, bad size, bad order
  LBO_ERR_FORMAT = -2,    // M/E/rounding outside the supported domain
  LBO_ERR_NAN_CODE = -3,  // an input byte is an E4M3 NaN code
  LBO_ERR_RANGE = -4,     // a value left the exact carrier or the binary32 output range
};

enum { LBO_ORDER_SEQUENTIAL = 0, LBO_ORDER_CHUNKED = 1 };
enum { LBO_STE_NONE = 0, LBO_STE_OF = 1, LBO_STE_DIFF = 2 };  // straight-through estimators of App. D

}  // extern "C"

namespace {

// ---------------------------------------------------------------- exact carrier
struct Dy {       // value = (-1)^neg * mag * 2^ex ; zero is {false, 0, 0}
  bool neg;
  u128 mag;
  int ex;
};

const Dy kZero = {false, 0, 0};

int bit_length(u128 v) {
  uint64_t hi = (uint64_t)(v >> 64), lo = (uint64_t)v;
  if (hi) return 128 - __builtin_clzll(hi);
  if (lo) return 64 - __builtin_clzll(lo);
  return 0;
}

Dy normalised(Dy a) {  // strip trailing zero bits so the magnitude stays short
  if (a.mag == 0) return kZero;
  uint64_t lo = (uint64_t)a.mag;
  int tz = lo ? __builtin_ctzll(lo) : 64 + __builtin_ctzll((uint64_t)(a.mag >> 64));
  a.mag >>= tz;
  a.ex += tz;
  return a;
}

// floor(log2|a|) for a != 0
int floor_log2(const Dy& a) { return bit_length(a.mag) - 1 + a.ex; }

// sign of |a| - |b|
int cmp_mag(const Dy& a, const Dy& b) {
  if (a.mag == 0 || b.mag == 0) return (a.mag != 0) - (b.mag != 0);
  int ea = floor_log2(a), eb = floor_log2(b);
  if (ea != eb) return ea < eb ? -1 : 1;
  // same leading bit position: align the least significant ends; no overflow since
  // both then have the bit length of the longer one (<= 128)
  int lo = std::min(a.ex, b.ex);
  u128 ma = a.mag << (a.ex - lo), mb = b.mag << (b.ex - lo);
  return ma < mb ? -1 : (ma > mb ? 1 : 0);
}

// exact a + b ; false when the aligned operands would not fit the carrier
bool add_exact(const Dy& a, const Dy& b, Dy* out) {
  if (a.mag == 0) { *out = b; return true; }
  if (b.mag == 0) { *out = a; return true; }
  int lo = std::min(a.ex, b.ex);
  int sa = a.ex - lo, sb = b.ex - lo;
  if (bit_length(a.mag) + sa > 126 || bit_length(b.mag) + sb > 126) return false;
  u128 ma = a.mag << sa, mb = b.mag << sb;
  Dy r;
  r.ex = lo;
  if (a.neg == b.neg) {
    r.neg = a.neg;
    r.mag = ma + mb;
  } else if (ma >= mb) {
    r.neg = a.neg;
    r.mag = ma - mb;
  } else {
    r.neg = b.neg;
    r.mag = mb - ma;
  }
  *out = normalised(r);
  return true;
}

Dy mul_exact(const Dy& a, const Dy& b) {  // operands here are at most 5 bits each
  if (a.mag == 0 || b.mag == 0) return kZero;
  Dy r = {a.neg != b.neg, a.mag * b.mag, a.ex + b.ex};
  return normalised(r);
}

bool from_double(double x, Dy* out) {
  if (!std::isfinite(x)) return false;
  if (x == 0.0) { *out = kZero; return true; }
  int e;
  double fr = std::frexp(std::fabs(x), &e);          // |x| = fr * 2^e, fr in [0.5, 1)
  uint64_t m = (uint64_t)std::ldexp(fr, 53);         // exact: 53-bit integer
  Dy r = {x < 0, (u128)m, e - 53};
  *out = normalised(r);
  return true;
}

bool to_double(const Dy& a, double* out) {           // exact or fail
  if (a.mag == 0) { *out = 0.0; return true; }
  if (bit_length(a.mag) > 53) return false;
  int e = floor_log2(a);
  if (e > 1023 || a.ex < -1074) return false;
  double v = std::ldexp((double)(uint64_t)a.mag, a.ex);
  *out = a.neg ? -v : v;
  return true;
}

bool to_float(const Dy& a, float* out) {             // exact, normal binary32, or fail
  if (a.mag == 0) { *out = 0.0f; return true; }
  if (bit_length(a.mag) > 24) return false;
  int e = floor_log2(a);
  if (e > 127 || e < -126) return false;
  float v = std::ldexp((float)(uint32_t)(uint64_t)a.mag, a.ex);
  *out = a.neg ? -v : v;
  return true;
}

// ---------------------------------------------------------------- E4M3 decode
// OCP E4M3: s eeee fff, exponent bias 7; e = 0 holds subnormals f/8 * 2^-6;
// S.1111.111 is NaN; there is no infinity; largest finite value 448.
bool decode_e4m3(uint8_t code, Dy* out) {
  int s = code >> 7, e = (code >> 3) & 0xF, f = code & 0x7;
  if (e == 15 && f == 7) return false;
  Dy r;
  r.neg = s != 0;
  if (e == 0) {
    r.mag = (u128)f;          // f/8 * 2^-6 = f * 2^-9
    r.ex = -9;
  } else {
    r.mag = (u128)(8 + f);    // (1 + f/8) * 2^(e-7) = (8+f) * 2^(e-10)
    r.ex = e - 10;
  }
  *out = normalised(r);
  return true;
}

// The paper's W/A format (Sec. 3.1, "M4E3"): s eee mmmm, Eq. 2 with M = 4, E = 3, b = 0, i.e.
// (-1)^s * 2^e * (1 + m/16) for e in 0..7; all 256 codes are numbers; e = m = 0 is zero.
bool decode_m4e3(uint8_t code, Dy* out) {
  int s = code >> 7, e = (code >> 4) & 0x7, m = code & 0xF;
  if (e == 0 && m == 0) { *out = kZero; return true; }
  Dy r = {s != 0, (u128)(16 + m), e - 4};   // (1 + m/16) * 2^e = (16 + m) * 2^(e-4)
  *out = normalised(r);
  return true;
}

// ---------------------------------------------------------------- Eq. 2
struct Fmt {
  int M, E, b;
  bool nearest;    // else floor on the magnitude
  bool underflow;  // the |x| < R_UF -> 0 branch of Eq. 2 is active
  Dy r_of;         // R_OF = 2^(2^E - b - 1) * (2 - 2^-M)
  bool fixed;      // Eq. 1 instead of Eq. 2: B = M bits in all, bias b
  bool wrap;       // fixed point: modulo 2^B instead of saturation
  bool in_m4e3;    // (read from the product format) the operands are M4E3 bytes
};

int make_fmt(const lbo_fmt* f, Fmt* out) {
  if (!f) return LBO_ERR_ARG;
  out->fixed = false;
  out->wrap = false;
  out->in_m4e3 = (f->flags & 4) != 0;
  if (f->exp_bits == 0) {  // Eq. 1
    if (f->man_bits < 2 || f->man_bits > 32 || f->rounding != 0) return LBO_ERR_FORMAT;
    if (f->bias < -64 || f->bias > 64) return LBO_ERR_FORMAT;
    out->fixed = true;
    out->wrap = (f->flags & 2) != 0;
    out->M = f->man_bits;
    out->E = 0;
    out->b = f->bias;
    out->nearest = false;
    out->underflow = false;
    out->r_of = kZero;
    return LBO_OK;
  }
  if (f->man_bits < 1 || f->man_bits > 52) return LBO_ERR_FORMAT;
  if (f->exp_bits < 1 || f->exp_bits > 10) return LBO_ERR_FORMAT;
  if (f->rounding != 0 && f->rounding != 1) return LBO_ERR_FORMAT;
  if (f->bias < -2000 || f->bias > 2000) return LBO_ERR_FORMAT;
  out->M = f->man_bits;
  out->E = f->exp_bits;
  out->b = f->bias;
  out->nearest = f->rounding == 1;
  out->underflow = (f->flags & 1) != 0;
  int emax = (1 << out->E) - out->b - 1;
  // (2 - 2^-M) * 2^emax = (2^(M+1) - 1) * 2^(emax - M)
  Dy r = {false, (((u128)1) << (out->M + 1)) - 1, emax - out->M};
  out->r_of = r;  // odd magnitude: already normalised
  return LBO_OK;
}

// Q^FIXED_{B,b}(x) of Eq. 1 with Round = floor: 2^-b * floor(x * 2^b), held to [R_min, R_max] =
// [-2^(B-1), 2^(B-1) - 1] * 2^-b by saturation (Eq. 1) or, with `wrap`, by two's-complement wrap-around.
// |x| here is far below 2^100 (sums of bounded terms), so the integer fits the carrier.
Dy quantise_fixed(const Fmt& f, const Dy& x) {
  if (x.mag == 0) return kZero;
  typedef __int128 i128;
  const int sh = x.ex + f.b;  // x * 2^b = mag * 2^sh
  i128 v;
  if (sh >= 0) {
    const int room = 120 - bit_length(x.mag);
    u128 q = sh <= room ? (x.mag << sh) : (((u128)1) << 120);  // beyond every admitted range: saturates below
    if (f.wrap && sh > room) q = sh >= 128 ? 0 : (x.mag << sh);  // modulo 2^B only the low bits matter (B <= 32)
    v = x.neg ? -(i128)q : (i128)q;
  } else {
    const int s = -sh;
    u128 q = s >= 128 ? 0 : (x.mag >> s);
    const bool rem = s >= 128 ? true : ((x.mag & ((((u128)1) << s) - 1)) != 0);
    if (x.neg && rem) q += 1;  // floor of a negative non-integer moves away from zero
    v = x.neg ? -(i128)q : (i128)q;
  }
  const i128 lo = -(((i128)1) << (f.M - 1)), hi = (((i128)1) << (f.M - 1)) - 1, span = ((i128)1) << f.M;
  if (f.wrap) {
    i128 r = (v - lo) % span;
    if (r < 0) r += span;
    v = r + lo;
  } else {
    v = v < lo ? lo : (v > hi ? hi : v);
  }
  if (v == 0) return kZero;
  Dy r = {v < 0, (u128)(v < 0 ? -v : v), -f.b};
  return normalised(r);
}

// Q^FLOAT_{M,E,b}(x), cases in the order Eq. 2 lists them.
Dy quantise(const Fmt& f, const Dy& x) {
  if (f.fixed) return quantise_fixed(f, x);
  if (x.mag == 0) return kZero;
  Dy sat = f.r_of;
  sat.neg = x.neg;
  if (cmp_mag(x, f.r_of) >= 0) return sat;             // |x| >= R_OF
  int e = floor_log2(x);                               // e = floor(log2|x|)
  if (f.underflow && e < -f.b) return kZero;           // |x| < R_UF = 2^-b
  // significand 2^M * (|x| 2^-e) = mag * 2^(ex + M - e), an integer in [2^M, 2^(M+1))
  // once rounded; s low bits of mag lie below the kept grid
  int s = (e - f.M) - x.ex;
  Dy r = x;
  if (s > 0) {
    u128 q = x.mag >> s;
    u128 rem = x.mag & ((((u128)1) << s) - 1);
    if (f.nearest) {
      u128 half = ((u128)1) << (s - 1);
      if (rem > half || (rem == half && (q & 1))) q += 1;
    }
    r.mag = q;
    r.ex = x.ex + s;
    r = normalised(r);
    if (cmp_mag(r, f.r_of) > 0) return sat;            // rounding carried past the top
  }
  return r;
}

// ---------------------------------------------------------------- Eq. 4, Eq. 8-9, chunks
struct Chain {
  const Fmt* prod;
  const Fmt* acc;
  int order;
  int64_t chunk;
  Dy first;        // running sum of the first hierarchy (S of Eq. 8-9, or the chunk sum)
  Dy second;       // running sum over finished chunks
  int64_t in_chunk;
  int status;
  int64_t steps;          // FMAq steps taken so far
  int64_t last_overflow;  // index of the last step with |Q_prod(x w) + S| >= R_OF(acc), or -1 (STE^OF of App. D)
  // straight-through estimators of App. D, evaluated for the step just taken (first hierarchy) and for
  // the chunk just folded (second hierarchy, where the chunk sum stands in for the product)
  int ste_kind;           // LBO_STE_NONE / LBO_STE_OF / LBO_STE_DIFF
  float eps1, eps2;       // DIFF only
  int ste_first, ste_second;
  int64_t chunks_closed;

  Chain(const Fmt* p, const Fmt* a, int ord, int64_t ch)
      : prod(p), acc(a), order(ord), chunk(ch), first(kZero), second(kZero), in_chunk(0), status(LBO_OK), steps(0),
        last_overflow(-1), ste_kind(0), eps1(0.0f), eps2(0.0f), ste_first(0), ste_second(0), chunks_closed(0) {}

  // STE^OF: 1 iff |term + S| < R_OF.   STE^DIFF: 1 iff |z - S| / (|u| + eps1) > eps2, u the unquantised product
  // (the chunk sum at the second hierarchy); the DIFF comparison is taken in binary32, round to nearest:
  // |fl(z - S)| > fl(eps2 * fl(|u| + eps1)).
  int ste(const Dy& exact_sum, const Dy& z, const Dy& s_before, const Dy& u) {
    if (ste_kind == LBO_STE_OF) return !(exact_sum.mag != 0 && cmp_mag(exact_sum, acc->r_of) >= 0);
    if (ste_kind == LBO_STE_DIFF) {
      float zf, sf, uf;
      if (!to_float(z, &zf) || !to_float(s_before, &sf) || !to_float(u, &uf)) { status = LBO_ERR_RANGE; return 0; }
      volatile float d = zf - sf;   // one binary32 subtraction (exact whenever the difference fits 24 bits)
      volatile float den = std::fabs(uf) + eps1;
      volatile float thr = eps2 * den;
      return std::fabs(d) > thr;
    }
    return 0;
  }

  void close_chunk() {
    Dy sum;
    if (!add_exact(first, second, &sum)) { status = LBO_ERR_RANGE; return; }
    Dy t = quantise(*acc, sum);
    if (ste_kind) ste_second = ste(sum, t, second, first);
    second = t;
    first = kZero;
    in_chunk = 0;
    ++chunks_closed;
  }

  // one FMAq step: first <- Q_acc(Q_prod(x*w) + first)
  void fmaq_step(uint8_t xcode, uint8_t wcode) {
    Dy x, w;
    if (prod->in_m4e3) {
      decode_m4e3(xcode, &x);
      decode_m4e3(wcode, &w);
    } else if (!decode_e4m3(xcode, &x) || !decode_e4m3(wcode, &w)) {
      status = LBO_ERR_NAN_CODE;
      return;
    }
    Dy xw = mul_exact(x, w);
    Dy p = quantise(*prod, xw);
    Dy sum;
    if (!add_exact(p, first, &sum)) { status = LBO_ERR_RANGE; return; }
    if (sum.mag != 0 && cmp_mag(sum, acc->r_of) >= 0) last_overflow = steps;
    ++steps;
    Dy z = quantise(*acc, sum);
    if (ste_kind) ste_first = ste(sum, z, first, xw);
    first = z;
  }

  // in chunked order, a full chunk is folded into the second hierarchy
  void end_of_step() {
    if (status == LBO_OK && order == LBO_ORDER_CHUNKED && ++in_chunk == chunk) close_chunk();
  }

  void push(uint8_t xcode, uint8_t wcode) {
    fmaq_step(xcode, wcode);
    end_of_step();
  }

  Dy finish() {
    if (order == LBO_ORDER_SEQUENTIAL) return first;
    if (in_chunk > 0) close_chunk();
    return second;
  }
};

// out = fl32(fl32(y*sa)*sb) (+ bias): three separate binary32 operations
float epilogue(float y, float sa, float sb, const float* bias_n) {
  volatile float t = y * sa;
  volatile float u = t * sb;
  if (bias_n) {
    volatile float v = u + *bias_n;
    return v;
  }
  return u;
}

int check_order(int order, int64_t chunk) {
  if (order != LBO_ORDER_SEQUENTIAL && order != LBO_ORDER_CHUNKED) return LBO_ERR_ARG;
  if (order == LBO_ORDER_CHUNKED && chunk < 1) return LBO_ERR_ARG;
  return LBO_OK;
}

int worker_count(int requested, int64_t items) {
  int n = requested;
  if (n <= 0) n = (int)std::thread::hardware_concurrency();
  if (n < 1) n = 1;
  if ((int64_t)n > items) n = (int)std::max<int64_t>(items, 1);
  return n;
}

template <class F>
int parallel_items(int64_t items, int nthreads, F body) {  // body(i) -> status
  int n = worker_count(nthreads, items);
  std::atomic<int> status(LBO_OK);
  auto run = [&](int t) {
    for (int64_t i = t; i < items; i += n) {
      if (status.load() != LBO_OK) return;
      int st = body(i);
      if (st != LBO_OK) { status.store(st); return; }
    }
  };
  if (n == 1) {
    run(0);
  } else {
    std::vector<std::thread> pool;
    for (int t = 0; t < n; ++t) pool.emplace_back(run, t);
    for (auto& th : pool) th.join();
  }
  return status.load();
}

struct GemmArgs {
  const uint8_t *A, *B;
  const float *sa, *sb, *bias;
  int sa_len, sb_len;
  int64_t M, N, K;
  Fmt prod, acc;
  int order;
  int64_t chunk;
};

int gemm_point(const GemmArgs& g, int64_t m, int64_t n, float* out) {
  Chain c(&g.prod, &g.acc, g.order, g.chunk);
  const uint8_t* x = g.A + m * g.K;   // x_i = X_mi
  const uint8_t* w = g.B + n * g.K;   // w_i = W_ni
  for (int64_t i = 0; i < g.K; ++i) {
    c.push(x[i], w[i]);
    if (c.status != LBO_OK) return c.status;
  }
  Dy y = c.finish();
  if (c.status != LBO_OK) return c.status;
  float yf;
  if (!to_float(y, &yf)) return LBO_ERR_RANGE;
  float sa = g.sa_len == 1 ? g.sa[0] : g.sa[m];
  float sb = g.sb_len == 1 ? g.sb[0] : g.sb[n];
  *out = epilogue(yf, sa, sb, g.bias ? g.bias + n : nullptr);
  return LBO_OK;
}

struct ConvArgs {
  const uint8_t *x, *w;
  const float *sx, *sw, *bias;
  int sx_len, sw_len;
  int64_t B, H, W, Cin, Cout, KH, KW, stride_h, stride_w, pad_h, pad_w, Hout, Wout;
  Fmt prod, acc;
  int order;
  int64_t chunk;
};

// one output scalar out[b][oh][ow][co]; m = (b*Hout + oh)*Wout + ow
int conv_point(const ConvArgs& c, int64_t m, int64_t co, float* out) {
  int64_t ow = m % c.Wout, oh = (m / c.Wout) % c.Hout, b = m / (c.Wout * c.Hout);
  Chain ch(&c.prod, &c.acc, c.order, c.chunk);
  for (int64_t kh = 0; kh < c.KH; ++kh)
    for (int64_t kw = 0; kw < c.KW; ++kw)
      for (int64_t ci = 0; ci < c.Cin; ++ci) {
        int64_t ih = oh * c.stride_h - c.pad_h + kh;
        int64_t iw = ow * c.stride_w - c.pad_w + kw;
        uint8_t xv = 0;  // a padded tap is the value 0
        if (ih >= 0 && ih < c.H && iw >= 0 && iw < c.W) xv = c.x[((b * c.H + ih) * c.W + iw) * c.Cin + ci];
        uint8_t wv = c.w[((co * c.KH + kh) * c.KW + kw) * c.Cin + ci];
        ch.push(xv, wv);
        if (ch.status != LBO_OK) return ch.status;
      }
  Dy y = ch.finish();
  if (ch.status != LBO_OK) return ch.status;
  float yf;
  if (!to_float(y, &yf)) return LBO_ERR_RANGE;
  float sx = c.sx_len == 1 ? c.sx[0] : c.sx[m];
  float sw = c.sw_len == 1 ? c.sw[0] : c.sw[co];
  *out = epilogue(yf, sx, sw, c.bias ? c.bias + co : nullptr);
  return LBO_OK;
}

int fill_gemm(GemmArgs* g, const uint8_t* A, const uint8_t* B, const float* sa, int sa_len, const float* sb,
              int sb_len, const float* bias, int64_t M, int64_t N, int64_t K, const lbo_fmt* pf,
              const lbo_fmt* af, int order, int64_t chunk) {
  if (!A || !B || !sa || !sb) return LBO_ERR_ARG;
  if (M < 0 || N < 0 || K < 0) return LBO_ERR_ARG;
  if (!(sa_len == 1 || sa_len == M) || !(sb_len == 1 || sb_len == N)) return LBO_ERR_ARG;
  int st = check_order(order, chunk);
  if (st != LBO_OK) return st;
  if ((st = make_fmt(pf, &g->prod)) != LBO_OK) return st;
  if ((st = make_fmt(af, &g->acc)) != LBO_OK) return st;
  g->A = A; g->B = B; g->sa = sa; g->sb = sb; g->bias = bias;
  g->sa_len = sa_len; g->sb_len = sb_len;
  g->M = M; g->N = N; g->K = K;
  g->order = order; g->chunk = chunk;
  return LBO_OK;
}

int fill_conv(ConvArgs* c, const uint8_t* x, const uint8_t* w, const float* sx, int sx_len, const float* sw,
              int sw_len, const float* bias, int64_t B, int64_t H, int64_t W, int64_t Cin, int64_t Cout,
              int64_t KH, int64_t KW, int64_t stride_h, int64_t stride_w, int64_t pad_h, int64_t pad_w,
              const lbo_fmt* pf, const lbo_fmt* af, int order, int64_t chunk) {
  if (!x || !w || !sx || !sw) return LBO_ERR_ARG;
  if (B < 1 || H < 1 || W < 1 || Cin < 1 || Cout < 1 || KH < 1 || KW < 1) return LBO_ERR_ARG;
  if (stride_h < 1 || stride_w < 1 || pad_h < 0 || pad_w < 0) return LBO_ERR_ARG;
  int64_t Hout = (H + 2 * pad_h - KH) / stride_h + 1, Wout = (W + 2 * pad_w - KW) / stride_w + 1;
  if (H + 2 * pad_h < KH || W + 2 * pad_w < KW || Hout < 1 || Wout < 1) return LBO_ERR_ARG;
  int64_t M = B * Hout * Wout;
  if (!(sx_len == 1 || sx_len == M) || !(sw_len == 1 || sw_len == Cout)) return LBO_ERR_ARG;
  int st = check_order(order, chunk);
  if (st != LBO_OK) return st;
  if ((st = make_fmt(pf, &c->prod)) != LBO_OK) return st;
  if ((st = make_fmt(af, &c->acc)) != LBO_OK) return st;
  c->x = x; c->w = w; c->sx = sx; c->sw = sw; c->bias = bias;
  c->sx_len = sx_len; c->sw_len = sw_len;
  c->B = B; c->H = H; c->W = W; c->Cin = Cin; c->Cout = Cout; c->KH = KH; c->KW = KW;
  c->stride_h = stride_h; c->stride_w = stride_w; c->pad_h = pad_h; c->pad_w = pad_w;
  c->Hout = Hout; c->Wout = Wout;
  c->order = order; c->chunk = chunk;
  return LBO_OK;
}

}  // namespace

extern "C" {

int lbo_version(void) { return 1; }

// value of one E4M3 byte
int lbo_decode_e4m3(uint8_t code, double* value) {
  if (!value) return LBO_ERR_ARG;
  Dy v;
  if (!decode_e4m3(code, &v)) return LBO_ERR_NAN_CODE;
  return to_double(v, value) ? LBO_OK : LBO_ERR_RANGE;
}

// value of one byte of the paper's M4E3 W/A format (bias 0)
int lbo_decode_m4e3(uint8_t code, double* value) {
  if (!value) return LBO_ERR_ARG;
  Dy v;
  decode_m4e3(code, &v);
  return to_double(v, value) ? LBO_OK : LBO_ERR_RANGE;
}

// R_OF and R_UF of Eq. 2 (as doubles; fails if R_OF is not a double)
int lbo_range(const lbo_fmt* f, double* r_of, double* r_uf) {
  Fmt fm;
  int st = make_fmt(f, &fm);
  if (st != LBO_OK) return st;
  if (r_of && !to_double(fm.r_of, r_of)) return LBO_ERR_RANGE;
  if (r_uf) *r_uf = std::ldexp(1.0, -fm.b);
  return LBO_OK;
}

// y = Q(x) for any finite double x (x is taken as the exact real number it holds)
int lbo_quantise(const lbo_fmt* f, double x, double* y) {
  Fmt fm;
  int st = make_fmt(f, &fm);
  if (st != LBO_OK) return st;
  Dy v;
  if (!y || !from_double(x, &v)) return LBO_ERR_ARG;
  return to_double(quantise(fm, v), y) ? LBO_OK : LBO_ERR_RANGE;
}

// One FMAq step (Eq. 4) from given running sums: out[(t * nx + i) * nw + j] = Q_acc(Q_prod(x_i * w_j) + s_t), for
// every running sum s_t (taken as the exact number the double holds), x code and w code.  Lets the tests take the
// last step of a chain from every state the chain can be in.
int lbo_fmaq_grid(const lbo_fmt* pf, const lbo_fmt* af, const uint8_t* xcodes, int64_t nx, const uint8_t* wcodes,
                  int64_t nw, const double* s_values, int64_t ns, double* out, int nthreads) {
  Fmt p, a;
  int st;
  if ((st = make_fmt(pf, &p)) != LBO_OK) return st;
  if ((st = make_fmt(af, &a)) != LBO_OK) return st;
  if (nx < 0 || nw < 0 || ns < 0 || (nx * nw * ns > 0 && (!xcodes || !wcodes || !s_values || !out))) return LBO_ERR_ARG;
  return parallel_items(ns * nx, nthreads, [&](int64_t item) {
    const int64_t t = item / nx, i = item % nx;
    Dy s0;
    if (!from_double(s_values[t], &s0)) return (int)LBO_ERR_ARG;
    for (int64_t j = 0; j < nw; ++j) {
      Chain c(&p, &a, LBO_ORDER_SEQUENTIAL, 1);
      c.first = s0;
      c.fmaq_step(xcodes[i], wcodes[j]);
      if (c.status != LBO_OK) return c.status;
      if (!to_double(c.first, &out[(t * nx + i) * nw + j])) return (int)LBO_ERR_RANGE;
    }
    return (int)LBO_OK;
  });
}

// One dot product over K byte pairs (element strides in bytes).  y receives the result.
// trace, if not null, has K entries: the first-hierarchy running sum after each step
// (in chunked order it restarts from 0 at each chunk; the entry of a chunk's last step
// is the chunk sum before it is folded into the second hierarchy).
int lbo_dot(const lbo_fmt* pf, const lbo_fmt* af, int order, int64_t chunk, const uint8_t* x, int64_t stride_x,
            const uint8_t* w, int64_t stride_w, int64_t K, double* y, double* trace) {
  Fmt p, a;
  int st = check_order(order, chunk);
  if (st != LBO_OK) return st;
  if ((st = make_fmt(pf, &p)) != LBO_OK) return st;
  if ((st = make_fmt(af, &a)) != LBO_OK) return st;
  if (K < 0 || !y || (K > 0 && (!x || !w))) return LBO_ERR_ARG;
  Chain c(&p, &a, order, chunk);
  for (int64_t i = 0; i < K; ++i) {
    c.fmaq_step(x[i * stride_x], w[i * stride_w]);
    if (c.status != LBO_OK) return c.status;
    if (trace && !to_double(c.first, &trace[i])) return LBO_ERR_RANGE;
    c.end_of_step();
    if (c.status != LBO_OK) return c.status;
  }
  Dy r = c.finish();
  if (c.status != LBO_OK) return c.status;
  return to_double(r, y) ? LBO_OK : LBO_ERR_RANGE;
}

// out[M][N] = epilogue(dot(A[m][:], B[n][:]))
int lbo_gemm(const uint8_t* A, const uint8_t* B, const float* sa, int sa_len, const float* sb, int sb_len,
             const float* bias, int64_t M, int64_t N, int64_t K, const lbo_fmt* pf, const lbo_fmt* af, int order,
             int64_t chunk, float* out, int nthreads) {
  GemmArgs g;
  int st = fill_gemm(&g, A, B, sa, sa_len, sb, sb_len, bias, M, N, K, pf, af, order, chunk);
  if (st != LBO_OK) return st;
  if (!out && M * N > 0) return LBO_ERR_ARG;
  return parallel_items(M, nthreads, [&](int64_t m) {
    for (int64_t n = 0; n < N; ++n) {
      int s = gemm_point(g, m, n, out + m * N + n);
      if (s != LBO_OK) return s;
    }
    return (int)LBO_OK;
  });
}

// last[M][N]: for the SEQUENTIAL chain of every output, the index of the last step whose exact sum
// Q_prod(x_i w_i) + S_i reached R_OF of the accumulator format (the step where STE^OF of App. D is 0), or -1
int lbo_gemm_last_overflow(const uint8_t* A, const uint8_t* B, int64_t M, int64_t N, int64_t K, const lbo_fmt* pf,
                           const lbo_fmt* af, int32_t* last, int nthreads) {
  GemmArgs g;
  const float one = 1.0f;
  int st = fill_gemm(&g, A, B, &one, 1, &one, 1, nullptr, M, N, K, pf, af, LBO_ORDER_SEQUENTIAL, 1);
  if (st != LBO_OK) return st;
  if (g.prod.fixed || g.acc.fixed) return LBO_ERR_FORMAT;  // the estimators are defined on Eq. 2
  if (!last && M * N > 0) return LBO_ERR_ARG;
  return parallel_items(M, nthreads, [&](int64_t m) {
    for (int64_t n = 0; n < N; ++n) {
      Chain c(&g.prod, &g.acc, g.order, g.chunk);
      for (int64_t i = 0; i < K; ++i) {
        c.push(A[m * K + i], B[n * K + i]);
        if (c.status != LBO_OK) return c.status;
      }
      last[m * N + n] = (int32_t)c.last_overflow;
    }
    return (int)LBO_OK;
  });
}

// STE bit masks of the re-computation pass (Sec. 4, App. D).  mask1[M][ceil(K/32)][N]: bit (i % 32) of word i / 32
// of output (m, n) is the STE value of step i of the first hierarchy (of the only one in sequential order).
// mask2[M][ceil(C/32)][N], C = ceil(K / chunk), chunked order only: the same for the step that folds chunk j into
// the second hierarchy.  Unused high bits of the last word are 0.
int lbo_gemm_ste_mask(const uint8_t* A, const uint8_t* B, int64_t M, int64_t N, int64_t K, const lbo_fmt* pf,
                      const lbo_fmt* af, int order, int64_t chunk, int kind, float eps1, float eps2, uint32_t* mask1,
                      uint32_t* mask2, int nthreads) {
  GemmArgs g;
  const float one = 1.0f;
  int st = fill_gemm(&g, A, B, &one, 1, &one, 1, nullptr, M, N, K, pf, af, order, chunk);
  if (st != LBO_OK) return st;
  if (kind != LBO_STE_OF && kind != LBO_STE_DIFF) return LBO_ERR_ARG;
  if (g.prod.fixed || g.acc.fixed) return LBO_ERR_FORMAT;  // the estimators are defined on Eq. 2
  if (kind == LBO_STE_DIFF && !(eps1 > 0.0f && eps2 > 0.0f)) return LBO_ERR_ARG;
  const bool chunked = order == LBO_ORDER_CHUNKED;
  const int64_t W1 = (K + 31) / 32;
  const int64_t C = chunked ? (K + chunk - 1) / chunk : 0;
  const int64_t W2 = (C + 31) / 32;
  if ((M * N * W1 > 0 && !mask1) || (M * N * W2 > 0 && !mask2)) return LBO_ERR_ARG;
  return parallel_items(M, nthreads, [&](int64_t m) {
    for (int64_t n = 0; n < N; ++n) {
      // word w of output (m, n): base[(m * words + w) * N + n]
      auto word1 = [&](int64_t w) -> uint32_t& { return mask1[(m * W1 + w) * N + n]; };
      auto word2 = [&](int64_t w) -> uint32_t& { return mask2[(m * W2 + w) * N + n]; };
      for (int64_t i = 0; i < W1; ++i) word1(i) = 0;
      for (int64_t i = 0; i < W2; ++i) word2(i) = 0;
      Chain c(&g.prod, &g.acc, g.order, g.chunk);
      c.ste_kind = kind;
      c.eps1 = eps1;
      c.eps2 = eps2;
      for (int64_t i = 0; i < K; ++i) {
        c.fmaq_step(A[m * K + i], B[n * K + i]);
        if (c.status != LBO_OK) return c.status;
        if (c.ste_first) word1(i / 32) |= 1u << (i % 32);
        const int64_t before = c.chunks_closed;
        c.end_of_step();
        if (c.status != LBO_OK) return c.status;
        if (c.chunks_closed != before && c.ste_second) word2(before / 32) |= 1u << (before % 32);
      }
      const int64_t before = c.chunks_closed;
      c.finish();   // folds a short last chunk
      if (c.status != LBO_OK) return c.status;
      if (c.chunks_closed != before && c.ste_second) word2(before / 32) |= 1u << (before % 32);
    }
    return (int)LBO_OK;
  });
}

// out[p] = element (ms[p], ns[p]) of the same GEMM
int lbo_gemm_points(const uint8_t* A, const uint8_t* B, const float* sa, int sa_len, const float* sb, int sb_len,
                    const float* bias, int64_t M, int64_t N, int64_t K, const lbo_fmt* pf, const lbo_fmt* af,
                    int order, int64_t chunk, const int64_t* ms, const int64_t* ns, int64_t P, float* out,
                    int nthreads) {
  GemmArgs g;
  int st = fill_gemm(&g, A, B, sa, sa_len, sb, sb_len, bias, M, N, K, pf, af, order, chunk);
  if (st != LBO_OK) return st;
  if (P < 0 || (P > 0 && (!ms || !ns || !out))) return LBO_ERR_ARG;
  for (int64_t p = 0; p < P; ++p)
    if (ms[p] < 0 || ms[p] >= M || ns[p] < 0 || ns[p] >= N) return LBO_ERR_ARG;
  return parallel_items(P, nthreads, [&](int64_t p) { return gemm_point(g, ms[p], ns[p], out + p); });
}

// x: [B][H][W][Cin] bytes, w: [Cout][KH][KW][Cin] bytes, out: [B][Hout][Wout][Cout]
int lbo_conv2d(const uint8_t* x, const uint8_t* w, const float* sx, int sx_len, const float* sw, int sw_len,
               const float* bias, int64_t B, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t KH,
               int64_t KW, int64_t stride_h, int64_t stride_w, int64_t pad_h, int64_t pad_w, const lbo_fmt* pf,
               const lbo_fmt* af, int order, int64_t chunk, float* out, int nthreads) {
  ConvArgs c;
  int st = fill_conv(&c, x, w, sx, sx_len, sw, sw_len, bias, B, H, W, Cin, Cout, KH, KW, stride_h, stride_w, pad_h,
                     pad_w, pf, af, order, chunk);
  if (st != LBO_OK) return st;
  if (!out) return LBO_ERR_ARG;
  int64_t M = c.B * c.Hout * c.Wout;
  return parallel_items(M, nthreads, [&](int64_t m) {
    for (int64_t co = 0; co < c.Cout; ++co) {
      int s = conv_point(c, m, co, out + m * c.Cout + co);
      if (s != LBO_OK) return s;
    }
    return (int)LBO_OK;
  });
}

// out[p] = output scalar at flattened position ms[p] = (b*Hout + oh)*Wout + ow, channel ns[p]
int lbo_conv2d_points(const uint8_t* x, const uint8_t* w, const float* sx, int sx_len, const float* sw, int sw_len,
                      const float* bias, int64_t B, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t KH,
                      int64_t KW, int64_t stride_h, int64_t stride_w, int64_t pad_h, int64_t pad_w,
                      const lbo_fmt* pf, const lbo_fmt* af, int order, int64_t chunk, const int64_t* ms,
                      const int64_t* ns, int64_t P, float* out, int nthreads) {
  ConvArgs c;
  int st = fill_conv(&c, x, w, sx, sx_len, sw, sw_len, bias, B, H, W, Cin, Cout, KH, KW, stride_h, stride_w, pad_h,
                     pad_w, pf, af, order, chunk);
  if (st != LBO_OK) return st;
  if (P < 0 || (P > 0 && (!ms || !ns || !out))) return LBO_ERR_ARG;
  int64_t M = c.B * c.Hout * c.Wout;
  for (int64_t p = 0; p < P; ++p)
    if (ms[p] < 0 || ms[p] >= M || ns[p] < 0 || ns[p] >= c.Cout) return LBO_ERR_ARG;
  return parallel_items(P, nthreads, [&](int64_t p) { return conv_point(c, ms[p], ns[p], out + p); });
}

}  // extern "C"
