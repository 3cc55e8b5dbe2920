// C ABI of liblba: argument checks, the per-call arithmetic plan, tile choice and dispatch.
// The definitions of the operations are in include/lba.h; the kernel is in lba_kernel.cuh.
#include <cfloat>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <atomic>
#include <mutex>

#include "../../include/lba.h"
#include "lba_kernel.cuh"

namespace lba {

// one definition per (QM, ORD), in the lba_fam_*.cu translation units
#define LBA_DECL(QM, ORD) template <> cudaError_t launch_family<QM, ORD>(int, int, const Problem&, cudaStream_t);
LBA_DECL(QM_FLOOR_FAST, ORD_SEQ) LBA_DECL(QM_FLOOR_FAST, ORD_CHUNK_SLAB) LBA_DECL(QM_FLOOR_FAST, ORD_CHUNK_ANY)
LBA_DECL(QM_FLOOR_FAST, ORD_CHUNK16) LBA_DECL(QM_FLOOR_FULL, ORD_CHUNK16) LBA_DECL(QM_RNE_FULL, ORD_CHUNK16)
LBA_DECL(QM_FLOOR_FULL, ORD_SEQ) LBA_DECL(QM_FLOOR_FULL, ORD_CHUNK_SLAB) LBA_DECL(QM_FLOOR_FULL, ORD_CHUNK_ANY)
LBA_DECL(QM_RNE_FULL, ORD_SEQ) LBA_DECL(QM_RNE_FULL, ORD_CHUNK_SLAB) LBA_DECL(QM_RNE_FULL, ORD_CHUNK_ANY)
LBA_DECL(QM_RNE_WIDE, ORD_SEQ) LBA_DECL(QM_RNE_WIDE, ORD_CHUNK_SLAB) LBA_DECL(QM_RNE_WIDE, ORD_CHUNK_ANY)
#undef LBA_DECL

cudaError_t launch_last_overflow(int qm, int load, const Problem& p, cudaStream_t stream);
cudaError_t launch_ste_mask(int qm, int ord, int diff, int load, const Problem& p, cudaStream_t stream);
cudaError_t launch_ste_packed(int pq, int chunk16, int load, const Problem& p, cudaStream_t stream);
cudaError_t launch_fixed(int ord, int load, const Problem& p, cudaStream_t stream);
cudaError_t launch_cluster_pair(int pq, int load, const Problem& p, cudaStream_t stream);

namespace {

thread_local int g_last_cuda_error = 0;
std::atomic<int> g_tile_override{-1};  // testing and tuning hook (lba_set_tile_override)

int cuda_fail(cudaError_t e) {
  g_last_cuda_error = (int)e;
  return LBA_ERR_CUDA;
}

const LaunchFn kLaunch[QM_COUNT][ORD_COUNT] = {
    // last column: chunk == 16 has a kernel of its own only for the floor quantisers (the plan never
    // selects it for the others; their entries repeat the general chunk-of-slabs family)
    {launch_family<QM_FLOOR_FAST, ORD_SEQ>, launch_family<QM_FLOOR_FAST, ORD_CHUNK_SLAB>,
     launch_family<QM_FLOOR_FAST, ORD_CHUNK_ANY>, launch_family<QM_FLOOR_FAST, ORD_CHUNK16>},
    {launch_family<QM_FLOOR_FULL, ORD_SEQ>, launch_family<QM_FLOOR_FULL, ORD_CHUNK_SLAB>,
     launch_family<QM_FLOOR_FULL, ORD_CHUNK_ANY>, launch_family<QM_FLOOR_FULL, ORD_CHUNK16>},
    {launch_family<QM_RNE_FULL, ORD_SEQ>, launch_family<QM_RNE_FULL, ORD_CHUNK_SLAB>,
     launch_family<QM_RNE_FULL, ORD_CHUNK_ANY>, launch_family<QM_RNE_FULL, ORD_CHUNK16>},
    {launch_family<QM_RNE_WIDE, ORD_SEQ>, launch_family<QM_RNE_WIDE, ORD_CHUNK_SLAB>,
     launch_family<QM_RNE_WIDE, ORD_CHUNK_ANY>, launch_family<QM_RNE_WIDE, ORD_CHUNK_SLAB>},
};

const char* const kQmName[QM_COUNT] = {"floor_fast", "floor_full", "rne_full", "rne_wide"};
const char* const kOrdName[ORD_COUNT] = {"seq", "chunk_slab", "chunk_any", "chunk16"};
const char* const kLdName[LD_COUNT] = {"gemm_vec", "conv_vec", "any"};

// What the host needs to know about the operand bytes: the largest |x*w|, the grid every product (hence every sum)
// lies on, the smallest non-zero |x*w| as a power of two at or below it, and the widest product significand.
struct InputInfo {
  double max_product;   // E4M3: 448^2; M4E3 (Sec. 3.1): 248^2
  int top_product_exp;  // max_product < 2^top_product_exp
  int grid_exp;         // every product is a multiple of 2^grid_exp
  int min_product_exp;  // the smallest non-zero |x*w| lies in [2^min_product_exp, 2^(min_product_exp+1))
  int product_bits;     // significant bits of a product, at most
  int decode_exp;       // generic kernel: its byte-to-binary32 step yields value * 2^-decode_exp
};
constexpr InputInfo kE4M3 = {448.0 * 448.0, 18, -18, -18, 8, 120};
constexpr InputInfo kM4E3 = {248.0 * 248.0, 16, -8, 0, 10, 0};
constexpr double kPartialRound = 0.5;          // share of the rounding-up of CTAs / SMs that a partial last round costs (measured)
constexpr double kPairEff = 0.91;              // MAC rate of the cluster-pair tile relative to the plain 64x64 tile (measured)

struct Plan {
  int qm, ord;
  float dec_a, dec_b, c, un1, un2;
  float pk_a, pk_b, nrm_scale, inv_top;
  float clamp_lim, slab_factor, fold_factor;
  int pq, rne_packed;
  float rne_k_acc, rne_k_prod;
  QConst qp, qa;
  int chunk_slabs, chunk;
  int kp, ka, sx;   // product carrier = value * 2^kp, accumulator carrier = value * 2^ka, A operand = x * 2^sx
  int in_m4e3;      // operands are M4E3 bytes
  int sum_grid;     // every sum is a multiple of 2^sum_grid
  bool a_flush;     // the flush of Q_acc is reachable
  int fused;        // Q_prod is the identity on every reachable product: PQ_FUSED applies (plain packed tiles)
  float pk_b_fused; // B operand scaling for it: 2^(sw + ka - kp), so that x' w' lands in the accumulator carrier
  double a_top;     // largest reachable accumulator magnitude (real domain)
  // fixed-point accumulation (Eq. 1): the integer kernel's constants
  bool fixed;
  int fx_shift0, fx_lo_p, fx_hi_p, fx_sh_p, fx_hold_p, fx_lo_a, fx_hi_a, fx_sh_a, fx_wrap_a, fx_dl, fx_dr;
  float fx_unit;
};

bool fmt_ok(const lba_fmt* f) {
  return f->man_bits >= 1 && f->man_bits <= 23 && f->exp_bits >= 1 && f->exp_bits <= 8 && f->bias >= -96 &&
         f->bias <= 192 && (f->rounding == LBA_ROUND_FLOOR || f->rounding == LBA_ROUND_NEAREST_EVEN);
}

double r_of(const lba_fmt* f) {  // Eq. 2; exact in double for the admitted M, E, b
  return std::ldexp(2.0 - std::ldexp(1.0, -f->man_bits), (1 << f->exp_bits) - f->bias - 1);
}

void fill_qconst(QConst* q, int M, float sat) {
  const int sh = 23 - M;
  q->mask = sh == 0 ? 0xFFFFFFFFu : ~((1u << sh) - 1u);
  q->rne_shift = sh;
  q->rne_add = sh == 0 ? 0u : ((1u << (sh - 1)) - 1u);
  q->rne_lsb = sh == 0 ? 0u : 1u;
  q->sat = sat;
}

// Work out, on the host, how the two formats are carried in binary32 registers and which of the
// branches of Eq. 2 can be reached at all from E4M3 inputs; refuse what cannot be carried exactly.
// Eq. 1 formats (exp_bits = 0): man_bits = B, 2..24, so that every held integer converts to binary32 exactly;
// floor only; biases for which no shift of the integer kernel can leave 32 bits.
int make_fixed_plan(const lba_fmt* pf, const lba_fmt* af, int order, int chunk, int64_t K, Plan* pl) {
  for (const lba_fmt* f : {pf, af})
    if (f->exp_bits != 0 || f->man_bits < 2 || f->man_bits > 24 || f->rounding != LBA_ROUND_FLOOR) return LBA_ERR_FORMAT;
  if (pf->flags & LBA_FLAG_INPUT_M4E3) return LBA_ERR_FORMAT;  // the integer kernel decodes E4M3 only
  const double kMaxProduct = kE4M3.max_product;
  if (order != LBA_ORDER_SEQUENTIAL && order != LBA_ORDER_CHUNKED) return LBA_ERR_ORDER;
  if (order == LBA_ORDER_CHUNKED && chunk < 1) return LBA_ERR_ORDER;
  // the product P * 2^(qx + qw), qx + qw in [-18, 10], is cut by a right shift of 22 - b_prod - qx - qw >= 0
  if (pf->bias > 12 || pf->bias < -64 || af->bias > 64 || af->bias < -64) return LBA_ERR_FORMAT;
  const int d = af->bias - pf->bias;  // product units -> accumulator units
  if (d > 0 && (pf->man_bits - 1) + d > 30) return LBA_ERR_FORMAT;
  std::memset(pl, 0, sizeof(*pl));
  pl->fixed = true;
  pl->qm = QM_FLOOR_FULL;
  pl->fx_shift0 = 22 - pf->bias;
  pl->fx_lo_p = -(1 << (pf->man_bits - 1));
  pl->fx_hi_p = (1 << (pf->man_bits - 1)) - 1;
  pl->fx_sh_p = 32 - pf->man_bits;
  // the largest product magnitude is 448^2 = 200704: if floor(448^2 * 2^b_prod) fits, Q_prod never has to hold
  const bool p_fits = std::floor(std::ldexp(kMaxProduct, pf->bias)) <= (double)pl->fx_hi_p;
  pl->fx_hold_p = p_fits ? 0 : ((pf->flags & LBA_FLAG_WRAP) ? 2 : 1);
  pl->fx_lo_a = -(1 << (af->man_bits - 1));
  pl->fx_hi_a = (1 << (af->man_bits - 1)) - 1;
  pl->fx_sh_a = 32 - af->man_bits;
  pl->fx_wrap_a = (af->flags & LBA_FLAG_WRAP) ? 1 : 0;
  pl->fx_dl = d > 0 ? d : 0;
  pl->fx_dr = d < 0 ? (-d > 31 ? 31 : -d) : 0;
  pl->fx_unit = (float)std::ldexp(1.0, -af->bias);
  pl->chunk = chunk;
  if (order == LBA_ORDER_SEQUENTIAL || (int64_t)chunk >= K) {
    pl->ord = ORD_SEQ;  // a single chunk: T = hold(C + 0) = C, already held
  } else if (chunk % BK == 0) {
    pl->ord = ORD_CHUNK_SLAB;
    pl->chunk_slabs = chunk / BK;
  } else {
    pl->ord = ORD_CHUNK_ANY;
  }
  return LBA_OK;
}

int make_plan(const lba_fmt* pf, const lba_fmt* af, int order, int chunk, int64_t K, Plan* pl) {
  if (!pf || !af) return LBA_ERR_NULL;
  if (pf->exp_bits == 0 || af->exp_bits == 0) return make_fixed_plan(pf, af, order, chunk, K, pl);
  pl->fixed = false;
  if (!fmt_ok(pf) || !fmt_ok(af)) return LBA_ERR_FORMAT;
  if (pf->rounding != af->rounding) return LBA_ERR_FORMAT;  // one rounding rule per FMAq unit
  if (order != LBA_ORDER_SEQUENTIAL && order != LBA_ORDER_CHUNKED) return LBA_ERR_ORDER;
  if (order == LBA_ORDER_CHUNKED && chunk < 1) return LBA_ERR_ORDER;
  const bool nearest = af->rounding == LBA_ROUND_NEAREST_EVEN;
  const InputInfo in = (pf->flags & LBA_FLAG_INPUT_M4E3) ? kM4E3 : kE4M3;
  const double kMaxProduct = in.max_product;
  pl->in_m4e3 = (pf->flags & LBA_FLAG_INPUT_M4E3) ? 1 : 0;

  // ---- Q_prod
  // the flush is reachable iff R_UF_prod = 2^-b exceeds the smallest non-zero product
  const bool p_flush = (pf->flags & LBA_FLAG_UNDERFLOW) && -pf->bias > in.min_product_exp;
  // carrier = value * 2^kp; without a flush the grid step 2^grid_exp is placed at the smallest normal number
  const int no_flush_carrier = -126 - in.grid_exp;
  const int kp = p_flush ? pf->bias - 126 : no_flush_carrier;
  const double p_rof = r_of(pf);
  // nearest-even can carry a value in the last half step below R_OF past it, so reachability
  // is assessed with that margin; floor never increases a magnitude
  const bool p_sat = p_rof <= kMaxProduct * (nearest ? 1.0 + std::ldexp(1.0, -pf->man_bits - 1) : 1.0);
  const bool p_round = pf->man_bits < in.product_bits - 1;  // an E4M3 product has at most 8 significant bits, an M4E3 one 10
  const int p_emax = (1 << pf->exp_bits) - pf->bias - 1;
  float p_sat_carrier = FLT_MAX;
  if (p_sat) {
    if (p_emax + kp < -126 || p_emax + kp > 127) return LBA_ERR_FORMAT;
    p_sat_carrier = (float)std::ldexp(p_rof, kp);
  }
  // ---- Q_acc
  const double a_rof = r_of(af);
  const double max_term = p_sat ? p_rof : kMaxProduct;
  // |S_i| <= i * max_term under floor; under nearest-even each step may add half a grid step
  const double growth = nearest ? std::exp(std::fmin((double)(K > 0 ? K : 1) * std::ldexp(1.0, -af->man_bits - 1), 80.0)) : 1.0;
  const double max_sum = (double)(K > 0 ? K : 1) * max_term * growth;
  const bool a_sat = a_rof <= max_sum;
  const int a_emax = (1 << af->exp_bits) - af->bias - 1;
  // every sum is a multiple of the grid step of the products, unless a saturation put R_OF into the chain: R_OF is a
  // multiple of 2^(e_max - M) only, of the product format where Q_prod saturates and of the accumulator's where Q_acc does
  int sum_grid = in.grid_exp;
  if (p_sat && p_emax - pf->man_bits < sum_grid) sum_grid = p_emax - pf->man_bits;
  if (a_sat && a_emax - af->man_bits < sum_grid) sum_grid = a_emax - af->man_bits;
  // a sum can cancel down to one grid step: the flush is reachable iff R_UF_acc exceeds it; without a flush the
  // carrier places that step at the smallest normal number
  const bool a_flush = (af->flags & LBA_FLAG_UNDERFLOW) && -af->bias > sum_grid;
  const int ka = a_flush ? af->bias - 126 : -126 - sum_grid;
  pl->sum_grid = sum_grid;
  pl->a_flush = a_flush;
  float a_sat_carrier = FLT_MAX;
  if (a_sat) {
    if (a_emax + ka < -126 || a_emax + ka > 127) return LBA_ERR_FORMAT;
    a_sat_carrier = (float)std::ldexp(a_rof, ka);
  } else if (std::ldexp(max_sum, ka) >= std::ldexp(1.0, 127)) {
    return LBA_ERR_FORMAT;
  }
  if (ka - kp < -126 || ka - kp > 126) return LBA_ERR_FORMAT;
  // the finished sum must be a normal binary32 number in the real domain: reachable magnitudes
  // lie in [2^-18, min(R_OF_acc, max_sum)]
  if ((a_sat ? a_rof : max_sum) >= std::ldexp(1.0, 128)) return LBA_ERR_FORMAT;

  // ---- quantiser mode
  if (!nearest) {
    pl->qm = (p_round || p_sat) ? QM_FLOOR_FULL : QM_FLOOR_FAST;
  } else if (af->man_bits == 23) {
    // a 24-bit accumulator is one IEEE addition, provided nothing else of Eq. 2 can happen
    if (p_flush || a_flush || p_sat || a_sat || p_round) return LBA_ERR_FORMAT;
    pl->qm = QM_RNE_WIDE;
  } else if (af->man_bits == 22) {
    return LBA_ERR_FORMAT;  // round-to-odd needs two spare bits below the kept mantissa
  } else {
    pl->qm = QM_RNE_FULL;
  }
  fill_qconst(&pl->qp, pf->man_bits, p_sat_carrier);
  fill_qconst(&pl->qa, af->man_bits, a_sat_carrier);

  const int sx = (kp >= 0) ? kp / 2 : -((-kp + 1) / 2);  // floor(kp / 2)
  const int sw = kp - sx;
  pl->kp = kp;
  pl->ka = ka;
  pl->sx = sx;
  pl->a_top = a_sat ? a_rof : max_sum;
  pl->dec_a = (float)std::ldexp(1.0, in.decode_exp + sx);
  pl->dec_b = (float)std::ldexp(1.0, in.decode_exp + sw);
  pl->c = (float)std::ldexp(1.0, ka - kp);
  const int u1 = (-ka) / 2, u2 = (-ka) - u1;
  pl->un1 = (float)std::ldexp(1.0, u1);
  pl->un2 = (float)std::ldexp(1.0, u2);
  // packed floor kernel: operands decoded by the hardware converter, then scaled by 2^sx, 2^sw; row
  // norms and |S| are measured as fractions of 2^(e_max_acc + 1), the first magnitude the mantissa
  // mask alone would not bring back to R_OF.  A scale that binary32 cannot hold switches the
  // clamp-free path off (infinite norms) rather than risk an underestimate.
  pl->pk_a = (float)std::ldexp(1.0, sx);
  pl->pk_b = (float)std::ldexp(1.0, sw);
  if (!a_sat) {
    pl->nrm_scale = 0.0f;
    pl->inv_top = 0.0f;
  } else {
    const int e1 = -(a_emax + 1), e2 = -ka - (a_emax + 1);
    if (e1 < -140 || e1 > 127 || e2 < -126 || e2 > 127) {
      pl->nrm_scale = INFINITY;
      pl->inv_top = 0.0f;
    } else {
      pl->nrm_scale = (float)std::ldexp(1.0, e1);
      pl->inv_top = (float)std::ldexp(1.0, e2);
    }
  }

  // clamp elision (see Problem::clamp_lim): floor never raises a magnitude; nearest-even raises it by at most half a
  // grid step per rounding, i.e. by the factor 1 + 2^-(M+1): sixteen accumulator roundings and the product's own in a
  // slab, one in a fold.  A sum at or below R_OF = 2^(e_max+1) (1 - 2^-(M+1)) rounds to at most R_OF.
  if (nearest) {
    const double ea = 1.0 + std::ldexp(1.0, -af->man_bits - 1), ep = p_round ? 1.0 + std::ldexp(1.0, -pf->man_bits - 1) : 1.0;
    pl->clamp_lim = (float)(0.999 * (1.0 - std::ldexp(1.0, -af->man_bits - 1)));
    pl->slab_factor = (float)(std::pow(ea, 16) * ep * 1.0001);
    pl->fold_factor = (float)(ea * 1.0001);
  } else {
    pl->clamp_lim = 0.999f;
    pl->slab_factor = 1.0f;
    pl->fold_factor = 1.0f;
  }

  // ---- packed kernel: what Q_prod does beyond the flush.  Nearest-even rounds on the FP32 pipe by adding and
  // subtracting 1.5 * 2^(23-M) * 2^e, which needs that much exponent headroom above the largest carried magnitude.
  // Its sum is one FMA rounded to nearest, which equals one rounding of the exact sum only under these conditions:
  //   * the quantised product has no more significant bits than the accumulator (else a product that is the larger
  //     operand can sit exactly on a tie of the accumulator's grid, which a far smaller sum must break);
  //   * M_acc <= 10, so that an operand small enough to be lost in the binary32 rounding (below 2^-12 of the larger
  //     one) is also too small to move the larger one, which lies on the grid, as far as the nearest tie;
  //   * the product carrier is not scaled down by more than 2^12 on its way into the sum, so that every sum below
  //     R_UF_acc is a subnormal binary32 number exactly and `.ftz` flushes it (a smaller term could be rounded
  //     away next to -R_UF_acc and leave R_UF_acc itself standing).
  // Everything else in nearest-even mode runs in the generic kernel (round-to-odd, then the cut).
  pl->pq = p_sat ? PQ_MASK_SAT : (p_round ? PQ_MASK : PQ_NONE);
  pl->rne_k_acc = (float)std::ldexp(1.0, 23 - af->man_bits);
  pl->rne_k_prod = (float)std::ldexp(1.0, 23 - pf->man_bits);
  pl->rne_packed = 0;
  if (pl->qm == QM_RNE_FULL) {
    const int top_acc = (a_sat ? a_emax + 1 : (int)std::ceil(std::log2(max_sum)) + 1) + ka;
    const int top_prod = in.top_product_exp + kp;
    // significant bits of a quantised product: the exact product's, cut to M_prod + 1; a saturated product is R_OF_prod,
    // which has all M_prod + 1
    const int prod_bits = (p_sat || pf->man_bits + 1 < in.product_bits) ? pf->man_bits + 1 : in.product_bits;
    pl->rne_packed = (top_acc + 25 - af->man_bits <= 127) && (top_prod + 25 - pf->man_bits <= 127) && af->man_bits <= 10 &&
                     prod_bits <= af->man_bits + 1 && ka - kp >= -12 && ka - kp <= 60;
  }

  // ---- fused product and sum: Q_prod must be the identity on every reachable product (no cut, no saturation, no
  // product under R_UF_prod), and the rescaled B operand must stay a normal binary32 number
  {
    const int swf = sw + (ka - kp);
    const bool packed_q = pl->qm == QM_FLOOR_FAST || (pl->qm == QM_RNE_FULL && pl->rne_packed);
    pl->fused = packed_q && !p_flush && !p_sat && !p_round && swf - 9 >= -126 && swf + 9 <= 126;
    pl->pk_b_fused = pl->fused ? (float)std::ldexp(1.0, swf) : 0.0f;
  }

  // ---- order mode
  pl->chunk = chunk;
  pl->chunk_slabs = 0;
  if (order == LBA_ORDER_SEQUENTIAL || (int64_t)chunk >= K) {
    pl->ord = ORD_SEQ;  // a single chunk: the second hierarchy adds it to 0, which changes nothing
  } else if (chunk % BK == 0) {
    const bool packed = pl->qm == QM_FLOOR_FAST || pl->qm == QM_FLOOR_FULL || (pl->qm == QM_RNE_FULL && pl->rne_packed);
    pl->ord = (chunk == BK && packed) ? ORD_CHUNK16 : ORD_CHUNK_SLAB;
    pl->chunk_slabs = chunk / BK;
  } else {
    pl->ord = ORD_CHUNK_ANY;
  }
  return LBA_OK;
}

// SM count of the current device, asked once per device (148 if the query fails).
int sm_count() {
  static std::atomic<int> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  int v = cached[dev].load(std::memory_order_relaxed);
  if (v > 0) return v;
  if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
  cached[dev].store(v, std::memory_order_relaxed);
  return v;
}

// Tile choice.  All CTAs of a launch have the same work and K is never split, so the launch ends when the
// busiest SM has run its ceil(CTAs / SMs) tiles; larger tiles spend fewer instructions per MAC (eff, measured
// on B200 with every SM loaded), smaller ones fill the SMs more evenly.  An SM that holds fewer CTAs than its
// neighbours runs each of them faster, so the last, partial round costs less than a full one: measured on
// 4096-row GEMMs of 768 to 3072 columns, counting half of the rounding-up reproduces the order of the tiles.
// Pick the cheapest by that model.
// pair_ok: the call qualifies for the 64x64 tile shared by a cluster of two CTAs (TILE_PAIR)
int choose_tile(int64_t M, int64_t N, int64_t batch, int qm, int ord, int load, bool pair_ok = false) {
  const int forced = g_tile_override.load(std::memory_order_relaxed);
  if (forced >= 0 && forced < TILE_COUNT) return forced;
  if (forced == TILE_PAIR && pair_ok) return TILE_PAIR;
  const int sms = sm_count();
  // relative MAC rate of each tile with every SM loaded (8192^2 x 1024 and 4096 x 3072 x 768 GEMMs)
  const double eff_seq[TILE_COUNT] = {1.00, 0.92, 0.96, 0.82};
  const double eff_chunk[TILE_COUNT] = {1.00, 0.96, 0.99, 0.87};
  // nearest-even: three more packed instructions per pair and step; the 8x8 micro-tile loses its lead
  const double eff_rne_seq[TILE_COUNT] = {1.00, 0.97, 0.99, 0.95};
  const double eff_rne_chunk[TILE_COUNT] = {0.88, 0.95, 1.00, 0.91};
  // byte-wise loader (ResNet stem, 401408 x 64 x 147): the fetch is costly, so the tile with the fewest
  // fetched rows per output wins as long as it keeps its registers
  const double eff_any[TILE_COUNT] = {0.55, 1.00, 0.87, 0.73};
  const bool rne = qm == QM_RNE_FULL;
  const double* eff = load == LD_ANY ? eff_any
                                     : (ord == ORD_SEQ ? (rne ? eff_rne_seq : eff_seq) : (rne ? eff_rne_chunk : eff_chunk));
  int best = 0;
  double best_cost = 1e300;
  for (int t = 0; t < TILE_COUNT; ++t) {
    const TileInfo ti = tile_info(t);
    const double ctas = (double)((M + ti.bm - 1) / ti.bm) * (double)((N + ti.bn - 1) / ti.bn) * (double)batch;
    const double rounds = std::ceil(ctas / sms);
    const double per_sm = std::fmax(1.0, ctas / sms + kPartialRound * (rounds - ctas / sms));
    double cost = per_sm * ti.bm * ti.bn / eff[t];
    if (t == 0 && rounds < 2) cost /= 0.85;  // one 8-warp CTA alone does not keep an SM's pipes busy
    if (cost < best_cost) {
      best_cost = cost;
      best = t;
    }
  }
  if (pair_ok) {
    // two CTAs per 64x64 tile, each with half the chunks: twice the CTAs at half the work, a few per cent for the
    // hand-over of the chunk sums and the cluster barrier
    const double ctas = 2.0 * (double)((M + 63) / 64) * (double)((N + 63) / 64) * (double)batch;
    const double per_sm = std::fmax(1.0, ctas / sms + kPartialRound * (std::ceil(ctas / sms) - ctas / sms));
    const double cost = per_sm * (64.0 * 64.0 / 2.0) / (eff[2] * kPairEff);
    if (cost < best_cost) best = TILE_PAIR;
  }
  return best;
}

int fill_scales(Problem* p, const float* sa, int sa_len, const float* sb, int sb_len, const float* bias) {
  if (!sa || !sb) return LBA_ERR_NULL;
  if (!(sa_len == 1 || (int64_t)sa_len == p->M) || !(sb_len == 1 || (int64_t)sb_len == p->N))
    return LBA_ERR_SCALE_LEN;
  p->sa = sa;
  p->sb = sb;
  p->bias = bias;
  p->sa_per_row = sa_len != 1 ? 1 : 0;
  p->sb_per_col = sb_len != 1 ? 1 : 0;
  return LBA_OK;
}

void apply_plan(Problem* p, const Plan& pl) {
  p->dec_a = pl.dec_a;
  p->dec_b = pl.dec_b;
  p->c = pl.c;
  p->un1 = pl.un1;
  p->un2 = pl.un2;
  p->qp = pl.qp;
  p->qa = pl.qa;
  p->chunk_slabs = pl.chunk_slabs;
  p->chunk = pl.chunk;
  p->pk_a = pl.pk_a;
  p->pk_b = pl.pk_b;
  p->nrm_scale = pl.nrm_scale;
  p->inv_top = pl.inv_top;
  p->clamp_lim = pl.clamp_lim;
  p->slab_factor = pl.slab_factor;
  p->fold_factor = pl.fold_factor;
  p->pq = pl.pq;
  p->rne_packed = pl.rne_packed;
  p->in_m4e3 = pl.in_m4e3;
  p->rne_k_acc = pl.rne_k_acc;
  p->rne_k_prod = pl.rne_k_prod;
  p->fx_shift0 = pl.fx_shift0;
  p->fx_lo_p = pl.fx_lo_p; p->fx_hi_p = pl.fx_hi_p; p->fx_sh_p = pl.fx_sh_p; p->fx_hold_p = pl.fx_hold_p;
  p->fx_lo_a = pl.fx_lo_a; p->fx_hi_a = pl.fx_hi_a; p->fx_sh_a = pl.fx_sh_a; p->fx_wrap_a = pl.fx_wrap_a;
  p->fx_dl = pl.fx_dl; p->fx_dr = pl.fx_dr;
  p->fx_unit = pl.fx_unit;
}

bool aligned16(const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15) == 0; }

int run(const Problem& p, const Plan& pl, int load, cudaStream_t stream) {
  if (p.M == 0 || p.N == 0 || p.batch == 0) return LBA_OK;
  if (p.batch > 65535) return LBA_ERR_SHAPE;
  if (pl.fixed) {  // Eq. 1: the integer kernel, one tile shape
    if ((p.N + 63) / 64 > 65535) return LBA_ERR_SHAPE;
    const cudaError_t e = launch_fixed(pl.ord, load, p, stream);
    return e == cudaSuccess ? LBA_OK : cuda_fail(e);
  }
  const bool pair_ok = pl.ord == ORD_CHUNK16 && (pl.qm == QM_FLOOR_FAST || pl.qm == QM_FLOOR_FULL) && load != LD_ANY &&
                       2 * ((p.M + 63) / 64) <= 2147483647LL;
  const int tile = choose_tile(p.M, p.N, p.batch, pl.qm, pl.ord, load, pair_ok);
  if (tile == TILE_PAIR) {
    if ((p.N + 63) / 64 > 65535) return LBA_ERR_SHAPE;
    const cudaError_t e = launch_cluster_pair(pl.qm == QM_FLOOR_FAST ? PQ_NONE : pl.pq, load, p, stream);
    return e == cudaSuccess ? LBA_OK : cuda_fail(e);
  }
  const TileInfo ti = tile_info(tile);
  if ((p.N + ti.bn - 1) / ti.bn > 65535 || (p.M + ti.bm - 1) / ti.bm > 2147483647LL) return LBA_ERR_SHAPE;
  if (pl.fused && pl.ord != ORD_CHUNK_ANY) {  // the plain packed tiles have the fused variant
    Problem q = p;
    q.pq = PQ_FUSED;
    q.pk_b = pl.pk_b_fused;
    const cudaError_t e = kLaunch[pl.qm][pl.ord](tile, load, q, stream);
    return e == cudaSuccess ? LBA_OK : cuda_fail(e);
  }
  const cudaError_t e = kLaunch[pl.qm][pl.ord](tile, load, p, stream);
  return e == cudaSuccess ? LBA_OK : cuda_fail(e);
}

struct ConvGeom {
  int Hout, Wout;
  int64_t M, K;
};

int conv_geom(int B, int H, int W, int C_in, int C_out, int KH, int KW, int sh, int sw, int ph, int pw,
              ConvGeom* g) {
  if (B < 1 || H < 1 || W < 1 || C_in < 1 || C_out < 1 || KH < 1 || KW < 1 || sh < 1 || sw < 1 || ph < 0 || pw < 0)
    return LBA_ERR_SHAPE;
  if ((int64_t)H + 2 * (int64_t)ph < KH || (int64_t)W + 2 * (int64_t)pw < KW) return LBA_ERR_SHAPE;
  g->Hout = (H + 2 * ph - KH) / sh + 1;
  g->Wout = (W + 2 * pw - KW) / sw + 1;
  if (g->Hout < 1 || g->Wout < 1) return LBA_ERR_SHAPE;
  g->M = (int64_t)B * g->Hout * g->Wout;
  g->K = (int64_t)KH * KW * C_in;
  if (g->K > 2147483647LL || (int64_t)H * W * C_in > 2147483647LL) return LBA_ERR_SHAPE;
  return LBA_OK;
}

__global__ void count_nan_codes_kernel(const uint8_t* codes, int64_t n, unsigned long long* count) {
  unsigned long long local = 0;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    local += (codes[i] & 0x7F) == 0x7F;
  if (local) atomicAdd(count, local);
}

size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Sizes of the host-buffer variants are formed in size_t; a shape whose operand or output byte count does not fit
// well inside 63 bits is refused before any product can wrap.
bool sizes_fit(double a_bytes, double b_bytes, double out_bytes) {
  const double limit = 4611686018427387904.0;  // 2^62
  return a_bytes < limit && b_bytes < limit && out_bytes < limit && a_bytes + b_bytes + out_bytes < limit;
}

}  // namespace
}  // namespace lba

using namespace lba;

extern "C" {

int lba_version(void) { return 1; }

int lba_last_cuda_error(void) { return g_last_cuda_error; }

int lba_set_tile_override(int tile) {
  if (tile < -1 || tile > TILE_PAIR || tile == TILE_COUNT) return LBA_ERR_SHAPE;
  g_tile_override.store(tile, std::memory_order_relaxed);
  return LBA_OK;
}

const char* lba_status_string(int status) {
  switch (status) {
    case LBA_OK: return "ok";
    case LBA_ERR_NULL: return "a required pointer is NULL";
    case LBA_ERR_SHAPE: return "bad shape";
    case LBA_ERR_FORMAT: return "format out of range or not exactly representable in the binary32 carrier";
    case LBA_ERR_ORDER: return "unknown accumulation order or chunk < 1";
    case LBA_ERR_SCALE_LEN: return "scale length must be 1 or the matching dimension";
    case LBA_ERR_CUDA: return "a CUDA call failed (see lba_last_cuda_error)";
    case LBA_ERR_WORKSPACE: return "workspace missing, too small or misaligned";
    case LBA_ERR_STATIC_LIMIT: return "problem too large for the built-in workspace of lba_gemm_host_static (LBA_STATIC_WORKSPACE_BYTES)";
    default: return "unknown status";
  }
}

int lba_gemm(const uint8_t* A, const uint8_t* B, const float* scale_a, int scale_a_len, const float* scale_b,
             int scale_b_len, const float* bias, int64_t M, int64_t N, int64_t K, const lba_fmt* prod_fmt,
             const lba_fmt* acc_fmt, int order, int chunk, float* out, void* stream) {
  if (M < 0 || N < 0 || K < 0 || K > 2147483647LL) return LBA_ERR_SHAPE;
  Plan pl;
  int st = make_plan(prod_fmt, acc_fmt, order, chunk, K, &pl);
  if (st != LBA_OK) return st;
  Problem p;
  std::memset(&p, 0, sizeof(p));
  p.M = M;
  p.N = N;
  p.K = K;
  p.batch = 1;
  if ((st = fill_scales(&p, scale_a, scale_a_len, scale_b, scale_b_len, bias)) != LBA_OK) return st;
  if (M > 0 && N > 0 && !out) return LBA_ERR_NULL;
  if (K > 0 && ((M > 0 && !A) || (N > 0 && !B))) return LBA_ERR_NULL;
  p.A = A;
  p.B = B;
  p.out = out;
  apply_plan(&p, pl);
  const bool vec = K % BK == 0 && aligned16(A) && aligned16(B);
  return run(p, pl, vec ? LD_GEMM_VEC : LD_ANY, (cudaStream_t)stream);
}

int lba_gemm_batched(const uint8_t* A, const uint8_t* B, const float* scale_a, int scale_a_len, const float* scale_b,
                     int scale_b_len, const float* bias, int64_t batch, int64_t M, int64_t N, int64_t K,
                     int64_t stride_a, int64_t stride_b, int64_t stride_out, const lba_fmt* prod_fmt,
                     const lba_fmt* acc_fmt, int order, int chunk, float* out, void* stream) {
  if (batch < 0 || M < 0 || N < 0 || K < 0 || K > 2147483647LL) return LBA_ERR_SHAPE;
  // problems may share an operand (stride 0) but outputs must not overlap
  if (stride_a < 0 || stride_b < 0 || stride_out < 0) return LBA_ERR_SHAPE;
  if (batch > 1 && ((stride_a != 0 && stride_a < M * K) || (stride_b != 0 && stride_b < N * K) || stride_out < M * N))
    return LBA_ERR_SHAPE;
  Plan pl;
  int st = make_plan(prod_fmt, acc_fmt, order, chunk, K, &pl);
  if (st != LBA_OK) return st;
  Problem p;
  std::memset(&p, 0, sizeof(p));
  p.M = M;
  p.N = N;
  p.K = K;
  if ((st = fill_scales(&p, scale_a, scale_a_len, scale_b, scale_b_len, bias)) != LBA_OK) return st;
  if (batch > 0 && M > 0 && N > 0 && !out) return LBA_ERR_NULL;
  if (batch > 0 && K > 0 && ((M > 0 && !A) || (N > 0 && !B))) return LBA_ERR_NULL;
  p.A = A;
  p.B = B;
  p.out = out;
  p.batch_a = stride_a;
  p.batch_b = stride_b;
  p.batch_out = stride_out;
  apply_plan(&p, pl);
  const bool vec = K % BK == 0 && aligned16(A) && aligned16(B) && stride_a % 16 == 0 && stride_b % 16 == 0;
  // the grid's third dimension holds at most 65535 problems
  for (int64_t b0 = 0; b0 < batch; b0 += 65535) {
    Problem q = p;
    q.batch = batch - b0 < 65535 ? batch - b0 : 65535;
    q.A = A + b0 * stride_a;
    q.B = B + b0 * stride_b;
    q.out = out + b0 * stride_out;
    if ((st = run(q, pl, vec ? LD_GEMM_VEC : LD_ANY, (cudaStream_t)stream)) != LBA_OK) return st;
  }
  return LBA_OK;
}

int lba_gemm_last_overflow(const uint8_t* A, const uint8_t* B, int64_t M, int64_t N, int64_t K, const lba_fmt* prod_fmt,
                           const lba_fmt* acc_fmt, int32_t* last, void* stream) {
  if (M < 0 || N < 0 || K < 0 || K > 2147483647LL) return LBA_ERR_SHAPE;
  Plan pl;
  const int st = make_plan(prod_fmt, acc_fmt, LBA_ORDER_SEQUENTIAL, 1, K, &pl);
  if (st != LBA_OK) return st;
  if (pl.fixed || pl.in_m4e3 || (pl.qm != QM_FLOOR_FAST && pl.qm != QM_FLOOR_FULL)) return LBA_ERR_FORMAT;  // Eq. 2, floor rounding, E4M3 operands
  if (M == 0 || N == 0) return LBA_OK;
  if (!last || (K > 0 && (!A || !B))) return LBA_ERR_NULL;
  if ((N + 63) / 64 > 65535) return LBA_ERR_SHAPE;
  Problem p;
  std::memset(&p, 0, sizeof(p));
  p.M = M;
  p.N = N;
  p.K = K;
  p.batch = 1;
  p.A = A;
  p.B = B;
  p.out = reinterpret_cast<float*>(last);
  apply_plan(&p, pl);
  const bool vec = K % BK == 0 && aligned16(A) && aligned16(B);
  const cudaError_t e = launch_last_overflow(pl.qm, vec ? LD_GEMM_VEC : LD_ANY, p, (cudaStream_t)stream);
  return e == cudaSuccess ? LBA_OK : cuda_fail(e);
}

int lba_gemm_ste_mask(const uint8_t* A, const uint8_t* B, int64_t M, int64_t N, int64_t K, const lba_fmt* prod_fmt,
                      const lba_fmt* acc_fmt, int order, int chunk, int ste, float eps1, float eps2, uint32_t* mask1,
                      uint32_t* mask2, void* stream) {
  if (M < 0 || N < 0 || K < 0 || K > 2147483647LL - 64) return LBA_ERR_SHAPE;
  if (ste != LBA_STE_OF && ste != LBA_STE_DIFF) return LBA_ERR_ORDER;
  Plan pl;
  const int st = make_plan(prod_fmt, acc_fmt, order, chunk, K, &pl);
  if (st != LBA_OK) return st;
  if (pl.fixed || pl.in_m4e3 || (pl.qm != QM_FLOOR_FAST && pl.qm != QM_FLOOR_FULL)) return LBA_ERR_FORMAT;  // Eq. 2, floor rounding, E4M3 operands
  const bool chunked = order == LBA_ORDER_CHUNKED;
  const int64_t chunks = chunked ? (K + chunk - 1) / chunk : 0;
  Problem p;
  std::memset(&p, 0, sizeof(p));
  if (ste == LBA_STE_DIFF) {
    // the comparison |z - S| > fl(eps2 * fl(|u| + eps1)) runs on values scaled by 2^kd relative to the real
    // domain; scaling by a power of two commutes with binary32 rounding as long as nothing leaves the normal
    // range on either side, which is checked here for the extreme operands
    if (!(eps1 > 0.0f) || !(eps2 > 0.0f) || !std::isfinite(eps1) || !std::isfinite(eps2)) return LBA_ERR_FORMAT;
    const int kd = pl.ka + 32;
    const auto normal = [kd](double v) {  // a normal binary32 magnitude in the real domain and after scaling
      const double lo = std::ldexp(1.0, -126), hi = std::ldexp(1.0, 127), w = std::ldexp(v, kd);
      return v >= lo && v < hi && w >= lo && w < hi;
    };
    const double u_max = std::fmax(std::ldexp(1.0, 18), pl.a_top);   // |x w| < 2^18; a chunk sum <= a_top
    const double u_min = std::ldexp(1.0, -18);                       // smallest non-zero |x w| and chunk sum
    // smallest non-zero |z - S|: one step of the accumulator's grid in its lowest binade where sums below R_UF are
    // flushed, else one step of the grid on which every sum lies
    const double d_min = pl.a_flush ? std::ldexp(1.0, -acc_fmt->bias - acc_fmt->man_bits) : std::ldexp(1.0, pl.sum_grid);
    for (const double v : {(double)eps1, u_max + eps1, (double)eps2 * eps1, (double)eps2 * (u_max + eps1), u_min, u_max,
                           d_min, 2.0 * pl.a_top})
      if (!normal(v)) return LBA_ERR_FORMAT;
    // A is rescaled so that A' * B' = |x w| * 2^kd; |x| lies in [2^-9, 448]
    const int sa = pl.sx + kd - pl.kp;
    if (sa - 9 < -126 || sa + 9 > 127) return LBA_ERR_FORMAT;
    const int kp = pl.kp;
    p.diff_scale = std::ldexp(1.0f, 32);
    p.diff_a_scale = std::ldexp(1.0f, kd - kp);
    p.diff_eps1 = std::ldexp(eps1, kd);
    p.diff_eps2 = eps2;
  }
  if (M == 0 || N == 0 || K == 0) return LBA_OK;
  if (!A || !B || !mask1 || (chunked && !mask2)) return LBA_ERR_NULL;
  if ((N + 63) / 64 > 65535) return LBA_ERR_SHAPE;
  p.M = M;
  p.N = N;
  p.K = K;
  p.batch = 1;
  p.A = A;
  p.B = B;
  apply_plan(&p, pl);
  p.mask1 = mask1;
  p.mask2 = mask2;
  p.mask2_words = (chunks + 31) / 32;
  p.ste_limit = (float)(0.999 * (1.0 - std::ldexp(1.0, -(acc_fmt->man_bits + 1))));
  // the single-chunk shortcut of the forward pass does not apply: the fold of that one chunk is a step too
  int ord = ORD_SEQ;
  if (chunked) {
    ord = chunk % BK == 0 ? ORD_CHUNK_SLAB : ORD_CHUNK_ANY;
    p.chunk = chunk;
    p.chunk_slabs = chunk / BK;
  }
  const bool vec = K % BK == 0 && aligned16(A) && aligned16(B);
  const int load = vec ? LD_GEMM_VEC : LD_ANY;
  // the overflow masks in sequential and chunk-16 order come from the packed kernel (tile override 3 keeps the
  // scalar tracking kernel, for tests and comparisons); everything else from the scalar one
  const bool packed = ste == LBA_STE_OF && (!chunked || chunk == BK) && g_tile_override.load(std::memory_order_relaxed) != 3;
  const cudaError_t e = packed ? launch_ste_packed(pl.qm == QM_FLOOR_FAST ? PQ_NONE : pl.pq, chunked ? 1 : 0, load, p, (cudaStream_t)stream)
                               : launch_ste_mask(pl.qm, ord, ste == LBA_STE_DIFF, load, p, (cudaStream_t)stream);
  return e == cudaSuccess ? LBA_OK : cuda_fail(e);
}

int lba_conv2d(const uint8_t* x, const uint8_t* w, const float* scale_x, int scale_x_len, const float* scale_w,
               int scale_w_len, const float* bias, int B, int H, int W, int C_in, int C_out, int KH, int KW,
               int stride_h, int stride_w, int pad_h, int pad_w, const lba_fmt* prod_fmt, const lba_fmt* acc_fmt,
               int order, int chunk, float* out, void* stream) {
  ConvGeom g;
  int st = conv_geom(B, H, W, C_in, C_out, KH, KW, stride_h, stride_w, pad_h, pad_w, &g);
  if (st != LBA_OK) return st;
  Plan pl;
  if ((st = make_plan(prod_fmt, acc_fmt, order, chunk, g.K, &pl)) != LBA_OK) return st;
  if (!x || !w || !out) return LBA_ERR_NULL;
  Problem p;
  std::memset(&p, 0, sizeof(p));
  p.M = g.M;
  p.N = C_out;
  p.K = g.K;
  p.batch = 1;
  if ((st = fill_scales(&p, scale_x, scale_x_len, scale_w, scale_w_len, bias)) != LBA_OK) return st;
  p.A = x;
  p.B = w;
  p.out = out;
  p.is_conv = 1;
  p.H = H; p.W = W; p.Cin = C_in; p.KH = KH; p.KW = KW;
  p.sh = stride_h; p.sw = stride_w; p.ph = pad_h; p.pw = pad_w;
  p.Hout = g.Hout; p.Wout = g.Wout;
  apply_plan(&p, pl);
  const bool vec = C_in % BK == 0 && aligned16(x) && aligned16(w);
  return run(p, pl, vec ? LD_CONV_VEC : LD_ANY, (cudaStream_t)stream);
}

size_t lba_gemm_host_workspace_bytes(int64_t M, int64_t N, int64_t K, int scale_a_len, int scale_b_len,
                                     int has_bias) {
  if (M < 0 || N < 0 || K < 0 || scale_a_len < 0 || scale_b_len < 0) return 0;
  if (!sizes_fit((double)M * (double)K, (double)N * (double)K, 4.0 * (double)M * (double)N)) return 0;
  size_t b = 0;
  b += round_up((size_t)M * K, 256) + round_up((size_t)N * K, 256);
  b += round_up((size_t)scale_a_len * 4, 256) + round_up((size_t)scale_b_len * 4, 256);
  if (has_bias) b += round_up((size_t)N * 4, 256);
  b += round_up((size_t)M * N * 4, 256);
  return b;
}

int lba_gemm_host(const uint8_t* A, const uint8_t* B, const float* scale_a, int scale_a_len, const float* scale_b,
                  int scale_b_len, const float* bias, int64_t M, int64_t N, int64_t K, const lba_fmt* prod_fmt,
                  const lba_fmt* acc_fmt, int order, int chunk, float* out, void* workspace,
                  size_t workspace_bytes, void* stream) {
  if (M < 0 || N < 0 || K < 0 || K > 2147483647LL) return LBA_ERR_SHAPE;
  if (!sizes_fit((double)M * (double)K, (double)N * (double)K, 4.0 * (double)M * (double)N)) return LBA_ERR_SHAPE;
  if (!scale_a || !scale_b) return LBA_ERR_NULL;
  if (!(scale_a_len == 1 || scale_a_len == M) || !(scale_b_len == 1 || scale_b_len == N)) return LBA_ERR_SCALE_LEN;
  Plan pl;
  int st = make_plan(prod_fmt, acc_fmt, order, chunk, K, &pl);  // reject bad formats before any copy
  if (st != LBA_OK) return st;
  const size_t need = lba_gemm_host_workspace_bytes(M, N, K, scale_a_len, scale_b_len, bias != nullptr);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255)) return LBA_ERR_WORKSPACE;
  if ((M * K > 0 && !A) || (N * K > 0 && !B) || (M * N > 0 && !out)) return LBA_ERR_NULL;
  cudaStream_t s = (cudaStream_t)stream;
  uint8_t* w = (uint8_t*)workspace;
  uint8_t* dA = w; w += round_up((size_t)M * K, 256);
  uint8_t* dB = w; w += round_up((size_t)N * K, 256);
  float* dsa = (float*)w; w += round_up((size_t)scale_a_len * 4, 256);
  float* dsb = (float*)w; w += round_up((size_t)scale_b_len * 4, 256);
  float* dbias = nullptr;
  if (bias) { dbias = (float*)w; w += round_up((size_t)N * 4, 256); }
  float* dout = (float*)w;
  cudaError_t e;
  if (M * K > 0 && (e = cudaMemcpyAsync(dA, A, (size_t)M * K, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
  if (N * K > 0 && (e = cudaMemcpyAsync(dB, B, (size_t)N * K, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
  if ((e = cudaMemcpyAsync(dsa, scale_a, (size_t)scale_a_len * 4, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
  if ((e = cudaMemcpyAsync(dsb, scale_b, (size_t)scale_b_len * 4, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
  if (bias && N > 0 && (e = cudaMemcpyAsync(dbias, bias, (size_t)N * 4, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
  st = lba_gemm(dA, dB, dsa, scale_a_len, dsb, scale_b_len, dbias, M, N, K, prod_fmt, acc_fmt, order, chunk, dout, stream);
  if (st != LBA_OK) return st;
  if (M * N > 0 && (e = cudaMemcpyAsync(out, dout, (size_t)M * N * 4, cudaMemcpyDeviceToHost, s)) != cudaSuccess) return cuda_fail(e);
  return LBA_OK;
}

size_t lba_conv2d_host_workspace_bytes(int B, int H, int W, int C_in, int C_out, int KH, int KW, int stride_h,
                                       int stride_w, int pad_h, int pad_w, int scale_x_len, int scale_w_len,
                                       int has_bias) {
  ConvGeom g;
  if (conv_geom(B, H, W, C_in, C_out, KH, KW, stride_h, stride_w, pad_h, pad_w, &g) != LBA_OK) return 0;
  if (scale_x_len < 0 || scale_w_len < 0) return 0;
  if (!sizes_fit((double)B * H * W * C_in, (double)C_out * (double)g.K, 4.0 * (double)g.M * C_out)) return 0;
  size_t b = 0;
  b += round_up((size_t)B * H * W * C_in, 256) + round_up((size_t)C_out * g.K, 256);
  b += round_up((size_t)scale_x_len * 4, 256) + round_up((size_t)scale_w_len * 4, 256);
  if (has_bias) b += round_up((size_t)C_out * 4, 256);
  b += round_up((size_t)g.M * C_out * 4, 256);
  return b;
}

int lba_conv2d_host(const uint8_t* x, const uint8_t* w, const float* scale_x, int scale_x_len,
                    const float* scale_w, int scale_w_len, const float* bias, int B, int H, int W, int C_in,
                    int C_out, int KH, int KW, int stride_h, int stride_w, int pad_h, int pad_w,
                    const lba_fmt* prod_fmt, const lba_fmt* acc_fmt, int order, int chunk, float* out,
                    void* workspace, size_t workspace_bytes, void* stream) {
  ConvGeom g;
  int st = conv_geom(B, H, W, C_in, C_out, KH, KW, stride_h, stride_w, pad_h, pad_w, &g);
  if (st != LBA_OK) return st;
  if (!sizes_fit((double)B * H * W * C_in, (double)C_out * (double)g.K, 4.0 * (double)g.M * C_out)) return LBA_ERR_SHAPE;
  if (!x || !w || !out || !scale_x || !scale_w) return LBA_ERR_NULL;
  if (!(scale_x_len == 1 || scale_x_len == g.M) || !(scale_w_len == 1 || scale_w_len == C_out)) return LBA_ERR_SCALE_LEN;
  Plan pl;
  if ((st = make_plan(prod_fmt, acc_fmt, order, chunk, g.K, &pl)) != LBA_OK) return st;
  const size_t need = lba_conv2d_host_workspace_bytes(B, H, W, C_in, C_out, KH, KW, stride_h, stride_w, pad_h, pad_w,
                                                      scale_x_len, scale_w_len, bias != nullptr);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255)) return LBA_ERR_WORKSPACE;
  cudaStream_t s = (cudaStream_t)stream;
  const size_t xb = (size_t)B * H * W * C_in, wb = (size_t)C_out * g.K, ob = (size_t)g.M * C_out * 4;
  uint8_t* ws = (uint8_t*)workspace;
  uint8_t* dx = ws; ws += round_up(xb, 256);
  uint8_t* dw = ws; ws += round_up(wb, 256);
  float* dsx = (float*)ws; ws += round_up((size_t)scale_x_len * 4, 256);
  float* dsw = (float*)ws; ws += round_up((size_t)scale_w_len * 4, 256);
  float* dbias = nullptr;
  if (bias) { dbias = (float*)ws; ws += round_up((size_t)C_out * 4, 256); }
  float* dout = (float*)ws;
  cudaError_t e;
  if ((e = cudaMemcpyAsync(dx, x, xb, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
  if ((e = cudaMemcpyAsync(dw, w, wb, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
  if ((e = cudaMemcpyAsync(dsx, scale_x, (size_t)scale_x_len * 4, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
  if ((e = cudaMemcpyAsync(dsw, scale_w, (size_t)scale_w_len * 4, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
  if (bias && (e = cudaMemcpyAsync(dbias, bias, (size_t)C_out * 4, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
  st = lba_conv2d(dx, dw, dsx, scale_x_len, dsw, scale_w_len, dbias, B, H, W, C_in, C_out, KH, KW, stride_h, stride_w,
                  pad_h, pad_w, prod_fmt, acc_fmt, order, chunk, dout, stream);
  if (st != LBA_OK) return st;
  if ((e = cudaMemcpyAsync(out, dout, ob, cudaMemcpyDeviceToHost, s)) != cudaSuccess) return cuda_fail(e);
  return LBA_OK;
}

int lba_count_nan_codes(const uint8_t* codes, int64_t n, unsigned long long* count, void* stream) {
  if (n < 0) return LBA_ERR_SHAPE;
  if (!count || (n > 0 && !codes)) return LBA_ERR_NULL;
  if (n == 0) return LBA_OK;
  int blocks = (int)((n + 255) / 256 < 1184 ? (n + 255) / 256 : 1184);
  count_nan_codes_kernel<<<blocks, 256, 0, (cudaStream_t)stream>>>(codes, n, count);
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? LBA_OK : cuda_fail(e);
}

int lba_describe_plan(int64_t M, int64_t N, int64_t K, const lba_fmt* prod_fmt, const lba_fmt* acc_fmt, int order,
                      int chunk, int is_conv, int vec_ok, char* buf, size_t buf_len) {
  return lba_describe_plan_batched(1, M, N, K, prod_fmt, acc_fmt, order, chunk, is_conv, vec_ok, buf, buf_len);
}

int lba_describe_plan_batched(int64_t batch, int64_t M, int64_t N, int64_t K, const lba_fmt* prod_fmt, const lba_fmt* acc_fmt,
                              int order, int chunk, int is_conv, int vec_ok, char* buf, size_t buf_len) {
  if (batch < 1 || M < 0 || N < 0 || K < 0) return LBA_ERR_SHAPE;
  Plan pl;
  const int st = make_plan(prod_fmt, acc_fmt, order, chunk, K, &pl);
  if (st != LBA_OK) return st;
  const int load = vec_ok ? (is_conv ? LD_CONV_VEC : LD_GEMM_VEC) : LD_ANY;
  if (pl.fixed) {
    if (buf && buf_len)
      std::snprintf(buf, buf_len, "tile=64x64x%d micro=4x4 q=fixed order=%s load=%s grid=%lldx%lld", BK, kOrdName[pl.ord],
                    kLdName[load], (long long)((M + 63) / 64), (long long)((N + 63) / 64));
    return LBA_OK;
  }
  const bool pair_ok = pl.ord == ORD_CHUNK16 && (pl.qm == QM_FLOOR_FAST || pl.qm == QM_FLOOR_FULL) && load != LD_ANY;
  const int tile = choose_tile(M > 0 ? M : 1, N > 0 ? N : 1, batch, pl.qm, pl.ord, load, pair_ok);
  // which kernel runs and what Q_prod costs there beyond the flush
  const bool packed = pl.ord != ORD_CHUNK_ANY &&
                      (pl.qm == QM_FLOOR_FAST || pl.qm == QM_FLOOR_FULL || (pl.qm == QM_RNE_FULL && pl.rne_packed));
  const char* const kern = packed ? "packed" : "generic";
  const char* const pq = (pl.fused && packed && tile != TILE_PAIR) ? "fused"
                         : (pl.qm == QM_FLOOR_FAST || pl.qm == QM_RNE_WIDE ? "none"
                            : (pl.pq == PQ_MASK_SAT ? "cut_sat" : (pl.pq == PQ_MASK ? "cut" : "none")));
  if (tile == TILE_PAIR) {
    if (buf && buf_len)
      std::snprintf(buf, buf_len, "tile=64x64x%d pair micro=4x8 q=%s pq=%s kernel=%s order=%s load=%s grid=%lldx%lld", BK,
                    kQmName[pl.qm], pq, kern, kOrdName[pl.ord], kLdName[load], (long long)(2 * ((M + 63) / 64)),
                    (long long)((N + 63) / 64));
    return LBA_OK;
  }
  const TileInfo ti = tile_info(tile);
  if (buf && buf_len)
    std::snprintf(buf, buf_len, "tile=%dx%dx%d micro=%dx%d q=%s pq=%s kernel=%s order=%s load=%s grid=%lldx%lld", ti.bm, ti.bn,
                  BK, ti.tm, ti.tn, kQmName[pl.qm], pq, kern, kOrdName[pl.ord], kLdName[load],
                  (long long)((M + ti.bm - 1) / ti.bm), (long long)((N + ti.bn - 1) / ti.bn));
  return LBA_OK;
}

}  // extern "C"

// ------------------------------------------------------------------ lba_gemm_host without allocation
// The device workspace of lba_gemm_host, as an array inside the library image.  In host code the
// name `g_static_workspace` is only a handle for the runtime, not a device address: the address the
// copies and the kernel need comes from cudaGetSymbolAddress, asked once per device.
namespace {

static __device__ __align__(256) unsigned char g_static_workspace[LBA_STATIC_WORKSPACE_BYTES];

constexpr int kMaxDevices = 64;
void* g_static_workspace_addr[kMaxDevices] = {};
std::mutex g_static_workspace_mutex;

// Device address of the array on the current device; looked up on the first call there.
int static_workspace(void** addr) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= kMaxDevices) return cuda_fail(cudaErrorInvalidDevice);
  std::lock_guard<std::mutex> lock(g_static_workspace_mutex);
  if (!g_static_workspace_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_workspace);
    if (e != cudaSuccess) return cuda_fail(e);
    if (!p) return cuda_fail(cudaErrorInvalidSymbol);
    g_static_workspace_addr[dev] = p;
  }
  *addr = g_static_workspace_addr[dev];
  return LBA_OK;
}

}  // namespace

extern "C" int lba_gemm_host_static(const uint8_t* A, const uint8_t* B, const float* scale_a, int scale_a_len,
                                    const float* scale_b, int scale_b_len, const float* bias, int64_t M, int64_t N,
                                    int64_t K, const lba_fmt* prod_fmt, const lba_fmt* acc_fmt, int order, int chunk,
                                    float* out, void* stream) {
  if (M < 0 || N < 0 || K < 0) return LBA_ERR_SHAPE;
  if (scale_a_len < 0 || scale_b_len < 0) return LBA_ERR_SCALE_LEN;
  // refuse before touching the device: sizes are compared in double first so that a huge shape cannot wrap size_t
  const double rough = (double)M * (double)K + (double)N * (double)K + 4.0 * (double)M * (double)N;
  if (rough > (double)LBA_STATIC_WORKSPACE_BYTES) return LBA_ERR_STATIC_LIMIT;
  const size_t need = lba_gemm_host_workspace_bytes(M, N, K, scale_a_len, scale_b_len, bias != nullptr);
  if (need > (size_t)LBA_STATIC_WORKSPACE_BYTES) return LBA_ERR_STATIC_LIMIT;
  void* ws = nullptr;
  const int st = static_workspace(&ws);
  if (st != LBA_OK) return st;
  return lba_gemm_host(A, B, scale_a, scale_a_len, scale_b, scale_b_len, bias, M, N, K, prod_fmt, acc_fmt, order, chunk,
                       out, ws, (size_t)LBA_STATIC_WORKSPACE_BYTES, stream);
}
