/* Sequential binary32 summation of binary32 products under a chosen IEEE rounding
 * direction, done by the host FPU.  Used to pin the oracle's wide-accumulator case:
 * with a 23-bit mantissa and nothing of Eq. 2 reachable, FMAq reduces to one IEEE
 * binary32 addition per step (round-to-nearest-even, or toward zero for floor). */
#include <fenv.h>
#include <stdint.h>

#pragma STDC FENV_ACCESS ON

float fp32_chain(const float* x, const float* w, int64_t K, int toward_zero) {
  int old = fegetround();
  fesetround(toward_zero ? FE_TOWARDZERO : FE_TONEAREST);
  volatile float s = 0.0f;
  for (int64_t i = 0; i < K; ++i) {
    volatile float p = x[i] * w[i]; /* exact: at most 8 significant bits */
    s = s + p;
  }
  fesetround(old);
  return s;
}
