// Pieces shared by the tensor-core attention kernels.
#pragma once
#include "tc_common.cuh"

namespace tc {

// 2^x on the FMA and integer pipes, for the share of a softmax tile's exponentials that the 16-lane
// special-function unit would otherwise make wait (x <= 8; below -125 the result is 2^-125 instead of 0):
// x + 1.5 * 2^23 leaves round(x) in the low mantissa bits, a degree-3 polynomial gives 2^f on
// [-0.5, 0.5] (relative error 7.5e-5, far below the bf16 rounding of the probabilities it feeds), and the
// integer part is added to the exponent field.
__device__ __forceinline__ float ex2_poly(float x) {
  x = fmaxf(x, -125.0f);
  const float y = x + 12582912.0f;
  const float f = x - (y - 12582912.0f);
  float p = fmaf(f, 0.055171624f, 0.24261113f);
  p = fmaf(p, f, 0.69326097f);
  p = fmaf(p, f, 0.99992806f);
  return __int_as_float(__float_as_int(p) + (__float_as_int(y) << 23));
}

}  // namespace tc
