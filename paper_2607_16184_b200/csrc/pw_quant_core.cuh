// The group quantizer shared by the kernels that build pages: codes of one row-group of 128 weights, held as
// four slices of 32 by four neighbouring lanes.  fp32, one rounding per operation, in the order the page
// format defines: scale = fp16((hi - lo) / L) (1.0 if hi == lo, 2^-24 if it rounds to zero), zero-point = lo,
// code = clamp(rint((w - lo) * (1 / scale)), 0, L); a minimum of -0 is stored as +0.
#pragma once

#include <cuda_fp16.h>
#include <stdint.h>

namespace pw {

// v: my 32 values; h16: the same as packed halves when the source was 16-bit (FROM_HALVES).  Returns my 32
// codes, the group's scale and its minimum (the zero-point), identical on the four lanes of the row-group.
// CLAMP = false leaves the codes as rint((w - lo) / scale) without the upper clamp (never negative; a huge
// quotient saturates at INT_MAX, NaN gives 0): for a caller whose packing saturates (pack_slice_sat).
template <bool FROM_HALVES, bool CLAMP = true>
__device__ __forceinline__ void group_quantize(const float (&v)[32], const __half2* h16, int L, int (&code)[32],
                                               __half& sh, float& lo_out) {
  // minimum and maximum of my 32 values (of fp16 sources taken on the packed halves: half as many operations,
  // and exact like the fp32 ones)
  float lo, hi;
  if constexpr (FROM_HALVES) {
    __half2 lo2 = h16[0], hi2 = h16[0];
#pragma unroll
    for (int i = 1; i < 16; ++i) {
      lo2 = __hmin2(lo2, h16[i]);
      hi2 = __hmax2(hi2, h16[i]);
    }
    const float2 lf = __half22float2(lo2), hf = __half22float2(hi2);
    lo = fminf(lf.x, lf.y);
    hi = fmaxf(hf.x, hf.y);
  } else {
    lo = v[0];
    hi = v[0];
#pragma unroll
    for (int i = 1; i < 32; ++i) {
      lo = fminf(lo, v[i]);
      hi = fmaxf(hi, v[i]);
    }
  }
#pragma unroll
  for (int d = 1; d <= 2; d <<= 1) {
    lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, d));
    hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, d));
  }
  if (lo == 0.0f) lo = 0.0f;  // store -0 as +0
  const float rng = __fsub_rn(hi, lo);
  if (rng == 0.0f) {
    sh = __ushort_as_half((unsigned short)0x3c00);
  } else {
    sh = __float2half_rn(__fdiv_rn(rng, (float)L));
    if ((__half_as_ushort(sh) & 0x7fff) == 0) sh = __ushort_as_half((unsigned short)0x0001);
  }
  const float rinv = __fdiv_rn(1.0f, __half2float(sh));
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    // round half to even and convert in one step (the product is never negative; a huge one saturates), then
    // clamp: the same code as clamp(rint(x), 0, L)
    if constexpr (CLAMP) {
      const uint32_t c = __float2uint_rn(__fmul_rn(__fsub_rn(v[i], lo), rinv));
      code[i] = (int)(c < (uint32_t)L ? c : (uint32_t)L);
    } else {
      code[i] = __float2int_rn(__fmul_rn(__fsub_rn(v[i], lo), rinv));
    }
  }
  lo_out = lo;
}

}  // namespace pw
