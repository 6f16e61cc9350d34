// Activation quantisation shared by the decode kernels (sm_100a): fp16 activations become 16-bit fixed point
// per (batch row, 128-channel group), split in two signed bytes, so that the 4-bit codes can go to the int8
// tensor-core MMA as they lie in memory.
#pragma once
#include <cuda_fp16.h>
#include <stdint.h>

namespace uniql {

// Sixteen consecutive lanes hold the 128 activations of one (batch row, group), eight each (`in`): 16-bit fixed
// point against the group's maximum, x_i = rint(x * 2^e) = 256 * hi + lo with both bytes signed.  Returns this
// lane's bytes in the order the nibbles leave a weight word (even codes first), the group's integer sum and
// 2^-e (NaN when the group holds a non-finite activation).  Every lane of the warp must call it (shuffles over the sixteen lanes).
__device__ inline void quantise16(const uint4& in, uint2& hi2, uint2& lo2, int& isum_out, float& inv_scale_out) {
  const __half2* h2 = reinterpret_cast<const __half2*>(&in);
  float f[8];
  // the group's maximum is taken on the magnitude bits as integers: Inf and NaN compare above every finite value,
  // where a floating-point maximum would drop a NaN
  uint32_t amax_bits = 0u;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 v = __half22float2(h2[i]);
    f[2 * i] = v.x; f[2 * i + 1] = v.y;
    amax_bits = max(amax_bits, max(__float_as_uint(v.x) & 0x7fffffffu, __float_as_uint(v.y) & 0x7fffffffu));
  }
#pragma unroll
  for (int o2 = 8; o2 >= 1; o2 >>= 1) amax_bits = max(amax_bits, __shfl_xor_sync(0xffffffffu, amax_bits, o2));
  const float amax = __uint_as_float(amax_bits);
  const bool finite = amax_bits < 0x7f800000u;
  int e = 0;
  if (amax_bits != 0u && finite) {
    e = 14 - ((int)(amax_bits >> 23) - 127);
    if (amax * __uint_as_float((uint32_t)(127 + e) << 23) > 32639.f) --e;     // keep the high byte of x_i + 128 signed
  }
  // a group that holds an Inf or a NaN gets a NaN factor: every output that uses the group becomes NaN
  const float scale = __uint_as_float((uint32_t)(127 + e) << 23);
  const float inv_scale = finite ? __uint_as_float((uint32_t)(127 - e) << 23) : __uint_as_float(0x7fc00000u);
  // t_k = x_i + 128 through the float adder: x * 2^e + (1.5 * 2^23 + 128) is rounded to an integer (nearest even,
  // as rint) whose low mantissa bits are t_k.  Byte 1 of t_k is hi, byte 0 of t_k xor 0x80 is lo; the bytes are
  // gathered with byte permutes.
  int tk[8];
  int isum = -8 * 128;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    tk[k] = __float_as_int(fmaf(f[k], scale, 12582912.f + 128.f)) - 0x4B400000;
    isum += tk[k];
  }
  const uint32_t hi_e = __byte_perm(__byte_perm(tk[0], tk[2], 0x0051), __byte_perm(tk[4], tk[6], 0x0051), 0x5410);
  const uint32_t hi_o = __byte_perm(__byte_perm(tk[1], tk[3], 0x0051), __byte_perm(tk[5], tk[7], 0x0051), 0x5410);
  const uint32_t lo_e = __byte_perm(__byte_perm(tk[0], tk[2], 0x0040), __byte_perm(tk[4], tk[6], 0x0040), 0x5410) ^ 0x80808080u;
  const uint32_t lo_o = __byte_perm(__byte_perm(tk[1], tk[3], 0x0040), __byte_perm(tk[5], tk[7], 0x0040), 0x5410) ^ 0x80808080u;
#pragma unroll
  for (int o2 = 8; o2 >= 1; o2 >>= 1) isum += __shfl_xor_sync(0xffffffffu, isum, o2);
  hi2 = make_uint2(hi_e, hi_o);
  lo2 = make_uint2(lo_e, lo_o);
  isum_out = isum;
  inv_scale_out = inv_scale;
}

}  // namespace uniql
