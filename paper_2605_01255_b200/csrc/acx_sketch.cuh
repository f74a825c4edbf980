// Device-side sketch generator "Gaussian v1": S[i][j] = z(seed, kind, i, j) * fp32(1/sqrt(r)).
//
// The paper only names its random-projection compressor (experimental setup of Section 5), so the
// generator is this library's own frozen format.  One Philox4x32-10 call with key = seed and counter
// (i, j/4, 0, kind) yields the four columns 4q..4q+3 of row i: words (x0, x1) make columns 4q, 4q+1
// and (x2, x3) make 4q+2, 4q+3 through a Box-Muller transform.  Every floating-point step is one
// correctly rounded binary32 operation (the _rn intrinsics are never contracted into FMAs), so any
// IEEE-754 machine that performs the same steps gets the same bits.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>

namespace acx {

struct SketchParams {
  uint32_t key0, key1;  // seed low / high word
  uint32_t kind;        // counter word 3
  float scale;          // fp32(1/sqrt(r)), computed on the host in double and rounded once
};

__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               uint32_t k0, uint32_t k1) {
  constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;  // round multipliers
  constexpr uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;  // Weyl key increments
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
    const uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
    c0 = hi1 ^ c1 ^ k0;
    c1 = lo1;
    c2 = hi0 ^ c3 ^ k1;
    c3 = lo0;
    k0 += W0;
    k1 += W1;
  }
  return make_uint4(c0, c1, c2, c3);
}

// Two words -> two independent N(0,1) values: radius from xa, angle from xb.
__device__ __forceinline__ void gaussian_pair(uint32_t xa, uint32_t xb, float& z0, float& z1) {
  // u = ((xa >> 9) + 0.5) * 2^-23 in (0, 1), exact
  const float u = __fmul_rn(__fadd_rn(__uint2float_rn(xa >> 9), 0.5f), 1.1920928955078125e-07f);
  // ln u = e*ln2 + ln(mant), mant in (0.7071, 1.4143), ln(mant) = 2 atanh(t), t = (mant-1)/(mant+1)
  const uint32_t bits = __float_as_uint(u);
  const uint32_t frac = bits & 0x7FFFFFu;
  const bool upper = frac > 0x3504F3u;  // mantissa above sqrt(2)
  const int e = int(bits >> 23) - 127 + (upper ? 1 : 0);
  const float mant = __uint_as_float((upper ? 0x3F000000u : 0x3F800000u) | frac);
  const float t = __fdiv_rn(__fsub_rn(mant, 1.0f), __fadd_rn(mant, 1.0f));
  const float t2 = __fmul_rn(t, t);
  float p = float(1.0 / 11.0);
  p = __fadd_rn(__fmul_rn(p, t2), float(1.0 / 9.0));
  p = __fadd_rn(__fmul_rn(p, t2), float(1.0 / 7.0));
  p = __fadd_rn(__fmul_rn(p, t2), float(1.0 / 5.0));
  p = __fadd_rn(__fmul_rn(p, t2), float(1.0 / 3.0));
  p = __fadd_rn(__fmul_rn(p, t2), 1.0f);
  const float ln_mant = __fmul_rn(__fmul_rn(2.0f, t), p);
  const float ln_u = __fadd_rn(__fmul_rn(__int2float_rn(e), float(0.6931471805599453)), ln_mant);
  const float rho = __fsqrt_rn(__fmul_rn(-2.0f, ln_u));

  // theta = (oct + a) * pi/4; odd octants measure the offset from their upper end (a <- 1 - a)
  const uint32_t oct = xb >> 29;
  float a = __fmul_rn(__uint2float_rn((xb >> 5) & 0xFFFFFFu), 5.9604644775390625e-08f);
  if (oct & 1u) a = __fsub_rn(1.0f, a);
  const float y = __fmul_rn(a, float(0.7853981633974483));
  const float y2 = __fmul_rn(y, y);
  float s = float(1.0 / 362880.0);
  s = __fadd_rn(__fmul_rn(s, y2), float(-1.0 / 5040.0));
  s = __fadd_rn(__fmul_rn(s, y2), float(1.0 / 120.0));
  s = __fadd_rn(__fmul_rn(s, y2), float(-1.0 / 6.0));
  s = __fadd_rn(__fmul_rn(s, y2), 1.0f);
  s = __fmul_rn(s, y);
  float c = float(-1.0 / 3628800.0);
  c = __fadd_rn(__fmul_rn(c, y2), float(1.0 / 40320.0));
  c = __fadd_rn(__fmul_rn(c, y2), float(-1.0 / 720.0));
  c = __fadd_rn(__fmul_rn(c, y2), float(1.0 / 24.0));
  c = __fadd_rn(__fmul_rn(c, y2), -0.5f);
  c = __fadd_rn(__fmul_rn(c, y2), 1.0f);
  const bool swap = ((oct + 1u) & 2u) != 0u;     // octants 1, 2, 5, 6
  float cos_t = swap ? s : c;
  float sin_t = swap ? c : s;
  if ((oct + 2u) & 4u) cos_t = -cos_t;           // octants 2..5: cos < 0
  if (oct & 4u) sin_t = -sin_t;                  // octants 4..7: sin < 0
  z0 = __fmul_rn(rho, cos_t);
  z1 = __fmul_rn(rho, sin_t);
}

// S[i][4q .. 4q+3] in binary32.
__device__ __forceinline__ float4 sketch_quad(const SketchParams& sp, uint32_t i, uint32_t q) {
  const uint4 x = philox4x32_10(i, q, 0u, sp.kind, sp.key0, sp.key1);
  float4 z;
  gaussian_pair(x.x, x.y, z.x, z.y);
  gaussian_pair(x.z, x.w, z.z, z.w);
  z.x = __fmul_rn(z.x, sp.scale);
  z.y = __fmul_rn(z.y, sp.scale);
  z.z = __fmul_rn(z.z, sp.scale);
  z.w = __fmul_rn(z.w, sp.scale);
  return z;
}

// The value a bf16 data path multiplies with: round to nearest even, back to binary32.
__device__ __forceinline__ float round_through_bf16(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

}  // namespace acx
