// Device-side sketch generator "Gaussian v1": S[i][j] = z(seed, kind, i, j) * fp32(1/sqrt(r)).
//
// The paper only names its random-projection compressor (experimental setup of Section 5), so the
// generator is this library's own frozen format.  One Philox4x32-10 call with key = seed and counter
// (i, j/4, 0, kind) yields the four columns 4q..4q+3 of row i: words (x0, x1) make columns 4q, 4q+1
// and (x2, x3) make 4q+2, 4q+3 through a Box-Muller transform.  Every floating-point step is one
// binary32 add, subtract or multiply rounded to nearest even (the _rn intrinsics are never contracted
// into FMAs); reciprocal and square root are fixed Newton iterations made of those steps, so any
// IEEE-754 machine that performs the same steps gets the same bits.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>

namespace acx {

struct SketchParams {
  uint32_t key0, key1;  // seed low / high word
  uint32_t kind;        // counter word 3
  float scale;          // fp32(1/sqrt(r)), computed on the host in double and rounded once
  // Philox round keys: key + round * Weyl increment.  The same for every element, so the host fills them
  // once (fill_round_keys) and the kernels read them as constants instead of re-deriving them per call.
  uint32_t rk0[10], rk1[10];
};

__host__ __device__ inline void fill_round_keys(SketchParams& sp) {
  uint32_t k0 = sp.key0, k1 = sp.key1;
  for (int round = 0; round < 10; ++round) {
    sp.rk0[round] = k0;
    sp.rk1[round] = k1;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
}

__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, const SketchParams& sp) {
  constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;  // round multipliers
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint64_t p0 = uint64_t(M0) * c0, p1 = uint64_t(M1) * c2;  // one widening multiply each
    const uint32_t hi0 = uint32_t(p0 >> 32), lo0 = uint32_t(p0);
    const uint32_t hi1 = uint32_t(p1 >> 32), lo1 = uint32_t(p1);
    c0 = hi1 ^ c1 ^ sp.rk0[round];
    c1 = lo1;
    c2 = hi0 ^ c3 ^ sp.rk1[round];
    c3 = lo0;
  }
  return make_uint4(c0, c1, c2, c3);
}

// 1/d for d in [1.70, 2.42]: linear start, three Newton steps y <- y*(2 - d*y).
__device__ __forceinline__ float newton_reciprocal(float d) {
  float y = __fsub_rn(0.99259f, __fmul_rn(0.24264f, d));
#pragma unroll
  for (int it = 0; it < 3; ++it) y = __fmul_rn(y, __fsub_rn(2.0f, __fmul_rn(d, y)));
  return y;
}

// 1/sqrt(w) for positive normal w: bit-shift start, three Newton steps y <- y*(1.5 - (0.5*w)*(y*y)).
__device__ __forceinline__ float newton_rsqrt(float w) {
  float y = __uint_as_float(0x5F3759DFu - (__float_as_uint(w) >> 1));
  const float h = __fmul_rn(0.5f, w);
#pragma unroll
  for (int it = 0; it < 3; ++it) y = __fmul_rn(y, __fsub_rn(1.5f, __fmul_rn(h, __fmul_rn(y, y))));
  return y;
}

// Two words -> two independent N(0,1) values: radius from xa, angle from xb.  Straight-line code:
// only +, -, * (each rounded once) and integer<->float bit moves; no division, sqrt, conversion or branch.
__device__ __forceinline__ void gaussian_pair(uint32_t xa, uint32_t xb, float& z0, float& z1) {
  // u = (2n+1) * 2^-24 in (0, 1) with n = xa >> 9: the float 1.n minus (1 - 2^-24), exact
  const float u = __fsub_rn(__uint_as_float(0x3F800000u | (xa >> 9)), __uint_as_float(0x3F7FFFFFu));
  // ln u = e*ln2 + ln(mant), mant in (0.7071, 1.4143), ln(mant) = 2 atanh(t), t = (mant-1)/(mant+1)
  const uint32_t bits = __float_as_uint(u);
  const uint32_t frac = bits & 0x7FFFFFu;
  const bool upper = frac > 0x3504F3u;  // mantissa above sqrt(2)
  const float mant = __uint_as_float((upper ? 0x3F000000u : 0x3F800000u) | frac);
  const uint32_t e_plus_127 = (bits >> 23) + (upper ? 1u : 0u);
  const float e_f = __fsub_rn(__uint_as_float((0x4B400000u - 127u) + e_plus_127), 12582912.0f);  // exact
  const float t = __fmul_rn(__fsub_rn(mant, 1.0f), newton_reciprocal(__fadd_rn(mant, 1.0f)));
  const float t2 = __fmul_rn(t, t);
  float p = float(1.0 / 11.0);
  p = __fadd_rn(__fmul_rn(p, t2), float(1.0 / 9.0));
  p = __fadd_rn(__fmul_rn(p, t2), float(1.0 / 7.0));
  p = __fadd_rn(__fmul_rn(p, t2), float(1.0 / 5.0));
  p = __fadd_rn(__fmul_rn(p, t2), float(1.0 / 3.0));
  p = __fadd_rn(__fmul_rn(p, t2), 1.0f);
  const float ln_mant = __fmul_rn(__fmul_rn(2.0f, t), p);
  const float ln_u = __fadd_rn(__fmul_rn(e_f, float(0.6931471805599453)), ln_mant);
  const float w = __fmul_rn(-2.0f, ln_u);
  const float rho = __fmul_rn(w, newton_rsqrt(w));

  // theta = (oct + a) * pi/4; odd octants measure the offset from their upper end (a <- 1 - a)
  const uint32_t oct = xb >> 29;
  float a = __fsub_rn(__uint_as_float(0x3F800000u | ((xb >> 6) & 0x7FFFFFu)), 1.0f);
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
  const uint4 x = philox4x32_10(i, q, 0u, sp.kind, sp);
  float4 z;
  gaussian_pair(x.x, x.y, z.x, z.y);
  gaussian_pair(x.z, x.w, z.z, z.w);
  z.x = __fmul_rn(z.x, sp.scale);
  z.y = __fmul_rn(z.y, sp.scale);
  z.z = __fmul_rn(z.z, sp.scale);
  z.w = __fmul_rn(z.w, sp.scale);
  return z;
}

// One thread's share of S^T in bfloat16 (r x d_in, row j = column j of S): rows 4q .. 4q+3, columns 2*ip and 2*ip + 1
// (d_in is even).  Consecutive ip in a warp make each row's stores contiguous.
__device__ __forceinline__ void sketch_transposed_store(const SketchParams& sp, __nv_bfloat16* St, int64_t d_in, uint32_t ip,
                                                        uint32_t q) {
  const float4 za = sketch_quad(sp, 2u * ip, q), zb = sketch_quad(sp, 2u * ip + 1u, q);
  __nv_bfloat16* dst = St + int64_t(4u * q) * d_in + 2u * ip;
  *reinterpret_cast<__nv_bfloat162*>(dst) = __floats2bfloat162_rn(za.x, zb.x);
  *reinterpret_cast<__nv_bfloat162*>(dst + d_in) = __floats2bfloat162_rn(za.y, zb.y);
  *reinterpret_cast<__nv_bfloat162*>(dst + 2 * d_in) = __floats2bfloat162_rn(za.z, zb.z);
  *reinterpret_cast<__nv_bfloat162*>(dst + 3 * d_in) = __floats2bfloat162_rn(za.w, zb.w);
}

// The value a bf16 data path multiplies with: round to nearest even, back to binary32.
__device__ __forceinline__ float round_through_bf16(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

}  // namespace acx
