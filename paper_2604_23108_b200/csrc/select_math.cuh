// Float32 arithmetic of the selection contract (Sec. 3.2, Eq. 2-6): the exponential and the
// sigmoid whose results decide indices.  Every operation is an explicit round-to-nearest
// intrinsic, so no compiler option can contract a multiply and an add into one rounding.
//   exp_s(z) for z <= 0:  zc = max(z, -100); n = rint(zc * 0x1.715476p+0);
//            r = zc - n * 0x1.62e4p-1;  r = r - n * 0x1.7f7d1cp-20;
//            p = Horner (separate multiply, add) with 1/7!, 1/6!, ..., 1/2!, 1, 1 rounded to
//            float32;  result p * 2^n;  z < -87 gives +0
//   sig_s(z) e = exp_s(-|z|);  z >= 0 ? 1/(1+e) : e/(1+e)
#pragma once

namespace mohge {

__device__ __forceinline__ float exp_s(float z) {
  const float zc = fmaxf(z, -100.0f);
  const float n = rintf(__fmul_rn(zc, 0x1.715476p+0f));
  float r = __fsub_rn(zc, __fmul_rn(n, 0x1.62e4p-1f));
  r = __fsub_rn(r, __fmul_rn(n, 0x1.7f7d1cp-20f));
  float p = 0x1.a01a02p-13f;
  p = __fadd_rn(__fmul_rn(p, r), 0x1.6c16c2p-10f);
  p = __fadd_rn(__fmul_rn(p, r), 0x1.111112p-7f);
  p = __fadd_rn(__fmul_rn(p, r), 0x1.555556p-5f);
  p = __fadd_rn(__fmul_rn(p, r), 0x1.555556p-3f);
  p = __fadd_rn(__fmul_rn(p, r), 0x1p-1f);
  p = __fadd_rn(__fmul_rn(p, r), 1.0f);
  p = __fadd_rn(__fmul_rn(p, r), 1.0f);
  int ni = (int)n;
  ni = ni < -126 ? -126 : (ni > 0 ? 0 : ni);
  const float scale = __int_as_float((ni + 127) << 23);
  const float out = __fmul_rn(p, scale);
  return z < -87.0f ? 0.0f : out;
}

__device__ __forceinline__ float sig_s(float z) {
  const float e = exp_s(-fabsf(z));
  const float den = __fadd_rn(1.0f, e);
  return z >= 0.0f ? __fdiv_rn(1.0f, den) : __fdiv_rn(e, den);
}

}  // namespace mohge
