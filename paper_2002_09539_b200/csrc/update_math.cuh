// The arithmetic of one parameter update, shared by the stand-alone fused
// update kernel and by the weight-gradient GEMM's fused epilogue so that both
// produce the same bits.
//
//   Eq. 3 with the local Nesterov buffer:  u <- mu u + g ;  x <- x - gamma (g + mu u)
//   Eq. 3 plain:                            x <- x - gamma g
//   Eq. 4 (sync steps):                     x <- x - alpha (x - z)
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

namespace olsgd {

template <bool MOM, bool SYNC>
__device__ __forceinline__ void update_scalar(float& x, float& u, float g, float z, float gamma,
                                              float mu, float alpha) {
  if (MOM) {
    u = fmaf(mu, u, g);
    x = fmaf(-gamma, fmaf(mu, u, g), x);
  } else {
    x = fmaf(-gamma, g, x);
  }
  if (SYNC) x = fmaf(-alpha, x - z, x);
}

template <bool MOM, bool SYNC>
__device__ __forceinline__ void update4(float4& x, float4& u, const float4& g, const float4& z,
                                        float gamma, float mu, float alpha) {
  update_scalar<MOM, SYNC>(x.x, u.x, g.x, z.x, gamma, mu, alpha);
  update_scalar<MOM, SYNC>(x.y, u.y, g.y, z.y, gamma, mu, alpha);
  update_scalar<MOM, SYNC>(x.z, u.z, g.z, z.z, gamma, mu, alpha);
  update_scalar<MOM, SYNC>(x.w, u.w, g.w, z.w, gamma, mu, alpha);
}

// The same arithmetic with the two switches taken at run time (kernels in which the update is
// a small tail, not the main loop).
__device__ __forceinline__ void update_scalar_rt(float& x, float& u, float g, float z, float gamma,
                                                 float mu, float alpha, bool mom, bool sync) {
  if (mom) {
    if (sync) update_scalar<true, true>(x, u, g, z, gamma, mu, alpha);
    else update_scalar<true, false>(x, u, g, z, gamma, mu, alpha);
  } else {
    if (sync) update_scalar<false, true>(x, u, g, z, gamma, mu, alpha);
    else update_scalar<false, false>(x, u, g, z, gamma, mu, alpha);
  }
}

// four floats -> four bf16 (round to nearest even), packed in 8 bytes
__device__ __forceinline__ uint2 pack_bf16x4(const float4& v) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
  __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 pk;
  pk.x = *reinterpret_cast<uint32_t*>(&lo);
  pk.y = *reinterpret_cast<uint32_t*>(&hi);
  return pk;
}

}  // namespace olsgd
