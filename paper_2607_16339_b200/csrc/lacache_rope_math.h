// Rotation and storage-format arithmetic shared by the RoPE-on-write kernel and
// the attention kernel's in-place rotation of a block's queries (Eq. 1): both
// must produce the same bits, so both call these.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cstdint>

namespace lacache {

// 8 consecutive source features starting at element offset elem_off
__device__ __forceinline__ void rope_load8(const void* base, size_t elem_off, bool bf16_in, float (&x)[8]) {
  if (bf16_in) {
    uint4 u = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(base) + elem_off);
    const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 f = __bfloat1622float2(p[i]);
      x[2 * i] = f.x;
      x[2 * i + 1] = f.y;
    }
  } else {
    const float4* p = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(base) + elem_off);
    float4 a = p[0], b = p[1];
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
    x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
  }
}

// (x1, x2) = features (c, c + d/2) rotated by the angle whose cos / sin are given;
// separate roundings on purpose (no fma contraction)
__device__ __forceinline__ void rope_rotate8(const float (&x1)[8], const float (&x2)[8], const float (&cs)[8],
                                             const float (&sn)[8], float (&y1)[8], float (&y2)[8]) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    y1[i] = __fsub_rn(__fmul_rn(x1[i], cs[i]), __fmul_rn(x2[i], sn[i]));
    y2[i] = __fadd_rn(__fmul_rn(x2[i], cs[i]), __fmul_rn(x1[i], sn[i]));
  }
}

// 8 values as split bf16: hi = bf16(y), lo = bf16(y - hi), 16 bytes each
__device__ __forceinline__ void rope_split8(const float (&y)[8], uint4& hi, uint4& lo) {
  __nv_bfloat162* ph = reinterpret_cast<__nv_bfloat162*>(&hi);
  __nv_bfloat162* pl = reinterpret_cast<__nv_bfloat162*>(&lo);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat16 h0 = __float2bfloat16_rn(y[2 * i]);
    __nv_bfloat16 h1 = __float2bfloat16_rn(y[2 * i + 1]);
    __nv_bfloat16 l0 = __float2bfloat16_rn(y[2 * i] - __bfloat162float(h0));
    __nv_bfloat16 l1 = __float2bfloat16_rn(y[2 * i + 1] - __bfloat162float(h1));
    ph[i] = __halves2bfloat162(h0, h1);
    pl[i] = __halves2bfloat162(l0, l1);
  }
}

// 8 values as fp16, saturated to the finite fp16 range (the storage format of V)
__device__ __forceinline__ uint4 rope_half8(const float (&y)[8]) {
  uint4 u;
  __half2* p = reinterpret_cast<__half2*>(&u);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float a = fminf(fmaxf(y[2 * i], -65504.f), 65504.f);
    float b = fminf(fmaxf(y[2 * i + 1], -65504.f), 65504.f);
    p[i] = __floats2half2_rn(a, b);
  }
  return u;
}

}  // namespace lacache
