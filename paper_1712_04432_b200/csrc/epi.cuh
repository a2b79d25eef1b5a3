// Epilogue operations shared by the tensor-core GEMM, the fp32 GEMM and the
// partial-sum reduction: what is done with a finished fp32 sum at (m, n).
#pragma once
#include "kernels.h"

namespace mbd {

__device__ __forceinline__ float bf16_bits_to_f32(uint32_t lo16) { return __uint_as_float(lo16 << 16); }

__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);   // .x = a (low half), .y = b
  return *reinterpret_cast<uint32_t*>(&h);
}

// One element.
__device__ __forceinline__ void epi_apply1(const Epi& e, int64_t m, int64_t n, float acc) {
  if (e.op == EPI_ACT) {
    float v = acc + (e.bias ? e.bias[n] : 0.f);
    if (e.relu) v = fmaxf(v, 0.f);
    if (e.out_bf16) reinterpret_cast<__nv_bfloat16*>(e.out)[m * e.ldo + n] = __float2bfloat16_rn(v);
    else reinterpret_cast<float*>(e.out)[m * e.ldo + n] = v;
  } else if (e.op == EPI_MASK) {
    float v = acc;
    if (e.mask) {
      float x = e.out_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(e.mask)[m * e.ldmask + n])
                           : reinterpret_cast<const float*>(e.mask)[m * e.ldmask + n];
      if (!(x > 0.f)) v = 0.f;
    }
    if (e.out_bf16) reinterpret_cast<__nv_bfloat16*>(e.out)[m * e.ldo + n] = __float2bfloat16_rn(v);
    else reinterpret_cast<float*>(e.out)[m * e.ldo + n] = v;
  } else {  // EPI_SGD
    if (e.out_bf16 && e.master) {
      float* w32 = e.master + m * e.ldo + n;
      const float v = fmaf(e.scale, acc, *w32);
      *w32 = v;
      reinterpret_cast<__nv_bfloat16*>(e.out)[m * e.ldo + n] = __float2bfloat16_rn(v);
    } else if (e.out_bf16) {
      __nv_bfloat16* w = reinterpret_cast<__nv_bfloat16*>(e.out) + m * e.ldo + n;
      *w = __float2bfloat16_rn(fmaf(e.scale, acc, __bfloat162float(*w)));
    } else {
      float* w = reinterpret_cast<float*>(e.out) + m * e.ldo + n;
      *w = fmaf(e.scale, acc, *w);
    }
  }
}

// Eight consecutive columns n0..n0+7 of row m; n0 and the leading dimensions are
// multiples of 8 and the bases 16-byte aligned (checked on the host).
__device__ __forceinline__ void epi_apply8(const Epi& e, int64_t m, int64_t n0, float* v) {
  if (e.op == EPI_ACT) {
    if (e.bias) {
      const float4 b0 = *reinterpret_cast<const float4*>(e.bias + n0);
      const float4 b1 = *reinterpret_cast<const float4*>(e.bias + n0 + 4);
      v[0] += b0.x; v[1] += b0.y; v[2] += b0.z; v[3] += b0.w;
      v[4] += b1.x; v[5] += b1.y; v[6] += b1.z; v[7] += b1.w;
    }
    if (e.relu) {
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = fmaxf(v[i], 0.f);
    }
  } else if (e.op == EPI_MASK) {
    if (e.mask) {
      if (e.out_bf16) {
        const uint4 q = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(e.mask) + m * e.ldmask + n0);
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (!(bf16_bits_to_f32(w[i] & 0xFFFFu) > 0.f)) v[2 * i] = 0.f;
          if (!(bf16_bits_to_f32(w[i] >> 16) > 0.f)) v[2 * i + 1] = 0.f;
        }
      } else {
        const float* x = reinterpret_cast<const float*>(e.mask) + m * e.ldmask + n0;
        const float4 a = *reinterpret_cast<const float4*>(x), b = *reinterpret_cast<const float4*>(x + 4);
        const float xs[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) if (!(xs[i] > 0.f)) v[i] = 0.f;
      }
    }
  } else {  // EPI_SGD: read-modify-write of the weights
    if (e.out_bf16 && e.master) {   // fp32 master weights: update the master, the bf16 copy is its rounding
      float* x = e.master + m * e.ldo + n0;
      const float4 a = *reinterpret_cast<const float4*>(x), b = *reinterpret_cast<const float4*>(x + 4);
      const float xs[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = fmaf(e.scale, v[i], xs[i]);
      *reinterpret_cast<float4*>(x) = make_float4(v[0], v[1], v[2], v[3]);
      *reinterpret_cast<float4*>(x + 4) = make_float4(v[4], v[5], v[6], v[7]);
    } else if (e.out_bf16) {
      uint4* p = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(e.out) + m * e.ldo + n0);
      const uint4 q = *p;
      const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        v[2 * i] = fmaf(e.scale, v[2 * i], bf16_bits_to_f32(w[i] & 0xFFFFu));
        v[2 * i + 1] = fmaf(e.scale, v[2 * i + 1], bf16_bits_to_f32(w[i] >> 16));
      }
    } else {
      float* x = reinterpret_cast<float*>(e.out) + m * e.ldo + n0;
      const float4 a = *reinterpret_cast<const float4*>(x), b = *reinterpret_cast<const float4*>(x + 4);
      const float xs[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = fmaf(e.scale, v[i], xs[i]);
    }
  }
  if (e.out_bf16) {
    uint4 o;
    o.x = pack_bf16x2(v[0], v[1]); o.y = pack_bf16x2(v[2], v[3]);
    o.z = pack_bf16x2(v[4], v[5]); o.w = pack_bf16x2(v[6], v[7]);
    *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(e.out) + m * e.ldo + n0) = o;
  } else {
    float* x = reinterpret_cast<float*>(e.out) + m * e.ldo + n0;
    *reinterpret_cast<float4*>(x) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(x + 4) = make_float4(v[4], v[5], v[6], v[7]);
  }
}

}  // namespace mbd
