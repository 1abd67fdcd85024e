// Rotary arithmetic shared by the kernels that re-encode keys (Sec. 4.3 / 4.4).  A rotated element is
// defined as fp32 products and sums without fused multiply-add followed by one round-to-nearest-even
// to bf16, so that an encoded key is a reproducible code.
#pragma once
#include "kvmem_internal.cuh"

namespace kvmem {

// 8 (lo, hi) pairs -> rotated pairs; t[w] = (cos, sin, cos, sin) of pairs 2w and 2w + 1.  sgn = +1 forward, -1 inverse.
__device__ __forceinline__ void rotate8_cs(const uint4& lo_in, const uint4& hi_in, const float4 (&t4)[4], float sgn,
                                           uint4& lo_out, uint4& hi_out) {
    const uint32_t li[4] = {lo_in.x, lo_in.y, lo_in.z, lo_in.w}, hi[4] = {hi_in.x, hi_in.y, hi_in.z, hi_in.w};
    uint32_t lo_o[4], hi_o[4];
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        const float4 t = t4[w];
        const float a0 = __uint_as_float(li[w] << 16), a1 = __uint_as_float(li[w] & 0xffff0000u);
        const float b0 = __uint_as_float(hi[w] << 16), b1 = __uint_as_float(hi[w] & 0xffff0000u);
        const float s0 = sgn * t.y, s1 = sgn * t.w;
        const float l0 = __fsub_rn(__fmul_rn(a0, t.x), __fmul_rn(b0, s0)), h0 = __fadd_rn(__fmul_rn(b0, t.x), __fmul_rn(a0, s0));
        const float l1 = __fsub_rn(__fmul_rn(a1, t.z), __fmul_rn(b1, s1)), h1 = __fadd_rn(__fmul_rn(b1, t.z), __fmul_rn(a1, s1));
        const __nv_bfloat162 lp = __floats2bfloat162_rn(l0, l1), hp = __floats2bfloat162_rn(h0, h1);
        lo_o[w] = *reinterpret_cast<const uint32_t*>(&lp);
        hi_o[w] = *reinterpret_cast<const uint32_t*>(&hp);
    }
    lo_out = make_uint4(lo_o[0], lo_o[1], lo_o[2], lo_o[3]);
    hi_out = make_uint4(hi_o[0], hi_o[1], hi_o[2], hi_o[3]);
}

// the same with the table row in global memory: cs points at the (cos, sin) of the first of the 8 pairs
__device__ __forceinline__ void rotate8(const uint4& lo_in, const uint4& hi_in, const float2* __restrict__ cs, float sgn,
                                        uint4& lo_out, uint4& hi_out) {
    const float4* cs4 = reinterpret_cast<const float4*>(cs);
    float4 t4[4];
#pragma unroll
    for (int w = 0; w < 4; ++w) t4[w] = __ldg(cs4 + w);
    rotate8_cs(lo_in, hi_in, t4, sgn, lo_out, hi_out);
}

}  // namespace kvmem
