// The quantizer of the pack, switch and retarget kernels, in IEEE double (Section IV-A: uniform quantization;
// group-wise asymmetric with fp16 scale and zero):
//   scale = fp16((max - min) / (2^b - 1))  (1.0 if that rounds to 0),  zero = fp16(min),
//   code  = clamp(rint((w - zero) / scale), 0, 2^b - 1)   (true division, ties to even).
#pragma once
#include "common.cuh"

namespace dyn {

__device__ __forceinline__ double bf16_to_double(__nv_bfloat16 v) { return (double)__bfloat162float(v); }

__device__ __forceinline__ void group_params(double lo, double hi, int bits, __half& s_h, __half& m_h, double& s,
                                             double& m) {
    const double L = (double)((1 << bits) - 1);
    s_h = __double2half(__ddiv_rn(__dsub_rn(hi, lo), L));
    if (__half2float(s_h) == 0.0f) s_h = __float2half(1.0f);
    m_h = __double2half(lo);
    s = (double)__half2float(s_h);
    m = (double)__half2float(m_h);
}

__device__ __forceinline__ int quantize_code(double w, double s, double m, int bits) {
    double t = rint(__ddiv_rn(__dsub_rn(w, m), s));
    const double L = (double)((1 << bits) - 1);
    t = t < 0.0 ? 0.0 : (t > L ? L : t);
    return (int)t;
}

}  // namespace dyn
