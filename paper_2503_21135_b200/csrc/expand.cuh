// Code expansion shared by the FFN kernels: packed codes of one atom -> fp16 A-operand register pairs.
// MAGIC = 0          : a field masked in place is the fp16 subnormal q * 2^(o-24)   (one AND per pair)
// MAGIC = 0x64006400 : the pair is (1024 + q * 2^o) in both halves                  (one AND-OR per pair)
// See layout.cuh for the field positions and the matching power-of-two scale of the activations.
#pragma once
#include "common.cuh"
#include "layout.cuh"

namespace dyn {

// Packed codes of one atom for one half chunk (64 k = 4 MMA steps), per lane, plus the shifted copies.
template <int BITS>
struct Codes;
template <>
struct Codes<2> { uint32_t w[2], ws[2]; };
template <>
struct Codes<3> { uint32_t w[2], ws[2], t0[2], t1[2]; };
template <>
struct Codes<4> { uint32_t w[4], ws[4]; };
template <>
struct Codes<8> { uint32_t w[8]; };
template <>
struct Codes<6> { uint32_t w[4], ws[4], t[2][4]; };  // low-nibble words and their >> 8; four copies of the high-bit words

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}

__device__ __forceinline__ uint32_t rotr32(uint32_t v, int n) { return __funnelshift_r(v, v, n); }

template <int BITS>
__device__ __forceinline__ void load_codes(Codes<BITS>& c, const uint8_t* atom, int lane, int half) {
    if constexpr (BITS == 4) {
        const uint4 v = *reinterpret_cast<const uint4*>(atom + half * 512 + lane * 16);
        c.w[0] = v.x; c.w[1] = v.y; c.w[2] = v.z; c.w[3] = v.w;
#pragma unroll
        for (int i = 0; i < 4; ++i) c.ws[i] = c.w[i] >> 8;
    } else if constexpr (BITS == 8) {
        const uint4 v0 = *reinterpret_cast<const uint4*>(atom + (2 * half) * 512 + lane * 16);
        const uint4 v1 = *reinterpret_cast<const uint4*>(atom + (2 * half + 1) * 512 + lane * 16);
        c.w[0] = v0.x; c.w[1] = v0.y; c.w[2] = v0.z; c.w[3] = v0.w;
        c.w[4] = v1.x; c.w[5] = v1.y; c.w[6] = v1.z; c.w[7] = v1.w;
    } else if constexpr (BITS == 6) {
        const uint4 v = *reinterpret_cast<const uint4*>(atom + half * 512 + lane * 16);
        c.w[0] = v.x; c.w[1] = v.y; c.w[2] = v.z; c.w[3] = v.w;
#pragma unroll
        for (int i = 0; i < 4; ++i) c.ws[i] = c.w[i] >> 8;
        const uint2 hb = *reinterpret_cast<const uint2*>(atom + 1024 + lane * 16 + half * 8);
        const uint32_t hw[2] = {hb.x, hb.y};
#pragma unroll
        for (int rh = 0; rh < 2; ++rh) {
            const uint32_t sw = prmt(hw[rh], 0u, 0x2301u);   // bytes of each 16-bit half swapped
            c.t[rh][0] = hw[rh];
            c.t[rh][1] = hw[rh] >> 2;
            c.t[rh][2] = sw;
            c.t[rh][3] = sw >> 2;
        }
    } else if constexpr (BITS == 2) {
        const uint2 v = *reinterpret_cast<const uint2*>(atom + lane * 16 + half * 8);
        c.w[0] = v.x; c.w[1] = v.y;
        c.ws[0] = v.x >> 10; c.ws[1] = v.y >> 10;
    } else {
        const uint2 v = *reinterpret_cast<const uint2*>(atom + lane * 16 + half * 8);
        const uint2 hb = *reinterpret_cast<const uint2*>(atom + 512 + lane * 8);
        c.w[0] = v.x; c.w[1] = v.y;
        c.ws[0] = v.x >> 8; c.ws[1] = v.y >> 8;
        c.t0[0] = rotr32(hb.x, half * 8); c.t0[1] = rotr32(hb.y, half * 8);
        c.t1[0] = rotr32(hb.x, half * 8 + 1); c.t1[1] = rotr32(hb.y, half * 8 + 1);
    }
}

// A-fragment registers of step S4 (0..3) of the loaded half chunk: fp16 pairs q * 2^(o-24).
template <int BITS, int S4, uint32_t MAGIC = 0u>
__device__ __forceinline__ void expand(const Codes<BITS>& c, uint32_t (&a)[4]) {
    if constexpr (BITS == 4) {
        constexpr int jj = S4 >> 1;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int phi = 2 * (S4 & 1) + h;
#pragma unroll
            for (int rh = 0; rh < 2; ++rh) {
                const uint32_t src = (phi < 2) ? c.w[rh * 2 + jj] : c.ws[rh * 2 + jj];
                a[rh + 2 * h] = (src & (0x000F000Fu << (4 * (phi & 1)))) | MAGIC;
            }
        }
    } else if constexpr (BITS == 6) {
        constexpr int jj = S4 >> 1;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int phi = 2 * (S4 & 1) + h;
#pragma unroll
            for (int rh = 0; rh < 2; ++rh) {
                const uint32_t lo = (phi < 2) ? c.w[rh * 2 + jj] : c.ws[rh * 2 + jj];
                a[rh + 2 * h] = (lo & (0x000F000Fu << (4 * h))) | ((c.t[rh][S4] & (0x00300030u << (4 * h))) | MAGIC);
            }
        }
    } else if constexpr (BITS == 8) {
        const uint32_t w0 = c.w[(S4 >> 1) * 4 + 2 * (S4 & 1)], w1 = c.w[(S4 >> 1) * 4 + 2 * (S4 & 1) + 1];
        a[0] = prmt(w0, MAGIC ? 0x64646464u : 0u, 0x4140u);
        a[1] = prmt(w0, MAGIC ? 0x64646464u : 0u, 0x4342u);
        a[2] = prmt(w1, MAGIC ? 0x64646464u : 0u, 0x4140u);
        a[3] = prmt(w1, MAGIC ? 0x64646464u : 0u, 0x4342u);
    } else if constexpr (BITS == 2) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int phi = 2 * S4 + h;
#pragma unroll
            for (int rh = 0; rh < 2; ++rh)
                a[rh + 2 * h] = ((phi <= 4) ? (c.w[rh] & (0x00030003u << (2 * phi)))
                                            : (c.ws[rh] & (0x00030003u << ((2 * phi - 10) & 31)))) | MAGIC;
        }
    } else {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int phi = 2 * S4 + h;
            const int i = phi & 3;
#pragma unroll
            for (int rh = 0; rh < 2; ++rh) {
                const uint32_t lo = (phi < 4) ? c.w[rh] : c.ws[rh];
                const uint32_t hi = (phi < 4) ? c.t0[rh] : c.t1[rh];
                a[rh + 2 * h] = (lo & (0x00030003u << (2 * i))) | ((hi & (0x00040004u << (2 * i))) | MAGIC);
            }
        }
    }
}

// In-place bit offset o of the code of (MMA step S4 of a half chunk, k pair h): see layout.cuh.
template <int BITS>
__host__ __device__ constexpr int code_offset(int s4, int h) {
    const int phi = 2 * s4 + h;
    return BITS == 2 ? (phi <= 4 ? 2 * phi : 2 * phi - 10) : BITS == 3 ? 2 * (phi & 3) : (BITS == 4 || BITS == 6) ? 4 * h : 0;
}

}  // namespace dyn
