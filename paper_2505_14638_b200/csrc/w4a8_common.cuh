// Device helpers shared by the W4A8 kernels: BF16 / E4M3 conversions and the INT4 -> E4M3
// look-up-table dequantizer that implements Eq. 10.  sm_100a only.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/w4a8.h"

namespace w4a8 {


constexpr int kGroup = 128;           // group size along K (Sec. 4.1: "group size of 128")
constexpr float kE4M3Max = 448.0f;    // Z_max of Eq. 3 / Eq. 13

// Device status word bits.
constexpr unsigned int kStatusTimeout = 1u;   // a bounded device-side wait gave up
constexpr unsigned int kStatusBadCode = 2u;   // prepack met a code the target format cannot hold
constexpr unsigned int kStatusPlacement = 4u; // run-time placement of a decode launch ended with a worker index unissued

__device__ __forceinline__ float bf16_bits_to_float(uint32_t bits16) {
    return __uint_as_float(bits16 << 16);
}

// Two fp32 values -> two E4M3 bytes (round-to-nearest-even, saturate to +-448).
// Result bits [7:0] = encode(lo), bits [15:8] = encode(hi).
__device__ __forceinline__ uint32_t cvt_e4m3x2(float hi, float lo) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return (uint32_t)r;
}

// Four fp32 values -> four E4M3 bytes, v0 in the lowest byte.
__device__ __forceinline__ uint32_t cvt_e4m3x4(float v0, float v1, float v2, float v3) {
    return cvt_e4m3x2(v1, v0) | (cvt_e4m3x2(v3, v2) << 16);
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// Two BF16 lanes: (x - off) * sc, the subtraction exact for the small integers it is used on, the
// product rounded once to nearest even.
__device__ __forceinline__ uint32_t bf16x2_sub_mul(uint32_t x, uint32_t off, uint32_t sc) {
    uint32_t d;
    asm("{\n\t"
        ".reg .b32 t;\n\t"
        "sub.rn.bf16x2 t, %1, %2;\n\t"
        "mul.rn.bf16x2 %0, t, %3;\n\t"
        "}\n"
        : "=r"(d)
        : "r"(x), "r"(off), "r"(sc));
    return d;
}

// Eq. 10 as a 16-entry table for one (row, group): entry u holds nearest_E4M3((u - z) * s).
// (u - z) is a small integer and s a BF16 value, so the fp32 product is exact and the table
// entry is the exact product rounded once -- the same bits as converting element by element.
struct DequantLut {
    uint32_t t[4];  // t[j] byte i = entry 4*j + i
    __device__ __forceinline__ void build(float s, int z) {
        float fz = (float)z;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float d0 = (float)(4 * j + 0) - fz;
            float d1 = (float)(4 * j + 1) - fz;
            float d2 = (float)(4 * j + 2) - fz;
            float d3 = (float)(4 * j + 3) - fz;
            t[j] = cvt_e4m3x4(__fmul_rn(d0, s), __fmul_rn(d1, s), __fmul_rn(d2, s),
                              __fmul_rn(d3, s));
        }
    }
    // w holds eight codes, element i in bits [4i+3 : 4i].  out0 = E4M3 bytes of elements 0..3,
    // out1 = elements 4..7 (element order = byte order).
    __device__ __forceinline__ void dequant8(uint32_t w, uint32_t& out0, uint32_t& out1) const {
        uint32_t lo3 = w & 0x77777777u;                               // low three bits: entry within a half table
        uint32_t pick = ((w >> 1) & 0x44444444u) | 0x32103210u;      // bit 3 chooses the half table
        uint32_t a0 = prmt(t[0], t[1], lo3);
        uint32_t b0 = prmt(t[2], t[3], lo3);
        out0 = prmt(a0, b0, pick);
        uint32_t lo3h = lo3 >> 16, pickh = pick >> 16;
        uint32_t a1 = prmt(t[0], t[1], lo3h);
        uint32_t b1 = prmt(t[2], t[3], lo3h);
        out1 = prmt(a1, b1, pickh);
    }
};

}  // namespace w4a8
