// Tiled ("prepacked") weight layout shared by the persistent GEMM kernels, the sign-magnitude
// look-up table for symmetric groups, and the offline prepack kernel.
//
// Layout (K = 128 KB k-blocks, N output channels, N a multiple of 8):
//   codes region  [KB][N/8][4 chunks][8 rows][16 bytes]: the 64 code bytes of row n of k-block kb
//                 are four 16-byte chunks; chunk c is stored at
//                 ((kb * N + (n & ~7)) * 64) + c * 128 + (n & 7) * 16, i.e. the same chunk of eight
//                 consecutive rows is one 128-byte line.  A thread that expands row n reads its
//                 chunks at a fixed 128-byte stride (no per-chunk address arithmetic), and eight
//                 consecutive rows read with 128-bit loads touch every shared-memory bank once.
//   meta region   [KB][N][MB bytes]   starts at KB * N * 64; MB = 2 (BF16 group scale) in the
//                 sign-magnitude format, 4 (BF16 scale, zero-point byte, one byte of padding) in
//                 the generic format
// Any run of consecutive eight-row units of one k-block is therefore one contiguous, 128-byte
// aligned piece of codes plus one contiguous piece of meta data: two bulk copies bring it into
// shared memory, whatever row partition the kernel picks at launch.
#pragma once

#include <cuda_bf16.h>

#include "w4a8_common.cuh"
#include "w4a8_ptx.cuh"

namespace w4a8 {

constexpr int kFmtCanonical = W4A8_FMT_CANONICAL;
constexpr int kFmtTiled = W4A8_FMT_TILED;
constexpr int kFmtTiledSignMag = W4A8_FMT_TILED_SIGNMAG;
constexpr int kFmtTiledFp8 = W4A8_FMT_TILED_FP8;   // FP8 weights (W8A8 comparison scheme): 128 bytes per row and k-block, no meta data

constexpr int kRowCodeBytes = 64;  // one row of one k-block: 128 INT4 codes
constexpr uint32_t kChunkStride = 128;  // bytes between two chunks of one row
// Offset of a row's first chunk within a piece of codes that starts on a multiple of eight rows.
__host__ __device__ constexpr uint32_t tiled_row_offset(int row) {
    return (uint32_t)(row >> 3) * 512u + (uint32_t)(row & 7) * 16u;
}
__host__ __device__ constexpr int meta_bytes(int fmt) { return fmt == kFmtTiledSignMag ? 2 : (fmt == kFmtTiledFp8 ? 0 : 4); }
// Bytes of one row of one k-block, and the offset of a row's first 16-byte chunk within a piece that
// starts on a multiple of eight rows (chunk c of the row sits c * 128 bytes further), per format.
__host__ __device__ constexpr int row_bytes(int fmt) { return fmt == kFmtTiledFp8 ? 128 : kRowCodeBytes; }
__host__ __device__ constexpr uint32_t row_offset(int fmt, int row) {
    return fmt == kFmtTiledFp8 ? (uint32_t)(row >> 3) * 1024u + (uint32_t)(row & 7) * 16u : tiled_row_offset(row);
}

// Sign-magnitude table of a symmetric group (z = 8): entry d = nearest_E4M3(d * s), d = 0..7.
// A stored nibble carries |u - 8| in its low three bits; the sign travels separately and is
// applied by flipping the E4M3 sign bit (the format is sign-magnitude and the rounding is
// symmetric, so nearest_E4M3(-d s) and nearest_E4M3(d s) differ in that bit only).
struct SignMagLut {
    uint32_t t0, t1;
    __device__ __forceinline__ void build(float s) {
        t0 = cvt_e4m3x4(__fmul_rn(0.0f, s), s, __fmul_rn(2.0f, s), __fmul_rn(3.0f, s));
        t1 = cvt_e4m3x4(__fmul_rn(4.0f, s), __fmul_rn(5.0f, s), __fmul_rn(6.0f, s), __fmul_rn(7.0f, s));
    }
    // Word layout: nibble i (i = 0..3) = magnitude of element i, nibble 4+i = magnitude of
    // element 4+i; sign of element i in bit 8i+7, sign of element 4+i in bit 8i+3.
    __device__ __forceinline__ void dequant8(uint32_t w, uint32_t& out0, uint32_t& out1) const {
        const uint32_t sel = w & 0x77777777u;
        out0 = prmt(t0, t1, sel) ^ (w & 0x80808080u);
        out1 = prmt(t0, t1, sel >> 16) ^ ((w << 4) & 0x80808080u);
    }
};

// The four code chunks of one row (constant address offsets: no arithmetic per chunk).
template <int C>
__device__ __forceinline__ void load_code_chunk(uint32_t src, uint32_t (&pk)[16]) {
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4+%5];"
                 : "=r"(pk[4 * C]), "=r"(pk[4 * C + 1]), "=r"(pk[4 * C + 2]), "=r"(pk[4 * C + 3])
                 : "r"(src), "n"(C * (int)kChunkStride));
}
__device__ __forceinline__ void load_row_codes(uint32_t src, uint32_t (&pk)[16]) {
    load_code_chunk<0>(src, pk);
    load_code_chunk<1>(src, pk);
    load_code_chunk<2>(src, pk);
    load_code_chunk<3>(src, pk);
}

// Expands one row of one k-block into 128 E4M3 bytes written as a row of a K-major tile with
// the 128-byte swizzle.  `src` = shared address of the row's first code chunk (piece base +
// tiled_row_offset(row)), `meta` = shared address of its meta entry, `row` = row index within
// the destination tile, `dst` = shared address of the destination row.
template <int FMT>
__device__ __forceinline__ void dequant_row_to_smem(uint32_t src, uint32_t meta, int row, uint32_t dst) {
    const uint32_t sw128 = (uint32_t)(row & 7);
    uint32_t mbits;
    if constexpr (FMT == kFmtTiledSignMag)
        asm volatile("ld.shared.u16 %0, [%1];" : "=r"(mbits) : "r"(meta));
    else
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(mbits) : "r"(meta));
    const float sc = bf16_bits_to_float(mbits & 0xFFFFu);
    uint32_t pk[16];
    load_row_codes(src, pk);
    SignMagLut slut;
    DequantLut glut;
    if constexpr (FMT == kFmtTiledSignMag)
        slut.build(sc);
    else
        glut.build(sc, (int)((mbits >> 16) & 0xFFu));
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        uint32_t o0, o1, o2, o3;
        if constexpr (FMT == kFmtTiledSignMag) {
            slut.dequant8(pk[2 * c], o0, o1);
            slut.dequant8(pk[2 * c + 1], o2, o3);
        } else {
            glut.dequant8(pk[2 * c], o0, o1);
            glut.dequant8(pk[2 * c + 1], o2, o3);
        }
        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (((uint32_t)c ^ sw128) << 4)), "r"(o0),
                     "r"(o1), "r"(o2), "r"(o3)
                     : "memory");
    }
}

// W4A16 comparison scheme, sign-magnitude codes: the row's 128 weights of the k-block as BF16
// values bf16_rn(+-d * s) -- the same one rounding as a BF16 multiplication of the integer by the
// group scale -- written as two rows of 128 bytes (64 values each) of two K-major panels with the
// 128-byte swizzle, the second panel 16384 bytes behind the first.  The table of the eight
// magnitudes is split into low and high bytes (a byte permute picks among eight bytes); the sign
// bits of the code words sit where the high bytes' sign bits go.
__device__ __forceinline__ void dequant_row_to_smem_bf16(uint32_t src, uint32_t meta, int row, uint32_t dst) {
    const uint32_t sw128 = (uint32_t)(row & 7);
    uint32_t mbits;
    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(mbits) : "r"(meta));
    const float sc = bf16_bits_to_float(mbits & 0xFFFFu);
    uint32_t pk[16];
    load_row_codes(src, pk);
    uint32_t tl0 = 0, tl1 = 0, th0 = 0, th1 = 0;
#pragma unroll
    for (int d = 0; d < 8; ++d) {
        const uint32_t b = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(__fmul_rn((float)d, sc)));
        if (d < 4) {
            tl0 |= (b & 0xFFu) << (8 * d);
            th0 |= (b >> 8) << (8 * d);
        } else {
            tl1 |= (b & 0xFFu) << (8 * (d - 4));
            th1 |= (b >> 8) << (8 * (d - 4));
        }
    }
#pragma unroll
    for (int j = 0; j < 16; ++j) {   // word j: elements 8j .. 8j+7 = one 16-byte chunk of BF16 values
        const uint32_t w = pk[j], sel = w & 0x77777777u;
        const uint32_t lo_a = prmt(tl0, tl1, sel), hi_a = prmt(th0, th1, sel) ^ (w & 0x80808080u);
        const uint32_t lo_b = prmt(tl0, tl1, sel >> 16), hi_b = prmt(th0, th1, sel >> 16) ^ ((w << 4) & 0x80808080u);
        const uint32_t o0 = prmt(lo_a, hi_a, 0x5140u), o1 = prmt(lo_a, hi_a, 0x7362u);
        const uint32_t o2 = prmt(lo_b, hi_b, 0x5140u), o3 = prmt(lo_b, hi_b, 0x7362u);
        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (uint32_t)((j >> 3) * 16384) + ((((uint32_t)j & 7u) ^ sw128) << 4)),
                     "r"(o0), "r"(o1), "r"(o2), "r"(o3)
                     : "memory");
    }
}

// Same expansion into registers and from there into tensor memory: the row's 128 E4M3 bytes go
// to 32 consecutive 32-bit columns starting at `taddr` (lane = this thread's lane within its
// warp's lane quarter), written as two 16-column stores to keep the live register count low.
// Warp-collective: every lane of the warp must call it with a readable row (a lane without a
// row of its own repeats another one; its tensor-memory lane is then never read out).
template <int FMT>
__device__ __forceinline__ void dequant_row_to_tmem(uint32_t src, uint32_t meta, uint32_t taddr) {
    uint32_t mbits;
    uint32_t pk[16];
    if constexpr (FMT == kFmtTiledSignMag)
        asm volatile("ld.shared.u16 %0, [%1];" : "=r"(mbits) : "r"(meta));
    else
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(mbits) : "r"(meta));
    load_row_codes(src, pk);
    const float sc = bf16_bits_to_float(mbits & 0xFFFFu);
    if constexpr (FMT == kFmtTiledSignMag) {
        SignMagLut lut;
        lut.build(sc);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t out[16];
#pragma unroll
            for (int w = 0; w < 8; ++w) lut.dequant8(pk[8 * h + w], out[2 * w], out[2 * w + 1]);
            ptx::tmem_st_32x32b_x16(taddr + 16u * h, out);
        }
    } else {
        DequantLut lut;
        lut.build(sc, (int)((mbits >> 16) & 0xFFu));
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t out[16];
#pragma unroll
            for (int w = 0; w < 8; ++w) lut.dequant8(pk[8 * h + w], out[2 * w], out[2 * w + 1]);
            ptx::tmem_st_32x32b_x16(taddr + 16u * h, out);
        }
    }
}

// FP8 weights (W8A8 comparison scheme): the row's 128 bytes of the k-block go to tensor memory as they are.
__device__ __forceinline__ void copy_fp8_row_to_tmem(uint32_t src, uint32_t taddr) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        uint32_t out[16];
#pragma unroll
        for (int c = 0; c < 4; ++c)
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(out[4 * c]), "=r"(out[4 * c + 1]), "=r"(out[4 * c + 2]), "=r"(out[4 * c + 3])
                         : "r"(src + (uint32_t)(4 * h + c) * kChunkStride));
        ptx::tmem_st_32x32b_x16(taddr + 16u * h, out);
    }
}

// [N][K] FP8 bytes -> tiled order (one thread per 16-byte chunk).
__global__ void prepack_fp8_kernel(const uint8_t* __restrict__ w8, int64_t N, int64_t K, uint8_t* __restrict__ out) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;   // chunk index: n * (K / 16) + k / 16
    const int64_t cpr = K >> 4;
    if (i >= N * cpr) return;
    const int64_t n = i / cpr, ck = i - n * cpr;
    const int64_t kb = ck >> 3, c = ck & 7;
    const uint4 v = *reinterpret_cast<const uint4*>(w8 + n * K + ck * 16);
    *reinterpret_cast<uint4*>(out + (kb * N + (n & ~(int64_t)7)) * 128 + c * 128 + (n & 7) * 16) = v;
}

// The expansion of one row whose codes and meta word are already in registers.
template <int FMT>
__device__ __forceinline__ void expand_row_to_tmem(const uint32_t (&pk)[16], uint32_t mbits, uint32_t taddr) {
    const float sc = bf16_bits_to_float(mbits & 0xFFFFu);
    if constexpr (FMT == kFmtTiledSignMag) {
        SignMagLut lut;
        lut.build(sc);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t out[16];
#pragma unroll
            for (int w = 0; w < 8; ++w) lut.dequant8(pk[8 * h + w], out[2 * w], out[2 * w + 1]);
            ptx::tmem_st_32x32b_x16(taddr + 16u * h, out);
        }
    } else {
        DequantLut lut;
        lut.build(sc, (int)((mbits >> 16) & 0xFFu));
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t out[16];
#pragma unroll
            for (int w = 0; w < 8; ++w) lut.dequant8(pk[8 * h + w], out[2 * w], out[2 * w + 1]);
            ptx::tmem_st_32x32b_x16(taddr + 16u * h, out);
        }
    }
}

__device__ __forceinline__ uint32_t load_meta_word(uint32_t meta, int fmt) {
    uint32_t mbits;
    if (fmt == kFmtTiledSignMag)
        asm volatile("ld.shared.u16 %0, [%1];" : "=r"(mbits) : "r"(meta));
    else
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(mbits) : "r"(meta));
    return mbits;
}

// Two rows (two items of one pipeline stage) expanded into 2 x 32 consecutive tensor-memory
// columns: all ten shared-memory loads are issued before the first look-up, so that the second
// row's loads are in flight while the first row is expanded.  Warp-collective.
template <int FMT>
__device__ __forceinline__ void dequant_two_rows_to_tmem(uint32_t src0, uint32_t meta0, uint32_t src1, uint32_t meta1,
                                                         uint32_t taddr) {
    uint32_t pa[16], pb[16];
    const uint32_t m0 = load_meta_word(meta0, FMT), m1 = load_meta_word(meta1, FMT);
    load_row_codes(src0, pa);
    load_row_codes(src1, pb);
    expand_row_to_tmem<FMT>(pa, m0, taddr);
    expand_row_to_tmem<FMT>(pb, m1, taddr + 32u);
}

// ---------------------------------------------------------------------------------------------
// Offline prepack: canonical [N][K/2] codes + [N][K/128] scales (+ zero-points) -> tiled buffer.
// One CTA per (128 rows, k-block), one thread per row.  In the sign-magnitude format a code 0
// (value -8 s) cannot be represented: it is stored as -7 s and the "unrepresentable code" status
// bit is raised.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t to_signmag_word(uint32_t w, bool& bad) {
    uint32_t out = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        int u = (int)((w >> (4 * i)) & 15u);
        int d = u - 8;
        uint32_t sign = d < 0 ? 1u : 0u;
        int mag = d < 0 ? -d : d;
        if (mag > 7) {
            bad = true;
            mag = 7;
        }
        out |= (uint32_t)mag << (4 * i);
        const int sign_bit = (i < 4) ? (8 * i + 7) : (8 * (i - 4) + 3);
        out |= sign << sign_bit;
    }
    return out;
}

__global__ void __launch_bounds__(128)
prepack_kernel(const uint8_t* __restrict__ codes, const uint16_t* __restrict__ gscale,
               const uint8_t* __restrict__ gzero, int64_t N, int64_t K, int fmt, uint8_t* __restrict__ out,
               unsigned int* status_word) {
    const int64_t KB = K >> 7;
    const int64_t rt = blockIdx.x / KB, kb = blockIdx.x - rt * KB;
    const int64_t n = rt * 128 + threadIdx.x;
    if (n >= N) return;
    const uint4* src = reinterpret_cast<const uint4*>(codes + n * (K >> 1) + kb * 64);
    uint4 w[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) w[c] = src[c];
    if (fmt == kFmtTiledSignMag) {
        bool bad = false;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            w[c].x = to_signmag_word(w[c].x, bad);
            w[c].y = to_signmag_word(w[c].y, bad);
            w[c].z = to_signmag_word(w[c].z, bad);
            w[c].w = to_signmag_word(w[c].w, bad);
        }
        if (bad) atomicOr(status_word, kStatusBadCode);
    }
    uint8_t* dst = out + (kb * N + (n & ~(int64_t)7)) * kRowCodeBytes + (n & 7) * 16;
#pragma unroll
    for (int c = 0; c < 4; ++c) *reinterpret_cast<uint4*>(dst + c * kChunkStride) = w[c];
    uint8_t* meta = out + KB * N * kRowCodeBytes + (kb * N + n) * meta_bytes(fmt);
    const uint16_t sc = gscale[n * KB + kb];
    if (fmt == kFmtTiledSignMag) {
        *reinterpret_cast<uint16_t*>(meta) = sc;
    } else {
        const uint32_t z = gzero ? (uint32_t)gzero[n * KB + kb] : 8u;
        *reinterpret_cast<uint32_t*>(meta) = (uint32_t)sc | (z << 16);
    }
}

}  // namespace w4a8
