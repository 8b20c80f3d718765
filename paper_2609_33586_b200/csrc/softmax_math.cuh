// Tile geometry and the per-element softmax arithmetic of the attention kernel.
//
// Instruction budget per score element (what the tensor cores leave for the softmax warps is about
// 8 issue slots at bf16 and 4 at fp8, per element, at full MMA rate), so the hot loops use packed
// two-lane fp32 instructions (fma.rn.f32x2 / add.rn.f32x2), the three-input max, and for the
// rounding maps an integer multiply-add that builds the fp32 weight pattern on the FMA pipe.
#pragma once
#include "attn_kernel_common.cuh"
#include "ptx.cuh"
#include "weight_map.cuh"

#include <cuda_bf16.h>
#include <cuda_fp16.h>

namespace rowmax {

template <int D, bool FP8>
struct TileCfg {
    static constexpr int kElem = FP8 ? 1 : 2;
    static constexpr int kRowBytes = D * kElem;
    // Swizzle span of the shared-memory tiles: 128 bytes, or 64 when a row has only 64 (fp8, D = 64).
    static constexpr int kSwizzle = kRowBytes >= 128 ? 128 : 64;
    static constexpr int kBoxElems = kSwizzle / kElem;      // one swizzle row
    static constexpr int kBoxes = kRowBytes / kSwizzle;     // boxes per tile along D
    static constexpr int kBoxBytes = 128 * kSwizzle;        // 128 rows x one swizzle row
    static constexpr int kTileBytes = kBoxes * kBoxBytes;   // 128 rows x D
    static constexpr int kStepsPerBox = kSwizzle / 32;      // MMA steps (32 bytes along K) per swizzle row
    static constexpr int kUmmaK = 32 / kElem;               // elements per MMA along K (32 bytes)
    static constexpr int kQkSteps = D / kUmmaK;
    static constexpr int kPvSteps = kTileN / kUmmaK;
    static_assert(kRowBytes % kSwizzle == 0, "row must be a whole number of swizzle rows");
};

// P is stored as weight * 2^kPOff so that it fills the range of its fp8 format: e4m3 holds the
// exact-mode weights up to 2^8 = 256 <= 448; e5m2 holds the lattice weights {1, 1.5} * 2^k exactly
// from 2^15 down to 2^-14 (k >= -29 relative to the row maximum).  The row sum carries the same
// factor, so it cancels in O and is subtracted from LSE.
template <bool FP8, int MODE>
struct PFormat {
    // e4m3 (3 fraction bits) for exact mode and for the eighth-octave family member, whose weights
    // carry 3 fraction bits; e5m2 for pot, h15 and the quarter-octave member (at most 2 fraction bits)
    static constexpr bool kE4M3 = FP8 && (is_exact_like(MODE) || MODE == kH15K3);
    static constexpr int kOffLog2 = FP8 ? (kE4M3 ? 8 : 15) : 0;
};

// ---- packed fp32 pairs and small helpers
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
    float2 d;
    asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%6, %7};\n\t"
        "fma.rn.f32x2 rd, ra, rb, rc;\n\t"
        "mov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d.x), "=f"(d.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
    return d;
}
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) {
    float2 d;
    asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
        "add.rn.f32x2 rd, ra, rb;\n\t"
        "mov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d.x), "=f"(d.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}
__device__ __forceinline__ float2 fmul2(float2 a, float2 b) {
    float2 d;
    asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
        "mul.rn.f32x2 rd, ra, rb;\n\t"
        "mov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d.x), "=f"(d.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// (a * b + c) mod 2^32 as one integer multiply-add; b arrives in a register so that the shift it
// stands for stays an FMA-pipe instruction.
__device__ __forceinline__ uint32_t imad(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t pack_bf16_rn(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t pack_e4m3x2(float lo, float hi) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint32_t pack_f16x2_rn(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Four fp32 values to four e5m2 bytes (first argument in the lowest byte) in one instruction.  The instruction rounds
// stochastically on the random bits it is given; every weight that goes through it here is a lattice weight, exactly
// representable in e5m2 (a power of two times 1, 1.25, 1.5 or 1.75) down to the format's subnormal grid, so the
// result does not depend on those bits; with the bits zero a value below that grid is cut off toward zero, as the
// upper byte of its fp16 pattern would be.
__device__ __forceinline__ uint32_t pack_e5m2x4_exact(float b0, float b1, float b2, float b3) {
    uint32_t d;
    asm("cvt.rs.satfinite.e5m2x4.f32 %0, {%1, %2, %3, %4}, %5;" : "=r"(d) : "f"(b3), "f"(b2), "f"(b1), "f"(b0), "r"(0u));
    return d;
}

// Row maximum of 128 scores held as 4 x 32 registers.
__device__ __forceinline__ float row_max128(const uint32_t (&s)[4][32]) {
    float m[8];
#pragma unroll
    for (int a = 0; a < 8; ++a) m[a] = -INFINITY;
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
#pragma unroll
        for (int i = 0; i < 32; i += 16) {
#pragma unroll
            for (int a = 0; a < 8; ++a)
                m[a] = max3(m[a], __uint_as_float(s[cc][i + 2 * a]), __uint_as_float(s[cc][i + 2 * a + 1]));
        }
    }
    return fmaxf(max3(m[0], m[1], m[2]), max3(m[3], m[4], max3(m[5], m[6], m[7])));
}

// Row minimum of the same 128 scores (decides whether the h15 clamp can be skipped for a tile).
__device__ __forceinline__ float min3(float a, float b, float c) {
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float row_min128(const uint32_t (&s)[4][32]) {
    float m[8];
#pragma unroll
    for (int a = 0; a < 8; ++a) m[a] = INFINITY;
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
#pragma unroll
        for (int i = 0; i < 32; i += 16) {
#pragma unroll
            for (int a = 0; a < 8; ++a)
                m[a] = min3(m[a], __uint_as_float(s[cc][i + 2 * a]), __uint_as_float(s[cc][i + 2 * a + 1]));
        }
    }
    return fminf(min3(m[0], m[1], m[2]), min3(m[3], m[4], min3(m[5], m[6], m[7])));
}

// Sum of |x| over the 16 * CHUNKS e4m3 bytes (128 or 64) at a 16-byte aligned shared-memory address, rounded up a little
// (the caller adds its own margin): pairs are widened to fp16 (exact), summed in eight fp16 lanes of at
// most 16 terms each (each partial sum <= 7168, so no overflow and an error below 0.5 %), then in fp32.
template <int CHUNKS>
__device__ __forceinline__ float abs_sum_e4m3_row(uint32_t saddr) {
    uint32_t acc[4] = {0u, 0u, 0u, 0u};   // four f16x2 accumulators
#pragma unroll
    for (int c = 0; c < CHUNKS; ++c) {
        uint32_t w[4];
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(saddr + 16u * c));
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t lo, hi;   // f16x2 of bytes (0,1) and (2,3)
            asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(lo) : "h"(static_cast<uint16_t>(w[i] & 0xFFFFu)));
            asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(hi) : "h"(static_cast<uint16_t>(w[i] >> 16)));
            lo &= 0x7FFF7FFFu;   // |x| of both halves
            hi &= 0x7FFF7FFFu;
            asm("add.rn.f16x2 %0, %0, %1;" : "+r"(acc[(2 * i) & 3]) : "r"(lo));
            asm("add.rn.f16x2 %0, %0, %1;" : "+r"(acc[(2 * i + 1) & 3]) : "r"(hi));
        }
    }
    float total = 0.f;
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const __half2 h = *reinterpret_cast<const __half2*>(&acc[a]);
        total += __low2float(h) + __high2float(h);
    }
    return total * 1.01f;
}

// Per-row constants of the weight map for one key tile.
struct RowScale {
    float2 c;      // multiplier of the raw score (c, or 2c for the doubled h15 input), both lanes
    float2 nmc;    // minus the scaled anchor (plus the P offset in exact mode), both lanes
    uint32_t two22;  // 1 << 22 held in a register (see imad)
    float clamp_lo;  // h15 family, clamped variant: lower bound of the scaled offset (see w_h15_doubled_pair)
    float pot_neg_cap;  // pot: lower clamp of the offset, -K_max (clamped tail) or -(K_max + 1) (dropped tail)
    float pot_drop_x;   // pot, dropped tail: offsets at or below this (-(K_max + 1/2)) weigh zero
    // saturating form (SAT, h15 family): u = sat(score * su + ou) is the distance below the anchor as a fraction
    // of the clamp distance R = 2^K * 126 (2^K * 127 in a tile with masked scores); sat_mul = -R
    float su, ou, sat_mul;
};

// fma with saturation to [0, 1] (NaN gives 0)
__device__ __forceinline__ float fma_sat(float a, float b, float c) {
    float d;
    asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// Turns 32 consecutive scores of one row into weights.  Adds them (times 2^kOffLog2) into `acc`
// (two independent packed accumulators, summed by the caller)
// and writes the packed P words: 16 words of 2 bf16 (2 fp16 with HALFP), or 8 words of 4 fp8.  In a MASKED tile
// columns >= limit are masked: their scores already hold -inf and their weights are forced to 0.
// CLAMP = false (h15 only) may be used when every doubled offset of the chunk is known to be >= -252.
// SAT (h15 family, anchor always current): the scale, the shift by the anchor and the lower clamp are one
// saturating multiply-add, u = sat((anchor - score) c' / R) in [0, 1], small and therefore accurate near the anchor;
// the second multiply-add puts R u back and adds the rounding constant in one rounding: t = 2^23 + 2^22 - R u, the
// integer n = -RNE(R u), clamped at -R.  No clamped or unclamped variants, no row minimum: a score further than R
// below its anchor, and a masked score (-inf), saturate.  With R = 2^K * 126 the saturated weight is the floor
// 2^-126 of Eq. h15; a key tile with masked scores uses R = 2^K * 127, whose saturated pattern is +0, so that a
// masked score weighs exactly nothing.  The integer is that of Eq. h15 up to the fp32 rounding of u (relative
// 2^-23 of the distance), i.e. it can differ only for offsets that close to a rounding tie.
template <bool FP8, int MODE, bool MASKED, bool CLAMP = true, bool HALFP = false, bool SAT = false>
__device__ __forceinline__ void weights_chunk32(const uint32_t (&s)[32], const RowScale& rs, int limit,
                                                float2 (&acc)[2], uint32_t* pw) {
    constexpr int kOff = PFormat<FP8, MODE>::kOffLog2;
    uint32_t half16[16];
    float2 w_even = make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float2 sv = make_float2(__uint_as_float(s[2 * i]), __uint_as_float(s[2 * i + 1]));
        float2 x = make_float2(0.f, 0.f);
        if constexpr (!SAT) x = ffma2(sv, rs.c, rs.nmc);
        float2 w;
        if constexpr (SAT && h15_family_k(MODE) > 0) {
            float2 t;
            t.x = fmaf(fma_sat(sv.x, rs.su, rs.ou), rs.sat_mul, kH15Magic);
            t.y = fmaf(fma_sat(sv.y, rs.su, rs.ou), rs.sat_mul, kH15Magic);
            w = h15_weight_pair_from_t<kOff, h15_family_k(MODE)>(t, rs.two22);
        } else if constexpr (exact_poly_eighths(MODE) > 0) {
            // e eighths of the pairs, spread evenly, take the polynomial route, the rest the hardware ex2; a masked
            // score (-inf) weighs nothing on either route
            constexpr int e = exact_poly_eighths(MODE);
            if (((i * e) & 7) < e) {
                w.x = w_exact_poly3(x.x);
                w.y = w_exact_poly3(x.y);
            } else {
                w.x = w_exact(x.x);
                w.y = w_exact(x.y);
            }
        } else if constexpr (is_exact_like(MODE)) {
            w.x = w_exact(x.x);  // masked scores are -inf -> weight 0
            w.y = w_exact(x.y);
        } else if constexpr (h15_family_k(MODE) > 0) {
            // Eq. h15 on the input scaled by 2^K (K = 1: doubled): clamp, add 2^23 + 2^22 (rounds to the
            // integer n, ties to even), then (bits << (23 - K)) + bias builds the weight times 2^kOff.
            w = w_h15_doubled_pair<kOff, CLAMP, h15_family_k(MODE)>(x, rs.two22, rs.clamp_lo);
        } else {
            w = pot_weight_pair_rne<kOff>(x, rs.pot_neg_cap, rs.two22 << 1);
            if constexpr (MODE == kPotDrop) {   // the index K_max + 1 stands for everything beyond K_max: weight zero
                if (x.x <= rs.pot_drop_x) w.x = 0.f;
                if (x.y <= rs.pot_drop_x) w.y = 0.f;
            }
        }
        if constexpr (!is_exact_like(MODE) && MASKED) {
            if (2 * i >= limit) w.x = 0.f;
            if (2 * i + 1 >= limit) w.y = 0.f;
        }
        acc[i & 1] = fadd2(acc[i & 1], w);
        if constexpr (!FP8 && HALFP) {
            pw[i] = pack_f16x2_rn(w.x, w.y);   // fp16 P: exact for the lattice weights down to 2^-14, rounded to nearest otherwise
        } else if constexpr (!FP8) {
            if constexpr (is_exact_like(MODE)) pw[i] = pack_bf16_rn(w.x, w.y);
            else pw[i] = __byte_perm(__float_as_uint(w.x), __float_as_uint(w.y), 0x7632);  // exact: at most 3 fraction bits
        } else {
            if constexpr (PFormat<FP8, MODE>::kE4M3) {
                half16[i] = pack_e4m3x2(w.x, w.y);
            } else if constexpr (is_pot(MODE)) {
                // e5m2 P of powers of two: four of them convert exactly at once (measured 2.5 % faster for pot than
                // the route below, 0.6 % slower for the h15 family, whose pipe mix differs)
                if (i & 1) pw[i >> 1] = pack_e5m2x4_exact(w_even.x, w_even.y, w.x, w.y);
                else w_even = w;
            } else {
                half16[i] = pack_f16x2_rn(w.x, w.y);  // at most 2 fraction bits: exact in fp16
            }
        }
    }
    if constexpr (FP8 && (PFormat<FP8, MODE>::kE4M3 || !is_pot(MODE))) {
        // e4m3 P: two converted pairs per word.  e5m2 P of the h15 family: e5m2 is the upper byte of an fp16 pattern,
        // and these weights have at most two fraction bits, so the upper bytes of the four halves are the exact P bytes.
#pragma unroll
        for (int i = 0; i < 8; ++i)
            pw[i] = __byte_perm(half16[2 * i], half16[2 * i + 1], PFormat<FP8, MODE>::kE4M3 ? 0x5410 : 0x7531);
    }
}

}  // namespace rowmax
