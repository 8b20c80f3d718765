// Device weight maps: exact (2^x), Rowmax-PoT (Eq. rowmax-pot) and Rowmax-H15 (Eq. h15), on fp32
// base-two offsets.  The fused kernel and the sweep entry point use these same functions.
#pragma once
#include <stdint.h>

namespace rowmax {

constexpr int kPotKmax = 20;  // K_max of Rowmax-PoT (App. A, main point)

// ---- exact: hardware ex2 (special-function unit), subnormal results flushed to zero.
__device__ __forceinline__ float w_exact(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// ---- exact, emulated on the FMA and ALU pipes (the partial emulation the paper's baseline kernel uses to
// take load off the special-function unit, Sec. 1 and App. B "FA4's own parameter space"): floor(x) by a
// round-down add of 2^23 + 2^22, a cubic for 2^f on the fraction f in [0,1), and floor(x) added to the
// exponent field.  The cubic is this build's own fit: it interpolates 2^0 and 2^1 (so the map is continuous
// across octaves) and minimises the largest relative error on [0,1], which is 1.03e-4.
// Valid for -127 <= x < 127; smaller inputs (a masked score is -inf) are clamped at -127, where floor = -127 and
// fraction = 0 give the exponent field 0 and the fraction 0: exactly +0, as the hardware ex2 with flush-to-zero
// gives.  Between -127 and -126 the result is a denormal pattern (2^-127 (1 + f) read as a fraction), below 2^-126.
__device__ __forceinline__ float w_exact_poly3(float x) {
    x = fmaxf(x, -127.0f);
    const float t = __fadd_rd(x, 12582912.0f);   // 2^23 + 2^22 + floor(x), exact
    const float f = x - (t - 12582912.0f);       // fraction in [0,1)
    const float p = fmaf(fmaf(fmaf(0.07826797f, f, 0.22630768f), f, 0.69542432f), f, 1.0f);   // 2^f in [1,2]
    return __uint_as_float(__float_as_uint(p) + (__float_as_uint(t) << 23));
}

// ---- Rowmax-H15 (Eq. h15; construction of App. B.1 "Implementation").
// Input is the DOUBLED offset 2x.  After the clamp at -252, adding 2^23 + 2^22 as an fp32 value
// rounds 2x to the nearest integer n (ties to even) and leaves 0x4B400000 + n in the bit pattern.
constexpr float kH15Magic = 12582912.0f;       // 2^23 + 2^22, bit pattern 0x4B400000
constexpr uint32_t kH15MagicBits = 0x4B400000u;

__device__ __forceinline__ uint32_t h15_tbits(float x2) {
    return __float_as_uint(fmaxf(x2, -252.0f) + kH15Magic);
}
// fp32 weight: shifting left by 22 drops the constant and puts bit 0 of n at the top of the
// fraction and the rest in the exponent; adding the pattern of 1.0 supplies the bias:
// bits = (n + 254) << 22, the value (1 + (n mod 2)/2) * 2^floor(n/2).
__device__ __forceinline__ float h15_weight_from_tbits(uint32_t tbits) {
    return __uint_as_float((tbits << 22) + 0x3F800000u);
}
__device__ __forceinline__ float w_h15_doubled(float x2) { return h15_weight_from_tbits(h15_tbits(x2)); }
// Two weights at once, the form the fused kernel uses, for the family member with input steps of
// 2^-K octaves (K = 1 is Rowmax-H15; K = 2, 3 are the quarter- and eighth-octave members of App. B
// "Exponential-map ablation": same add, shift by 23 - K).  Input is the offset times 2^K.  Packed fp32
// add of the magic constant, then (bits << (23 - K)) + bias per lane: the low K bits of n become the
// top fraction bits and the rest the exponent, i.e. 2^floor(n / 2^K) * (1 + (n mod 2^K) / 2^K).  One
// lane uses the shift-add (ALU pipe), the other the equivalent integer multiply-add (FMA pipe), which
// balances the two pipes; `two22` must hold 1 << 22 and arrives in a register so that the
// multiply-add is not turned back into a shift.  kOff scales the weight by 2^kOff (an exact exponent
// shift) for the fp8 P formats.  kClamp = false skips the clamp; the caller must know that both
// inputs are at or above -126 * 2^K.  The clamp value is -126 * 2^K (Eq. h15: the weight floor 2^-126);
// the fused kernel passes -127 * 2^K in a key tile that holds masked scores: that input gives the
// bit pattern of +0 when kOff = 0 (16-bit inputs): a masked score (-inf) then weighs exactly nothing.  With the fp8
// P offset (kOff = 15) the pattern is 2^(kOff - 127) = 2^-112 instead: P, which is what multiplies V, still rounds to
// zero, and the row sum takes 2^-112 against terms of at least 2^15, below one part in 2^127.
// Two rounded patterns t = 2^23 + 2^22 + n (as floats) -> the two weights (1 + (n mod 2^K) / 2^K) 2^floor(n / 2^K)
// times 2^kOff: (bits << (23 - K)) + bias, one lane by shift-add (ALU pipe), the other by the equivalent integer
// multiply-add (FMA pipe).
template <int kOff, int K>
__device__ __forceinline__ float2 h15_weight_pair_from_t(float2 t, uint32_t two22) {
    constexpr uint32_t bias = 0x3F800000u + (static_cast<uint32_t>(kOff) << 23);
    const uint32_t b0 = (__float_as_uint(t.x) << (23 - K)) + bias;
    uint32_t b1;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(b1) : "r"(__float_as_uint(t.y)), "r"(two22 >> (K - 1)), "r"(bias));
    return make_float2(__uint_as_float(b0), __uint_as_float(b1));
}
template <int K>
__device__ __forceinline__ constexpr float h15_clamp_floor() { return -126.0f * (1 << K); }
template <int K>
__device__ __forceinline__ constexpr float h15_clamp_zero() { return -127.0f * (1 << K); }
template <int kOff, bool kClamp = true, int K = 1>
__device__ __forceinline__ float2 w_h15_doubled_pair(float2 x2, uint32_t two22, float clamp_lo = h15_clamp_floor<K>()) {
    static_assert(K >= 1 && K <= 3, "family members k = 1, 2, 3");
    if constexpr (kClamp) {
        x2.x = fmaxf(x2.x, clamp_lo);
        x2.y = fmaxf(x2.y, clamp_lo);
    }
    float2 t;
    asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %4};\n\t"
        "add.rn.f32x2 rd, ra, rb;\n\t"
        "mov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(t.x), "=f"(t.y)
        : "f"(x2.x), "f"(x2.y), "f"(kH15Magic));
    return h15_weight_pair_from_t<kOff, K>(t, two22);
}

// ---- Rowmax-PoT (Eq. rowmax-pot): d = min{K_max, floor(y + 1/2)}, y = -x, w = 2^-d.
// floor(y + 1/2) without double rounding: one round-DOWN add of 2^22 + 64.5 leaves
// 2^22 + floor(2 (y + 64.5)) / 2 exactly, whose integer part is floor(y + 1/2) + 64.
// Capping y at K_max + 1/4 first makes the min{K_max, .} implicit (floor(y + 1/2) = K_max for every
// y in [K_max - 1/2, K_max + 1/2)) and keeps huge and infinite y in range.  y >= -64 is required
// (offsets above the anchor occur only with a deferred rescale, whose threshold is at most 32).
constexpr float kPotMagic = 4194368.5f;        // 2^22 + 64.5, bit pattern 0x4A800081
constexpr uint32_t kPotMagicBase = 0x4A800000u;  // bit pattern of 2^22
constexpr float kPotCapDefault = static_cast<float>(kPotKmax) + 0.25f;
// `cap` = K_max + 1/4 (1 <= K_max <= 126) for the clamped tail.  For the dropped tail the callers cap at
// K_max + 1 + 1/4, so that the index K_max + 1 survives, and give that index the weight zero.
__device__ __forceinline__ uint32_t pot_tbits(float y, float cap = kPotCapDefault) {
    return __float_as_uint(__fadd_rd(fminf(y, cap), kPotMagic));
}
__device__ __forceinline__ int pot_index_from_y(float y, float cap = kPotCapDefault) {
    return static_cast<int>((pot_tbits(y, cap) - kPotMagicBase) >> 1) - 64;   // (2 (t - 2^22)) / 2 - 64
}
__device__ __forceinline__ int pot_index(float x) { return pot_index_from_y(-x); }
// fp32 pattern of 2^(kOff - d): exponent field 127 + kOff - d = (191 + kOff) - (d + 64), and d + 64 is
// the t pattern without its lowest bit, shifted right by one: ((tbits & ~1) << 22) puts it at bit 23
// (the bits of 2^22's own pattern fall off the top).
template <int kOff>
__device__ __forceinline__ float pot_weight_from_tbits(uint32_t tbits) {
    return __uint_as_float((static_cast<uint32_t>(191 + kOff) << 23) - ((tbits & ~1u) << 22));
}
template <int kOff>
__device__ __forceinline__ float pot_weight_from_y(float y, float cap = kPotCapDefault) {
    return pot_weight_from_tbits<kOff>(pot_tbits(y, cap));
}
// Two at once, the form the fused kernel uses, on the offsets x themselves.  -floor(-x + 1/2) = ceil(x - 1/2) is x
// rounded to the nearest integer with ties going DOWN; adding 2^23 + 2^22 rounds to nearest with ties to EVEN, the
// same integer except at an exact tie (x = k + 1/2 with k odd).  Inside the fused kernel x is itself an fp32
// rounding of the true offset, so an exact tie carries no information and this costs nothing; the stand-alone map
// above keeps the definition.  Then the pattern of 2^(n + kOff) is (bits << 23) + bias, one lane by shift-add, the
// other by the equivalent integer multiply-add (two23 must hold 1 << 23).  The lower clamp -cap (cap = K_max, or
// K_max + 1 with a dropped tail, at most 125) keeps the index in range and makes min{K_max, .} implicit.
template <int kOff>
__device__ __forceinline__ float2 pot_weight_pair_rne(float2 x, float neg_cap, uint32_t two23) {
    x.x = fmaxf(x.x, neg_cap);
    x.y = fmaxf(x.y, neg_cap);
    float2 t;
    asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %4};\n\t"
        "add.rn.f32x2 rd, ra, rb;\n\t"
        "mov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(t.x), "=f"(t.y)
        : "f"(x.x), "f"(x.y), "f"(kH15Magic));
    constexpr uint32_t bias = 0x3F800000u + (static_cast<uint32_t>(kOff) << 23);
    const uint32_t b0 = (__float_as_uint(t.x) << 23) + bias;
    uint32_t b1;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(b1) : "r"(__float_as_uint(t.y)), "r"(two23), "r"(bias));
    return make_float2(__uint_as_float(b0), __uint_as_float(b1));
}
__device__ __forceinline__ float w_pot(float x) { return pot_weight_from_y<0>(-x); }
// General tail: K_max as a run-time value, clamped (every key keeps 2^-K_max) or dropped (weight zero
// beyond K_max; ties of y + 1/2 go up in the index, so y = K_max + 1/2 is already dropped).
__device__ __forceinline__ float w_pot_tail(float x, int kmax, bool drop_tail) {
    const float y = -x;
    const float w = pot_weight_from_y<0>(y, static_cast<float>(kmax) + (drop_tail ? 1.25f : 0.25f));
    return (drop_tail && y >= static_cast<float>(kmax) + 0.5f) ? 0.0f : w;
}

}  // namespace rowmax
