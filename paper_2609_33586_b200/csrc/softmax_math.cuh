// Tile geometry and the per-element softmax arithmetic shared by the attention kernels.
#pragma once
#include "attn_kernel_common.cuh"
#include "ptx.cuh"
#include "weight_map.cuh"

#include <cuda_bf16.h>

namespace rowmax {

template <int D, bool FP8>
struct TileCfg {
    static constexpr int kElem = FP8 ? 1 : 2;
    static constexpr int kRowBytes = D * kElem;
    static constexpr int kBoxElems = 128 / kElem;           // one 128-byte swizzle row
    static constexpr int kBoxes = kRowBytes / 128;          // boxes per tile along D
    static constexpr int kBoxBytes = 128 * 128;             // 128 rows x 128 bytes
    static constexpr int kTileBytes = kBoxes * kBoxBytes;   // 128 rows x D
    static constexpr int kUmmaK = 32 / kElem;               // elements per MMA along K (32 bytes)
    static constexpr int kQkSteps = D / kUmmaK;
    static constexpr int kPvSteps = kTileN / kUmmaK;
    static constexpr int kPCols = kTileN * kElem / 4;       // TMEM columns holding one P tile
    static_assert(kRowBytes % 128 == 0, "row must be a whole number of 128-byte swizzle rows");
};

__device__ __forceinline__ uint32_t pack_bf16_rn(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t pack_e4m3x2(float lo, float hi) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}

// exact-mode fp8 path stores P = w * 2^8 in e4m3 (largest value 256 <= 448)
constexpr int kP8ExactOffsetLog2 = 8;

// Turns 32 consecutive scores of one row into weights: returns their sum and writes the packed P
// words (16 words of 2 bf16, or 8 words of 4 fp8).  `limit` = first masked column of the chunk
// (MASKED tiles only; masked scores must already hold -inf for the exact map).
template <bool FP8, int MODE, bool MASKED>
__device__ __forceinline__ float weights_chunk32(const uint32_t (&sraw)[32], float c_eff, float mc_eff,
                                                 int limit, uint32_t* pw) {
    float acc0 = 0.f, acc1 = 0.f;
    uint32_t pb[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        const float s = __uint_as_float(sraw[i]);
        const bool masked = MASKED && i >= limit;
        float w;
        uint32_t bits;  // P pattern: bf16 in the low 16 bits, or an fp8 byte
        if constexpr (MODE == kExact) {
            w = w_exact(fmaf(s, c_eff, -mc_eff));  // masked scores are -inf -> weight 0
            bits = 0;
        } else if constexpr (MODE == kH15) {
            const uint32_t tb = h15_tbits(fmaf(s, c_eff, -mc_eff));  // c_eff = 2c: doubled input
            w = h15_weight_from_tbits(tb);
            bits = FP8 ? h15_e5m2_from_tbits(tb) : (__float_as_uint(w) >> 16);
        } else {
            const int d = pot_index(fmaf(s, c_eff, -mc_eff));
            w = __uint_as_float(static_cast<uint32_t>(127 - d) << 23);
            bits = FP8 ? static_cast<uint32_t>(15 + kP8OffsetLog2 - d) << 2 : (__float_as_uint(w) >> 16);
        }
        if constexpr (MODE != kExact && MASKED) {
            if (masked) { w = 0.f; bits = 0; }
        }
        pb[i] = (MODE == kExact) ? __float_as_uint(w) : bits;
        if (i & 1) acc1 += w; else acc0 += w;
    }
    if constexpr (!FP8) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            if constexpr (MODE == kExact)
                pw[i] = pack_bf16_rn(__uint_as_float(pb[2 * i]), __uint_as_float(pb[2 * i + 1]));
            else
                pw[i] = pb[2 * i] | (pb[2 * i + 1] << 16);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if constexpr (MODE == kExact)
                pw[i] = pack_e4m3x2(__uint_as_float(pb[4 * i]), __uint_as_float(pb[4 * i + 1])) |
                        (pack_e4m3x2(__uint_as_float(pb[4 * i + 2]), __uint_as_float(pb[4 * i + 3])) << 16);
            else
                pw[i] = pb[4 * i] | (pb[4 * i + 1] << 8) | (pb[4 * i + 2] << 16) | (pb[4 * i + 3] << 24);
        }
    }
    return acc0 + acc1;
}


}  // namespace rowmax
