// Parameters and small helpers shared by the attention kernels and the host launcher.
#pragma once
#include <cuda.h>
#include <stdint.h>

namespace rowmax {

constexpr int kTileM = 128;  // query rows per tile
constexpr int kTileN = 128;  // keys per tile

// storage type of q, k, v (the values of ATTN_IN_* in the C interface)
enum InType : int { kInBF16 = 0, kInFP8 = 1, kInFP16 = 2 };
// kPotDrop is internal: Rowmax-PoT with a dropped tail (the C interface selects it through attn_fwd_pot), a
// separate instance so that the clamped tail does not pay for the comparison that drops.
// kExactPoly1/3/4 are internal too: the partly emulated exact mode with 1, 3 or 4 eighths of the scores on the
// polynomial route (kExactPoly itself: 2 eighths), selected through attn_fwd_exact_emulated.
enum WeightMode : int { kExact = 0, kPot = 1, kH15 = 2, kH15K2 = 3, kH15K3 = 4, kExactPoly = 5, kPotDrop = 6,
                        kExactPoly1 = 7, kExactPoly3 = 8, kExactPoly4 = 9 };
// eighths of the scores whose 2^x is evaluated by the polynomial instead of the special-function unit (0: none)
__host__ __device__ constexpr int exact_poly_eighths(int mode) {
    return mode == kExactPoly ? 2 : mode == kExactPoly1 ? 1 : mode == kExactPoly3 ? 3 : mode == kExactPoly4 ? 4 : 0;
}
__host__ __device__ constexpr bool is_pot(int mode) { return mode == kPot || mode == kPotDrop; }
// modes whose weight is 2^x itself (with the P offset folded into x)
__host__ __device__ constexpr bool is_exact_like(int mode) { return mode == kExact || exact_poly_eighths(mode) > 0; }
// input-rounding exponent of the h15 family member: steps of 2^-k octaves (0: not a family member)
__host__ __device__ constexpr int h15_family_k(int mode) {
    return mode == kH15 ? 1 : mode == kH15K2 ? 2 : mode == kH15K3 ? 3 : 0;
}

struct AttnParams {
    void* o;          // (B,Sq,Hq,D) bf16
    float* lse;       // (B,Hq,Sq) or nullptr
    int B, Hq, Hkv, Sq, Sk;
    int causal;
    int group;        // Hq / Hkv
    float c;          // softmax_scale * q_descale * k_descale * log2(e), rounded once to fp32
    float v_descale;  // 1 for bf16
    float tau;        // rescale threshold in octaves (0 = the anchor is always the running maximum)
    uint32_t two22;   // 1 << 22, kept in a register for the h15 integer multiply-add
    // Rowmax-PoT tail (Eq. rowmax-pot and the sentence after it): index cap K_max and what happens beyond it
    float pot_neg_cap;  // lower clamp of the offset: -K_max (clamped tail) or -(K_max + 1) (dropped tail)
    float pot_drop_x;   // dropped tail: offsets below -(K_max + 1/2) weigh zero
    int* status;      // device-global sticky status word
#ifdef ROWMAX_TRACE
    long long* trace;  // optional per-role cycle stamps of one CTA: [role 4][tile 64][slot 8]
    int trace_block;
#endif
};

// Status codes written by expired waits: role << 8 | barrier id.
enum : int {
    kRoleSerial = 1, kRoleLoad = 2, kRoleMma = 3, kRoleSoftmax = 4, kRoleCorr = 5, kRoleEpi = 6, kRoleSelftest = 7
};

}  // namespace rowmax
