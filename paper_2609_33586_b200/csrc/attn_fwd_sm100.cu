// Fused attention forward for sm_100a: TMA-staged Q/K/V tiles, tcgen05 MMAs with TMEM accumulators,
// online softmax with a selectable weight map (exact / Rowmax-PoT / Rowmax-H15), bf16 O + fp32 LSE.
//
// Loop structure per query tile (Sec. 5.2; App. B.1): for each key tile in ascending order
//   S = Q K^T -> tile row maximum -> running maximum m (always adopted, threshold 0) ->
//   x = s*c - m*c -> weight map -> row sum l and P (same weights) -> O = alpha*O + P V;
// at the end O = v_descale * O / l and LSE = ln2 * (m*c + log2 l).
#include "attn_kernel_common.cuh"
#include "ptx.cuh"
#include "weight_map.cuh"

#include <cuda_bf16.h>

namespace rowmax {

namespace {

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
// words (16 words of 2 bf16, or 8 words of 4 fp8).  `limit` = first masked column of the chunk.
template <bool FP8, int MODE>
__device__ __forceinline__ float weights_chunk32(const uint32_t (&sraw)[32], float c_eff, float mc_eff,
                                                 int limit, uint32_t* pw) {
    float acc0 = 0.f, acc1 = 0.f;
    uint32_t pb[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        const float s = __uint_as_float(sraw[i]);
        const bool masked = i >= limit;
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
        if constexpr (MODE != kExact) {
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

}  // namespace

// ------------------------------------------------------------------------------------------------
// Serial kernel: one CTA of 128 threads per (query tile, head, batch); thread t owns query row t.
// Every step waits for the previous one (no overlap).  It fixes the data layouts and descriptors.
// ------------------------------------------------------------------------------------------------
template <int D, bool FP8, int MODE>
__global__ void __launch_bounds__(128, 1)
attn_fwd_serial_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                       const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
    using C = TileCfg<D, FP8>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const uint32_t sQ = smem_u32(smem), sK = sQ + C::kTileBytes, sV = sK + C::kTileBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 3 * C::kTileBytes);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const uint32_t bar_q = smem_u32(&bars[0]), bar_kv = smem_u32(&bars[1]), bar_mma = smem_u32(&bars[2]);
    const int tid = threadIdx.x, warp = tid >> 5;
    const WaitCtx wctx{abort_flag, p.status};

    if (tid == 0) {
        mbar_init(bar_q, 1);
        mbar_init(bar_kv, 1);
        mbar_init(bar_mma, 1);
        *abort_flag = (*reinterpret_cast<volatile int*>(p.status) != 0);
        fence_mbar_init();
    }
    constexpr uint32_t kTmemCols = 256;
    if (warp == 0) {
        tmem_alloc(smem_u32(tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const uint32_t tmem_S = tmem, tmem_P = tmem, tmem_O = tmem + 128;
    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;

    const int q0 = blockIdx.x * kTileM, h = blockIdx.y, b = blockIdx.z, hk = h / p.group;
    const int shift = p.Sk - p.Sq;
    int kv_end = p.Sk;
    if (p.causal) kv_end = min(p.Sk, q0 + kTileM + shift);
    const int n_tiles = kv_end > 0 ? (kv_end + kTileN - 1) / kTileN : 0;
    const int row = q0 + tid;
    const int row_limit = p.causal ? min(p.Sk, row + shift + 1) : p.Sk;  // visible keys of this row

    constexpr uint32_t fmt_ab = FP8 ? kFmtE4M3 : kFmtBF16;
    constexpr uint32_t fmt_p = FP8 ? (MODE == kExact ? kFmtE4M3 : kFmtE5M2) : kFmtBF16;
    constexpr uint32_t idesc_s = umma_idesc(fmt_ab, fmt_ab, false, false, kTileM, kTileN);
    constexpr uint32_t idesc_pv = umma_idesc(fmt_p, fmt_ab, false, true, kTileM, D);

    auto load_kv = [&](int j) {
        mbar_arrive_expect_tx(bar_kv, 2 * C::kTileBytes);
#pragma unroll
        for (int bx = 0; bx < C::kBoxes; ++bx) {
            tma_load_4d(sK + bx * C::kBoxBytes, &tmK, bar_kv, bx * C::kBoxElems, hk, j * kTileN, b);
            tma_load_4d(sV + bx * C::kBoxBytes, &tmV, bar_kv, bx * C::kBoxElems, hk, j * kTileN, b);
        }
    };

    if (tid == 0 && n_tiles > 0 && !*abort_flag) {
        mbar_arrive_expect_tx(bar_q, C::kTileBytes);
#pragma unroll
        for (int bx = 0; bx < C::kBoxes; ++bx)
            tma_load_4d(sQ + bx * C::kBoxBytes, &tmQ, bar_q, bx * C::kBoxElems, h, q0, b);
        load_kv(0);
    }

    // exact: x = s*c - m*c (+ the fp8 P offset);  h15: doubled input 2x = s*(2c) - m*(2c)
    const float c_eff = (MODE == kH15) ? 2.0f * p.c : p.c;
    const float x_bias = (FP8 && MODE == kExact) ? static_cast<float>(kP8ExactOffsetLog2) : 0.0f;
    float m_run = -INFINITY, l_run = 0.f;
    uint32_t ph_mma = 0;

    for (int j = 0; j < n_tiles; ++j) {
        if (tid == 0 && !*abort_flag) {
            if (j == 0) mbar_wait(bar_q, 0, wctx, (kRoleSerial << 8) | 0);
            mbar_wait(bar_kv, j & 1, wctx, (kRoleSerial << 8) | 1);
            tc_fence_after();
            if (!*abort_flag) {
#pragma unroll
                for (int ks = 0; ks < C::kQkSteps; ++ks) {
                    const uint32_t off = (ks / 4) * C::kBoxBytes + (ks % 4) * 32;
                    umma_ss<FP8>(tmem_S, umma_desc_sw128(sQ + off, 16, 1024), umma_desc_sw128(sK + off, 16, 1024),
                                 idesc_s, ks > 0);
                }
                umma_commit(bar_mma);
            }
        }
        mbar_wait(bar_mma, ph_mma, wctx, (kRoleSerial << 8) | 2);
        ph_mma ^= 1;
        __syncwarp();
        tc_fence_after();

        uint32_t s[4][32];
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) tmem_ld32(tmem_S + lane_base + cc * 32, s[cc]);
        tmem_wait_ld();

        const int col_limit = row_limit - j * kTileN;  // columns >= col_limit are masked
        float m_t = -INFINITY;
        if (col_limit < kTileN) {
#pragma unroll
            for (int cc = 0; cc < 4; ++cc)
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (cc * 32 + i >= col_limit) s[cc][i] = __float_as_uint(-INFINITY);
        }
#pragma unroll
        for (int cc = 0; cc < 4; ++cc)
#pragma unroll
            for (int i = 0; i < 32; ++i) m_t = fmaxf(m_t, __uint_as_float(s[cc][i]));

        const float m_new = fmaxf(m_run, m_t);
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
        const float alpha = ex2_approx((m_run - m_use) * p.c);
        const float mc_eff = m_use * c_eff - x_bias;
        m_run = m_new;

        // every S column is in registers now, so P may overwrite the S columns
        float l_tile = 0.f;
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
            uint32_t pw[16];
            l_tile += weights_chunk32<FP8, MODE>(s[cc], c_eff, mc_eff, col_limit - cc * 32, pw);
            if constexpr (FP8) tmem_st8(tmem_P + lane_base + cc * 8, pw);
            else tmem_st16(tmem_P + lane_base + cc * 16, pw);
        }
        l_run = l_run * alpha + l_tile;

        if (j > 0 && __any_sync(0xffffffffu, alpha != 1.0f)) {
#pragma unroll
            for (int cc = 0; cc < D / 32; ++cc) {
                uint32_t o[32];
                tmem_ld32(tmem_O + lane_base + cc * 32, o);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                tmem_st32(tmem_O + lane_base + cc * 32, o);
            }
        }
        tmem_wait_st();
        tc_fence_before();
        __syncthreads();

        if (tid == 0 && !*abort_flag) {
            tc_fence_after();
#pragma unroll
            for (int ks = 0; ks < C::kPvSteps; ++ks) {
                const uint64_t bdesc = umma_desc_sw128(sV + ks * C::kUmmaK * 128, C::kBoxBytes, 1024);
                umma_ts<FP8>(tmem_O, tmem_P + ks * 8, bdesc, idesc_pv, (j > 0 || ks > 0) ? 1u : 0u);
            }
            umma_commit(bar_mma);
        }
        mbar_wait(bar_mma, ph_mma, wctx, (kRoleSerial << 8) | 3);
        ph_mma ^= 1;
        if (tid == 0 && j + 1 < n_tiles && !*abort_flag) load_kv(j + 1);
        __syncwarp();
    }
    tc_fence_after();

    // epilogue: O = v_descale * acc / l (undoing the P offset), LSE = ln2 * (m c + log2 l)
    const bool has_keys = l_run > 0.f;
    const float p_unscale = (FP8 && MODE != kExact) ? exp2f(-static_cast<float>(kP8OffsetLog2)) : 1.0f;
    const float inv = has_keys ? p.v_descale * p_unscale / l_run : 0.f;
    if (row < p.Sq && p.lse != nullptr) {
        const float lse = has_keys ? 0.6931471805599453f * (m_run * p.c + log2f(l_run) - x_bias) : -INFINITY;
        p.lse[(static_cast<size_t>(b) * p.Hq + h) * p.Sq + row] = lse;
    }
    __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(p.o) +
                          ((static_cast<size_t>(b) * p.Sq + row) * p.Hq + h) * D;
#pragma unroll
    for (int cc = 0; cc < D / 32; ++cc) {
        uint32_t o[32];
        if (n_tiles > 0) {
            tmem_ld32(tmem_O + lane_base + cc * 32, o);
            tmem_wait_ld();
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = 0;
        }
        if (row < p.Sq) {
#pragma unroll
            for (int v4 = 0; v4 < 4; ++v4) {
                uint4 pk;
                pk.x = pack_bf16_rn(__uint_as_float(o[v4 * 8 + 0]) * inv, __uint_as_float(o[v4 * 8 + 1]) * inv);
                pk.y = pack_bf16_rn(__uint_as_float(o[v4 * 8 + 2]) * inv, __uint_as_float(o[v4 * 8 + 3]) * inv);
                pk.z = pack_bf16_rn(__uint_as_float(o[v4 * 8 + 4]) * inv, __uint_as_float(o[v4 * 8 + 5]) * inv);
                pk.w = pack_bf16_rn(__uint_as_float(o[v4 * 8 + 6]) * inv, __uint_as_float(o[v4 * 8 + 7]) * inv);
                *reinterpret_cast<uint4*>(orow + cc * 32 + v4 * 8) = pk;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// ------------------------------------------------------------------------------------------------
// Host launcher
// ------------------------------------------------------------------------------------------------
template <int D, bool FP8, int MODE>
static cudaError_t launch_serial(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                                 const AttnParams& p, cudaStream_t stream) {
    using C = TileCfg<D, FP8>;
    constexpr int smem_bytes = 3 * C::kTileBytes + 64 + 1024;
    auto kern = attn_fwd_serial_kernel<D, FP8, MODE>;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    dim3 grid((p.Sq + kTileM - 1) / kTileM, p.Hq, p.B);
    kern<<<grid, 128, smem_bytes, stream>>>(tq, tk, tv, p);
    return cudaGetLastError();
}

template <int D, bool FP8>
static cudaError_t dispatch_mode(int mode, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                                 const AttnParams& p, cudaStream_t stream) {
    switch (mode) {
        case kExact: return launch_serial<D, FP8, kExact>(tq, tk, tv, p, stream);
        case kPot: return launch_serial<D, FP8, kPot>(tq, tk, tv, p, stream);
        default: return launch_serial<D, FP8, kH15>(tq, tk, tv, p, stream);
    }
}

// Returns cudaErrorInvalidValue for a combination that is not built.
cudaError_t launch_attn_fwd(int D, bool fp8, int mode, const CUtensorMap& tq, const CUtensorMap& tk,
                            const CUtensorMap& tv, const AttnParams& p, cudaStream_t stream) {
    if (!fp8 && D == 128) return dispatch_mode<128, false>(mode, tq, tk, tv, p, stream);
    if (!fp8 && D == 64) return dispatch_mode<64, false>(mode, tq, tk, tv, p, stream);
    if (fp8 && D == 128) return dispatch_mode<128, true>(mode, tq, tk, tv, p, stream);
    return cudaErrorInvalidValue;
}

// ------------------------------------------------------------------------------------------------
// Weight-map sweep: the same device functions on a flat array of offsets.
// ------------------------------------------------------------------------------------------------
__global__ void weight_map_kernel(const float* __restrict__ x, float* __restrict__ w, size_t n, int mode) {
    const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
    for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += stride) {
        const float xi = x[i];
        float wi;
        if (mode == kExact) wi = w_exact(xi);
        else if (mode == kPot) wi = w_pot(xi);
        else wi = w_h15_doubled(xi * 2.0f);
        w[i] = wi;
    }
}

cudaError_t launch_weight_map(const float* x, float* w, size_t n, int mode, cudaStream_t stream) {
    if (n == 0) return cudaSuccess;
    const int threads = 256;
    size_t blocks = (n + threads - 1) / threads;
    if (blocks > 148 * 8) blocks = 148 * 8;
    weight_map_kernel<<<static_cast<unsigned>(blocks), threads, 0, stream>>>(x, w, n, mode);
    return cudaGetLastError();
}

__device__ int g_attn_status = 0;

cudaError_t status_word_address(int** out) {
    return cudaGetSymbolAddress(reinterpret_cast<void**>(out), g_attn_status);
}

}  // namespace rowmax
