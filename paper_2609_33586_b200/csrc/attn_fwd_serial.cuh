#pragma once
#include "softmax_math.cuh"

namespace rowmax {

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
            l_tile += weights_chunk32<FP8, MODE, true>(s[cc], c_eff, mc_eff, col_limit - cc * 32, pw);
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


}  // namespace rowmax
