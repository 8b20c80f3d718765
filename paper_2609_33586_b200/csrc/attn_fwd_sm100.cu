// Fused attention forward for sm_100a: TMA-staged Q/K/V tiles, tcgen05 MMAs with TMEM accumulators,
// online softmax with a selectable weight map (exact / Rowmax-PoT / Rowmax-H15), bf16 O + fp32 LSE.
//
// Loop structure per query tile (Sec. 5.2; App. B.1): for each key tile in ascending order
//   S = Q K^T -> tile row maximum -> running maximum m (always adopted, threshold 0) ->
//   x = s*c - m*c -> weight map -> row sum l and P (same weights) -> O = alpha*O + P V;
// at the end O = v_descale * O / l and LSE = ln2 * (m*c + log2 l).
//
// One CTA (16 warps) owns two query tiles of 128 rows of one (batch, head) and walks their key
// tiles once, so every K/V tile staged in shared memory feeds four MMAs:
//   warpgroup 0/1  softmax of query tile 0/1: one thread per row (no shuffles needed: a thread
//                  reads its whole score row from TMEM), weight map, row sum, P written back to
//                  TMEM over the S columns
//   warpgroup 2    correction: rescales the O accumulators in TMEM when a running maximum moved,
//                  and runs the epilogue
//   warp 12        MMA issuer (one thread): S_t = Q_t K^T and O_t += P_t V on the tensor cores
//   warp 13        TMA producer (one thread): Q once, then K/V through a ring of shared-memory slots
// While warpgroup 0 works on S_0(j), the tensor cores compute P_1 V(j-1) and S_1(j), and vice versa.
// TMEM columns: S_0/P_0 [0,128), S_1/P_1 [128,256), O_0 [256,384), O_1 [384,512).
#include "softmax_math.cuh"

namespace rowmax {

namespace {

template <int D, bool FP8>
struct WsCfg {
    using C = TileCfg<D, FP8>;
    static constexpr int kSlots = FP8 ? 8 : (D == 128 ? 4 : 8);  // K/V ring slots (one tile each)
    static constexpr int kQBytes = 2 * C::kTileBytes;
    static constexpr int kRingBytes = kSlots * C::kTileBytes;
    static constexpr int kScaleOff = kQBytes + kRingBytes;        // float alpha[2][128]
    static constexpr int kFinalOff = kScaleOff + 2 * 128 * 4;     // float2 (l, m)[2][128]
    static constexpr int kBarOff = kFinalOff + 2 * 128 * 8;
    static constexpr int kNumBars = 2 + 2 * kSlots + 6 * 2 + 8;
    static constexpr int kMiscOff = kBarOff + kNumBars * 8;
    static constexpr int kSmemBytes = kMiscOff + 16 + 1024;       // + manual 1024-byte alignment slack
    static_assert(kSmemBytes <= 232448, "exceeds the 227 KB shared memory of an sm_100 CTA");
};

__device__ __forceinline__ void reg_dec_48() { asm volatile("setmaxnreg.dec.sync.aligned.u32 48;"); }
__device__ __forceinline__ void reg_dec_80() { asm volatile("setmaxnreg.dec.sync.aligned.u32 80;"); }
__device__ __forceinline__ void reg_inc_192() { asm volatile("setmaxnreg.inc.sync.aligned.u32 192;"); }

// Optional cycle stamps (compiled in only with -DROWMAX_TRACE): one representative thread per role of
// one chosen CTA writes clock64() at fixed points of its first 64 key tiles.
#ifdef ROWMAX_TRACE
#define ROWMAX_STAMP(role, j, slot)                                                              \
    do {                                                                                         \
        if (p.trace != nullptr && static_cast<int>(blockIdx.x) == p.trace_block && (j) < 64)     \
            p.trace[((role) * 64 + (j)) * 8 + (slot)] = clock64();                               \
    } while (0)
#else
#define ROWMAX_STAMP(role, j, slot) do { } while (0)
#endif

// Whether the two softmax warps of a scheduler alternate strictly (see the softmax role).  Measured
// slower than free-running on every workload tried, so it is off; the barriers stay for experiments.
constexpr bool kTakeTurns = false;
constexpr bool kStagger = true;

enum BarId : int { kBarQ = 0, kBarKvFull = 1, kBarKvEmpty = 2, kBarSFull = 3, kBarPFull = 4, kBarOFull = 5,
                   kBarScale = 6, kBarORescaled = 7, kBarFinal = 8, kBarTurn = 9 };

}  // namespace

template <int D, bool FP8, int MODE>
__global__ void __launch_bounds__(512, 1)
attn_fwd_ws_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
    using C = TileCfg<D, FP8>;
    using W = WsCfg<D, FP8>;
    constexpr int NS = W::kSlots;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const uint32_t sQ = smem_u32(smem);
    const uint32_t sRing = sQ + W::kQBytes;
    float* sScale = reinterpret_cast<float*>(smem + W::kScaleOff);
    float2* sFinal = reinterpret_cast<float2*>(smem + W::kFinalOff);
    const uint32_t bar0 = smem_u32(smem + W::kBarOff);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + W::kMiscOff);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + W::kMiscOff + 4);
    const WaitCtx wctx{abort_flag, p.status};

    // barrier addresses
    auto bar_q = [&](int t) { return bar0 + 8u * t; };
    auto bar_kv_full = [&](int s) { return bar0 + 8u * (2 + s); };
    auto bar_kv_empty = [&](int s) { return bar0 + 8u * (2 + NS + s); };
    auto bar_x = [&](int which, int t) { return bar0 + 8u * (2 + 2 * NS + 2 * which + t); };
    auto bar_s_full = [&](int t) { return bar_x(0, t); };      // MMA -> softmax: S_t(j) is in TMEM
    auto bar_p_full = [&](int t) { return bar_x(1, t); };      // softmax -> MMA: P_t(j) is in TMEM
    auto bar_o_full = [&](int t) { return bar_x(2, t); };      // MMA -> correction: P_t V(j) accumulated
    auto bar_scale = [&](int t) { return bar_x(3, t); };       // softmax -> correction: alpha_t(j) in smem
    auto bar_o_rescaled = [&](int t) { return bar_x(4, t); };  // correction -> MMA: O_t rescaled for tile j
    auto bar_final = [&](int t) { return bar_x(5, t); };       // softmax -> correction: (l, m) in smem
    // turn token of the softmax warp pair that shares scheduler w: bar_turn(t, w) lets tile t's warp go
    auto bar_turn = [&](int t, int w) { return bar0 + 8u * (2 + 2 * NS + 12 + 4 * t + w); };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, wg = warp >> 2;

    // work item: heaviest query tiles first (they have the most key tiles under a causal mask)
    const int n_pairs = (p.Sq + 2 * kTileM - 1) / (2 * kTileM);
    const int bh = p.Hq * p.B;
    const int pair = n_pairs - 1 - static_cast<int>(blockIdx.x) / bh;
    const int rem = static_cast<int>(blockIdx.x) % bh;
    const int h = rem % p.Hq, b = rem / p.Hq, hk = h / p.group;
    const int shift = p.Sk - p.Sq;
    int q0t[2], n_t[2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        q0t[t] = pair * 2 * kTileM + t * kTileM;
        int kv_end = p.causal ? min(p.Sk, q0t[t] + kTileM + shift) : p.Sk;
        n_t[t] = (q0t[t] < p.Sq && kv_end > 0) ? (kv_end + kTileN - 1) / kTileN : 0;
    }
    const int n_max = max(n_t[0], n_t[1]);

    if (tid == 0) {
        mbar_init(bar_q(0), 1);
        mbar_init(bar_q(1), 1);
        for (int s = 0; s < NS; ++s) {
            mbar_init(bar_kv_full(s), 1);
            mbar_init(bar_kv_empty(s), 1);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(bar_s_full(t), 1);
            mbar_init(bar_p_full(t), 4);      // one arrival per softmax warp
            mbar_init(bar_o_full(t), 1);
            mbar_init(bar_scale(t), 4);
            mbar_init(bar_o_rescaled(t), 4);  // one arrival per correction warp
            mbar_init(bar_final(t), 4);
            for (int w = 0; w < 4; ++w) mbar_init(bar_turn(t, w), 1);
        }
        *abort_flag = (*reinterpret_cast<volatile int*>(p.status) != 0);
        fence_mbar_init();
    }
    constexpr uint32_t kTmemCols = 512;
    if (warp == 12) {
        tmem_alloc(smem_u32(tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    auto tmem_S = [&](int t) { return tmem + 128u * t; };
    auto tmem_O = [&](int t) { return tmem + 256u + 128u * t; };

    constexpr uint32_t fmt_ab = FP8 ? kFmtE4M3 : kFmtBF16;
    constexpr uint32_t fmt_p = FP8 ? (MODE == kExact ? kFmtE4M3 : kFmtE5M2) : kFmtBF16;
    constexpr uint32_t idesc_s = umma_idesc(fmt_ab, fmt_ab, false, false, kTileM, kTileN);
    constexpr uint32_t idesc_pv = umma_idesc(fmt_p, fmt_ab, false, true, kTileM, D);
    constexpr float p_off = static_cast<float>(PFormat<FP8, MODE>::kOffLog2);  // log2 of the P / row-sum scale

    if (wg == 3) {
        reg_dec_48();
        if (warp == 13 && lane == 0) {
            // ------------------------------------------------------------ TMA producer
            auto load_tile = [&](const CUtensorMap* tm, uint32_t dst, uint32_t bar, int head, int row0) {
                mbar_arrive_expect_tx(bar, C::kTileBytes);
#pragma unroll
                for (int bx = 0; bx < C::kBoxes; ++bx)
                    tma_load_4d(dst + bx * C::kBoxBytes, tm, bar, bx * C::kBoxElems, head, row0, b);
            };
            if (!*abort_flag) {
                if (n_t[0] > 0) load_tile(&tmQ, sQ, bar_q(0), h, q0t[0]);
                for (int j = 0; j < n_max; ++j) {
#pragma unroll
                    for (int kv = 0; kv < 2; ++kv) {
                        const int idx = 2 * j + kv, slot = idx % NS, use = idx / NS;
                        mbar_wait(bar_kv_empty(slot), (use & 1) ^ 1, wctx, (kRoleLoad << 8) | kBarKvEmpty);
                        if (*abort_flag) break;
                        load_tile(kv == 0 ? &tmK : &tmV, sRing + slot * C::kTileBytes, bar_kv_full(slot), hk, j * kTileN);
                        if (j == 0 && kv == 0 && n_t[1] > 0) load_tile(&tmQ, sQ + C::kTileBytes, bar_q(1), h, q0t[1]);
                    }
                }
            }
        } else if (warp == 12) {
            // ------------------------------------------------------------ MMA issuer
            // The whole warp walks the loop (so addresses and descriptors stay warp-uniform values);
            // one elected lane issues the MMAs and commits.
            const bool leader = elect_one();
            constexpr uint32_t desc_hi = umma_desc_hi_sw128(1024);
            const uint32_t q_lo0 = umma_desc_lo(sQ, 16);
            const uint32_t ring_lo_k = umma_desc_lo(sRing, 16);               // K tiles: K-major
            const uint32_t ring_lo_v = umma_desc_lo(sRing, C::kBoxBytes);     // V tiles: MN-major, LBO = next 128-byte column block
            constexpr uint32_t kTileLo = C::kTileBytes >> 4;
            auto issue_s = [&](int t, uint32_t k_lo) {
                const uint32_t q_lo = q_lo0 + t * kTileLo;
#pragma unroll
                for (int ks = 0; ks < C::kQkSteps; ++ks) {
                    const uint32_t off = ((ks / 4) * C::kBoxBytes + (ks % 4) * 32) >> 4;
                    umma_ss_lo<FP8>(tmem_S(t), q_lo + off, k_lo + off, desc_hi, idesc_s, ks > 0 ? 1u : 0u);
                }
            };
            auto issue_pv = [&](int t, uint32_t v_lo, bool accumulate) {
#pragma unroll
                for (int ks = 0; ks < C::kPvSteps; ++ks) {
                    const uint32_t off = (ks * C::kUmmaK * 128) >> 4;
                    umma_ts_lo<FP8>(tmem_O(t), tmem_S(t) + ks * 8, v_lo + off, desc_hi, idesc_pv,
                                    (accumulate || ks > 0) ? 1u : 0u);
                }
            };
            auto slot_lo = [&](int idx) { return static_cast<uint32_t>(idx % NS) * kTileLo; };
            auto wait_full = [&](int idx) {
                mbar_wait(bar_kv_full(idx % NS), (idx / NS) & 1, wctx, (kRoleMma << 8) | kBarKvFull);
            };
            if (n_max > 0) {
                wait_full(0);
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    if (n_t[t] > 0) {
                        mbar_wait(bar_q(t), 0, wctx, (kRoleMma << 8) | kBarQ);
                        // Stagger the two query tiles: tile 1 starts once tile 0's first P is done, which
                        // spreads the two tiles' softmax phases apart for the first iterations.
                        if (kStagger && t == 1 && n_t[0] > 0)
                            mbar_wait(bar_p_full(0), 0, wctx, (kRoleMma << 8) | kBarPFull);
                        tc_fence_after();
                        if (leader) {
                            if (!*abort_flag) issue_s(t, ring_lo_k + slot_lo(0));
                            umma_commit(bar_s_full(t));
                        }
                    }
                }
                if (leader) umma_commit(bar_kv_empty(0));
                for (int j = 0; j < n_max; ++j) {
                    wait_full(2 * j + 1);
                    bool k_ready = false;
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        if (j < n_t[t]) {
                            mbar_wait(bar_p_full(t), j & 1, wctx, (kRoleMma << 8) | kBarPFull);
                            if (leader) ROWMAX_STAMP(3, j, t * 4 + 0);
                            mbar_wait(bar_o_rescaled(t), j & 1, wctx, (kRoleMma << 8) | kBarORescaled);
                            if (leader) ROWMAX_STAMP(3, j, t * 4 + 1);
                            tc_fence_after();
                            if (leader) {
                                if (!*abort_flag) issue_pv(t, ring_lo_v + slot_lo(2 * j + 1), j > 0);
                                umma_commit(bar_o_full(t));
                                ROWMAX_STAMP(3, j, t * 4 + 2);
                            }
                        }
                        if (j + 1 < n_t[t]) {
                            if (!k_ready) {
                                wait_full(2 * j + 2);
                                tc_fence_after();
                                k_ready = true;
                            }
                            if (leader) {
                                if (!*abort_flag) issue_s(t, ring_lo_k + slot_lo(2 * j + 2));
                                umma_commit(bar_s_full(t));
                                ROWMAX_STAMP(3, j, t * 4 + 3);
                            }
                        }
                    }
                    if (leader) {
                        umma_commit(bar_kv_empty((2 * j + 1) % NS));
                        if (j + 1 < n_max) umma_commit(bar_kv_empty((2 * j + 2) % NS));
                    }
                    __syncwarp();
                }
            }
        }
    } else if (wg == 2) {
        // ---------------------------------------------------------------- correction + epilogue
        reg_dec_80();
        const int r = tid & 127;
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        for (int j = 0; j < n_max; ++j) {
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                if (j < n_t[t]) {
                    mbar_wait(bar_scale(t), j & 1, wctx, (kRoleCorr << 8) | kBarScale);
                    if (r == 0) ROWMAX_STAMP(2, j, t * 4 + 0);
                    const float alpha = sScale[t * 128 + r];
                    if (j > 0) {
                        mbar_wait(bar_o_full(t), (j - 1) & 1, wctx, (kRoleCorr << 8) | kBarOFull);
                        if (r == 0) ROWMAX_STAMP(2, j, t * 4 + 1);
                        __syncwarp();
                        tc_fence_after();
                        if (__any_sync(0xffffffffu, alpha != 1.0f)) {
#pragma unroll
                            for (int cc = 0; cc < D / 32; ++cc) {
                                uint32_t o[32];
                                tmem_ld32(tmem_O(t) + lane_base + cc * 32, o);
                                tmem_wait_ld();
#pragma unroll
                                for (int i = 0; i < 32; i += 2) {
                                    const float2 v = fmul2(make_float2(__uint_as_float(o[i]), __uint_as_float(o[i + 1])),
                                                           make_float2(alpha, alpha));
                                    o[i] = __float_as_uint(v.x);
                                    o[i + 1] = __float_as_uint(v.y);
                                }
                                tmem_st32(tmem_O(t) + lane_base + cc * 32, o);
                            }
                            tmem_wait_st();
                        }
                        tc_fence_before();
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_o_rescaled(t));
                    if (r == 0) ROWMAX_STAMP(2, j, t * 4 + 2);
                }
            }
        }
        // epilogue: O = v_descale * acc / l (undoing the P offset), LSE = ln2 * (m c + log2 l)
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const int row = q0t[t] + r;
            if (q0t[t] >= p.Sq) continue;
            float l_run = 0.f, m_run = -INFINITY;
            if (n_t[t] > 0) {
                mbar_wait(bar_final(t), 0, wctx, (kRoleEpi << 8) | kBarFinal);
                const float2 lm = sFinal[t * 128 + r];
                l_run = lm.x;
                m_run = lm.y;
                mbar_wait(bar_o_full(t), (n_t[t] - 1) & 1, wctx, (kRoleEpi << 8) | kBarOFull);
                __syncwarp();
                tc_fence_after();
            }
            const bool has_keys = l_run > 0.f;
            const float inv = has_keys ? p.v_descale / l_run : 0.f;
            if (row < p.Sq && p.lse != nullptr) {
                const float lse = has_keys ? 0.6931471805599453f * (m_run * p.c + log2f(l_run) - p_off) : -INFINITY;
                p.lse[(static_cast<size_t>(b) * p.Hq + h) * p.Sq + row] = lse;
            }
            __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(p.o) +
                                  ((static_cast<size_t>(b) * p.Sq + row) * p.Hq + h) * D;
#pragma unroll
            for (int cc = 0; cc < D / 32; ++cc) {
                uint32_t o[32];
                if (n_t[t] > 0) {
                    tmem_ld32(tmem_O(t) + lane_base + cc * 32, o);
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
        }
    } else {
        // ---------------------------------------------------------------- softmax of query tile t
        reg_inc_192();
        const int t = wg;
        const int r = tid & 127;
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_S(t) + lane_base;
        const int q0 = t == 0 ? q0t[0] : q0t[1];
        const int nt = t == 0 ? n_t[0] : n_t[1];
        // The two softmax warps on one scheduler take turns on their arithmetic-heavy section, tile by
        // tile (0, 1, 0, 1, ...), so that each runs it alone and the two query tiles stay half a period
        // apart: while one warp computes weights, the other's MMAs and hand-offs are in flight.
        const int n_both = kTakeTurns ? min(n_t[0], n_t[1]) : 0;   // tiles for which both warps are active
        const int w4 = warp & 3;
        const int row = q0 + r;
        const int row_limit = p.causal ? min(p.Sk, row + shift + 1) : p.Sk;  // visible keys of this row
        // first key index that some row of this tile cannot see (tile-uniform)
        const int tile_limit = p.causal ? min(p.Sk, q0 + shift + 1) : p.Sk;
        const float c_eff = (MODE == kH15) ? 2.0f * p.c : p.c;
        float m_run = -INFINITY, l_run = 0.f;
        for (int j = 0; j < nt; ++j) {
            mbar_wait(bar_s_full(t), j & 1, wctx, (kRoleSoftmax << 8) | kBarSFull);
            if (t == 0) {
                if (j > 0 && j < n_both) mbar_wait(bar_turn(0, w4), (j - 1) & 1, wctx, (kRoleSoftmax << 8) | kBarTurn);
            } else {
                if (j < n_both) mbar_wait(bar_turn(1, w4), j & 1, wctx, (kRoleSoftmax << 8) | kBarTurn);
            }
            if (r == 0) ROWMAX_STAMP(t, j, 0);
            __syncwarp();
            tc_fence_after();
            uint32_t s[4][32];
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) tmem_ld32(tS + cc * 32, s[cc]);
            tmem_wait_ld();
            if (r == 0) ROWMAX_STAMP(t, j, 1);

            const bool masked_tile = (j + 1) * kTileN > tile_limit;
            const int col_limit = row_limit - j * kTileN;
            if (masked_tile) {
#pragma unroll
                for (int cc = 0; cc < 4; ++cc)
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (cc * 32 + i >= col_limit) s[cc][i] = __float_as_uint(-INFINITY);
            }
            const float m_t = row_max128(s);
            const float m_new = fmaxf(m_run, m_t);
            const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
            const float alpha = ex2_approx((m_run - m_use) * p.c);
            m_run = m_new;
            sScale[t * 128 + r] = alpha;
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_scale(t));
            if (r == 0) ROWMAX_STAMP(t, j, 2);

            // exact: x = s*c - m*c + P offset;  h15: doubled input 2x = s*(2c) - m*(2c);  pot: x = s*c - m*c
            RowScale rs;
            rs.c = make_float2(c_eff, c_eff);
            const float nmc = (MODE == kExact ? p_off : 0.0f) - m_use * c_eff;
            rs.nmc = make_float2(nmc, nmc);
            rs.two22 = p.two22;
            float2 acc[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
            if (masked_tile) {
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    uint32_t pw[16];
                    weights_chunk32<FP8, MODE, true>(s[cc], rs, col_limit - cc * 32, acc, pw);
                    if constexpr (FP8) tmem_st8(tS + cc * 8, pw);
                    else tmem_st16(tS + cc * 16, pw);
                }
            } else {
                // h15: the clamp at -252 is a no-op unless some score of the warp's rows lies more than
                // 126 octaves below its running maximum; the row minimum (one more three-input pass)
                // tells, and the common case runs without the per-score clamp.
                bool clamp = false;
                if constexpr (MODE == kH15) {
                    const float lowest = (row_min128(s) - m_use) * c_eff;   // smallest doubled offset of the row
                    clamp = __any_sync(0xffffffffu, !(lowest >= -250.0f));
                }
                if (clamp) {
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        uint32_t pw[16];
                        weights_chunk32<FP8, MODE, false, true>(s[cc], rs, 32, acc, pw);
                        if constexpr (FP8) tmem_st8(tS + cc * 8, pw);
                        else tmem_st16(tS + cc * 16, pw);
                    }
                } else {
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        uint32_t pw[16];
                        weights_chunk32<FP8, MODE, false, false>(s[cc], rs, 32, acc, pw);
                        if constexpr (FP8) tmem_st8(tS + cc * 8, pw);
                        else tmem_st16(tS + cc * 16, pw);
                    }
                }
            }
            const float l_tile = (acc[0].x + acc[0].y) + (acc[1].x + acc[1].y);
            if (r == 0) ROWMAX_STAMP(t, j, 3);
            __syncwarp();
            if (lane == 0) {   // pass the turn to the other tile's warp
                if (t == 0) {
                    if (j < n_both) mbar_arrive(bar_turn(1, w4));
                } else {
                    if (j + 1 < n_both) mbar_arrive(bar_turn(0, w4));
                }
            }
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_p_full(t));
            if (r == 0) ROWMAX_STAMP(t, j, 4);
            l_run = l_run * alpha + l_tile;
        }
        if (nt > 0) {
            sFinal[t * 128 + r] = make_float2(l_run, m_run);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_final(t));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 12) tmem_dealloc(tmem, kTmemCols);
}

// ------------------------------------------------------------------------------------------------
// Host launcher
// ------------------------------------------------------------------------------------------------
template <int D, bool FP8, int MODE>
static cudaError_t launch_ws(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                             const AttnParams& p, cudaStream_t stream) {
    using W = WsCfg<D, FP8>;
    auto kern = attn_fwd_ws_kernel<D, FP8, MODE>;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, W::kSmemBytes);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const long long n_pairs = (p.Sq + 2 * kTileM - 1) / (2 * kTileM);
    const long long blocks = n_pairs * p.Hq * p.B;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
    kern<<<static_cast<unsigned>(blocks), 512, W::kSmemBytes, stream>>>(tq, tk, tv, p);
    return cudaGetLastError();
}

template <int D, bool FP8>
static cudaError_t dispatch_mode(int mode, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                                 const AttnParams& p, cudaStream_t stream) {
    switch (mode) {
        case kExact: return launch_ws<D, FP8, kExact>(tq, tk, tv, p, stream);
        case kPot: return launch_ws<D, FP8, kPot>(tq, tk, tv, p, stream);
        default: return launch_ws<D, FP8, kH15>(tq, tk, tv, p, stream);
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
__global__ void weight_map_kernel(const float* __restrict__ x, float* __restrict__ w, size_t n, int mode,
                                  uint32_t two22) {
    const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
    for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += stride) {
        const float xi = x[i];
        float wi;
        if (mode == kExact) wi = w_exact(xi);
        else if (mode == kPot) wi = w_pot(xi);
        else wi = w_h15_doubled_pair<0>(make_float2(xi * 2.0f, xi * 2.0f), two22).x;
        w[i] = wi;
    }
}

cudaError_t launch_weight_map(const float* x, float* w, size_t n, int mode, cudaStream_t stream) {
    if (n == 0) return cudaSuccess;
    const int threads = 256;
    size_t blocks = (n + threads - 1) / threads;
    if (blocks > 148 * 8) blocks = 148 * 8;
    weight_map_kernel<<<static_cast<unsigned>(blocks), threads, 0, stream>>>(x, w, n, mode, 1u << 22);
    return cudaGetLastError();
}

__device__ int g_attn_status = 0;

cudaError_t status_word_address(int** out) {
    return cudaGetSymbolAddress(reinterpret_cast<void**>(out), g_attn_status);
}

}  // namespace rowmax
