// Fused attention forward for sm_100a: TMA-staged Q/K/V tiles, tcgen05 MMAs with TMEM accumulators,
// online softmax with a selectable weight map (exact / Rowmax-PoT / Rowmax-H15), bf16 O + fp32 LSE.
//
// Loop structure per query tile (Sec. 5.2; App. B.1): for each key tile in ascending order
//   S = Q K^T -> tile row maximum -> running maximum m (always adopted, threshold 0) ->
//   x = s*c - m*c -> weight map -> row sum l and P (same weights) -> O = alpha*O + P V;
// at the end O = v_descale * O / l and LSE = ln2 * (m*c + log2 l).
//
// Persistent grid: one CTA (16 warps) per SM walks work items, each a pair of query tiles of 128 rows
// of one (batch, head) whose key tiles it visits once, so every K/V tile staged in shared memory
// feeds four MMAs:
//   warpgroup 0/1  softmax of query tile 0/1: one thread per row (no shuffles needed: a thread
//                  reads its whole score row from TMEM), weight map, row sum, P written back to
//                  TMEM over the S columns; after the last key tile the epilogue of its rows
//   warpgroup 2    correction: rescales the O accumulators in TMEM when a running maximum moved
//   warp 12        MMA issuer (one thread): S_t = Q_t K^T and O_t += P_t V on the tensor cores
//   warp 13        TMA producer (one thread): Q per item, K/V through a ring of shared-memory slots
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
    static constexpr int kBarOff = kScaleOff + 2 * 128 * 4;
    static constexpr int kNumBars = 2 * kSlots + 8 * 2 + 1;
    static constexpr int kMiscOff = kBarOff + kNumBars * 8;
    static constexpr int kSmemBytes = kMiscOff + 16 + 1024;       // + manual 1024-byte alignment slack
    static_assert(kSmemBytes <= 232448, "exceeds the 227 KB shared memory of an sm_100 CTA");
};

// Register split of the 512 threads x 128 registers the CTA is launched with (setmaxnreg can only
// redistribute that allocation; a larger total would make the increase wait for ever): softmax /
// correction / MMA+TMA warpgroups.
constexpr int kRegSoftmax = 192, kRegCorr = 80, kRegMma = 48;
static_assert(256 * kRegSoftmax + 128 * kRegCorr + 128 * kRegMma <= 512 * 128, "setmaxnreg targets exceed the launch allocation");
template <int N> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }

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

// Tile 1 of a CTA's first work item starts once tile 0's first P is done, which spreads the two
// tiles' softmax phases apart for the first iterations.
constexpr bool kStagger = true;

constexpr int kBarSelftest = 0x7F;
enum BarId : int { kBarQFull = 0, kBarQEmpty = 1, kBarKvFull = 2, kBarKvEmpty = 3, kBarSFull = 4, kBarPFull = 5,
                   kBarOFull = 6, kBarScale = 7, kBarORescaled = 8, kBarOFree = 9 };

// One work item = two query tiles of 128 rows of one (batch, head).
struct WorkItem {
    int h, b, hk;
    int q0[2];   // first query row of each tile
    int n[2];    // key tiles of each tile (0: the tile is out of range or sees no key)
    int n_max;
};

// Items are numbered heaviest first (under a causal mask the last query tiles have the most key
// tiles).  CTA c of G walks them in a snake: round k takes item k*G + c (k even) or k*G + G-1-c (k odd),
// so every CTA gets one item of each weight class and the loads even out without a global counter.
__device__ __forceinline__ int item_index(int round, int cta, int n_ctas) {
    return round * n_ctas + ((round & 1) ? (n_ctas - 1 - cta) : cta);
}
__device__ __forceinline__ WorkItem decode_item(int w, const AttnParams& p, int n_pairs, int bh) {
    WorkItem it;
    const int pair = n_pairs - 1 - w / bh;
    const int rem = w % bh;
    it.h = rem % p.Hq;
    it.b = rem / p.Hq;
    it.hk = it.h / p.group;
    const int shift = p.Sk - p.Sq;
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        it.q0[t] = pair * 2 * kTileM + t * kTileM;
        const int kv_end = p.causal ? min(p.Sk, it.q0[t] + kTileM + shift) : p.Sk;
        it.n[t] = (it.q0[t] < p.Sq && kv_end > 0) ? (kv_end + kTileN - 1) / kTileN : 0;
    }
    it.n_max = max(it.n[0], it.n[1]);
    return it;
}

}  // namespace

// IN: storage type of q, k, v (kInBF16 / kInFP8 / kInFP16).  P has the type of V at 16 bits (the f16
// kind wants both MMA operands in one format) and one of the two fp8 formats at 8 bits.
template <int D, int IN, int MODE>
__global__ void __launch_bounds__(512, 1)
attn_fwd_ws_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
    constexpr bool FP8 = IN == kInFP8;
    constexpr bool HALF = IN == kInFP16;
    using C = TileCfg<D, FP8>;
    using W = WsCfg<D, FP8>;
    constexpr int NS = W::kSlots;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const uint32_t sQ = smem_u32(smem);
    const uint32_t sRing = sQ + W::kQBytes;
    float* sScale = reinterpret_cast<float*>(smem + W::kScaleOff);
    const uint32_t bar0 = smem_u32(smem + W::kBarOff);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + W::kMiscOff);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + W::kMiscOff + 4);
    const WaitCtx wctx{abort_flag, p.status, kWaitLimitCycles};

    // barrier addresses
    auto bar_kv_full = [&](int s) { return bar0 + 8u * s; };
    auto bar_kv_empty = [&](int s) { return bar0 + 8u * (NS + s); };
    auto bar_x = [&](int which, int t) { return bar0 + 8u * (2 * NS + 2 * which + t); };
    auto bar_q_full = [&](int t) { return bar_x(0, t); };      // TMA -> MMA: Q_t of the current item landed
    auto bar_q_empty = [&](int t) { return bar_x(1, t); };     // MMA -> TMA: last S_t MMA of the item done
    auto bar_s_full = [&](int t) { return bar_x(2, t); };      // MMA -> softmax: S_t(j) is in TMEM
    auto bar_p_full = [&](int t) { return bar_x(3, t); };      // softmax -> MMA: P_t(j) is in TMEM
    auto bar_o_full = [&](int t) { return bar_x(4, t); };      // MMA -> correction / epilogue: P_t V(j) accumulated
    auto bar_scale = [&](int t) { return bar_x(5, t); };       // softmax -> correction: alpha_t(j) in smem
    auto bar_o_rescaled = [&](int t) { return bar_x(6, t); };  // correction -> MMA: O_t rescaled for tile j
    auto bar_o_free = [&](int t) { return bar_x(7, t); };      // epilogue -> MMA: O_t has been read out
    const uint32_t bar_drain = bar0 + 8u * (2 * NS + 16);      // abort path only: the MMA warp's last commit

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, wg = warp >> 2;
    // The status word is sticky: once a wait has expired (in an earlier launch, or in another CTA of this one) and
    // until the host clears it, a CTA that starts is a no-op: it touches neither its outputs nor TMEM nor TMA.
    // One thread reads the word so that the whole CTA takes the same way.
    if (tid == 0) *abort_flag = (*reinterpret_cast<volatile int*>(p.status) != 0);
    __syncthreads();
    if (*abort_flag) return;
#ifdef ROWMAX_TRACE
    const long long trace_t0 = clock64();
#endif
    if (tid == 256) ROWMAX_STAMP(2, 63, 0);

    const int n_pairs = (p.Sq + 2 * kTileM - 1) / (2 * kTileM);
    const int bh = p.Hq * p.B;
    const int n_items = n_pairs * bh;
    const int cta = blockIdx.x, n_ctas = gridDim.x;
    const int shift = p.Sk - p.Sq;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(bar_kv_full(s), 1);
            mbar_init(bar_kv_empty(s), 1);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(bar_q_full(t), 1);
            mbar_init(bar_q_empty(t), 1);
            mbar_init(bar_s_full(t), 1);
            mbar_init(bar_p_full(t), 4);      // one arrival per softmax warp
            mbar_init(bar_o_full(t), 1);
            mbar_init(bar_scale(t), 4);
            mbar_init(bar_o_rescaled(t), 4);  // one arrival per correction warp
            mbar_init(bar_o_free(t), 4);      // one arrival per softmax warp (epilogue)
        }
        mbar_init(bar_drain, 1);
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
    if (tid == 256) ROWMAX_STAMP(2, 63, 1);
    auto tmem_S = [&](int t) { return tmem + 128u * t; };
    auto tmem_O = [&](int t) { return tmem + 256u + 128u * t; };

    constexpr uint32_t fmt_16 = HALF ? kFmtF16 : kFmtBF16;
    constexpr uint32_t fmt_ab = FP8 ? kFmtE4M3 : fmt_16;
    constexpr uint32_t fmt_p = FP8 ? (PFormat<FP8, MODE>::kE4M3 ? kFmtE4M3 : kFmtE5M2) : fmt_16;
    constexpr uint32_t idesc_s = umma_idesc(fmt_ab, fmt_ab, false, false, kTileM, kTileN);
    constexpr uint32_t idesc_pv = umma_idesc(fmt_p, fmt_ab, false, true, kTileM, D);
    constexpr float p_off = static_cast<float>(PFormat<FP8, MODE>::kOffLog2);  // log2 of the P / row-sum scale

    if (wg == 3) {
        reg_dec<kRegMma>();
        if (warp == 13 && lane == 0) {
            // ------------------------------------------------------------ TMA producer
            int kv_idx = 0;             // K/V tiles loaded so far (ring position), over all items
            int q_use[2] = {0, 0};      // items that used Q buffer t so far
            for (int round = 0;; ++round) {
                const int w = item_index(round, cta, n_ctas);
                if (w >= n_items || *abort_flag) break;
                const WorkItem it = decode_item(w, p, n_pairs, bh);
                auto load_tile = [&](const CUtensorMap* tm, uint32_t dst, uint32_t bar, int head, int row0) {
                    mbar_arrive_expect_tx(bar, C::kTileBytes);
#pragma unroll
                    for (int bx = 0; bx < C::kBoxes; ++bx)
                        tma_load_4d(dst + bx * C::kBoxBytes, tm, bar, bx * C::kBoxElems, head, row0, it.b);
                };
                // After an expired wait nothing more is loaded: a wait then returns at once, and a copy into a buffer
                // whose last copy may still be under way would leave more in flight than the waits below account for.
                auto load_q = [&](int t) {
                    if (it.n[t] > 0) {
                        mbar_wait(bar_q_empty(t), (q_use[t] & 1) ^ 1, wctx, (kRoleLoad << 8) | kBarQEmpty);
                        if (*abort_flag) return;
                        load_tile(&tmQ, sQ + t * C::kTileBytes, bar_q_full(t), it.h, it.q0[t]);
                        ++q_use[t];
                    }
                };
                if (round == 0) ROWMAX_STAMP(3, 63, 0);
                load_q(0);
                for (int j = 0; j < it.n_max && !*abort_flag; ++j) {
#pragma unroll
                    for (int kv = 0; kv < 2; ++kv) {
                        const int slot = kv_idx % NS, use = kv_idx / NS;
                        mbar_wait(bar_kv_empty(slot), (use & 1) ^ 1, wctx, (kRoleLoad << 8) | kBarKvEmpty);
                        if (*abort_flag) break;
                        load_tile(kv == 0 ? &tmK : &tmV, sRing + slot * C::kTileBytes, bar_kv_full(slot), it.hk,
                                  j * kTileN);
                        ++kv_idx;
                        if (j == 0 && kv == 0) load_q(1);
                    }
                }
                if (it.n_max == 0) load_q(1);
            }
            // Before the CTA ends every load this thread issued must have landed.  Normally the consumers have
            // seen to that and these waits return at once; after an expired wait they may have stopped waiting while
            // copies were still writing shared memory, so wait (bounded) for the last use of every ring slot and
            // Q buffer.
            for (int idx = kv_idx > NS ? kv_idx - NS : 0; idx < kv_idx; ++idx)
                mbar_wait_quiet(bar_kv_full(idx % NS), (idx / NS) & 1, kDrainLimitCycles);
#pragma unroll
            for (int t = 0; t < 2; ++t)
                if (q_use[t] > 0) mbar_wait_quiet(bar_q_full(t), (q_use[t] - 1) & 1, kDrainLimitCycles);
        } else if (warp == 12) {
            // ------------------------------------------------------------ MMA issuer
            // The whole warp walks the loop (so addresses and descriptors stay warp-uniform values);
            // one elected lane issues the MMAs and commits.
            const bool leader = elect_one();
            constexpr uint32_t desc_hi = umma_desc_hi_sw(C::kSwizzle);
            const uint32_t q_lo0 = umma_desc_lo(sQ, 16);
            const uint32_t ring_lo_k = umma_desc_lo(sRing, 16);               // K tiles: K-major
            const uint32_t ring_lo_v = umma_desc_lo(sRing, C::kBoxBytes);     // V tiles: MN-major, LBO = next 128-byte column block
            constexpr uint32_t kTileLo = C::kTileBytes >> 4;
            auto issue_s = [&](int t, uint32_t k_lo) {
                const uint32_t q_lo = q_lo0 + t * kTileLo;
#pragma unroll
                for (int ks = 0; ks < C::kQkSteps; ++ks) {
                    const uint32_t off = ((ks / C::kStepsPerBox) * C::kBoxBytes + (ks % C::kStepsPerBox) * 32) >> 4;
                    umma_ss_lo<FP8>(tmem_S(t), q_lo + off, k_lo + off, desc_hi, idesc_s, ks > 0 ? 1u : 0u);
                }
            };
            auto issue_pv = [&](int t, uint32_t v_lo, bool accumulate) {
#pragma unroll
                for (int ks = 0; ks < C::kPvSteps; ++ks) {
                    const uint32_t off = (ks * C::kUmmaK * C::kSwizzle) >> 4;   // kUmmaK keys down the MN-major V tile
                    umma_ts_lo<FP8>(tmem_O(t), tmem_S(t) + ks * 8, v_lo + off, desc_hi, idesc_pv,
                                    (accumulate || ks > 0) ? 1u : 0u);
                }
            };
            auto slot_lo = [&](int idx) { return static_cast<uint32_t>(idx % NS) * kTileLo; };
            auto wait_full = [&](int idx) {
                mbar_wait(bar_kv_full(idx % NS), (idx / NS) & 1, wctx, (kRoleMma << 8) | kBarKvFull);
            };
            int kv_base = 0;            // ring index of K_0 of the current item
            int tiles[2] = {0, 0};      // key tiles of query tile t finished in earlier items (barrier phases)
            int q_use[2] = {0, 0};      // items that used Q buffer / O accumulator t so far
            for (int round = 0;; ++round) {
                const int w = item_index(round, cta, n_ctas);
                if (w >= n_items) break;
                const WorkItem it = decode_item(w, p, n_pairs, bh);
                if (it.n_max > 0) {
                    wait_full(kv_base);
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        if (it.n[t] > 0) {
                            mbar_wait(bar_q_full(t), q_use[t] & 1, wctx, (kRoleMma << 8) | kBarQFull);
                            if (kStagger && round == 0 && t == 1 && it.n[0] > 0)
                                mbar_wait(bar_p_full(0), 0, wctx, (kRoleMma << 8) | kBarPFull);
                            tc_fence_after();
                            if (leader) {
                                if (round == 0) ROWMAX_STAMP(3, 63, 1 + t);
                                if (!*abort_flag) issue_s(t, ring_lo_k + slot_lo(kv_base));
                                umma_commit(bar_s_full(t));
                                if (it.n[t] == 1) umma_commit(bar_q_empty(t));
                            }
                        }
                    }
                    if (leader) umma_commit(bar_kv_empty(kv_base % NS));
                    for (int j = 0; j < it.n_max; ++j) {
                        // Everything the next MMAs need besides P is awaited first (it is normally there long
                        // before), so that once P_t(j) arrives the P V and next-S MMAs go out back to back.  (The flag
                        // is read here, off that path: if one of the waits below expires, this step's MMAs still go
                        // out, on stale operands; nothing is stored after that and the MMAs are awaited at the end.)
                        const bool ok = !*abort_flag;
                        wait_full(kv_base + 2 * j + 1);
                        if (j + 1 < it.n_max) wait_full(kv_base + 2 * j + 2);
#pragma unroll
                        for (int t = 0; t < 2; ++t) {
                            if (j < it.n[t]) {
                                const uint32_t ph = (tiles[t] + j) & 1;
                                mbar_wait(bar_o_rescaled(t), ph, wctx, (kRoleMma << 8) | kBarORescaled);
                                // the accumulator of the previous item must have been read out
                                if (j == 0) mbar_wait(bar_o_free(t), (q_use[t] & 1) ^ 1, wctx, (kRoleMma << 8) | kBarOFree);
                                mbar_wait(bar_p_full(t), ph, wctx, (kRoleMma << 8) | kBarPFull);
                                if (leader) ROWMAX_STAMP(3, j, t * 4 + 0);
                                tc_fence_after();
                                if (leader) {
                                    if (ok) issue_pv(t, ring_lo_v + slot_lo(kv_base + 2 * j + 1), j > 0);
                                    umma_commit(bar_o_full(t));
                                    ROWMAX_STAMP(3, j, t * 4 + 2);
                                    if (j + 1 < it.n[t]) {
                                        if (ok) issue_s(t, ring_lo_k + slot_lo(kv_base + 2 * j + 2));
                                        umma_commit(bar_s_full(t));
                                        if (j + 2 == it.n[t]) umma_commit(bar_q_empty(t));   // last S of this item
                                        ROWMAX_STAMP(3, j, t * 4 + 3);
                                    }
                                }
                            }
                        }
                        if (leader) {
                            umma_commit(bar_kv_empty((kv_base + 2 * j + 1) % NS));
                            if (j + 1 < it.n_max) umma_commit(bar_kv_empty((kv_base + 2 * j + 2) % NS));
                        }
                        __syncwarp();
                    }
                }
                kv_base += 2 * it.n_max;
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    tiles[t] += it.n[t];
                    if (it.n[t] > 0) ++q_use[t];
                }
            }
            // No MMA of this thread may still be running when TMEM is handed back: one last commit, awaited with a
            // bound (it arrives at once unless a wait expired and the roles left their loops early).
            if (leader) umma_commit(bar_drain);
            mbar_wait_quiet(bar_drain, 0, kDrainLimitCycles);
        }
    } else if (wg == 2) {
        // ---------------------------------------------------------------- correction
        reg_dec<kRegCorr>();
        const int r = tid & 127;
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        int tiles[2] = {0, 0};
        for (int round = 0;; ++round) {
            const int w = item_index(round, cta, n_ctas);
            if (w >= n_items) break;
            const WorkItem it = decode_item(w, p, n_pairs, bh);
            for (int j = 0; j < it.n_max; ++j) {
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    if (j < it.n[t]) {
                        mbar_wait(bar_scale(t), (tiles[t] + j) & 1, wctx, (kRoleCorr << 8) | kBarScale);
                        if (r == 0) ROWMAX_STAMP(2, j, t * 4 + 0);
                        const float alpha = sScale[t * 128 + r];
                        if (j > 0) {
                            mbar_wait(bar_o_full(t), (tiles[t] + j - 1) & 1, wctx, (kRoleCorr << 8) | kBarOFull);
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
            tiles[0] += it.n[0];
            tiles[1] += it.n[1];
        }
    } else {
        // ---------------------------------------------------------------- softmax + epilogue of query tile t
        reg_inc<kRegSoftmax>();
        const int t = wg;
        const int r = tid & 127;
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_S(t) + lane_base;
        const uint32_t tO = tmem_O(t) + lane_base;
        constexpr int kFam = h15_family_k(MODE);   // h15 family: the map takes the offset times 2^kFam
        const float c_eff = static_cast<float>(1 << kFam) * p.c;
        // 16-bit inputs: the h15 family uses the saturating form of weights_chunk32 (no row-minimum pass, no
        // clamped or masked variants) whenever the anchor is always current (offsets <= 0); the deferred rescale,
        // where a score may lie above its anchor, keeps the form with explicit clamps.  fp8 inputs keep the
        // packed form: there a bound on the key magnitude already removes the row-minimum pass, and the
        // scalar multiply-adds of the saturating form cost more issue slots than they save (measured 4 to 6 %).
        constexpr bool kLattice = kFam > 0 && !FP8;
        const bool sat_form = kLattice && (IN != kInBF16 || !(p.tau > 0.0f));
        int tiles = 0;
        for (int round = 0;; ++round) {
            const int w = item_index(round, cta, n_ctas);
            if (w >= n_items) break;
            const WorkItem it = decode_item(w, p, n_pairs, bh);
            const int q0 = t == 0 ? it.q0[0] : it.q0[1];
            const int nt = t == 0 ? it.n[0] : it.n[1];
            const int row = q0 + r;
            const int row_limit = p.causal ? min(p.Sk, row + shift + 1) : p.Sk;  // visible keys of this row
            // first key index that some row of this tile cannot see (tile-uniform)
            const int tile_limit = p.causal ? min(p.Sk, q0 + shift + 1) : p.Sk;
            float m_run = -INFINITY, l_run = 0.f;
            // h15 family at fp8: a lower bound of every raw score of this row that costs nothing per score.
            // |q . k| <= (sum_i |q_i|) * max_i |k_i| and an e4m3 key element is at most 448 in magnitude, so
            // s >= -448 * sum_i |q_i|.  When that bound already keeps the scaled offsets of a tile above the
            // clamp, the tile needs neither the row-minimum pass nor the clamped variant.  The row of Q is
            // read from shared memory (a sum does not care about the swizzle, which stays within the row), which
            // is safe while S_t(1) has not been issued, i.e. for items with at least two key tiles (used from four on).
            float score_floor = -INFINITY;
            if constexpr (FP8 && kFam > 0) {
                if (nt >= 4) {   // the sum costs about three row-minimum passes
                    mbar_wait(bar_s_full(t), tiles & 1, wctx, (kRoleSoftmax << 8) | kBarSFull);   // Q_t has landed
                    score_floor = -448.0f * 1.02f * abs_sum_e4m3_row<D / 16>(sQ + t * C::kTileBytes + r * D);
                }
            }
            for (int j = 0; j < nt; ++j) {
                mbar_wait(bar_s_full(t), (tiles + j) & 1, wctx, (kRoleSoftmax << 8) | kBarSFull);
                if (r == 0) ROWMAX_STAMP(t, j, 0);
                __syncwarp();
                tc_fence_after();
                uint32_t s[4][32];
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) tmem_ld32(tS + cc * 32, s[cc]);
                tmem_wait_ld();
                if (r == 0) ROWMAX_STAMP(t, j, 1);

                // Masked scores are set to -inf.  exact: their weight is then 0 by itself.  h15 family: a masked
                // tile takes the clamped variant with the clamp one octave lower, at the input whose
                // weight pattern is +0 (there a real score more than 126 octaves below its anchor also weighs 0,
                // or a denormal, instead of 2^-126: nothing against a row sum >= 1).  pot and the partly emulated
                // exact mode zero the masked weights explicitly (pot's floor 2^-20 is not nothing, and the
                // polynomial route does not take -inf).  Keeping a masked variant out of the common modes
                // makes their hot loop markedly faster.
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
                // The tile maximum becomes the new anchor when there is none yet or when it exceeds the
                // anchor by more than tau octaves (tau = 0: always, so the anchor is the running maximum).
                const bool adopt = (m_run == -INFINITY) || ((m_t - m_run) * p.c > p.tau);
                const float m_new = adopt ? fmaxf(m_run, m_t) : m_run;
                const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
                const float alpha = ex2_approx((m_run - m_use) * p.c);
                m_run = m_new;
                // exact-like modes post the rescale factor after the first 32 weights are under way, so that its
                // special-function latency, the shared-memory store and the arrival hide behind them (measured +2 %);
                // their weight phase is long enough for the correction warps to rescale O in what is left of it.  The
                // rounding maps post it at once: their weight phase is shorter, and posting late put the correction on
                // the critical path (measured 5 to 8 % slower).
                constexpr bool kPostLate = is_exact_like(MODE);
                auto post_alpha_now = [&]() {
                    sScale[t * 128 + r] = alpha;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_scale(t));
                    if (r == 0) ROWMAX_STAMP(t, j, 2);
                };
                auto post_alpha = [&]() { if constexpr (kPostLate) post_alpha_now(); };
                if constexpr (!kPostLate) post_alpha_now();

                // exact: x = s*c - m*c + P offset;  h15 family: scaled input 2^K x = s*(2^K c) - m*(2^K c);  pot: x = s*c - m*c
                RowScale rs;
                float nmc = (is_exact_like(MODE) ? p_off : 0.0f) - m_use * c_eff;
                float c_row = c_eff;
                rs.c = make_float2(c_row, c_row);
                rs.nmc = make_float2(nmc, nmc);
                rs.two22 = p.two22;
                rs.pot_neg_cap = p.pot_neg_cap;
                rs.pot_drop_x = p.pot_drop_x;
                rs.clamp_lo = 0.f;
                if constexpr (kFam > 0) rs.clamp_lo = masked_tile ? h15_clamp_zero<kFam>() : h15_clamp_floor<kFam>();
                float2 acc[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                if (kLattice && sat_form) {
                    // distance below the anchor as a fraction of the clamp distance R, which is also where a masked
                    // score (-inf) ends up: 2^K * 126 (weight floor 2^-126, Eq. h15), in a tile with masked scores
                    // 2^K * 127 (pattern of +0)
                    constexpr float kR = 126.0f * (1 << kFam), kRm = 127.0f * (1 << kFam);
                    const float big_r = masked_tile ? kRm : kR;
                    const float inv_r = masked_tile ? 1.0f / kRm : 1.0f / kR;
                    rs.su = -c_eff * inv_r;
                    rs.ou = (m_use * c_eff) * inv_r;
                    rs.sat_mul = -big_r;
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        uint32_t pw[16];
                        weights_chunk32<FP8, MODE, false, true, HALF, true>(s[cc], rs, 32, acc, pw);
                        tmem_st16(tS + cc * 16, pw);
                        if (cc == 0) post_alpha();
                    }
                } else if (is_pot(MODE) && masked_tile) {
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        uint32_t pw[16];
                        weights_chunk32<FP8, MODE, true, true, HALF>(s[cc], rs, col_limit - cc * 32, acc, pw);
                        if constexpr (FP8) tmem_st8(tS + cc * 8, pw);
                        else tmem_st16(tS + cc * 16, pw);
                        if (cc == 0) post_alpha();
                    }
                } else {
                    // h15: the clamp is a no-op unless some score of the warp's rows lies more than 126 octaves
                    // below its anchor; the row minimum (one more three-input pass) tells, and the common case
                    // runs without the per-score clamp.  A tile with masked scores always takes the clamp.
                    bool clamp = false;
                    if constexpr (kFam > 0) {
                        if (masked_tile) {
                            clamp = true;
                        } else if (!__all_sync(0xffffffffu, (score_floor - m_use) * c_eff >= -125.0f * (1 << kFam))) {
                            const float lowest = (row_min128(s) - m_use) * c_eff;   // smallest scaled offset of the row
                            clamp = __any_sync(0xffffffffu, !(lowest >= -125.0f * (1 << kFam)));
                        }
                    }
                    if (clamp) {
#pragma unroll
                        for (int cc = 0; cc < 4; ++cc) {
                            uint32_t pw[16];
                            weights_chunk32<FP8, MODE, false, true, HALF>(s[cc], rs, 32, acc, pw);
                            if constexpr (FP8) tmem_st8(tS + cc * 8, pw);
                            else tmem_st16(tS + cc * 16, pw);
                            if (cc == 0) post_alpha();
                        }
                    } else {
#pragma unroll
                        for (int cc = 0; cc < 4; ++cc) {
                            uint32_t pw[16];
                            weights_chunk32<FP8, MODE, false, false, HALF>(s[cc], rs, 32, acc, pw);
                            if constexpr (FP8) tmem_st8(tS + cc * 8, pw);
                            else tmem_st16(tS + cc * 16, pw);
                            if (cc == 0) post_alpha();
                        }
                    }
                }
                const float l_tile = (acc[0].x + acc[0].y) + (acc[1].x + acc[1].y);
                if (r == 0) ROWMAX_STAMP(t, j, 3);
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_p_full(t));
                if (r == 0) ROWMAX_STAMP(t, j, 4);
                l_run = l_run * alpha + l_tile;
            }

            // epilogue of this tile: O = v_descale * acc / l (the P offset cancels), LSE = ln2 * (m c + log2 l)
            if (q0 < p.Sq) {
                const bool has_keys = (m_run != -INFINITY) && l_run > 0.f;
                const float inv = has_keys ? p.v_descale / l_run : 0.f;
                const bool alive = !*abort_flag;      // after an expired wait the accumulators are not to be trusted: store nothing
                if (alive && row < p.Sq && p.lse != nullptr) {
                    const float lse = has_keys ? 0.6931471805599453f * (m_run * p.c + log2f(l_run) - p_off) : -INFINITY;
                    p.lse[(static_cast<size_t>(it.b) * p.Hq + it.h) * p.Sq + row] = lse;
                }
                if (nt > 0) {
                    mbar_wait(bar_o_full(t), (tiles + nt - 1) & 1, wctx, (kRoleEpi << 8) | kBarOFull);
                    __syncwarp();
                    tc_fence_after();
                }
                if (r == 0 && round == 0) ROWMAX_STAMP(2, 63, 2 + 2 * t);
                __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(p.o) +
                                      ((static_cast<size_t>(it.b) * p.Sq + row) * p.Hq + it.h) * D;
#pragma unroll
                for (int cc = 0; cc < D / 32; ++cc) {
                    uint32_t o[32];
                    if (nt > 0) {
                        tmem_ld32(tO + cc * 32, o);
                        tmem_wait_ld();
                        if (cc == D / 32 - 1) {   // the accumulator is in registers: the next item may overwrite it
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(bar_o_free(t));
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = 0;
                    }
                    if (alive && row < p.Sq) {
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
            tiles += nt;
        }
    }

    if (tid == 256) ROWMAX_STAMP(2, 63, 6);
    tc_fence_before();
    __syncthreads();
    if (tid == 256) ROWMAX_STAMP(2, 63, 7);
#ifdef ROWMAX_TRACE
    if (tid == 0 && p.trace != nullptr && p.trace_block < 0) p.trace[blockIdx.x] = clock64() - trace_t0;   // per-CTA busy time
#endif
    if (warp == 12) tmem_dealloc(tmem, kTmemCols);
}

// ------------------------------------------------------------------------------------------------
// Host launcher
// ------------------------------------------------------------------------------------------------
template <int D, int IN, int MODE>
static cudaError_t launch_ws(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                             const AttnParams& p, cudaStream_t stream) {
    using W = WsCfg<D, IN == kInFP8>;
    auto kern = attn_fwd_ws_kernel<D, IN, MODE>;
    // per-device launch set-up: the shared-memory opt-in of this instance and the SM count
    static bool configured[64] = {};
    static int sm_counts[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, W::kSmemBytes);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sm_counts[dev], cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    const int sm_count = sm_counts[dev];
    const long long n_pairs = (p.Sq + 2 * kTileM - 1) / (2 * kTileM);
    const long long items = n_pairs * p.Hq * p.B;
    if (items > 0x7fffffffLL) return cudaErrorInvalidValue;
    // persistent CTAs: one per SM (shared memory and TMEM allow no more), each walking its share of the items
    const unsigned blocks = static_cast<unsigned>(items < sm_count ? items : sm_count);
    kern<<<blocks, 512, W::kSmemBytes, stream>>>(tq, tk, tv, p);
    return cudaGetLastError();
}

template <int D, int IN>
static cudaError_t dispatch_mode(int mode, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                                 const AttnParams& p, cudaStream_t stream) {
    switch (mode) {
        case kExact: return launch_ws<D, IN, kExact>(tq, tk, tv, p, stream);
        case kPot: return launch_ws<D, IN, kPot>(tq, tk, tv, p, stream);
        case kPotDrop: return launch_ws<D, IN, kPotDrop>(tq, tk, tv, p, stream);
        case kH15: return launch_ws<D, IN, kH15>(tq, tk, tv, p, stream);
        default: break;
    }
    if constexpr (IN != kInFP16) {   // the family members and the emulated control are built for bf16 and fp8 only
        switch (mode) {
            case kH15K2: return launch_ws<D, IN, kH15K2>(tq, tk, tv, p, stream);
            case kH15K3: return launch_ws<D, IN, kH15K3>(tq, tk, tv, p, stream);
            case kExactPoly: return launch_ws<D, IN, kExactPoly>(tq, tk, tv, p, stream);
            default: break;
        }
        if constexpr (D == 128) {   // the other emulation shares: the paper's main head dimension only
            switch (mode) {
                case kExactPoly1: return launch_ws<D, IN, kExactPoly1>(tq, tk, tv, p, stream);
                case kExactPoly3: return launch_ws<D, IN, kExactPoly3>(tq, tk, tv, p, stream);
                case kExactPoly4: return launch_ws<D, IN, kExactPoly4>(tq, tk, tv, p, stream);
                default: break;
            }
        }
    }
    return cudaErrorInvalidValue;
}

// Returns cudaErrorInvalidValue for a combination that is not built.
cudaError_t launch_attn_fwd(int D, int in_type, int mode, const CUtensorMap& tq, const CUtensorMap& tk,
                            const CUtensorMap& tv, const AttnParams& p, cudaStream_t stream) {
    if (in_type == kInBF16 && D == 128) return dispatch_mode<128, kInBF16>(mode, tq, tk, tv, p, stream);
    if (in_type == kInBF16 && D == 64) return dispatch_mode<64, kInBF16>(mode, tq, tk, tv, p, stream);
    if (in_type == kInFP16 && D == 128) return dispatch_mode<128, kInFP16>(mode, tq, tk, tv, p, stream);
    if (in_type == kInFP16 && D == 64) return dispatch_mode<64, kInFP16>(mode, tq, tk, tv, p, stream);
    if (in_type == kInFP8 && D == 128) return dispatch_mode<128, kInFP8>(mode, tq, tk, tv, p, stream);
    if (in_type == kInFP8 && D == 64) return dispatch_mode<64, kInFP8>(mode, tq, tk, tv, p, stream);
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
        else if (mode == kExactPoly) wi = w_exact_poly3(xi);
        else if (mode == kPot) wi = w_pot(xi);
        else {
            // both lanes of the pair function are exercised: even indices take the shift-add lane, odd
            // indices the multiply-add lane
            float2 r;
            if (mode == kH15K2) r = w_h15_doubled_pair<0, true, 2>(make_float2(xi * 4.0f, xi * 4.0f), two22);
            else if (mode == kH15K3) r = w_h15_doubled_pair<0, true, 3>(make_float2(xi * 8.0f, xi * 8.0f), two22);
            else r = w_h15_doubled_pair<0, true, 1>(make_float2(xi * 2.0f, xi * 2.0f), two22);
            wi = (i & 1) ? r.y : r.x;
        }
        w[i] = wi;
    }
}

// Rowmax-PoT with a run-time tail (index cap K_max, clamped or dropped), the function of the 16-bit paths.
__global__ void weight_map_pot_kernel(const float* __restrict__ x, float* __restrict__ w, size_t n, int kmax, int drop) {
    const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
    for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += stride)
        w[i] = w_pot_tail(x[i], kmax, drop != 0);
}

cudaError_t launch_weight_map_pot(const float* x, float* w, size_t n, int kmax, int drop, cudaStream_t stream) {
    if (n == 0) return cudaSuccess;
    size_t blocks = (n + 255) / 256;
    if (blocks > 148 * 8) blocks = 148 * 8;
    weight_map_pot_kernel<<<static_cast<unsigned>(blocks), 256, 0, stream>>>(x, w, n, kmax, drop);
    return cudaGetLastError();
}

// The weights as the fused kernel's hot loop produces and stores them: every thread takes 32 consecutive offsets
// as one chunk of a score row (score = offset, scale 1, anchor 0), runs weights_chunk32 with the template
// arguments of the fused kernel for that storage type (fp8: its choice between the unclamped and the clamped h15
// variant, here per chunk, in the fused kernel per warp and key tile; 16 bit: the saturating form), and decodes
// the packed P words back to fp32, divided by the P scale.
template <bool FP8, bool HALF, int MODE>
__global__ void weight_map_fused_kernel(const float* __restrict__ x, float* __restrict__ w, size_t n, uint32_t two22,
                                        float pot_neg_cap, float pot_drop_x) {
    constexpr int kFam = h15_family_k(MODE);
    constexpr int kOff = PFormat<FP8, MODE>::kOffLog2;
    const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
    for (size_t chunk = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; chunk * 32 < n; chunk += stride) {
        uint32_t s[32];
        float lowest = INFINITY;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const size_t idx = chunk * 32 + i;
            const float xi = idx < n ? x[idx] : 0.0f;
            s[i] = __float_as_uint(xi);
            lowest = fminf(lowest, xi);
        }
        RowScale rs;
        const float c_row = static_cast<float>(1 << kFam);
        const float nmc = is_exact_like(MODE) ? static_cast<float>(kOff) : 0.0f;
        rs.c = make_float2(c_row, c_row);
        rs.nmc = make_float2(nmc, nmc);
        rs.two22 = two22;
        rs.pot_neg_cap = pot_neg_cap;
        rs.pot_drop_x = pot_drop_x;
        rs.clamp_lo = 0.f;
        if constexpr (kFam > 0) rs.clamp_lo = h15_clamp_floor<kFam>();
        float2 acc[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
        uint32_t pw[16];
        if constexpr (kFam > 0 && !FP8) {
            // 16-bit inputs: the saturating form, as in a key tile without masked scores
            constexpr float kR = 126.0f * (1 << kFam);
            rs.su = -static_cast<float>(1 << kFam) * (1.0f / kR);
            rs.ou = 0.0f;
            rs.sat_mul = -kR;
            weights_chunk32<FP8, MODE, false, true, HALF, true>(s, rs, 32, acc, pw);
        } else {
            const bool clamp = kFam > 0 && !(lowest * (1 << kFam) >= -125.0f * (1 << kFam));
            if (clamp) weights_chunk32<FP8, MODE, false, true, HALF>(s, rs, 32, acc, pw);
            else weights_chunk32<FP8, MODE, false, false, HALF>(s, rs, 32, acc, pw);
        }
        const float unscale = __uint_as_float(static_cast<uint32_t>(127 - kOff) << 23);   // 2^-kOff
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            float v;
            if constexpr (FP8) {
                const uint32_t byte = (pw[i / 4] >> (8 * (i % 4))) & 0xFFu;
                if constexpr (PFormat<FP8, MODE>::kE4M3) {
                    uint32_t h2;
                    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(static_cast<uint16_t>(byte)));
                    v = __half2float(__ushort_as_half(static_cast<unsigned short>(h2 & 0xFFFFu)));
                } else {
                    v = __half2float(__ushort_as_half(static_cast<unsigned short>(byte << 8)));   // e5m2 = upper byte of fp16
                }
            } else {
                const uint32_t h = (pw[i / 2] >> (16 * (i % 2))) & 0xFFFFu;
                if constexpr (HALF) v = __half2float(__ushort_as_half(static_cast<unsigned short>(h)));
                else v = __uint_as_float(h << 16);
            }
            const size_t idx = chunk * 32 + i;
            if (idx < n) w[idx] = v * unscale;
        }
    }
}

template <bool FP8, bool HALF>
static cudaError_t launch_fused_map_mode(const float* x, float* w, size_t n, int mode, float pot_neg_cap, float pot_drop_x,
                                         cudaStream_t stream) {
    size_t blocks = ((n + 31) / 32 + 127) / 128;
    if (blocks > 148 * 8) blocks = 148 * 8;
    const unsigned g = static_cast<unsigned>(blocks);
    switch (mode) {
        case kExact: weight_map_fused_kernel<FP8, HALF, kExact><<<g, 128, 0, stream>>>(x, w, n, 1u << 22, pot_neg_cap, pot_drop_x); break;
        case kPot: weight_map_fused_kernel<FP8, HALF, kPot><<<g, 128, 0, stream>>>(x, w, n, 1u << 22, pot_neg_cap, pot_drop_x); break;
        case kPotDrop: weight_map_fused_kernel<FP8, HALF, kPotDrop><<<g, 128, 0, stream>>>(x, w, n, 1u << 22, pot_neg_cap, pot_drop_x); break;
        case kH15: weight_map_fused_kernel<FP8, HALF, kH15><<<g, 128, 0, stream>>>(x, w, n, 1u << 22, pot_neg_cap, pot_drop_x); break;
        default:
            if constexpr (!HALF) {
                switch (mode) {
                    case kH15K2: weight_map_fused_kernel<FP8, HALF, kH15K2><<<g, 128, 0, stream>>>(x, w, n, 1u << 22, pot_neg_cap, pot_drop_x); break;
                    case kH15K3: weight_map_fused_kernel<FP8, HALF, kH15K3><<<g, 128, 0, stream>>>(x, w, n, 1u << 22, pot_neg_cap, pot_drop_x); break;
                    case kExactPoly: weight_map_fused_kernel<FP8, HALF, kExactPoly><<<g, 128, 0, stream>>>(x, w, n, 1u << 22, pot_neg_cap, pot_drop_x); break;
                    default: return cudaErrorInvalidValue;
                }
            } else {
                return cudaErrorInvalidValue;
            }
    }
    return cudaGetLastError();
}

cudaError_t launch_weight_map_fused(const float* x, float* w, size_t n, int mode, int in_type, float pot_neg_cap,
                                    float pot_drop_x, cudaStream_t stream) {
    if (n == 0) return cudaSuccess;
    if (in_type == kInFP8) return launch_fused_map_mode<true, false>(x, w, n, mode, pot_neg_cap, pot_drop_x, stream);
    if (in_type == kInFP16) return launch_fused_map_mode<false, true>(x, w, n, mode, pot_neg_cap, pot_drop_x, stream);
    return launch_fused_map_mode<false, false>(x, w, n, mode, pot_neg_cap, pot_drop_x, stream);
}

cudaError_t launch_weight_map(const float* x, float* w, size_t n, int mode, cudaStream_t stream) {
    if (n == 0) return cudaSuccess;
    const int threads = 256;
    size_t blocks = (n + threads - 1) / threads;
    if (blocks > 148 * 8) blocks = 148 * 8;
    weight_map_kernel<<<static_cast<unsigned>(blocks), threads, 0, stream>>>(x, w, n, mode, 1u << 22);
    return cudaGetLastError();
}

// One warp waits on a barrier nobody arrives on, with a short limit: the wait gives up, records its code in the
// status word and the kernel returns.  Exercises the bounded-wait path without touching the attention kernels.
__global__ void selftest_wait_kernel(int* status, long long limit_cycles) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int cta_abort;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        cta_abort = 0;
        fence_mbar_init();
    }
    __syncthreads();
    const WaitCtx ctx{&cta_abort, status, limit_cycles};
    mbar_wait(smem_u32(&bar), 0, ctx, (kRoleSelftest << 8) | kBarSelftest);
}

cudaError_t launch_selftest_wait(int* status, long long limit_cycles, cudaStream_t stream) {
    selftest_wait_kernel<<<1, 32, 0, stream>>>(status, limit_cycles);
    return cudaGetLastError();
}

__device__ int g_attn_status = 0;

cudaError_t status_word_address(int** out) {
    return cudaGetSymbolAddress(reinterpret_cast<void**>(out), g_attn_status);
}

}  // namespace rowmax
