/*
 * CPU oracle for the Rowmax attention forward.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, double-precision statement of what the fused attention forward computes, written
 * from the paper's definitions.  It exists so that tests, the smoke check and the bench's
 * cpu_baseline leg have something independent to compare the CUDA path with.  It shares no code,
 * header, table or constant generator with the CUDA path, and the product path never calls it.
 *
 * Passages followed:
 *   - exact softmax attention, masked entries have probability zero ........ Eq. m-exact (Sec. 3.1),
 *                                                                            Eq. exact-attention (App. A)
 *   - Rowmax-PoT: d = min{K_max, floor(Delta/ln2 + 1/2)}, w = 2^-d ........... Eq. rowmax-pot (App. A)
 *   - Rowmax-H15: n = RNE(2x), w = (1 + (n mod 2)/2) * 2^floor(n/2) .......... Eq. m-h15 (Sec. 5.2), Eq. h15 (App. B.1)
 *   - lower clamp of the H15 input at x = -126 (doubled input at -252) ...... App. B.1 "Implementation",
 *                                                                            App. B "Exponential-map ablation"
 *   - the H15 family S(Q_{2^-k}(x)), k = 2, 3 ................................. App. B "Exponential-map ablation",
 *                                                                            App. B.1 "Relation to classical bit-level exponentiation"
 *   - anchor = the running row maximum of the online loop, tile of 128 keys,
 *     rescale rule, per-row decision; row sum and PV use the same weights ... Sec. 5.2, App. B.1,
 *                                                                            App. B "Semantic simulation"
 *
 * Pins (see tests, all run without a GPU): worked example n = -3 -> 1.5 * 2^-2; h15(0) = pot(0) = 1;
 * range, monotonicity, octave equivariance; error envelope [-0.25, log2(1.5) - 0.25]; identity with
 * the unshifted Schraudolph construction on half-integer-rounded inputs; the add-and-shift bit
 * construction; brute-force and library softmax on tiny inputs; Q = 0 closed form; two-key hand
 * example; whole-row equivalence when one tile covers the row; a second, independent NumPy coding
 * of the online loop; with a rescale threshold: exact mode equals the definition for any threshold,
 * and a hand example with a lagging anchor (positive offsets); Rowmax-PoT tail: clamp and drop values
 * at and beyond K_max.  The tie-widening rule (oracle_attn's widen outputs) and the p_round diagnostic
 * are this build's own devices with no counterpart in the paper; they are pinned as what they claim
 * to be: p_round against a library's casts to bfloat16 / e4m3 / e5m2, the widening as a bound, by
 * moving every flagged score across its boundary.
 */
#include <fenv.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_W_EXACT = 0, ORACLE_W_POT = 1, ORACLE_W_H15 = 2, ORACLE_W_H15K2 = 3, ORACLE_W_H15K3 = 4 };
enum { ORACLE_IN_BF16 = 0, ORACLE_IN_FP8_E4M3 = 1, ORACLE_IN_FP16 = 2 };
enum { ORACLE_P_NONE = 0, ORACLE_P_BF16 = 1, ORACLE_P_E4M3 = 2, ORACLE_P_E5M2 = 3 };

/* ---------------------------------------------------------------------------------------------
 * Storage formats, decoded from their definitions.
 * ------------------------------------------------------------------------------------------- */

/* bfloat16: 1 sign, 8 exponent (bias 127), 7 fraction bits. */
double oracle_decode_bf16(uint16_t h) {
    int sign = (h >> 15) & 1;
    int e = (h >> 7) & 0xFF;
    int f = h & 0x7F;
    double v;
    if (e == 0xFF) {
        v = f ? NAN : INFINITY;
    } else if (e == 0) {
        v = ldexp((double)f / 128.0, -126);
    } else {
        v = ldexp(1.0 + (double)f / 128.0, e - 127);
    }
    return sign ? -v : v;
}

/* IEEE binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits. */
double oracle_decode_fp16(uint16_t h) {
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1F;
    int f = h & 0x3FF;
    double v;
    if (e == 0x1F) {
        v = f ? NAN : INFINITY;
    } else if (e == 0) {
        v = ldexp((double)f / 1024.0, -14);
    } else {
        v = ldexp(1.0 + (double)f / 1024.0, e - 15);
    }
    return sign ? -v : v;
}

/* float8 e4m3 ("fn" flavour): 1 sign, 4 exponent (bias 7), 3 fraction bits; no infinity; the
 * all-ones pattern S.1111.111 is NaN; largest finite value 448. */
double oracle_decode_e4m3(uint8_t b) {
    int sign = (b >> 7) & 1;
    int e = (b >> 3) & 0xF;
    int f = b & 0x7;
    double v;
    if (e == 0xF && f == 0x7) {
        v = NAN;
    } else if (e == 0) {
        v = ldexp((double)f / 8.0, -6);
    } else {
        v = ldexp(1.0 + (double)f / 8.0, e - 7);
    }
    return sign ? -v : v;
}

/* Round a non-negative double to a format with `fbits` fraction bits, minimum normal exponent
 * `emin` and largest finite value `vmax`, ties to even, saturating.  Used only by the p_round
 * diagnostic below (pinned in the tests against a library's casts to bfloat16, e4m3 and e5m2). */
static double round_to_small_float(double v, int fbits, int emin, double vmax) {
    if (!(v > 0.0)) return 0.0;
    int e;
    (void)frexp(v, &e); /* v = m * 2^e, m in [0.5, 1) -> exponent of the leading bit is e - 1 */
    int lead = e - 1;
    if (lead < emin) lead = emin; /* subnormal range: fixed spacing */
    double ulp = ldexp(1.0, lead - fbits);
    double r = nearbyint(v / ulp) * ulp;
    if (r > vmax) r = vmax;
    return r;
}

static double p_round_apply(double w, int p_round, int p_off) {
    double s = ldexp(w, p_off), r;
    switch (p_round) {
        case ORACLE_P_BF16: r = round_to_small_float(s, 7, -126, 3.3895313892515355e38); break;
        case ORACLE_P_E4M3: r = round_to_small_float(s, 3, -6, 448.0); break;
        case ORACLE_P_E5M2: r = round_to_small_float(s, 2, -14, 57344.0); break;
        default: return w;
    }
    return ldexp(r, -p_off);
}

/* The p_round diagnostic on one value, exported so that tests can pin it:
 * the weight w >= 0 times 2^p_off rounded to the format, divided by 2^p_off again. */
double oracle_p_round(double w, int p_round, int p_off) { return p_round_apply(w, p_round, p_off); }

/* ---------------------------------------------------------------------------------------------
 * Weight maps on an fp32 base-two offset x (x = 0 at the anchor, negative below it).
 * ------------------------------------------------------------------------------------------- */

/* Exact mode: w = 2^x (Eq. m-exact rewritten in base two: exp(-Delta) = 2^(-Delta/ln 2)). */
double oracle_w_exact(float x) { return exp2((double)x); }

/* Rowmax-PoT (Eq. rowmax-pot): with y = Delta/ln2 = -x, d = min{K_max, floor(y + 1/2)}, w = 2^-d.
 * Ties in y + 1/2 go up in d, that is toward the smaller weight.  The main point clamps the tail
 * (every key keeps at least 2^-K_max: full support); the tail-drop variant (App. A, the sentence
 * after Eq. rowmax-pot) gives weight zero to the keys whose index floor(y + 1/2) exceeds K_max. */
double oracle_w_pot_tail(float x, int kmax, int drop_tail) {
    if (isnan(x)) return NAN;
    double y = -(double)x;
    double d = floor(y + 0.5); /* exact: y is an fp32 value, the sum is representable in double */
    if (d > (double)kmax) {
        if (drop_tail) return 0.0;
        d = (double)kmax;
    }
    return ldexp(1.0, -(int)d);
}
double oracle_w_pot(float x, int kmax) { return oracle_w_pot_tail(x, kmax, 0); }

/* Rowmax-H15 (Eq. h15): n = RNE(2x), w = (1 + (n mod 2)/2) * 2^floor(n/2), floor toward -inf and
 * n mod 2 the non-negative residue; the input is first clamped from below at -126 (the doubled
 * input at -252). */
double oracle_w_h15(float x) {
    if (isnan(x)) return NAN;
    double xd = (double)x;
    if (xd < -126.0) xd = -126.0;
    double n = nearbyint(2.0 * xd); /* rounding mode is to-nearest-even, set by the callers below */
    double k = floor(n / 2.0);
    double b = n - 2.0 * k; /* 0 or 1 */
    return (1.0 + 0.5 * b) * ldexp(1.0, (int)k);
}

/* The family Rowmax-H15 belongs to (App. B "Exponential-map ablation"): the unshifted Schraudolph
 * construction S(q) = 2^floor(q) (1 + q - floor(q)) evaluated on the input rounded to steps of 2^-k,
 * q = RNE(2^k x) / 2^k, after the same lower clamp max(x, -126).  k = 1 is Rowmax-H15 itself;
 * k = 2, 3 are the quarter- and eighth-octave members. */
double oracle_w_h15_family(float x, int k) {
    if (isnan(x)) return NAN;
    double xd = (double)x;
    if (xd < -126.0) xd = -126.0;
    double steps = ldexp(1.0, k);
    double q = nearbyint(steps * xd) / steps;
    double fl = floor(q);
    return ldexp(1.0 + (q - fl), (int)fl);
}

static double weight_of(float x, int mode, int kmax, int drop_tail) {
    switch (mode) {
        case ORACLE_W_POT: return oracle_w_pot_tail(x, kmax, drop_tail);
        case ORACLE_W_H15: return oracle_w_h15(x);
        case ORACLE_W_H15K2: return oracle_w_h15_family(x, 2);
        case ORACLE_W_H15K3: return oracle_w_h15_family(x, 3);
        default: return oracle_w_exact(x);
    }
}

/* Array form used by the sweep tests.  Returns 0, or -1 for a bad mode. */
int oracle_weight_map(const float* x, double* w, size_t n, int mode, int kmax, int drop_tail) {
    if (mode < 0 || mode > 4) return -1;
    fesetround(FE_TONEAREST);
    for (size_t i = 0; i < n; ++i) w[i] = weight_of(x[i], mode, kmax, drop_tail);
    return 0;
}

/* ---------------------------------------------------------------------------------------------
 * Attention.
 * Layouts: q (B,Sq,Hq,D), k and v (B,Sk,Hkv,D), D contiguous; raw storage bytes (bf16 = 2 bytes
 * little endian, e4m3 = 1 byte).  Outputs are compact over the requested query rows:
 * O (B,Hq,nrows,D), LSE (B,Hq,nrows), natural log.
 * Causal masking is aligned to the bottom-right corner: key j is visible to query i iff
 * j <= i + Sk - Sq.  A row with no visible key gives O = 0 and LSE = -inf.
 * GQA: query head h reads kv head h / (Hq/Hkv).
 * ------------------------------------------------------------------------------------------- */

static double* decode_tensor(const void* p, size_t n, int in_dtype) {
    double* out = (double*)malloc(n * sizeof(double));
    if (!out) return NULL;
    if (in_dtype == ORACLE_IN_BF16) {
        const uint16_t* s = (const uint16_t*)p;
        for (size_t i = 0; i < n; ++i) out[i] = oracle_decode_bf16(s[i]);
    } else if (in_dtype == ORACLE_IN_FP16) {
        const uint16_t* s = (const uint16_t*)p;
        for (size_t i = 0; i < n; ++i) out[i] = oracle_decode_fp16(s[i]);
    } else {
        const uint8_t* s = (const uint8_t*)p;
        for (size_t i = 0; i < n; ++i) out[i] = oracle_decode_e4m3(s[i]);
    }
    return out;
}

/* One query row, exact mode, straight from the definition (whole row, no tiles):
 * s_j = scale * q.k_j over visible j; m = max s; w = exp(s - m); O = dv * sum w v / sum w;
 * LSE = m + ln sum w. */
static void row_exact_definition(const double* qrow, const double* kbase, const double* vbase,
                                 size_t kv_stride, int nvis, int D, double scale, double dv,
                                 double* s_buf, double* o, double* lse) {
    if (nvis <= 0) {
        for (int d = 0; d < D; ++d) o[d] = 0.0;
        *lse = -INFINITY;
        return;
    }
    double m = -INFINITY;
    for (int j = 0; j < nvis; ++j) {
        const double* kr = kbase + (size_t)j * kv_stride;
        double dot = 0.0;
        for (int d = 0; d < D; ++d) dot += qrow[d] * kr[d];
        s_buf[j] = scale * dot;
        if (s_buf[j] > m) m = s_buf[j];
    }
    double l = 0.0;
    for (int d = 0; d < D; ++d) o[d] = 0.0;
    for (int j = 0; j < nvis; ++j) {
        double w = exp(s_buf[j] - m);
        const double* vr = vbase + (size_t)j * kv_stride;
        l += w;
        for (int d = 0; d < D; ++d) o[d] += w * vr[d];
    }
    for (int d = 0; d < D; ++d) o[d] = dv * o[d] / l;
    *lse = m + log(l);
}

/* One query row, online loop over key tiles (App. B.1; App. B "Semantic simulation"):
 *   for each tile (in kv_order) that holds a visible key:
 *     m_t = max of the raw dot products z_j of the tile's visible keys
 *     adopt m_new = max(m, m_t) when m is -inf or m_t exceeds m by more than tau octaves
 *       (tau = 0: always adopt, so the anchor is current and x <= 0 up to rounding);
 *       on adoption l and acc are multiplied by alpha = 2^((m - m_new) c)
 *     x_j = fl32(z_j c - fl32(m c)),  w_j = MAP(x_j),  l += w_j,  acc += P(w_j) v_j
 *   O = dv acc / l,  LSE = ln2 (m c + log2 l)
 * c is the single fp32 constant fl32(scale dq dk log2 e).  tau is in octaves of the scaled score.
 * With tau > 0 the last adopted anchor may lag the true maximum; the final formulas hold as they
 * are because l, acc and m stay mutually consistent.
 *
 * Tie bookkeeping (not from the paper): a weight map that rounds is discontinuous, and a score
 * that differs in its last fp32 bits can land on the other side of a rounding boundary.  Elements
 * whose rounded quantity lies within tie_eps * max(1, |quantity|) of a boundary are counted, and
 * a bound on what flipping them could do to O and LSE is returned so that a comparison can widen
 * its tolerance on exactly those rows. */
static void row_online(const double* qrow, const double* kbase, const double* vbase,
                       size_t kv_stride, int nvis, int D, float c32, double dv, int mode,
                       int tile_n, int kv_order, double tau, int kmax, int drop_tail, int p_round,
                       int p_off, double tie_eps, double* z_buf, double* o, double* lse, double* widen_o,
                       double* widen_lse, int32_t* nflag) {
    double c = (double)c32;
    double m = -INFINITY, l = 0.0;
    double flip = 0.0, flip_down = 0.0, flip_vmax = 0.0;
    int32_t flagged = 0;
    for (int d = 0; d < D; ++d) o[d] = 0.0;
    if (nvis <= 0) {
        *lse = -INFINITY;
        if (widen_o) *widen_o = 0.0;
        if (widen_lse) *widen_lse = 0.0;
        if (nflag) *nflag = 0;
        return;
    }
    int ntiles = (nvis + tile_n - 1) / tile_n;
    for (int tt = 0; tt < ntiles; ++tt) {
        int t = kv_order >= 0 ? tt : ntiles - 1 - tt;
        int j0 = t * tile_n;
        int j1 = j0 + tile_n < nvis ? j0 + tile_n : nvis;
        double m_t = -INFINITY;
        for (int j = j0; j < j1; ++j) {
            const double* kr = kbase + (size_t)j * kv_stride;
            double dot = 0.0;
            for (int d = 0; d < D; ++d) dot += qrow[d] * kr[d];
            z_buf[j - j0] = dot;
            if (dot > m_t) m_t = dot;
        }
        if (m == -INFINITY || (m_t - m) * c > tau) {
            double m_new = m_t > m ? m_t : m;
            double alpha = (m == -INFINITY) ? 0.0 : exp2((m - m_new) * c);
            l *= alpha;
            flip *= alpha;
            flip_down *= alpha;
            for (int d = 0; d < D; ++d) o[d] *= alpha;
            m = m_new;
        }
        double mc = (double)(float)(m * c);
        for (int j = j0; j < j1; ++j) {
            float x = (float)(z_buf[j - j0] * c - mc);
            double w = weight_of(x, mode, kmax, drop_tail);
            const double* vr = vbase + (size_t)j * kv_stride;
            double pw = p_round_apply(w, p_round, p_off);
            l += w;
            for (int d = 0; d < D; ++d) o[d] += pw * vr[d];
            if (mode != ORACLE_W_EXACT && tie_eps > 0.0) {
                double u, dist;
                const int kk = mode == ORACLE_W_H15 ? 1 : mode == ORACLE_W_H15K2 ? 2 : mode == ORACLE_W_H15K3 ? 3 : 0;
                if (kk > 0) {
                    u = ldexp((double)x < -126.0 ? -126.0 : (double)x, kk);   /* the quantity that is rounded */
                } else {
                    u = -(double)x; /* boundaries of floor(y + 1/2) sit at half-integers too */
                }
                dist = fabs(u - (floor(u) + 0.5));
                if (dist < tie_eps * (fabs(u) > 1.0 ? fabs(u) : 1.0) &&
                    !(mode == ORACLE_W_POT && u > (double)kmax + 1.0)) {
                    double vmax = 0.0;
                    for (int d = 0; d < D; ++d)
                        if (fabs(vr[d]) > vmax) vmax = fabs(vr[d]);
                    /* one lattice step is at most w / 2^k (pot: w; a dropped tail weight may come back as 2^-K_max) */
                    flip += kk > 0 ? ldexp(w, -kk) : (w > 0.0 ? w : ldexp(1.0, -kmax));
                    /* the largest step DOWN is w / (2^k + 1) (from (1 + 2^-k) 2^e to 2^e; pot: w / 2); a
                     * tail weight 2^-K_max that is dropped loses all of itself */
                    flip_down += (kk == 0 && drop_tail && w <= ldexp(1.0, -kmax)) ? w : w / (ldexp(1.0, kk) + 1.0);
                    if (vmax > flip_vmax) flip_vmax = vmax;
                    ++flagged;
                }
            }
        }
    }
    double omax = 0.0;
    for (int d = 0; d < D; ++d) {
        o[d] = dv * o[d] / l;
        if (fabs(o[d]) > omax) omax = fabs(o[d]);
    }
    *lse = M_LN2 * (m * c + log2(l));
    /* O' - O = sum_j delta_j (dv v_j - O) / l' with l' = l + sum_j delta_j >= l - flip_down */
    if (widen_o) *widen_o = (flip / (l - flip_down)) * (dv * flip_vmax + omax);
    if (widen_lse) *widen_lse = flip / l;
    if (nflag) *nflag = flagged;
}

/*
 * oracle_attn: attention forward for the query rows listed in `rows` (NULL = every row 0..Sq-1),
 * for every (batch, query head).
 *   mode        ORACLE_W_EXACT / _POT / _H15
 *   tile_n      0 with mode exact = the whole-row definition (the parity reference of exact mode);
 *               > 0 = the online loop with tiles of tile_n keys (any mode)
 *   kv_order    +1 ascending key tiles, -1 descending
 *   tau         rescale threshold in octaves (0 = always rescale)
 *   kmax, drop_tail   Rowmax-PoT: tail index K_max and what happens beyond it (0 = clamp, 1 = drop)
 *   p_round     diagnostic only: round the weight (times 2^p_off) to bf16 / e4m3 / e5m2 before it
 *               multiplies V; the row sum always uses the unrounded weight
 *   tie_eps     0 disables the tie bookkeeping; widen_o, widen_lse, nflag may be NULL
 * Returns the number of threads used (>= 1), or a negative value on a bad argument / no memory.
 */
int oracle_attn(const void* q, const void* k, const void* v, int in_dtype, int B, int Hq, int Hkv,
                int Sq, int Sk, int D, int causal, float softmax_scale, float q_descale,
                float k_descale, float v_descale, int mode, int tile_n, int kv_order, double tau,
                int kmax, int drop_tail, int p_round, int p_off, double tie_eps, const int32_t* rows, int nrows,
                double* O, double* LSE, double* widen_o, double* widen_lse, int32_t* nflag,
                int nthreads) {
    if (!q || !k || !v || !O || !LSE) return -1;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || D <= 0 || Hq % Hkv) return -2;
    if (mode < 0 || mode > 4 || in_dtype < 0 || in_dtype > 2 || tile_n < 0) return -3;
    if (tile_n == 0 && mode != ORACLE_W_EXACT) return -3;
    fesetround(FE_TONEAREST);
    if (!rows) nrows = Sq;
    double* qd = decode_tensor(q, (size_t)B * Sq * Hq * D, in_dtype);
    double* kd = decode_tensor(k, (size_t)B * Sk * Hkv * D, in_dtype);
    double* vd = decode_tensor(v, (size_t)B * Sk * Hkv * D, in_dtype);
    if (!qd || !kd || !vd) {
        free(qd); free(kd); free(vd);
        return -4;
    }
    double dq = in_dtype != ORACLE_IN_FP8_E4M3 ? 1.0 : (double)q_descale;
    double dk = in_dtype != ORACLE_IN_FP8_E4M3 ? 1.0 : (double)k_descale;
    double dv = in_dtype != ORACLE_IN_FP8_E4M3 ? 1.0 : (double)v_descale;
    double scale = (double)softmax_scale * dq * dk;
    float c32 = (float)(scale * 1.4426950408889634074); /* log2 e */
    int group = Hq / Hkv;
    size_t kv_stride = (size_t)Hkv * D;
    long total = (long)B * Hq * nrows;
    int used = 1;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
    used = omp_get_max_threads();
#endif
    int bufn = tile_n > 0 ? tile_n : Sk;
    int failed = 0;
#pragma omp parallel
    {
        double* buf = (double*)malloc((size_t)bufn * sizeof(double));
        if (!buf) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 8)
        for (long it = 0; it < total; ++it) {
            if (!buf) continue;
            int r = (int)(it % nrows);
            int h = (int)((it / nrows) % Hq);
            int b = (int)(it / ((long)nrows * Hq));
            int i = rows ? rows[r] : r;
            int hk = h / group;
            int nvis = causal ? i + Sk - Sq + 1 : Sk;
            if (nvis > Sk) nvis = Sk;
            const double* qrow = qd + (((size_t)b * Sq + i) * Hq + h) * D;
            const double* kbase = kd + ((size_t)b * Sk * Hkv + hk) * D;
            const double* vbase = vd + ((size_t)b * Sk * Hkv + hk) * D;
            double* o = O + (size_t)it * D;
            if (tile_n == 0) {
                row_exact_definition(qrow, kbase, vbase, kv_stride, nvis, D, scale, dv, buf, o,
                                     LSE + it);
                if (widen_o) widen_o[it] = 0.0;
                if (widen_lse) widen_lse[it] = 0.0;
                if (nflag) nflag[it] = 0;
            } else {
                row_online(qrow, kbase, vbase, kv_stride, nvis, D, c32, dv, mode, tile_n,
                           kv_order, tau, kmax, drop_tail, p_round, p_off, tie_eps, buf, o,
                           LSE + it,
                           widen_o ? widen_o + it : NULL, widen_lse ? widen_lse + it : NULL,
                           nflag ? nflag + it : NULL);
            }
        }
        free(buf);
    }
    free(qd); free(kd); free(vd);
    return failed ? -4 : used;
}
