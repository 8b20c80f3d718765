/*
 * attn.h — C interface of the B200 (sm_100a) fused attention forward with Rowmax weight maps.
 *
 * The library computes, for every batch b, query head h and query row i,
 *
 *     O[b,i,h,:] = v_descale * sum_j w_ij V[b,j,g(h),:] / sum_j w_ij,      LSE[b,h,i] = ln sum_j w_ij (+ anchor)
 *
 * over the keys j visible to row i, where the weight w_ij of a score is one of
 *   exact : 2^x               softmax, Eq. m-exact (Sec. 3.1) / Eq. exact-attention (App. A)
 *   pot   : 2^-min{K,floor(-x+1/2)}   Rowmax-PoT, Eq. rowmax-pot (App. A), K = K_max = 20
 *   h15   : (1 + (n mod 2)/2) 2^floor(n/2), n = RNE(2x)   Rowmax-H15, Eq. m-h15 (Sec. 5.2) / Eq. h15 (App. B.1)
 *   h15k2, h15k3 : 2^floor(q) (1 + q - floor(q)), q = RNE(2^k x)/2^k, k = 2, 3   the family H15 belongs to
 *           (k = 1), App. B "Exponential-map ablation": same add-and-shift with 2^k x and a shift by 23 - k
 *   exact_poly : 2^x as in exact, but every fourth pair of scores evaluated by floor + cubic + exponent insert
 *           instead of the special-function unit (relative error <= 1.1e-4): the partial emulation of the
 *           paper's baseline kernel, a stronger control than plain exact (App. B "FA4's own parameter space")
 * and x is the score's base-two offset from the running row maximum of the online-softmax loop
 * over key tiles (Sec. 5.2, App. B.1): x = s*c - m*c with c = softmax_scale*q_descale*k_descale*log2(e).
 * In pot and h15 mode the result depends on the key-tile schedule, which attn_get_schedule reports.
 *
 * Conventions shared by every entry point
 *   - All data pointers are DEVICE pointers owned by the caller.  The library never allocates,
 *     frees or keeps them.  Calls are asynchronous on `stream` (a cudaStream_t passed as void*;
 *     NULL = the legacy default stream) and do not synchronise the host.
 *   - Return value: ATTN_OK (0) or a negative ATTN_ERR_* code.  Nothing is thrown, printed or aborted.
 *   - The library keeps a little per-process state without locks (the address of each device's status
 *     word, the code of the last failing CUDA call, per-device launch set-up): call from one host thread
 *     at a time.
 */
#ifndef ROWMAX_ATTN_H_
#define ROWMAX_ATTN_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { ATTN_W_EXACT = 0, ATTN_W_POT = 1, ATTN_W_H15 = 2,
       ATTN_W_H15K2 = 3, ATTN_W_H15K3 = 4,     /* quarter- and eighth-octave members of the H15 family */
       ATTN_W_EXACT_POLY = 5 };               /* exact, a quarter of the 2^x evaluated by a cubic on the FMA pipe */
enum { ATTN_IN_BF16 = 0, ATTN_IN_FP8_E4M3 = 1, ATTN_IN_FP16 = 2 };
/* format of the probability tile P fed to the P.V contraction, as reported by attn_get_schedule */
enum { ATTN_P_BF16 = 0, ATTN_P_E4M3 = 1, ATTN_P_E5M2 = 2, ATTN_P_FP16 = 3 };

/* Rowmax-PoT tail index K_max: default (the paper's main point) and the largest value whose weights the
 * format of P still holds exactly (bf16: the fp32 exponent range; fp16 P: down to its subnormals; fp8:
 * e5m2 P with a power-of-two offset, 29 octaves). */
enum { ATTN_POT_KMAX_DEFAULT = 20, ATTN_POT_KMAX_BF16 = 125, ATTN_POT_KMAX_FP16 = 23, ATTN_POT_KMAX_FP8 = 29 };

enum {
    ATTN_OK = 0,
    ATTN_ERR_NULLPTR = -1,          /* a required pointer is NULL */
    ATTN_ERR_BAD_SHAPE = -2,        /* B, H, S <= 0; Hq % Hkv != 0; unsupported D; size overflow */
    ATTN_ERR_BAD_ENUM = -3,         /* weight_mode / in_dtype outside the enums above */
    ATTN_ERR_MISALIGNED = -4,       /* q, k, v or o not 16-byte aligned */
    ATTN_ERR_UNSUPPORTED_ARCH = -5, /* current device is not compute capability 10.x */
    ATTN_ERR_CUDA = -6,             /* a CUDA runtime/driver call failed; see attn_last_cuda_error */
    ATTN_ERR_TIMEOUT = -7,          /* returned by attn_device_status: a bounded device-side wait has expired */
    ATTN_ERR_UNSUPPORTED = -8,      /* valid arguments, combination not built (e.g. a deferred rescale on fp8 inputs) */
    ATTN_ERR_BAD_VALUE = -9         /* softmax_scale or an fp8 descale not positive and finite; rescale_tau or K_max out of range */
};

/*
 * attn_fwd — fused attention forward (Sec. 5.2; App. B.1 for the loop the weight map lives in).
 *
 *   q            (B, Sq, Hq, D)   bf16, IEEE half (ATTN_IN_FP16; the FP16 rows of the timing tables in
 *                                 App. B), or e4m3 bytes (ATTN_IN_FP8_E4M3); D contiguous
 *   k, v         (B, Sk, Hkv, D)  same storage type as q
 *   o            (B, Sq, Hq, D)   bf16, written
 *   lse          (B, Hq, Sq)      fp32, natural log, written; may be NULL
 *   D            64 or 128
 *   causal       != 0: key j is visible to query i iff j <= i + Sk - Sq (aligned to the bottom-right
 *                corner); a row that sees no key gets O = 0 and LSE = -inf
 *   Hq, Hkv      query head h reads key/value head h / (Hq / Hkv)
 *   softmax_scale  multiplies q.k before the softmax (natural-exponent units)
 *   weight_mode  ATTN_W_EXACT / ATTN_W_POT / ATTN_W_H15 / ATTN_W_H15K2 / ATTN_W_H15K3 / ATTN_W_EXACT_POLY
 *                (fp16 inputs: the first three; the others return ATTN_ERR_UNSUPPORTED)
 *   q/k/v_descale  per-tensor factors of the fp8 inputs (value = stored * descale); ignored for bf16 / fp16
 *
 * All tensors are contiguous; q, k, v, o must be 16-byte aligned.  In pot/h15 mode LSE is the log
 * of the approximated denominator.
 */
int attn_fwd(const void* q, const void* k, const void* v, void* o, float* lse,
             int B, int Hq, int Hkv, int Sq, int Sk, int D,
             int causal, float softmax_scale, int weight_mode, int in_dtype,
             float q_descale, float k_descale, float v_descale, void* stream);

/*
 * attn_fwd_tau — attn_fwd with a deferred rescale (App. B "Conditional rescaling moves the anchor";
 * the rule of the paper's BF16 kernel, which uses rescale_tau = 8): a key tile's maximum replaces the
 * row's anchor only when it exceeds the anchor by more than rescale_tau octaves of the scaled score,
 * so O is rescaled far less often and x can be positive (Eq. h15 covers both signs).  Exact mode is
 * unchanged by this up to rounding; pot and h15 results differ from rescale_tau = 0 because the
 * lattice is anchored at the lagging maximum.  bf16 inputs only (ATTN_ERR_UNSUPPORTED for fp8, whose P
 * formats have no headroom above the anchor, and for fp16); 0 <= rescale_tau <= 32, else ATTN_ERR_BAD_VALUE.
 * attn_fwd is attn_fwd_tau with rescale_tau = 0.
 */
int attn_fwd_tau(const void* q, const void* k, const void* v, void* o, float* lse,
                 int B, int Hq, int Hkv, int Sq, int Sk, int D,
                 int causal, float softmax_scale, int weight_mode, int in_dtype,
                 float q_descale, float k_descale, float v_descale, float rescale_tau, void* stream);

/*
 * attn_fwd_pot — attn_fwd in Rowmax-PoT mode with the tail chosen by the caller (App. A, Eq. rowmax-pot and the
 * sentence after it: the main point clamps the tail at K_max = 20, a K_max sweep and a tail-drop variant are
 * reported beside it; results figure, panel B).  The index of a key is d = min{K_max, floor(-x + 1/2)} and its
 * weight 2^-d (clamped tail, drop_tail = 0: every visible key keeps at least 2^-K_max), or, with drop_tail != 0,
 * d = floor(-x + 1/2) and weight 0 where d > K_max.  x is the offset from the running maximum of the online
 * loop, so with a dropped tail a key is dropped relative to the anchor of its own key tile; what earlier tiles
 * accumulated is rescaled, not dropped.  1 <= pot_kmax <= ATTN_POT_KMAX_BF16 / _FP16 / _FP8 for the storage type,
 * else ATTN_ERR_BAD_VALUE.  attn_fwd(..., ATTN_W_POT, ...) is attn_fwd_pot with pot_kmax = 20, drop_tail = 0.
 */
int attn_fwd_pot(const void* q, const void* k, const void* v, void* o, float* lse,
                 int B, int Hq, int Hkv, int Sq, int Sk, int D,
                 int causal, float softmax_scale, int in_dtype,
                 float q_descale, float k_descale, float v_descale,
                 int pot_kmax, int drop_tail, void* stream);

/*
 * attn_fwd_exact_emulated — attn_fwd in exact mode with share_eighths / 8 of the 2^x evaluated by floor + cubic +
 * exponent insert on the FMA and integer pipes instead of the special-function unit (relative error <= 1.1e-4):
 * the partial emulation that the paper's baseline kernel uses, with its share as a parameter (App. B "FA4's own
 * parameter space": shares 0 to 75 %, the fastest stock setting at 37.5 %).  share_eighths = 1, 2, 3, 4 (12.5, 25,
 * 37.5, 50 %), else ATTN_ERR_BAD_VALUE; attn_fwd(..., ATTN_W_EXACT_POLY, ...) is share_eighths = 2.  Shares other
 * than 2 are built for D = 128 and bf16 / fp8 inputs (ATTN_ERR_UNSUPPORTED otherwise).  Same tolerances as exact.
 */
int attn_fwd_exact_emulated(const void* q, const void* k, const void* v, void* o, float* lse,
                            int B, int Hq, int Hkv, int Sq, int Sk, int D,
                            int causal, float softmax_scale, int in_dtype,
                            float q_descale, float k_descale, float v_descale,
                            int share_eighths, void* stream);

/*
 * attn_weight_map — applies the weight map of `weight_mode` to n fp32 offsets with the same device
 * function the fused kernel uses (Eq. m-exact / Eq. rowmax-pot / Eq. h15; the h15 input is clamped
 * below at -126, App. B.1 "Implementation"; inside the fused kernel a key tile that holds masked scores
 * clamps at -127 instead, the input whose weight pattern is +0, so that a masked key weighs nothing; on fp8 inputs, whose weights
 * carry a 2^15 offset, that pattern is 2^-112: zero in P, and below one part in 2^127 of a row sum).  x and w are device arrays
 * of n floats; they may alias.
 * pot and h15 results are bit-exact by definition; exact uses the hardware ex2 approximation with
 * subnormal results flushed to zero.
 */
int attn_weight_map(const float* x, float* w, size_t n, int weight_mode, void* stream);

/*
 * attn_weight_map_pot — the Rowmax-PoT map with the tail of attn_fwd_pot (Eq. rowmax-pot and the sentence after
 * it): w = 2^-min{K_max, floor(-x + 1/2)}, or with drop_tail != 0 zero where floor(-x + 1/2) > K_max.  Bit-exact
 * by definition.  1 <= pot_kmax <= ATTN_POT_KMAX_BF16, else ATTN_ERR_BAD_VALUE.
 */
int attn_weight_map_pot(const float* x, float* w, size_t n, int pot_kmax, int drop_tail, void* stream);

/*
 * attn_weight_map_fused — the weights as the hot loop of attn_fwd produces them and stores them in P for inputs of
 * storage type in_dtype (Eq. m-exact / Eq. rowmax-pot / Eq. h15 again, but through the instantiations the fused
 * kernel runs, which attn_weight_map does not reach).  The n offsets are taken 32 at a time as one chunk of a
 * score row (score = offset, anchor 0, scale 1); the packed P words are decoded again and divided by the P scale.
 *   fp8 inputs, h15 family: the packed form without the per-score clamp wherever the 32 offsets all lie above -125
 *     octaves, with the clamp elsewhere; weights scaled by the P offset.  Equal to attn_weight_map bit for bit
 *     wherever P holds the weight: down to 2^-29 (e5m2 P: h15, h15k2) or 2^-14 (e4m3 P: h15k3).
 *   16-bit inputs, h15 family: the saturating form (scale, anchor shift and lower clamp in one saturating
 *     multiply-add on the distance below the anchor, then one multiply-add that rounds).  The rounded integer is
 *     that of Eq. h15 except possibly for offsets within 2^-20 (relative) of a rounding tie, where the fp32
 *     rounding of the scaled distance decides; everywhere else equal to attn_weight_map bit for bit (bf16 P
 *     holds every weight; fp16 P down to 2^-23).
 *   Rowmax-PoT: the offset rounded to the nearest integer by the same add as h15 (ties to even, where Eq. rowmax-pot
 *     sends ties down: the two differ only at an exact tie x = -(d + 1/2), d odd, where the fused loop gives the
 *     larger neighbour; the boundary of a dropped tail is kept as defined), with the tail given here; bit for bit
 *     elsewhere, wherever P holds the weight (fp16 P: 2^-24, e5m2 P: 2^-29).
 *   exact-like modes: 2^x rounded to the format of P.
 * Below the range of P the stored weight rounds in the subnormal range of the format and then underflows to zero.
 * pot_kmax / drop_tail matter in ATTN_W_POT mode only (limits as for attn_fwd_pot).
 */
int attn_weight_map_fused(const float* x, float* w, size_t n, int weight_mode, int in_dtype,
                          int pot_kmax, int drop_tail, void* stream);

/*
 * attn_get_schedule — what a reference implementation must mirror to reproduce pot/h15 results
 * (App. B "Semantic simulation": per-tile running maximum, tile of 128 keys, rescale rule).
 * Host-only query, no CUDA call.  Any output pointer may be NULL.
 *   tile_m, tile_n   query rows / keys per tile
 *   kv_order         +1: key tiles visited in ascending order
 *   rescale_tau      anchor adoption threshold in octaves used by attn_fwd (0 = the anchor is always current);
 *                    attn_fwd_tau takes its own
 *   pot_kmax         K_max of Rowmax-PoT as attn_fwd uses it (attn_fwd_pot takes its own)
 *   p_format         ATTN_P_*; p_offset_log2: P is stored as weight * 2^p_offset_log2
 */
int attn_get_schedule(int D, int in_dtype, int weight_mode, int causal,
                      int* tile_m, int* tile_n, int* kv_order, float* rescale_tau,
                      int* pot_kmax, int* p_format, int* p_offset_log2);

/*
 * Device-side waits and the status word.  (No counterpart in the paper: safety net of the mbarrier / TMEM pipeline.)
 * Every wait inside the kernels is bounded (about one second).  A wait that runs out writes a code, role << 8 |
 * barrier id, into one status word per device, and the kernel winds down: the roles leave their loops, copies and
 * MMAs in flight are awaited with a bound, nothing more is stored, TMEM is released.  No trap, no hang.
 * The word is STICKY: it stays set across launches until attn_device_status_reset.  While it is set, attn_fwd,
 * attn_fwd_tau and attn_fwd_pot still return ATTN_OK (they are asynchronous and do not read the word), but their
 * kernels return at once WITHOUT writing o or lse.  So: after a batch of launches call attn_device_status; on
 * ATTN_ERR_TIMEOUT treat every output since the last clean check as invalid, reset, and launch again.
 *   attn_device_status        synchronises the current device; ATTN_OK, ATTN_ERR_TIMEOUT (the word is set), or
 *                             ATTN_ERR_CUDA
 *   attn_device_status_code   same, but returns the word itself (0, or role << 8 | barrier id of the first wait
 *                             that ran out) or a negative ATTN_ERR_*
 *   attn_device_status_reset  synchronises and clears the word
 *   attn_selftest_wait        launches one warp that waits, for at most limit_cycles SM clocks (1 .. 2e9), on a
 *                             barrier that nothing arrives on: the wait runs out, the word is set (role 7, barrier
 *                             0x7f) and the kernel returns.  For tests of the path above; clear the word afterwards.
 */
int attn_device_status(void);
int attn_device_status_code(void);
int attn_device_status_reset(void);
int attn_selftest_wait(long long limit_cycles, void* stream);

/* Number of kernels this library has launched in this process (all entry points). */
unsigned long long attn_launch_count(void);

const char* attn_status_string(int status);
int attn_last_cuda_error(void);     /* cudaError_t / CUresult of the last failing call, else 0 */
const char* attn_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ROWMAX_ATTN_H_ */
