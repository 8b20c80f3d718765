// C interface (include/attn.h): argument validation, TMA tensor maps, dispatch.  No torch types.
#include "../../include/attn.h"
#include "attn_kernel_common.cuh"

#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstdint>

namespace rowmax {
cudaError_t launch_attn_fwd(int D, int in_type, int mode, const CUtensorMap& tq, const CUtensorMap& tk,
                            const CUtensorMap& tv, const AttnParams& p, cudaStream_t stream);
cudaError_t launch_weight_map(const float* x, float* w, size_t n, int mode, cudaStream_t stream);
cudaError_t launch_weight_map_pot(const float* x, float* w, size_t n, int kmax, int drop, cudaStream_t stream);
cudaError_t launch_weight_map_fused(const float* x, float* w, size_t n, int mode, int in_type, float pot_neg_cap,
                                    float pot_drop_x, cudaStream_t stream);
cudaError_t status_word_address(int** out);
cudaError_t launch_selftest_wait(int* status, long long limit_cycles, cudaStream_t stream);
}  // namespace rowmax

namespace {

std::atomic<unsigned long long> g_launches{0};
#ifdef ROWMAX_TRACE
long long* g_trace = nullptr;
int g_trace_block = 0;
#endif
int g_last_cuda_error = 0;

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                   CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres);
        if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || sym == nullptr) {
            g_last_cuda_error = static_cast<int>(e != cudaSuccess ? e : cudaErrorUnknown);
            return nullptr;
        }
        fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// Tensor (B, S, H, D) with D contiguous, viewed innermost-first as (D, H, S, B); one box is
// 128 bytes along D (64 when a row has only 64: fp8 with D = 64) by 128 rows along S of a single
// head, swizzled in shared memory with that span.
// Rows past S read as zero.
int make_tile_map(CUtensorMap* map, const void* base, bool fp8, bool half_in, int B, int S, int H, int D) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (enc == nullptr) return ATTN_ERR_CUDA;
    const cuuint64_t es = fp8 ? 1 : 2;
    cuuint64_t dims[4] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(H), static_cast<cuuint64_t>(S),
                          static_cast<cuuint64_t>(B)};
    cuuint64_t strides[3] = {static_cast<cuuint64_t>(D) * es, static_cast<cuuint64_t>(H) * D * es,
                             static_cast<cuuint64_t>(S) * H * D * es};
    const cuuint64_t row_bytes = static_cast<cuuint64_t>(D) * es;
    const cuuint64_t span = row_bytes >= 128 ? 128 : 64;   // swizzle span: a whole row when it has only 64 bytes
    cuuint32_t box[4] = {static_cast<cuuint32_t>(span / es), 1, 128, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(map, fp8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                              : (half_in ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16), 4,
                     const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     span == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        g_last_cuda_error = static_cast<int>(r);
        return ATTN_ERR_CUDA;
    }
    return ATTN_OK;
}

int check_arch() {
    static int cached_dev = -1, cached_ok = 0;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { g_last_cuda_error = e; return ATTN_ERR_CUDA; }
    if (dev != cached_dev) {
        int major = 0;
        e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) { g_last_cuda_error = e; return ATTN_ERR_CUDA; }
        cached_dev = dev;
        cached_ok = (major == 10);
    }
    return cached_ok ? ATTN_OK : ATTN_ERR_UNSUPPORTED_ARCH;
}

int status_word(int** out) {
    // one status word per device; looked up once per device
    static int* words[64] = {nullptr};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= 64) { g_last_cuda_error = e; return ATTN_ERR_CUDA; }
    if (words[dev] == nullptr) {
        e = rowmax::status_word_address(&words[dev]);
        if (e != cudaSuccess) { g_last_cuda_error = e; words[dev] = nullptr; return ATTN_ERR_CUDA; }
    }
    *out = words[dev];
    return ATTN_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" {

#ifdef ROWMAX_TRACE
// Trace builds only: device buffer of 4 * 64 * 8 int64 that CTA `block` fills with cycle stamps.
void attn_set_trace(long long* device_buffer, int block) {
    g_trace = device_buffer;
    g_trace_block = block;
}
#endif

}  // extern "C"

namespace {

// Every forward entry point ends here.  pot_kmax / pot_drop_tail matter in ATTN_W_POT mode only.
int fwd_impl(const void* q, const void* k, const void* v, void* o, float* lse, int B, int Hq, int Hkv, int Sq,
             int Sk, int D, int causal, float softmax_scale, int weight_mode, int in_dtype, float q_descale,
             float k_descale, float v_descale, float rescale_tau, int pot_kmax, int pot_drop_tail, int poly_eighths,
             void* stream) {
    if (!q || !k || !v || !o) return ATTN_ERR_NULLPTR;
    if (weight_mode < ATTN_W_EXACT || weight_mode > ATTN_W_EXACT_POLY) return ATTN_ERR_BAD_ENUM;
    if (in_dtype != ATTN_IN_BF16 && in_dtype != ATTN_IN_FP8_E4M3 && in_dtype != ATTN_IN_FP16) return ATTN_ERR_BAD_ENUM;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || Hq % Hkv != 0) return ATTN_ERR_BAD_SHAPE;
    if (D != 64 && D != 128) return ATTN_ERR_BAD_SHAPE;
    if (B > 65535 || Hq > 65535) return ATTN_ERR_BAD_SHAPE;  // grid y/z limits
    if (static_cast<long long>(Sq) + Sk >= (1ll << 30)) return ATTN_ERR_BAD_SHAPE;
    const bool fp8 = in_dtype == ATTN_IN_FP8_E4M3;
    if (!(softmax_scale > 0.f) || !std::isfinite(softmax_scale)) return ATTN_ERR_BAD_VALUE;
    if (fp8 && (!(q_descale > 0.f) || !(k_descale > 0.f) || !(v_descale > 0.f) || !std::isfinite(q_descale) ||
                !std::isfinite(k_descale) || !std::isfinite(v_descale)))
        return ATTN_ERR_BAD_VALUE;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return ATTN_ERR_MISALIGNED;
    if (!(rescale_tau >= 0.f) || !std::isfinite(rescale_tau) || rescale_tau > 32.f) return ATTN_ERR_BAD_VALUE;
    if (fp8 && rescale_tau != 0.f) return ATTN_ERR_UNSUPPORTED;   // the fp8 P formats have no headroom above the anchor
    if (in_dtype == ATTN_IN_FP16 && rescale_tau != 0.f) return ATTN_ERR_UNSUPPORTED;   // fp16 P: not built
    if (in_dtype == ATTN_IN_FP16 && weight_mode != ATTN_W_EXACT && weight_mode != ATTN_W_POT && weight_mode != ATTN_W_H15)
        return ATTN_ERR_UNSUPPORTED;
    const bool drop = pot_drop_tail != 0;
    if (weight_mode == ATTN_W_POT) {
        // the tail index must stay inside what the format of P can hold exactly (see attn_fwd_pot in attn.h)
        const int kmax_hi = fp8 ? ATTN_POT_KMAX_FP8 : (in_dtype == ATTN_IN_FP16 ? ATTN_POT_KMAX_FP16 : ATTN_POT_KMAX_BF16);
        if (pot_kmax < 1 || pot_kmax > kmax_hi) return ATTN_ERR_BAD_VALUE;
    }
    int rc = check_arch();
    if (rc != ATTN_OK) return rc;

    rowmax::AttnParams p{};
    p.o = o;
    p.lse = lse;
    p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.Sq = Sq; p.Sk = Sk;
    p.causal = causal != 0;
    p.group = Hq / Hkv;
    const double dq = fp8 ? static_cast<double>(q_descale) : 1.0;
    const double dk = fp8 ? static_cast<double>(k_descale) : 1.0;
    p.c = static_cast<float>(static_cast<double>(softmax_scale) * dq * dk * 1.4426950408889634074);
    p.v_descale = fp8 ? v_descale : 1.0f;
    p.two22 = 1u << 22;
    p.tau = rescale_tau;
    p.pot_neg_cap = -static_cast<float>(drop ? pot_kmax + 1 : pot_kmax);
    p.pot_drop_x = -(static_cast<float>(pot_kmax) + 0.5f);

#ifdef ROWMAX_TRACE
    p.trace = g_trace;
    p.trace_block = g_trace_block;
#endif
    rc = status_word(&p.status);
    if (rc != ATTN_OK) return rc;

    CUtensorMap tq, tk, tv;
    const bool half_in = in_dtype == ATTN_IN_FP16;
    if ((rc = make_tile_map(&tq, q, fp8, half_in, B, Sq, Hq, D)) != ATTN_OK) return rc;
    if ((rc = make_tile_map(&tk, k, fp8, half_in, B, Sk, Hkv, D)) != ATTN_OK) return rc;
    if ((rc = make_tile_map(&tv, v, fp8, half_in, B, Sk, Hkv, D)) != ATTN_OK) return rc;

    static_assert(ATTN_IN_BF16 == rowmax::kInBF16 && ATTN_IN_FP8_E4M3 == rowmax::kInFP8 && ATTN_IN_FP16 == rowmax::kInFP16,
                  "the kernel's storage-type codes are those of the C interface");
    int kernel_mode = (weight_mode == ATTN_W_POT && drop) ? rowmax::kPotDrop : weight_mode;
    if (weight_mode == ATTN_W_EXACT_POLY) {
        if (poly_eighths < 1 || poly_eighths > 4) return ATTN_ERR_BAD_VALUE;
        const int by_share[5] = {0, rowmax::kExactPoly1, rowmax::kExactPoly, rowmax::kExactPoly3, rowmax::kExactPoly4};
        kernel_mode = by_share[poly_eighths];
    }
    cudaError_t e = rowmax::launch_attn_fwd(D, in_dtype, kernel_mode, tq, tk, tv, p, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) {
        g_last_cuda_error = static_cast<int>(e);
        return e == cudaErrorInvalidValue ? ATTN_ERR_UNSUPPORTED : ATTN_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return ATTN_OK;
}

}  // namespace

extern "C" {

int attn_fwd_tau(const void* q, const void* k, const void* v, void* o, float* lse, int B, int Hq, int Hkv, int Sq,
                 int Sk, int D, int causal, float softmax_scale, int weight_mode, int in_dtype, float q_descale,
                 float k_descale, float v_descale, float rescale_tau, void* stream) {
    return fwd_impl(q, k, v, o, lse, B, Hq, Hkv, Sq, Sk, D, causal, softmax_scale, weight_mode, in_dtype, q_descale,
                    k_descale, v_descale, rescale_tau, ATTN_POT_KMAX_DEFAULT, 0, 2, stream);
}

int attn_fwd_exact_emulated(const void* q, const void* k, const void* v, void* o, float* lse, int B, int Hq, int Hkv,
                            int Sq, int Sk, int D, int causal, float softmax_scale, int in_dtype, float q_descale,
                            float k_descale, float v_descale, int share_eighths, void* stream) {
    return fwd_impl(q, k, v, o, lse, B, Hq, Hkv, Sq, Sk, D, causal, softmax_scale, ATTN_W_EXACT_POLY, in_dtype, q_descale,
                    k_descale, v_descale, 0.0f, ATTN_POT_KMAX_DEFAULT, 0, share_eighths, stream);
}

int attn_fwd_pot(const void* q, const void* k, const void* v, void* o, float* lse, int B, int Hq, int Hkv, int Sq,
                 int Sk, int D, int causal, float softmax_scale, int in_dtype, float q_descale, float k_descale,
                 float v_descale, int pot_kmax, int drop_tail, void* stream) {
    return fwd_impl(q, k, v, o, lse, B, Hq, Hkv, Sq, Sk, D, causal, softmax_scale, ATTN_W_POT, in_dtype, q_descale,
                    k_descale, v_descale, 0.0f, pot_kmax, drop_tail, 2, stream);
}

int attn_fwd(const void* q, const void* k, const void* v, void* o, float* lse, int B, int Hq, int Hkv, int Sq,
             int Sk, int D, int causal, float softmax_scale, int weight_mode, int in_dtype, float q_descale,
             float k_descale, float v_descale, void* stream) {
    return attn_fwd_tau(q, k, v, o, lse, B, Hq, Hkv, Sq, Sk, D, causal, softmax_scale, weight_mode, in_dtype,
                        q_descale, k_descale, v_descale, 0.0f, stream);
}

int attn_weight_map(const float* x, float* w, size_t n, int weight_mode, void* stream) {
    if (n == 0) return ATTN_OK;
    if (!x || !w) return ATTN_ERR_NULLPTR;
    if (weight_mode < ATTN_W_EXACT || weight_mode > ATTN_W_EXACT_POLY) return ATTN_ERR_BAD_ENUM;
    cudaError_t e = rowmax::launch_weight_map(x, w, n, weight_mode, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) {
        g_last_cuda_error = static_cast<int>(e);
        return ATTN_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return ATTN_OK;
}

int attn_weight_map_pot(const float* x, float* w, size_t n, int pot_kmax, int drop_tail, void* stream) {
    if (n == 0) return ATTN_OK;
    if (!x || !w) return ATTN_ERR_NULLPTR;
    if (pot_kmax < 1 || pot_kmax > ATTN_POT_KMAX_BF16) return ATTN_ERR_BAD_VALUE;
    cudaError_t e = rowmax::launch_weight_map_pot(x, w, n, pot_kmax, drop_tail != 0, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) {
        g_last_cuda_error = static_cast<int>(e);
        return ATTN_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return ATTN_OK;
}

int attn_weight_map_fused(const float* x, float* w, size_t n, int weight_mode, int in_dtype, int pot_kmax, int drop_tail,
                          void* stream) {
    if (n == 0) return ATTN_OK;
    if (!x || !w) return ATTN_ERR_NULLPTR;
    if (weight_mode < ATTN_W_EXACT || weight_mode > ATTN_W_EXACT_POLY) return ATTN_ERR_BAD_ENUM;
    if (in_dtype != ATTN_IN_BF16 && in_dtype != ATTN_IN_FP8_E4M3 && in_dtype != ATTN_IN_FP16) return ATTN_ERR_BAD_ENUM;
    const int kmax_hi = in_dtype == ATTN_IN_FP8_E4M3 ? ATTN_POT_KMAX_FP8 : (in_dtype == ATTN_IN_FP16 ? ATTN_POT_KMAX_FP16 : ATTN_POT_KMAX_BF16);
    if (weight_mode == ATTN_W_POT && (pot_kmax < 1 || pot_kmax > kmax_hi)) return ATTN_ERR_BAD_VALUE;
    const bool drop = drop_tail != 0;
    const int kernel_mode = (weight_mode == ATTN_W_POT && drop) ? rowmax::kPotDrop : weight_mode;
    cudaError_t e = rowmax::launch_weight_map_fused(x, w, n, kernel_mode, in_dtype, -static_cast<float>(drop ? pot_kmax + 1 : pot_kmax),
                                                    -(static_cast<float>(pot_kmax) + 0.5f), static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) {
        g_last_cuda_error = static_cast<int>(e);
        return e == cudaErrorInvalidValue ? ATTN_ERR_UNSUPPORTED : ATTN_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return ATTN_OK;
}

int attn_get_schedule(int D, int in_dtype, int weight_mode, int causal, int* tile_m, int* tile_n, int* kv_order,
                      float* rescale_tau, int* pot_kmax, int* p_format, int* p_offset_log2) {
    (void)causal;
    if (D != 64 && D != 128) return ATTN_ERR_BAD_SHAPE;
    if (in_dtype != ATTN_IN_BF16 && in_dtype != ATTN_IN_FP8_E4M3 && in_dtype != ATTN_IN_FP16) return ATTN_ERR_BAD_ENUM;
    if (weight_mode < ATTN_W_EXACT || weight_mode > ATTN_W_EXACT_POLY) return ATTN_ERR_BAD_ENUM;
    const bool fp8 = in_dtype == ATTN_IN_FP8_E4M3;
    if (tile_m) *tile_m = rowmax::kTileM;
    if (tile_n) *tile_n = rowmax::kTileN;
    if (kv_order) *kv_order = +1;
    if (rescale_tau) *rescale_tau = 0.0f;
    if (pot_kmax) *pot_kmax = ATTN_POT_KMAX_DEFAULT;
    const bool e4m3 = weight_mode == ATTN_W_EXACT || weight_mode == ATTN_W_EXACT_POLY || weight_mode == ATTN_W_H15K3;
    if (p_format) *p_format = in_dtype == ATTN_IN_FP16 ? ATTN_P_FP16 : !fp8 ? ATTN_P_BF16 : (e4m3 ? ATTN_P_E4M3 : ATTN_P_E5M2);
    if (p_offset_log2) *p_offset_log2 = !fp8 ? 0 : (e4m3 ? 8 : 15);
    return ATTN_OK;
}

// Synchronises the device and reads the status word; *code gets the raw word.
static int read_status_word(int* code) {
    int* word = nullptr;
    int rc = status_word(&word);
    if (rc != ATTN_OK) return rc;
    int host = 0;
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(&host, word, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) { g_last_cuda_error = static_cast<int>(e); return ATTN_ERR_CUDA; }
    *code = host;
    return ATTN_OK;
}

int attn_device_status(void) {
    int code = 0;
    int rc = read_status_word(&code);
    if (rc != ATTN_OK) return rc;
    return code != 0 ? ATTN_ERR_TIMEOUT : ATTN_OK;
}

int attn_device_status_code(void) {
    int code = 0;
    int rc = read_status_word(&code);
    return rc != ATTN_OK ? rc : code;
}

int attn_selftest_wait(long long limit_cycles, void* stream) {
    if (limit_cycles <= 0 || limit_cycles > 2000000000LL) return ATTN_ERR_BAD_VALUE;
    int rc = check_arch();
    if (rc != ATTN_OK) return rc;
    int* word = nullptr;
    rc = status_word(&word);
    if (rc != ATTN_OK) return rc;
    cudaError_t e = rowmax::launch_selftest_wait(word, limit_cycles, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { g_last_cuda_error = static_cast<int>(e); return ATTN_ERR_CUDA; }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return ATTN_OK;
}

int attn_device_status_reset(void) {
    int* word = nullptr;
    int rc = status_word(&word);
    if (rc != ATTN_OK) return rc;
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemset(word, 0, sizeof(int));
    if (e != cudaSuccess) { g_last_cuda_error = static_cast<int>(e); return ATTN_ERR_CUDA; }
    return ATTN_OK;
}

unsigned long long attn_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* attn_status_string(int status) {
    switch (status) {
        case ATTN_OK: return "ok";
        case ATTN_ERR_NULLPTR: return "null pointer";
        case ATTN_ERR_BAD_SHAPE: return "bad shape";
        case ATTN_ERR_BAD_ENUM: return "bad enum value";
        case ATTN_ERR_MISALIGNED: return "pointer not 16-byte aligned";
        case ATTN_ERR_UNSUPPORTED_ARCH: return "device is not sm_100";
        case ATTN_ERR_CUDA: return "CUDA call failed";
        case ATTN_ERR_TIMEOUT: return "device-side wait expired";
        case ATTN_ERR_UNSUPPORTED: return "combination not built";
        case ATTN_ERR_BAD_VALUE: return "scale or descale not positive and finite";
        default: return "unknown status";
    }
}

int attn_last_cuda_error(void) { return g_last_cuda_error; }

const char* attn_version(void) { return "rowmax-attn-b200 0.1"; }

}  // extern "C"
