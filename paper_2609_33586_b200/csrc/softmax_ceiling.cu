// Stand-alone measurement of what the SIMT side of the attention kernel can do at best: the softmax
// arithmetic of one key tile (scores read from TMEM, row maximum, anchor update, weight map, row sum,
// P packed and written back to TMEM) in a loop, with no tensor-core work, no barriers and no other
// warps.  It uses the same device functions as the fused kernel (softmax_math.cuh, weight_map.cuh)
// and prints scores per clock per SM for several numbers of resident warps and scores per thread.
// Built and run by `python -m paper_2609_33586_b200.softmax_ceiling`.
#include <cstdint>
#include <cstdio>

#include <cuda_runtime.h>

#include "softmax_math.cuh"

using namespace rowmax;

namespace {

constexpr int kIters = 64;

template <int NC>
__device__ __forceinline__ float max_chunks(const uint32_t (&s)[NC][32]) {
    float m[8];
#pragma unroll
    for (int a = 0; a < 8; ++a) m[a] = -INFINITY;
#pragma unroll
    for (int cc = 0; cc < NC; ++cc)
#pragma unroll
        for (int i = 0; i < 32; i += 16)
#pragma unroll
            for (int a = 0; a < 8; ++a)
                m[a] = max3(m[a], __uint_as_float(s[cc][i + 2 * a]), __uint_as_float(s[cc][i + 2 * a + 1]));
    return fmaxf(max3(m[0], m[1], m[2]), max3(m[3], m[4], max3(m[5], m[6], m[7])));
}
template <int NC>
__device__ __forceinline__ float min_chunks(const uint32_t (&s)[NC][32]) {
    float m[8];
#pragma unroll
    for (int a = 0; a < 8; ++a) m[a] = INFINITY;
#pragma unroll
    for (int cc = 0; cc < NC; ++cc)
#pragma unroll
        for (int i = 0; i < 32; i += 16)
#pragma unroll
            for (int a = 0; a < 8; ++a)
                m[a] = min3(m[a], __uint_as_float(s[cc][i + 2 * a]), __uint_as_float(s[cc][i + 2 * a + 1]));
    return fminf(min3(m[0], m[1], m[2]), min3(m[3], m[4], min3(m[5], m[6], m[7])));
}

// NC chunks of 32 scores per thread; MINPASS: the h15 row-minimum pass that decides about the clamp.
template <bool FP8, int MODE, int NC, int THREADS, bool MINPASS>
__global__ void __launch_bounds__(THREADS, 1) ceiling_kernel(uint32_t* out, long long* cycles, float c, uint32_t two22) {
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5;
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_base + ((warp >> 2) * (NC * 32)) % 512;
    {   // finite, varied scores
        uint32_t z[32];
        for (int i = 0; i < 32; ++i) z[i] = __float_as_uint(-static_cast<float>((threadIdx.x * 7 + i * 13) % 97));
        for (int cc = 0; cc < NC; ++cc) tmem_st32(tS + cc * 32, z);
        tmem_wait_st();
    }
    float m_run = -INFINITY, l_run = 0.f, drift = 0.f;
    __syncthreads();
    const long long t0 = clock64();
    for (int it = 0; it < kIters; ++it) {
        uint32_t s[NC][32];
#pragma unroll
        for (int cc = 0; cc < NC; ++cc) tmem_ld32(tS + cc * 32, s[cc]);
        tmem_wait_ld();
        const float m_new = fmaxf(m_run, max_chunks<NC>(s));
        const float alpha = ex2_approx((m_run - m_new) * c);
        m_run = m_new;
        constexpr int kFam = h15_family_k(MODE);
        const float c_eff = static_cast<float>(1 << kFam) * c;
        RowScale rs;
        rs.c = make_float2(c_eff, c_eff);
        const float nmc = -m_new * c_eff + drift;   // drifts so that iterations are not identical
        rs.nmc = make_float2(nmc, nmc);
        rs.two22 = two22;
        rs.clamp_lo = -126.0f * (1 << kFam);
        float2 acc[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
        bool clamp = false;
        if (MINPASS && kFam > 0) {
            const float lowest = (min_chunks<NC>(s) - m_new) * c_eff;
            clamp = __any_sync(0xffffffffu, !(lowest >= -125.0f * (1 << kFam)));
        }
        if (clamp) {
#pragma unroll
            for (int cc = 0; cc < NC; ++cc) {
                uint32_t pw[16];
                weights_chunk32<FP8, MODE, false, true>(s[cc], rs, 32, acc, pw);
                if constexpr (FP8) tmem_st8(tS + cc * 8, pw);
                else tmem_st16(tS + cc * 16, pw);
            }
        } else {
#pragma unroll
            for (int cc = 0; cc < NC; ++cc) {
                uint32_t pw[16];
                weights_chunk32<FP8, MODE, false, false>(s[cc], rs, 32, acc, pw);
                if constexpr (FP8) tmem_st8(tS + cc * 8, pw);
                else tmem_st16(tS + cc * 16, pw);
            }
        }
        tmem_wait_st();
        l_run = l_run * alpha + (acc[0].x + acc[0].y) + (acc[1].x + acc[1].y);
        drift += 0.0625f;
    }
    const long long t1 = clock64();
    out[blockIdx.x * blockDim.x + threadIdx.x] = __float_as_uint(l_run);
    if (threadIdx.x == 0 && blockIdx.x == 0) *cycles = t1 - t0;
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

template <bool FP8, int MODE, int NC, int THREADS, bool MINPASS>
void run(const char* name, uint32_t* out, long long* cycles, int sms) {
    for (int rep = 0; rep < 2; ++rep)
        ceiling_kernel<FP8, MODE, NC, THREADS, MINPASS><<<sms, THREADS>>>(out, cycles, 0.1275f, 1u << 22);
    long long h = 0;
    cudaError_t e = cudaMemcpy(&h, cycles, sizeof(h), cudaMemcpyDeviceToHost);
    const double per_iter = static_cast<double>(h) / kIters;
    const double scores = static_cast<double>(THREADS) * NC * 32;
    printf("%-22s %3d scores/thread %2d warps/SM : %7.1f clocks/iteration  %5.2f scores/clock/SM  (128x128 tile in %4.0f clocks)  %s\n",
           name, NC * 32, THREADS / 32, per_iter, scores / per_iter, 16384.0 * per_iter / scores, cudaGetErrorString(e));
}

}  // namespace

int main() {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0) != cudaSuccess || sms <= 0) {
        fprintf(stderr, "no CUDA device\n");
        return 1;
    }
    uint32_t* out = nullptr;
    long long* cycles = nullptr;
    if (cudaMalloc(&out, 1 << 20) != cudaSuccess || cudaMalloc(&cycles, sizeof(long long)) != cudaSuccess) return 1;
    run<true, kH15, 4, 128, false>("fp8 h15", out, cycles, sms);
    run<true, kH15, 4, 256, false>("fp8 h15", out, cycles, sms);
    run<true, kH15, 2, 512, false>("fp8 h15", out, cycles, sms);
    run<true, kH15, 1, 1024, false>("fp8 h15", out, cycles, sms);
    run<true, kH15, 4, 256, true>("fp8 h15 + min pass", out, cycles, sms);
    run<true, kExact, 4, 128, false>("fp8 exact", out, cycles, sms);
    run<true, kExact, 4, 256, false>("fp8 exact", out, cycles, sms);
    run<true, kExact, 2, 512, false>("fp8 exact", out, cycles, sms);
    run<true, kPot, 4, 256, false>("fp8 pot", out, cycles, sms);
    run<false, kH15, 4, 256, false>("bf16 h15", out, cycles, sms);
    run<false, kH15, 4, 256, true>("bf16 h15 + min pass", out, cycles, sms);
    run<false, kExact, 4, 256, false>("bf16 exact", out, cycles, sms);
    const cudaError_t e = cudaDeviceSynchronize();
    printf("%s\n", cudaGetErrorString(e));
    cudaFree(out);
    cudaFree(cycles);
    return e == cudaSuccess ? 0 : 1;
}
