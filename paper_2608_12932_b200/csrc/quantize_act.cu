// Per-token dynamic activation quantisation, bf16 -> int8 (Sec. 3.4: activations are quantised to 8 bits).
//
// One CTA per token row.  Each thread owns 16-byte chunks (8 bf16) of the row, keeps them
// in registers across the two passes (absmax, then quantise), so the row is read from
// HBM once: 2 B in, 1 B out per element.  The scale is fp16_rne(amax/127); codes are
// cvt.rni(x / s_a) with an IEEE fp32 division (never a reciprocal multiply: a bf16 over
// an fp16 value is either an exact tie or at least 2^-12 from one, so the correctly
// rounded fp32 quotient rounds to the same integer as the exact one; a reciprocal would
// break exact ties).  Group sums of the codes (the zero-point correction term) come from
// a 16-lane segmented shuffle: 16 chunks of 8 = one group of 128.
#include <cuda_fp16.h>
#include "ptx_sm100.cuh"
#include "w4a8_internal.cuh"

namespace w4a8 {
namespace {

constexpr int QA_CACHE_CHUNKS = 1536;   // 16-byte chunks of a row kept in registers: rows up to 12288 read once

__device__ __forceinline__ uint32_t absmax_bits_bf16x8(const uint4& v, uint32_t run) {
    // bf16 magnitudes order like their 15-bit patterns: keep a packed running max of two lanes
    run = __vmaxu2(run, v.x & 0x7FFF7FFFu);
    run = __vmaxu2(run, v.y & 0x7FFF7FFFu);
    run = __vmaxu2(run, v.z & 0x7FFF7FFFu);
    run = __vmaxu2(run, v.w & 0x7FFF7FFFu);
    return run;
}

__device__ __forceinline__ int quant1(uint32_t bf16_hi_bits, float s) {
    // bf16_hi_bits: the value's bits already in the upper half of a 32-bit word
    float q = __fdiv_rn(__uint_as_float(bf16_hi_bits), s);
    int r;
    asm("cvt.rni.sat.s8.f32 %0, %1;" : "=r"(r) : "f"(q));   // ties to even, saturates to [-128,127]
    return max(r, -127);
}

__device__ __forceinline__ uint2 quant8(const uint4& v, float s, int& sum) {
    int q0 = quant1(v.x << 16, s), q1 = quant1(v.x & 0xFFFF0000u, s);
    int q2 = quant1(v.y << 16, s), q3 = quant1(v.y & 0xFFFF0000u, s);
    int q4 = quant1(v.z << 16, s), q5 = quant1(v.z & 0xFFFF0000u, s);
    int q6 = quant1(v.w << 16, s), q7 = quant1(v.w & 0xFFFF0000u, s);
    sum = q0 + q1 + q2 + q3 + q4 + q5 + q6 + q7;
    uint2 o;
    o.x = (q0 & 0xFF) | ((q1 & 0xFF) << 8) | ((q2 & 0xFF) << 16) | ((uint32_t)q3 << 24);
    o.y = (q4 & 0xFF) | ((q5 & 0xFF) << 8) | ((q6 & 0xFF) << 16) | ((uint32_t)q7 << 24);
    return o;
}

// QA_THREADS threads per token row: 256 for many rows (more rows in flight per SM), 512 or 1024 for fewer
// (a row's latency chain - load, row maximum, divisions, store - is then shorter per thread).
template <int QA_THREADS>
__global__ void __launch_bounds__(QA_THREADS)
quantize_act_kernel(const uint4* __restrict__ x, int K, uint2* __restrict__ qa,
                    uint16_t* __restrict__ sa, int32_t* __restrict__ asum) {
    // Under programmatic dependent launch this grid may start while its predecessor still runs:
    // let the next grid start as early, and touch no memory before the predecessor is complete.
    ptx::pdl_launch_dependents();
    ptx::pdl_wait();
    const int m = blockIdx.x;
    const int chunks = K >> 3;                    // 16-byte chunks per row; a multiple of 16
    const int G = K >> 7;
    const uint4* xr = x + (size_t)m * chunks;
    uint2* qr = qa + (size_t)m * chunks;
    const int tid = threadIdx.x;
    constexpr int QA_CACHE = QA_CACHE_CHUNKS / QA_THREADS;

    uint4 cache[QA_CACHE];
    uint32_t run = 0;
#pragma unroll
    for (int i = 0; i < QA_CACHE; ++i) {
        int c = tid + i * QA_THREADS;
        if (c < chunks) {
            cache[i] = __ldcg(xr + c);
            run = absmax_bits_bf16x8(cache[i], run);
        }
    }
    for (int c = tid + QA_CACHE * QA_THREADS; c < chunks; c += QA_THREADS)
        run = absmax_bits_bf16x8(__ldcg(xr + c), run);

    uint32_t mx = max(run & 0xFFFFu, run >> 16);
    mx = __reduce_max_sync(0xFFFFFFFFu, mx);
    __shared__ uint32_t warp_max[QA_THREADS / 32];
    if ((tid & 31) == 0) warp_max[tid >> 5] = mx;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < QA_THREADS / 32; ++w) mx = max(mx, warp_max[w]);

    const float amax = __uint_as_float(mx << 16);
    const __half sh = __float2half_rn(fminf(__fdiv_rn(amax, 127.0f), 65504.0f));
    const float s = __half2float(sh);
    if (tid == 0) sa[m] = __half_as_ushort(sh);

    // chunks c..c+15 (c a multiple of 16) are one group of 128 and sit in the 16 lanes of one
    // half-warp; chunks is a multiple of 16, so a half-warp is in range or out of it as a whole
    // and shuffles under its own 16-lane mask.
    const uint32_t seg_mask = (tid & 16) ? 0xFFFF0000u : 0x0000FFFFu;
    auto emit = [&](int c, const uint4& v) {
        int sum = 0;
        uint2 o = make_uint2(0u, 0u);
        if (s != 0.0f) o = quant8(v, s, sum);
        qr[c] = o;
        sum += __shfl_xor_sync(seg_mask, sum, 8);
        sum += __shfl_xor_sync(seg_mask, sum, 4);
        sum += __shfl_xor_sync(seg_mask, sum, 2);
        sum += __shfl_xor_sync(seg_mask, sum, 1);
        if ((c & 15) == 0) asum[(size_t)m * G + (c >> 4)] = sum;
    };
#pragma unroll
    for (int i = 0; i < QA_CACHE; ++i) {
        int c = tid + i * QA_THREADS;
        if (c < chunks) emit(c, cache[i]);
    }
    for (int c = tid + QA_CACHE * QA_THREADS; c < chunks; c += QA_THREADS) emit(c, __ldcg(xr + c));
}

}  // namespace

cudaError_t launch_quantize_act(const void* x, int M, int K, int8_t* qa, uint16_t* sa, int32_t* asum,
                                cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)M, 1, 1);
    // measured on B200 (K = 4096 and 12288): 512 threads per row are best up to 512 rows except between
    // about 64 and 128 rows, where 1024 are; from 1024 rows on 256 are
    const int threads = M > 512 ? 256 : ((M > 48 && M <= 192) ? 1024 : 512);
    cfg.blockDim = dim3((unsigned)threads, 1, 1);
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    if (threads == 1024)
        return cudaLaunchKernelEx(&cfg, quantize_act_kernel<1024>, reinterpret_cast<const uint4*>(x), K,
                                  reinterpret_cast<uint2*>(qa), sa, asum);
    if (threads == 512)
        return cudaLaunchKernelEx(&cfg, quantize_act_kernel<512>, reinterpret_cast<const uint4*>(x), K,
                                  reinterpret_cast<uint2*>(qa), sa, asum);
    return cudaLaunchKernelEx(&cfg, quantize_act_kernel<256>, reinterpret_cast<const uint4*>(x), K,
                              reinterpret_cast<uint2*>(qa), sa, asum);
}

}  // namespace w4a8
