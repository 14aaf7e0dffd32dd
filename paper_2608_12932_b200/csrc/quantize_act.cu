// Per-token dynamic activation quantisation, bf16 -> int8 (Sec. 3.4: activations are quantised to 8 bits).
//
// One CTA per token row.  Each thread owns 16-byte chunks (8 bf16) of the row, keeps them
// in registers across the two passes (absmax, then quantise), so the row is read from
// HBM once: 2 B in, 1 B out per element.  The scale is fp16_rne(amax/127); codes are
// rne(x / s_a) of the exact quotient.  A bf16 over an fp16 value is either an exact tie or at
// least 2^-12 from one, so the correctly rounded fp32 quotient (IEEE division) rounds to the same
// integer as the exact one.  A reciprocal multiply alone would break exact ties, but it is within
// 2^-16 of the quotient: the kernel multiplies, rounds with the 1.5 * 2^23 trick (the code is then
// the low byte of the sum's mantissa), and sends only the 16-byte chunks in which some product came
// within 2^-13 of a half-integer - every exact tie, and nothing that is not nearly one - back to the
// division.  Eight instructions per element instead of about thirty.  Group sums of the codes (the
// zero-point correction term) come from a 16-lane segmented shuffle: 16 chunks of 8 = one group of 128.
#include <cuda_fp16.h>
#include "ptx_sm100.cuh"
#include "quant_common.cuh"
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

// Fast path of a chunk (see the header): products with the row's reciprocal scale.  `worst` returns the largest
// distance of a product from the integer it was rounded to.  Valid for rows whose scale did not saturate
// (|x / s_a| < 127.1, so the rounded value needs no clamp).
__device__ __forceinline__ uint32_t quant4_fast(uint32_t lo_pair, uint32_t hi_pair, float rinv, float& worst) {
    constexpr float MAGIC = 12582912.0f;                     // 1.5 * 2^23: adding it rounds to an integer, ties to even
    const float t0 = __fmul_rn(__uint_as_float(lo_pair << 16), rinv), t1 = __fmul_rn(__uint_as_float(lo_pair & 0xFFFF0000u), rinv);
    const float t2 = __fmul_rn(__uint_as_float(hi_pair << 16), rinv), t3 = __fmul_rn(__uint_as_float(hi_pair & 0xFFFF0000u), rinv);
    const float y0 = __fadd_rn(t0, MAGIC), y1 = __fadd_rn(t1, MAGIC), y2 = __fadd_rn(t2, MAGIC), y3 = __fadd_rn(t3, MAGIC);
    worst = fmaxf(worst, fmaxf(fmaxf(fabsf(__fsub_rn(t0, __fsub_rn(y0, MAGIC))), fabsf(__fsub_rn(t1, __fsub_rn(y1, MAGIC)))),
                               fmaxf(fabsf(__fsub_rn(t2, __fsub_rn(y2, MAGIC))), fabsf(__fsub_rn(t3, __fsub_rn(y3, MAGIC))))));
    // low mantissa bytes of y0..y3 -> one word
    const uint32_t a = __byte_perm(__float_as_uint(y0), __float_as_uint(y1), 0x0040);
    const uint32_t b = __byte_perm(__float_as_uint(y2), __float_as_uint(y3), 0x0040);
    return __byte_perm(a, b, 0x5410);
}

// QA_THREADS threads per token row: 256 for many rows (more rows in flight per SM), 512 or 1024 for fewer
// (a row's latency chain - load, row maximum, divisions, store - is then shorter per thread).
// QA_CACHE: 16-byte chunks per thread kept in registers between the two passes (rows up to QA_THREADS * QA_CACHE * 8
// elements are read once; a small cache leaves room for more rows per SM).  FAST: reciprocal multiply with the
// division as the tie fallback - for many rows, where instruction issue matters; with few rows the kernel is a single
// latency chain and the shorter code of the plain division is quicker (1.8 against 1.9 us at 8 rows, 2.0 against
// 2.7 us at 128).
//
// SILU: the input row is the bf16 output of a fused gate+up projection, 2 K values in 16-byte chunks that
// alternate between eight gate channels and the eight up channels of the same indices; the row that is quantised
// is h = bf16(SiLU(gate) * up), K values, computed chunk by chunk as it is loaded (Sec. 3.5: the element-wise
// step merged into its consumer) and, if h_out is given, also stored.
template <int QA_THREADS, int QA_CACHE, bool FAST, bool SILU>
__global__ void __launch_bounds__(QA_THREADS, QA_THREADS == 256 ? (QA_CACHE == 2 ? 8 : 5) : (QA_THREADS == 512 ? 3 : 1))
quantize_act_kernel(const uint4* __restrict__ x, int K, uint2* __restrict__ qa,
                    uint16_t* __restrict__ sa, int32_t* __restrict__ asum, uint4* __restrict__ h_out) {
    // Under programmatic dependent launch this grid may start while its predecessor still runs:
    // let the next grid start as early, and touch no memory before the predecessor is complete.
    ptx::pdl_launch_dependents();
    ptx::pdl_wait();
    const int m = blockIdx.x;
    const int chunks = K >> 3;                    // 16-byte chunks per row; a multiple of 16
    const int G = K >> 7;
    const uint4* xr = x + (size_t)m * chunks * (SILU ? 2 : 1);
    uint2* qr = qa + (size_t)m * chunks;
    // chunk c of the row to quantise
    auto load = [&](int c) -> uint4 {
        if (!SILU) return __ldcg(xr + c);
        const uint4 g = __ldcg(xr + 2 * c), u = __ldcg(xr + 2 * c + 1);
        uint4 h;
        h.x = silu_mul_bf16x2(g.x, u.x);
        h.y = silu_mul_bf16x2(g.y, u.y);
        h.z = silu_mul_bf16x2(g.z, u.z);
        h.w = silu_mul_bf16x2(g.w, u.w);
        return h;
    };
    const int tid = threadIdx.x;

    uint4 cache[QA_CACHE];
    uint32_t run = 0;
#pragma unroll
    for (int i = 0; i < QA_CACHE; ++i) {
        int c = tid + i * QA_THREADS;
        if (c < chunks) {
            cache[i] = load(c);
            run = absmax_bits_bf16x8(cache[i], run);
        }
    }
    for (int c = tid + QA_CACHE * QA_THREADS; c < chunks; c += QA_THREADS)
        run = absmax_bits_bf16x8(load(c), run);

    uint32_t mx = max(run & 0xFFFFu, run >> 16);
    mx = __reduce_max_sync(0xFFFFFFFFu, mx);
    __shared__ uint32_t warp_max[QA_THREADS / 32];
    if ((tid & 31) == 0) warp_max[tid >> 5] = mx;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < QA_THREADS / 32; ++w) mx = max(mx, warp_max[w]);

    const __half sh = row_scale_from_amax_bits(mx);
    const float s = __half2float(sh);
    if (tid == 0) sa[m] = __half_as_ushort(sh);
    // the fast path needs a quotient that cannot leave [-127.1, 127.1]: not for a saturated scale
    const bool fast_row = FAST && __half_as_ushort(sh) < 0x7BFFu;
    const float rinv = s != 0.0f ? __frcp_rn(s) : 0.0f;

    // chunks c..c+15 (c a multiple of 16) are one group of 128 and sit in the 16 lanes of one
    // half-warp; chunks is a multiple of 16, so a half-warp is in range or out of it as a whole
    // and shuffles under its own 16-lane mask.
    const uint32_t seg_mask = (tid & 16) ? 0xFFFF0000u : 0x0000FFFFu;
    auto emit = [&](int c, const uint4& v) {
        int sum = 0;
        uint2 o = make_uint2(0u, 0u);
        if (s != 0.0f) {
            float worst = 1.0f;
            if (fast_row) {
                worst = 0.0f;
                o.x = quant4_fast(v.x, v.y, rinv, worst);
                o.y = quant4_fast(v.z, v.w, rinv, worst);
                sum = __dp4a((int)o.x, 0x01010101, __dp4a((int)o.y, 0x01010101, 0));
            }
            if (worst > 0.5f - 0.0001220703125f) o = quant8(v, s, sum);      // 2^-13: a possible tie in this chunk
        }
        qr[c] = o;
        if (SILU && h_out) h_out[(size_t)m * chunks + c] = v;
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
    for (int c = tid + QA_CACHE * QA_THREADS; c < chunks; c += QA_THREADS) emit(c, load(c));
}

}  // namespace

namespace {
template <bool SILU>
cudaError_t launch_quantize(const void* x, int M, int K, int8_t* qa, uint16_t* sa, int32_t* asum, void* h_out,
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
    const uint4* xp = reinterpret_cast<const uint4*>(x);
    uint2* qp = reinterpret_cast<uint2*>(qa);
    uint4* hp = reinterpret_cast<uint4*>(h_out);
    if (threads == 1024)
        return cudaLaunchKernelEx(&cfg, quantize_act_kernel<1024, QA_CACHE_CHUNKS / 1024, false, SILU>, xp, K, qp, sa, asum, hp);
    if (threads == 512)
        return cudaLaunchKernelEx(&cfg, quantize_act_kernel<512, QA_CACHE_CHUNKS / 512, false, SILU>, xp, K, qp, sa, asum, hp);
    if (K <= 256 * 2 * 8)                                    // rows of up to 4096: two chunks per thread, eight rows per SM
        return cudaLaunchKernelEx(&cfg, quantize_act_kernel<256, 2, true, SILU>, xp, K, qp, sa, asum, hp);
    return cudaLaunchKernelEx(&cfg, quantize_act_kernel<256, QA_CACHE_CHUNKS / 256, true, SILU>, xp, K, qp, sa, asum, hp);
}
}  // namespace

cudaError_t launch_quantize_act(const void* x, int M, int K, int8_t* qa, uint16_t* sa, int32_t* asum,
                                cudaStream_t stream) {
    return launch_quantize<false>(x, M, K, qa, sa, asum, nullptr, stream);
}

// y_gate_up: bf16 [M, 2 I] in the chunk-interleaved layout; quantises h = SiLU(gate) * up, [M, I]
cudaError_t launch_silu_mul_quantize(const void* y_gate_up, int M, int I, void* h_out, int8_t* qa, uint16_t* sa,
                                     int32_t* asum, cudaStream_t stream) {
    return launch_quantize<true>(y_gate_up, M, I, qa, sa, asum, h_out, stream);
}

}  // namespace w4a8
