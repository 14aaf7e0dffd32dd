// Two pieces of streaming prefill that sit beside the quantised linears (Sec. 3.1, "Streaming design").
//
// rope_shifted_keys_kernel: keys are cached BEFORE the rotary embedding, because a cached token's position changes
// when the window slides (what was at p is now at p - delta); the rotation is applied when the keys are used, at
// the shifted positions.  Rotate-half form: with i < D/2, theta_i = base^(-2i/D), phi = (pos[t] - delta) theta_i,
//   out[i] = k[i] cos(phi) - k[i + D/2] sin(phi),   out[i + D/2] = k[i + D/2] cos(phi) + k[i] sin(phi).
// One warp per token, all its heads (the angles do not depend on the head); a lane owns the same two i for every token
// it meets, so its two theta are computed once, in fp64; the angle is formed and reduced to [-pi, pi] in fp64 (a position of several thousand times theta_0 = 1
// has no bits to spare in fp32), its sine and cosine are taken in fp32, the products and sums in fp32, one rounding to
// bf16.  Memory-bound: 2 B in and 2 B out per element, 4-byte accesses that a warp makes in two 128-byte runs.
//
// streaming_mask_kernel: the new frame's tokens are inserted at the last-frame place of each camera view (the
// sequence is view-major), only they are queries, and attention stays causal in that order:
//   mask[q][j] = (j <= position of query q),  position of query (v, i) = ((v F + F - 1) n + i).
#include <cuda_bf16.h>
#include "w4a8_internal.cuh"

namespace w4a8 {
namespace {

constexpr int ROPE_WARPS = 8;

__global__ void __launch_bounds__(ROPE_WARPS * 32)
rope_shifted_keys_kernel(const uint32_t* __restrict__ k_pre, const int32_t* __restrict__ pos, int delta, int T, int H, int D,
                         double log2_base, uint32_t* __restrict__ k_rot) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int half = D >> 1, pairs = half >> 1;              // 32-bit words (two bf16) per half row
    const double two_pi = 6.283185307179586476925286766559, inv_two_pi = 0.15915494309189533576888376337251;
    for (int w0 = lane; w0 < pairs; w0 += 32) {
        // this lane's elements i = 2 w0 and 2 w0 + 1 of the first half and their partners in the second
        const double th0 = exp2(-(double)(4 * w0) / (double)D * log2_base), th1 = exp2(-(double)(4 * w0 + 2) / (double)D * log2_base);
        // a warp per token: the angles do not depend on the head, so sine and cosine are taken once for all H rows
        for (int t = blockIdx.x * ROPE_WARPS + warp; t < T; t += gridDim.x * ROPE_WARPS) {
            const double p = (double)(__ldg(pos + t) - delta);
            double a0 = p * th0, a1 = p * th1;
            a0 -= two_pi * rint(a0 * inv_two_pi);
            a1 -= two_pi * rint(a1 * inv_two_pi);
            float s0, c0, s1, c1;
            sincosf((float)a0, &s0, &c0);
            sincosf((float)a1, &s1, &c1);
            for (int h0 = 0; h0 < H; h0 += 8) {
                uint32_t lo[8], hi[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const size_t base_w = ((size_t)t * H + h0 + j) * (D >> 1);
                    if (h0 + j < H) { lo[j] = __ldg(k_pre + base_w + w0); hi[j] = __ldg(k_pre + base_w + pairs + w0); }
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (h0 + j >= H) break;
                    const size_t base_w = ((size_t)t * H + h0 + j) * (D >> 1);
                    const float x0 = __uint_as_float(lo[j] << 16), x1 = __uint_as_float(lo[j] & 0xFFFF0000u);
                    const float y0 = __uint_as_float(hi[j] << 16), y1 = __uint_as_float(hi[j] & 0xFFFF0000u);
                    const __nv_bfloat162 olo = __floats2bfloat162_rn(x0 * c0 - y0 * s0, x1 * c1 - y1 * s1);
                    const __nv_bfloat162 ohi = __floats2bfloat162_rn(y0 * c0 + x0 * s0, y1 * c1 + x1 * s1);
                    k_rot[base_w + w0] = *reinterpret_cast<const uint32_t*>(&olo);
                    k_rot[base_w + pairs + w0] = *reinterpret_cast<const uint32_t*>(&ohi);
                }
            }
        }
    }
}

__global__ void __launch_bounds__(256)
streaming_mask_kernel(int V, int F, int n, uint8_t* __restrict__ mask) {
    const long long kv = (long long)V * F * n, total = (long long)V * n * kv;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long long)gridDim.x * blockDim.x) {
        const long long q = idx / kv, j = idx - q * kv;
        const long long v = q / n, i = q - v * n;
        const long long p = (v * F + F - 1) * n + i;
        mask[idx] = j <= p ? 1 : 0;
    }
}

}  // namespace

cudaError_t launch_rope_shifted_keys(const void* k_pre, const int32_t* pos, int delta, int T, int H, int D, double base,
                                     void* k_rot, cudaStream_t stream) {
    int grid = (T + ROPE_WARPS - 1) / ROPE_WARPS;
    const int cap = device_sm_count() * 8;
    if (grid > cap) grid = cap;
    rope_shifted_keys_kernel<<<grid, ROPE_WARPS * 32, 0, stream>>>(static_cast<const uint32_t*>(k_pre), pos, delta, T, H, D,
                                                                   log2(base), static_cast<uint32_t*>(k_rot));
    return cudaGetLastError();
}

cudaError_t launch_streaming_mask(int V, int F, int n, uint8_t* mask, cudaStream_t stream) {
    const long long total = (long long)V * n * V * F * n;
    long long grid = (total + 255) / 256;
    const long long cap = (long long)device_sm_count() * 8;
    if (grid > cap) grid = cap;
    streaming_mask_kernel<<<(unsigned)grid, 256, 0, stream>>>(V, F, n, mask);
    return cudaGetLastError();
}

}  // namespace w4a8
