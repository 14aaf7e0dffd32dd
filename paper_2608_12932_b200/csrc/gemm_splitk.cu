// Small-M W4A8 GEMM: a weight-streaming split-K kernel for decode / speculative-verify sized
// token counts (Sec. 3.2: one draft block is 8 tokens; Sec. 4: decode is bound by the bytes
// of weights the GPU must load).  HBM-bound by design:
//
//  * grid = (128-channel tiles) x (S slices of consecutive groups); a CTA owns at most
//    SPLITK_MAX_GROUPS blobs and requests ALL of them with 1-D bulk async copies (TMA) the
//    moment it starts, one mbarrier per blob, so every SM has its whole share of the weight
//    stream in flight at once and nothing is ever re-fetched.
//  * compute is mma.sync m16n8k32 (u8 x s8 -> s32) with the weights as the 16-row operand and
//    8 tokens as the 8 columns; the nibble interleave of the packed layout makes a lane's
//    16-byte chunk unpack (one AND, one shift+AND per word) straight into fragment registers.
//    k is visited in a permuted order inside each group, identically for both operands.
//  * zero points: D = P - z * sum_k(q_a) with the group sums from the quantise kernel;
//    group scales in fp32, slices written to the workspace, and the last CTA to arrive
//    at a tile sums the slices in slice order (deterministic), applies the token scale and
//    stores bf16.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include "ptx_sm100.cuh"
#include "w4a8_internal.cuh"

namespace w4a8 {

// the self-test entry point asks for the instantiation that withholds a copy by passing this address as the
// debug pointer (never dereferenced)
int32_t* withhold_marker() {
    static int32_t marker;
    return &marker;
}

namespace {
constexpr int SK_THREADS = 256;
constexpr int SK_BAR_BYTES = 128;
constexpr int SK_ACT_PAD = 16;     // bytes added to each activation row: kills the 2-way bank conflict

__host__ __device__ inline int sk_act_stride(int ng) { return ng * GROUP + SK_ACT_PAD; }
__host__ __device__ inline size_t sk_smem_bytes(int mb, int ng) {
    return SK_BAR_BYTES + (size_t)ng * BLOB_BYTES + (size_t)8 * mb * sk_act_stride(ng) + (size_t)8 * mb * ng * 4;
}

__device__ __forceinline__ void mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// WITHHOLD: a self-test instantiation.  Every CTA leaves the copy of its last blob out and waits for at most
// 200 microseconds: the wait for that blob expires, the CTA takes the give-up path below (status word, bounded wait
// for the copies in flight) and the kernel returns normally; its output is invalid.
constexpr uint64_t SK_TEST_LIMIT_NS = 200000ull;
template <int MB, bool WITHHOLD = false>
__global__ void __launch_bounds__(SK_THREADS)
gemm_splitk_kernel(const int8_t* __restrict__ qa, const uint16_t* __restrict__ sa,
                   const int32_t* __restrict__ asum, const uint8_t* __restrict__ packed,
                   __nv_bfloat16* __restrict__ y, int M, int N, int K, int S, int ng_max,
                   float* __restrict__ slices, uint32_t* __restrict__ counters,
                   uint32_t* __restrict__ status, int32_t* __restrict__ debug_partials) {
    extern __shared__ __align__(128) uint8_t smem[];
    const int G = K / GROUP;
    const int ntile = blockIdx.x / S, slice = blockIdx.x % S;
    const int g0 = (int)(((long long)slice * G) / S), g1 = (int)(((long long)(slice + 1) * G) / S);
    const int ng = g1 - g0;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    uint64_t* bars = reinterpret_cast<uint64_t*>(smem);
    uint8_t* blobs = smem + SK_BAR_BYTES;
    const int act_stride = sk_act_stride(ng_max);
    uint8_t* act = blobs + (size_t)ng_max * BLOB_BYTES;
    int32_t* asum_s = reinterpret_cast<int32_t*>(act + (size_t)8 * MB * act_stride);
    __shared__ uint32_t abort_flag, is_last;

    if (tid == 0) {
        abort_flag = 0;
        for (int i = 0; i < ng; ++i) ptx::mbar_init(ptx::smem_u32(bars + i), 1);
        ptx::fence_mbar_init();
        const uint8_t* src = packed + ((size_t)ntile * G + g0) * BLOB_BYTES;
        for (int i = 0; i < ng; ++i) {
            uint32_t bar = ptx::smem_u32(bars + i);
            ptx::mbar_arrive_expect_tx(bar, BLOB_BYTES);
            if (WITHHOLD && i == ng - 1) continue;          // announced, never sent: its barrier cannot complete
            ptx::bulk_g2s(ptx::smem_u32(blobs + (size_t)i * BLOB_BYTES), src + (size_t)i * BLOB_BYTES, BLOB_BYTES, bar);
        }
    }
    // activation slice [8*MB rows][ng*128 bytes] (rows >= M zero) and its group sums
    {
        const int row_chunks = ng * (GROUP / 16);
        for (int i = tid; i < 8 * MB * row_chunks; i += SK_THREADS) {
            int m = i / row_chunks, c = i % row_chunks;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (m < M) v = __ldg(reinterpret_cast<const uint4*>(qa + (size_t)m * K + (size_t)g0 * GROUP) + c);
            *reinterpret_cast<uint4*>(act + (size_t)m * act_stride + c * 16) = v;
        }
        for (int i = tid; i < 8 * MB * ng; i += SK_THREADS) {
            int m = i / ng, gi = i % ng;
            asum_s[m * ng_max + gi] = (m < M) ? __ldg(asum + (size_t)m * G + g0 + gi) : 0;
        }
    }
    __syncthreads();

    const int r = lane >> 2, j = lane & 3;
    const int row_lo = warp * 16 + r, row_hi = row_lo + 8;
    float facc[MB][4];
#pragma unroll
    for (int mb = 0; mb < MB; ++mb) facc[mb][0] = facc[mb][1] = facc[mb][2] = facc[mb][3] = 0.0f;

    bool ok = true;
    for (int gi = 0; gi < ng && ok; ++gi) {
        ok = ptx::mbar_wait_limit(ptx::smem_u32(bars + gi), 0, &abort_flag, WITHHOLD ? SK_TEST_LIMIT_NS : ptx::WAIT_LIMIT_NS);
        if (!ok) break;
        const uint8_t* blob = blobs + (size_t)gi * BLOB_BYTES;
        // chunk j of the two rows (rows r and r + 8 share their swizzle)
        const uint4 wa = *reinterpret_cast<const uint4*>(blob + row_lo * 64 + blob_chunk_pos(row_lo, j) * 16);
        const uint4 wb = *reinterpret_cast<const uint4*>(blob + row_hi * 64 + blob_chunk_pos(row_lo, j) * 16);
        const uint32_t wlo[4] = {wa.x, wa.y, wa.z, wa.w}, whi[4] = {wb.x, wb.y, wb.z, wb.w};
        uint32_t a[4][4];
#pragma unroll
        for (int s = 0; s < 4; ++s) {
            a[s][0] = wlo[s] & 0x0F0F0F0Fu;            // row_lo, k = 32j + blob_word_k(s) + 0..3
            a[s][1] = whi[s] & 0x0F0F0F0Fu;            // row_hi, same k
            a[s][2] = (wlo[s] >> 4) & 0x0F0F0F0Fu;     // row_lo, eight k further on
            a[s][3] = (whi[s] >> 4) & 0x0F0F0F0Fu;     // row_hi
        }
        const float s_lo = __half2float(__ushort_as_half(reinterpret_cast<const uint16_t*>(blob + BLOB_SCALE_OFF)[row_lo]));
        const float s_hi = __half2float(__ushort_as_half(reinterpret_cast<const uint16_t*>(blob + BLOB_SCALE_OFF)[row_hi]));
        const int z_lo = (blob[BLOB_ZERO_OFF + (row_lo >> 1)] >> ((row_lo & 1) * 4)) & 0xF;
        const int z_hi = (blob[BLOB_ZERO_OFF + (row_hi >> 1)] >> ((row_hi & 1) * 4)) & 0xF;
#pragma unroll
        for (int mb = 0; mb < MB; ++mb) {
            const uint8_t* arow = act + (size_t)(8 * mb + r) * act_stride + gi * GROUP + 32 * j;
            const uint4 b0 = *reinterpret_cast<const uint4*>(arow);
            const uint4 b1 = *reinterpret_cast<const uint4*>(arow + 16);
            const uint32_t bq[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
            int c[4] = {0, 0, 0, 0};
#pragma unroll
            for (int s = 0; s < 4; ++s)
                mma_u8s8(c, a[s][0], a[s][1], a[s][2], a[s][3], bq[blob_word_k(s) / 4], bq[blob_word_k(s) / 4 + 2]);
            const int m0 = 8 * mb + 2 * j;
            const int A0 = asum_s[m0 * ng_max + gi], A1 = asum_s[(m0 + 1) * ng_max + gi];
            const int d0 = c[0] - z_lo * A0, d1 = c[1] - z_lo * A1;
            const int d2 = c[2] - z_hi * A0, d3 = c[3] - z_hi * A1;
            facc[mb][0] = fmaf(s_lo, (float)d0, facc[mb][0]);
            facc[mb][1] = fmaf(s_lo, (float)d1, facc[mb][1]);
            facc[mb][2] = fmaf(s_hi, (float)d2, facc[mb][2]);
            facc[mb][3] = fmaf(s_hi, (float)d3, facc[mb][3]);
            if (debug_partials) {
                const size_t n_lo = (size_t)ntile * TILE_N + row_lo, n_hi = n_lo + 8;
                const int g = g0 + gi;
                if (m0 < M) {
                    debug_partials[((size_t)m0 * G + g) * N + n_lo] = d0;
                    debug_partials[((size_t)m0 * G + g) * N + n_hi] = d2;
                }
                if (m0 + 1 < M) {
                    debug_partials[((size_t)(m0 + 1) * G + g) * N + n_lo] = d1;
                    debug_partials[((size_t)(m0 + 1) * G + g) * N + n_hi] = d3;
                }
            }
        }
    }
    if (!ok && lane == 0) atomicExch(status, (uint32_t)W4A8_ERR_TIMEOUT);
    if (!ok) {
        // every blob this CTA requested must land before its shared memory is released:
        // bounded wait for the copies still in flight
        const uint64_t t0 = ptx::globaltimer_ns();
        for (int gi = 0; gi < ng; ++gi) {
            uint32_t bar = ptx::smem_u32(bars + gi);
            while (!ptx::mbar_test_wait(bar, 0) && ptx::globaltimer_ns() - t0 < (WITHHOLD ? SK_TEST_LIMIT_NS : 100000000ull)) __nanosleep(200);
        }
    }

    const size_t n_lo = (size_t)ntile * TILE_N + row_lo, n_hi = n_lo + 8;
    if (S == 1) {
#pragma unroll
        for (int mb = 0; mb < MB; ++mb) {
            const int m0 = 8 * mb + 2 * j;
            if (m0 < M) {
                const float t = __half2float(__ushort_as_half(__ldg(sa + m0)));
                y[(size_t)m0 * N + n_lo] = __float2bfloat16_rn(facc[mb][0] * t);
                y[(size_t)m0 * N + n_hi] = __float2bfloat16_rn(facc[mb][2] * t);
            }
            if (m0 + 1 < M) {
                const float t = __half2float(__ushort_as_half(__ldg(sa + m0 + 1)));
                y[(size_t)(m0 + 1) * N + n_lo] = __float2bfloat16_rn(facc[mb][1] * t);
                y[(size_t)(m0 + 1) * N + n_hi] = __float2bfloat16_rn(facc[mb][3] * t);
            }
        }
        return;
    }

    float* mine = slices + (size_t)slice * M * N;
#pragma unroll
    for (int mb = 0; mb < MB; ++mb) {
        const int m0 = 8 * mb + 2 * j;
        if (m0 < M) {
            __stcg(mine + (size_t)m0 * N + n_lo, facc[mb][0]);
            __stcg(mine + (size_t)m0 * N + n_hi, facc[mb][2]);
        }
        if (m0 + 1 < M) {
            __stcg(mine + (size_t)(m0 + 1) * N + n_lo, facc[mb][1]);
            __stcg(mine + (size_t)(m0 + 1) * N + n_hi, facc[mb][3]);
        }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        uint32_t prev = atomicAdd(counters + ntile, 1u);
        is_last = (prev == (uint32_t)(S - 1));
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    for (int i = tid; i < M * TILE_N; i += SK_THREADS) {
        const int m = i / TILE_N, nn = i % TILE_N;
        const size_t off = (size_t)m * N + (size_t)ntile * TILE_N + nn;
        float acc = 0.0f;
        for (int s = 0; s < S; ++s) acc += __ldcg(slices + (size_t)s * M * N + off);
        const float t = __half2float(__ushort_as_half(__ldg(sa + m)));
        y[off] = __float2bfloat16_rn(acc * t);
    }
    if (tid == 0) counters[ntile] = 0;     // leave the header zero for the next call
}

template <int MB>
cudaError_t launch_mb(const int8_t* qa, const uint16_t* sa, const int32_t* asum, const void* packed, void* y,
                      int M, int N, int K, int S, void* workspace, float* slices, int32_t* debug_partials, cudaStream_t stream) {
    const int G = K / GROUP;
    const int ng_max = (G + S - 1) / S;
    const size_t smem = sk_smem_bytes(MB, ng_max);
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    static bool attr_set[64] = {false};      // function attributes are per device; one array per template instance
    if (!attr_set[dev]) {
        e = cudaFuncSetAttribute(gemm_splitk_kernel<MB>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    if (debug_partials == withhold_marker()) {
        static bool attr_set_t[64] = {false};
        if (!attr_set_t[dev]) {
            e = cudaFuncSetAttribute(gemm_splitk_kernel<MB, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
            if (e != cudaSuccess) return e;
            attr_set_t[dev] = true;
        }
        gemm_splitk_kernel<MB, true><<<(N / TILE_N) * S, SK_THREADS, smem, stream>>>(
            qa, sa, asum, static_cast<const uint8_t*>(packed), static_cast<__nv_bfloat16*>(y), M, N, K, S, ng_max,
            slices, reinterpret_cast<uint32_t*>(ws + WS_COUNTER_OFF), reinterpret_cast<uint32_t*>(ws + WS_STATUS_OFF), nullptr);
        return cudaGetLastError();
    }
    gemm_splitk_kernel<MB><<<(N / TILE_N) * S, SK_THREADS, smem, stream>>>(
        qa, sa, asum, static_cast<const uint8_t*>(packed), static_cast<__nv_bfloat16*>(y), M, N, K, S, ng_max,
        slices, reinterpret_cast<uint32_t*>(ws + WS_COUNTER_OFF),
        reinterpret_cast<uint32_t*>(ws + WS_STATUS_OFF), debug_partials);
    return cudaGetLastError();
}
}  // namespace

// Number of K slices: enough CTAs for about two per SM, never more than SPLITK_MAX_GROUPS
// groups per CTA, never more slices than groups.  Depends on the shape only (not on M), so
// that the workspace size does not depend on M either.
int splitk_num_slices(int /*M*/, int N, int K) {
    const int G = K / GROUP, tiles = N / TILE_N;
    const int s_min = (G + SPLITK_MAX_GROUPS - 1) / SPLITK_MAX_GROUPS;
    int s = (2 * 148 + tiles / 2) / tiles;
    if (s < s_min) s = s_min;
    if (s > G) s = G;
    if (s < 1) s = 1;
    return s;
}

cudaError_t launch_gemm_splitk(const int8_t* qa, const uint16_t* sa, const int32_t* asum, const void* packed,
                               void* y, int M, int N, int K, void* workspace, float* slices, int32_t* debug_partials,
                               cudaStream_t stream) {
    const int S = splitk_num_slices(M, N, K);
    if (M <= 8) return launch_mb<1>(qa, sa, asum, packed, y, M, N, K, S, workspace, slices, debug_partials, stream);
    if (M <= 16) return launch_mb<2>(qa, sa, asum, packed, y, M, N, K, S, workspace, slices, debug_partials, stream);
    if (M <= 32) return launch_mb<4>(qa, sa, asum, packed, y, M, N, K, S, workspace, slices, debug_partials, stream);
    return launch_mb<8>(qa, sa, asum, packed, y, M, N, K, S, workspace, slices, debug_partials, stream);
}

}  // namespace w4a8

// ---------------------------------------------------------------------------------------------
// Allocation-free variant of the split-K GEMM (declared in w4a8.h as w4a8_gemm_static_scratch).
// The split-K slices, arrival counters and status word live in a fixed array that is part of the
// library image on every GPU that loads it, instead of a caller-provided workspace.
namespace w4a8 {
namespace {
static __device__ __align__(256) unsigned char g_static_scratch[W4A8_STATIC_SCRATCH_BYTES];

// Device address of g_static_scratch on the current device (0 on failure).  In host code the
// array's name is only a handle for the runtime, not an address a kernel could use, so the
// address is looked up once per device with that device current, and cached.
void* static_scratch_ptr(int dev, cudaError_t* err) {
    static void* cached[64] = {nullptr};
    if (!cached[dev]) {
        void* p = nullptr;
        *err = cudaGetSymbolAddress(&p, g_static_scratch);
        if (*err != cudaSuccess) return nullptr;
        cached[dev] = p;
    }
    *err = cudaSuccess;
    return cached[dev];
}
}  // namespace

void* static_scratch_address() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    cudaError_t e = cudaSuccess;
    return static_scratch_ptr(dev, &e);
}
}  // namespace w4a8

extern "C" w4a8_status w4a8_gemm_static_scratch(const int8_t* qa, const uint16_t* sa, const int32_t* asum,
                                                const void* packed_w, void* y_bf16,
                                                int M, int N, int K, int group, void* stream) {
    using namespace w4a8;
    if (group != GROUP || N <= 0 || K <= 0 || N % TILE_N != 0 || K % GROUP != 0 || N / TILE_N > MAX_N_TILES || M < 0)
        return W4A8_ERR_SHAPE;
    if (M > SPLITK_MAX_M) return W4A8_ERR_SHAPE;
    if (M == 0) return W4A8_OK;
    if (!qa || !sa || !asum || !packed_w || !y_bf16) return W4A8_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(qa) & 15) || (reinterpret_cast<uintptr_t>(sa) & 1) ||
        (reinterpret_cast<uintptr_t>(asum) & 3) || (reinterpret_cast<uintptr_t>(packed_w) & 127) ||
        (reinterpret_cast<uintptr_t>(y_bf16) & 1))
        return W4A8_ERR_ALIGN;
    const int S = splitk_num_slices(M, N, K);
    const size_t need = (size_t)WS_HEADER_BYTES + (S > 1 ? (size_t)S * M * N * sizeof(float) : 0);
    if (need > (size_t)W4A8_STATIC_SCRATCH_BYTES) return W4A8_ERR_WORKSPACE;   // beyond the fixed scratch
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return W4A8_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return W4A8_ERR_CUDA;
    if (major != 10) return W4A8_ERR_ARCH;
    cudaError_t e = cudaSuccess;
    void* scratch = static_scratch_ptr(dev, &e);
    if (!scratch) return W4A8_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array keeps whatever the previous call left: the arrival counters must be zero when the
    // kernel starts.  The status word ahead of them is left alone, so that a wait that timed out in an
    // earlier call stays readable (w4a8_check_status with a NULL workspace) until it is read.
    if (cudaMemsetAsync(static_cast<uint8_t*>(scratch) + WS_COUNTER_OFF, 0, WS_HEADER_BYTES - WS_COUNTER_OFF, st) != cudaSuccess)
        return W4A8_ERR_CUDA;
    e = launch_gemm_splitk(qa, sa, asum, packed_w, y_bf16, M, N, K, scratch,
                           reinterpret_cast<float*>(static_cast<uint8_t*>(scratch) + WS_HEADER_BYTES), nullptr, st);
    return e == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
}
