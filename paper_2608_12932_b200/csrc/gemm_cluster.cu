// Small-M W4A8 GEMM, cluster variant: the K slices of one 128-channel tile form a thread-block
// cluster and are reduced through distributed shared memory, so the kernel needs no global
// scratch, no atomics and no memory fence.  (Sec. 3.2: a draft block is 8 tokens; Sec. 4: decode is
// bound by the weight bytes the GPU must load - this kernel streams them once at HBM width.)
//
//  * grid = tiles x S, cluster = the S slices of a tile (S <= 8).  A CTA walks its consecutive
//    groups through a ring of R stages; one stage = one packed blob (1-D bulk copy, 8512 B) plus
//    the matching 128-byte-wide activation tile (2-D TMA, 128-byte swizzle, rows >= M read as 0).
//  * a producer warp issues the copies; the weight copies of the first R stages are issued before
//    griddepcontrol.wait, so under programmatic dependent launch the weight stream of this
//    kernel overlaps the tail of the previous kernel in the stream.
//  * sixteen consumer warps in two sets of eight or four sets of four (set s takes groups s,
//    s + sets, ... of the slice; a set's warp owns one or two blocks of 16 of the 128 rows):
//    mma.sync m16n8k32 (u8 x s8 -> s32), weights as the 16-row operand; D = P - z * sum(q_a) with
//    the group sums from the quantise kernel; fp32 group scales; the sets' partial sums are added
//    through shared memory (fixed order).
//  * reduction: the tile's M x 128 outputs are split into S contiguous shares, one per CTA of the
//    cluster.  A CTA lays its fp32 partials out as [token][channel] in its own shared memory and
//    pushes them in 16-byte pieces into the owners' shared memory (slot = pusher's rank) with
//    st.shared::cluster (one store instruction of a warp then goes to one owner), then one cluster
//    barrier (release/acquire); the owner sums its S slots in rank order (fixed order:
//    deterministic), applies the token scale and stores bf16.  After the barrier a CTA reads only
//    its own shared memory, so it may exit freely.
//  * sizing: the number of slices minimises ceil(CTAs / SMs) * ceil(G / S); a launch that fits in
//    one wave keeps its CTAs under half an SM's shared memory and prefetches as much of its slice
//    as fits, so that two consecutive launches can be resident together and the weight stream of
//    the next overlaps the tail of the current one.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include "ptx_sm100.cuh"
#include "w4a8_internal.cuh"

namespace w4a8 {
namespace {

constexpr int CL_ROW_WARPS = 8;                           // 16 weight rows each: one 128-row blob
constexpr int CL_CONSUMER_WARPS = 2 * CL_ROW_WARPS;        // split into warp sets that take groups in turn
constexpr int CL_THREADS = (CL_CONSUMER_WARPS + 1) * 32;   // + one producer warp
constexpr int CL_MAX_STAGES = 12;
constexpr int CL_PART_STRIDE = TILE_N + 4;                 // floats per token row of a partial-sum buffer: the pad spreads the four
                                                           // token pairs of a warp's store over all banks (a 128-float row puts them in one)
constexpr int CL_BLOB_STRIDE = 8704;                       // BLOB_BYTES rounded up to a multiple of 128
constexpr int CL_MAX_S = 8;

struct ClLayout {
    int act_off, blob_off, bar_off, asum_off, red_off, set_off, misc_off, total;
};
// warp sets of a kernel whose warps own rb blocks of 16 rows each, and the buffers of partial sums
__host__ __device__ constexpr int cl_sets(int rb) { return 2 * rb; }
__host__ __device__ constexpr int cl_parts(int mb, int rb) { return (mb <= 2 && mb * cl_sets(rb) <= 8) ? cl_sets(rb) : 1; }
__host__ __device__ inline ClLayout cl_layout(int mb, int rb, int stages, int ng_max) {
    ClLayout L;
    L.act_off = 0;                                            // stages x (8*mb rows x 128 B), 1024-aligned
    L.blob_off = L.act_off + stages * 1024 * mb;
    L.bar_off = L.blob_off + stages * CL_BLOB_STRIDE;
    L.asum_off = L.bar_off + 2 * CL_MAX_STAGES * 8;
    L.red_off = (L.asum_off + 8 * mb * ng_max * 4 + 15) & ~15;
    L.set_off = L.red_off + (8 * mb * (TILE_N / 4) + CL_MAX_S) * 16;   // S slots x ceil(M*32/S) float4
    L.misc_off = L.set_off + cl_parts(mb, rb) * 8 * mb * CL_PART_STRIDE * 4;   // partial sums, [token][channel] fp32
    L.total = L.misc_off + 16;
    return L;
}

__device__ __forceinline__ void mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// MINB = 2 caps the registers so that two CTAs fit on an SM: wanted when a launch has more CTAs than
// SMs anyway (they then share SMs instead of queueing); with fewer CTAs than SMs it only invites the
// cluster scheduler to pack two of them onto one SM and leave others idle.
template <int MB, int MINB, int RB>
__global__ void __launch_bounds__(CL_THREADS, MINB)
gemm_cluster_kernel(const __grid_constant__ CUtensorMap tmap_qa, const uint16_t* __restrict__ sa,
                    const int32_t* __restrict__ asum, const uint8_t* __restrict__ packed,
                    __nv_bfloat16* y, const __nv_bfloat16* residual, int M, int N, int K, int S, int ng_max, int stages,
                    uint32_t* __restrict__ status, int32_t* __restrict__ debug_partials) {
    ptx::pdl_launch_dependents();
    ptx::cluster_arrive_relaxed();     // "this CTA runs": peers wait for it before they write into it
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    const ClLayout L = cl_layout(MB, RB, stages, ng_max);
    constexpr int MP = 8 * MB;
    constexpr uint32_t ACT_BYTES = MP * GROUP;
    constexpr int NSETS = cl_sets(RB);                    // warp sets: set s takes groups s, s + NSETS, ...
    constexpr int WPS = CL_CONSUMER_WARPS / NSETS;        // warps per set, RB blocks of 16 rows each
    constexpr int NPARTS = cl_parts(MB, RB);              // buffers of partial sums: one per set, or one
    static_assert(NPARTS == NSETS || RB == 1, "in-place merge is written for two sets");

    const int G = K / GROUP;
    const int ntile = blockIdx.x / S;
    const int slice = (int)ptx::cluster_ctarank();             // == blockIdx.x % S
    const int g0 = (int)(((long long)slice * G) / S), g1 = (int)(((long long)(slice + 1) * G) / S);
    const int ng = g1 - g0;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    auto full_bar = [&](int s) { return smem_base + L.bar_off + 8 * s; };
    auto empty_bar = [&](int s) { return smem_base + L.bar_off + 8 * (CL_MAX_STAGES + s); };
    int32_t* asum_s = reinterpret_cast<int32_t*>(smem + L.asum_off);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + L.misc_off);
    const uint8_t* src = packed + ((size_t)ntile * G + g0) * BLOB_BYTES;

    if (warp == CL_CONSUMER_WARPS && lane == 0) {
        *abort_flag = 0;
        for (int s = 0; s < stages; ++s) {
            ptx::mbar_init(full_bar(s), 1);
            ptx::mbar_init(empty_bar(s), WPS);                       // the one set that consumed the stage
        }
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tmap_qa);
        // weights do not depend on the previous kernel: start their stream at once
        const int first = ng < stages ? ng : stages;
        for (int gi = 0; gi < first; ++gi) {
            ptx::mbar_expect_tx(full_bar(gi), BLOB_BYTES);
            ptx::bulk_g2s(smem_base + L.blob_off + gi * CL_BLOB_STRIDE, src + (size_t)gi * BLOB_BYTES, BLOB_BYTES,
                          full_bar(gi));
        }
    }
    __syncthreads();
    // Activations, their scales and group sums come from the previous kernel.  They are read
    // only after this wait and only through L2 (TMA, ld.global.cg): an L1 line filled by an
    // older grid that shared this SM could otherwise be stale.
    ptx::pdl_wait();

    float facc[RB][MB][4];
#pragma unroll
    for (int b = 0; b < RB; ++b)
#pragma unroll
        for (int mb = 0; mb < MB; ++mb) facc[b][mb][0] = facc[b][mb][1] = facc[b][mb][2] = facc[b][mb][3] = 0.0f;
    const int r = lane >> 2, j = lane & 3;
    const int set = (warp / WPS) % NSETS;
    const int row0 = (warp % WPS) * (16 * RB) + r;        // block b of this warp: rows row0 + 16b and + 8
    const int jx = blob_chunk_pos(r, j) * 16;             // chunk j of those rows (they all share the swizzle of r)

    if (warp == CL_CONSUMER_WARPS) {
        // ------------------------------------------------------------------ producer ----
        if (lane == 0) {
            bool ok = true;
            int s = 0;
            uint32_t phase = 1;                 // parity of the previous use's "empty" phase
            for (int gi = 0; gi < ng && ok; ++gi, ++s) {
                if (s == stages) { s = 0; phase ^= 1; }
                if (gi >= stages) {
                    ok = ptx::mbar_wait(empty_bar(s), phase, abort_flag);
                    if (!ok) break;
                    ptx::mbar_arrive_expect_tx(full_bar(s), BLOB_BYTES + ACT_BYTES);
                    ptx::bulk_g2s(smem_base + L.blob_off + s * CL_BLOB_STRIDE, src + (size_t)gi * BLOB_BYTES,
                                  BLOB_BYTES, full_bar(s));
                } else {
                    ptx::mbar_arrive_expect_tx(full_bar(s), ACT_BYTES);    // blob bytes were announced above
                }
                ptx::tma_load_2d(smem_base + L.act_off + s * 1024 * MB, &tmap_qa, (g0 + gi) * GROUP, 0, full_bar(s));
            }
        }
    } else {
        // ----------------------------------------------------------------- consumers ----
        for (int i = tid; i < MP * ng; i += CL_CONSUMER_WARPS * 32) {
            const int m = i / ng, gi = i % ng;
            asum_s[gi * MP + m] = (m < M) ? __ldcg(asum + (size_t)m * G + g0 + gi) : 0;      // group-major: see the loads
        }
        ptx::named_bar_sync(1, CL_CONSUMER_WARPS * 32);
        bool ok = true;
        int s = set;
        uint32_t phase = 0;
        for (int gi = set; gi < ng; gi += NSETS, s += NSETS) {
            while (s >= stages) { s -= stages; phase ^= 1; }
            ok = ptx::mbar_wait(full_bar(s), phase, abort_flag);
            if (!ok) break;
            const uint8_t* blob = smem + L.blob_off + s * CL_BLOB_STRIDE;
            const uint8_t* act = smem + L.act_off + s * 1024 * MB;
#pragma unroll
            for (int b = 0; b < RB; ++b) {
                const int row_lo = row0 + 16 * b, row_hi = row_lo + 8;
                const uint4 wa = *reinterpret_cast<const uint4*>(blob + row_lo * 64 + jx);
                const uint4 wb = *reinterpret_cast<const uint4*>(blob + row_hi * 64 + jx);
                const uint32_t wlo[4] = {wa.x, wa.y, wa.z, wa.w}, whi[4] = {wb.x, wb.y, wb.z, wb.w};
                uint32_t a[4][4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    a[q][0] = wlo[q] & 0x0F0F0F0Fu;            // row_lo, k = 32j + blob_word_k(q) + 0..3
                    a[q][1] = whi[q] & 0x0F0F0F0Fu;            // row_hi, same k
                    a[q][2] = (wlo[q] >> 4) & 0x0F0F0F0Fu;     // row_lo, eight k further on
                    a[q][3] = (whi[q] >> 4) & 0x0F0F0F0Fu;     // row_hi
                }
                const uint16_t* sc = reinterpret_cast<const uint16_t*>(blob + BLOB_SCALE_OFF);
                const float s_lo = __half2float(__ushort_as_half(sc[row_lo]));
                const float s_hi = __half2float(__ushort_as_half(sc[row_hi]));
                const int z_lo = (blob[BLOB_ZERO_OFF + (row_lo >> 1)] >> ((row_lo & 1) * 4)) & 0xF;
                const int z_hi = (blob[BLOB_ZERO_OFF + (row_hi >> 1)] >> ((row_hi & 1) * 4)) & 0xF;
#pragma unroll
                for (int mb = 0; mb < MB; ++mb) {
                    // token row 8*mb + r of the stage: 128 B, 16-byte chunks XOR-swizzled by the row index
                    const uint8_t* arow = act + mb * 1024 + r * 128;
                    const uint4 b0 = *reinterpret_cast<const uint4*>(arow + (((2 * j) ^ r) << 4));
                    const uint4 b1 = *reinterpret_cast<const uint4*>(arow + (((2 * j + 1) ^ r) << 4));
                    const uint32_t bq[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
                    const int m0 = 8 * mb + 2 * j;
                    // the two tokens' group sums: one 8-byte load, the four j of a quarter-warp side by side (token-major
                    // rows of 16 or 32 words put them all into one bank)
                    const int2 A01 = *reinterpret_cast<const int2*>(asum_s + gi * MP + m0);
                    const int A0 = A01.x, A1 = A01.y;
                    int d0, d1, d2, d3;       // D = P - z * sum(q_a)
                    if (MB == 2) {
                        // two token blocks give two independent chains: the four MMAs of a block add
                        // onto one accumulator that starts at the zero-point term (fewer instructions)
                        int c[4] = {-z_lo * A0, -z_lo * A1, -z_hi * A0, -z_hi * A1};
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            mma_u8s8(c, a[q][0], a[q][1], a[q][2], a[q][3], bq[blob_word_k(q) / 4], bq[blob_word_k(q) / 4 + 2]);
                        d0 = c[0]; d1 = c[1]; d2 = c[2]; d3 = c[3];
                    } else {
                        // four independent MMAs (one per k-step) instead of a dependent chain of four
                        int cq[4][4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            cq[q][0] = cq[q][1] = cq[q][2] = cq[q][3] = 0;
                            mma_u8s8(cq[q], a[q][0], a[q][1], a[q][2], a[q][3], bq[blob_word_k(q) / 4], bq[blob_word_k(q) / 4 + 2]);
                        }
                        int c[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) c[e] = (cq[0][e] + cq[1][e]) + (cq[2][e] + cq[3][e]);
                        d0 = c[0] - z_lo * A0; d1 = c[1] - z_lo * A1;
                        d2 = c[2] - z_hi * A0; d3 = c[3] - z_hi * A1;
                    }
                    facc[b][mb][0] = fmaf(s_lo, (float)d0, facc[b][mb][0]);
                    facc[b][mb][1] = fmaf(s_lo, (float)d1, facc[b][mb][1]);
                    facc[b][mb][2] = fmaf(s_hi, (float)d2, facc[b][mb][2]);
                    facc[b][mb][3] = fmaf(s_hi, (float)d3, facc[b][mb][3]);
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
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(empty_bar(s));
        }
        if (!ok) {
            // copies of stages not yet consumed may still be in flight: give them a bounded time to land
            for (int st = 0; st < stages; ++st)
                for (int spin = 0; spin < (1 << 16) && !ptx::mbar_try_wait(full_bar(st), 0); ++spin) {}
        }
        // The CTA's partial sums go to shared memory as [token][channel]: the exchange below moves
        // 16-byte pieces of that layout.  With few tokens each warp set has a buffer of its own and
        // the two are added (even + odd: fixed order) when a piece is read; otherwise the odd set
        // writes, the even set adds its own values in place.
        float* part = reinterpret_cast<float*>(smem + L.set_off);
        auto put = [&](float* buf) {
#pragma unroll
            for (int b = 0; b < RB; ++b) {
                const int row_lo = row0 + 16 * b, row_hi = row_lo + 8;
#pragma unroll
                for (int mb = 0; mb < MB; ++mb) {
                    float* p = buf + (8 * mb + 2 * j) * CL_PART_STRIDE;
                    p[row_lo] = facc[b][mb][0]; p[CL_PART_STRIDE + row_lo] = facc[b][mb][1];
                    p[row_hi] = facc[b][mb][2]; p[CL_PART_STRIDE + row_hi] = facc[b][mb][3];
                }
            }
        };
        if (NPARTS > 1) {
            put(part + set * (MP * CL_PART_STRIDE));
        } else {
            if (set == 1) put(part);
            ptx::named_bar_sync(1, CL_CONSUMER_WARPS * 32);
            if (set == 0) {
                const int row_lo = row0, row_hi = row_lo + 8;
#pragma unroll
                for (int mb = 0; mb < MB; ++mb) {
                    const float* p = part + (8 * mb + 2 * j) * CL_PART_STRIDE;
                    facc[0][mb][0] += p[row_lo]; facc[0][mb][1] += p[CL_PART_STRIDE + row_lo];
                    facc[0][mb][2] += p[row_hi]; facc[0][mb][3] += p[CL_PART_STRIDE + row_hi];
                }
                put(part);
            }
        }
    }
    if (*abort_flag && lane == 0) atomicExch(status, (uint32_t)W4A8_ERR_TIMEOUT);

    __syncwarp();
    ptx::cluster_wait();       // every CTA of the cluster has started: its shared memory may be written
    // The tile's M x 128 sums, as M*32 pieces of four channels, are split into S contiguous shares.
    const int T4 = M * (TILE_N / 4), chunk4 = (T4 + S - 1) / S;
    const int lo4 = slice * chunk4;
    const int cnt4 = (T4 - lo4) < chunk4 ? (T4 - lo4) : chunk4;       // may be <= 0 for the last ranks
    // the token scale of this thread's first output piece: loaded now, needed after the barrier
    float t_first = 0.0f;
    uint2 r_first = make_uint2(0u, 0u);
    if (tid < cnt4) {
        t_first = __half2float(__ushort_as_half(__ldcg(sa + ((lo4 + tid) >> 5))));
        if (residual)
            r_first = __ldcg(reinterpret_cast<const uint2*>(residual + (size_t)((lo4 + tid) >> 5) * N + (size_t)ntile * TILE_N + ((lo4 + tid) & 31) * 4));
    }
    __syncthreads();           // the CTA's partial sums are complete in shared memory
    const float4* part4 = reinterpret_cast<const float4*>(smem + L.set_off);
    auto piece = [&](int q) {
        const int q4 = q + (q >> 5);                       // piece q = token q / 32, channels 4 (q % 32)..; rows of 33 float4
        float4 v = part4[q4];
#pragma unroll
        for (int p = 1; p < NPARTS; ++p) {                 // set order: deterministic
            const float4 o = part4[q4 + p * MP * (CL_PART_STRIDE / 4)];
            v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
        }
        return v;
    };
    if (S > 1) {
        // push every piece to the CTA that owns it: slot `slice` of the owner's buffer
        const uint32_t red_addr = smem_base + L.red_off;
        for (int q = tid; q < T4; q += CL_THREADS) {
            const int owner = q / chunk4;
            const uint32_t off = (uint32_t)(slice * chunk4 + q - owner * chunk4) * 16u;
            ptx::st_dsmem_f32x4(ptx::map_to_cta(red_addr + off, (uint32_t)owner), piece(q));
        }
        __syncwarp();
        ptx::cluster_sync();   // arrive.release after the pushes, wait.acquire before the sums
    }
    {
        const float4* red4 = reinterpret_cast<const float4*>(smem + L.red_off);
        for (int i = tid; i < cnt4; i += CL_THREADS) {
            float4 acc;
            if (S == 1) {
                acc = piece(i);            // a single slice owns the whole K range: no exchange
            } else {
                acc = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                for (int s = 0; s < S; ++s) {                          // rank order: deterministic
                    const float4 v = red4[s * chunk4 + i];
                    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                }
            }
            const int m = (lo4 + i) >> 5, nn = ((lo4 + i) & 31) * 4;
            const float t = (i == tid) ? t_first : __half2float(__ushort_as_half(__ldcg(sa + m)));
            float r0 = 0.0f, r1 = 0.0f, r2 = 0.0f, r3 = 0.0f;
            if (residual) {
                // the projection's output joins the residual stream: added in fp32 before the one rounding (y may be
                // the residual buffer itself: this thread reads the four values it then overwrites)
                const uint2 rv = (i == tid) ? r_first : __ldcg(reinterpret_cast<const uint2*>(residual + (size_t)m * N + (size_t)ntile * TILE_N + nn));
                r0 = __uint_as_float(rv.x << 16); r1 = __uint_as_float(rv.x & 0xFFFF0000u);
                r2 = __uint_as_float(rv.y << 16); r3 = __uint_as_float(rv.y & 0xFFFF0000u);
            }
            float v0 = acc.x * t, v1 = acc.y * t, v2 = acc.z * t, v3 = acc.w * t;
            if (residual) { v0 += r0; v1 += r1; v2 += r2; v3 += r3; }
            __nv_bfloat162 o01 = __floats2bfloat162_rn(v0, v1);
            __nv_bfloat162 o23 = __floats2bfloat162_rn(v2, v3);
            uint2 o;
            o.x = *reinterpret_cast<uint32_t*>(&o01);
            o.y = *reinterpret_cast<uint32_t*>(&o23);
            *reinterpret_cast<uint2*>(y + (size_t)m * N + (size_t)ntile * TILE_N + nn) = o;
        }
    }
}

template <int MB, int MINB, int RB>
cudaError_t launch_mb(const int8_t* qa, const uint16_t* sa, const int32_t* asum, const void* packed, void* y, const void* residual,
                      int M, int N, int K, int S, void* workspace, int32_t* debug_partials, cudaStream_t stream) {
    const int G = K / GROUP;
    const int ng_max = (G + S - 1) / S;
    // shared-memory budget per CTA: a launch of at most one wave leaves room for the next launch's
    // CTAs on the same SMs; larger launches share the SM between ceil(CTAs/SMs) CTAs of their own
    const int ctas = (N / TILE_N) * S, sms = device_sm_count();
    const int waves = (ctas + sms - 1) / sms;
    int budget = waves <= 1 ? 110 * 1024 : (220 * 1024) / waves;
    if (budget < 40 * 1024) budget = 40 * 1024;
    const int fixed = cl_layout(MB, RB, 0, ng_max).total + 1024;
    int stages = (budget - fixed) / (CL_BLOB_STRIDE + 1024 * MB);
    if (stages > CL_MAX_STAGES) stages = CL_MAX_STAGES;
    if (stages >= ng_max) {
        stages = ng_max;                       // every stage is used once
    } else {
        // Stages are reused.  Consecutive groups go to different warp sets and a parity wait can
        // only tell consecutive uses of a barrier apart, so each stage must always serve the same
        // set: the ring length has to be a multiple of the number of sets.
        constexpr int NSETS = cl_sets(RB);
        stages -= stages % NSETS;
        if (stages < NSETS) stages = NSETS;
    }
    const ClLayout L = cl_layout(MB, RB, stages, ng_max);
    const size_t smem = (size_t)L.total + 1024;
    if (smem > 227 * 1024) return cudaErrorInvalidConfiguration;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    static bool attr_done[64] = {false};
    if (!attr_done[dev]) {
        e = cudaFuncSetAttribute(gemm_cluster_kernel<MB, MINB, RB>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return e;
        attr_done[dev] = true;
    }
    CUtensorMap tmap;
    e = make_qa_tensor_map(&tmap, qa, M, K, 8 * MB);
    if (e != cudaSuccess) return e;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((N / TILE_N) * S), 1, 1);
    cfg.blockDim = dim3(CL_THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attrs[3];
    attrs[0].id = cudaLaunchAttributeClusterDimension;
    attrs[0].val.clusterDim.x = (unsigned)S;
    attrs[0].val.clusterDim.y = 1;
    attrs[0].val.clusterDim.z = 1;
    attrs[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[1].val.programmaticStreamSerializationAllowed = 1;
    attrs[2].id = cudaLaunchAttributeClusterSchedulingPolicyPreference;     // one CTA per SM before doubling up
    attrs[2].val.clusterSchedulingPolicyPreference = cudaClusterSchedulingPolicySpread;
    cfg.attrs = attrs;
    cfg.numAttrs = 3;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    return cudaLaunchKernelEx(&cfg, gemm_cluster_kernel<MB, MINB, RB>, tmap, sa, asum, static_cast<const uint8_t*>(packed),
                              static_cast<__nv_bfloat16*>(y), static_cast<const __nv_bfloat16*>(residual), M, N, K, S, ng_max, stages,
                              reinterpret_cast<uint32_t*>(ws + WS_STATUS_OFF), debug_partials);
}
}  // namespace

// Slices per tile for the cluster kernel, at most 8 (portable cluster size) and never more than
// the number of groups.  Measured on the four layer shapes: one m-block (M <= 8) runs best with
// about 1.4 CTAs per SM (two co-resident CTAs per SM leave room for the next launch to prefetch);
// larger M, whose CTAs hold more registers and shared memory, with the largest power of two that
// keeps the launch within 0.9 CTAs per SM (clusters of 3 were always slower than 2 or 4).
int cluster_num_slices(int M, int N, int K) {
    const int G = K / GROUP, tiles = N / TILE_N, sms = device_sm_count();
    int s;
    // Powers of two only (clusters of other sizes schedule worse).  Up to 8 tokens two CTAs share an
    // SM, so up to 1.75 CTAs per SM still run as one wave; above that one CTA per SM.
    const int cta_limit = M <= 8 ? (sms * 7) / 4 : (sms * 9) / 10;
    s = 1;
    while (2 * s <= CL_MAX_S && tiles * 2 * s <= cta_limit) s *= 2;
    if (s > CL_MAX_S) s = CL_MAX_S;
    if (s > G) s = G;
    if (s < 1) s = 1;
    return s;
}

cudaError_t launch_gemm_cluster(const int8_t* qa, const uint16_t* sa, const int32_t* asum, const void* packed,
                                void* y, const void* residual, int M, int N, int K, void* workspace, int32_t* debug_partials,
                                cudaStream_t stream) {
    const int S = cluster_num_slices(M, N, K);
    if (M <= 8) {
        // two launches co-resident.  Four warp sets (each warp two blocks of 16 rows) when a slice is
        // long enough to give every set at least two groups: more groups in flight per CTA and the
        // activation fragments are loaded once for both blocks.
        const int ng_max = (K / GROUP + S - 1) / S;
        if (ng_max >= 8) return launch_mb<1, 2, 2>(qa, sa, asum, packed, y, residual, M, N, K, S, workspace, debug_partials, stream);
        return launch_mb<1, 2, 1>(qa, sa, asum, packed, y, residual, M, N, K, S, workspace, debug_partials, stream);
    }
    if (M <= 16) {
        if ((N / TILE_N) * S > device_sm_count())
            return launch_mb<2, 2, 1>(qa, sa, asum, packed, y, residual, M, N, K, S, workspace, debug_partials, stream);
        return launch_mb<2, 1, 1>(qa, sa, asum, packed, y, residual, M, N, K, S, workspace, debug_partials, stream);
    }
    if (M <= 32) return launch_mb<4, 1, 1>(qa, sa, asum, packed, y, residual, M, N, K, S, workspace, debug_partials, stream);
    return launch_mb<8, 1, 1>(qa, sa, asum, packed, y, residual, M, N, K, S, workspace, debug_partials, stream);
}

}  // namespace w4a8
