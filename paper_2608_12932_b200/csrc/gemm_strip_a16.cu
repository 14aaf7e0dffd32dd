// W4A16 small-M GEMM (up to 16 tokens): the same packed 4-bit weights against UNQUANTISED bf16 activations - the
// weight-only scheme that Sec. 3.4 contrasts W4A8 with (it shrinks the weights, which is what the memory-bound
// decode needs, and leaves the arithmetic in 16-bit floating point).  Built to measure that argument on the same
// layers with the same streaming skeleton as the W4A8 strip kernel (gemm_strip.cu): persistent CTAs, strips of R
// output channels over the whole K dealt out in equal contiguous ranges of stages, a ring of asynchronous copies fed
// by three producer warps, eight consumer warps with two 16-row units per stage each, one epilogue warp, the
// neighbour hand-over of a shared strip through tagged 64-bit words in the workspace, programmatic dependent launch.
//
// What differs is the consumer:
//  * a nibble becomes the bf16 number 128 + code by OR-ing it into the mantissa of 0x4300; subtracting the bf16
//    number 128 + z (sub.bf16x2, exact) leaves code - z: integers of magnitude <= 15, exact in bf16.  The zero point
//    is thus applied before the product and there are no group sums;
//  * mma.sync m16n8k16 bf16 x bf16 -> fp32, weights as the 16-row operand, eight per group; which k a fragment slot
//    means is free as long as both operands agree: a weight register pairs the codes k and k + 2 (nibbles 16 bits
//    apart in a packed word), so the two activation registers of an MMA are re-paired the same way with a byte permute;
//  * the group's fp32 sum P (products exact, additions rounded) is scaled by the group scale in fp32 and added to the
//    running sum: y = bf16(sum_g s_w P_g).  No weight is rounded before it is multiplied.
//  * activations are 256 B per token and group: a stage's tile is one 3-D box of 64-element (128-byte, swizzled) rows,
//    [half-group][token]; strips are at least 32 rows wide so that the tiles leave room for a ring.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include "ptx_sm100.cuh"
#include "w4a8_internal.cuh"

namespace w4a8 {
namespace {

constexpr int A16_CONSUMER_WARPS = 8;
constexpr int A16_PRODUCER_WARPS = 3;
constexpr int A16_THREADS = (A16_CONSUMER_WARPS + A16_PRODUCER_WARPS + 1) * 32;
constexpr int A16_MAX_STAGES = 8;
constexpr int A16_W_BYTES = 17408;                        // weight part of a stage (16 KB of nibbles + scales + zero points, padded)
constexpr int A16_SMEM_BUDGET = 112 * 1024;               // two CTAs per SM

struct A16Layout {
    int ring_off, bar_off, part_off, take_off, ystage_off, misc_off, total;
};
__host__ __device__ constexpr int a16_stage_bytes(int mb, int rblk) { return A16_W_BYTES + (16 / rblk) * 8 * mb * 2 * GROUP; }
__host__ __device__ inline A16Layout a16_layout(int mb, int rblk, int stages) {
    const int mp = 8 * mb;
    A16Layout L;
    L.ring_off = 0;
    L.bar_off = stages * a16_stage_bytes(mb, rblk);
    L.part_off = (L.bar_off + (2 * A16_MAX_STAGES + 2) * 8 + 15) & ~15;
    L.take_off = L.part_off + A16_CONSUMER_WARPS * 2 * mb * 32 * 16;     // one float4 per consumer lane, row block and token block
    L.ystage_off = L.take_off + rblk * mb * 32 * 16;
    L.misc_off = L.ystage_off + mp * (32 * rblk + 16);
    L.total = L.misc_off + 16;
    return L;
}

__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// two codes of a packed word (nibbles at bits sh and sh + 16) minus the zero point, as a pair of bf16
__device__ __forceinline__ uint32_t code_pair(uint32_t w, int sh, uint32_t zc) {
    const uint32_t v = ((w >> sh) & 0x000F000Fu) | 0x43004300u;         // (128 + code, 128 + code')
    uint32_t d;
    asm("sub.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(v), "r"(zc));          // exact
    return d;
}

__device__ __forceinline__ bool a16_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    uint64_t t0 = 0;
    for (uint32_t spin = 1;; ++spin) {
        if (ptx::mbar_try_wait_parked(bar, parity, 4000u)) return true;
        if ((spin & 63) == 0) {
            if (*abort_flag) return false;
            const uint64_t now = ptx::globaltimer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > ptx::WAIT_LIMIT_NS) { *abort_flag = 1; return false; }
        }
    }
}

struct A16Args {
    const uint8_t* packed;
    __nv_bfloat16* y;
    int M, N, K;
    int stages, sps, total_stages;
    uint32_t* status;
    unsigned long long* slots;
};

template <int MB, int RBLK>
__global__ void __launch_bounds__(A16_THREADS, MB == 1 ? 2 : 1)      // two token blocks need more than half an SM's registers
gemm_strip_a16_kernel(const __grid_constant__ CUtensorMap tm_act, const __grid_constant__ CUtensorMap tm_nib,
                      const __grid_constant__ CUtensorMap tm_scale, const __grid_constant__ CUtensorMap tm_zero,
                      const A16Args a) {
    ptx::pdl_launch_dependents();
    static_assert(RBLK >= 2, "strips of at least 32 rows");
    constexpr int R = 16 * RBLK, GS = 16 / RBLK, MP = 8 * MB;
    constexpr int STRIPS_PER_TILE = TILE_N / R;
    constexpr bool WHOLE = (R == TILE_N);
    constexpr int ZB = R / 2;
    constexpr uint32_t STAGE_BYTES = a16_stage_bytes(MB, RBLK);
    constexpr uint32_t HALF_BYTES = MP * 128;                 // one half-group of the activation tile: [token][128 B]
    constexpr uint32_t ACT_BYTES = GS * 2 * HALF_BYTES;
    constexpr uint32_t NARROW_W_BYTES = 16384 + GS * 2 * R + GS * ZB;
    constexpr int NIB_G = WHOLE ? BLOB_BYTES : R * 64;
    constexpr int SC_BASE = WHOLE ? BLOB_SCALE_OFF : 16384, SC_G = WHOLE ? BLOB_BYTES : 2 * R;
    constexpr int Z_BASE = WHOLE ? BLOB_ZERO_OFF : 16384 + GS * 2 * R, Z_G = WHOLE ? BLOB_BYTES : ZB;
    static_assert(NARROW_W_BYTES <= A16_W_BYTES && 2 * BLOB_BYTES <= A16_W_BYTES, "weight part of a stage");

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    const int G = a.K / GROUP;
    const int stages = a.stages, sps = a.sps;
    const A16Layout L = a16_layout(MB, RBLK, stages);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    const int lo = (int)(((long long)blockIdx.x * a.total_stages) / gridDim.x);
    const int hi = (int)(((long long)(blockIdx.x + 1) * a.total_stages) / gridDim.x);
    const int n = hi - lo;
    const int first_strip = lo / sps, last_strip = (hi - 1) / sps;

    const uint32_t bar_base = smem_base + L.bar_off;       // full[s] at 8 s, empty[s] at 8 (MAX + s)
    const uint32_t part_full = bar_base + 8 * (2 * A16_MAX_STAGES), part_empty = part_full + 8;
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + L.misc_off);

    auto load_weights = [&](int t, int s) {
        const int strip = t / sps, sg = t - strip * sps;
        const int tile = strip / STRIPS_PER_TILE, r0 = (strip % STRIPS_PER_TILE) * R, g0 = sg * GS;
        const uint32_t dst = smem_base + s * STAGE_BYTES, bar = bar_base + 8 * s;
        if (WHOLE) {
            const int valid = (G - g0) < GS ? (G - g0) : GS;
            const uint32_t bytes = (uint32_t)valid * BLOB_BYTES;
            ptx::mbar_expect_tx(bar, bytes);
            ptx::bulk_g2s(dst, a.packed + ((size_t)tile * G + g0) * BLOB_BYTES, bytes, bar);
        } else {
            ptx::mbar_expect_tx(bar, NARROW_W_BYTES);
            ptx::tma_load_4d(dst, &tm_nib, 0, r0, g0, tile, bar);
            ptx::tma_load_3d(dst + SC_BASE, &tm_scale, r0, g0, tile, bar);
            ptx::tma_load_3d(dst + Z_BASE, &tm_zero, r0 / 2, g0, tile, bar);
        }
    };

    if (warp == A16_CONSUMER_WARPS && lane == 0) {
        *abort_flag = 0;
        for (int s = 0; s < stages; ++s) {
            ptx::mbar_init(bar_base + 8 * s, 1);
            ptx::mbar_init(bar_base + 8 * (A16_MAX_STAGES + s), A16_CONSUMER_WARPS);
        }
        ptx::mbar_init(part_full, A16_CONSUMER_WARPS);
        ptx::mbar_init(part_empty, 1);
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tm_act);
        if (!WHOLE) {
            ptx::prefetch_tmap(&tm_nib);
            ptx::prefetch_tmap(&tm_scale);
            ptx::prefetch_tmap(&tm_zero);
        }
    }
    __syncthreads();
    const int pw = warp - A16_CONSUMER_WARPS;
    const bool producer = pw >= 0 && pw < A16_PRODUCER_WARPS;
    if (producer && lane == 0) {
        // weights do not depend on the previous kernel: start their stream at once
        const int first = n < stages ? n : stages;
        for (int i = pw; i < first; i += A16_PRODUCER_WARPS) load_weights(lo + i, i);
    }
    // activations and the workspace belong to the previous kernel until this wait returns
    ptx::pdl_wait();

    if (producer) {
        if (lane == 0) {
            bool go = pw < stages;
            const int uses = (n + stages - 1) / stages;
            for (int use = 0; go && use < uses; ++use) {
                for (int s = pw; s < stages; s += A16_PRODUCER_WARPS) {      // slot s belongs to producer s mod 3
                    const int i = use * stages + s;
                    if (i >= n) { go = false; break; }
                    const int t = lo + i;
                    const uint32_t bar = bar_base + 8 * s;
                    if (use > 0) {
                        if (!a16_wait(bar_base + 8 * (A16_MAX_STAGES + s), (uint32_t)((use - 1) & 1), abort_flag)) { go = false; break; }
                        load_weights(t, s);
                    }
                    ptx::mbar_arrive_expect_tx(bar, ACT_BYTES);
                    ptx::tma_load_3d(smem_base + s * STAGE_BYTES + A16_W_BYTES, &tm_act, 0, 0, (t % sps) * GS * 2, bar);
                }
            }
        }
    } else if (warp < A16_CONSUMER_WARPS) {
        // ----------------------------------------------------------------- consumers ----
        // the warp's two units of a stage: two 16-row blocks, rows 32 rp .. 32 rp + 31, of group gi
        constexpr int WPG = RBLK / 2;
        const int gi = warp / WPG, rp = warp % WPG;
        const int r = lane >> 2, j = lane & 3;
        const int row = rp * 32 + r;
        const uint32_t nib_off = gi * NIB_G + row * 64 + blob_chunk_pos(r, j) * 16;   // rows r, r + 8, r + 16, r + 24 share their swizzle
        const uint32_t sc_off = SC_BASE + gi * SC_G + 2 * row;
        const uint32_t z_off = Z_BASE + gi * Z_G + (row >> 1);
        const int zsh = (r & 1) * 4;
        // token r of a token block, k 32 j .. 32 j + 31 of the group: half-group j / 2, 16-byte chunks 4 (j % 2) + i
        const uint32_t act_off = A16_W_BYTES + (gi * 2 + (j >> 1)) * HALF_BYTES + r * 128;
        const uint32_t part_lane = smem_base + L.part_off + (warp * 2 * MB * 32 + lane) * 16;
        float facc[2][MB][4];
#pragma unroll
        for (int f = 0; f < 2; ++f)
#pragma unroll
            for (int mb = 0; mb < MB; ++mb) facc[f][mb][0] = facc[f][mb][1] = facc[f][mb][2] = facc[f][mb][3] = 0.0f;

        bool ok = true;
        int flushed = 0;
        auto flush = [&]() {
            if (flushed > 0) ok = ok && a16_wait(part_empty, (uint32_t)((flushed - 1) & 1), abort_flag);
            if (ok) {
#pragma unroll
                for (int f = 0; f < 2; ++f)
#pragma unroll
                    for (int mb = 0; mb < MB; ++mb) {
                        ptx::sts128(part_lane + (f * MB + mb) * 512,
                                    make_float4(facc[f][mb][0], facc[f][mb][1], facc[f][mb][2], facc[f][mb][3]));
                        facc[f][mb][0] = facc[f][mb][1] = facc[f][mb][2] = facc[f][mb][3] = 0.0f;
                    }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(part_full);
            }
            ++flushed;
        };

        int strip = first_strip, sg = lo - first_strip * sps;
        uint32_t stage = smem_base, full = bar_base, phase = 0;
        int s = 0;
        for (int i = 0; i < n; ++i) {
            ok = a16_wait(full, phase, abort_flag);
            if (!ok) break;
            {
                const int g0 = sg * GS + gi;
                const uint4 wa0 = ptx::lds128(stage + nib_off), wb0 = ptx::lds128(stage + nib_off + 8 * 64);
                const uint4 wa1 = ptx::lds128(stage + nib_off + 16 * 64), wb1 = ptx::lds128(stage + nib_off + 24 * 64);
                float s_lo0 = __half2float(__ushort_as_half((unsigned short)ptx::lds_u16(stage + sc_off)));
                float s_hi0 = __half2float(__ushort_as_half((unsigned short)ptx::lds_u16(stage + sc_off + 16)));
                float s_lo1 = __half2float(__ushort_as_half((unsigned short)ptx::lds_u16(stage + sc_off + 32)));
                float s_hi1 = __half2float(__ushort_as_half((unsigned short)ptx::lds_u16(stage + sc_off + 48)));
                // 128 + z as a pair of equal bf16 numbers, per row
                const uint32_t zl0 = (0x4300u | ((ptx::lds_u8(stage + z_off) >> zsh) & 0xFu)) * 0x00010001u;
                const uint32_t zh0 = (0x4300u | ((ptx::lds_u8(stage + z_off + 4) >> zsh) & 0xFu)) * 0x00010001u;
                const uint32_t zl1 = (0x4300u | ((ptx::lds_u8(stage + z_off + 8) >> zsh) & 0xFu)) * 0x00010001u;
                const uint32_t zh1 = (0x4300u | ((ptx::lds_u8(stage + z_off + 12) >> zsh) & 0xFu)) * 0x00010001u;
                // groups past the end of K (a ragged last stage): the slot holds finite numbers there (any nibble is a
                // finite bf16 after the OR, activations past K arrive as zeros), a zero scale makes them add nothing
                if (g0 >= G) s_lo0 = s_hi0 = s_lo1 = s_hi1 = 0.0f;
#pragma unroll
                for (int mb = 0; mb < MB; ++mb) {
                    float c0[4] = {0.0f, 0.0f, 0.0f, 0.0f}, c1[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                    const uint32_t ab = stage + act_off + mb * 1024;
#pragma unroll
                    for (int i4 = 0; i4 < 4; ++i4) {
                        // activations k0 .. k0 + 7, k0 = 32 j + 8 i4, of this lane's token
                        const uint4 p = ptx::lds128(ab + (uint32_t)((((j & 1) * 4 + i4) ^ r) << 4));
                        const uint32_t b00 = __byte_perm(p.x, p.y, 0x5410), b01 = __byte_perm(p.x, p.y, 0x7632);   // (k, k+2), (k+1, k+3)
                        const uint32_t b10 = __byte_perm(p.z, p.w, 0x5410), b11 = __byte_perm(p.z, p.w, 0x7632);   // the next four k
                        // the packed words that hold those eight k: x and y of the chunk for i4 < 2, z and w above; low
                        // nibbles for even i4, high for odd
                        const uint32_t xa0 = i4 < 2 ? wa0.x : wa0.z, ya0 = i4 < 2 ? wa0.y : wa0.w;
                        const uint32_t xb0 = i4 < 2 ? wb0.x : wb0.z, yb0 = i4 < 2 ? wb0.y : wb0.w;
                        const uint32_t xa1 = i4 < 2 ? wa1.x : wa1.z, ya1 = i4 < 2 ? wa1.y : wa1.w;
                        const uint32_t xb1 = i4 < 2 ? wb1.x : wb1.z, yb1 = i4 < 2 ? wb1.y : wb1.w;
                        const int sh = (i4 & 1) * 4;
                        mma_bf16(c0, code_pair(xa0, sh, zl0), code_pair(xb0, sh, zh0), code_pair(xa0, sh + 8, zl0), code_pair(xb0, sh + 8, zh0), b00, b01);
                        mma_bf16(c1, code_pair(xa1, sh, zl1), code_pair(xb1, sh, zh1), code_pair(xa1, sh + 8, zl1), code_pair(xb1, sh + 8, zh1), b00, b01);
                        mma_bf16(c0, code_pair(ya0, sh, zl0), code_pair(yb0, sh, zh0), code_pair(ya0, sh + 8, zl0), code_pair(yb0, sh + 8, zh0), b10, b11);
                        mma_bf16(c1, code_pair(ya1, sh, zl1), code_pair(yb1, sh, zh1), code_pair(ya1, sh + 8, zl1), code_pair(yb1, sh + 8, zh1), b10, b11);
                    }
                    facc[0][mb][0] = fmaf(s_lo0, c0[0], facc[0][mb][0]);
                    facc[0][mb][1] = fmaf(s_lo0, c0[1], facc[0][mb][1]);
                    facc[0][mb][2] = fmaf(s_hi0, c0[2], facc[0][mb][2]);
                    facc[0][mb][3] = fmaf(s_hi0, c0[3], facc[0][mb][3]);
                    facc[1][mb][0] = fmaf(s_lo1, c1[0], facc[1][mb][0]);
                    facc[1][mb][1] = fmaf(s_lo1, c1[1], facc[1][mb][1]);
                    facc[1][mb][2] = fmaf(s_hi1, c1[2], facc[1][mb][2]);
                    facc[1][mb][3] = fmaf(s_hi1, c1[3], facc[1][mb][3]);
                }
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(full + 8 * A16_MAX_STAGES);
            ++s; stage += STAGE_BYTES; full += 8;
            if (s == stages) { s = 0; stage = smem_base; full = bar_base; phase ^= 1; }
            if (++sg == sps) { flush(); sg = 0; ++strip; if (!ok) break; }
        }
        if (ok && sg != 0) flush();                          // the range ends inside a strip
    } else {
        // ------------------------------------------------------------------ epilogue ----
        bool ok = true;
        const int r = lane >> 2, j = lane & 3;
        const int nseg = last_strip - first_strip + 1;
        constexpr int ITEMS = RBLK * MB;
        constexpr int YPITCH = 2 * R + 16;
        const uint32_t part_lane = smem_base + L.part_off + lane * 16, take_lane = smem_base + L.take_off + lane * 16;
        const uint32_t ystage = smem_base + L.ystage_off;
        constexpr size_t SLOT = (size_t)R * MP * 8;
        ulonglong2* mine = reinterpret_cast<ulonglong2*>(reinterpret_cast<uint8_t*>(a.slots) + (size_t)blockIdx.x * SLOT);
        ulonglong2* theirs = reinterpret_cast<ulonglong2*>(reinterpret_cast<uint8_t*>(a.slots) + (size_t)(blockIdx.x + 1) * SLOT);
        constexpr unsigned long long TAG = 1ull << 32;
        for (int q = 0; q < nseg && ok; ++q) {
            const int strip = first_strip + q;
            const bool has_start = lo <= strip * sps, has_end = hi >= (strip + 1) * sps;
            const bool take = has_start && !has_end;       // the neighbour holds the strip's later groups
            if (take) {
                constexpr int BATCH = 2 * ITEMS < 8 ? 2 * ITEMS : 8;
                for (int base = 0; base < 2 * ITEMS && ok; base += BATCH) {
                    ulonglong2 v[BATCH];
                    uint64_t t0 = 0;
                    for (uint32_t spin = 0;; ++spin) {
                        bool all = true;
#pragma unroll
                        for (int e = 0; e < BATCH; ++e) {
                            v[e] = __ldcg(theirs + (base + e) * 32 + lane);
                            all = all && (v[e].x >> 32) == 1ull && (v[e].y >> 32) == 1ull;
                        }
                        if (__all_sync(0xFFFFFFFFu, all)) break;
                        if (*abort_flag) { ok = false; break; }
                        const uint64_t now = ptx::globaltimer_ns();
                        if (t0 == 0) t0 = now;
                        else if (now - t0 > ptx::WAIT_LIMIT_NS) { *abort_flag = 1; ok = false; break; }
                        __nanosleep(200);
                    }
                    if (!ok) break;
#pragma unroll
                    for (int e = 0; e < BATCH; ++e) {
                        const uint32_t dst = take_lane + ((base + e) >> 1) * 512 + ((base + e) & 1) * 8;
                        asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(dst), "r"((uint32_t)v[e].x), "r"((uint32_t)v[e].y) : "memory");
                        __stcg(theirs + (base + e) * 32 + lane, make_ulonglong2(0ull, 0ull));
                    }
                }
                if (!ok) break;
                __syncwarp();
            }
            ok = a16_wait(part_full, (uint32_t)(q & 1), abort_flag);
            if (!ok) break;
#pragma unroll 1
            for (int item = 0; item < ITEMS; ++item) {
                const int rb = item / MB, mb = item % MB;
                float4 acc = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                constexpr int WPG = RBLK / 2;
#pragma unroll
                for (int gi = 0; gi < A16_CONSUMER_WARPS / WPG; ++gi) {        // the warps that hold this row block, in warp order
                    const int w = gi * WPG + rb / 2, f = rb % 2;
                    const float4 v = ptx::lds128f(part_lane + ((w * 2 + f) * MB + mb) * 512);
                    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                }
                if (!has_start) {
                    __stcg(mine + (2 * item) * 32 + lane, make_ulonglong2(TAG | __float_as_uint(acc.x), TAG | __float_as_uint(acc.y)));
                    __stcg(mine + (2 * item + 1) * 32 + lane, make_ulonglong2(TAG | __float_as_uint(acc.z), TAG | __float_as_uint(acc.w)));
                    continue;
                }
                if (take) {
                    const float4 o = ptx::lds128f(take_lane + item * 512);
                    acc.x += o.x; acc.y += o.y; acc.z += o.z; acc.w += o.w;      // earlier groups + later groups
                }
                const int m0 = 8 * mb + 2 * j;
                const uint32_t yo = ystage + m0 * YPITCH + (rb * 16 + r) * 2;
                const __nv_bfloat16 o0 = __float2bfloat16_rn(acc.x), o1 = __float2bfloat16_rn(acc.y);
                const __nv_bfloat16 o2 = __float2bfloat16_rn(acc.z), o3 = __float2bfloat16_rn(acc.w);
                asm volatile("st.shared.u16 [%0], %1;" ::"r"(yo), "h"(__bfloat16_as_ushort(o0)) : "memory");
                asm volatile("st.shared.u16 [%0], %1;" ::"r"(yo + YPITCH), "h"(__bfloat16_as_ushort(o1)) : "memory");
                asm volatile("st.shared.u16 [%0], %1;" ::"r"(yo + 16), "h"(__bfloat16_as_ushort(o2)) : "memory");
                asm volatile("st.shared.u16 [%0], %1;" ::"r"(yo + YPITCH + 16), "h"(__bfloat16_as_ushort(o3)) : "memory");
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(part_empty);
            if (has_start) {
                constexpr int CPR = R / 8;
                for (int c = lane; c < a.M * CPR; c += 32) {
                    const int m = c / CPR, col = c - m * CPR;
                    const uint4 v = ptx::lds128(ystage + m * YPITCH + col * 16);
                    *reinterpret_cast<uint4*>(a.y + (size_t)m * a.N + (size_t)strip * R + col * 8) = v;
                }
                __syncwarp();
            }
        }
    }
    __syncwarp();
    if (*abort_flag) {
        if (lane == 0) atomicExch(a.status, (uint32_t)W4A8_ERR_TIMEOUT);
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);      // copies in flight: a bounded time to land
    }
}

template <int MB, int RBLK>
cudaError_t launch_a16(const void* x, const void* packed, void* y, int M, int N, int K, int ctas, void* workspace,
                       cudaStream_t stream) {
    constexpr int R = 16 * RBLK, GS = 16 / RBLK, MP = 8 * MB;
    const int G = K / GROUP;
    const int fixed = a16_layout(MB, RBLK, 0).total + 1024;
    int stages = (A16_SMEM_BUDGET - fixed) / a16_stage_bytes(MB, RBLK);
    if (stages > A16_MAX_STAGES) stages = A16_MAX_STAGES;
    if (stages < 2) return cudaErrorInvalidConfiguration;
    const size_t smem = (size_t)a16_layout(MB, RBLK, stages).total + 1024;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    static bool attr_done[64] = {false};
    if (!attr_done[dev]) {
        e = cudaFuncSetAttribute(gemm_strip_a16_kernel<MB, RBLK>, cudaFuncAttributeMaxDynamicSharedMemorySize, A16_SMEM_BUDGET);
        if (e != cudaSuccess) return e;
        attr_done[dev] = true;
    }
    CUtensorMap tm_act, tm_nib, tm_scale, tm_zero;
    e = make_x_half_group_map(&tm_act, x, M, K, MP, 2 * GS);
    if (e != cudaSuccess) return e;
    e = make_strip_weight_maps(&tm_nib, &tm_scale, &tm_zero, packed, N, K, R, GS);
    if (e != cudaSuccess) return e;

    uint8_t* ws = static_cast<uint8_t*>(workspace);
    A16Args a;
    a.packed = static_cast<const uint8_t*>(packed);
    a.y = static_cast<__nv_bfloat16*>(y);
    a.M = M; a.N = N; a.K = K;
    a.stages = stages;
    a.sps = (G + GS - 1) / GS;
    a.total_stages = (N / R) * a.sps;
    a.status = reinterpret_cast<uint32_t*>(ws + WS_STATUS_OFF);
    a.slots = reinterpret_cast<unsigned long long*>(ws + WS_HEADER_BYTES);

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctas, 1, 1);
    cfg.blockDim = dim3(A16_THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attrs[1];
    attrs[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attrs;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemm_strip_a16_kernel<MB, RBLK>, tm_act, tm_nib, tm_scale, tm_zero, a);
}

}  // namespace

bool a16_supported(int M, int N, int K) {
    (void)K;
    return M >= 1 && M <= STRIP_MAX_M && N >= 32;
}

// Strip width and CTA count (the W4A8 strip kernel's rule, with 32 rows as the narrowest strip: an activation tile is
// twice as large here): up to 8 tokens the widest strip that still gives about 1.25 strips per SM, one step narrower
// if that puts two CTAs on every SM; 64 rows and one CTA per SM for two token blocks.
void a16_plan(int M, int N, int K, int* strip_rows, int* ctas) {
    (void)K;
    const int sms = device_sm_count();
    int R = 128;
    if (M <= 8) {
        while (R > 32 && N / R < (sms * 5) / 4) R /= 2;
        if (R > 32 && N / R < 2 * sms) R /= 2;
    } else {
        R = 64;
    }
    int limit = (M <= 8 ? 2 : 1) * sms;
    const int slot_limit = (STRIP_MAX_CTAS * STRIP_SLOT_BYTES) / (R * (M <= 8 ? 8 : 16) * 8);
    if (limit > slot_limit) limit = slot_limit;
    int c = N / R;
    if (c > limit) c = limit;
    if (strip_rows) *strip_rows = R;
    if (ctas) *ctas = c;
}

cudaError_t launch_gemm_strip_a16(const void* x, const void* packed, void* y, int M, int N, int K, void* workspace,
                                  cudaStream_t stream) {
    int R = 0, ctas = 0;
    a16_plan(M, N, K, &R, &ctas);
    if (M <= 8) {
        if (R == 128) return launch_a16<1, 8>(x, packed, y, M, N, K, ctas, workspace, stream);
        if (R == 64) return launch_a16<1, 4>(x, packed, y, M, N, K, ctas, workspace, stream);
        return launch_a16<1, 2>(x, packed, y, M, N, K, ctas, workspace, stream);
    }
    return launch_a16<2, 4>(x, packed, y, M, N, K, ctas, workspace, stream);
}

}  // namespace w4a8
