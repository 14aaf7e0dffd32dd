// Small-M W4A8 GEMM, strip variant (up to 16 tokens): one persistent CTA per SM, no split of K
// between CTAs and therefore no exchange on the critical path.  (Sec. 3.2: a draft block is 8
// tokens; Sec. 4: decode is bound by the weight bytes the GPU must load - this kernel streams
// them once, at HBM width, evenly over the SMs.)
//
//  * A strip is R = 16 * RBLK consecutive output channels (rows of a 128-channel tile of the packed
//    layout) over the whole K range; R is the widest of 128 / 64 / 32 / 16 that still gives about
//    one strip per SM.  A pipeline stage holds GS = 256 / R consecutive groups of one strip: always
//    16 KB of nibbles, i.e. sixteen units of 16 rows x one group, one per consumer warp.
//  * Copies are few and large, because what a copy costs its issuing thread does not depend on its
//    size (measured on B200: one thread gets a bulk copy or a TMA box issued every 480 ns, be it 1 KB
//    or 17 KB, however deep the ring; threads of different warps issue in parallel; 64-byte box rows
//    are as fast as 2 KB ones).  With R = 128 a stage's weights are ONE bulk copy of two whole blobs
//    (17 024 B, scales and zero points included); narrower strips take one 4-D box for the nibbles
//    and two small 3-D boxes for their own scales and zero points.  The activation tiles of the
//    stage's groups are one 3-D box (128-byte swizzle).  Three producer warps share the ring (slot s
//    belongs to warp s % 3: a parity wait tells only consecutive phases apart, so one slot must never
//    be re-armed by two threads out of turn).
//  * Work is dealt out in stages: strips x stages-per-strip, cut into gridDim.x equal contiguous
//    ranges.  With at least as many strips as CTAs a strip is shared by at most two CTAs: the one
//    that holds its later groups meets them first (they open its range), writes its fp32 sums to
//    its slot of the workspace, each as a 64-bit word that carries a tag beside the float (so a
//    word says for itself that it has been written: no flag, no fence, one round trip to read);
//    the one that holds the earlier groups meets them last, fetches the neighbour's words while its
//    own last strip is still being multiplied (bounded retries), zeroes them for the next call,
//    adds (earlier + later groups: a fixed order) and stores the strip.  Every SM thus streams the
//    same number of bytes, whatever the layer's width.
//  * Consumers: eight warps, each with two of a stage's sixteen units, whose loads and MMAs interleave: two
//    16-row blocks of one group (they share the activation fragments), or, in 16-row strips, the one block of
//    two groups.  mma.sync m16n8k32 (u8 x s8 -> s32), weights as the 16-row operand.  The low nibbles
//    feed one chain of two MMAs that starts at the zero-point term -z * sum(q_a), the high nibbles -
//    masked in place, i.e. as 16 x code - a second chain; D = low + high / 16 exactly (int32), scaled
//    by the group scale in fp32.  A warp keeps its sums over the groups it meets in registers; at the
//    end of a strip all eight warps put them into shared memory and go on, and the epilogue warp
//    adds them in warp order (fixed: deterministic), applies the token scale and stores bf16 - or
//    hands the sums over as described above.
//  * Launched with programmatic stream serialisation: the weight copies of the first ring fill
//    are requested before griddepcontrol.wait, so this kernel's weight stream starts under the
//    tail of its predecessor; activations, token scales, group sums and the workspace are touched
//    only after the wait.  A CTA stays under half an SM's shared memory and registers, so that
//    two consecutive launches are resident together.
//  * Every wait is bounded; on expiry the CTA sets its abort flag, every role leaves its loop, the
//    status word becomes W4A8_ERR_TIMEOUT and the kernel returns.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#ifdef W4A8_TUNING
#include <cstdlib>
#endif
#include "ptx_sm100.cuh"
#include "quant_common.cuh"
#include "w4a8_internal.cuh"

namespace w4a8 {
namespace {

// Eight consumer warps, each taking two of a stage's sixteen units (the same 16 rows of two groups): with twelve
// warps in the CTA two CTAs per SM leave 80 registers per thread, enough to keep every per-lane offset in a
// register.  (Sixteen thin warps at 48 registers re-derived them from the thread index in every unit: 119
// instructions per unit, more than half of them address arithmetic.  Twelve consumer warps at 64 registers and
// 24-unit stages, -DST_CW=12, give the same results 10 % slower: 14.4 against 12.9 us on the 4096 -> 24576 layer.)
#ifndef ST_CW
#define ST_CW 8
#endif
constexpr int ST_CONSUMER_WARPS = ST_CW;
constexpr int ST_UNITS = 2 * ST_CONSUMER_WARPS;           // units (16 rows x one group) per stage
constexpr int ST_NIB_BYTES = ST_UNITS * 1024;             // nibbles of a stage
// three producer warps: two or four (-DST_PW) move every layer by less than 2 % either way
#ifndef ST_PW
#define ST_PW 3
#endif
constexpr int ST_PRODUCER_WARPS = ST_PW;
constexpr int ST_EPILOGUE_WARP = ST_CONSUMER_WARPS + ST_PRODUCER_WARPS;
constexpr int ST_THREADS = (ST_CONSUMER_WARPS + ST_PRODUCER_WARPS + 1) * 32;
constexpr int ST_MAX_STAGES = 8;
constexpr int ST_W_BYTES = ST_CW == 8 ? 17408 : (ST_CW == 12 ? 26624 : 34816);                         // weight part of a stage (16 KB of nibbles + scales + zero points, padded)
// CTAs per SM.  One CTA per SM with sixteen consumer warps (-DST_CW=16 -DST_MINB=1: 96 registers, no spills with two
// token blocks, a 220 KB ring) was measured equal to 17 % slower at up to 8 tokens and equal to 10 % faster at 16
// (the 4096 -> 24576 layer: 17.3 against 19.2 us); not worth a second build of the kernel.
#ifndef ST_MINB
#define ST_MINB 2
#endif
constexpr int ST_SMEM_BUDGET = (ST_MINB == 2 ? 112 : 220) * 1024;   // per CTA: two CTAs share an SM
constexpr uint32_t ST_STAY = 128;                         // one-kernel fused form: CTAs that stay to requantise (swept 32..296 on B200)
constexpr int ST_MAX_ASUM_WORDS = 4096;                   // group sums of all tokens kept in shared memory

struct StLayout {
    int ring_off, bar_off, asum_off, sa_off, part_off, take_off, ystage_off, misc_off, total;
};
__host__ __device__ constexpr int st_stage_bytes(int mb, int rblk) { return ST_W_BYTES + (ST_UNITS / rblk) * 8 * mb * GROUP; }
__host__ __device__ inline StLayout st_layout(int mb, int rblk, int stages, int G, bool fp32_stage = false) {
    const int mp = 8 * mb;
    StLayout L;
    L.ring_off = 0;                                         // stages x (weights, then GS activation tiles), 1024-aligned
    L.bar_off = stages * st_stage_bytes(mb, rblk);
    L.asum_off = (L.bar_off + (2 * ST_MAX_STAGES + 2) * 8 + 15) & ~15;
    L.sa_off = L.asum_off + G * mp * 4;                     // group sums, [group][token]
    L.part_off = (L.sa_off + mp * 4 + 15) & ~15;            // token scales as fp32
    L.take_off = L.part_off + ST_CONSUMER_WARPS * (rblk >= 2 ? 2 : 1) * mb * 32 * 16;   // one float4 per consumer lane, row block and token block
    L.ystage_off = L.take_off + rblk * mb * 32 * 16;        // the neighbour's sums of a shared strip
    // a strip's outputs, [token][channel], rows padded by 16 B: bf16, or fp32 when a residual is added at the store
    L.misc_off = L.ystage_off + mp * ((fp32_stage ? 64 : 32) * rblk + 16);
    L.total = L.misc_off + 16;
    return L;
}

// the same with a zero accumulator going in (no registers to clear)
__device__ __forceinline__ void mma_u8s8_z(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                           uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(0));
}

__device__ __forceinline__ void mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Bounded wait without back-off: a pending try_wait lets the hardware park the thread (up to the hint) until the
// phase completes, so the loop turns rarely and costs the working warps no issue slots; the clock is looked at
// every 64 turns.
__device__ __forceinline__ bool st_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
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

// h[m, 128 g .. 128 g + 127] -> codes, group sum and (for g == 0) the token's scale; one warp, four values per lane
__device__ __forceinline__ void requant_unit(const __nv_bfloat16* h, int I, int Gh, int u, int lane, int8_t* qa_h,
                                             uint16_t* sa_h, int32_t* asum_h, const uint32_t* sync) {
    const int m = u / Gh, g = u - m * Gh;
    const size_t at = (size_t)m * I + (size_t)g * GROUP + 4 * lane;
    const uint2 hv = __ldcg(reinterpret_cast<const uint2*>(h + at));
    const __half sh = row_scale_from_amax_bits(__ldcg(sync + m));
    const float s = __half2float(sh);
    int q0 = 0, q1 = 0, q2 = 0, q3 = 0;
    if (s != 0.0f) {
        q0 = quant1(hv.x << 16, s); q1 = quant1(hv.x & 0xFFFF0000u, s);
        q2 = quant1(hv.y << 16, s); q3 = quant1(hv.y & 0xFFFF0000u, s);
    }
    *reinterpret_cast<uint32_t*>(qa_h + at) =
        (uint32_t)(q0 & 0xFF) | ((uint32_t)(q1 & 0xFF) << 8) | ((uint32_t)(q2 & 0xFF) << 16) | ((uint32_t)q3 << 24);
    const int sum = __reduce_add_sync(0xFFFFFFFFu, q0 + q1 + q2 + q3);
    if (lane == 0) {
        asum_h[(size_t)m * Gh + g] = sum;
        if (g == 0) sa_h[m] = __half_as_ushort(sh);
    }
}

#ifdef W4A8_TRACE
// working builds only: time stamps of one launch's stages, [launch % 64][CTA < 320][96] words
__device__ unsigned long long g_strip_trace[64 * 320 * 96];
__device__ unsigned int g_strip_trace_count[320];
#define ST_STAMP(k) do { g_strip_trace[((size_t)(trace_launch & 63) * 320 + blockIdx.x) * 96 + (k)] = ptx::globaltimer_ns(); } while (0)
#define ST_PUT(k, v) do { g_strip_trace[((size_t)(trace_launch & 63) * 320 + blockIdx.x) * 96 + (k)] = (unsigned long long)(v); } while (0)
#define ST_CLK() clock64()
#else
#define ST_STAMP(k) do { } while (0)
#define ST_PUT(k, v) do { } while (0)
#define ST_CLK() 0ll
#endif

struct StripArgs {
    const uint16_t* sa;
    const int32_t* asum;
    const uint8_t* packed;
    __nv_bfloat16* y;
    int M, N, K;
    int stages;              // ring length
    int pre;                 // ring slots whose weights are requested before griddepcontrol.wait (the rest: L2 prefetch).
                             // The whole ring: fewer (1..3 slots, so that the first activation tile would not queue behind
                             // them) changed nothing on the wide layers and cost 2 to 19 % on the narrow ones - the first
                             // tile takes 1.5-2 us under the weight stream however little this CTA has in flight.
    int sps;                 // stages per strip = ceil(G / GS)
    int total_stages;        // strips x sps
    uint32_t* status;
    unsigned long long* slots;   // one strip of tagged fp32 sums per CTA (STRIP_SLOT_BYTES each), zero between calls
    int32_t* debug_partials;
    const __nv_bfloat16* residual;   // null, or bf16 [M,N] added to the projection before the one rounding (may be y)
    // fused form only (gate+up projection -> SiLU * up -> requantise): N = 2 I
    __nv_bfloat16* h;        // [M, I] bf16, written before and read after the grid-wide barrier
    int8_t* qa_h;            // [M, I]
    uint16_t* sa_h;          // [M]
    int32_t* asum_h;         // [M, I / 128]
    uint32_t* sync;          // workspace words: amax[16] (bf16 magnitudes), arrivals, departures; zero between calls
};

// FUSE (Sec. 3.5, "Kernel Fusion"): the layer is a fused gate+up projection whose output channels alternate in
// runs of eight (rows 16 b .. 16 b + 7 of the packed layer are gate channels 8 b .. 8 b + 7, rows 16 b + 8 .. 16 b + 15
// the up channels of the same indices), so that a lane of the epilogue warp holds gate and up of one channel.  The
// epilogue rounds both to bf16 as the plain kernel would, computes h = bf16(SiLU(gate) * up), stores h and keeps
// the largest |h| per token (atomic maxima in the workspace); y is never stored.  What remains is to quantise h once
// every token's maximum is final, one (token, group of 128) per warp.  FUSE == 2: a second, small kernel does that
// (requant_kernel below; the kernel boundary is the grid-wide wait).  FUSE == 1, the one-kernel form: every CTA
// counts itself in; the last 128 to do so stay, wait (bounded) until the count is complete, and quantise.
// FUSE == 3 is unrelated to gate+up: the plain projection with a residual added at the store (fp32 staging, the
// residual's 16-byte pieces requested before the wait for the consumers), for the O and down projections.
template <int MB, int RBLK, bool DEBUG, int FUSE>
__global__ void __launch_bounds__(ST_THREADS, ST_MINB)
gemm_strip_kernel(const __grid_constant__ CUtensorMap tm_act, const __grid_constant__ CUtensorMap tm_nib,
                  const __grid_constant__ CUtensorMap tm_scale, const __grid_constant__ CUtensorMap tm_zero,
                  const StripArgs a) {
    ptx::pdl_launch_dependents();
#ifdef W4A8_TRACE
    __shared__ unsigned int trace_launch_s;
    if (threadIdx.x == 0) trace_launch_s = atomicAdd(&g_strip_trace_count[blockIdx.x], 1u);
    __syncthreads();
    const unsigned int trace_launch = trace_launch_s;
    if (threadIdx.x == 0) ST_STAMP(0);
#endif
    constexpr int R = 16 * RBLK, GS = ST_UNITS / RBLK, MP = 8 * MB;
    constexpr int STRIPS_PER_TILE = TILE_N / R;
    constexpr bool WHOLE = (R == TILE_N);                  // whole blobs: weights, scales and zero points in one bulk copy
    constexpr int ZB = R / 2 < 16 ? 16 : R / 2;            // bytes of zero points fetched per group (16-byte granules)
    constexpr uint32_t STAGE_BYTES = st_stage_bytes(MB, RBLK);
    constexpr uint32_t ACT_BYTES = GS * MP * GROUP;
    constexpr uint32_t NARROW_W_BYTES = ST_NIB_BYTES + GS * 2 * R + GS * ZB;
    // byte offsets inside a stage
    constexpr int NIB_G = WHOLE ? BLOB_BYTES : R * 64;               // from one group's rows to the next group's
    constexpr int SC_BASE = WHOLE ? BLOB_SCALE_OFF : ST_NIB_BYTES, SC_G = WHOLE ? BLOB_BYTES : 2 * R;
    constexpr int Z_BASE = WHOLE ? BLOB_ZERO_OFF : ST_NIB_BYTES + GS * 2 * R, Z_G = WHOLE ? BLOB_BYTES : ZB;
    static_assert(NARROW_W_BYTES <= ST_W_BYTES && (ST_UNITS / 8) * BLOB_BYTES <= ST_W_BYTES, "weight part of a stage");

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    const int G = a.K / GROUP;
    const int stages = a.stages, sps = a.sps;
    constexpr bool SILU = FUSE == 1 || FUSE == 2;          // gate+up epilogue; FUSE == 3: residual epilogue
    const StLayout L = st_layout(MB, RBLK, stages, G, FUSE == 3);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // this CTA's contiguous range of stages, [lo, hi), and the strips it touches
    const int lo = (int)(((long long)blockIdx.x * a.total_stages) / gridDim.x);
    const int hi = (int)(((long long)(blockIdx.x + 1) * a.total_stages) / gridDim.x);
    const int n = hi - lo;
    const int first_strip = lo / sps, last_strip = (hi - 1) / sps;

    const uint32_t bar_base = smem_base + L.bar_off;       // full[s] at 8 s, empty[s] at 8 (MAX + s)
    const uint32_t part_full = bar_base + 8 * (2 * ST_MAX_STAGES), part_empty = part_full + 8;
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + L.misc_off);

    // weight copies of stage t (global stage index) into ring slot s, announced to the slot's barrier
    auto load_weights = [&](int t, int s) {
        const int strip = t / sps, sg = t - strip * sps;
        const int tile = strip / STRIPS_PER_TILE, r0 = (strip % STRIPS_PER_TILE) * R, g0 = sg * GS;
        const uint32_t dst = smem_base + s * STAGE_BYTES, bar = bar_base + 8 * s;
        if (WHOLE) {
            const int valid = (G - g0) < GS ? (G - g0) : GS;           // never past the tile's last blob
            const uint32_t bytes = (uint32_t)valid * BLOB_BYTES;
            ptx::mbar_expect_tx(bar, bytes);
            ptx::bulk_g2s(dst, a.packed + ((size_t)tile * G + g0) * BLOB_BYTES, bytes, bar);
        } else {
            ptx::mbar_expect_tx(bar, NARROW_W_BYTES);      // boxes deliver their full size (zeros past the last group)
            ptx::tma_load_4d(dst, &tm_nib, 0, r0, g0, tile, bar);
            ptx::tma_load_3d(dst + SC_BASE, &tm_scale, r0, g0, tile, bar);
            // zero points: R / 2 bytes from byte r0 / 2 of the blob's 64; a 16-row strip fetches its 32-row granule
            ptx::tma_load_3d(dst + Z_BASE, &tm_zero, R < 32 ? (r0 >> 5) * 16 : r0 / 2, g0, tile, bar);
        }
    };

    if (warp == ST_CONSUMER_WARPS && lane == 0) {
        *abort_flag = 0;
        for (int s = 0; s < stages; ++s) {
            ptx::mbar_init(bar_base + 8 * s, 1);
            ptx::mbar_init(bar_base + 8 * (ST_MAX_STAGES + s), ST_CONSUMER_WARPS);
        }
        ptx::mbar_init(part_full, ST_CONSUMER_WARPS);
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
    const int pw = warp - ST_CONSUMER_WARPS;               // producer index, 0..2, for the producer warps
    const bool producer = pw >= 0 && pw < ST_PRODUCER_WARPS;
    if (producer && lane == 0) {
        // weights do not depend on the previous kernel: start their stream at once
        const int first = n < a.pre ? n : a.pre;
        for (int i = pw; i < first; i += ST_PRODUCER_WARPS) load_weights(lo + i, i);
        // what the ring cannot hold is asked into L2 meanwhile, so that HBM keeps streaming under the previous
        // kernel and the ring refills from L2 (a third of the latency) once this one runs
        for (int i = first + pw; i < n; i += ST_PRODUCER_WARPS) {
            const int t = lo + i, strip = t / sps, sg = t - strip * sps;
            const int tile = strip / STRIPS_PER_TILE, r0 = (strip % STRIPS_PER_TILE) * R, g0 = sg * GS;
            if (WHOLE) {
                const int valid = (G - g0) < GS ? (G - g0) : GS;
                ptx::bulk_prefetch_l2(a.packed + ((size_t)tile * G + g0) * BLOB_BYTES, (uint32_t)valid * BLOB_BYTES);
            } else {
                ptx::tma_prefetch_4d(&tm_nib, 0, r0, g0, tile);
                ptx::tma_prefetch_3d(&tm_scale, r0, g0, tile);
                ptx::tma_prefetch_3d(&tm_zero, R < 32 ? (r0 >> 5) * 16 : r0 / 2, g0, tile);
            }
        }
    }
    // Activations, their scales and group sums, and the workspace belong to the previous kernel until
    // this wait returns.  They are read only after it and only through L2 (TMA, ld.global.cg).
    ptx::pdl_wait();
    if (tid == 0) ST_STAMP(1);

    if (producer) {
        // ----------------------------------------------------------------- producers ----
        if (lane == 0) {
            bool go = pw < stages;                              // a short ring leaves the last producer without a slot
            const int uses = (n + stages - 1) / stages;
            for (int use = 0; go && use < uses; ++use) {
                for (int s = pw; s < stages; s += ST_PRODUCER_WARPS) {
                    const int i = use * stages + s;
                    if (i >= n) { go = false; break; }
                    const int t = lo + i;
                    const uint32_t bar = bar_base + 8 * s;
                    if (use > 0) {
                        if (!st_wait(bar_base + 8 * (ST_MAX_STAGES + s), (uint32_t)((use - 1) & 1), abort_flag)) { go = false; break; }
                        load_weights(t, s);
                    } else if (s >= a.pre) {
                        load_weights(t, s);                                   // ring slots not filled before the wait
                    }
                    if (i < 40) ST_STAMP(56 + i);
                    ptx::mbar_arrive_expect_tx(bar, ACT_BYTES);           // the weight bytes are announced by load_weights
                    ptx::tma_load_3d(smem_base + s * STAGE_BYTES + ST_W_BYTES, &tm_act, 0, 0, (t % sps) * GS, bar);
                }
            }
        }
    } else if (warp < ST_CONSUMER_WARPS) {
        // ----------------------------------------------------------------- consumers ----
        int32_t* asum_s = reinterpret_cast<int32_t*>(smem + L.asum_off);
        for (int i = tid; i < MP * G; i += ST_CONSUMER_WARPS * 32) {
            const int m = i / G, g = i - m * G;
            asum_s[g * MP + m] = (m < a.M) ? __ldcg(a.asum + (size_t)m * G + g) : 0;      // group-major: see the loads
        }
        ptx::named_bar_sync(1, ST_CONSUMER_WARPS * 32);

        // The warp's two units of a stage.  SHARE (strips of 32 rows and more): two 16-row blocks, rows 32 rp ..
        // 32 rp + 31, of ONE group gi - the activation fragments and group sums are loaded once for both.
        // Strips of 16 rows: the one block of groups gi and gi + GS / 2.
        constexpr bool SHARE = RBLK >= 2;
        constexpr int NF = SHARE ? 2 : 1;                    // row blocks a lane accumulates
        constexpr int WPG = SHARE ? RBLK / 2 : 1;            // warps per group
        constexpr int HALF_GS = GS / 2;
        const int gi = warp / WPG, rp = warp % WPG;
        const int r = lane >> 2, j = lane & 3;
        const int row = rp * (SHARE ? 32 : 16) + r;          // first unit's row inside the strip (its second row is + 8)
        // second unit relative to the first, in bytes inside a stage
        constexpr uint32_t U1_NIB = SHARE ? 16 * 64 : HALF_GS * NIB_G, U1_SC = SHARE ? 32 : HALF_GS * SC_G;
        constexpr uint32_t U1_Z = SHARE ? 8 : HALF_GS * Z_G, U1_ACT = SHARE ? 0 : HALF_GS * MP * GROUP;
        constexpr uint32_t U1_ASUM = SHARE ? 0 : HALF_GS * MP * 4;
        // per-lane offsets inside a stage, first unit
        const uint32_t nib_off = gi * NIB_G + row * 64 + blob_chunk_pos(r, j) * 16;   // rows r, r + 8, r + 16, r + 24 share their swizzle
        const uint32_t sc_off = SC_BASE + gi * SC_G + 2 * row;
        const uint32_t z_off = Z_BASE + gi * Z_G + (row >> 1);
        const int zsh = (r & 1) * 4;
        const uint32_t b0_off = ST_W_BYTES + gi * (MP * GROUP) + r * 128 + (((2 * j) ^ r) << 4);   // chunk 2j of the token row; 2j + 1 is ^ 16
        const uint32_t asum_lane = smem_base + L.asum_off + (gi * MP + 2 * j) * 4;
        const uint32_t part_lane = smem_base + L.part_off + (warp * NF * MB * 32 + lane) * 16;
        float facc[NF][MB][4];
#pragma unroll
        for (int f = 0; f < NF; ++f)
#pragma unroll
            for (int mb = 0; mb < MB; ++mb) facc[f][mb][0] = facc[f][mb][1] = facc[f][mb][2] = facc[f][mb][3] = 0.0f;

        bool ok = true;
        int flushed = 0;                                     // strips of this CTA flushed so far
        // the warp's sums over the groups of a strip it met go to shared memory; it starts the next strip at zero
        auto flush = [&]() {
            if (flushed > 0) ok = ok && st_wait(part_empty, (uint32_t)((flushed - 1) & 1), abort_flag);
            if (ok) {
#pragma unroll
                for (int f = 0; f < NF; ++f)
#pragma unroll
                    for (int mb = 0; mb < MB; ++mb) {
                        // the high-nibble chain carried 16 x code: the sums are 16 x D, a power of two taken out here
                        ptx::sts128(part_lane + (f * MB + mb) * 512,
                                    make_float4(facc[f][mb][0] * 0.0625f, facc[f][mb][1] * 0.0625f, facc[f][mb][2] * 0.0625f,
                                                facc[f][mb][3] * 0.0625f));
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
        long long cw = 0, ct0 = 0;
        for (int i = 0; i < n; ++i) {
            const long long c0 = ST_CLK();
            ok = st_wait(full, phase, abort_flag);
            if (!ok) break;
            cw += ST_CLK() - c0;
            if (tid == 0 && i == 0) { ST_STAMP(2); cw = 0; ct0 = ST_CLK(); }
            if (tid == 0 && i < 40) ST_STAMP(16 + i);
#if !defined(ST_ABL) || ST_ABL != 1
            {
                const int g0 = sg * GS + gi, g1 = SHARE ? g0 : g0 + HALF_GS;
                // narrow strips of 16 rows fetch the zero points of 32 rows: the odd strip's are the second half
                const uint32_t zo = stage + z_off + ((R == 16 && (strip & 1)) ? 8 : 0);
                const uint4 wa0 = ptx::lds128(stage + nib_off), wb0 = ptx::lds128(stage + nib_off + 8 * 64);
                const uint4 wa1 = ptx::lds128(stage + nib_off + U1_NIB), wb1 = ptx::lds128(stage + nib_off + U1_NIB + 8 * 64);
                float s_lo0 = __half2float(__ushort_as_half((unsigned short)ptx::lds_u16(stage + sc_off)));
                float s_hi0 = __half2float(__ushort_as_half((unsigned short)ptx::lds_u16(stage + sc_off + 16)));
                float s_lo1 = __half2float(__ushort_as_half((unsigned short)ptx::lds_u16(stage + sc_off + U1_SC)));
                float s_hi1 = __half2float(__ushort_as_half((unsigned short)ptx::lds_u16(stage + sc_off + U1_SC + 16)));
                const int z_lo0 = (ptx::lds_u8(zo) >> zsh) & 0xF, z_hi0 = (ptx::lds_u8(zo + 4) >> zsh) & 0xF;
                const int z_lo1 = (ptx::lds_u8(zo + U1_Z) >> zsh) & 0xF, z_hi1 = (ptx::lds_u8(zo + U1_Z + 4) >> zsh) & 0xF;
                // groups past the end of K (a ragged last stage): whatever the slot holds there must add nothing
                if (g0 >= G) s_lo0 = s_hi0 = 0.0f;
                if (g1 >= G) s_lo1 = s_hi1 = 0.0f;
                const uint32_t asum_g = asum_lane + sg * (GS * MP * 4);
                constexpr uint32_t LO = 0x0F0F0F0Fu, HI = 0xF0F0F0F0u;
#pragma unroll
                for (int mb = 0; mb < MB; ++mb) {
                    // token row 8*mb + r of a group's tile: 128 B, 16-byte chunks XOR-swizzled by the row index
                    const uint32_t ab = stage + b0_off + mb * 1024;
                    const uint4 p0 = ptx::lds128(ab), p1 = ptx::lds128(ab ^ 16u);
                    const uint2 A0 = ptx::lds64(asum_g + mb * 32);                        // the two tokens' group sums
                    uint4 q0 = p0, q1 = p1;
                    uint2 A1 = A0;
                    if (!SHARE) {
                        q0 = ptx::lds128(ab + U1_ACT);
                        q1 = ptx::lds128((ab + U1_ACT) ^ 16u);
                        A1 = ptx::lds64(asum_g + U1_ASUM + mb * 32);
                    }
                    int cl0[4] = {-z_lo0 * (int)A0.x, -z_lo0 * (int)A0.y, -z_hi0 * (int)A0.x, -z_hi0 * (int)A0.y};
                    int cl1[4] = {-z_lo1 * (int)A1.x, -z_lo1 * (int)A1.y, -z_hi1 * (int)A1.x, -z_hi1 * (int)A1.y};
                    int ch0[4], ch1[4];
                    // Words x, y of a packed chunk carry the runs of four k (a0, a2) and (a1, a3) in their (low, high)
                    // nibbles, words z, w the runs (a4, a6) and (a5, a7): the low nibbles of a word pair go with
                    // activation words (0, 1) or (4, 5), the high ones - left in place, i.e. 16 x code - with (2, 3) or (6, 7).
#if defined(ST_ABL) && ST_ABL == 2
                    cl0[0] += wa0.x + p0.x; cl1[0] += wa1.x + q0.x; ch0[0] = ch0[1] = ch0[2] = ch0[3] = wb0.y + p1.y; ch1[0] = ch1[1] = ch1[2] = ch1[3] = wb1.y + q1.y;
#else
                    mma_u8s8(cl0, wa0.x & LO, wb0.x & LO, wa0.y & LO, wb0.y & LO, p0.x, p0.y);
                    mma_u8s8(cl1, wa1.x & LO, wb1.x & LO, wa1.y & LO, wb1.y & LO, q0.x, q0.y);
                    mma_u8s8_z(ch0, wa0.x & HI, wb0.x & HI, wa0.y & HI, wb0.y & HI, p0.z, p0.w);
                    mma_u8s8_z(ch1, wa1.x & HI, wb1.x & HI, wa1.y & HI, wb1.y & HI, q0.z, q0.w);
                    mma_u8s8(cl0, wa0.z & LO, wb0.z & LO, wa0.w & LO, wb0.w & LO, p1.x, p1.y);
                    mma_u8s8(cl1, wa1.z & LO, wb1.z & LO, wa1.w & LO, wb1.w & LO, q1.x, q1.y);
                    mma_u8s8(ch0, wa0.z & HI, wb0.z & HI, wa0.w & HI, wb0.w & HI, p1.z, p1.w);
                    mma_u8s8(ch1, wa1.z & HI, wb1.z & HI, wa1.w & HI, wb1.w & HI, q1.z, q1.w);
#endif
                    const int d00 = (cl0[0] << 4) + ch0[0], d01 = (cl0[1] << 4) + ch0[1];      // 16 x D, exact
                    const int d02 = (cl0[2] << 4) + ch0[2], d03 = (cl0[3] << 4) + ch0[3];
                    const int d10 = (cl1[0] << 4) + ch1[0], d11 = (cl1[1] << 4) + ch1[1];
                    const int d12 = (cl1[2] << 4) + ch1[2], d13 = (cl1[3] << 4) + ch1[3];
                    if (SHARE) {
                        facc[0][mb][0] = fmaf(s_lo0, (float)d00, facc[0][mb][0]);
                        facc[0][mb][1] = fmaf(s_lo0, (float)d01, facc[0][mb][1]);
                        facc[0][mb][2] = fmaf(s_hi0, (float)d02, facc[0][mb][2]);
                        facc[0][mb][3] = fmaf(s_hi0, (float)d03, facc[0][mb][3]);
                        facc[NF - 1][mb][0] = fmaf(s_lo1, (float)d10, facc[NF - 1][mb][0]);
                        facc[NF - 1][mb][1] = fmaf(s_lo1, (float)d11, facc[NF - 1][mb][1]);
                        facc[NF - 1][mb][2] = fmaf(s_hi1, (float)d12, facc[NF - 1][mb][2]);
                        facc[NF - 1][mb][3] = fmaf(s_hi1, (float)d13, facc[NF - 1][mb][3]);
                    } else {
                        // ascending group order within the warp: the earlier group first
                        facc[0][mb][0] = fmaf(s_lo1, (float)d10, fmaf(s_lo0, (float)d00, facc[0][mb][0]));
                        facc[0][mb][1] = fmaf(s_lo1, (float)d11, fmaf(s_lo0, (float)d01, facc[0][mb][1]));
                        facc[0][mb][2] = fmaf(s_hi1, (float)d12, fmaf(s_hi0, (float)d02, facc[0][mb][2]));
                        facc[0][mb][3] = fmaf(s_hi1, (float)d13, fmaf(s_hi0, (float)d03, facc[0][mb][3]));
                    }
                    if (DEBUG) {
                        const int m0 = 8 * mb + 2 * j;
                        const size_t n0 = (size_t)strip * R + row, n1 = SHARE ? n0 + 16 : n0;
                        if (g0 < G) {
                            if (m0 < a.M) {
                                a.debug_partials[((size_t)m0 * G + g0) * a.N + n0] = d00 >> 4;
                                a.debug_partials[((size_t)m0 * G + g0) * a.N + n0 + 8] = d02 >> 4;
                            }
                            if (m0 + 1 < a.M) {
                                a.debug_partials[((size_t)(m0 + 1) * G + g0) * a.N + n0] = d01 >> 4;
                                a.debug_partials[((size_t)(m0 + 1) * G + g0) * a.N + n0 + 8] = d03 >> 4;
                            }
                        }
                        if (g1 < G) {
                            if (m0 < a.M) {
                                a.debug_partials[((size_t)m0 * G + g1) * a.N + n1] = d10 >> 4;
                                a.debug_partials[((size_t)m0 * G + g1) * a.N + n1 + 8] = d12 >> 4;
                            }
                            if (m0 + 1 < a.M) {
                                a.debug_partials[((size_t)(m0 + 1) * G + g1) * a.N + n1] = d11 >> 4;
                                a.debug_partials[((size_t)(m0 + 1) * G + g1) * a.N + n1 + 8] = d13 >> 4;
                            }
                        }
                    }
                }
            }
#endif
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(full + 8 * ST_MAX_STAGES);
            ++s; stage += STAGE_BYTES; full += 8;
            if (s == stages) { s = 0; stage = smem_base; full = bar_base; phase ^= 1; }
            if (++sg == sps) { flush(); sg = 0; ++strip; if (!ok) break; }
        }
        if (tid == 0) { ST_STAMP(3); ST_PUT(10, cw); ST_PUT(11, ST_CLK() - ct0); }
        if (ok && sg != 0) flush();                          // the range ends inside a strip
        if (tid == 0) ST_STAMP(4);
    } else {
        // ------------------------------------------------------------------ epilogue ----
        float* sa_s = reinterpret_cast<float*>(smem + L.sa_off);
        if (lane < MP) sa_s[lane] = lane < a.M ? __half2float(__ushort_as_half(__ldcg(a.sa + lane))) : 0.0f;
        __syncwarp();
        bool ok = true;
        const int r = lane >> 2, j = lane & 3;
        const int nseg = last_strip - first_strip + 1;
        constexpr int ITEMS = RBLK * MB;                          // (16-row block, token block) pairs of a strip
        constexpr int YPITCH = 2 * R + 16;                        // bytes per token row of the staged outputs
        const uint32_t part_lane = smem_base + L.part_off + lane * 16, take_lane = smem_base + L.take_off + lane * 16;
        const uint32_t ystage = smem_base + L.ystage_off;
        // Hand-over words: a float in the low half, the tag 1 in the high half, written and read as one 64-bit
        // word each (no flag, no fence: a word says for itself that it has been written); a lane's four sums of an
        // item are two 16-byte pairs, pair h of item i at ulonglong2 index (2 i + h) * 32 + lane of the CTA's slot.
        constexpr size_t SLOT = (size_t)R * MP * 8;               // a CTA's slot: one 64-bit word per sum of a strip
        ulonglong2* mine = reinterpret_cast<ulonglong2*>(reinterpret_cast<uint8_t*>(a.slots) + (size_t)blockIdx.x * SLOT);
        ulonglong2* theirs = reinterpret_cast<ulonglong2*>(reinterpret_cast<uint8_t*>(a.slots) + (size_t)(blockIdx.x + 1) * SLOT);
        constexpr unsigned long long TAG = 1ull << 32;
        constexpr int HPITCH = R + 16;                            // fused form: bytes per token row of the staged h (R / 2 channels)
        constexpr int FPITCH = 4 * R + 16;                        // with a residual: bytes per token row of the staged fp32 outputs
        uint32_t hmax[MB][2];                                     // fused form: largest |h| (bf16 bits) of this lane's tokens
#pragma unroll
        for (int mb = 0; mb < MB; ++mb) hmax[mb][0] = hmax[mb][1] = 0u;
        for (int q = 0; q < nseg && ok; ++q) {
            const int strip = first_strip + q;
            const bool has_start = lo <= strip * sps, has_end = hi >= (strip + 1) * sps;
            const bool take = has_start && !has_end;       // the neighbour holds the strip's later groups
            if (take) {
                // The neighbour wrote its sums early (they open its range).  Fetch them while the consumers still
                // work on this strip: up to eight 16-byte loads in flight per lane and round trip to L2, retried
                // (bounded) until every word carries its tag; the words are zeroed again for the next call.
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
            // a residual joins at the store: its 16-byte pieces, in the layout of the final stores, are asked for now and
            // have arrived by the time the consumers are done with the strip
            constexpr int RES_CHUNKS = (MP * (R / 8) + 31) / 32;
            uint4 rv[RES_CHUNKS];
            constexpr bool with_res = FUSE == 3;
            if (with_res && has_start) {
#pragma unroll
                for (int k = 0; k < RES_CHUNKS; ++k) {
                    const int c = lane + 32 * k, m = c / (R / 8), col = c - m * (R / 8);
                    rv[k] = make_uint4(0u, 0u, 0u, 0u);
                    if (c < a.M * (R / 8))
                        rv[k] = __ldcg(reinterpret_cast<const uint4*>(a.residual + (size_t)m * a.N + (size_t)strip * R + col * 8));
                }
            }
            ok = st_wait(part_full, (uint32_t)(q & 1), abort_flag);
            if (!ok) break;
            if (lane == 0 && q == nseg - 1) ST_STAMP(5);
#pragma unroll 1
            for (int item = 0; item < ITEMS; ++item) {
                const int rb = item / MB, mb = item % MB;
                float4 acc = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                // the warps that hold this row block, in warp order: deterministic
                constexpr bool SHARE = RBLK >= 2;
                constexpr int WPG = SHARE ? RBLK / 2 : 1, NF = SHARE ? 2 : 1;
#pragma unroll
                for (int gi = 0; gi < ST_CONSUMER_WARPS / WPG; ++gi) {
                    const int w = gi * WPG + (SHARE ? rb / 2 : 0), f = SHARE ? rb % 2 : 0;
                    const float4 v = ptx::lds128f(part_lane + ((w * NF + f) * MB + mb) * 512);
                    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                }
                if (!has_start) {                                  // the strip's earlier groups are the previous CTA's
                    __stcg(mine + (2 * item) * 32 + lane, make_ulonglong2(TAG | __float_as_uint(acc.x), TAG | __float_as_uint(acc.y)));
                    __stcg(mine + (2 * item + 1) * 32 + lane, make_ulonglong2(TAG | __float_as_uint(acc.z), TAG | __float_as_uint(acc.w)));
                    continue;
                }
                if (take) {
                    const float4 o = ptx::lds128f(take_lane + item * 512);
                    acc.x += o.x; acc.y += o.y; acc.z += o.z; acc.w += o.w;      // earlier groups + later groups
                }
                // bf16 outputs into the staging rows: token 8 mb + 2 j (and the next one), channels rb 16 + r and + 8
                const int m0 = 8 * mb + 2 * j;
                const float t0 = sa_s[m0], t1 = sa_s[m0 + 1];
                if (with_res) {
                    // fp32 staging: the rounding comes after the residual has been added
                    const uint32_t fo = ystage + m0 * FPITCH + (rb * 16 + r) * 4;
                    asm volatile("st.shared.f32 [%0], %1;" ::"r"(fo), "f"(acc.x * t0) : "memory");
                    asm volatile("st.shared.f32 [%0], %1;" ::"r"(fo + FPITCH), "f"(acc.y * t1) : "memory");
                    asm volatile("st.shared.f32 [%0], %1;" ::"r"(fo + 32), "f"(acc.z * t0) : "memory");
                    asm volatile("st.shared.f32 [%0], %1;" ::"r"(fo + FPITCH + 32), "f"(acc.w * t1) : "memory");
                    continue;
                }
                const uint32_t yo = ystage + m0 * YPITCH + (rb * 16 + r) * 2;
                const __nv_bfloat16 o0 = __float2bfloat16_rn(acc.x * t0), o1 = __float2bfloat16_rn(acc.y * t1);
                const __nv_bfloat16 o2 = __float2bfloat16_rn(acc.z * t0), o3 = __float2bfloat16_rn(acc.w * t1);
                if (SILU) {
                    // (o0, o2) = (gate, up) of channel 8 rb + r for token m0, (o1, o3) for token m0 + 1
                    const uint32_t h0 = silu_mul_bf16_bits(__bfloat162float(o0), __bfloat162float(o2));
                    const uint32_t h1 = silu_mul_bf16_bits(__bfloat162float(o1), __bfloat162float(o3));
                    hmax[mb][0] = max(hmax[mb][0], h0 & 0x7FFFu);
                    hmax[mb][1] = max(hmax[mb][1], h1 & 0x7FFFu);
                    const uint32_t ho = ystage + m0 * HPITCH + (rb * 8 + r) * 2;
                    asm volatile("st.shared.u16 [%0], %1;" ::"r"(ho), "h"((unsigned short)h0) : "memory");
                    asm volatile("st.shared.u16 [%0], %1;" ::"r"(ho + HPITCH), "h"((unsigned short)h1) : "memory");
                    continue;
                }
                asm volatile("st.shared.u16 [%0], %1;" ::"r"(yo), "h"(__bfloat16_as_ushort(o0)) : "memory");
                asm volatile("st.shared.u16 [%0], %1;" ::"r"(yo + YPITCH), "h"(__bfloat16_as_ushort(o1)) : "memory");
                asm volatile("st.shared.u16 [%0], %1;" ::"r"(yo + 16), "h"(__bfloat16_as_ushort(o2)) : "memory");
                asm volatile("st.shared.u16 [%0], %1;" ::"r"(yo + YPITCH + 16), "h"(__bfloat16_as_ushort(o3)) : "memory");
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(part_empty);
            if (has_start && with_res) {
                constexpr int CPR = R / 8;
#pragma unroll
                for (int k = 0; k < RES_CHUNKS; ++k) {
                    const int c = lane + 32 * k, m = c / CPR, col = c - m * CPR;
                    if (c < a.M * CPR) {
                        const float4 f0 = ptx::lds128f(ystage + m * FPITCH + col * 32), f1 = ptx::lds128f(ystage + m * FPITCH + col * 32 + 16);
                        const uint4 rr = rv[k];
                        uint4 v;
                        __nv_bfloat162 b;
                        b = __floats2bfloat162_rn(f0.x + __uint_as_float(rr.x << 16), f0.y + __uint_as_float(rr.x & 0xFFFF0000u));
                        v.x = *reinterpret_cast<uint32_t*>(&b);
                        b = __floats2bfloat162_rn(f0.z + __uint_as_float(rr.y << 16), f0.w + __uint_as_float(rr.y & 0xFFFF0000u));
                        v.y = *reinterpret_cast<uint32_t*>(&b);
                        b = __floats2bfloat162_rn(f1.x + __uint_as_float(rr.z << 16), f1.y + __uint_as_float(rr.z & 0xFFFF0000u));
                        v.z = *reinterpret_cast<uint32_t*>(&b);
                        b = __floats2bfloat162_rn(f1.z + __uint_as_float(rr.w << 16), f1.w + __uint_as_float(rr.w & 0xFFFF0000u));
                        v.w = *reinterpret_cast<uint32_t*>(&b);
                        *reinterpret_cast<uint4*>(a.y + (size_t)m * a.N + (size_t)strip * R + col * 8) = v;
                    }
                }
                __syncwarp();
            }
            if (has_start && FUSE == 0) {
                // the strip leaves in 16-byte pieces: R / 8 per token row
                constexpr int CPR = R / 8;
                for (int c = lane; c < a.M * CPR; c += 32) {
                    const int m = c / CPR, col = c - m * CPR;
                    const uint4 v = ptx::lds128(ystage + m * YPITCH + col * 16);
                    *reinterpret_cast<uint4*>(a.y + (size_t)m * a.N + (size_t)strip * R + col * 8) = v;
                }
                __syncwarp();
            }
            if (has_start && SILU) {
                // the strip's R / 2 channels of h, 16-byte pieces
                constexpr int CPR = R / 16;
                const int I = a.N / 2;
                for (int c = lane; c < a.M * CPR; c += 32) {
                    const int m = c / CPR, col = c - m * CPR;
                    const uint4 v = ptx::lds128(ystage + m * HPITCH + col * 16);
                    *reinterpret_cast<uint4*>(a.h + (size_t)m * I + (size_t)strip * (R / 2) + col * 8) = v;
                }
                __syncwarp();
            }
        }
        if (SILU) {
            // largest |h| per token over this CTA's strips: lanes of equal j hold the same two tokens
#pragma unroll
            for (int mb = 0; mb < MB; ++mb)
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    uint32_t v = hmax[mb][t];
                    v = max(v, __shfl_xor_sync(0xFFFFFFFFu, v, 4));
                    v = max(v, __shfl_xor_sync(0xFFFFFFFFu, v, 8));
                    v = max(v, __shfl_xor_sync(0xFFFFFFFFu, v, 16));
                    const int m = 8 * mb + 2 * j + t;
                    if (r == 0 && m < a.M && v != 0u) atomicMax(a.sync + m, v);
                }
            __syncwarp();                                      // the lanes' stores of h and maxima, then one release
            // one-kernel form: the CTA's place in the order of arrival decides whether it stays for the requantisation
            if (FUSE == 1 && lane == 0) {
                uint32_t place;
                asm volatile("atom.add.release.gpu.global.u32 %0, [%1], 1;" : "=r"(place) : "l"(a.sync + 16) : "memory");
                *reinterpret_cast<volatile uint32_t*>(smem + L.misc_off + 4) = place;
            }
        }
        if (lane == 0) ST_STAMP(6);
    }
    __syncwarp();
    if (FUSE == 1) {
        // ---- the last CTAs to arrive wait for the rest and requantise h; the others leave at once ----
        // (a CTA that leaves frees its place for the next kernel's CTAs, which start their weight stream under this
        // kernel's tail; a stayer waits only for CTAs that run or will run whether it holds its place or not, so the
        // grid need not be resident as a whole)
        __syncthreads();
        const uint32_t stay = gridDim.x < ST_STAY ? gridDim.x : ST_STAY;
        const uint32_t place = *reinterpret_cast<volatile uint32_t*>(smem + L.misc_off + 4);
        if (tid == 0) { ST_STAMP(7); ST_PUT(12, place); }
        if (place >= gridDim.x - stay) {
            const uint32_t rank = place - (gridDim.x - stay);
            if (tid == 0) {
                uint64_t t0 = 0;
                for (uint32_t spin = 0; !*abort_flag; ++spin) {
                    uint32_t v;
                    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(a.sync + 16) : "memory");
                    if (v >= gridDim.x) break;
                    if ((spin & 15) == 15) {
                        const uint64_t now = ptx::globaltimer_ns();
                        if (t0 == 0) t0 = now;
                        else if (now - t0 > ptx::WAIT_LIMIT_NS) { *abort_flag = 1; break; }
                    }
                }
                __threadfence();
                ST_STAMP(8);
            }
            __syncthreads();
            if (!*abort_flag) {
                const int I = a.N / 2, Gh = I / GROUP;
                constexpr int WARPS = ST_THREADS / 32;
                for (int u = (int)rank * WARPS + warp; u < a.M * Gh; u += (int)stay * WARPS)
                    requant_unit(a.h, I, Gh, u, lane, a.qa_h, a.sa_h, a.asum_h, a.sync);
            }
            __syncthreads();
            // the last stayer to leave puts the words back to zero for the next call
            if (tid == 0) ST_STAMP(9);
            if (tid == 0) {
                const uint32_t old = atomicAdd(a.sync + 17, 1u);
                if (old == stay - 1) {
                    for (int i = 0; i < 18; ++i) a.sync[i] = 0u;
                    __threadfence();
                }
                ST_STAMP(13);
            }
        }
    }
    if (*abort_flag) {
        if (lane == 0) atomicExch(a.status, (uint32_t)W4A8_ERR_TIMEOUT);
        // copies that were requested may still be in flight: give them a bounded time to land before the
        // shared memory is handed back
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
}

// The quantisation of h after the gate+up kernel in its two-kernel form: one (token, group of 128) per warp, the
// token's scale from its final maximum.  The last CTA to finish puts the maxima back to zero for the next call.
__global__ void __launch_bounds__(256) requant_kernel(const __nv_bfloat16* __restrict__ h, int M, int I, int8_t* __restrict__ qa_h,
                                                      uint16_t* __restrict__ sa_h, int32_t* __restrict__ asum_h, uint32_t* sync) {
    ptx::pdl_launch_dependents();
    ptx::pdl_wait();
    const int Gh = I / GROUP, lane = threadIdx.x & 31;
    const int u = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (u < M * Gh) requant_unit(h, I, Gh, u, lane, qa_h, sa_h, asum_h, sync);
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const uint32_t old = atomicAdd(sync + 17, 1u);
        if (old == gridDim.x - 1) {
            for (int i = 0; i < 18; ++i) sync[i] = 0u;
            __threadfence();
        }
    }
}

struct FuseOut {
    void* h;
    int8_t* qa_h;
    uint16_t* sa_h;
    int32_t* asum_h;
    bool one_kernel;
};

template <int MB, int RBLK, bool DEBUG, int FUSE>
cudaError_t launch_strip(const int8_t* qa, const uint16_t* sa, const int32_t* asum, const void* packed, void* y,
                         const void* residual, int M, int N, int K, int ctas, void* workspace, int32_t* debug_partials,
                         const FuseOut* fuse, cudaStream_t stream) {
    constexpr int R = 16 * RBLK, GS = ST_UNITS / RBLK, MP = 8 * MB;
    const int G = K / GROUP;
    const bool fp32_stage = FUSE == 3;
    const int fixed = st_layout(MB, RBLK, 0, G, fp32_stage).total + 1024;
    int stages = (ST_SMEM_BUDGET - fixed) / st_stage_bytes(MB, RBLK);
    if (stages > ST_MAX_STAGES) stages = ST_MAX_STAGES;
    if (stages < 2) return cudaErrorInvalidConfiguration;
    const size_t smem = (size_t)st_layout(MB, RBLK, stages, G, fp32_stage).total + 1024;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    static bool attr_done[64] = {false};
    static int resident[64] = {0};                          // CTAs of this instance that fit on the device at once
    if (!attr_done[dev]) {
        e = cudaFuncSetAttribute(gemm_strip_kernel<MB, RBLK, DEBUG, FUSE>, cudaFuncAttributeMaxDynamicSharedMemorySize, ST_SMEM_BUDGET);
        if (e != cudaSuccess) return e;
        int per_sm = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, gemm_strip_kernel<MB, RBLK, DEBUG, FUSE>, ST_THREADS, ST_SMEM_BUDGET);
        if (e != cudaSuccess) return e;
        resident[dev] = per_sm * device_sm_count();
        attr_done[dev] = true;
    }
    if (FUSE == 1) {
        // keep the grid within what is resident at once: the stayers then never wait for a CTA that has yet to start
        if (resident[dev] < 1) return cudaErrorInvalidConfiguration;
        if (ctas > resident[dev]) ctas = resident[dev];
    }
    CUtensorMap tm_act, tm_nib, tm_scale, tm_zero;
    e = make_qa_group_map(&tm_act, qa, M, K, MP, GS);
    if (e != cudaSuccess) return e;
    e = make_strip_weight_maps(&tm_nib, &tm_scale, &tm_zero, packed, N, K, R, GS);
    if (e != cudaSuccess) return e;

    uint8_t* ws = static_cast<uint8_t*>(workspace);
    StripArgs a;
    a.sa = sa;
    a.asum = asum;
    a.packed = static_cast<const uint8_t*>(packed);
    a.y = static_cast<__nv_bfloat16*>(y);
    a.M = M; a.N = N; a.K = K;
    a.stages = stages;
    a.pre = stages;
#ifdef W4A8_TUNING
    if (const char* e = getenv("W4A8_STRIP_PRE")) { const int v = atoi(e); if (v >= 1 && v < stages) a.pre = v; }
#endif
    a.sps = (G + GS - 1) / GS;
    a.total_stages = (N / R) * a.sps;
    a.status = reinterpret_cast<uint32_t*>(ws + WS_STATUS_OFF);
    a.slots = reinterpret_cast<unsigned long long*>(ws + WS_HEADER_BYTES);
    a.debug_partials = debug_partials;
    a.residual = static_cast<const __nv_bfloat16*>(residual);
    a.h = fuse ? static_cast<__nv_bfloat16*>(fuse->h) : nullptr;
    a.qa_h = fuse ? fuse->qa_h : nullptr;
    a.sa_h = fuse ? fuse->sa_h : nullptr;
    a.asum_h = fuse ? fuse->asum_h : nullptr;
    a.sync = reinterpret_cast<uint32_t*>(ws + WS_FUSE_SYNC_OFF);

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctas, 1, 1);
    cfg.blockDim = dim3(ST_THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attrs[1];
    attrs[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attrs;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, gemm_strip_kernel<MB, RBLK, DEBUG, FUSE>, tm_act, tm_nib, tm_scale, tm_zero, a);
    if (e != cudaSuccess || FUSE != 2) return e;
    // two-kernel form: the requantisation once every maximum is final
    const int units = M * (N / 2 / GROUP);
    cfg.gridDim = dim3((unsigned)((units + 7) / 8), 1, 1);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.dynamicSmemBytes = 0;
    return cudaLaunchKernelEx(&cfg, requant_kernel, (const __nv_bfloat16*)a.h, M, N / 2, a.qa_h, a.sa_h, a.asum_h, a.sync);
}

template <int MB, int RBLK>
cudaError_t launch_strip_dbg(const int8_t* qa, const uint16_t* sa, const int32_t* asum, const void* packed, void* y,
                             const void* residual, int M, int N, int K, int ctas, void* workspace, int32_t* debug_partials, const FuseOut* fuse,
                             cudaStream_t stream) {
    if (fuse) {
        // two token blocks always run on 32-row strips (strip_plan): the other widths are not built in the fused form
        if constexpr (MB == 2 && RBLK != 2) return cudaErrorInvalidConfiguration;
        else if (fuse->one_kernel)
            return launch_strip<MB, RBLK, false, 1>(qa, sa, asum, packed, nullptr, nullptr, M, N, K, ctas, workspace, nullptr, fuse, stream);
        else
            return launch_strip<MB, RBLK, false, 2>(qa, sa, asum, packed, nullptr, nullptr, M, N, K, ctas, workspace, nullptr, fuse, stream);
    }
    if (residual) {                                      // its own instantiation: the plain kernel's epilogue stays as small as it was
        if constexpr (MB == 2 && RBLK != 2) return cudaErrorInvalidConfiguration;
        else return launch_strip<MB, RBLK, false, 3>(qa, sa, asum, packed, y, residual, M, N, K, ctas, workspace, nullptr, nullptr, stream);
    }
    if (debug_partials)
        return launch_strip<MB, RBLK, true, 0>(qa, sa, asum, packed, y, nullptr, M, N, K, ctas, workspace, debug_partials, nullptr, stream);
    return launch_strip<MB, RBLK, false, 0>(qa, sa, asum, packed, y, nullptr, M, N, K, ctas, workspace, nullptr, nullptr, stream);
}

}  // namespace

#ifdef W4A8_TRACE
extern "C" int w4a8_strip_trace_read(unsigned long long* host_out, unsigned int* host_counts) {
    if (cudaMemcpyFromSymbol(host_out, g_strip_trace, sizeof(unsigned long long) * 64 * 320 * 96) != cudaSuccess) return 1;
    if (cudaMemcpyFromSymbol(host_counts, g_strip_trace_count, sizeof(unsigned int) * 320) != cudaSuccess) return 2;
    return 0;
}
#endif

bool strip_supported(int M, int N, int K) {
    const int mp = M <= 8 ? 8 : 16;
    return M >= 1 && M <= STRIP_MAX_M && (K / GROUP) * mp <= ST_MAX_ASUM_WORDS && N >= 16;
}

// Strip width and CTA count for a problem (measured on B200, sweep of widths 16..128 and 148..296 CTAs on the
// four layer shapes of an 8B-class decoder, 4 to 16 tokens): the widest strip that still gives about 1.25 strips
// per SM (one step narrower if a wide strip would leave SMs with a single CTA), and up to two CTAs per SM - the second CTA's warps multiply while the first one's wait for data, which is
// worth more than a whole SM's shared memory held free for the next launch; the next launch's CTAs still start
// (and prefetch) as soon as the first CTAs of this one leave.  Wide strips share an activation tile between more
// rows (less traffic from L2 into shared memory); 16-row strips are left to up to 8 tokens, where their 16
// activation tiles per stage still leave room for a ring.  The grid never exceeds the number of strips, so that a
// strip is shared by at most two CTAs.
void strip_plan(int M, int N, int K, int* strip_rows, int* ctas) {
    (void)K;
    const int sms = device_sm_count();
    int R = 128;
    if (M <= 8) {
        while (R > 16 && N / R < (sms * 5) / 4) R /= 2;
        if (R > 32 && N / R < 2 * sms) R /= 2;               // wide strips: enough of them for two CTAs on every SM
    } else {
        R = 32;                                              // two token blocks: 32-row strips measured best (wider: fewer CTAs or more
    }                                                        // hand-over; narrower: the activation tiles crowd the ring)
#ifdef W4A8_TUNING
    if (const char* e = getenv("W4A8_STRIP_R")) {
        const int v = atoi(e);
        if (v == 16 || v == 32 || v == 64 || v == 128) R = v;
    }
#endif
    int limit = ST_MINB * sms;
#ifdef W4A8_TUNING
    if (const char* e = getenv("W4A8_STRIP_CTAS")) { const int v = atoi(e); if (v >= 1) limit = v; }
#endif
    const int slot_limit = (STRIP_MAX_CTAS * STRIP_SLOT_BYTES) / (R * (M <= 8 ? 8 : 16) * 8);    // hand-over slots in the workspace
    if (limit > slot_limit) limit = slot_limit;
    int c = N / R;
    if (c > limit) c = limit;
    if (strip_rows) *strip_rows = R;
    if (ctas) *ctas = c;
}

namespace {
cudaError_t strip_dispatch(const int8_t* qa, const uint16_t* sa, const int32_t* asum, const void* packed,
                           void* y, const void* residual, int M, int N, int K, void* workspace, int32_t* debug_partials, const FuseOut* fuse,
                           cudaStream_t stream) {
    int R = 0, ctas = 0;
    strip_plan(M, N, K, &R, &ctas);
#define W4A8_STRIP_CASE(MBV, RBV) \
    return launch_strip_dbg<MBV, RBV>(qa, sa, asum, packed, y, residual, M, N, K, ctas, workspace, debug_partials, fuse, stream)
    if (M <= 8) {
        if (R == 128) W4A8_STRIP_CASE(1, 8);
        if (R == 64) W4A8_STRIP_CASE(1, 4);
        if (R == 32) W4A8_STRIP_CASE(1, 2);
        W4A8_STRIP_CASE(1, 1);
    }
    if (R == 128) W4A8_STRIP_CASE(2, 8);
    if (R == 64) W4A8_STRIP_CASE(2, 4);
    if (R == 32) W4A8_STRIP_CASE(2, 2);
    W4A8_STRIP_CASE(2, 1);
#undef W4A8_STRIP_CASE
}
}  // namespace

cudaError_t launch_gemm_strip(const int8_t* qa, const uint16_t* sa, const int32_t* asum, const void* packed,
                              void* y, const void* residual, int M, int N, int K, void* workspace, int32_t* debug_partials,
                              cudaStream_t stream) {
    return strip_dispatch(qa, sa, asum, packed, y, residual, M, N, K, workspace, debug_partials, nullptr, stream);
}

// The fused gate+up form: packed = the 2 I = N channels in runs of eight gate / eight up; outputs h [M, I] bf16 and the
// quantised input of the down projection (codes, token scales, group sums).  I must be a multiple of 128.
cudaError_t launch_gemm_strip_gate_up(const int8_t* qa, const uint16_t* sa, const int32_t* asum, const void* packed,
                                      int M, int N, int K, void* h, int8_t* qa_h, uint16_t* sa_h, int32_t* asum_h,
                                      bool one_kernel, void* workspace, cudaStream_t stream) {
    const FuseOut f = {h, qa_h, sa_h, asum_h, one_kernel};
    return strip_dispatch(qa, sa, asum, packed, nullptr, nullptr, M, N, K, workspace, nullptr, &f, stream);
}

}  // namespace w4a8
