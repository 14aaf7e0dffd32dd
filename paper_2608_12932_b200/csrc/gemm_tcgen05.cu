// Large-M W4A8 GEMM for sm_100a: bulk copies -> shared memory -> int4->int8 unpack into TENSOR
// MEMORY -> tcgen05.mma kind::i8 (weights from TMEM, activations from shared memory) with int32
// accumulators in TMEM -> per-group fp32 scaling -> bf16.
// (Sec. 3.4: quantising the activations to 8 bits is what lets the compute-bound prefill run on
// INT8 tensor cores; Sec. 4: prefill is one long matrix multiplication.)
//
// Orientation ("swap-AB"): the 128 output channels of a tile are the MMA's M side (TMEM lanes),
// the tokens are its N side (TMEM columns).  A drain thread therefore owns ONE output channel:
// its group scale is a per-thread scalar and the per-group work on the CUDA cores is one
// int->float convert and one FMA per accumulator element.
//
// One pipeline step = one quantisation group = 128 k = four K=32 MMAs; the accumulator must be
// drained after every group because the scale changes, so TMEM holds two accumulator buffers:
// the tensor core fills one while the drain warps empty the other.  The first MMA of a group
// overwrites its buffer, so a buffer needs no preparation: the drain hands it back as soon as
// its columns are in registers.
//
// The tensor pipe is not what bounds this kernel (it is busy under a third of the time): the CUDA
// cores must take every accumulator element out of TMEM after every group and spend two
// instructions on it, the unpack shares the integer pipe with that conversion, and shared memory
// (about 128 B/clk per SM) is shared by the tensor core's operand reads, the bulk-copy fills and
// ordinary loads.  Design choices made on measurements:
//  * the unpacked weights never touch shared memory: an unpack thread owns one weight row
//    (= one TMEM lane), converts its 64 packed bytes in registers and writes the 128 signed
//    bytes to 32 TMEM columns with tcgen05.st; the MMA takes its A operand from TMEM.  That
//    removes a 16 KB store and a 16 KB operand read per group from shared memory;
//  * the token tile is 208 rows, not 256: two accumulator buffers of 208 columns plus three
//    32-column weight stages fill the 512 TMEM columns exactly, and M = 1024 or 4096 splits
//    into 208-row tiles with 1.5 % padding;
//  * there is no accumulator bias / re-arm (which would turn the int->float conversion into an
//    FMA-pipe add): tcgen05.st traffic to TMEM costs as much port time as tcgen05.ld traffic, more
//    than the conversion;
//  * two warps issue the MMAs, one for the even and one for the odd steps (a step costs its issuer
//    three barrier waits, four MMAs and a commit); the whole warp walks the loop and an elected lane
//    issues, which keeps the MMA operands in uniform registers (from inside a one-lane branch every
//    MMA cost its thread about a hundred cycles of register-to-uniform moves);
//  * one tcgen05.commit per step, on a ring of "step done" barriers, frees the step's weight and
//    activation stages and publishes its accumulator.
//
// Zero points are subtracted while unpacking (weights become signed, -15..15), so the int32
// accumulator is directly D = sum (q_w - z) q_a; identical to P - z*sum(q_a), and it moves the
// correction from the per-(token, channel, group) drain to the per-weight unpack.
//
// Warp roles (512 threads, four warpgroups so that setmaxnreg can move registers to the drain:
// 40 / 40 / 216 / 216 per thread for 208-row tiles, 40 / 96 / 160 / 160 for shorter ones):
//   warp 0       producer of the activation tiles (2-D TMA loads)
//   warps 1, 3   MMA issuers (even and odd pipeline steps; an elected lane issues); warp 1 owns TMEM allocation
//   warp 2       producer of the packed blobs (1-D bulk copies)
//   warps 4-7    unpack: raw blob -> signed int8 weight rows in TMEM
//   warps 8-15   drain: tcgen05.ld -> convert -> FMA with the group scale; final bf16 store
//
// Split-K variant (SPLIT): when an [M, N] problem has fewer tiles than half the SMs, a tile is given
// to a thread-block cluster of S CTAs, each walking G / S of the K groups (a CTA's time is close to
// proportional to its number of groups, whatever the tile height).  The fp32 partials are reduced
// like the small-M kernel's: after a cluster barrier (every CTA has finished its MMAs, so the
// activation ring is free) each drain thread pushes its partials with st.shared::cluster into the
// ring area of the CTA that owns that share of the tile (slot = pusher's rank), a second cluster
// barrier, and the owner sums its S slots in rank order, applies the token scale and stores bf16.
// (Pushing 16 bytes at a time into a channel-major buffer was measured slightly slower.)
// Every wait is bounded; on expiry the CTA records W4A8_ERR_TIMEOUT, frees TMEM and exits.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include "ptx_sm100.cuh"
#include "w4a8_internal.cuh"

namespace w4a8 {
namespace {

constexpr int TC_THREADS = 512;
constexpr int WARP_PRODUCER = 0, WARP_MMA = 1, WARP_RAW_PRODUCER = 2, WARP_MMA_ODD = 3, WARP_UNPACK0 = 4, WARP_DRAIN0 = 8;
constexpr int DONE_RING = 8;                     // "group finished" barriers; every role stays within 8 groups of the others
constexpr int NUM_UNPACK_WARPS = 4, NUM_DRAIN_WARPS = 8;
constexpr int RAW_STRIDE = 8576;                 // BLOB_BYTES rounded up to a multiple of 128
constexpr int A_COLS = GROUP / 4;                // 32 TMEM columns hold one group of a weight row (4 bytes per column)
constexpr int TMEM_COLS = 512;
// cost model of tcgen05_plan (nanoseconds, measured): per launch; per group of a 208-, 128-, 64-row tile; for splitting K
// (cluster launch, two cluster barriers, exchange and reduction of a 208-, 128-, 64-row tile)
constexpr long TC_FIXED_NS = 4000, TC_GROUP_NS[3] = {650, 540, 440}, TC_SPLIT_NS[3] = {10000, 7000, 4000};
constexpr int TC_MAX_SPLIT = 4;
// balanced walk: hand-over of two partial tiles (208-, 128-, 64-row) and a slower pipeline around them
constexpr long TC_BALANCE_NS[3] = {12000, 8000, 5000};

// Shared-memory rings.  The activation tile comes from L2 through TMA with a latency of roughly
// 2000 cycles, the packed blob from HBM likewise: both rings are deep enough to cover it.
template <int TILE_M>
struct Cfg {
    static constexpr int B_BYTES = TILE_M * GROUP;                            // one activation stage
    static constexpr int SB = TILE_M > 128 ? 5 : (TILE_M == 128 ? 6 : 8);     // activation stages
    static constexpr int SR = TILE_M > 128 ? 8 : (TILE_M == 128 ? 12 : 16);   // packed-blob stages: a short tile finishes a group
                                                                              // quickly, so more blobs must be in flight to cover HBM latency
// (four accumulator buffers at 64-row tiles, where tensor memory has the room, -DTC_NB64=4: same results, 0.5-2 % faster
// - the MMA -> drain -> MMA round trip of a buffer is not what bounds the short-tile step)
#ifndef TC_NB64
#define TC_NB64 2
#endif
    static constexpr int NB = TILE_M == 64 ? TC_NB64 : 2;                      // accumulator buffers in flight
    static constexpr int SA_MAX = (TMEM_COLS - NB * TILE_M) / A_COLS;
    static constexpr int SA = SA_MAX > 4 ? 4 : SA_MAX;                        // weight stages in TMEM
    static constexpr int A_COL0 = NB * TILE_M;                                // first weight column (after the accumulators)
    static constexpr int B_OFF = 0;
    static constexpr int RAW_OFF = B_OFF + SB * B_BYTES;
    static constexpr int BAR_OFF = RAW_OFF + SR * RAW_STRIDE;
    static constexpr int NUM_BARS = 2 * SR + SB + SA + 4 + DONE_RING + 2 + 2;
    static constexpr int MISC_OFF = (BAR_OFF + NUM_BARS * 8 + 15) & ~15;      // 16-byte aligned: staging is read with 16-byte loads
    static constexpr int W = TILE_M / 2;                                      // accumulator columns (tokens) per drain warp
    static constexpr int NCH = (W + 31) / 32;                                 // 32-column chunks per drain warp (the last may be 8 wide)
    static constexpr int LAST = W - 32 * (NCH - 1);                           // width of the last chunk
    static constexpr int SA_OFF = MISC_OFF + 16;   // per drain warp: token scales as fp32
    static constexpr int OUT_OFF = (SA_OFF + NUM_DRAIN_WARPS * NCH * 32 * 4 + 127) & ~127;   // per drain warp: 32 tokens x 32 channels bf16 (TMA source: 128-byte aligned)
    static constexpr int SMEM_BYTES = OUT_OFF + NUM_DRAIN_WARPS * 2048;
    static constexpr int SMEM_ALLOC = SMEM_BYTES + 1024;       // slack to align the base to 1024 B
    static_assert(TILE_M == 64 || TILE_M == 128 || TILE_M == 208, "token tile");
    static_assert(TILE_M % 16 == 0, "MMA N granularity; 8-row swizzle atoms");
    static_assert(LAST == 32 || LAST == 8, "chunk widths the drain knows how to load");
    static_assert(SA >= 2 && A_COL0 + SA * A_COLS <= TMEM_COLS, "tensor memory");
    static_assert(SB <= DONE_RING && SA <= DONE_RING, "a stage is freed by the group that used it, at most DONE_RING groups ago");
    static_assert(SMEM_ALLOC <= 227 * 1024, "shared memory");
    static_assert(OUT_OFF % 128 == 0 && SA_OFF % 16 == 0 && B_BYTES % 1024 == 0, "alignment");
};

__device__ __forceinline__ uint32_t sub_zero4(uint32_t q, uint32_t kz) {
    // bytes of q in 0..15, bytes of kz = 0x80 - z with z in 0..15: per byte (q + 0x80 - z) ^ 0x80
    // is q - z as a signed int8; no carry crosses a byte (0x71 <= q + 0x80 - z <= 0x8F).  (The per-byte subtract
    // intrinsic __vsub4 in its place was measured 7-10 % slower on the whole kernel: it is not one instruction here.)
    return (q + kz) ^ 0x80808080u;
}

// PC ("per channel"): the scales of a channel are the same in every group, so the integer sums of all
// groups of a tile add up in one accumulator and the tile is drained once (see w4a8_gemm_per_channel).
// BAL: balanced walk (see `segment` below).
// RES: the epilogue adds a residual (its own instantiations: the extra registers of the residual block would
// otherwise spill in the plain kernels).
template <int TILE_M, bool DEBUG, bool SPLIT, bool PC = false, bool BAL = false, bool RES = false>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_qa, const __grid_constant__ CUtensorMap tmap_y,
                    const uint8_t* __restrict__ packed,
                    const uint16_t* __restrict__ sa, __nv_bfloat16* y, const __nv_bfloat16* residual,
                    int32_t* __restrict__ debug_partials, uint32_t* __restrict__ status,
                    int M, int N, int K, int m_tiles, int total_tiles, int S,
                    float* __restrict__ handover, uint32_t* __restrict__ handover_flags) {
    // Programmatic dependent launch: the kernel after this one may start its prologue now; this one sets up tensor
    // memory, barriers and its weight stream (weights never depend on the previous kernel) while its predecessor may
    // still run, and the roles that touch activations, token scales, the workspace or the output wait below.
    ptx::pdl_launch_dependents();
    using C = Cfg<TILE_M>;
    static_assert(!SPLIT || C::SB * C::B_BYTES >= TILE_M * TILE_N * 4 + 64, "the split-K exchange buffer lives in the activation ring");
    static_assert(!(SPLIT && PC), "the per-channel form is not split along K");
    static_assert(!BAL || (!SPLIT && !PC), "the balanced walk is for the plain persistent form");
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    const int GK = K / GROUP;                                   // groups of the whole K range (blob and output indexing)
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // SPLIT: a cluster of S CTAs per tile (one tile per cluster, no persistence); this CTA walks groups [g_lo, g_lo + G)
    const int slice = SPLIT ? (int)ptx::cluster_ctarank() : 0;
    const int unit = SPLIT ? (int)blockIdx.x / S : (int)blockIdx.x;
    const int num_units = SPLIT ? (int)gridDim.x / S : (int)gridDim.x;
    const int g_lo = SPLIT ? (int)(((long long)slice * GK) / S) : 0;
    const int G = SPLIT ? (int)(((long long)(slice + 1) * GK) / S) - g_lo : GK;

    auto bar = [&](int i) { return smem_base + C::BAR_OFF + 8 * i; };
    // DONE[j % DONE_RING] completes its phase j / DONE_RING when the MMAs of pipeline step j have finished: that
    // one event frees the step's weight stage (unpack warps wait for step it - SA), its activation
    // stage (producer waits for step it - SB) and publishes its accumulator (drain warps wait for it).
    const int RAW_FULL = 0, RAW_EMPTY = C::SR, B_FULL = 2 * C::SR, A_FULL = B_FULL + C::SB, ACC_EMPTY = A_FULL + C::SA,
              DONE = ACC_EMPTY + 4, FINAL = DONE + DONE_RING, TILE_DONE = FINAL + 2;
    auto done_bar = [&](uint32_t step) { return bar(DONE + (int)(step % DONE_RING)); };
    auto done_parity = [](uint32_t step) { return (step / DONE_RING) & 1u; };
    volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(smem + C::MISC_OFF);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + C::MISC_OFF + 4);

    if (warp == WARP_MMA) {
        if (lane == 0) {
            *abort_flag = 0;
            for (int i = 0; i < C::SR; ++i) {
                ptx::mbar_init(bar(RAW_FULL + i), 1);
                ptx::mbar_init(bar(RAW_EMPTY + i), NUM_UNPACK_WARPS);
            }
            for (int i = 0; i < C::SB; ++i) ptx::mbar_init(bar(B_FULL + i), 1);
            for (int i = 0; i < C::SA; ++i) ptx::mbar_init(bar(A_FULL + i), NUM_UNPACK_WARPS);
            for (int i = 0; i < 4; ++i) ptx::mbar_init(bar(ACC_EMPTY + i), NUM_DRAIN_WARPS);
            for (int i = 0; i < DONE_RING; ++i) ptx::mbar_init(bar(DONE + i), 1);
            for (int i = 0; i < 2; ++i) ptx::mbar_init(bar(FINAL + i), 1);
            for (int i = 0; i < 2; ++i) ptx::mbar_init(bar(TILE_DONE + i), 2);      // both MMA issuers
            ptx::fence_mbar_init();
        }
        __syncwarp();
        ptx::tmem_alloc(smem_base + C::MISC_OFF, TMEM_COLS);
        ptx::tmem_relinquish();
    }
    if (warp == WARP_PRODUCER && lane == 0) ptx::prefetch_tmap(&tmap_qa);
    if (warp == WARP_DRAIN0 && lane == 0) ptx::prefetch_tmap(&tmap_y);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_holder;
    // tile of iteration t of this CTA: channel tile and token tile
    auto tile_of = [&](int t, int& ntile, int& mtile) {
        ntile = t / m_tiles;
        mtile = t % m_tiles;
    };

    // The work of a CTA as a list of segments (tile, groups [gb, ge) of it).  Plain persistent walk: whole
    // tiles unit, unit + num_units, ...  Balanced walk (more tiles than CTAs): the tiles x groups units are
    // dealt out in equal contiguous ranges, so a CTA's first and last segment may be part of a tile; the CTA
    // that holds the later groups of such a tile reaches them first (they open its range) and hands its
    // fp32 sums over through global memory to the CTA that holds the earlier groups (they close its range).
    const long bal_lo = BAL ? ((long)blockIdx.x * total_tiles * G) / gridDim.x : 0;
    const long bal_hi = BAL ? ((long)(blockIdx.x + 1) * total_tiles * G) / gridDim.x : 0;
    auto segment = [&](int idx, int& tile, int& gb, int& ge) -> bool {
        if (BAL) {
            tile = (int)(bal_lo / G) + idx;
            gb = idx == 0 ? (int)(bal_lo % G) : 0;
            const long left = bal_hi - (long)tile * G;
            ge = left < G ? (int)left : G;
            return gb < ge;
        }
        tile = unit + idx * num_units;
        gb = 0;
        ge = G;
        return tile < total_tiles;
    };

    bool exchanged = false;                     // SPLIT: this thread has passed the first cluster barrier
    if (warp < 4) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
        if (warp == WARP_PRODUCER && lane == 0) {
            // ------------------------------------------------ producer: activation tiles ----
            ptx::pdl_wait();                                    // the activations are the previous kernel's output
            uint32_t it = 0;
            bool ok = true;
            for (int si = 0; ok; ++si) {
                int tile, gb, ge, ntile, mtile;
                if (!segment(si, tile, gb, ge)) break;
                tile_of(tile, ntile, mtile);
                for (int g = gb; g < ge; ++g, ++it) {
                    const uint32_t sb = it % C::SB;
                    if (it >= (uint32_t)C::SB && !(ok = ptx::mbar_wait(done_bar(it - C::SB), done_parity(it - C::SB), abort_flag))) break;
                    ptx::mbar_arrive_expect_tx(bar(B_FULL + sb), C::B_BYTES);
                    ptx::tma_load_2d(smem_base + C::B_OFF + sb * C::B_BYTES, &tmap_qa, (g_lo + g) * GROUP, mtile * TILE_M,
                                     bar(B_FULL + sb));
                }
            }
            if (!ok) {   // let copies already in flight land before shared memory is released
                const uint64_t t0 = ptx::globaltimer_ns();
                while (ptx::globaltimer_ns() - t0 < 200000ull) {}
            }
        } else if (warp == WARP_RAW_PRODUCER && lane == 0) {
            // --------------------------------------------------- producer: packed blobs ----
            uint32_t it = 0;
            bool ok = true;
            for (int si = 0; ok; ++si) {
                int tile, gb, ge, ntile, mtile;
                if (!segment(si, tile, gb, ge)) break;
                tile_of(tile, ntile, mtile);
                const uint8_t* src = packed + ((size_t)ntile * GK + g_lo) * BLOB_BYTES;
                for (int g = gb; g < ge; ++g, ++it) {
                    const uint32_t sr = it % C::SR, pr = (it / C::SR) & 1;
                    if (!(ok = ptx::mbar_wait(bar(RAW_EMPTY + sr), pr ^ 1, abort_flag))) break;
                    ptx::mbar_arrive_expect_tx(bar(RAW_FULL + sr), BLOB_BYTES);
                    ptx::bulk_g2s(smem_base + C::RAW_OFF + sr * RAW_STRIDE, src + (size_t)g * BLOB_BYTES, BLOB_BYTES,
                                  bar(RAW_FULL + sr));
                }
            }
            if (!ok) {
                const uint64_t t0 = ptx::globaltimer_ns();
                while (ptx::globaltimer_ns() - t0 < 200000ull) {}
            }
        } else if (warp == WARP_MMA || warp == WARP_MMA_ODD) {
            // ---------------------------------------------------------------- MMA issuers ----
            // Two warps, one for the even pipeline steps (accumulator buffer 0) and one for the odd
            // ones (buffer 1).  A step costs its issuer several dependent shared-memory and
            // tensor-pipe round trips (three barrier probes, four MMAs, a commit); with two issuers the
            // round trips of one step overlap the MMAs of the other.
            // The whole warp walks the loop and one elected lane issues: with warp-uniform control flow the
            // MMA operands (addresses, descriptors) are computed once per warp in uniform registers, which
            // is where the tensor instructions take them from; issued from inside a one-lane branch, every
            // operand of every MMA went through a register-to-uniform move first.
            const uint32_t par = __shfl_sync(0xFFFFFFFFu, (warp == WARP_MMA) ? 0u : 1u, 0);
            const uint32_t tmem_u = __shfl_sync(0xFFFFFFFFu, tmem_base, 0);
            constexpr uint32_t idesc = ptx::idesc_i8(TILE_N, TILE_M, true, true);
            // descriptor of activation stage 0; a stage and a K slice of 32 bytes are plain
            // additions to its (address >> 4) field
            const uint64_t b_desc0 = ptx::smem_desc_k_sw128(smem_base + C::B_OFF);
            uint32_t it = 0, tcount = 0;
            bool ok = true;
            for (int si = 0; ok; ++si, ++tcount) {
                int tile, gb, ge;
                if (!segment(si, tile, gb, ge)) break;
                // PC: both threads add into the buffer of the tile, which the drain warps left zeroed
                // (integer sums commute, so the order of the two threads' MMAs does not matter)
                uint32_t buf = PC ? (tcount & 1u) : par;
                uint32_t d_tmem = tmem_u + buf * TILE_M;
                bool mine = false;
                for (int g = gb; g < ge; ++g, ++it) {
                    if ((it & 1u) != par) continue;
                    const uint32_t sb = it % C::SB, pb = (it / C::SB) & 1;
                    const uint32_t sa_ = it % C::SA, pas = (it / C::SA) & 1;
                    // accumulator drained; activations landed; weights unpacked
                    // Parking waits, one after the other: polling the three barriers in a loop gained nothing at tall
                    // tiles (the accumulator hand-back this warp waits for there is 1 000 cycles away) and cost 3-4 %
                    // at short ones, where the probes queue up in front of the unpack warp's shared-memory accesses
                    // on the same scheduler.  At short tiles the unpacked weights arrive last by far.
                    // (Order as measured: weights first at short tiles; activations first at tall ones, 1.5 % there.)
                    if (TILE_M <= 128) {
                        if (!(ok = ptx::mbar_wait(bar(A_FULL + sa_), pas, abort_flag))) break;
                        if (!(ok = ptx::mbar_wait(bar(B_FULL + sb), pb, abort_flag))) break;
                    } else {
                        if (!(ok = ptx::mbar_wait(bar(B_FULL + sb), pb, abort_flag))) break;
                        if (!(ok = ptx::mbar_wait(bar(A_FULL + sa_), pas, abort_flag))) break;
                    }
                    if (!PC && C::NB == 4) { buf = it & 3u; d_tmem = tmem_u + buf * TILE_M; }      // this issuer's two buffers in turn
                    if (!(ok = ptx::mbar_wait(bar(ACC_EMPTY + buf), (PC ? (tcount >> 1) : (it / C::NB)) & 1, abort_flag))) break;
                    ptx::tc_fence_after_sync();
                    const uint64_t bd = b_desc0 + (uint64_t)(sb * (C::B_BYTES / 16));
                    const uint32_t a_tmem = tmem_u + C::A_COL0 + sa_ * A_COLS;
                    const uint32_t done = done_bar(it);
                    if (ptx::elect_one()) {
#pragma unroll
                        for (int kk = 0; kk < GROUP / 32; ++kk)   // not PC: the first K slice overwrites the buffer
                            ptx::mma_i8_ts(d_tmem, a_tmem + 8 * kk, bd + 2 * kk, idesc, (PC || kk) ? 1u : 0u);
                        ptx::tc_commit(done);                     // stages consumed (not PC: accumulator complete)
                    }
                    __syncwarp();
                    mine = true;
                }
                if (PC && ok) {
                    // the tile is complete when the MMAs of both issuers are: a commit tracks only its own thread's
                    // (elect.sync names the same lane of a full warp every time)
                    if (ptx::elect_one()) {
                        if (mine) ptx::tc_commit(bar(TILE_DONE + buf));
                        else ptx::mbar_arrive(bar(TILE_DONE + buf));
                    }
                    __syncwarp();
                }
            }
            if (ptx::elect_one()) ptx::tc_commit(bar(FINAL + par));
            __syncwarp();
            // nothing may still be executing on the tensor core when TMEM is freed
            ptx::mbar_wait(bar(FINAL + par), 0, abort_flag);
        }
    } else if (warp < WARP_DRAIN0) {
        // short tiles leave the drain registers to spare: the unpack gets them (its loads, arithmetic and
        // TMEM stores then overlap better; measured 4 % on single-tile problems)
        if (TILE_M > 128) asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
        else asm volatile("setmaxnreg.dec.sync.aligned.u32 96;");
        // -------------------------------------------------------------------- unpack ----
        // One weight row (= one TMEM lane) per thread: 64 packed bytes -> 128 signed bytes -> 32
        // TMEM columns of this group's weight stage, k ascending (4 consecutive k per column).
        const int u = tid - WARP_UNPACK0 * 32;
        const int sw0 = blob_chunk_pos(u, 0);
        const uint32_t a_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + C::A_COL0;
        uint32_t it = 0;
        bool ok = true;
        for (int si = 0; ok; ++si) {
            int tile, gb, ge;
            if (!segment(si, tile, gb, ge)) break;
            for (int g = gb; g < ge; ++g, ++it) {
                const uint32_t sr = it % C::SR, pr = (it / C::SR) & 1;
                const uint32_t sa_ = it % C::SA;
                if (!(ok = ptx::mbar_wait(bar(RAW_FULL + sr), pr, abort_flag))) break;
                const uint8_t* raw = smem + C::RAW_OFF + sr * RAW_STRIDE;
                const uint32_t z = (raw[BLOB_ZERO_OFF + (u >> 1)] >> ((u & 1) * 4)) & 0xFu;
                const uint32_t kz = 0x80808080u - z * 0x01010101u;       // per byte: 0x80 - z, no borrow
                // chunk p of row u sits at position p ^ ((u >> 1) & 3): eight consecutive rows hit eight bank groups
                const uint4* rawrow = reinterpret_cast<const uint4*>(raw + u * 64);
                const uint4 w0 = rawrow[sw0], w1 = rawrow[sw0 ^ 1], w2 = rawrow[sw0 ^ 2], w3 = rawrow[sw0 ^ 3];
                // the MMAs that read this stage's previous contents have completed
                if (it >= (uint32_t)C::SA && !(ok = ptx::mbar_wait(done_bar(it - C::SA), done_parity(it - C::SA), abort_flag))) break;
                ptx::tc_fence_after_sync();
                const uint32_t a_addr = a_lane + sa_ * A_COLS;
                auto put = [&](const uint4& w, int j) {                  // 16 packed bytes = k 32j .. 32j+31
                    // words 0..3 of a chunk hold the runs of four k (a0, a2), (a1, a3), (a4, a6), (a5, a7) in their
                    // (low, high) nibbles: columns in k order are lo(x), lo(y), hi(x), hi(y), lo(z), lo(w), hi(z), hi(w)
                    ptx::tmem_st_32x8(a_addr + 8 * j,
                                      sub_zero4(w.x & 0x0F0F0F0Fu, kz), sub_zero4(w.y & 0x0F0F0F0Fu, kz),
                                      sub_zero4((w.x >> 4) & 0x0F0F0F0Fu, kz), sub_zero4((w.y >> 4) & 0x0F0F0F0Fu, kz),
                                      sub_zero4(w.z & 0x0F0F0F0Fu, kz), sub_zero4(w.w & 0x0F0F0F0Fu, kz),
                                      sub_zero4((w.z >> 4) & 0x0F0F0F0Fu, kz), sub_zero4((w.w >> 4) & 0x0F0F0F0Fu, kz));
                };
                put(w0, 0);
                put(w1, 1);
                put(w2, 2);
                put(w3, 3);
                ptx::tmem_st_wait();
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) {
                    ptx::mbar_arrive(bar(A_FULL + sa_));
                    ptx::mbar_arrive(bar(RAW_EMPTY + sr));
                }
            }
        }
    } else {
        if (TILE_M > 128) asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
        else asm volatile("setmaxnreg.inc.sync.aligned.u32 160;");
        // --------------------------------------------------------------------- drain ----
        // Warp (q, h): TMEM lanes 32q..32q+31 (output channels), accumulator columns h*W.. (tokens).
        ptx::pdl_wait();                                        // token scales, hand-over flags, residual and output
        const int q = warp & 3, h = (warp - WARP_DRAIN0) >> 2;
        const int n_local = q * 32 + lane;
        const uint32_t lane_taddr = tmem_base + ((uint32_t)(q * 32) << 16) + h * C::W;
        // PC: this warp's part of an accumulator buffer back to zero (every MMA of a tile adds)
        auto zero_fill = [&](uint32_t taddr) {
#pragma unroll
            for (int c = 0; c < C::W; c += 8) ptx::tmem_st_32x8(taddr + c, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u);
            ptx::tmem_st_wait();
        };
        if (PC) {
            zero_fill(lane_taddr);
            zero_fill(lane_taddr + TILE_M);
            ptx::tc_fence_before_sync();
            __syncwarp();
        }
        if (lane == 0) {                                          // the accumulator buffers start out free
            for (int i = 0; i < 4; ++i) ptx::mbar_arrive(bar(ACC_EMPTY + i));
        }
        uint32_t it = 0, tcount = 0;
        bool ok = true;
        // token scales (raw fp16 bits) and first group scale of the next segment, requested before the epilogue of
        // the current one so that their latency is not added to the time the tensor pipe waits for this warp
        uint16_t next_sa_bits[C::NCH], next_sw_bits = 0;
        bool have_next = false;
        auto request = [&](int idx) {
            int t2, gb2, ge2, nt2, mt2;
            have_next = segment(idx, t2, gb2, ge2);
            if (!have_next) return;
            tile_of(t2, nt2, mt2);
            const int mb2 = mt2 * TILE_M + h * C::W;
#pragma unroll
            for (int k = 0; k < C::NCH; ++k) {
                const int i = lane + 32 * k;
                next_sa_bits[k] = (i < C::W && mb2 + i < M) ? __ldg(sa + mb2 + i) : (uint16_t)0;
            }
            next_sw_bits = __ldg(reinterpret_cast<const uint16_t*>(packed + ((size_t)nt2 * GK + g_lo + gb2) * BLOB_BYTES +
                                                                   BLOB_SCALE_OFF + 2 * n_local));
        };
        request(0);
        for (int si = 0; ok; ++si, ++tcount) {
            int tile, gb, ge, ntile, mtile;
            if (!segment(si, tile, gb, ge)) break;
            tile_of(tile, ntile, mtile);
            const int n = ntile * TILE_N + n_local;
            const int m_base = mtile * TILE_M + h * C::W;
            const uint8_t* sw_ptr = packed + ((size_t)ntile * GK + g_lo) * BLOB_BYTES + BLOB_SCALE_OFF + 2 * n_local;
            float facc[C::W];
#pragma unroll
            for (int i = 0; i < C::W; ++i) facc[i] = 0.0f;
            if (RES) {
                // the residual of this warp's part of the tile (W tokens x 64 bytes) is asked into L2 now; the epilogue's
                // loads then find it there
#pragma unroll
                for (int k = 0; k < C::NCH; ++k) {
                    const int m = m_base + lane + 32 * k;
                    if (lane + 32 * k < C::W && m < M)
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(residual + (size_t)m * N + (size_t)ntile * TILE_N + q * 32));
                }
            }
            // this warp's token scales, widened once per tile (rows past M get 0 and are never stored)
            float* sa_w = reinterpret_cast<float*>(smem + C::SA_OFF) + (warp - WARP_DRAIN0) * (C::NCH * 32);
            __syncwarp();
#pragma unroll
            for (int k = 0; k < C::NCH; ++k)
                if (lane + 32 * k < C::W) sa_w[lane + 32 * k] = __half2float(__ushort_as_half(next_sa_bits[k]));
            __syncwarp();
            uint16_t sw_bits = next_sw_bits;
            if (PC) {
                // one drain per tile: the buffer holds the sum of D over all groups (|sum| < 2^31 for K < 2^13 * 128)
                const uint32_t buf = tcount & 1u;
                const float sw = __half2float(__ushort_as_half(sw_bits));
                if (!(ok = ptx::mbar_wait_hot(bar(TILE_DONE + buf), (tcount >> 1) & 1, abort_flag))) break;
                ptx::tc_fence_after_sync();
                const uint32_t taddr = lane_taddr + buf * TILE_M;
                uint32_t v[C::NCH][32];
#pragma unroll
                for (int ch = 0; ch < C::NCH; ++ch) {
                    if (ch == C::NCH - 1 && C::LAST == 8) ptx::tmem_ld_32x8(taddr + ch * 32, reinterpret_cast<uint32_t(&)[8]>(v[ch]));
                    else ptx::tmem_ld_32x32(taddr + ch * 32, v[ch]);
                }
                ptx::tmem_ld_wait();
                zero_fill(taddr);
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(bar(ACC_EMPTY + buf));
#pragma unroll
                for (int ch = 0; ch < C::NCH; ++ch) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        if (ch * 32 + i < C::W) {
                            const int32_t di = (int32_t)v[ch][i];
                            // exact while |sum| < 2^24; beyond that one rounding of relative size 2^-24
                            facc[ch * 32 + i] = sw * (float)di;
                            if (DEBUG) {
                                const int m = m_base + ch * 32 + i;
                                if (m < M) debug_partials[(size_t)m * N + n] = di;
                            }
                        }
                    }
                }
            }
            for (int g = gb; g < (PC ? gb : ge); ++g, ++it) {
                const uint32_t buf = it & (C::NB - 1);
                const float sw = __half2float(__ushort_as_half(sw_bits));
                if (g + 1 < ge) sw_bits = __ldg(reinterpret_cast<const uint16_t*>(sw_ptr + (size_t)(g + 1) * BLOB_BYTES));
                // (short tiles: this warp mostly waits, and a polling loop's probes queue up in front of the unpack
                // warp's shared-memory accesses on the same scheduler; the parking wait leaves the queue alone)
                if (!(ok = (TILE_M <= 128 ? ptx::mbar_wait(done_bar(it), done_parity(it), abort_flag)
                                          : ptx::mbar_wait_hot(done_bar(it), done_parity(it), abort_flag)))) break;
                ptx::tc_fence_after_sync();
                const uint32_t taddr = lane_taddr + buf * TILE_M;
                // All of this warp's columns go to registers with back-to-back loads, then the buffer is
                // handed back: the MMA -> drain -> MMA round trip of a buffer, not the arithmetic
                // below, sets the pace of the pipeline.
                uint32_t v[C::NCH][32];
#pragma unroll
                for (int ch = 0; ch < C::NCH; ++ch) {
                    if (ch == C::NCH - 1 && C::LAST == 8) ptx::tmem_ld_32x8(taddr + ch * 32, reinterpret_cast<uint32_t(&)[8]>(v[ch]));
                    else ptx::tmem_ld_32x32(taddr + ch * 32, v[ch]);
                }
                ptx::tmem_ld_wait();
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(bar(ACC_EMPTY + buf));
#pragma unroll
                for (int ch = 0; ch < C::NCH; ++ch) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        if (ch * 32 + i < C::W) {
                            const int32_t di = (int32_t)v[ch][i];
                            facc[ch * 32 + i] = fmaf(sw, (float)di, facc[ch * 32 + i]);     // exact convert: |D| < 2^24
                            if (DEBUG) {
                                const int m = m_base + ch * 32 + i;
                                if (m < M) debug_partials[((size_t)m * GK + g_lo + g) * N + n] = di;
                            }
                        }
                    }
                }
            }
            if (!ok) break;
            request(si + 1);
            if (BAL && gb > 0) {
                // Balanced walk: the tile's earlier groups belong to the CTA before this one, which reaches
                // them at the end of its range.  Hand this CTA's sums over: element (token t, channel n) at
                // t * 128 + n of this CTA's slot, then the flag (release) once all eight drain warps have written.
                float* slot = handover + (size_t)blockIdx.x * (TILE_M * TILE_N);
#pragma unroll
                for (int i = 0; i < C::W; ++i) __stcg(slot + (size_t)(h * C::W + i) * TILE_N + n_local, facc[i]);
                // the barrier orders the eight warps' stores before the one release below (cumulative at gpu scope)
                ptx::named_bar_sync(2, NUM_DRAIN_WARPS * 32);
                if (warp == WARP_DRAIN0 && lane == 0) ptx::st_release_gpu_u32(handover_flags + blockIdx.x, 1u);
                continue;                       // the other CTA stores the tile
            }
            if (BAL && ge < G) {
                // ... and this CTA holds the earlier groups of a tile whose later groups the next CTA summed
                // long ago (they opened its range): wait for its flag (bounded), add its sums, clear the flag
                if (warp == WARP_DRAIN0 && lane == 0) {
                    if (!ptx::wait_flag_acquire_gpu(handover_flags + blockIdx.x + 1, 1u, abort_flag)) ok = false;
                }
                ptx::named_bar_sync(2, NUM_DRAIN_WARPS * 32);
                if (*abort_flag) { ok = false; break; }
                const float* slot = handover + (size_t)(blockIdx.x + 1) * (TILE_M * TILE_N);
#pragma unroll
                for (int i = 0; i < C::W; ++i) facc[i] += __ldcg(slot + (size_t)(h * C::W + i) * TILE_N + n_local);
                ptx::named_bar_sync(2, NUM_DRAIN_WARPS * 32);
                if (warp == WARP_DRAIN0 && lane == 0) handover_flags[blockIdx.x + 1] = 0u;     // zero again for the next call
            }
            if (SPLIT) {
                // every CTA of the cluster is past its last MMA: the activation rings are free and become
                // the exchange buffers; push this thread's partials to the CTAs that own them
                ptx::cluster_sync();
                exchanged = true;
                // element (token t, channel n) of the tile has index t * 128 + n; the indices are dealt out to
                // the S CTAs in contiguous chunks
                const int chunk = (TILE_M * TILE_N + S - 1) / S;
                const uint32_t red = smem_base + C::B_OFF;
#pragma unroll
                for (int i = 0; i < C::W; ++i) {
                    const int idx = (h * C::W + i) * TILE_N + n_local, owner = idx / chunk;
                    ptx::st_dsmem_f32(ptx::map_to_cta(red + (uint32_t)(slice * chunk + idx - owner * chunk) * 4u, (uint32_t)owner), facc[i]);
                }
                break;                          // one tile per cluster
            }
            // Epilogue: token scale, bf16, and a transpose through shared memory so that global
            // stores are 16 bytes per lane along the channel dimension (a thread owns a channel,
            // the output is token-major).  Blocks of up to 32 tokens x this warp's 32 channels.
            uint8_t* ob = smem + C::OUT_OFF + (warp - WARP_DRAIN0) * 2048;
            const uint32_t ob_addr = smem_base + C::OUT_OFF + (warp - WARP_DRAIN0) * 2048;
            __nv_bfloat16* yrow = y + (size_t)ntile * TILE_N + q * 32 + 8 * (lane & 3);
            uint4 rv[4];
            // residual rows 8 k + lane / 4 of block b, this lane's 16-byte piece of the warp's 64-byte row (zeros past M or W)
            auto load_res = [&](int b, uint4 (&dst)[4]) {
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int t = b * 32 + 8 * k + (lane >> 2), m = m_base + t;
                    dst[k] = make_uint4(0u, 0u, 0u, 0u);
                    if (RES && t < C::W && m < M)
                        dst[k] = __ldcg(reinterpret_cast<const uint4*>(residual + (size_t)m * N + (size_t)ntile * TILE_N + q * 32 + 8 * (lane & 3)));
                }
            };
#pragma unroll
            for (int b2 = 0; b2 < C::NCH; ++b2) {
                // The chunk's 32 token scales go to registers first: read one by one between the stores below
                // they would each wait for the store before them (both are shared-memory accesses the compiler
                // must keep in order), a chain of 32 round trips per chunk.
                float sc[32];
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float4 t = *reinterpret_cast<const float4*>(sa_w + b2 * 32 + 4 * k);
                    sc[4 * k] = t.x; sc[4 * k + 1] = t.y; sc[4 * k + 2] = t.z; sc[4 * k + 3] = t.w;
                }
                if (RES) {
                    // The projection's output joins the residual stream, added in fp32 before the one rounding.  A block's
                    // residual (32 tokens x this warp's 32 channels) is fetched in the layout of the stores - 16 bytes per
                    // lane, rows of 64 bytes, one block ahead - and written into the output block, from which each lane
                    // reads its own channel's column back, adds, rounds and overwrites.  y may be the residual buffer:
                    // this warp reads a block before it stores it.
                    if (b2 == 0) load_res(0, rv);
                    uint4 rv_next[4];
                    if (b2 + 1 < C::NCH) load_res(b2 + 1, rv_next);
                    if (lane == 0) ptx::bulk_wait_group_read0();
                    __syncwarp();
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        *reinterpret_cast<uint4*>(ob + (8 * k + (lane >> 2)) * 64 + 16 * (lane & 3)) = rv[k];
                    __syncwarp();
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        float rs[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            rs[i] = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(ob + (16 * half + i) * 64)[lane]);
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            if (b2 * 32 + 16 * half + i < C::W)
                                reinterpret_cast<__nv_bfloat16*>(ob + (16 * half + i) * 64)[lane] =
                                    __float2bfloat16_rn(facc[b2 * 32 + 16 * half + i] * sc[16 * half + i] + rs[i]);
                    }
#pragma unroll
                    for (int k = 0; k < 4; ++k) rv[k] = rv_next[k];
                } else {
                if (lane == 0) ptx::bulk_wait_group_read0();      // the previous block's TMA store has read `ob`
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (b2 * 32 + i < C::W)
                        reinterpret_cast<__nv_bfloat16*>(ob + i * 64)[lane] = __float2bfloat16_rn(facc[b2 * 32 + i] * sc[i]);
                }
                if (b2 < C::NCH - 1 || C::LAST == 32) {
                    // a full block of 32 tokens: one TMA store (rows past M are clipped by the map), the warp moves on
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        ptx::tma_store_2d(&tmap_y, ntile * TILE_N + q * 32, m_base + b2 * 32, ob_addr);
                        ptx::bulk_commit_group();
                    }
                } else {
                    // the 8-token tail of a 208-row tile: 16-byte stores per lane
                    __syncwarp();
                    const int row = lane >> 2;
                    const int m = m_base + b2 * 32 + row;
                    if (b2 * 32 + row < C::W && m < M) {
                        const uint4 val = *reinterpret_cast<const uint4*>(ob + row * 64 + 16 * (lane & 3));
                        *reinterpret_cast<uint4*>(yrow + (size_t)m * N) = val;
                    }
                }
            }
        }
        if (lane == 0) ptx::bulk_wait_group0();                   // every tile store of this warp has completed
        __syncwarp();
    }

    ptx::pdl_wait();                            // every thread, before the split-K tail's stores and the status word
    if (SPLIT) {
        // first barrier for every thread that has not passed it in the drain role, then the second one
        // (release after the pushes, acquire before the sums); this CTA then reduces its share of the tile
        if (!exchanged) ptx::cluster_sync();
        ptx::cluster_sync();
        if (unit < total_tiles && !*abort_flag) {
            int ntile, mtile;
            tile_of(unit, ntile, mtile);
            const int chunk = (TILE_M * TILE_N + S - 1) / S;
            const int lo = slice * chunk;
            const int cnt = (TILE_M * TILE_N - lo) < chunk ? (TILE_M * TILE_N - lo) : chunk;
            const float* red = reinterpret_cast<const float*>(smem + C::B_OFF);
            for (int i = tid; i < cnt; i += TC_THREADS) {
                float acc = 0.0f;
                for (int s2 = 0; s2 < S; ++s2) acc += red[s2 * chunk + i];        // rank order: deterministic
                const int idx = lo + i, m = mtile * TILE_M + idx / TILE_N, nn = idx % TILE_N;
                if (m < M) {
                    const float t = __half2float(__ushort_as_half(__ldg(sa + m)));
                    float v = acc * t;
                    if (RES) v += __bfloat162float(residual[(size_t)m * N + (size_t)ntile * TILE_N + nn]);
                    y[(size_t)m * N + (size_t)ntile * TILE_N + nn] = __float2bfloat16_rn(v);
                }
            }
        }
    }
    if (*abort_flag && lane == 0) atomicExch(status, (uint32_t)W4A8_ERR_TIMEOUT);
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == WARP_MMA) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

template <int TILE_M, bool DEBUG, bool SPLIT, bool PC = false, bool BAL = false, bool RES = false>
cudaError_t launch_tile(const int8_t* qa, const uint16_t* sa, const void* packed, void* y, const void* residual, int M, int N, int K, int S,
                        void* workspace, int32_t* debug_partials, cudaStream_t stream) {
    using C = Cfg<TILE_M>;
    CUtensorMap tmap, tmap_y;
    cudaError_t te = make_qa_tensor_map(&tmap, qa, M, K, TILE_M);
    if (te != cudaSuccess) return te;
    te = make_y_tensor_map(&tmap_y, y, M, N);
    if (te != cudaSuccess) return te;

    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    static bool attr_done[64] = {false};
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    const int sms = device_sm_count();
    if (!attr_done[dev]) {
        e = cudaFuncSetAttribute(gemm_tcgen05_kernel<TILE_M, DEBUG, SPLIT, PC, BAL, RES>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 C::SMEM_ALLOC);
        if (e != cudaSuccess) return e;
        attr_done[dev] = true;
    }
    const int m_tiles = (M + TILE_M - 1) / TILE_M;
    const int total = m_tiles * (N / TILE_N);
    // persistent: at most one CTA per SM; split-K: one cluster of S CTAs per tile
    const int grid = SPLIT ? total * S : (total < sms ? total : sms);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    // BAL: the tiles x groups units are dealt out evenly (a tile may then be shared by two neighbouring
    // CTAs, which meet through the hand-over area of the workspace); the caller has checked that it applies
    if (BAL && !(total > grid && grid <= HANDOVER_SLOTS && handover_bytes(M, N, K) > 0)) return cudaErrorInvalidConfiguration;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(TC_THREADS, 1, 1);
    cfg.dynamicSmemBytes = C::SMEM_ALLOC;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = SPLIT ? (unsigned)S : 1u;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, gemm_tcgen05_kernel<TILE_M, DEBUG, SPLIT, PC, BAL, RES>, tmap, tmap_y, static_cast<const uint8_t*>(packed), sa,
                              static_cast<__nv_bfloat16*>(y), static_cast<const __nv_bfloat16*>(residual), debug_partials,
                              reinterpret_cast<uint32_t*>(ws + WS_STATUS_OFF),
                              M, N, K, m_tiles, total, S, reinterpret_cast<float*>(ws + WS_SHARED_OFF),
                              reinterpret_cast<uint32_t*>(ws + WS_COUNTER_OFF));
}

// Clusters of S CTAs of the split-K kernel that the device can hold at once (S CTAs need S free SMs
// of one GPC, so this is less than SMs / S); 0 if the query fails.  Cached per device.
template <int TILE_M>
int max_active_clusters(int S) {
    static int cached[64][TC_MAX_SPLIT + 1] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64 || S < 2 || S > TC_MAX_SPLIT) return 0;
    if (cached[dev][S] == 0) {
        using C = Cfg<TILE_M>;
        int n = 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(S * 64), 1, 1);
        cfg.blockDim = dim3(TC_THREADS, 1, 1);
        cfg.dynamicSmemBytes = C::SMEM_ALLOC;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = (unsigned)S;
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        if (cudaFuncSetAttribute(gemm_tcgen05_kernel<TILE_M, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 C::SMEM_ALLOC) != cudaSuccess ||
            cudaOccupancyMaxActiveClusters(&n, gemm_tcgen05_kernel<TILE_M, false, true>, &cfg) != cudaSuccess)
            n = -1;
        cached[dev][S] = n > 0 ? n : -1;
    }
    return cached[dev][S] > 0 ? cached[dev][S] : 0;
}

template <bool DEBUG, bool PC = false, bool RES = false>
cudaError_t launch_plan(int tile_m, int S, bool balanced, const int8_t* qa, const uint16_t* sa, const void* packed, void* y,
                        const void* residual, int M, int N, int K, void* workspace, int32_t* debug_partials, cudaStream_t stream) {
    if (S > 1 && !PC) {
        if (tile_m == 64) return launch_tile<64, DEBUG, true, false, false, RES>(qa, sa, packed, y, residual, M, N, K, S, workspace, debug_partials, stream);
        if (tile_m == 128) return launch_tile<128, DEBUG, true, false, false, RES>(qa, sa, packed, y, residual, M, N, K, S, workspace, debug_partials, stream);
        return launch_tile<208, DEBUG, true, false, false, RES>(qa, sa, packed, y, residual, M, N, K, S, workspace, debug_partials, stream);
    }
    if (balanced && !PC) {
        if (tile_m == 64) return launch_tile<64, DEBUG, false, false, true, RES>(qa, sa, packed, y, residual, M, N, K, 1, workspace, debug_partials, stream);
        if (tile_m == 128) return launch_tile<128, DEBUG, false, false, true, RES>(qa, sa, packed, y, residual, M, N, K, 1, workspace, debug_partials, stream);
        return launch_tile<208, DEBUG, false, false, true, RES>(qa, sa, packed, y, residual, M, N, K, 1, workspace, debug_partials, stream);
    }
    if (tile_m == 64) return launch_tile<64, DEBUG, false, PC, false, RES>(qa, sa, packed, y, residual, M, N, K, 1, workspace, debug_partials, stream);
    if (tile_m == 128) return launch_tile<128, DEBUG, false, PC, false, RES>(qa, sa, packed, y, residual, M, N, K, 1, workspace, debug_partials, stream);
    return launch_tile<208, DEBUG, false, PC, false, RES>(qa, sa, packed, y, residual, M, N, K, 1, workspace, debug_partials, stream);
}

}  // namespace

// Tile height and K split for an [M, N, K] problem, from a cost model fitted to measurements on B200:
// a CTA spends about TC_FIXED_NS on launch, set-up and pipeline fill, then TC_GROUP_NS[height] per
// 128-k group of every tile it walks (the weight unpack, whose cost does not depend on the height,
// dominates a group, so taller tiles are cheaper per token); a K split into S slices costs
// TC_SPLIT_NS for the cluster exchange.  Tall tiles win when there are several waves of them, short
// ones when a tall tiling would leave SMs idle, and a K split when even the shortest tiling does.
long tcgen05_plan(int M, int N, int K, int sms, int* tile_m, int* split, int max_split, int* balanced) {
    const int heights[3] = {208, 128, 64};
    const int n_tiles = N / TILE_N, G = K / GROUP;
    long best_ns = -1;
    *tile_m = 64;
    *split = 1;
    if (balanced) *balanced = 0;
    for (int i = 0; i < 3; ++i) {
        if (heights[i] > 64 && M <= heights[i + 1]) continue;        // the next height down already covers M in one tile
        const long tiles = (long)((M + heights[i] - 1) / heights[i]) * n_tiles;
        const long waves = (tiles + sms - 1) / sms;
        for (int S = 1; S <= TC_MAX_SPLIT && S <= max_split; ++S) {
            if (S > 1) {
                if (tiles * S > sms || G / S < 4) break;
                const int room = i == 0 ? max_active_clusters<208>(S) : (i == 1 ? max_active_clusters<128>(S) : max_active_clusters<64>(S));
                if (tiles > room) continue;                          // the clusters must all be resident at once
            }
            const long ns = TC_FIXED_NS + waves * TC_GROUP_NS[i] * ((G + S - 1) / S) + (S > 1 ? TC_SPLIT_NS[i] : 0);
            if (best_ns < 0 || ns < best_ns) {                        // ties: taller tile, fewer slices
                best_ns = ns; *tile_m = heights[i]; *split = S;
                if (balanced) *balanced = 0;
            }
            // no split, more tiles than SMs: an even share of all tiles x groups units per CTA, at the price of
            // handing partial tiles over between neighbours
            if (S == 1 && balanced && tiles > sms && tiles % sms != 0 && sms <= HANDOVER_SLOTS && handover_bytes(M, N, K) > 0) {
                const long nb = TC_FIXED_NS + TC_GROUP_NS[i] * ((tiles * G + sms - 1) / sms) + TC_BALANCE_NS[i];
                if (nb < best_ns) { best_ns = nb; *tile_m = heights[i]; *split = 1; *balanced = 1; }
            }
        }
    }
    return best_ns;                                                   // the estimate, for the caller's choice of kernel family
}

cudaError_t launch_gemm_tcgen05(const int8_t* qa, const uint16_t* sa, const void* packed, void* y, const void* residual,
                                int M, int N, int K, void* workspace, int32_t* debug_partials,
                                cudaStream_t stream) {
    int tile_m = 64, S = 1, balanced = 0;
    tcgen05_plan(M, N, K, device_sm_count(), &tile_m, &S, TC_MAX_SPLIT, &balanced);
    if (residual)                                   // (no partials dump in this form)
        return launch_plan<false, false, true>(tile_m, S, balanced != 0, qa, sa, packed, y, residual, M, N, K, workspace, nullptr, stream);
    if (debug_partials)
        return launch_plan<true>(tile_m, S, balanced != 0, qa, sa, packed, y, nullptr, M, N, K, workspace, debug_partials, stream);
    return launch_plan<false>(tile_m, S, balanced != 0, qa, sa, packed, y, nullptr, M, N, K, workspace, debug_partials, stream);
}

// The same pipeline with one drain per tile: for weights whose scale does not change along K.
// debug_sums, if not null, receives the int32 sum over all groups per (token, channel), [M][N].
cudaError_t launch_gemm_tcgen05_per_channel(const int8_t* qa, const uint16_t* sa, const void* packed, void* y,
                                            int M, int N, int K, void* workspace, int32_t* debug_sums,
                                            cudaStream_t stream) {
    int tile_m = 64, S = 1;
    tcgen05_plan(M, N, K, device_sm_count(), &tile_m, &S, 1, nullptr);
    if (debug_sums)
        return launch_plan<true, true>(tile_m, 1, false, qa, sa, packed, y, nullptr, M, N, K, workspace, debug_sums, stream);
    return launch_plan<false, true>(tile_m, 1, false, qa, sa, packed, y, nullptr, M, N, K, workspace, debug_sums, stream);
}

}  // namespace w4a8
