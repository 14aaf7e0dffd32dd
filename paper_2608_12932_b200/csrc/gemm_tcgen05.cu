// Large-M W4A8 GEMM for sm_100a: TMA -> shared memory -> int4->int8 unpack in shared memory
// -> tcgen05.mma kind::i8 with int32 accumulators in TMEM -> per-group fp32 scaling -> bf16.
// (Sec. 3.4: "8-bit activations unlock faster INT8 matrix multiplies for the compute-heavy
// prefill"; Sec. 4: prefill is one long matrix multiplication.)
//
// Orientation ("swap-AB"): the 128 output channels of a tile are the MMA's M side (TMEM lanes),
// the tokens are its N side (TMEM columns).  A drain thread therefore owns ONE output channel:
// its group scale is a per-thread scalar and the per-group work on the CUDA cores is one
// int->float convert and one FMA per accumulator element.
//
// One pipeline step = one quantisation group = 128 k = four K=32 MMAs; the accumulator must
// be drained after every group because the scale changes, so TMEM holds two accumulator
// buffers: the tensor core fills one while the drain warps empty the other.
//
// The drain does no int->float conversion: the drain warps re-arm each accumulator buffer with
// the bit pattern 0x4B400000 (the float 1.5 * 2^23) and every MMA accumulates on top of it.
// |D| <= 128*15*127 < 2^22, so the int32 sum 0x4B400000 + D read back as a float IS
// 12582912 + D exactly; one add (minus 12582912) and one FMA with the group scale per element
// finish the job on the FMA pipe, leaving the ALU pipe to the unpack.  (Packed f32x2
// arithmetic was measured slower than scalar here.)
//
// Zero points are subtracted while unpacking (weights become signed, -15..15), so the int32
// accumulator is directly D = sum (q_w - z) q_a; identical to P - z*sum(q_a), and it moves the
// correction from the per-(token, channel, group) drain to the per-weight unpack.
//
// CTA pairs (token counts above 128, N a multiple of 256): two CTAs of a cluster run one
// tcgen05.mma.cta_group::2 of M = 256 output channels (128 per CTA) x 256 tokens.  Each CTA
// unpacks its own 128 weight rows and loads only HALF of the activation tile (128 tokens); the
// tensor cores of the pair read both halves.  Per MMA this cuts the bytes a CTA pulls from L2
// from 8.5 + 32 KB to 8.5 + 16 KB - the activation re-reads from L2, not HBM or the tensor
// pipe, were what bounded the single-CTA kernel.  The leader CTA issues the MMAs; the peer's
// unpack and drain warps arrive on the leader's barriers through the cluster's shared memory
// window, and MMA completion is committed to the barriers of both CTAs.  No TMA multicast.
//
// Warp roles (512 threads, four warpgroups so that setmaxnreg can move registers to the drain):
//   warp 0       producer of the activation tiles (2-D TMA loads)
//   warp 1       MMA issuer (one thread), owns TMEM allocation
//   warp 2       producer of the packed blobs (1-D bulk copies)
//   warps 4-7    unpack: raw blob -> signed int8 A tile in the 128-byte-swizzled K-major layout
//   warps 8-15   drain: tcgen05.ld -> convert -> FMA with the group scale; final bf16 store
// Every wait is bounded; on expiry the CTA records W4A8_ERR_TIMEOUT, frees TMEM and exits.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include "ptx_sm100.cuh"
#include "w4a8_internal.cuh"

namespace w4a8 {
namespace {

constexpr int TC_THREADS = 512;
constexpr int WARP_PRODUCER = 0, WARP_MMA = 1, WARP_RAW_PRODUCER = 2, WARP_UNPACK0 = 4, WARP_DRAIN0 = 8;
constexpr int NUM_UNPACK_WARPS = 4, NUM_DRAIN_WARPS = 8;
constexpr int RAW_STRIDE = 8576;                 // BLOB_BYTES rounded up to a multiple of 128
constexpr int A_BYTES = TILE_N * GROUP;          // 16384: 128 rows x 128 B, signed int8

// Shared-memory rings.  The activation tile comes from L2 through TMA with a latency of roughly
// 2000 cycles, the packed blob likewise, while the unpacked weight tile is produced locally:
// the three have separate rings, deep for the two that cover memory latency, shallow for the third.
template <int TILE_M, bool PAIR>
struct Cfg {
    static constexpr int B_ROWS = PAIR ? TILE_M / 2 : TILE_M;  // token rows of the activation tile this CTA loads
    static constexpr int B_BYTES = B_ROWS * GROUP;
    static constexpr int SB = B_ROWS == 256 ? 4 : (B_ROWS == 128 ? 6 : 8);    // activation stages
    static constexpr int SA = B_ROWS == 256 ? 2 : 3;                          // unpacked-weight stages
    static constexpr int SR = B_ROWS == 256 ? 5 : 6;                          // packed-blob stages
    static constexpr int B_OFF = 0;
    static constexpr int A_OFF = B_OFF + SB * B_BYTES;
    static constexpr int RAW_OFF = A_OFF + SA * A_BYTES;
    static constexpr int BAR_OFF = RAW_OFF + SR * RAW_STRIDE;
    static constexpr int NUM_BARS = 2 * SR + 2 * SB + 2 * SA + 4 + 1;
    static constexpr int MISC_OFF = (BAR_OFF + NUM_BARS * 8 + 15) & ~15;      // 16-byte aligned: staging is read with 16-byte loads
    static constexpr int SA_OFF = MISC_OFF + 16;   // per drain warp: token scales as fp32
    static constexpr int OUT_OFF = SA_OFF + NUM_DRAIN_WARPS * (TILE_M / 2) * 4;   // per drain warp: 32 tokens x 32 channels bf16
    static constexpr int SMEM_BYTES = OUT_OFF + NUM_DRAIN_WARPS * 2048;
    static constexpr int SMEM_ALLOC = SMEM_BYTES + 1024;       // slack to align the base to 1024 B
    static constexpr int TMEM_COLS = 2 * TILE_M;               // two accumulator buffers
    static constexpr int HALF = TILE_M / 2;                    // columns per drain warp
    static constexpr int CTAS = PAIR ? 2 : 1;
    static_assert(TILE_M == 64 || TILE_M == 128 || TILE_M == 256, "token tile");
    static_assert(!PAIR || TILE_M == 256, "pairs run 256-token tiles");
    static_assert(SMEM_ALLOC <= 227 * 1024, "shared memory");
    static_assert(OUT_OFF % 16 == 0 && SA_OFF % 16 == 0 && A_OFF % 1024 == 0, "alignment");
};

__device__ __forceinline__ uint32_t sub_zero4(uint32_t q, uint32_t kz) {
    // bytes of q in 0..15, bytes of kz = 0x80 - z with z in 0..15: per byte (q + 0x80 - z) ^ 0x80
    // is q - z as a signed int8; no carry crosses a byte (0x71 <= q + 0x80 - z <= 0x8F)
    return (q + kz) ^ 0x80808080u;
}

template <int TILE_M, bool DEBUG, bool PAIR>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_qa, const uint8_t* __restrict__ packed,
                    const uint16_t* __restrict__ sa, __nv_bfloat16* __restrict__ y,
                    int32_t* __restrict__ debug_partials, uint32_t* __restrict__ status,
                    int M, int N, int K, int m_tiles, int total_tiles) {
    using C = Cfg<TILE_M, PAIR>;
    // In a pair, rank 0 is the leader (issues the MMAs, owns the barriers the peer arrives on).
    const uint32_t rank = PAIR ? ptx::cluster_ctarank() : 0u;
    const int unit = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;          // CTA or CTA pair
    const int num_units = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    const int G = K / GROUP;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    auto bar = [&](int i) { return smem_base + C::BAR_OFF + 8 * i; };
    const int RAW_FULL = 0, RAW_EMPTY = C::SR, B_FULL = 2 * C::SR, B_EMPTY = B_FULL + C::SB, A_FULL = B_EMPTY + C::SB,
              A_EMPTY = A_FULL + C::SA, ACC_FULL = A_EMPTY + C::SA, ACC_EMPTY = ACC_FULL + 2, FINAL = ACC_EMPTY + 2;
    volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(smem + C::MISC_OFF);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + C::MISC_OFF + 4);

    if (warp == WARP_MMA) {
        if (lane == 0) {
            *abort_flag = 0;
            for (int i = 0; i < C::SR; ++i) {
                ptx::mbar_init(bar(RAW_FULL + i), 1);
                ptx::mbar_init(bar(RAW_EMPTY + i), NUM_UNPACK_WARPS);
            }
            for (int i = 0; i < C::SB; ++i) {
                ptx::mbar_init(bar(B_FULL + i), 1);
                ptx::mbar_init(bar(B_EMPTY + i), 1);
            }
            for (int i = 0; i < C::SA; ++i) {
                ptx::mbar_init(bar(A_FULL + i), NUM_UNPACK_WARPS * C::CTAS);     // leader's copy is the one waited on
                ptx::mbar_init(bar(A_EMPTY + i), 1);
            }
            for (int i = 0; i < 2; ++i) {
                ptx::mbar_init(bar(ACC_FULL + i), 1);
                ptx::mbar_init(bar(ACC_EMPTY + i), NUM_DRAIN_WARPS * C::CTAS);   // leader's copy is the one waited on
            }
            ptx::mbar_init(bar(FINAL), 1);
            ptx::fence_mbar_init();
        }
        __syncwarp();
        if (PAIR) {
            ptx::tmem_alloc_pair(smem_base + C::MISC_OFF, C::TMEM_COLS);
            ptx::tmem_relinquish_pair();
        } else {
            ptx::tmem_alloc(smem_base + C::MISC_OFF, C::TMEM_COLS);
            ptx::tmem_relinquish();
        }
    }
    if (warp == WARP_PRODUCER && lane == 0) ptx::prefetch_tmap(&tmap_qa);
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (PAIR) ptx::cluster_sync();      // the peer's barriers exist before anything arrives on them
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_holder;
    // tile of iteration i of this CTA (or pair): channel tile and token tile
    auto tile_of = [&](int t, int& ntile, int& mtile) {
        ntile = PAIR ? 2 * (t / m_tiles) + (int)rank : t / m_tiles;
        mtile = t % m_tiles;
    };

    if (warp < 4) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
        if (warp == WARP_PRODUCER && lane == 0) {
            // ------------------------------------------------ producer: activation tiles ----
            uint32_t it = 0;
            bool ok = true;
            for (int tile = unit; tile < total_tiles && ok; tile += num_units) {
                int ntile, mtile;
                tile_of(tile, ntile, mtile);
                for (int g = 0; g < G; ++g, ++it) {
                    const uint32_t sb = it % C::SB, pb = (it / C::SB) & 1;
                    if (!(ok = ptx::mbar_wait(bar(B_EMPTY + sb), pb ^ 1, abort_flag))) break;
                    ptx::mbar_arrive_expect_tx(bar(B_FULL + sb), C::B_BYTES);
                    ptx::tma_load_2d(smem_base + C::B_OFF + sb * C::B_BYTES, &tmap_qa, g * GROUP,
                                     mtile * TILE_M + (int)rank * C::B_ROWS, bar(B_FULL + sb));
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
            for (int tile = unit; tile < total_tiles && ok; tile += num_units) {
                int ntile, mtile;
                tile_of(tile, ntile, mtile);
                const uint8_t* src = packed + (size_t)ntile * G * BLOB_BYTES;
                for (int g = 0; g < G; ++g, ++it) {
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
        } else if (warp == WARP_MMA && lane == 0) {
            if (rank == 0) {
                // ------------------------------------------------------------ MMA issuer ----
                constexpr uint32_t idesc = ptx::idesc_i8(TILE_N * C::CTAS, TILE_M, true, true);
                // completion of the MMAs issued so far -> barrier `b` of this CTA and, in a pair, of the peer
                auto commit = [&](int b) {
                    if (PAIR) {
                        ptx::tc_commit_pair(bar(b));
                        ptx::tc_commit_pair(ptx::map_to_cta(bar(b), 1u));
                    } else {
                        ptx::tc_commit(bar(b));
                    }
                };
                uint32_t it = 0;
                bool ok = true;
                for (int tile = unit; tile < total_tiles && ok; tile += num_units) {
                    for (int g = 0; g < G; ++g, ++it) {
                        const uint32_t sb = it % C::SB, pb = (it / C::SB) & 1;
                        const uint32_t sa_ = it % C::SA, pas = (it / C::SA) & 1;
                        const uint32_t buf = it & 1, pa = (it >> 1) & 1;
                        // accumulator re-armed with the bias; weights unpacked and activations landed
                        // (in a pair the peer's unpack warps vouch for both on the leader's A_FULL barrier)
                        if (PAIR) {
                            if (!(ok = ptx::mbar_wait_cluster(bar(ACC_EMPTY + buf), pa, abort_flag))) break;
                            if (!(ok = ptx::mbar_wait_cluster(bar(A_FULL + sa_), pas, abort_flag))) break;
                        } else {
                            if (!(ok = ptx::mbar_wait_hot(bar(ACC_EMPTY + buf), pa, abort_flag))) break;
                            if (!(ok = ptx::mbar_wait_hot(bar(B_FULL + sb), pb, abort_flag))) break;
                            if (!(ok = ptx::mbar_wait_hot(bar(A_FULL + sa_), pas, abort_flag))) break;
                        }
                        ptx::tc_fence_after_sync();
                        const uint32_t a_addr = smem_base + C::A_OFF + sa_ * A_BYTES;
                        const uint32_t b_addr = smem_base + C::B_OFF + sb * C::B_BYTES;
                        const uint32_t d_tmem = tmem_base + buf * TILE_M;
#pragma unroll
                        for (int kk = 0; kk < GROUP / 32; ++kk) {
                            const uint64_t ad = ptx::smem_desc_k_sw128(a_addr + kk * 32);
                            const uint64_t bd = ptx::smem_desc_k_sw128(b_addr + kk * 32);
                            if (PAIR) ptx::mma_i8_ss_pair(d_tmem, ad, bd, idesc, 1u);           // on top of the bias
                            else ptx::mma_i8_ss(d_tmem, ad, bd, idesc, 1u);
                        }
                        commit(A_EMPTY + sa_);     // operands of these stages consumed
                        commit(B_EMPTY + sb);
                        commit(ACC_FULL + buf);    // accumulator of this group complete
                    }
                }
                commit(FINAL);
            }
            // nothing may still be executing on the tensor core when TMEM is freed
            ptx::mbar_wait(bar(FINAL), 0, abort_flag);
        }
    } else if (warp < WARP_DRAIN0) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
        // -------------------------------------------------------------------- unpack ----
        const int u = tid - WARP_UNPACK0 * 32;
        uint32_t it = 0;
        bool ok = true;
        for (int tile = unit; tile < total_tiles && ok; tile += num_units) {
            for (int g = 0; g < G; ++g, ++it) {
                const uint32_t sr = it % C::SR, pr = (it / C::SR) & 1;
                const uint32_t sa_ = it % C::SA, pas = (it / C::SA) & 1;
                if (!(ok = ptx::mbar_wait(bar(RAW_FULL + sr), pr, abort_flag))) break;
                if (!(ok = ptx::mbar_wait(bar(A_EMPTY + sa_), pas ^ 1, abort_flag))) break;
                const uint8_t* raw = smem + C::RAW_OFF + sr * RAW_STRIDE;
                uint8_t* a_tile = smem + C::A_OFF + sa_ * A_BYTES;
                // one weight row (64 packed bytes -> 128 signed bytes) per thread: its zero point is
                // fetched once; the four 16-byte chunks are visited in a lane-rotated order so that
                // the loads of a warp spread over the banks
                const uint32_t z = (raw[BLOB_ZERO_OFF + (u >> 1)] >> ((u & 1) * 4)) & 0xFu;
                const uint32_t kz = 0x80808080u - z * 0x01010101u;       // per byte: 0x80 - z, no borrow
                const uint8_t* rawrow = raw + u * 64;
                uint8_t* rowp = a_tile + u * 128;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int j = (i + u) & 3;                            // chunk j: k = 32j .. 32j+31
                    const uint4 w = *reinterpret_cast<const uint4*>(rawrow + j * 16);
                    uint4 o0, o1;
                    o0.x = sub_zero4(w.x & 0x0F0F0F0Fu, kz);
                    o0.y = sub_zero4((w.x >> 4) & 0x0F0F0F0Fu, kz);
                    o0.z = sub_zero4(w.y & 0x0F0F0F0Fu, kz);
                    o0.w = sub_zero4((w.y >> 4) & 0x0F0F0F0Fu, kz);
                    o1.x = sub_zero4(w.z & 0x0F0F0F0Fu, kz);
                    o1.y = sub_zero4((w.z >> 4) & 0x0F0F0F0Fu, kz);
                    o1.z = sub_zero4(w.w & 0x0F0F0F0Fu, kz);
                    o1.w = sub_zero4((w.w >> 4) & 0x0F0F0F0Fu, kz);
                    // K-major row of 128 B; 16-byte chunk index XOR (row % 8): the 128-byte swizzle
                    *reinterpret_cast<uint4*>(rowp + (((2 * j) ^ (u & 7)) << 4)) = o0;
                    *reinterpret_cast<uint4*>(rowp + (((2 * j + 1) ^ (u & 7)) << 4)) = o1;
                }
                ptx::fence_proxy_async_smem();
                if (PAIR) {
                    // the leader cannot see this CTA's TMA barrier: "operands ready" on the leader's
                    // barrier also vouches for the activation tile of this group having landed here
                    const uint32_t sb = it % C::SB, pb = (it / C::SB) & 1;
                    if (!(ok = ptx::mbar_wait(bar(B_FULL + sb), pb, abort_flag))) break;
                }
                __syncwarp();
                if (lane == 0) {
                    if (PAIR) ptx::mbar_arrive_remote(bar(A_FULL + sa_), 0u);     // the leader's barrier
                    else ptx::mbar_arrive(bar(A_FULL + sa_));
                    ptx::mbar_arrive(bar(RAW_EMPTY + sr));
                }
            }
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
        // --------------------------------------------------------------------- drain ----
        const int q = warp & 3, h = (warp - WARP_DRAIN0) >> 2;
        const int n_local = q * 32 + lane;
        constexpr int NCH = C::HALF / 32;                       // 32-column chunks per drain warp
        constexpr uint32_t ACC_BIAS_BITS = 0x4B400000u;         // 12582912.0f
        const uint32_t lane_taddr = tmem_base + ((uint32_t)(q * 32) << 16) + h * C::HALF;
        // arm both accumulator buffers (this warp's lanes and columns) before the first MMA
#pragma unroll
        for (int b2 = 0; b2 < 2; ++b2)
#pragma unroll
            for (int cc = 0; cc < NCH; ++cc) ptx::tmem_fill_32x32(lane_taddr + b2 * TILE_M + cc * 32, ACC_BIAS_BITS);
        ptx::tmem_st_wait();
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) {
            if (PAIR) {
                ptx::mbar_arrive_remote(bar(ACC_EMPTY + 0), 0u);
                ptx::mbar_arrive_remote(bar(ACC_EMPTY + 1), 0u);
            } else {
                ptx::mbar_arrive(bar(ACC_EMPTY + 0));
                ptx::mbar_arrive(bar(ACC_EMPTY + 1));
            }
        }
        uint32_t it = 0;
        bool ok = true;
        for (int tile = unit; tile < total_tiles && ok; tile += num_units) {
            int ntile, mtile;
            tile_of(tile, ntile, mtile);
            const int n = ntile * TILE_N + n_local;
            const int m_base = mtile * TILE_M + h * C::HALF;
            const uint8_t* sw_ptr = packed + (size_t)ntile * G * BLOB_BYTES + BLOB_SCALE_OFF + 2 * n_local;
            float facc[C::HALF];
#pragma unroll
            for (int i = 0; i < C::HALF; ++i) facc[i] = 0.0f;
            // this warp's token scales, widened once per tile (rows past M get 0 and are never stored)
            float* sa_w = reinterpret_cast<float*>(smem + C::SA_OFF) + (warp - WARP_DRAIN0) * C::HALF;
            __syncwarp();
            for (int i = lane; i < C::HALF; i += 32)
                sa_w[i] = (m_base + i < M) ? __half2float(__ushort_as_half(__ldg(sa + m_base + i))) : 0.0f;
            __syncwarp();
            uint16_t sw_bits = __ldg(reinterpret_cast<const uint16_t*>(sw_ptr));
            for (int g = 0; g < G; ++g, ++it) {
                const uint32_t buf = it & 1, pa = (it >> 1) & 1;
                const float sw = __half2float(__ushort_as_half(sw_bits));
                if (g + 1 < G) sw_bits = __ldg(reinterpret_cast<const uint16_t*>(sw_ptr + (size_t)(g + 1) * BLOB_BYTES));
                if (!(ok = ptx::mbar_wait_hot(bar(ACC_FULL + buf), pa, abort_flag))) break;
                ptx::tc_fence_after_sync();
                const uint32_t taddr = lane_taddr + buf * TILE_M;
                uint32_t v[2][32];
                ptx::tmem_ld_32x32(taddr, v[0]);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int ch = 0; ch < NCH; ++ch) {
                    if (ch + 1 < NCH) {
                        ptx::tmem_ld_32x32(taddr + (ch + 1) * 32, v[(ch + 1) & 1]);     // in flight during the math below
                    } else {
                        // every column of this buffer is in registers: re-arm it and hand it back to the
                        // MMA warp before the math of the last chunk (the buffer is the scarce resource)
#pragma unroll
                        for (int cc = 0; cc < NCH; ++cc) ptx::tmem_fill_32x32(taddr + cc * 32, ACC_BIAS_BITS);
                        ptx::tmem_st_wait();
                        ptx::tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) {
                            if (PAIR) ptx::mbar_arrive_remote(bar(ACC_EMPTY + buf), 0u);
                            else ptx::mbar_arrive(bar(ACC_EMPTY + buf));
                        }
                    }
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float d = __uint_as_float(v[ch & 1][i]) - 12582912.0f;       // exact: D as a float
                        facc[ch * 32 + i] = fmaf(sw, d, facc[ch * 32 + i]);
                        if (DEBUG) {
                            const int m = m_base + ch * 32 + i;
                            if (m < M) debug_partials[((size_t)m * G + g) * N + n] = (int)(v[ch & 1][i] - ACC_BIAS_BITS);
                        }
                    }
                    if (ch + 1 < NCH) ptx::tmem_ld_wait();
                }
            }
            if (!ok) break;
            // Epilogue: token scale, bf16, and a transpose through shared memory so that global
            // stores are 16 bytes per lane along the channel dimension (a thread owns a channel,
            // the output is token-major).  Blocks of 32 tokens x this warp's 32 channels.
            uint8_t* ob = smem + C::OUT_OFF + (warp - WARP_DRAIN0) * 2048;
            __nv_bfloat16* yrow = y + (size_t)ntile * TILE_N + q * 32 + 8 * (lane & 3);
#pragma unroll
            for (int b2 = 0; b2 < C::HALF / 32; ++b2) {
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    reinterpret_cast<__nv_bfloat16*>(ob + i * 64)[lane] = __float2bfloat16_rn(facc[b2 * 32 + i] * sa_w[b2 * 32 + i]);
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int row = (lane >> 2) + 8 * i;
                    const int m = m_base + b2 * 32 + row;
                    const uint4 val = *reinterpret_cast<const uint4*>(ob + row * 64 + 16 * (lane & 3));
                    if (m < M) *reinterpret_cast<uint4*>(yrow + (size_t)m * N) = val;
                }
            }
        }
    }

    if (*abort_flag && lane == 0) atomicExch(status, (uint32_t)W4A8_ERR_TIMEOUT);
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (PAIR) ptx::cluster_sync();      // neither CTA leaves while the other may still arrive on its barriers
    if (warp == WARP_MMA) {
        ptx::tc_fence_after_sync();
        if (PAIR) ptx::tmem_dealloc_pair(tmem_base, C::TMEM_COLS);
        else ptx::tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

template <int TILE_M, bool DEBUG, bool PAIR>
cudaError_t launch_tile(const int8_t* qa, const uint16_t* sa, const void* packed, void* y, int M, int N, int K,
                        void* workspace, int32_t* debug_partials, cudaStream_t stream) {
    using C = Cfg<TILE_M, PAIR>;
    CUtensorMap tmap;
    cudaError_t te = make_qa_tensor_map(&tmap, qa, M, K, C::B_ROWS);
    if (te != cudaSuccess) return te;

    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    static bool attr_done[64] = {false};
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    const int sms = device_sm_count();
    if (!attr_done[dev]) {
        e = cudaFuncSetAttribute(gemm_tcgen05_kernel<TILE_M, DEBUG, PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 C::SMEM_ALLOC);
        if (e != cudaSuccess) return e;
        attr_done[dev] = true;
    }
    const int m_tiles = (M + TILE_M - 1) / TILE_M;
    const int total = m_tiles * (N / (TILE_N * C::CTAS));           // tiles per CTA, or per CTA pair
    const int units = PAIR ? sms / 2 : sms;
    const int grid = (total < units ? total : units) * C::CTAS;
    uint8_t* ws = static_cast<uint8_t*>(workspace);

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(TC_THREADS, 1, 1);
    cfg.dynamicSmemBytes = C::SMEM_ALLOC;
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = C::CTAS;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemm_tcgen05_kernel<TILE_M, DEBUG, PAIR>, tmap, static_cast<const uint8_t*>(packed),
                              sa, static_cast<__nv_bfloat16*>(y), debug_partials,
                              reinterpret_cast<uint32_t*>(ws + WS_STATUS_OFF), M, N, K, m_tiles, total);
}

}  // namespace

// Token-tile height for an [M, N] problem.  A CTA's time per tile is dominated by unpacking the
// tile's weights, which does not depend on the tile height: measured on B200 a 64-, 128- and
// 256-token tile cost 1 : 1.13 : 1.47.  The persistent grid runs ceil(tiles / SMs) tiles per CTA,
// so the height with the smallest (tiles per CTA) x (cost per tile) wins: tall tiles when there
// are several waves of them, short ones when a tall tiling would leave SMs idle.
int tcgen05_tile_m(int M, int N, int sms) {
    const int heights[3] = {256, 128, 64};
    const int cost[3] = {147, 113, 100};
    const int n_tiles = N / TILE_N;
    int best = 64;
    long best_cost = -1;
    for (int i = 0; i < 3; ++i) {
        if (heights[i] > 64 && M <= heights[i] / 2) continue;       // half the height already covers M in one tile
        const long tiles = (long)((M + heights[i] - 1) / heights[i]) * n_tiles;
        const long c = ((tiles + sms - 1) / sms) * cost[i];
        if (best_cost < 0 || c < best_cost) { best_cost = c; best = heights[i]; }   // ties go to the taller tile
    }
    return best;
}

namespace {
template <bool DEBUG>
cudaError_t launch_height(int tile_m, bool pair, const int8_t* qa, const uint16_t* sa, const void* packed, void* y,
                          int M, int N, int K, void* workspace, int32_t* debug_partials, cudaStream_t stream) {
    if (pair) return launch_tile<256, DEBUG, true>(qa, sa, packed, y, M, N, K, workspace, debug_partials, stream);
    if (tile_m == 64) return launch_tile<64, DEBUG, false>(qa, sa, packed, y, M, N, K, workspace, debug_partials, stream);
    if (tile_m == 128) return launch_tile<128, DEBUG, false>(qa, sa, packed, y, M, N, K, workspace, debug_partials, stream);
    return launch_tile<256, DEBUG, false>(qa, sa, packed, y, M, N, K, workspace, debug_partials, stream);
}
}  // namespace

cudaError_t launch_gemm_tcgen05(const int8_t* qa, const uint16_t* sa, const void* packed, void* y,
                                int M, int N, int K, void* workspace, int32_t* debug_partials,
                                cudaStream_t stream, bool want_pair) {
    const bool pair = want_pair && M > 128 && N % (2 * TILE_N) == 0;
    const int sms = device_sm_count();
    const int tile_m = tcgen05_tile_m(M, N, sms);
    if (debug_partials)
        return launch_height<true>(tile_m, pair, qa, sa, packed, y, M, N, K, workspace, debug_partials, stream);
    return launch_height<false>(tile_m, pair, qa, sa, packed, y, M, N, K, workspace, debug_partials, stream);
}

}  // namespace w4a8
