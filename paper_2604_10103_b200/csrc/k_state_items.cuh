// Layer-batched state update (Eq. 3; Alg. 2 "if KV full: pop(0) -> update LN" for every layer of the model at once).
//
// All layers evict at the same moment (once per chunk, after the clean pass), and the update of one layer's state does
// not depend on anything else, so the evicted chunks of L layers go through ONE persistent launch: 30 x 28.75 MB at the
// 832x480 shape instead of thirty 28.75 MB launches that are each over before the memory pipeline has filled.
//
// The token range of a (layer, batch*head) item is cut into `nsplit` splits, and the splits into `ngroup` groups of
// consecutive splits (the same cuts, and the same order of additions, as k_absorb_tc5 + k_reduce_fold use for one layer:
// same operations on the same operands in the same order, so both paths leave the same bits in S and z).
// Work unit = (item, group); thread block c takes units c, c + gridDim.x, ... and sums a unit's splits on chip:
//   TMA warp        K (row-major) and V (128-byte swizzle) tiles of 64 tokens, ring of four stages, running ahead over
//                   split and unit boundaries
//   16 phi warps    phi(K) of a tile in fp32 -> bf16 hi + lo halves -> tensor memory (A operand, M = key feature,
//                   K = token), sum of phi(K) per feature in a register        [absorb_phi_tile, shared with k_absorb_tc5]
//   MMA warp        P_s += A_hi V + A_lo V over the tiles of split s, two P accumulators in tensor memory alternating
//   4 merge warps   R = P of the unit's first split, R += P_s for the others, likewise the phi(K) sums; when the unit ends R
//                   and the sums go to the unit's slot of the scratch buffer.  They run beside the next split's tiles.
// k_reduce_fold then adds the ngroup slots of every item to its state in ascending order and refolds S W^T.  With two
// groups per item the scratch traffic is 2 x 66 KB per item (against 2.4 MB of K, V read), and 720 units spread over the
// SMs within 3 % of evenly where 360 whole items would leave a third of them idle for the last third of the launch.
// Tensor memory (512 columns at head dim 128): R [0, D), P_0 [D, 2D), P_1 [2D, 3D), A_0 / A_1 (hi 32 + lo 32 columns each).
// Every wait is bounded and reports through the device status word; nothing traps.
#pragma once
#include "k_state_tc5.cuh"

#define HF_MAX_BATCH_LAYERS 64

template <int D>
struct AbsorbItems {
    typedef AbsorbTc5<D> A;
    static constexpr int TT = A::TT, NST = A::NST, NQ = A::NQ, SUB = A::SUB;
    static constexpr int K_BYTES = A::K_BYTES, VSUB_BYTES = A::VSUB_BYTES, V_BYTES = A::V_BYTES;
    static constexpr int OFF_K = 0, OFF_V = NST * K_BYTES, OFF_BAR = OFF_V + NST * V_BYTES;
    static constexpr int OFF_Z = OFF_BAR + 256;          // phi(K) sums of a split, [2 buffers][NQ][D] floats
    static constexpr int SMEM_BYTES = OFF_Z + 2 * NQ * D * 4 + 1024;
    static constexpr int WARP_MERGE = 4 * NQ;            // four merge warps: warp index % 4 = TMEM lane quadrant
    static constexpr int WARP_TMA = 4 * NQ + 4, WARP_MMA = 4 * NQ + 5;
    static constexpr int THREADS = 32 * (4 * NQ + 6);
    static constexpr int COL_R = 0, COL_P = D, COL_A = 3 * D;
    static constexpr int TMEM_COLS = 512;
    static_assert(3 * D + 128 <= TMEM_COLS, "tensor memory layout does not fit");
};

struct AbsorbItemsParams {
    int n_tokens;             // tokens per item
    int BH, n_units;          // units = layers of the call x B*H x ngroup; unit u: item u / ngroup (layer item / BH, batch*head item % BH), group u % ngroup
    int nsplit, ngroup;       // splits of an item's token range and groups of consecutive splits (the summation order)
    float* partials;          // [items][ngroup][D*D + D]: per unit the sum of its splits' phi(K)^T V, then of their phi(K) sums
    int slot[HF_MAX_BATCH_LAYERS];   // coordinate 3 of the tensor maps for each layer of the call
    const float* cos_k;       // rotation tables (ROPE instantiation only)
    const float* sin_k;
    int rope_rows;
    int* dev_status;
};

// grid: min(n_units, SMs); thread block c takes units c, c + gridDim.x, ...
// tm_k: [D, n_tokens, B*H, slots] box {D, 64}, no swizzle.  tm_v: same tensor, box {64, 64}, 128-byte swizzle.
template <int D, bool ROPE>
__global__ void __launch_bounds__(AbsorbItems<D>::THREADS, 1)
k_absorb_items(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
               const __grid_constant__ AbsorbItemsParams p) {
    using namespace tc5;
    typedef AbsorbItems<D> C;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t s_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* s_gen = smem_raw + (s_base - smem_u32(smem_raw));
    const uint32_t sK = s_base + C::OFF_K, sV = s_base + C::OFF_V, bar0 = s_base + C::OFF_BAR;
    // bar_full[s] completes for a tile when its K / V bytes have landed AND the A buffer the tile will use is free again
    // (the tensor core has consumed the tile two before it): one wait per tile for the phi warps instead of two.
    const uint32_t bar_full = bar0, bar_kfree = bar0 + 32, bar_vfree = bar0 + 64, bar_afull = bar0 + 96,
                   bar_dfull = bar0 + 128, bar_pfree = bar0 + 144, bar_zfull = bar0 + 160;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(s_gen + C::OFF_BAR + 176);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(s_gen + C::OFF_BAR + 180);
    float* z_x = reinterpret_cast<float*>(s_gen + C::OFF_Z);            // [2][NQ][D]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = (p.n_tokens + C::TT - 1) / C::TT;
    const int nsplit = p.nsplit;
    const int ngroup = p.ngroup;
    const int my_units = (p.n_units - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    auto split_lo = [&](int s) { return (int)(((long long)n_tiles * s) / nsplit); };       // first tile of split s
    auto group_lo = [&](int g) { return (int)(((long long)nsplit * g) / ngroup); };        // first split of group g
    int my_tiles = 0;                                                                       // tiles of all units of this thread block
    for (int n = 0; n < my_units; ++n) {
        const int grp = (blockIdx.x + n * gridDim.x) % ngroup;
        my_tiles += split_lo(group_lo(grp + 1)) - split_lo(group_lo(grp));
    }

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::NST; ++s) { mbar_init(bar_full + 8 * s, 2); mbar_init(bar_kfree + 8 * s, C::NQ * D); mbar_init(bar_vfree + 8 * s, 1); }
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar_afull + 8 * s, C::NQ * D);
            mbar_init(bar_dfull + 8 * s, 1); mbar_init(bar_pfree + 8 * s, D); mbar_init(bar_zfull + 8 * s, C::NQ * D);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        mbar_arrive(bar_full); mbar_arrive(bar_full + 8);     // the A buffers of the first two tiles are free from the start
    }
    if (warp == C::WARP_MMA) {
        tmem_alloc(smem_u32(tmem_slot), C::TMEM_COLS);
        tmem_relinquish();
    }
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    pdl_wait();                 // (set-up above may overlap the tail of the kernel before this one in the stream)

    if (warp == C::WARP_TMA) {
        // ================================================================= TMA producer
        if (lane == 0) {
            bool ok = true;
            int g = 0;                                        // tiles issued so far
            for (int n = 0; ok && n < my_units; ++n) {
                const int unit = blockIdx.x + n * gridDim.x;
                const int item = unit / ngroup, grp = unit - item * ngroup;
                const int lay = item / p.BH, bh = item - lay * p.BH;
                const int slot = p.slot[lay];
                const int t_lo = split_lo(group_lo(grp)), t_hi = split_lo(group_lo(grp + 1));
                for (int tile = t_lo; ok && tile < t_hi; ++tile, ++g) {
                    const int s = g % C::NST;
                    if (g >= C::NST) {
                        const uint32_t par_free = ((g / C::NST) & 1) ^ 1;
                        if (!(ok = mbar_wait<true>(bar_kfree + 8 * s, par_free, abort_flag, p.dev_status, 61))) break;
                        if (!(ok = mbar_wait<true>(bar_vfree + 8 * s, par_free, abort_flag, p.dev_status, 62))) break;
                    }
                    const int row0 = tile * C::TT;
                    mbar_expect_tx(bar_full + 8 * s, C::K_BYTES + C::V_BYTES);
                    tma_load_4d(sK + s * C::K_BYTES, &tm_k, 0, row0, bh, slot, bar_full + 8 * s);
#pragma unroll
                    for (int u = 0; u < C::SUB; ++u)
                        tma_load_4d(sV + s * C::V_BYTES + u * C::VSUB_BYTES, &tm_v, u * 64, row0, bh, slot, bar_full + 8 * s);
                }
            }
            if (!ok) {
                const long long t0 = clock64();
                while (clock64() - t0 < 400000) {}
            }
        }
    } else if (warp == C::WARP_MMA) {
        // ================================================================= MMA issuer (warp-uniform, one elected lane issues)
        constexpr uint32_t IDESC = idesc_bf16(D, true);
        const uint64_t dv0 = smem_desc_sw128(sV, C::VSUB_BYTES, 1024);
        bool ok = true;
        int g = 0, q = 0;                                     // tiles / splits so far
        for (int n = 0; ok && n < my_units; ++n) {
            const int grp = (blockIdx.x + n * gridDim.x) % ngroup;
            for (int sp = group_lo(grp); ok && sp < group_lo(grp + 1); ++sp, ++q) {
                const int lo = split_lo(sp), hi = split_lo(sp + 1);
                const int pb = q & 1;
                // the accumulator of this split was read by the merge warps two splits ago
                if (q >= 2 && !(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_pfree + 8 * pb, ((q >> 1) & 1) ^ 1, abort_flag, p.dev_status, 63)))) break;
                fence_after_sync();
                const uint32_t tP = tmem + C::COL_P + pb * D;
                for (int tile = lo; ok && tile < hi; ++tile, ++g) {
                    const int s = g % C::NST, ab = g & 1;
                    if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_afull + 8 * ab, (g >> 1) & 1, abort_flag, p.dev_status, 64)))) break;
                    if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_full + 8 * s, (g / C::NST) & 1, abort_flag, p.dev_status, 65)))) break;
                    fence_after_sync();
                    if (elect_one()) {
                        const uint32_t tA = tmem + C::COL_A + ab * 64;
                        const uint64_t dv = dv0 + (uint64_t)((s * C::V_BYTES) >> 4);
#pragma unroll
                        for (int ks = 0; ks < C::TT / 16; ++ks) {
                            const uint64_t db = dv + (uint64_t)(ks * (2048 >> 4));
                            mma_ts(tP, tA + ks * 8, db, IDESC, tile > lo || ks > 0);        // hi half
                            mma_ts(tP, tA + 32 + ks * 8, db, IDESC, true);                  // lo half
                        }
                        if (g + 2 < my_tiles) mma_commit(bar_full + 8 * ((g + 2) % C::NST));    // this tile's A buffer is the next-but-one's
                        mma_commit(bar_vfree + 8 * s);
                        if (tile == hi - 1) mma_commit(bar_dfull + 8 * pb);
                    }
                    __syncwarp();
                }
            }
        }
    } else if (warp >= C::WARP_MERGE) {
        // ================================================================= merge warps: the item's state lives in R
        const int quad = warp & 3;
        const int a = quad * 32 + lane;                         // key feature = TMEM lane = row of S
        const bool active = a < D;                              // (warp-uniform)
        const uint32_t lane_base = tmem + ((uint32_t)(quad * 32) << 16);
        bool ok = true;
        int q = 0;
        for (int n = 0; ok && active && n < my_units; ++n) {
            const int unit = blockIdx.x + n * gridDim.x;
            const int grp = unit % ngroup;
            float* out = p.partials + (size_t)unit * (D * D + D);
            float zsum = 0.f;
            const int sp0 = group_lo(grp), sp1 = group_lo(grp + 1);
            for (int sp = sp0; ok && sp < sp1; ++sp, ++q) {
                const int pb = q & 1;
                const uint32_t par = (q >> 1) & 1;
                ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_dfull + 8 * pb, par, abort_flag, p.dev_status, 66));
                if (ok) ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_zfull + 8 * pb, par, abort_flag, p.dev_status, 67));
                if (!ok) break;
                fence_after_sync();
                // R = P for the unit's first split, R += P for the others (R is this role's own: nothing else touches it)
#pragma unroll 1
                for (int c = 0; c < D; c += 32) {
                    uint32_t r[32], x[32];
                    tmem_ld32(lane_base + C::COL_P + pb * D + c, x);
                    if (sp > sp0) {
                        tmem_ld32(lane_base + C::COL_R + c, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) x[e] = __float_as_uint(__fadd_rn(__uint_as_float(r[e]), __uint_as_float(x[e])));
                    } else {
                        tmem_wait_ld();
                    }
                    tmem_st32(lane_base + C::COL_R + c, x);
                }
                const float* zp = z_x + pb * C::NQ * D;
                float zs = zp[a];
#pragma unroll
                for (int w = 1; w < C::NQ; ++w) zs += zp[w * D + a];
                zsum = sp > sp0 ? zsum + zs : zs;
                tmem_wait_st();
                fence_before_sync();
                mbar_arrive(bar_pfree + 8 * pb);
            }
            if (!ok) break;
            // the unit's sums to its slot of the scratch buffer (row a of the matrix: 4 D contiguous bytes per thread)
#pragma unroll 1
            for (int c = 0; c < D; c += 32) {
                uint32_t r[32];
                tmem_ld32(lane_base + C::COL_R + c, r);
                tmem_wait_ld();
#pragma unroll
                for (int v = 0; v < 8; ++v)
                    *reinterpret_cast<float4*>(out + (size_t)a * D + c + 4 * v) =
                        make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]), __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
            }
            out[D * D + a] = zsum;
        }
    } else {
        // ================================================================= phi(K) into tensor memory
        // NQ warps per TMEM lane quadrant: warps w, w + 4, ... own the same 32 key features (lanes) and convert consecutive
        // groups of TT / NQ tokens of a tile.  Warps whose lanes lie past the head dimension stay out of the loop.
        const int part = warp >> 2;
        const int a = (warp & 3) * 32 + lane;
        const bool active = a < D;                              // (warp-uniform)
        const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        bool ok = true;
        int g = 0, q = 0;
        for (int n = 0; ok && active && n < my_units; ++n) {
            const int grp = (blockIdx.x + n * gridDim.x) % ngroup;
            for (int sp = group_lo(grp); ok && sp < group_lo(grp + 1); ++sp, ++q) {
                const int lo = split_lo(sp), hi = split_lo(sp + 1);
                const int pb = q & 1;
                float2 zacc = make_float2(0.f, 0.f);
                for (int tile = lo; ok && tile < hi; ++tile, ++g) {
                    const int s = g % C::NST, ab = g & 1;
                    ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_full + 8 * s, (g / C::NST) & 1, abort_flag, p.dev_status, 68));
                    if (!ok) break;
                    fence_after_sync();
                    absorb_phi_tile<D, ROPE>(s_gen + C::OFF_K + s * C::K_BYTES, p.n_tokens, tile * C::TT, part, a,
                                             lane_base + C::COL_A + ab * 64, p.cos_k, p.sin_k, p.rope_rows, zacc);
                    tmem_wait_st();
                    fence_before_sync();
                    mbar_arrive(bar_afull + 8 * ab);
                    mbar_arrive(bar_kfree + 8 * s);
                }
                if (!ok) break;
                // the split's sums: the buffer was read by the merge warps two splits ago
                if (q >= 2) {
                    ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_pfree + 8 * pb, ((q >> 1) & 1) ^ 1, abort_flag, p.dev_status, 70));
                    if (!ok) break;
                }
                z_x[(pb * C::NQ + part) * D + a] = zacc.x + zacc.y;
                mbar_arrive(bar_zfull + 8 * pb);
            }
        }
    }
    pdl_trigger();
    fence_before_sync();
    __syncthreads();
    if (warp == C::WARP_MMA) {
        fence_after_sync();
        tmem_dealloc(tmem, C::TMEM_COLS);
    }
}
