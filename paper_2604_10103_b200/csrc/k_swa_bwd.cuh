// Gradient of the block-sparse attention (Eq. 6) with respect to the queries, on the Blackwell tensor path: the first
// piece of the backward pass that the training rollout needs for its step with gradient (Alg. 1).  128-token blocks.
//
// With p = softmax(s) over the kept keys of a query row, s = q k^T / sqrt(d), and g = dL/dO_local:
//     dq = (1 / sqrt(d)) * sum_c p_c (g . v_c - delta) k_c,     delta = g . o_local     (= sum_c p_c g . v_c)
// The forward pass leaves lse = log sum_c exp(s_c) per row (hf_sparse_swa), so p = exp(s - lse) needs no running maximum,
// and k_rowdot forms delta; the block mask is the forward's (held fixed: the top-K choice is piecewise constant).
//
// Per (batch*head, query block) unit and kept key tile t, three tensor-core products:
//   S  = Q K_t^T          A = Q  (smem, K-major),  B = K_t (smem, K-major)          -> TMEM [0, 128) / [384, 512), t even / odd
//   dP = dO V_t^T         A = dO (smem, K-major),  B = V_t (smem, K-major)          -> TMEM [128, 256)
//   dQ += dS K_t          A = dS (TMEM, bf16, written over S),  B = K_t (MN-major)   -> TMEM [256, 256 + D)
// and between them, on the softmax warps (thread = query row x half of the 128 key columns):
//   dS = exp2(S c - lse log2 e) * (dP - delta) / sqrt(d)        (columns past a short block's end: 0)
// The two score products of tile t + 1 are issued while the softmax warps work on tile t: S has two buffers, and the
// softmax threads free dP's one buffer as soon as their share of it is in registers.  A K tile is held from S to dS K
// (three stages), a V tile only until dP (two); with less, the latency of the tile loads (~3 000 clk here) is what a
// tile costs.  Every wait is bounded and reports through the device status word.
#pragma once
#include "k_swa_tc5.cuh"

// delta[r] = sum_d dO[r][d] * O[r][d], one warp per row.  grid: ceil(rows / 8), 256 threads.
template <int D>
__global__ void __launch_bounds__(256) k_rowdot(const bf16* __restrict__ a, const bf16* __restrict__ b, float* __restrict__ out, long long rows) {
    const long long r = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (r >= rows) return;
    float acc = 0.f;
    for (int c = lane * 2; c < D; c += 64) {
        const float2 x = unpack_bf16(*reinterpret_cast<const uint32_t*>(a + r * D + c));
        const float2 y = unpack_bf16(*reinterpret_cast<const uint32_t*>(b + r * D + c));
        acc = fmaf(x.x, y.x, fmaf(x.y, y.y, acc));
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (lane == 0) out[r] = acc;
}

template <int D>
struct SwaBwd {
    static constexpr int BLK = 128;
    static constexpr int SUB = D / 64, SUB_BYTES = BLK * 128, TILE_BYTES = SUB * SUB_BYTES;
    // a K tile is held until its dS K product has completed, a V tile only until dP has: three and two stages
    static constexpr int KST = 3, VST = 2;
    static constexpr int OFF_Q = 0, OFF_DO = TILE_BYTES, OFF_K = 2 * TILE_BYTES, OFF_V = OFF_K + KST * TILE_BYTES;
    static constexpr int OFF_BAR = OFF_V + VST * TILE_BYTES;
    static constexpr int USED_BYTES = OFF_BAR + 256;
    static constexpr int SMEM_BYTES = USED_BYTES + 1024;
    static constexpr int THREADS = 320;                  // warps 0-7: softmax (two column groups), 8: TMA, 9: MMA
    static constexpr int WARP_TMA = 8, WARP_MMA = 9;
    // S alternates between two buffers (tile t in buffer t % 2, the bf16 dS written over it); dP has one, which the softmax
    // threads free as soon as they hold their share of it in registers
    static constexpr int COL_S = 0, COL_S1 = 384, COL_DP = 128, COL_DQ = 256, TMEM_COLS = 512;
};

struct SwaBwdParams {
    const int32_t* idx;      // [B*H, T_m, keep]
    int keep, Tc, n_b, n_cached, ring_head, P, n_sink, Tm, n_units;
    float scale_log2, scale; // log2(e) / sqrt(d), 1 / sqrt(d)
    const float* lse;        // [B*H, T_c] natural log of the row's sum of exponentials (forward)
    const float* delta;      // [B*H, T_c] g . o_local
    bf16* dq;                // [B*H, T_c, D]
    int* dev_status;
};

template <int D>
__global__ void __launch_bounds__(SwaBwd<D>::THREADS, 1)
k_swa_bwd_dq(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_do,
             const __grid_constant__ CUtensorMap tm_kring, const __grid_constant__ CUtensorMap tm_vring,
             const __grid_constant__ CUtensorMap tm_kcur, const __grid_constant__ CUtensorMap tm_vcur,
             const __grid_constant__ SwaBwdParams p) {
    using namespace tc5;
    typedef SwaBwd<D> C;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t s_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* s_gen = smem_raw + (s_base - smem_u32(smem_raw));
    const uint32_t sQ = s_base + C::OFF_Q, sDO = s_base + C::OFF_DO, sK = s_base + C::OFF_K, sV = s_base + C::OFF_V;
    const uint32_t bar0 = s_base + C::OFF_BAR;
    const uint32_t bar_kf = bar0 + 128, bar_ke = bar0 + 152, bar_vf = bar0 + 32, bar_ve = bar0 + 48, bar_qf = bar0 + 64, bar_qe = bar0 + 72,
                   bar_sd = bar0 + 80, bar_ds = bar0 + 88, bar_dqf = bar0 + 96, bar_dqe = bar0 + 104, bar_dpf = bar0 + 120;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(s_gen + C::OFF_BAR + 112);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(s_gen + C::OFF_BAR + 116);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int keep = p.keep;
    const int my_units = (p.n_units - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const int n_tiles = my_units * keep;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::KST; ++s) { mbar_init(bar_kf + 8 * s, 1); mbar_init(bar_ke + 8 * s, 1); }
        for (int s = 0; s < C::VST; ++s) { mbar_init(bar_vf + 8 * s, 1); mbar_init(bar_ve + 8 * s, 1); }
        mbar_init(bar_qf, 1); mbar_init(bar_qe, 1); mbar_init(bar_sd, 1); mbar_init(bar_ds, 256); mbar_init(bar_dqf, 1); mbar_init(bar_dqe, 256); mbar_init(bar_dpf, 256);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == C::WARP_MMA) {
        tmem_alloc(smem_u32(tmem_slot), C::TMEM_COLS);
        tmem_relinquish();
    }
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    pdl_wait();

    if (warp == C::WARP_TMA) {
        // ================================================================= TMA producer: Q and dO per unit, K and V per tile
        if (lane == 0) {
            bool ok = true;
            int t = 0;
            const int Tn = (p.n_sink + p.n_cached + 1) * p.n_b;
            for (int n = 0; ok && n < my_units; ++n) {
                const int u = blockIdx.x + n * gridDim.x;
                const int bh = u / p.Tm, i = u - bh * p.Tm;
                const int32_t* my_idx = p.idx + (size_t)u * keep;
                if (n >= 1 && !(ok = mbar_wait<true>(bar_qe, (n - 1) & 1, abort_flag, p.dev_status, 81))) break;
                mbar_expect_tx(bar_qf, 2 * C::TILE_BYTES);
#pragma unroll
                for (int s = 0; s < C::SUB; ++s) {
                    tma_load_4d(sQ + s * C::SUB_BYTES, &tm_q, s * 64, i * C::BLK, bh, 0, bar_qf);
                    tma_load_4d(sDO + s * C::SUB_BYTES, &tm_do, s * 64, i * C::BLK, bh, 0, bar_qf);
                }
                for (int j = 0; j < keep; ++j, ++t) {
                    const int blk = checked_block(__ldg(my_idx + j), Tn, p.dev_status, u);
                    int c = 0, jb = blk;
                    while (jb >= p.n_b) { jb -= p.n_b; ++c; }
                    const bool cur = (c == p.n_sink + p.n_cached);
                    int slot = 0;
                    if (!cur) {
                        if (c < p.n_sink) slot = p.P + c;
                        else { slot = p.ring_head + c - p.n_sink; if (slot >= p.P) slot -= p.P; }
                    }
                    const int kst = t % C::KST, vst = t % C::VST;
                    if (t >= C::VST && !(ok = mbar_wait<true>(bar_ve + 8 * vst, ((t / C::VST) & 1) ^ 1, abort_flag, p.dev_status, 83))) break;
                    mbar_expect_tx(bar_vf + 8 * vst, C::TILE_BYTES);
#pragma unroll
                    for (int s = 0; s < C::SUB; ++s)
                        tma_load_4d(sV + vst * C::TILE_BYTES + s * C::SUB_BYTES, cur ? &tm_vcur : &tm_vring, s * 64, jb * C::BLK, bh, slot, bar_vf + 8 * vst);
                    if (t >= C::KST && !(ok = mbar_wait<true>(bar_ke + 8 * kst, ((t / C::KST) & 1) ^ 1, abort_flag, p.dev_status, 82))) break;
                    mbar_expect_tx(bar_kf + 8 * kst, C::TILE_BYTES);
#pragma unroll
                    for (int s = 0; s < C::SUB; ++s)
                        tma_load_4d(sK + kst * C::TILE_BYTES + s * C::SUB_BYTES, cur ? &tm_kcur : &tm_kring, s * 64, jb * C::BLK, bh, slot, bar_kf + 8 * kst);
                }
            }
            if (!ok) {
                const long long t0 = clock64();
                while (clock64() - t0 < 400000) {}
            }
        }
    } else if (warp == C::WARP_MMA) {
        // ================================================================= MMA issuer (warp-uniform, one elected lane issues)
        constexpr uint32_t IDESC_S = idesc_bf16(128, false);
        constexpr uint32_t IDESC_DQ = idesc_bf16(D, true);
        constexpr uint32_t TILE_STEP = C::TILE_BYTES >> 4;
        const uint64_t dq0 = smem_desc_sw128(sQ, 16, 1024), dd0 = smem_desc_sw128(sDO, 16, 1024);
        const uint64_t dk0 = smem_desc_sw128(sK, 16, 1024), dv0 = smem_desc_sw128(sV, 16, 1024);
        const uint64_t dkm = smem_desc_sw128(sK, C::SUB_BYTES, 1024);        // the K tile again, as the MN-major operand of dS K
        const uint32_t hi_k = (uint32_t)(dq0 >> 32), hi_m = (uint32_t)(dkm >> 32);
        bool ok = true;
        // S_t = Q K_t^T and dP_t = dO V_t^T, one tile ahead of the softmax warps: tile t + 1 is issued while they turn
        // tile t into dS (S into the other buffer; dP as soon as they have taken tile t's out of tensor memory)
        int n_s = 0, j_s = 0, t_s = 0;
        auto issue_scores = [&]() -> bool {
            if (j_s == 0 && !__all_sync(0xffffffffu, mbar_wait<true>(bar_qf, n_s & 1, abort_flag, p.dev_status, 84))) return false;
            const int kst = t_s % C::KST, vst = t_s % C::VST;
            if (!__all_sync(0xffffffffu, mbar_wait<true>(bar_kf + 8 * kst, (t_s / C::KST) & 1, abort_flag, p.dev_status, 85))) return false;
            if (!__all_sync(0xffffffffu, mbar_wait<true>(bar_vf + 8 * vst, (t_s / C::VST) & 1, abort_flag, p.dev_status, 86))) return false;
            fence_after_sync();
            if (elect_one()) {
                mma_ss_tile<D>(tmem + ((t_s & 1) ? C::COL_S1 : C::COL_S), (uint32_t)dq0, (uint32_t)dk0 + kst * TILE_STEP, hi_k, IDESC_S);
                mma_ss_tile<D>(tmem + C::COL_DP, (uint32_t)dd0, (uint32_t)dv0 + vst * TILE_STEP, hi_k, IDESC_S);
                mma_commit(bar_sd);
                mma_commit(bar_ve + 8 * vst);
                if (j_s == keep - 1) mma_commit(bar_qe);          // Q and dO of this unit have been read for the last time
            }
            __syncwarp();
            ++t_s;
            if (++j_s == keep) { j_s = 0; ++n_s; }
            return true;
        };
        if (n_tiles > 0) ok = issue_scores();
        int t = 0;
        for (int n = 0; ok && n < my_units; ++n) {
            for (int j = 0; ok && j < keep; ++j, ++t) {
                const int kst = t % C::KST;
                if (t + 1 < n_tiles) {
                    // dP of tile t is in the softmax threads' registers: the buffer may take tile t + 1
                    if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_dpf, t & 1, abort_flag, p.dev_status, 91)))) break;
                    if (!(ok = issue_scores())) break;
                }
                if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_ds, t & 1, abort_flag, p.dev_status, 87)))) break;
                // the accumulator of the previous unit has been read out before this unit's first product overwrites it
                if (j == 0 && n >= 1 && !(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_dqe, (n - 1) & 1, abort_flag, p.dev_status, 88)))) break;
                fence_after_sync();
                if (elect_one()) {
                    const uint32_t tS = tmem + ((t & 1) ? C::COL_S1 : C::COL_S);
                    mma_ts_tile_split(tmem + C::COL_DQ, tS, tS + 64, (uint32_t)dkm + kst * TILE_STEP, hi_m, IDESC_DQ, j > 0);
                    mma_commit(bar_ke + 8 * kst);
                    if (j == keep - 1) mma_commit(bar_dqf);
                }
                __syncwarp();
            }
        }
    } else {
        // ================================================================= softmax warps: dS from S and dP; dQ out at the unit's end
        const int grp = warp >> 2;                          // key columns [64 grp, 64 grp + 64) of a tile
        const int row = (warp & 3) * 32 + lane;
        const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        bool ok = true;
        int t = 0;
        for (int n = 0; ok && n < my_units; ++n) {
            const int u = blockIdx.x + n * gridDim.x;
            const int bh = u / p.Tm, i = u - bh * p.Tm;
            const int32_t* my_idx = p.idx + (size_t)u * keep;
            const int q0 = i * C::BLK, nq = min(C::BLK, p.Tc - q0);
            const size_t g_row = (size_t)bh * p.Tc + q0 + row;
            const float neg_lse2 = row < nq ? -p.lse[g_row] * 1.4426950408889634f : 0.f;
            const float delta = row < nq ? p.delta[g_row] : 0.f;
            for (int j = 0; j < keep; ++j, ++t) {
                const int blk = __ldg(my_idx + j);
                bool tail = false;
#pragma unroll
                for (int c = 1; c <= HF_MAX_CHUNKS; ++c) tail |= (blk + 1 == c * p.n_b);
                const int nv = tail ? p.Tc - (p.n_b - 1) * C::BLK : C::BLK;
                ok = __all_sync(0xffffffffu, mbar_wait(bar_sd, t & 1, abort_flag, p.dev_status, 89));
                if (!ok) break;
                fence_after_sync();
                const uint32_t tS = lane_base + ((t & 1) ? C::COL_S1 : C::COL_S) + grp * 64;
                // this thread's share of dP first, all of it: the MMA warp refills the buffer as soon as every thread has it
                uint32_t dp[2][32], s[32];
                tmem_ld32(lane_base + C::COL_DP + grp * 64, dp[0]);
                tmem_ld32(lane_base + C::COL_DP + grp * 64 + 32, dp[1]);
                tmem_ld32(tS, s);
                tmem_wait_ld();
                fence_before_sync();
                mbar_arrive(bar_dpf);
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t pk[16];
                    if (c == 1) {
                        tmem_ld32(tS + 32, s);
                        tmem_wait_ld();
                    }
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        const float p0 = fast_exp2(fmaf(__uint_as_float(s[e]), p.scale_log2, neg_lse2));
                        const float p1 = fast_exp2(fmaf(__uint_as_float(s[e + 1]), p.scale_log2, neg_lse2));
                        float d0 = p0 * (__uint_as_float(dp[c][e]) - delta) * p.scale;
                        float d1 = p1 * (__uint_as_float(dp[c][e + 1]) - delta) * p.scale;
                        if (grp * 64 + c * 32 + e >= nv) d0 = 0.f;
                        if (grp * 64 + c * 32 + e + 1 >= nv) d1 = 0.f;
                        pk[e >> 1] = pack_bf16_alu(d0, d1);
                    }
                    // (all of this thread's S columns of the chunk are in registers: the bf16 dS may go over them)
                    tmem_st16(tS + c * 16, pk);
                }
                tmem_wait_st();
                fence_before_sync();
                mbar_arrive(bar_ds);
            }
            if (!ok) break;
            ok = __all_sync(0xffffffffu, mbar_wait(bar_dqf, n & 1, abort_flag, p.dev_status, 90));
            if (!ok) break;
            fence_after_sync();
#pragma unroll
            for (int c = 0; c < D / 64; ++c) {
                uint32_t o[32];
                tmem_ld32(lane_base + C::COL_DQ + grp * (D / 2) + c * 32, o);
                tmem_wait_ld();
                if (row < nq) {
                    bf16* dst = p.dq + g_row * D + grp * (D / 2) + c * 32;
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        uint4 w;
                        w.x = pack_bf16(__uint_as_float(o[v * 8]), __uint_as_float(o[v * 8 + 1]));
                        w.y = pack_bf16(__uint_as_float(o[v * 8 + 2]), __uint_as_float(o[v * 8 + 3]));
                        w.z = pack_bf16(__uint_as_float(o[v * 8 + 4]), __uint_as_float(o[v * 8 + 5]));
                        w.w = pack_bf16(__uint_as_float(o[v * 8 + 6]), __uint_as_float(o[v * 8 + 7]));
                        *reinterpret_cast<uint4*>(dst + v * 8) = w;
                    }
                }
            }
            fence_before_sync();
            mbar_arrive(bar_dqe);
        }
    }
    fence_before_sync();
    __syncthreads();
    if (warp == C::WARP_MMA) {
        fence_after_sync();
        tmem_dealloc(tmem, C::TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------------------------
// dK and dV of the current chunk (the keys and values that carry gradient in the rollout: the cache holds clean chunks of
// earlier, gradient-free passes).  The transposed walk: unit = (batch*head, key block j of the current chunk); for every
// query block i that keeps j (read off the selection's bit mask), with rows = keys and columns = queries:
//   S^T  = K_j Q_i^T      A = K_j (smem), B = Q_i (smem)                      -> TMEM [0, 128)
//   dP^T = V_j dO_i^T     A = V_j (smem), B = dO_i (smem)                     -> TMEM [128, 256)
//   P^T  = exp2(S^T c - lse_i log2 e)  (bf16, over S^T),   dS^T = P^T (dP^T - delta_i) / sqrt(d)  (bf16, over dP^T)
//   dV_j += P^T dO_i      A = P^T (TMEM), B = dO_i (MN-major)                  -> TMEM [256, 256 + D)
//   dK_j += dS^T Q_i      A = dS^T (TMEM), B = Q_i (MN-major)                  -> TMEM [384, 384 + D)
// lse and delta are per QUERY, i.e. per column here: staged in shared memory per tile.  First version: S^T / dP^T
// single-buffered; Q / dO tiles double-buffered.
// ------------------------------------------------------------------------------------------------------------
template <int D>
struct SwaBwdKV {
    static constexpr int BLK = 128;
    static constexpr int SUB = D / 64, SUB_BYTES = BLK * 128, TILE_BYTES = SUB * SUB_BYTES;
    static constexpr int STAGES = 2;
    static constexpr int OFF_K = 0, OFF_V = TILE_BYTES, OFF_Q = 2 * TILE_BYTES, OFF_DO = OFF_Q + STAGES * TILE_BYTES;
    static constexpr int OFF_BAR = OFF_DO + STAGES * TILE_BYTES;
    static constexpr int OFF_ROW = OFF_BAR + 256;        // [2 stages][lse log2 e, delta][128] floats
    static constexpr int USED_BYTES = OFF_ROW + 2 * 2 * BLK * 4;
    static constexpr int SMEM_BYTES = USED_BYTES + 1024;
    static constexpr int THREADS = 320;                  // warps 0-7: softmax (two column groups), 8: TMA, 9: MMA
    static constexpr int WARP_TMA = 8, WARP_MMA = 9;
    static constexpr int COL_S = 0, COL_DP = 128, COL_DV = 256, COL_DK = 384, TMEM_COLS = 512;
};

struct SwaBwdKVParams {
    const uint32_t* mask;    // [B*H, T_m, mask_words]: the forward's selection
    int mask_words, first_block;     // logical index of the current chunk's first key block
    int Tc, n_b, Tm, n_units;        // units = B*H x n_b
    float scale_log2, scale;
    const float* lse;        // [B*H, T_c]
    const float* delta;      // [B*H, T_c]
    bf16* dk;                // [B*H, T_c, D]
    bf16* dv;
    int* dev_status;
};

template <int D>
__global__ void __launch_bounds__(SwaBwdKV<D>::THREADS, 1)
k_swa_bwd_dkv(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_do,
              const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
              const __grid_constant__ SwaBwdKVParams p) {
    using namespace tc5;
    typedef SwaBwdKV<D> C;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t s_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* s_gen = smem_raw + (s_base - smem_u32(smem_raw));
    const uint32_t sK = s_base + C::OFF_K, sV = s_base + C::OFF_V, sQ = s_base + C::OFF_Q, sDO = s_base + C::OFF_DO;
    const uint32_t bar0 = s_base + C::OFF_BAR;
    const uint32_t bar_kvf = bar0, bar_kve = bar0 + 8, bar_qf = bar0 + 16, bar_qe = bar0 + 32, bar_sd = bar0 + 48, bar_ds = bar0 + 56,
                   bar_accf = bar0 + 64, bar_acce = bar0 + 72;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(s_gen + C::OFF_BAR + 80);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(s_gen + C::OFF_BAR + 84);
    float* row_vals = reinterpret_cast<float*>(s_gen + C::OFF_ROW);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int my_units = (p.n_units - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    // does query block i of batch*head bh keep the unit's key block?  (the same answer in every role: all walk i = 0 .. T_m - 1)
    auto keeps = [&](int bh, int i, int jlog) -> bool {
        return (__ldg(p.mask + ((size_t)bh * p.Tm + i) * p.mask_words + (jlog >> 5)) >> (jlog & 31)) & 1u;
    };

    if (threadIdx.x == 0) {
        mbar_init(bar_kvf, 1); mbar_init(bar_kve, 1);
        for (int s = 0; s < C::STAGES; ++s) { mbar_init(bar_qf + 8 * s, 1); mbar_init(bar_qe + 8 * s, 1); }
        mbar_init(bar_sd, 1); mbar_init(bar_ds, 256); mbar_init(bar_accf, 1); mbar_init(bar_acce, 256);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == C::WARP_MMA) {
        tmem_alloc(smem_u32(tmem_slot), C::TMEM_COLS);
        tmem_relinquish();
    }
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    pdl_wait();

    if (warp == C::WARP_TMA) {
        // ================================================================= TMA producer: K_j, V_j per unit; Q_i, dO_i per kept pair
        if (lane == 0) {
            bool ok = true;
            int t = 0;
            for (int n = 0; ok && n < my_units; ++n) {
                const int u = blockIdx.x + n * gridDim.x;
                const int bh = u / p.n_b, jb = u - bh * p.n_b;
                const int jlog = p.first_block + jb;
                if (n >= 1 && !(ok = mbar_wait<true>(bar_kve, (n - 1) & 1, abort_flag, p.dev_status, 91))) break;
                mbar_expect_tx(bar_kvf, 2 * C::TILE_BYTES);
#pragma unroll
                for (int s = 0; s < C::SUB; ++s) {
                    tma_load_4d(sK + s * C::SUB_BYTES, &tm_k, s * 64, jb * C::BLK, bh, 0, bar_kvf);
                    tma_load_4d(sV + s * C::SUB_BYTES, &tm_v, s * 64, jb * C::BLK, bh, 0, bar_kvf);
                }
                for (int i = 0; ok && i < p.Tm; ++i) {
                    if (!keeps(bh, i, jlog)) continue;
                    const int st = t % C::STAGES;
                    if (t >= C::STAGES && !(ok = mbar_wait<true>(bar_qe + 8 * st, ((t / C::STAGES) & 1) ^ 1, abort_flag, p.dev_status, 92))) break;
                    mbar_expect_tx(bar_qf + 8 * st, 2 * C::TILE_BYTES);
#pragma unroll
                    for (int s = 0; s < C::SUB; ++s) {
                        tma_load_4d(sQ + st * C::TILE_BYTES + s * C::SUB_BYTES, &tm_q, s * 64, i * C::BLK, bh, 0, bar_qf + 8 * st);
                        tma_load_4d(sDO + st * C::TILE_BYTES + s * C::SUB_BYTES, &tm_do, s * 64, i * C::BLK, bh, 0, bar_qf + 8 * st);
                    }
                    ++t;
                }
            }
            if (!ok) {
                const long long t0 = clock64();
                while (clock64() - t0 < 400000) {}
            }
        }
    } else if (warp == C::WARP_MMA) {
        // ================================================================= MMA issuer (warp-uniform, one elected lane issues)
        constexpr uint32_t IDESC_S = idesc_bf16(128, false);
        constexpr uint32_t IDESC_ACC = idesc_bf16(D, true);
        constexpr uint32_t TILE_STEP = C::TILE_BYTES >> 4;
        const uint64_t dk0 = smem_desc_sw128(sK, 16, 1024), dv0 = smem_desc_sw128(sV, 16, 1024);
        const uint64_t dq0 = smem_desc_sw128(sQ, 16, 1024), dd0 = smem_desc_sw128(sDO, 16, 1024);
        const uint64_t dqm = smem_desc_sw128(sQ, C::SUB_BYTES, 1024), ddm = smem_desc_sw128(sDO, C::SUB_BYTES, 1024);   // as MN-major operands
        const uint32_t hi_k = (uint32_t)(dk0 >> 32), hi_m = (uint32_t)(dqm >> 32);
        bool ok = true;
        int t = 0;
        for (int n = 0; ok && n < my_units; ++n) {
            const int u = blockIdx.x + n * gridDim.x;
            const int bh = u / p.n_b, jb = u - bh * p.n_b;
            const int jlog = p.first_block + jb;
            if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_kvf, n & 1, abort_flag, p.dev_status, 93)))) break;
            int pairs = 0;
            for (int i = 0; ok && i < p.Tm; ++i) {
                if (!keeps(bh, i, jlog)) continue;
                const int st = t % C::STAGES;
                if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_qf + 8 * st, (t / C::STAGES) & 1, abort_flag, p.dev_status, 94)))) break;
                fence_after_sync();
                if (elect_one()) {
                    mma_ss_tile<D>(tmem + C::COL_S, (uint32_t)dk0, (uint32_t)dq0 + st * TILE_STEP, hi_k, IDESC_S);
                    mma_ss_tile<D>(tmem + C::COL_DP, (uint32_t)dv0, (uint32_t)dd0 + st * TILE_STEP, hi_k, IDESC_S);
                    mma_commit(bar_sd);
                }
                __syncwarp();
                if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_ds, t & 1, abort_flag, p.dev_status, 95)))) break;
                // the accumulators of the previous unit have been read out before this unit's first products overwrite them
                if (pairs == 0 && n >= 1 && !(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_acce, (n - 1) & 1, abort_flag, p.dev_status, 96)))) break;
                fence_after_sync();
                if (elect_one()) {
                    mma_ts_tile_split(tmem + C::COL_DV, tmem + C::COL_S, tmem + C::COL_S + 64, (uint32_t)ddm + st * TILE_STEP, hi_m, IDESC_ACC, pairs > 0);
                    mma_ts_tile_split(tmem + C::COL_DK, tmem + C::COL_DP, tmem + C::COL_DP + 64, (uint32_t)dqm + st * TILE_STEP, hi_m, IDESC_ACC, pairs > 0);
                    mma_commit(bar_qe + 8 * st);
                }
                __syncwarp();
                ++pairs; ++t;
            }
            if (!ok) break;
            if (elect_one()) { mma_commit(bar_accf); mma_commit(bar_kve); }      // everything of this unit has completed
            __syncwarp();
            if (pairs == 0 && n >= 1) {     // (nothing was issued: the previous unit's read-out still has to be waited for, to keep the phases in step)
                if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_acce, (n - 1) & 1, abort_flag, p.dev_status, 97)))) break;
            }
        }
    } else {
        // ================================================================= softmax warps (rows = keys, columns = queries)
        const int grp = warp >> 2;                          // query columns [64 grp, 64 grp + 64) of the pair
        const int row = (warp & 3) * 32 + lane;             // key row of the block
        const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        bool ok = true;
        int t = 0;
        for (int n = 0; ok && n < my_units; ++n) {
            const int u = blockIdx.x + n * gridDim.x;
            const int bh = u / p.n_b, jb = u - bh * p.n_b;
            const int jlog = p.first_block + jb;
            const int k0 = jb * C::BLK, nk = min(C::BLK, p.Tc - k0);
            int pairs = 0;
            for (int i = 0; ok && i < p.Tm; ++i) {
                if (!keeps(bh, i, jlog)) continue;
                const int q0 = i * C::BLK, nq = min(C::BLK, p.Tc - q0);
                // per-query values of this pair into shared memory (the buffer of pair t - 2 was read before its arrival on bar_ds)
                float* rv = row_vals + (t & 1) * 2 * C::BLK;
                if (threadIdx.x < C::BLK) {
                    const bool v = (int)threadIdx.x < nq;
                    rv[threadIdx.x] = v ? -p.lse[(size_t)bh * p.Tc + q0 + threadIdx.x] * 1.4426950408889634f : 0.f;
                    rv[C::BLK + threadIdx.x] = v ? p.delta[(size_t)bh * p.Tc + q0 + threadIdx.x] : 0.f;
                }
                asm volatile("bar.sync 1, 256;\n" ::: "memory");
                ok = __all_sync(0xffffffffu, mbar_wait(bar_sd, t & 1, abort_flag, p.dev_status, 98));
                if (!ok) break;
                fence_after_sync();
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t s[32], dp[32], pk[16], dk_[16];
                    tmem_ld32(lane_base + C::COL_S + grp * 64 + c * 32, s);
                    tmem_ld32(lane_base + C::COL_DP + grp * 64 + c * 32, dp);
                    tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        const int col = grp * 64 + c * 32 + e;
                        float p0 = fast_exp2(fmaf(__uint_as_float(s[e]), p.scale_log2, rv[col]));
                        float p1 = fast_exp2(fmaf(__uint_as_float(s[e + 1]), p.scale_log2, rv[col + 1]));
                        if (row >= nk || col >= nq) p0 = 0.f;               // rows past the key block's end, columns past the query block's
                        if (row >= nk || col + 1 >= nq) p1 = 0.f;
                        const float d0 = p0 * (__uint_as_float(dp[e]) - rv[C::BLK + col]) * p.scale;
                        const float d1 = p1 * (__uint_as_float(dp[e + 1]) - rv[C::BLK + col + 1]) * p.scale;
                        pk[e >> 1] = pack_bf16(p0, p1);
                        dk_[e >> 1] = pack_bf16(d0, d1);
                    }
                    tmem_st16(lane_base + C::COL_S + grp * 64 + c * 16, pk);
                    tmem_st16(lane_base + C::COL_DP + grp * 64 + c * 16, dk_);
                }
                tmem_wait_st();
                fence_before_sync();
                mbar_arrive(bar_ds);
                ++pairs; ++t;
            }
            if (!ok) break;
            ok = __all_sync(0xffffffffu, mbar_wait(bar_accf, n & 1, abort_flag, p.dev_status, 99));
            if (!ok) break;
            fence_after_sync();
            const size_t g_row = (size_t)bh * p.Tc + k0 + row;
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                bf16* out = which == 0 ? p.dv : p.dk;
#pragma unroll
                for (int c = 0; c < D / 64; ++c) {
                    uint32_t o[32];
                    tmem_ld32(lane_base + (which == 0 ? C::COL_DV : C::COL_DK) + grp * (D / 2) + c * 32, o);
                    tmem_wait_ld();
                    if (row < nk) {
                        bf16* dst = out + g_row * D + grp * (D / 2) + c * 32;
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            uint4 w;
                            if (pairs == 0) w = make_uint4(0u, 0u, 0u, 0u);     // no query block keeps this key block: no gradient
                            else {
                                w.x = pack_bf16(__uint_as_float(o[v * 8]), __uint_as_float(o[v * 8 + 1]));
                                w.y = pack_bf16(__uint_as_float(o[v * 8 + 2]), __uint_as_float(o[v * 8 + 3]));
                                w.z = pack_bf16(__uint_as_float(o[v * 8 + 4]), __uint_as_float(o[v * 8 + 5]));
                                w.w = pack_bf16(__uint_as_float(o[v * 8 + 6]), __uint_as_float(o[v * 8 + 7]));
                            }
                            *reinterpret_cast<uint4*>(dst + v * 8) = w;
                        }
                    }
                }
            }
            fence_before_sync();
            mbar_arrive(bar_acce);
        }
    }
    fence_before_sync();
    __syncthreads();
    if (warp == C::WARP_MMA) {
        fence_after_sync();
        tmem_dealloc(tmem, C::TMEM_COLS);
    }
}
