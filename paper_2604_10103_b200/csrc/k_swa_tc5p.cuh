// Block-sparse sliding-window attention (Eq. 6; Alg. 3 inner loops) on the Blackwell tensor path, "ping-pong"
// arrangement of the softmax: the kept tiles of a (batch*head, query block) unit alternate between two groups of
// four warps.  Each group owns one S buffer and one O accumulator in tensor memory and runs a complete online
// softmax over its own tiles (one query row per thread, no exchange between the groups inside a unit); while one
// group waits for its P V and next S to come back from the tensor core, the other group's exponentials have the
// special-function unit to themselves.  At the end of the unit the two partial results are merged:
//     O = (O_A 2^(m_A - m) + O_B 2^(m_B - m)) / (l_A 2^(m_A - m) + l_B 2^(m_B - m)),   m = max(m_A, m_B).
//   S = Q K_t^T        A = Q (smem, K-major, 128B swizzle), B = K_t (smem, K-major)     -> TMEM cols 128 (t & 1)
//   P = exp2(S*c - m)  bf16, written over the first 64 columns of its S buffer
//   O_g += P V_t       A = P (TMEM), B = V_t (smem, MN-major, 128B swizzle)              -> TMEM cols 256 + D (t & 1)
// Loader warps (Q + three-stage K ring; two-stage V ring) and the MMA warp as in k_swa_tc5.  Each tile group may be
// split further into CG column groups of four warps (thread = one row, 128 / CG columns; the column groups of a
// tile group exchange their row maxima through shared memory once per tile, as in k_swa_tc5), which puts 4 CG
// softmax warps of two different tiles on every scheduler.  A row share of S is read from tensor memory twice,
// 32 columns at a time (maximum, then exponentials), so that a thread holds 32 values at a time.  Every wait is
// bounded (~1 s) and reports through the device status word.
#pragma once
#include "tc5_common.cuh"
#include "k_swa_tc5.cuh"      // Tc5Params, RingPos

template <int D, int CG>
struct SwaTc5P {
    static constexpr int NCOL = 128 / CG;              // S columns per thread
    static constexpr int NSM = 256 * CG;               // softmax threads
    static constexpr int BLK = 128;
    static constexpr int SUB = D / 64;
    static constexpr int SUB_BYTES = BLK * 128;
    static constexpr int TILE_BYTES = SUB * SUB_BYTES;
    static constexpr int KSTAGES = 3, VSTAGES = 2;
    static constexpr int OFF_Q = 0, OFF_K = TILE_BYTES, OFF_V = OFF_K + KSTAGES * TILE_BYTES;
    static constexpr int OFF_BAR = OFF_V + VSTAGES * TILE_BYTES;
    static constexpr int OFF_X = OFF_BAR + 256;        // per tile group, column group and row: (m, l) of the unit, [2][CG][128] float2
    static constexpr int OFF_XM = OFF_X + 2 * CG * BLK * 8;   // row-max exchange [2 tile groups][2 parities][CG][128] floats
    static constexpr int USED_BYTES = OFF_XM + 4 * CG * BLK * 4;
    static constexpr int SMEM_BYTES = (USED_BYTES + 1024) > 120 * 1024 ? (USED_BYTES + 1024) : 120 * 1024;
    static constexpr int THREADS = NSM + 96;
    static constexpr int WARP_LOAD_K = NSM / 32, WARP_LOAD_V = NSM / 32 + 1, WARP_MMA = NSM / 32 + 2;
    static constexpr int TMEM_COLS = 512;
    static constexpr int COL_O = 2 * BLK;              // O_A at 256, O_B at 256 + D
};

template <int D, int CG>
__global__ void __launch_bounds__(SwaTc5P<D, CG>::THREADS, 1)
k_swa_tc5p(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kring,
           const __grid_constant__ CUtensorMap tm_vring, const __grid_constant__ CUtensorMap tm_kcur,
           const __grid_constant__ CUtensorMap tm_vcur, const Tc5Params p) {
    using namespace tc5;
    typedef SwaTc5P<D, CG> C;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t s_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* s_gen = smem_raw + (s_base - smem_u32(smem_raw));
    const uint32_t sQ = s_base + C::OFF_Q, sK = s_base + C::OFF_K, sV = s_base + C::OFF_V;
    const uint32_t bar0 = s_base + C::OFF_BAR;
    const uint32_t bar_kf = bar0, bar_ke = bar0 + 24, bar_vf = bar0 + 48, bar_ve = bar0 + 64, bar_sf = bar0 + 80,
                   bar_pf = bar0 + 96, bar_pv = bar0 + 112, bar_qf = bar0 + 128, bar_qe = bar0 + 136, bar_ep = bar0 + 144,
                   bar_ep2 = bar0 + 152, bar_drain = bar0 + 160, bar_mx = bar0 + 168, bar_mx2 = bar0 + 200;   // bar_mx*, [tile group][parity]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(s_gen + C::OFF_BAR + 240);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(s_gen + C::OFF_BAR + 244);
    float2* x_ml = reinterpret_cast<float2*>(s_gen + C::OFF_X);           // [2][CG][128]
    float* x_max = reinterpret_cast<float*>(s_gen + C::OFF_XM);           // [2][2][CG][128]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int keep = p.keep;
    const int my_units = (p.n_units - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const int n_tiles = my_units * keep;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 3; ++s) { mbar_init(bar_kf + 8 * s, 1); mbar_init(bar_ke + 8 * s, 1); }
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar_vf + 8 * s, 1); mbar_init(bar_ve + 8 * s, 1); mbar_init(bar_sf + 8 * s, 1);
            mbar_init(bar_pf + 8 * s, 128 * CG); mbar_init(bar_pv + 8 * s, 1);
            mbar_init(bar_mx + 16 * s, 128 * CG); mbar_init(bar_mx + 16 * s + 8, 128 * CG);
            mbar_init(bar_mx2 + 16 * s, 128 * CG); mbar_init(bar_mx2 + 16 * s + 8, 128 * CG);
        }
        mbar_init(bar_qf, 1); mbar_init(bar_qe, 1); mbar_init(bar_ep, C::NSM); mbar_init(bar_ep2, C::NSM); mbar_init(bar_drain, 1);
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

    if (warp == C::WARP_LOAD_K || warp == C::WARP_LOAD_V) {
        // ================================================================= TMA producers
        if (lane == 0) {
            const bool is_k = (warp == C::WARP_LOAD_K);
            bool ok = true;
            RingPos<C::KSTAGES> rk;
            RingPos<C::VSTAGES> rv;
            int t = 0;
            const int Tn = (p.n_sink + p.n_cached + 1) * p.n_b;
            for (int n = 0; ok && n < my_units; ++n) {
                const int u = blockIdx.x + n * gridDim.x;
                const int bh = u / p.Tm, i = u - bh * p.Tm;
                const int32_t* my_idx = p.idx + (size_t)u * keep;
                if (is_k) {   // Q of this unit, once the last S of the previous unit has read the buffer
                    if (n >= 1 && !(ok = mbar_wait<true>(bar_qe, (n - 1) & 1, abort_flag, p.dev_status, 1))) break;
                    mbar_expect_tx(bar_qf, C::TILE_BYTES);
#pragma unroll
                    for (int s = 0; s < C::SUB; ++s)
                        tma_load_4d(sQ + s * C::SUB_BYTES, &tm_q, s * 64, i * C::BLK, bh, 0, bar_qf);
                }
                for (int j = 0; j < keep; ++j, ++t) {
                    const int blk = checked_block(__ldg(my_idx + j), Tn, is_k ? p.dev_status : nullptr, u);
                    int c = 0, jb = blk;
                    while (jb >= p.n_b) { jb -= p.n_b; ++c; }          // at most HF_MAX_CHUNKS - 1 steps; no XU-pipe division
                    // logical chunk order: sink chunks (slots P, P + 1, ...), cached chunks oldest first (ring), current chunk
                    const bool cur = (c == p.n_sink + p.n_cached);
                    int slot = 0;
                    if (!cur) {
                        if (c < p.n_sink) slot = p.P + c;
                        else { slot = p.ring_head + c - p.n_sink; if (slot >= p.P) slot -= p.P; }
                    }
                    if (is_k) {
                        const CUtensorMap* mk = cur ? &tm_kcur : &tm_kring;
                        if (t >= C::KSTAGES && !(ok = mbar_wait<true>(bar_ke + 8 * rk.stage, rk.phase ^ 1u, abort_flag, p.dev_status, 2))) break;
                        mbar_expect_tx(bar_kf + 8 * rk.stage, C::TILE_BYTES);
#pragma unroll
                        for (int s = 0; s < C::SUB; ++s)
                            tma_load_4d(sK + rk.stage * C::TILE_BYTES + s * C::SUB_BYTES, mk, s * 64, jb * C::BLK, bh, slot, bar_kf + 8 * rk.stage);
                        rk.advance();
                    } else {
                        const CUtensorMap* mv = cur ? &tm_vcur : &tm_vring;
                        if (t >= C::VSTAGES && !(ok = mbar_wait<true>(bar_ve + 8 * rv.stage, rv.phase ^ 1u, abort_flag, p.dev_status, 3))) break;
                        mbar_expect_tx(bar_vf + 8 * rv.stage, C::TILE_BYTES);
#pragma unroll
                        for (int s = 0; s < C::SUB; ++s)
                            tma_load_4d(sV + rv.stage * C::TILE_BYTES + s * C::SUB_BYTES, mv, s * 64, jb * C::BLK, bh, slot, bar_vf + 8 * rv.stage);
                        rv.advance();
                    }
                }
            }
            if (!ok) {   // gave up: let the copies already in flight land before the CTA leaves
                const long long t0 = clock64();
                while (clock64() - t0 < 400000) {}
            }
        }
    } else if (warp == C::WARP_MMA) {
        // ================================================================= MMA issuer (warp-uniform, one elected lane issues)
        constexpr uint32_t IDESC_S = idesc_bf16(128, false);
        constexpr uint32_t IDESC_PV = idesc_bf16(D, true);
        constexpr uint32_t TILE_STEP = C::TILE_BYTES >> 4;
        const uint64_t dq0 = smem_desc_sw128(sQ, 16, 1024), dk0 = smem_desc_sw128(sK, 16, 1024);
        const uint64_t dv0 = smem_desc_sw128(sV, C::SUB_BYTES, 1024);
        const uint32_t q_lo = (uint32_t)dq0, k_lo = (uint32_t)dk0, v_lo = (uint32_t)dv0;
        const uint32_t qk_hi = (uint32_t)(dq0 >> 32), v_hi = (uint32_t)(dv0 >> 32);
        bool ok = true;
        int n_s = 0, j_s = 0, t_s = 0;                // unit, position in its list and stream index of the next S tile
        RingPos<C::KSTAGES> rk;
        // S_t = Q K_t^T into S buffer t & 1.  The buffer still holds P of tile t - 2: its P V is issued before this
        // call (the tensor pipe runs in order).
        auto issue_s = [&]() -> bool {
            if (j_s == 0 && !__all_sync(0xffffffffu, mbar_wait<true>(bar_qf, n_s & 1, abort_flag, p.dev_status, 4))) return false;
            if (!__all_sync(0xffffffffu, mbar_wait<true>(bar_kf + 8 * rk.stage, rk.phase, abort_flag, p.dev_status, 5))) return false;
            fence_after_sync();
            if (elect_one()) {
                mma_ss_tile<D>(tmem + (t_s & 1) * C::BLK, q_lo, k_lo + rk.stage * TILE_STEP, qk_hi, IDESC_S);
                mma_commit(bar_sf + 8 * (t_s & 1));
                mma_commit(bar_ke + 8 * rk.stage);
                if (j_s == keep - 1) mma_commit(bar_qe);
            }
            __syncwarp();
            rk.advance();
            ++t_s;
            if (++j_s == keep) { j_s = 0; ++n_s; }
            return true;
        };
        if (n_tiles > 0) ok = issue_s();
        if (ok && n_tiles > 1) ok = issue_s();
        int j_pv = 0;
        RingPos<C::VSTAGES> rv;
        for (int t = 0; ok && t < n_tiles; ++t) {
            const int g = t & 1;
            if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_pf + 8 * g, (t >> 1) & 1, abort_flag, p.dev_status, 6)))) break;
            if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_vf + 8 * rv.stage, rv.phase, abort_flag, p.dev_status, 7)))) break;
            fence_after_sync();
            if (elect_one()) {
                // the first tile of each group in a unit (positions 0 and 1) starts its accumulator afresh
                mma_ts_tile(tmem + C::COL_O + g * D, tmem + g * C::BLK, v_lo + rv.stage * TILE_STEP, v_hi, IDESC_PV, j_pv >= 2);
                mma_commit(bar_pv + 8 * g);
                mma_commit(bar_ve + 8 * rv.stage);
            }
            __syncwarp();
            rv.advance();
            if (++j_pv == keep) j_pv = 0;
            if (t + 2 < n_tiles && !(ok = issue_s())) break;
        }
        if (elect_one()) mma_commit(bar_drain);
        __syncwarp();
        {
            const long long t0 = clock64();
            while (!mbar_try_wait(bar_drain, 0) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
        }
    } else {
        // ================================================================= softmax groups / merge / epilogue
        const int g = warp / (4 * CG);                      // tile group: tiles with stream index t & 1 == g
        const int cg = (warp >> 2) % CG;                    // column group inside the tile group
        const int row = (warp & 3) * 32 + lane;             // query row of the tile = TMEM lane
        const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        const uint32_t tS = lane_base + g * C::BLK;
        constexpr int OC = D / CG;                          // accumulator columns this thread rescales
        const uint32_t tO_mine = lane_base + C::COL_O + g * D + cg * OC;
        const int tail_cols = p.Tc - (p.n_b - 1) * C::BLK;
        constexpr int NCH = C::NCOL / 32;                   // 32-column chunks of this thread's S share
        const int col0 = cg * C::NCOL;
        bool ok = true;
        int n_mine = 0;                                     // tiles this group has processed (exchange barrier phases)
        for (int n = 0; ok && n < my_units; ++n) {
            const int u = blockIdx.x + n * gridDim.x;
            const int bh = u / p.Tm, i = u - bh * p.Tm;
            const int32_t* my_idx = p.idx + (size_t)u * keep;
            const int q0 = i * C::BLK;
            const int nq = min(C::BLK, p.Tc - q0);
            const int t0 = n * keep;                        // stream index of the unit's first tile
            float m_used = -INFINITY, l_run = 0.f;          // l_run: this thread's share of the row sum
            bool first = true;
            int j = (t0 & 1) == g ? 0 : 1;                  // this group's first position in the unit
            const int Tn = (p.n_sink + p.n_cached + 1) * p.n_b;
            int blk_next = j < keep ? checked_block(__ldg(my_idx + j), Tn, nullptr, 0) : 0;
            if (n >= 1) {
                // every softmax thread has read both accumulators of the previous unit before either is started afresh
                ok = __all_sync(0xffffffffu, mbar_wait(bar_ep2, (n - 1) & 1, abort_flag, p.dev_status, 14));
                if (!ok) break;
            }
            for (; j < keep; j += 2, ++n_mine) {
                const int t = t0 + j;
                bool tail = false;
#pragma unroll
                for (int c = 1; c <= HF_MAX_CHUNKS; ++c) tail |= (blk_next + 1 == c * p.n_b);
                if (j + 2 < keep) blk_next = checked_block(__ldg(my_idx + j + 2), Tn, nullptr, 0);
                const int nv = tail ? tail_cols : C::BLK;
                // S of this tile has landed; so has P V of this group's previous tile (it precedes this S in the tensor pipe)
                ok = __all_sync(0xffffffffu, mbar_wait(bar_sf + 8 * g, (t >> 1) & 1, abort_flag, p.dev_status, 8));
                if (!ok) break;
                fence_after_sync();
                // ---- pass 1: maximum of this thread's share of the row, 32 columns at a time
                float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll 1
                for (int c = 0; c < NCH; ++c) {
                    uint32_t r[32];
                    tmem_ld32(tS + col0 + c * 32, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        float v0 = __uint_as_float(r[e]), v1 = __uint_as_float(r[e + 1]);
                        if (nv < C::BLK) {
                            if (col0 + c * 32 + e >= nv) v0 = -INFINITY;
                            if (col0 + c * 32 + e + 1 >= nv) v1 = -INFINITY;
                        }
                        mx[(e >> 1) & 3] = fmax3(mx[(e >> 1) & 3], v0, v1);
                    }
                }
                float mrow = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                if (CG > 1) {
                    // the column groups of this tile group learn the maximum of the whole row; the exchange also tells
                    // them that this thread has finished pass 1 (P columns written in pass 2 overlap other groups' S)
                    const int par = n_mine & 1;
                    float* xm = x_max + ((g * 2 + par) * CG) * C::BLK;
                    xm[cg * C::BLK + row] = mrow;
                    mbar_arrive(bar_mx + 16 * g + 8 * par);
                    ok = __all_sync(0xffffffffu, mbar_wait(bar_mx + 16 * g + 8 * par, (n_mine >> 1) & 1, abort_flag, p.dev_status, 11));
                    if (!ok) break;
#pragma unroll
                    for (int q = 0; q < CG; ++q) mrow = fmaxf(mrow, xm[q * C::BLK + row]);
                }
                const float m_new = fmaxf(m_used, mrow * p.scale_log2);
                // ---- lazy rescale of this group's accumulator: only when some row of the warp moved its maximum by more than 2^8
                if (first) {
                    m_used = m_new;
                    first = false;
                } else {
                    const bool need = (m_new - m_used) > 8.f;
                    if (__any_sync(0xffffffffu, need)) {
                        const float alpha = need ? fast_exp2(m_used - m_new) : 1.f;
                        if (need) { m_used = m_new; l_run *= alpha; }
#pragma unroll 1
                        for (int c = 0; c < OC / 32; ++c) {
                            uint32_t o[32];
                            tmem_ld32(tO_mine + c * 32, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                            tmem_st32(tO_mine + c * 32, o);
                        }
                    }
                }
                // ---- pass 2: P = exp2(S*c - m), row sum, bf16 pairs over the first 64 columns of the S buffer.  With one
                // column group a chunk of P overwrites columns this thread has already read.  With several, a group's P
                // columns overlap another group's S columns: every thread first turns its whole share into packed P in
                // registers, the groups meet (second exchange barrier), then all store.
                float2 rsum[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                const float2 scale2 = make_float2(p.scale_log2, p.scale_log2), negm2 = make_float2(-m_used, -m_used);
                uint32_t pk[NCH][16];
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    uint32_t r[32];
                    tmem_ld32(tS + col0 + c * 32, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        float2 x = ffma2(make_float2(__uint_as_float(r[e]), __uint_as_float(r[e + 1])), scale2, negm2);
                        if (nv < C::BLK) {
                            if (col0 + c * 32 + e >= nv) x.x = -INFINITY;
                            if (col0 + c * 32 + e + 1 >= nv) x.y = -INFINITY;
                        }
                        const float2 pe = make_float2(fast_exp2(x.x), fast_exp2(x.y));
                        rsum[(e >> 1) & 1] = fadd2(rsum[(e >> 1) & 1], pe);
                        pk[c][e >> 1] = pack_bf16(pe.x, pe.y);
                    }
                    if (CG == 1) tmem_st16(tS + c * 16, pk[c]);
                }
                if (CG > 1) {
                    // all column groups have read their S values of this tile: P may now overwrite the buffer's first half
                    const int par = n_mine & 1;
                    mbar_arrive(bar_mx2 + 16 * g + 8 * par);
                    ok = __all_sync(0xffffffffu, mbar_wait(bar_mx2 + 16 * g + 8 * par, (n_mine >> 1) & 1, abort_flag, p.dev_status, 15));
                    if (!ok) break;
#pragma unroll
                    for (int c = 0; c < NCH; ++c) tmem_st16(tS + col0 / 2 + c * 16, pk[c]);
                }
                l_run += (rsum[0].x + rsum[0].y) + (rsum[1].x + rsum[1].y);
                tmem_wait_st();
                fence_before_sync();
                mbar_arrive(bar_pf + 8 * g);
            }
            if (!ok) break;
            // ---- merge of the two tile groups and epilogue: O / l (+ history term), one rounding to bf16
            x_ml[(g * CG + cg) * C::BLK + row] = make_float2(m_used, l_run);
            mbar_arrive(bar_ep);
            ok = __all_sync(0xffffffffu, mbar_wait(bar_ep, n & 1, abort_flag, p.dev_status, 12));
            if (!ok) break;
            float mA = x_ml[row].x, lA = 0.f, mB = x_ml[CG * C::BLK + row].x, lB = 0.f;
#pragma unroll
            for (int q = 0; q < CG; ++q) { lA += x_ml[q * C::BLK + row].y; lB += x_ml[(CG + q) * C::BLK + row].y; }
            const float m = fmaxf(mA, mB);
            const float fA = lA > 0.f ? fast_exp2(mA - m) : 0.f;
            const float fB = lB > 0.f ? fast_exp2(mB - m) : 0.f;
            const float l = lA * fA + lB * fB;
            // last P V of each group in this unit: stream index of the last tile with that parity
            const int t_last = t0 + keep - 1;
#pragma unroll
            for (int gg = 0; gg < 2; ++gg) {
                const int tl = ((t_last & 1) == gg) ? t_last : t_last - 1;
                if (tl >= t0) {
                    ok = __all_sync(0xffffffffu, mbar_wait(bar_pv + 8 * gg, (tl >> 1) & 1, abort_flag, p.dev_status, 10));
                    if (!ok) break;
                }
            }
            if (!ok) break;
            fence_after_sync();
            const float inv = 1.f / l;
            const float wA = fA * inv, wB = fB * inv;
            const size_t g_row = (size_t)bh * p.Tc + q0 + row;
            if (g == 0 && cg == 0 && row < nq && p.lse) p.lse[g_row] = (m + log2f(l)) * 0.6931471805599453f;
            constexpr int EC = D / (2 * CG);                // output columns per thread: the 2 CG warps of a row quadrant split the row
            static_assert(EC % 16 == 0, "output share must be a multiple of 16 columns");
            const int ecol0 = (g * CG + cg) * EC;
#pragma unroll 1
            for (int c = 0; c < EC / 16; ++c) {
                const int col = ecol0 + c * 16;
                uint32_t oa[16], ob[16];
                tmem_ld16(lane_base + C::COL_O + col, oa);
                tmem_ld16(lane_base + C::COL_O + D + col, ob);
                tmem_wait_ld();
                if (row < nq) {
                    const size_t off = g_row * D + col;
                    bf16* dst = p.o + off;
                    const float* hsrc = p.hist ? p.hist + off : nullptr;
#pragma unroll
                    for (int v = 0; v < 2; ++v) {
                        float x[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            // an accumulator whose group had no tile in this unit holds stale values: weight 0 must win
                            const float a = wA != 0.f ? __uint_as_float(oa[v * 8 + e]) * wA : 0.f;
                            const float b = wB != 0.f ? __uint_as_float(ob[v * 8 + e]) * wB : 0.f;
                            x[e] = a + b;
                        }
                        if (hsrc) {
                            const float4 h0 = *reinterpret_cast<const float4*>(hsrc + v * 8);
                            const float4 h1 = *reinterpret_cast<const float4*>(hsrc + v * 8 + 4);
                            x[0] += h0.x; x[1] += h0.y; x[2] += h0.z; x[3] += h0.w;
                            x[4] += h1.x; x[5] += h1.y; x[6] += h1.z; x[7] += h1.w;
                        }
                        uint4 w;
                        w.x = pack_bf16(x[0], x[1]); w.y = pack_bf16(x[2], x[3]);
                        w.z = pack_bf16(x[4], x[5]); w.w = pack_bf16(x[6], x[7]);
                        *reinterpret_cast<uint4*>(dst + v * 8) = w;
                    }
                }
            }
            fence_before_sync();
            mbar_arrive(bar_ep2);
        }
    }
    fence_before_sync();
    __syncthreads();
    if (warp == C::WARP_MMA) {
        fence_after_sync();
        tmem_dealloc(tmem, C::TMEM_COLS);
    }
}
