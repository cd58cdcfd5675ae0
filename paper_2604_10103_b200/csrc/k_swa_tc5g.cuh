// Block-sparse sliding-window attention (Eq. 6; Alg. 3 with b_q = b_kv = 16 or 64) on the Blackwell tensor path.
//
// The tensor core works on 128 x 128 tiles; blocks of 16 or 64 tokens are therefore grouped:
//   unit  = 128 consecutive query rows of one (batch, head) = G = 128 / BLK query blocks ("row groups"), each with its
//           own kept list;
//   tile  = G key blocks side by side (G boxes of BLK rows from TMA, anywhere in the window) = 128 keys;
//   k_union_tiles  merges the G kept lists of a unit into one list of key blocks, each with the set of row groups that
//           keep it, and cuts it into tiles; the attention kernel then walks those tiles exactly like the 128-token kernel
//           walks its kept blocks, and masks, per (row group, key block), what a row group does not keep (-inf before the
//           exponential, so those keys have weight exactly zero, as in the definition).
// Work done on masked (row group, key block) pairs is wasted tensor time: the union of G random lists is larger than
// any one of them (k / |union| of the products are wanted: ~57 % for two lists that keep a quarter each, ~100 % when
// neighbouring query blocks keep the same blocks, as trained attention maps tend to).
// The first tile of a unit holds the FIRST kept block of every row group, so that every row has a finite maximum in the
// tile from which the softmax reference is taken (see k_swa_tc5.cuh for the fixed reference and for the second pass with
// the running maximum that takes over when a row leaves its range; here that pass runs per query block).
// Roles, barriers, tensor-memory layout and shared-memory layout are those of k_swa_tc5<D, 2, false>.
#pragma once
#include "k_swa_tc5.cuh"

// One list entry: key block index (10 bits) | row groups that keep it (8 bits) << 10 | valid tokens in the block << 18.
__host__ __device__ __forceinline__ uint32_t union_entry(int blk, uint32_t rows, int nv) { return (uint32_t)blk | (rows << 10) | ((uint32_t)nv << 18); }

// grid (units per batch*head, B*H), 256 threads.  idx: [B*H, T_m, keep] kept lists (ascending).  Out: entries
// [B*H * units, max_tiles, G] and tiles [B*H * units]; slots past the union in a unit's last tile repeat its first block with
// no row group (they are loaded -- every box of a tile must hold finite numbers -- and fully masked).
template <int BLK>
__global__ void __launch_bounds__(256) k_union_tiles(const int32_t* __restrict__ idx, int keep, int Tm, int Tn, int n_b, int Tc, int max_tiles,
                                                     uint32_t* __restrict__ entries, int* __restrict__ tiles, int* dev_status) {
    constexpr int G = 128 / BLK;
    __shared__ uint32_t rows[HF_MAX_TN];          // bits 0..7: row groups keeping the block; bit 8: some row group's first kept block
    __shared__ int warp_tot[2][8];
    const int mt = blockIdx.x, bh = blockIdx.y, units = gridDim.x;
    const int unit = bh * units + mt;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int j = threadIdx.x; j < Tn; j += 256) rows[j] = 0;
    __syncthreads();
    pdl_wait();                 // the lists come from the selection kernel launched before this one
    pdl_trigger();
    for (int e = threadIdx.x; e < G * keep; e += 256) {
        const int r = e / keep, jj = e - r * keep, qb = mt * G + r;
        if (qb < Tm) {
            const int j = checked_block(__ldg(idx + ((size_t)bh * Tm + qb) * keep + jj), Tn, dev_status, bh * Tm + qb);
            atomicOr(&rows[j], (1u << r) | (jj == 0 ? 0x100u : 0u));
        }
    }
    __syncthreads();
    // compaction: the first-kept blocks (ascending), then the rest of the union (ascending); thread t looks at blocks 4t .. 4t+3
    uint32_t w[4];
    int nA = 0, nB = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int j = threadIdx.x * 4 + i;
        w[i] = j < Tn ? rows[j] : 0u;
        nA += (w[i] & 0x100u) != 0;
        nB += (w[i] & 0xffu) != 0 && !(w[i] & 0x100u);
    }
    int pA = nA, pB = nB;       // inclusive scans inside the warp
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int a = __shfl_up_sync(0xffffffffu, pA, off), b = __shfl_up_sync(0xffffffffu, pB, off);
        if (lane >= off) { pA += a; pB += b; }
    }
    if (lane == 31) { warp_tot[0][warp] = pA; warp_tot[1][warp] = pB; }
    __syncthreads();
    int baseA = 0, baseB = 0, totA = 0, totB = 0;
#pragma unroll
    for (int x = 0; x < 8; ++x) {
        if (x < warp) { baseA += warp_tot[0][x]; baseB += warp_tot[1][x]; }
        totA += warp_tot[0][x]; totB += warp_tot[1][x];
    }
    int posA = baseA + pA - nA, posB = totA + baseB + pB - nB;
    uint32_t* out = entries + (size_t)unit * max_tiles * G;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int j = threadIdx.x * 4 + i;
        if ((w[i] & 0xffu) == 0) continue;
        int jb = j;
        while (jb >= n_b) jb -= n_b;
        const int nv = jb == n_b - 1 ? Tc - jb * BLK : BLK;
        const uint32_t ent = union_entry(j, w[i] & 0xffu, nv);
        if (w[i] & 0x100u) out[posA++] = ent; else out[posB++] = ent;
    }
    __syncthreads();
    const int total = totA + totB, n_tiles = (total + G - 1) / G;
    if (threadIdx.x < n_tiles * G - total) out[total + threadIdx.x] = union_entry((int)(out[0] & 1023u), 0u, BLK);
    if (threadIdx.x == 0) tiles[unit] = n_tiles;
}

struct Tc5GParams {
    const uint32_t* entries;     // [units, max_tiles, G] from k_union_tiles
    const int* tiles;            // [units]
    int max_tiles;
    int Tmt, n_units;            // units per batch*head; units in all
    const int32_t* idx;          // [B*H, T_m, keep]: the kept lists themselves (second pass with the running maximum)
    int keep, Tm;
    int Tc, n_b, n_cached, ring_head, P, n_sink;
    float scale_log2;
    const float* hist;           // optional fp32 [B*H, T_c, D]: history term added in the epilogue
    const bf16* q;
    bf16* o;
    float* lse;
    int* dev_status;
    ChunkTable tab;
};

template <int D, int BLK>
__global__ void __launch_bounds__(SwaTc5<D, 2>::THREADS, 1)
k_swa_tc5g(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kring,
           const __grid_constant__ CUtensorMap tm_vring, const __grid_constant__ CUtensorMap tm_kcur,
           const __grid_constant__ CUtensorMap tm_vcur, const __grid_constant__ CUtensorMap tm_o,
           const __grid_constant__ Tc5GParams p) {
    using namespace tc5;
    typedef SwaTc5<D, 2> C;
    constexpr int NG = 2;
    constexpr int G = 128 / BLK;                       // key blocks per tile = row groups per unit
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t s_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    if (s_base - smem_u32(smem_raw) + C::USED_BYTES > C::SMEM_BYTES) {
        if (threadIdx.x == 0) { atomicOr(p.dev_status, HF_DEV_TIMEOUT_FLAG); atomicExch(p.dev_status + 1, 98); }
        return;
    }
    uint8_t* s_gen = smem_raw + (s_base - smem_u32(smem_raw));
    const uint32_t sQ = s_base + C::OFF_Q, sK = s_base + C::OFF_K, sV = s_base + C::OFF_V;
    const uint32_t bar0 = s_base + C::OFF_BAR;
    const uint32_t bar_kf = bar0, bar_ke = bar0 + 24, bar_vf = bar0 + 48, bar_ve = bar0 + 64, bar_sf = bar0 + 80,
                   bar_pf = bar0 + 104, bar_pv = bar0 + 128, bar_mx = bar0 + 160, bar_qf = bar0 + 176, bar_qe = bar0 + 184,
                   bar_ep = bar0 + 192, bar_drain = bar0 + 200, bar_rd = bar0 + 216;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(s_gen + C::OFF_BAR + 208);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(s_gen + C::OFF_BAR + 212);
    constexpr int REDO_CAP = 8;
    int* redo_cnt = reinterpret_cast<int*>(s_gen + C::OFF_BAR + 264);
    int* redo_last = redo_cnt + 1;
    int* redo_list = redo_cnt + 2;
    float* x_max = reinterpret_cast<float*>(s_gen + C::OFF_XM);          // [2][NG][128]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int my_units = (p.n_units - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 3; ++s) { mbar_init(bar_kf + 8 * s, 1); mbar_init(bar_ke + 8 * s, 1); mbar_init(bar_sf + 8 * s, 1); mbar_init(bar_pf + 8 * s, 128 * NG); }
        for (int s = 0; s < 2; ++s) { mbar_init(bar_vf + 8 * s, 1); mbar_init(bar_ve + 8 * s, 1); mbar_init(bar_mx + 8 * s, 128 * NG); }
        for (int s = 0; s < 4; ++s) mbar_init(bar_pv + 8 * s, 1);
        mbar_init(bar_qf, 1); mbar_init(bar_qe, 1); mbar_init(bar_ep, 128 * NG); mbar_init(bar_drain, 1); mbar_init(bar_rd, 128 * NG);
        *abort_flag = 0;
        *redo_cnt = 0; *redo_last = -1;
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
    pdl_wait();                 // the tile lists come from k_union_tiles, launched before this kernel
    if (C::SMEM_BYTES > 200 * 1024) pdl_trigger();

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
                const int bh = u / p.Tmt, mt = u - bh * p.Tmt;
                const int cnt = __ldg(p.tiles + u);
                const uint32_t* ent = p.entries + (size_t)u * p.max_tiles * G;
                if (is_k) {   // Q of this unit, once the last S of the previous unit has read the buffer
                    if (n >= 1 && !(ok = mbar_wait<true>(bar_qe, (n - 1) & 1, abort_flag, p.dev_status, 1))) break;
                    mbar_expect_tx(bar_qf, C::TILE_BYTES);
#pragma unroll
                    for (int s = 0; s < C::SUB; ++s)
                        tma_load_4d(sQ + s * C::SUB_BYTES, &tm_q, s * 64, mt * 128, bh, 0, bar_qf);
                }
                for (int j = 0; j < cnt; ++j, ++t) {
                    uint32_t dst, bar;
                    if (is_k) {
                        if (t >= C::KSTAGES && !(ok = mbar_wait<true>(bar_ke + 8 * rk.stage, rk.phase ^ 1u, abort_flag, p.dev_status, 2))) break;
                        dst = sK + rk.stage * C::TILE_BYTES; bar = bar_kf + 8 * rk.stage;
                        rk.advance();
                    } else {
                        if (t >= C::VSTAGES && !(ok = mbar_wait<true>(bar_ve + 8 * rv.stage, rv.phase ^ 1u, abort_flag, p.dev_status, 3))) break;
                        dst = sV + rv.stage * C::TILE_BYTES; bar = bar_vf + 8 * rv.stage;
                        rv.advance();
                    }
                    mbar_expect_tx(bar, C::TILE_BYTES);
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        int blk = (int)(__ldg(ent + j * G + g) & 1023u);
                        if (blk >= Tn) blk = 0;                            // (the list builder has checked every entry already)
                        int c = 0, jb = blk;
                        while (jb >= p.n_b) { jb -= p.n_b; ++c; }
                        const bool cur = (c == p.n_sink + p.n_cached);
                        int slot = 0;
                        if (!cur) {
                            if (c < p.n_sink) slot = p.P + c;
                            else { slot = p.ring_head + c - p.n_sink; if (slot >= p.P) slot -= p.P; }
                        }
                        const CUtensorMap* m = is_k ? (cur ? &tm_kcur : &tm_kring) : (cur ? &tm_vcur : &tm_vring);
#pragma unroll
                        for (int s = 0; s < C::SUB; ++s)
                            tma_load_4d(dst + s * C::SUB_BYTES + g * BLK * 128, m, s * 64, jb * BLK, bh, slot, bar);
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
        const uint32_t tO = tmem + C::COL_O;
        const uint64_t dq0 = smem_desc_sw128(sQ, 16, 1024), dk0 = smem_desc_sw128(sK, 16, 1024);
        const uint64_t dv0 = smem_desc_sw128(sV, C::SUB_BYTES, 1024);
        const uint32_t q_lo = (uint32_t)dq0, k_lo = (uint32_t)dk0, v_lo = (uint32_t)dv0;
        const uint32_t qk_hi = (uint32_t)(dq0 >> 32), v_hi = (uint32_t)(dv0 >> 32);
        bool ok = true;
        int n_s = 0, j_s = 0;                         // unit and position in its tile list of the next S tile to issue
        int cnt_s = my_units > 0 ? __ldg(p.tiles + blockIdx.x) : 0;
        RingPos<C::KSTAGES> rk;
        RingPos<C::SBUFS> rb;
        auto issue_s = [&]() -> bool {                // S_t = Q K_t^T into S buffer t % 3
            if (j_s == 0 && !__all_sync(0xffffffffu, mbar_wait<true>(bar_qf, n_s & 1, abort_flag, p.dev_status, 4))) return false;
            if (!__all_sync(0xffffffffu, mbar_wait<true>(bar_kf + 8 * rk.stage, rk.phase, abort_flag, p.dev_status, 5))) return false;
            fence_after_sync();
            if (elect_one()) {
                mma_ss_tile<D>(tmem + rb.stage * 128, q_lo, k_lo + rk.stage * TILE_STEP, qk_hi, IDESC_S);
                mma_commit(bar_sf + 8 * rb.stage);
                mma_commit(bar_ke + 8 * rk.stage);
                if (j_s == cnt_s - 1) mma_commit(bar_qe);
            }
            __syncwarp();
            rk.advance();
            rb.advance();
            if (++j_s == cnt_s) {
                j_s = 0; ++n_s;
                cnt_s = n_s < my_units ? __ldg(p.tiles + blockIdx.x + n_s * gridDim.x) : 0;
            }
            return true;
        };
        if (n_s < my_units) ok = issue_s();
        if (ok && n_s < my_units) ok = issue_s();
        int t = 0;
        RingPos<C::SBUFS> rp;
        RingPos<C::VSTAGES> rv;
        for (int n = 0; ok && n < my_units; ++n) {
            const int cnt = __ldg(p.tiles + blockIdx.x + n * gridDim.x);
            for (int j = 0; ok && j < cnt; ++j, ++t) {
                if (n_s < my_units && !(ok = issue_s())) break;
                if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_pf + 8 * rp.stage, rp.phase, abort_flag, p.dev_status, 6)))) break;
                if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_vf + 8 * rv.stage, rv.phase, abort_flag, p.dev_status, 7)))) break;
                fence_after_sync();
                if (elect_one()) {
                    mma_ts_tile_split(tO, tmem + rp.stage * 128, tmem + rp.stage * 128 + C::GCOLS,
                                      v_lo + rv.stage * TILE_STEP, v_hi, IDESC_PV, j > 0);
                    mma_commit(bar_pv + 8 * (t & 3));
                    mma_commit(bar_ve + 8 * rv.stage);
                }
                __syncwarp();
                rp.advance();
                rv.advance();
            }
        }
        if (elect_one()) mma_commit(bar_drain);
        __syncwarp();
        {
            const long long t0 = clock64();
            while (!mbar_try_wait(bar_drain, 0) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
        }
    } else {
        // ================================================================= softmax / epilogue
        const int grp = warp >> 2;                          // column group: key columns [64 grp, 64 grp + 64) of a tile
        const int row = (warp & 3) * 32 + lane;             // query row of the unit = TMEM lane
        const int rg = row / BLK;                           // row group (query block within the unit)
        const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        const uint32_t tO = lane_base + C::COL_O + grp * C::OCOLS;
        constexpr int NC = C::GCOLS / 32;                   // 32-column register chunks of S per thread (2)
        constexpr int EPT = 64 / BLK;                       // list entries (key blocks) under this thread's 64 columns
        bool ok = true;
        int t = 0;
        RingPos<C::SBUFS> rs;
        auto note_redo = [&](int n) {
            if (atomicExch(redo_last, n) != n) {
                const int slot = atomicAdd(redo_cnt, 1);
                if (slot < REDO_CAP) redo_list[slot] = n;
            }
        };
        auto wait_pv_prev = [&](int where) -> bool {
            return __all_sync(0xffffffffu, mbar_wait(bar_pv + 8 * ((t - 1) & 3), ((t - 1) >> 2) & 1, abort_flag, p.dev_status, where));
        };
        for (int n = 0; ok && n < my_units; ++n) {
            const int u = blockIdx.x + n * gridDim.x;
            const int bh = u / p.Tmt, mt = u - bh * p.Tmt;
            const int q0 = mt * 128;
            const int nq = min(128, p.Tc - q0);
            const int cnt = __ldg(p.tiles + u);
            const uint32_t* ent = p.entries + (size_t)u * p.max_tiles * G + grp * EPT;
            float m_used = 0.f, l_run = 0.f;
            uint32_t e_next[EPT];                           // this thread's entries of the next tile, read one tile ahead
#pragma unroll
            for (int x = 0; x < EPT; ++x) e_next[x] = __ldg(ent + x);
            for (int j = 0; j < cnt; ++j, ++t) {
                uint32_t e_cur[EPT];
#pragma unroll
                for (int x = 0; x < EPT; ++x) e_cur[x] = e_next[x];
                if (j + 1 < cnt) {
#pragma unroll
                    for (int x = 0; x < EPT; ++x) e_next[x] = __ldg(ent + (j + 1) * G + x);
                }
                const uint32_t tS = lane_base + rs.stage * 128;
                ok = __all_sync(0xffffffffu, mbar_wait(bar_sf + 8 * rs.stage, rs.phase, abort_flag, p.dev_status, 8));
                if (!ok) break;
                rs.advance();
                fence_after_sync();
                uint32_t r[NC][32];
#pragma unroll
                for (int c = 0; c < NC; ++c) tmem_ld32(tS + grp * C::GCOLS + c * 32, r[c]);
                tmem_wait_ld();
                // ---- what this row does not keep, and the columns past a short block's end: -inf
#pragma unroll
                for (int x = 0; x < EPT; ++x) {
                    const bool kept = (e_cur[x] >> (10 + rg)) & 1u;
                    const int nv = kept ? (int)((e_cur[x] >> 18) & 127u) : 0;
                    if (nv < BLK) {
#pragma unroll
                        for (int e = 0; e < BLK; ++e)
                            if (e >= nv) r[(x * BLK + e) >> 5][(x * BLK + e) & 31] = 0xff800000u;
                    }
                }
                if (j == 0) {
                    // ---- the reference exponent of the row for the whole unit (see k_swa_tc5.cuh): maximum of the first
                    // tile, which holds the first kept block of every row group, times 2^HEADROOM
                    float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int c = 0; c < NC; ++c)
#pragma unroll
                        for (int e = 0; e < 32; e += 2)
                            mx[(e >> 1) & 3] = fmax3(mx[(e >> 1) & 3], __uint_as_float(r[c][e]), __uint_as_float(r[c][e + 1]));
                    float mrow = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                    float* xm = x_max + (n & 1) * NG * 128;
                    xm[grp * 128 + row] = mrow;
                    mbar_arrive(bar_mx + 8 * (n & 1));
                    ok = __all_sync(0xffffffffu, mbar_wait(bar_mx + 8 * (n & 1), (n >> 1) & 1, abort_flag, p.dev_status, 11));
                    if (!ok) break;
#pragma unroll
                    for (int g = 0; g < NG; ++g) mrow = fmaxf(mrow, xm[g * 128 + row]);
                    mbar_arrive(bar_rd);
                    // rows of a row group past the last query block keep nothing at all: any finite reference will do
                    m_used = mrow == -INFINITY ? 0.f : fmaf(mrow, p.scale_log2, C::HEADROOM);
                }
                float2 rsum[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                const float2 scale2 = make_float2(p.scale_log2, p.scale_log2), negm2 = make_float2(-m_used, -m_used);
#pragma unroll
                for (int c = 0; c < NC; ++c) {
                    uint32_t pk[16];
#pragma unroll
                    for (int e0 = 0; e0 < 32; e0 += 8) {
                        float2 x[4], pe[4];
#pragma unroll
                        for (int v = 0; v < 4; ++v)
                            x[v] = ffma2(make_float2(__uint_as_float(r[c][e0 + 2 * v]), __uint_as_float(r[c][e0 + 2 * v + 1])), scale2, negm2);
#pragma unroll
                        for (int v = 0; v < 4; ++v) pe[v] = make_float2(fast_exp2(x[v].x), fast_exp2(x[v].y));
#pragma unroll
                        for (int v = 0; v < 4; ++v) rsum[v] = fadd2(rsum[v], pe[v]);
#pragma unroll
                        for (int v = 0; v < 4; ++v) pk[(e0 >> 1) + v] = pack_bf16_alu(pe[v].x, pe[v].y);
                    }
                    tmem_st16(tS + grp * C::GCOLS + c * 16, pk);
                }
                l_run += ((rsum[0].x + rsum[0].y) + (rsum[1].x + rsum[1].y)) + ((rsum[2].x + rsum[2].y) + (rsum[3].x + rsum[3].y));
                tmem_wait_st();
                fence_before_sync();
                mbar_arrive(bar_pf + 8 * (rs.stage == 0 ? C::SBUFS - 1 : rs.stage - 1));
            }
            if (!ok) break;
            // ---- end of the unit: row sums of the two column groups, range test, output
            ok = __all_sync(0xffffffffu, mbar_wait(bar_rd, n & 1, abort_flag, p.dev_status, 17));
            if (!ok) break;
            float* x_l = x_max + (n & 1) * NG * 128;
            x_l[grp * 128 + row] = l_run;
            mbar_arrive(bar_ep);
            ok = __all_sync(0xffffffffu, mbar_wait(bar_ep, n & 1, abort_flag, p.dev_status, 12));
            if (!ok) break;
            l_run = x_l[row] + x_l[128 + row];
            ok = wait_pv_prev(10);
            if (!ok) break;
            fence_after_sync();
            const float inv = 1.f / l_run;
            if (!(l_run < 1e30f)) note_redo(n);         // overflow (or NaN): a later tile rose too far above the first one
            const size_t g_row = (size_t)bh * p.Tc + q0 + row;
            if (grp == 0 && row < nq && p.lse) p.lse[g_row] = (m_used + log2f(l_run)) * 0.6931471805599453f;
            if constexpr (C::FUSE) {
                // output through shared memory and one bulk tensor store per warp (32 rows x 64 columns)
                uint8_t* stage = s_gen + C::OFF_H + grp * C::SUB_BYTES + (warp & 3) * 4096 + lane * 128;
                if (lane == 0) bulk_wait_read();            // this warp's previous store has read its part
                __syncwarp();
#pragma unroll
                for (int c = 0; c < C::OCOLS / 32; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tO + c * 32, o);
                    tmem_wait_ld();
                    const float* hsrc = p.hist ? p.hist + g_row * D + grp * C::OCOLS + c * 32 : nullptr;
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        float x[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) x[e] = __uint_as_float(o[v * 8 + e]) * inv;
                        if (hsrc && row < nq) {
                            const float4 h0 = *reinterpret_cast<const float4*>(hsrc + v * 8);
                            const float4 h1 = *reinterpret_cast<const float4*>(hsrc + v * 8 + 4);
                            x[0] += h0.x; x[1] += h0.y; x[2] += h0.z; x[3] += h0.w;
                            x[4] += h1.x; x[5] += h1.y; x[6] += h1.z; x[7] += h1.w;
                        }
                        uint4 w;
                        w.x = pack_bf16(x[0], x[1]); w.y = pack_bf16(x[2], x[3]);
                        w.z = pack_bf16(x[4], x[5]); w.w = pack_bf16(x[6], x[7]);
                        *reinterpret_cast<uint4*>(stage + (((c * 4 + v) ^ (lane & 7)) << 4)) = w;
                    }
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0 && q0 + (warp & 3) * 32 < p.Tc) {     // rows past the chunk's end are clipped by the map
                    tma_store_4d(&tm_o, s_base + C::OFF_H + grp * C::SUB_BYTES + (warp & 3) * 4096, grp * 64, q0 + (warp & 3) * 32, bh, 0);
                    bulk_commit();
                }
            } else {
#pragma unroll
                for (int c = 0; c < C::OCOLS / 32; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tO + c * 32, o);
                    tmem_wait_ld();
                    if (row < nq) {
                        const size_t off = g_row * D + grp * C::OCOLS + c * 32;
                        bf16* dst = p.o + off;
                        const float* hsrc = p.hist ? p.hist + off : nullptr;
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            float x[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e) x[e] = __uint_as_float(o[v * 8 + e]) * inv;
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
            }
            fence_before_sync();
        }
    }
    if (C::FUSE && warp < 4 * NG && lane == 0) bulk_wait_all();     // output tiles still on their way out of shared memory
    fence_before_sync();
    __syncthreads();
    if (warp == C::WARP_MMA) {
        fence_after_sync();
        tmem_dealloc(tmem, C::TMEM_COLS);
    }
    // ---- second pass (rare): the listed units again, query block by query block, with the running maximum
    const int n_redo = *redo_cnt;
    if (n_redo > 0 && *abort_flag == 0 && threadIdx.x < SwaMma<BLK, D>::THREADS) {
        fence_proxy_async();
        const int total = n_redo > REDO_CAP ? my_units : n_redo;
        for (int r = 0; r < total; ++r) {
            const int n = n_redo > REDO_CAP ? r : redo_list[r];
            const int u = (int)blockIdx.x + n * (int)gridDim.x;
            const int bh = u / p.Tmt, mt = u - bh * p.Tmt;
            for (int g = 0; g < G; ++g) {
                const int qb = mt * G + g;
                if (qb >= p.Tm) break;
                if (threadIdx.x == 0) atomicAdd(p.dev_status + 2, 1);
                swa_mma_unit<BLK, D>(s_gen, p.q, p.tab, p.idx + ((size_t)bh * p.Tm + qb) * p.keep, p.keep, p.Tc, p.n_b, p.scale_log2,
                                     p.hist ? p.hist + ((size_t)bh * p.Tc + (size_t)qb * BLK) * D : nullptr, p.o, p.lse, p.dev_status,
                                     qb, bh, bh * p.Tm + qb);
            }
        }
    }
}
