// Backward of the history read-out (Eq. 4 with the Linear folded into the state) with respect to the queries.
//
// Forward, per query row r of a (batch, head):  f = phi(q_r),  den = f . z + eps,  y_r = (f S') / den + bias,
// S' = S W^T the folded state.  With g_r = dL/dy_r:
//     u   = S' g_r                      (u[a] = sum_c S'[a, c] g_r[c])           -- the one contraction: U = G S'^T
//     df  = (u - (f . u / den) z) / den
//     dq_r = df * phi'(q_r),            phi'(x) = 1 for x > 0, e^x otherwise
// The state itself comes from evicted chunks of earlier, gradient-free passes of the rollout (Alg. 1 back-propagates
// through the sampled step only), so nothing flows into S, z or the cached K / V here.
//
// Persistent kernel; a thread block takes a contiguous range of (batch*head, 128-row tile) units:
//   warp 4   TMA: the tile of G (bf16, K-major, 128-byte swizzle; two buffers) and, when the (batch, head) changes, the
//            hi and lo halves of S' ([a][c] bf16 -- as the B operand that is N = a by K = c, K-major)
//   warp 5   tcgen05.mma: U = G S'_hi^T + G S'_lo^T into one of two TMEM accumulators (D columns each)
//   warps 0-3  thread = row: two passes over U in 32-column chunks (TMEM is read twice; q and z come through L1):
//            f . u and f . z first, then df, dq -> bf16 -> global
// Every wait is bounded; on expiry the thread block raises the device status word and leaves through the common exit.
#pragma once
#include "tc5_common.cuh"

template <int D>
struct ReadoutBwd {
    static constexpr int ROWS = 128;
    static constexpr int SUB = D / 64;
    static constexpr int G_BYTES = ROWS * D * 2, S_BYTES = D * D * 2;
    static constexpr int OFF_G = 0, OFF_S = 2 * G_BYTES, OFF_BAR = OFF_S + 2 * S_BYTES;
    static constexpr int SMEM_BYTES = OFF_BAR + 128 + 1024;
    static constexpr int THREADS = 192, WARP_TMA = 4, WARP_MMA = 5;
    static constexpr int TMEM_COLS = 2 * D < 32 ? 32 : 2 * D;
};

struct ReadoutBwdParams {
    const bf16* q;            // [B*H, T_c, D]
    const float* z;           // [B*H, D]
    bf16* dq;                 // [B*H, T_c, D]
    int Tc, Tm, n_units;
    float eps;
    int* dev_status;
};

// tm_g: [D, T_c, B*H, 1] box {64, 128}; tm_sh, tm_sl: [D, D, B*H, 1] box {64, D}; all 128-byte swizzle.
template <int D>
__global__ void __launch_bounds__(ReadoutBwd<D>::THREADS, 1)
k_readout_bwd_dq(const __grid_constant__ CUtensorMap tm_g, const __grid_constant__ CUtensorMap tm_sh,
                 const __grid_constant__ CUtensorMap tm_sl, const ReadoutBwdParams p) {
    using namespace tc5;
    typedef ReadoutBwd<D> C;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t s_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* s_gen = smem_raw + (s_base - smem_u32(smem_raw));
    const uint32_t bar0 = s_base + C::OFF_BAR;
    const uint32_t bar_gfull = bar0, bar_gfree = bar0 + 16, bar_ufull = bar0 + 32, bar_ufree = bar0 + 48, bar_sfull = bar0 + 64,
                   bar_drain = bar0 + 72;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(s_gen + C::OFF_BAR + 80);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(s_gen + C::OFF_BAR + 84);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int upc = (p.n_units + (int)gridDim.x - 1) / (int)gridDim.x;
    const int u0 = min((int)blockIdx.x * upc, p.n_units);
    const int my_units = min(upc, p.n_units - u0);

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar_gfull + 8 * s, 1); mbar_init(bar_gfree + 8 * s, 1);
            mbar_init(bar_ufull + 8 * s, 1); mbar_init(bar_ufree + 8 * s, 128);
        }
        mbar_init(bar_sfull, 1); mbar_init(bar_drain, 1);
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

    if (warp == C::WARP_TMA) {
        if (lane == 0) {
            bool ok = true;
            int bh_prev = -1;
            for (int n = 0; ok && n < my_units; ++n) {
                const int u = u0 + n;
                const int bh = u / p.Tm, i = u - bh * p.Tm;
                const int s = n & 1;
                if (bh != bh_prev) {
                    // the products of the previous unit (the last one of the other head) have read S'
                    if (n >= 1 && !(ok = mbar_wait<true>(bar_gfree + 8 * ((n - 1) & 1), ((n - 1) >> 1) & 1, abort_flag, p.dev_status, 61))) break;
                    bh_prev = bh;
                    mbar_expect_tx(bar_sfull, 2 * C::S_BYTES);
#pragma unroll
                    for (int v = 0; v < C::SUB; ++v) {
                        tma_load_4d(s_base + C::OFF_S + v * D * 128, &tm_sh, v * 64, 0, bh, 0, bar_sfull);
                        tma_load_4d(s_base + C::OFF_S + C::S_BYTES + v * D * 128, &tm_sl, v * 64, 0, bh, 0, bar_sfull);
                    }
                }
                if (n >= 2 && !(ok = mbar_wait<true>(bar_gfree + 8 * s, ((n >> 1) & 1) ^ 1, abort_flag, p.dev_status, 62))) break;
                mbar_expect_tx(bar_gfull + 8 * s, C::G_BYTES);
#pragma unroll
                for (int v = 0; v < C::SUB; ++v)
                    tma_load_4d(s_base + C::OFF_G + s * C::G_BYTES + v * C::ROWS * 128, &tm_g, v * 64, i * C::ROWS, bh, 0, bar_gfull + 8 * s);
            }
            if (!ok) {   // gave up: let the copies already in flight land before the thread block leaves
                const long long t0 = clock64();
                while (clock64() - t0 < 400000) {}
            }
        }
    } else if (warp == C::WARP_MMA) {
        constexpr uint32_t IDESC = idesc_bf16(D, false);
        bool ok = true;
        int bh_prev = -1, epoch = -1;
        for (int n = 0; ok && n < my_units; ++n) {
            const int s = n & 1;
            const uint32_t par = (n >> 1) & 1;
            const int bh = (u0 + n) / p.Tm;
            if (bh != bh_prev) {
                bh_prev = bh; ++epoch;
                if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_sfull, epoch & 1, abort_flag, p.dev_status, 63)))) break;
            }
            if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_gfull + 8 * s, par, abort_flag, p.dev_status, 64)))) break;
            if (n >= 2 && !(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_ufree + 8 * s, par ^ 1u, abort_flag, p.dev_status, 65)))) break;
            fence_after_sync();
            if (elect_one()) {
                const uint32_t tU = tmem + s * D;
                const uint64_t dg = smem_desc_sw128(s_base + C::OFF_G + s * C::G_BYTES, 16, 1024);
                const uint64_t dsh = smem_desc_sw128(s_base + C::OFF_S, 16, 1024);
                const uint64_t dsl = smem_desc_sw128(s_base + C::OFF_S + C::S_BYTES, 16, 1024);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    // 16 contraction columns = 32 bytes inside a 128-byte row; the next 64-column sub-tile is ROWS (or D) rows on
                    const uint64_t og = (uint64_t)(((ks >> 2) * C::ROWS * 128 + (ks & 3) * 32) >> 4);
                    const uint64_t os = (uint64_t)(((ks >> 2) * D * 128 + (ks & 3) * 32) >> 4);
                    mma_ss(tU, dg + og, dsh + os, IDESC, ks > 0);
                    mma_ss(tU, dg + og, dsl + os, IDESC, true);
                }
                mma_commit(bar_ufull + 8 * s);
                mma_commit(bar_gfree + 8 * s);
            }
            __syncwarp();
        }
        if (elect_one()) mma_commit(bar_drain);
        __syncwarp();
        {
            const long long t0 = clock64();
            while (!mbar_try_wait(bar_drain, 0) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
        }
    } else {
        const int row = warp * 32 + lane;
        const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
        bool ok = true;
        for (int n = 0; ok && n < my_units; ++n) {
            const int u = u0 + n;
            const int bh = u / p.Tm, i = u - bh * p.Tm;
            const int s = n & 1;
            const int r = i * C::ROWS + row;
            const bool valid = r < p.Tc;
            const bf16* q_row = p.q + ((size_t)bh * p.Tc + (valid ? r : 0)) * D;
            const float* z_row = p.z + (size_t)bh * D;
            ok = __all_sync(0xffffffffu, mbar_wait(bar_ufull + 8 * s, (n >> 1) & 1, abort_flag, p.dev_status, 66));
            if (!ok) break;
            fence_after_sync();
            const uint32_t tU = lane_base + s * D;
            // ---- pass 1: f . u and f . z
            float fu = 0.f, fz = 0.f;
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
                uint32_t uu[32];
                tmem_ld32(tU + c * 32, uu);
                uint4 qw[4];
#pragma unroll
                for (int v = 0; v < 4; ++v) qw[v] = __ldg(reinterpret_cast<const uint4*>(q_row + c * 32) + v);
                tmem_wait_ld();
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const uint32_t ws[4] = {qw[v].x, qw[v].y, qw[v].z, qw[v].w};
                    const float4 z0 = __ldg(reinterpret_cast<const float4*>(z_row + c * 32 + v * 8));
                    const float4 z1 = __ldg(reinterpret_cast<const float4*>(z_row + c * 32 + v * 8 + 4));
                    const float zz[8] = {z0.x, z0.y, z0.z, z0.w, z1.x, z1.y, z1.z, z1.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 x = unpack_bf16(ws[e]);
                        const float f0 = phi_elu1(x.x), f1 = phi_elu1(x.y);
                        fu = fmaf(f0, __uint_as_float(uu[v * 8 + 2 * e]), fmaf(f1, __uint_as_float(uu[v * 8 + 2 * e + 1]), fu));
                        fz = fmaf(f0, zz[2 * e], fmaf(f1, zz[2 * e + 1], fz));
                    }
                }
            }
            const float inv = 1.f / (fz + p.eps);
            const float ratio = fu * inv;
            // ---- pass 2: df = (u - ratio z) / den, dq = df phi'(q)
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
                uint32_t uu[32];
                tmem_ld32(tU + c * 32, uu);
                uint4 qw[4];
#pragma unroll
                for (int v = 0; v < 4; ++v) qw[v] = __ldg(reinterpret_cast<const uint4*>(q_row + c * 32) + v);
                tmem_wait_ld();
                if (c == D / 32 - 1) {          // U is in registers: the accumulator may take the unit after the next
                    fence_before_sync();
                    mbar_arrive(bar_ufree + 8 * s);
                }
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const uint32_t ws[4] = {qw[v].x, qw[v].y, qw[v].z, qw[v].w};
                    const float4 z0 = __ldg(reinterpret_cast<const float4*>(z_row + c * 32 + v * 8));
                    const float4 z1 = __ldg(reinterpret_cast<const float4*>(z_row + c * 32 + v * 8 + 4));
                    const float zz[8] = {z0.x, z0.y, z0.z, z0.w, z1.x, z1.y, z1.z, z1.w};
                    uint32_t w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 x = unpack_bf16(ws[e]);
                        const float d0 = fmaf(-ratio, zz[2 * e], __uint_as_float(uu[v * 8 + 2 * e])) * inv;
                        const float d1 = fmaf(-ratio, zz[2 * e + 1], __uint_as_float(uu[v * 8 + 2 * e + 1])) * inv;
                        // phi'(x): 1 above zero, e^x (= phi(x)) at and below it
                        w[e] = pack_bf16(x.x > 0.f ? d0 : d0 * phi_elu1(x.x), x.y > 0.f ? d1 : d1 * phi_elu1(x.y));
                    }
                    if (valid) *(reinterpret_cast<uint4*>(p.dq + ((size_t)bh * p.Tc + r) * D + c * 32) + v) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
        }
    }
    fence_before_sync();
    __syncthreads();
    if (warp == C::WARP_MMA) {
        fence_after_sync();
        tmem_dealloc(tmem, C::TMEM_COLS);
    }
}
