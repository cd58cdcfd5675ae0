// Block-sparse sliding-window attention (Eq. 6; Alg. 3 inner loops) on the warp-level tensor path
// (ldmatrix + mma.sync).  Generic over block size {16, 64, 128} and head dim {64, 128}: it is the
// path for the small-block shapes and the cross-check for the tcgen05 kernel.
//
// One CTA per (query block, batch*head); BLK/16 warps, each owning 16 query rows.  The kept key
// blocks of the row are streamed through two shared-memory stages with cp.async; per block
// S = Q K^T (fp32), running max / sum in the exp2 domain, P rounded to bf16, O += P V (fp32).
#pragma once
#include "hf_common.cuh"

template <int BLK, int D>
struct SwaMma {
    static constexpr int WARPS = BLK / 16;
    static constexpr int THREADS = WARPS * 32;
    static constexpr int ROW_BYTES = D * 2;
    static constexpr int TILE_BYTES = BLK * ROW_BYTES;
    static constexpr int SMEM_BYTES = 5 * TILE_BYTES;          // Q + 2 x (K, V)
    static constexpr int CHUNKS_PER_ROW = D / 8;
    static constexpr int CHUNKS_PER_THREAD = (BLK * CHUNKS_PER_ROW) / THREADS;   // = D / 16
};

template <int BLK, int D>
__device__ __forceinline__ void swa_load_tile(uint32_t smem_tile, const bf16* __restrict__ src, int n_valid) {
    typedef SwaMma<BLK, D> C;
#pragma unroll
    for (int i = 0; i < C::CHUNKS_PER_THREAD; ++i) {
        const int id = threadIdx.x + i * C::THREADS;
        const int row = id / C::CHUNKS_PER_ROW, ch = id % C::CHUNKS_PER_ROW;
        const bool ok = row < n_valid;
        cp_async16(smem_tile + swz<C::ROW_BYTES>(row, ch), src + (ok ? (size_t)row * D + ch * 8 : 0), ok);
    }
}

// One (batch*head, query block) unit with the first SwaMma::THREADS threads of the thread block (thread index tid), in the
// shared-memory window starting at `smem` (SwaMma::SMEM_BYTES, 128-byte aligned).  The participating threads meet on
// named barrier 1, so the function can run inside a larger thread block (the tcgen05 kernel calls it for the units it
// hands back, see k_swa_tc5.cuh) as well as be the whole body of k_swa_mma.
// hist_rows: optional fp32 rows [nq, D] of the unit (row stride D; global or shared memory), added to the normalised
// output before the single rounding to bf16.
template <int BLK, int D>
__device__ __forceinline__ void swa_mma_unit(uint8_t* smem, const bf16* __restrict__ q, const ChunkTable& tab,
                                             const int32_t* __restrict__ my_idx, int keep, int Tc, int n_b, float scale_log2,
                                             const float* hist_rows, bf16* __restrict__ o, float* __restrict__ lse,
                                             int* dev_status, int i, int bh, int unit) {
    typedef SwaMma<BLK, D> C;
    auto sync_unit = [] { asm volatile("bar.sync 1, %0;\n" ::"n"(C::THREADS) : "memory"); };
    typedef SwaMma<BLK, D> C;
    const uint32_t sQ = smem_u32(smem);
    const uint32_t sKV = sQ + C::TILE_BYTES;   // stage s: K at sKV + s*2*TILE, V right after

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int q0 = i * BLK;
    const int nq = min(BLK, Tc - q0);

    const int Tn = tab.n_chunks * n_b;
    auto issue = [&](int it, int stage) {
        const int j = checked_block(my_idx[it], Tn, dev_status, unit);
        const int c = j / n_b, jb = j - c * n_b;
        const int nv = min(BLK, Tc - jb * BLK);
        const size_t off = ((size_t)bh * Tc + (size_t)jb * BLK) * D;
        swa_load_tile<BLK, D>(sKV + stage * 2 * C::TILE_BYTES, tab.k[c] + off, nv);
        swa_load_tile<BLK, D>(sKV + stage * 2 * C::TILE_BYTES + C::TILE_BYTES, tab.v[c] + off, nv);
    };

    swa_load_tile<BLK, D>(sQ, q + ((size_t)bh * Tc + q0) * D, nq);
    issue(0, 0);
    cp_async_commit();

    float o_acc[D / 8][4];
#pragma unroll
    for (int n = 0; n < D / 8; ++n) { o_acc[n][0] = o_acc[n][1] = o_acc[n][2] = o_acc[n][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY};
    float l_run[2] = {0.f, 0.f};

    for (int it = 0; it < keep; ++it) {
        const int stage = it & 1;
        if (it + 1 < keep) issue(it + 1, stage ^ 1);
        cp_async_commit();
        cp_async_wait<1>();
        sync_unit();

        const int j = checked_block(my_idx[it], Tn, nullptr, 0);
        const int jb = j % n_b;
        const int nv = min(BLK, Tc - jb * BLK);
        const uint32_t sK = sKV + stage * 2 * C::TILE_BYTES, sV = sK + C::TILE_BYTES;

        // ---- S = Q K^T
        float s[BLK / 8][4];
#pragma unroll
        for (int n = 0; n < BLK / 8; ++n) { s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
            uint32_t a0, a1, a2, a3;
            ldsm_x4(sQ + swz<C::ROW_BYTES>(warp * 16 + (lane & 15), ks * 2 + (lane >> 4)), a0, a1, a2, a3);
#pragma unroll
            for (int np = 0; np < BLK / 16; ++np) {
                uint32_t b0, b1, b2, b3;
                ldsm_x4(sK + swz<C::ROW_BYTES>(np * 16 + (lane & 7) + ((lane >> 4) << 3), ks * 2 + ((lane >> 3) & 1)),
                        b0, b1, b2, b3);
                mma_bf16(s[2 * np], a0, a1, a2, a3, b0, b1);
                mma_bf16(s[2 * np + 1], a0, a1, a2, a3, b2, b3);
            }
        }
        // ---- mask the padded columns of a short key block
        if (nv < BLK) {
#pragma unroll
            for (int n = 0; n < BLK / 8; ++n) {
                const int c0 = n * 8 + 2 * (lane & 3);
                if (c0 >= nv) { s[n][0] = -INFINITY; s[n][2] = -INFINITY; }
                if (c0 + 1 >= nv) { s[n][1] = -INFINITY; s[n][3] = -INFINITY; }
            }
        }
        // ---- running max / sum (rows g = lane/4 and g + 8)
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int n = 0; n < BLK / 8; ++n) {
            mx[0] = fmaxf(mx[0], fmaxf(s[n][0], s[n][1]));
            mx[1] = fmaxf(mx[1], fmaxf(s[n][2], s[n][3]));
        }
        float alpha[2], m_new[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
            m_new[r] = fmaxf(m_run[r], mx[r] * scale_log2);
            alpha[r] = fast_exp2(m_run[r] - m_new[r]);
            m_run[r] = m_new[r];
        }
        float rs[2] = {0.f, 0.f};
#pragma unroll
        for (int n = 0; n < BLK / 8; ++n) {
            s[n][0] = fast_exp2(fmaf(s[n][0], scale_log2, -m_new[0]));
            s[n][1] = fast_exp2(fmaf(s[n][1], scale_log2, -m_new[0]));
            s[n][2] = fast_exp2(fmaf(s[n][2], scale_log2, -m_new[1]));
            s[n][3] = fast_exp2(fmaf(s[n][3], scale_log2, -m_new[1]));
            rs[0] += s[n][0] + s[n][1];
            rs[1] += s[n][2] + s[n][3];
        }
        l_run[0] = l_run[0] * alpha[0] + rs[0];
        l_run[1] = l_run[1] * alpha[1] + rs[1];
#pragma unroll
        for (int n = 0; n < D / 8; ++n) {
            o_acc[n][0] *= alpha[0]; o_acc[n][1] *= alpha[0];
            o_acc[n][2] *= alpha[1]; o_acc[n][3] *= alpha[1];
        }
        // ---- O += P V
#pragma unroll
        for (int kk = 0; kk < BLK / 16; ++kk) {
            const uint32_t a0 = pack_bf16(s[2 * kk][0], s[2 * kk][1]);
            const uint32_t a1 = pack_bf16(s[2 * kk][2], s[2 * kk][3]);
            const uint32_t a2 = pack_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1]);
            const uint32_t a3 = pack_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
            for (int dp = 0; dp < D / 16; ++dp) {
                uint32_t b0, b1, b2, b3;
                ldsm_x4_t(sV + swz<C::ROW_BYTES>(kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3), dp * 2 + (lane >> 4)),
                          b0, b1, b2, b3);
                mma_bf16(o_acc[2 * dp], a0, a1, a2, a3, b0, b1);
                mma_bf16(o_acc[2 * dp + 1], a0, a1, a2, a3, b2, b3);
            }
        }
        sync_unit();       // every warp is done with this stage before the next prefetch overwrites it
    }
    cp_async_wait<0>();

    // ---- epilogue
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int row = warp * 16 + (lane >> 2) + r * 8;
        if (row >= nq) continue;
        const float inv = 1.f / l_run[r];
        const size_t g = ((size_t)bh * Tc + q0 + row);
        if (lse && (lane & 3) == 0) lse[g] = (m_run[r] + log2f(l_run[r])) * 0.6931471805599453f;
#pragma unroll
        for (int n = 0; n < D / 8; ++n) {
            const int col = n * 8 + 2 * (lane & 3);
            float x0 = o_acc[n][2 * r] * inv, x1 = o_acc[n][2 * r + 1] * inv;
            if (hist_rows) {
                const float2 h = *reinterpret_cast<const float2*>(hist_rows + (size_t)row * D + col);
                x0 += h.x; x1 += h.y;
            }
            *reinterpret_cast<uint32_t*>(o + g * D + col) = pack_bf16(x0, x1);
        }
    }
}

// hist: optional fp32 [B*H, T_c, D] added to the normalised output before the single rounding to bf16.
template <int BLK, int D>
__global__ void __launch_bounds__(SwaMma<BLK, D>::THREADS)
k_swa_mma(const bf16* __restrict__ q, ChunkTable tab, const int32_t* __restrict__ idx, int keep,
          int Tc, int n_b, float scale_log2, const float* __restrict__ hist,
          bf16* __restrict__ o, float* __restrict__ lse, int* dev_status) {
    extern __shared__ __align__(128) uint8_t smem[];
    const int i = blockIdx.x, bh = blockIdx.y;
    const int unit = bh * gridDim.x + i;
    swa_mma_unit<BLK, D>(smem, q, tab, idx + (size_t)unit * keep, keep, Tc, n_b, scale_log2,
                         hist ? hist + ((size_t)bh * Tc + (size_t)i * BLK) * D : nullptr, o, lse, dev_status, i, bh, unit);
}
