// Linear-attention state kernels off the tcgen05 path:
//   k_absorb_mma   Eq. 3, first half, on the warp-level tensor path (ldmatrix + mma.sync): per (batch, head) the token
//                  range is split over thread blocks, each writing its partial phi(K_ev)^T V_ev and sum_t phi(K_ev[t])
//                  to scratch.  Used by the entry point that may not allocate; the context's path is k_absorb_tc5.
//   k_reduce_fold  Eq. 3, second half: S, z += the partials in a fixed order (deterministic), then
//                  S' = S W^T split into bf16 hi/lo halves (the per-row divisor of Eq. 4 commutes with W)
// phi(K) is carried as a bf16 hi + lo pair so that the products keep ~16 mantissa bits; accumulation is fp32.
#pragma once
#include "hf_common.cuh"

template <int D>
struct AbsorbMma {
    static constexpr int THREADS = D * 2;          // D/16 warps, each owning 16 state rows (key features)
    static constexpr int TT = 64;                  // tokens per shared-memory tile
    static constexpr int ROW_BYTES = D * 2;
    static constexpr int TILE_BYTES = TT * ROW_BYTES;
    static constexpr int STAGES = 3;
    static constexpr int SMEM_BYTES = STAGES * 2 * TILE_BYTES;   // stages x (K, V)
    static constexpr int CHUNKS_PER_ROW = D / 8;
    static constexpr int CHUNKS_PER_THREAD = (TT * CHUNKS_PER_ROW) / THREADS;   // = 4
    static constexpr int PART_FLOATS = D * D + D;  // one partial: S then z
};

template <int D>
__device__ __forceinline__ void absorb_load_tile(uint32_t smem_tile, const bf16* __restrict__ src, int n_valid) {
    typedef AbsorbMma<D> C;
#pragma unroll
    for (int i = 0; i < C::CHUNKS_PER_THREAD; ++i) {
        const int id = threadIdx.x + i * C::THREADS;
        const int row = id / C::CHUNKS_PER_ROW, ch = id % C::CHUNKS_PER_ROW;
        const bool ok = row < n_valid;
        cp_async16(smem_tile + swz<C::ROW_BYTES>(row, ch), src + (ok ? (size_t)row * D + ch * 8 : 0), ok);
    }
}

// grid (nsplit, B*H).  k_ev, v_ev: [B*H, n_tokens, D].  partials: [B*H, nsplit, D*D + D] scratch, every element
// of which is written (S part, then z part); k_reduce_fold adds them to the state.
template <int D>
__global__ void __launch_bounds__(AbsorbMma<D>::THREADS)
k_absorb_mma(const bf16* __restrict__ k_ev, const bf16* __restrict__ v_ev, int n_tokens, float* __restrict__ partials) {
    typedef AbsorbMma<D> C;
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t s0 = smem_u32(smem);
    const int split = blockIdx.x, nsplit = gridDim.x, bh = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    // token range of this split, in whole tiles
    const int n_tiles = (n_tokens + C::TT - 1) / C::TT;
    const int tile_lo = (int)(((long long)n_tiles * split) / nsplit);
    const int tile_hi = (int)(((long long)n_tiles * (split + 1)) / nsplit);
    const bf16* kb = k_ev + (size_t)bh * n_tokens * D;
    const bf16* vb = v_ev + (size_t)bh * n_tokens * D;

    auto issue = [&](int tile, int stage) {
        if (tile < tile_hi) {
            const int t0 = tile * C::TT;
            const int nv = min(C::TT, n_tokens - t0);
            absorb_load_tile<D>(s0 + stage * 2 * C::TILE_BYTES, kb + (size_t)t0 * D, nv);
            absorb_load_tile<D>(s0 + stage * 2 * C::TILE_BYTES + C::TILE_BYTES, vb + (size_t)t0 * D, nv);
        }
        cp_async_commit();      // one group per call, empty past the end, so that the wait below counts uniformly
    };

    float acc[D / 8][4];
#pragma unroll
    for (int n = 0; n < D / 8; ++n) { acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f; }
    float zs[2] = {0.f, 0.f};

#pragma unroll
    for (int s = 0; s < C::STAGES - 1; ++s) issue(tile_lo + s, s);
    int stage = 0;
    for (int tile = tile_lo; tile < tile_hi; ++tile) {
        cp_async_wait<C::STAGES - 2>();
        __syncthreads();          // tile landed for every thread; the stage refilled below was read in the previous pass
        issue(tile + C::STAGES - 1, (stage + C::STAGES - 1) % C::STAGES);
        const uint32_t sK = s0 + stage * 2 * C::TILE_BYTES, sV = sK + C::TILE_BYTES;
        const int nv = min(C::TT, n_tokens - tile * C::TT);
#pragma unroll
        for (int ks = 0; ks < C::TT / 16; ++ks) {
            // A = phi(K)^T: rows = key features warp*16.., columns = tokens ks*16..
            uint32_t r[4];
            ldsm_x4_t(sK + swz<C::ROW_BYTES>(ks * 16 + (lane & 7) + ((lane >> 4) << 3), warp * 2 + ((lane >> 3) & 1)),
                      r[0], r[1], r[2], r[3]);
            uint32_t ahi[4], alo[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                float2 kv = unpack_bf16(r[x]);
                float f0 = phi_elu1(kv.x), f1 = phi_elu1(kv.y);
                if (nv < C::TT) {   // padded token rows contribute nothing (phi(0) = 1 otherwise)
                    const int t = ks * 16 + 2 * (lane & 3) + ((x >> 1) << 3);
                    if (t >= nv) f0 = 0.f;
                    if (t + 1 >= nv) f1 = 0.f;
                }
                zs[x & 1] += f0 + f1;
                const __nv_bfloat16 h0 = __float2bfloat16_rn(f0), h1 = __float2bfloat16_rn(f1);
                ahi[x] = pack_bf16(f0, f1);
                alo[x] = pack_bf16(f0 - __bfloat162float(h0), f1 - __bfloat162float(h1));
            }
#pragma unroll
            for (int np = 0; np < D / 16; ++np) {
                uint32_t b0, b1, b2, b3;
                ldsm_x4_t(sV + swz<C::ROW_BYTES>(ks * 16 + (lane & 7) + (((lane >> 3) & 1) << 3), np * 2 + (lane >> 4)),
                          b0, b1, b2, b3);
                mma_bf16(acc[2 * np], ahi[0], ahi[1], ahi[2], ahi[3], b0, b1);
                mma_bf16(acc[2 * np], alo[0], alo[1], alo[2], alo[3], b0, b1);
                mma_bf16(acc[2 * np + 1], ahi[0], ahi[1], ahi[2], ahi[3], b2, b3);
                mma_bf16(acc[2 * np + 1], alo[0], alo[1], alo[2], alo[3], b2, b3);
            }
        }
        stage = (stage + 1) % C::STAGES;
    }
    cp_async_wait<0>();

    // ---- write this split's partial
    float* part = partials + ((size_t)bh * nsplit + split) * C::PART_FLOATS;
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        zs[r] += __shfl_xor_sync(0xffffffffu, zs[r], 1);
        zs[r] += __shfl_xor_sync(0xffffffffu, zs[r], 2);
        const int a = warp * 16 + (lane >> 2) + r * 8;
        if ((lane & 3) == 0) part[D * D + a] = zs[r];
#pragma unroll
        for (int n = 0; n < D / 8; ++n) {
            const int c = n * 8 + 2 * (lane & 3);
            *reinterpret_cast<float2*>(part + (size_t)a * D + c) = make_float2(acc[n][2 * r], acc[n][2 * r + 1]);
        }
    }
}

// grid (D / 16, B*H, layers), D threads.  Adds the nsplit partials of every (layer, batch*head) to S (rows a0 .. a0 + 15 per
// block) and z (block 0), then folds the updated rows: Sf = S W_h^T (or S where the layer has no matrix) as bf16 hi and lo
// halves.  Order of the additions (it fixes the bits of the state, whichever kernel produced the partials): the splits are
// taken in `ngroup` groups of consecutive splits, group g = splits [nsplit g / ngroup, nsplit (g + 1) / ngroup); a group is
// summed from its first split upwards, and the group sums are added to the state in ascending g.  (The layer-batched
// kernel sums a group on chip and hands over one partial per group: nsplit == ngroup there.)
// The fold is a 16 x D x D product per block on the warp-level tensor path: the fp32 rows are split exactly into three bf16
// terms (hi + mid + lo = all 24 mantissa bits), W_h is bf16 already, so every product is exact and only the fp32
// accumulation of mma.sync rounds; warp w owns output columns [32 w, 32 w + 32).
// nsplit == 0: fold only.  sf_hi == nullptr: state update only.  z_scale: 1 for z = sum of phi(K) rows, 1 / tokens-per-frame
// for the per-frame-mean reading of Eq. 3.  partials: [layers][B*H][nsplit][D*D + D]; S, sf_hi, sf_lo: [layers][B*H][D][D];
// z: [layers][B*H][D]; W: [layers][H][D][D] or nullptr, used for the layers whose bit is set in has_w_mask.
template <int D>
__global__ void __launch_bounds__(D)
k_reduce_fold(const float* __restrict__ partials, int nsplit, int ngroup, float* __restrict__ S, float* __restrict__ z, float z_scale,
              const bf16* __restrict__ W, int heads, int BH, bf16* __restrict__ sf_hi, bf16* __restrict__ sf_lo,
              unsigned long long has_w_mask) {
    constexpr int ROWS = 16;
    constexpr int PART_FLOATS = D * D + D;
    constexpr int ROW_BYTES = D * 2;
    __shared__ __align__(128) uint8_t sW[D * ROW_BYTES];            // W_h [c'][c], 16-byte chunks XOR-swizzled by the row
    __shared__ __align__(128) uint8_t sA[3][ROWS * ROW_BYTES];      // the block's rows of S as bf16 hi / mid / lo, same swizzle
    const int a0 = blockIdx.x * ROWS, bh = blockIdx.y, lay = blockIdx.z, h = bh % heads;
    const size_t item = (size_t)lay * BH + bh;
    const int cp = threadIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool fold = sf_hi != nullptr, with_w = fold && W != nullptr && ((has_w_mask >> lay) & 1ull);
    if (with_w) {       // the matrix does not depend on the kernel before this one: fetched while that kernel drains
        const bf16* wsrc = W + ((size_t)lay * heads + h) * D * D;
        constexpr int CPR = D / 8;                                  // 16-byte chunks per row
#pragma unroll
        for (int i = 0; i < CPR; ++i) {
            const int id = threadIdx.x + i * D, row = id / CPR, ch = id % CPR;
            cp_async16(smem_u32(sW) + swz<ROW_BYTES>(row, ch), wsrc + (size_t)row * D + ch * 8, true);
        }
        cp_async_commit();
    }
    pdl_wait();         // launched under the tail of the partials kernel: its partials (and the state) are complete from here on
    const float* base = partials + item * nsplit * PART_FLOATS;
    float* S_it = S + item * D * D;
    float sum[ROWS];
#pragma unroll
    for (int r = 0; r < ROWS; ++r) sum[r] = S_it[(size_t)(a0 + r) * D + cp];
    float ztot = 0.f;           // this call's sum of phi(K) rows; enters z scaled (1, or 1 / tokens per frame)
    const bool do_z = blockIdx.x == 0 && nsplit > 0;
    for (int g = 0; g < ngroup && nsplit > 0; ++g) {
        const int s0 = (int)(((long long)nsplit * g) / ngroup), s1 = (int)(((long long)nsplit * (g + 1)) / ngroup);
        float sg[ROWS], zg = 0.f;
#pragma unroll
        for (int r = 0; r < ROWS; ++r) sg[r] = __ldcg(base + (size_t)s0 * PART_FLOATS + (size_t)(a0 + r) * D + cp);
        if (do_z) zg = __ldcg(base + (size_t)s0 * PART_FLOATS + D * D + cp);
#pragma unroll 2
        for (int s = s0 + 1; s < s1; ++s) {      // ascending split order per element; several splits' loads in flight
#pragma unroll
            for (int r = 0; r < ROWS; ++r) sg[r] += __ldcg(base + (size_t)s * PART_FLOATS + (size_t)(a0 + r) * D + cp);
            if (do_z) zg += __ldcg(base + (size_t)s * PART_FLOATS + D * D + cp);
        }
#pragma unroll
        for (int r = 0; r < ROWS; ++r) sum[r] += sg[r];
        ztot += zg;
    }
    if (nsplit > 0) {
#pragma unroll
        for (int r = 0; r < ROWS; ++r) S_it[(size_t)(a0 + r) * D + cp] = sum[r];
        if (do_z) z[item * D + cp] += ztot * z_scale;
    }
    if (!fold) return;
    if (!with_w) {
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            const __nv_bfloat16 hi = __float2bfloat16_rn(sum[r]);
            const size_t o = (item * D + a0 + r) * D + cp;
            sf_hi[o] = hi;
            sf_lo[o] = __float2bfloat16_rn(sum[r] - __bfloat162float(hi));
        }
        return;
    }
    // ---- the rows as three bf16 terms (each difference is exact in fp32), column cp of every row
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
        const __nv_bfloat16 t0 = __float2bfloat16_rn(sum[r]);
        const float r1 = sum[r] - __bfloat162float(t0);
        const __nv_bfloat16 t1 = __float2bfloat16_rn(r1);
        const __nv_bfloat16 t2 = __float2bfloat16_rn(r1 - __bfloat162float(t1));
        const uint32_t off = swz<ROW_BYTES>(r, cp >> 3) + (cp & 7) * 2;
        *reinterpret_cast<__nv_bfloat16*>(sA[0] + off) = t0;
        *reinterpret_cast<__nv_bfloat16*>(sA[1] + off) = t1;
        *reinterpret_cast<__nv_bfloat16*>(sA[2] + off) = t2;
    }
    cp_async_wait<0>();
    __syncthreads();
    // ---- out[a][c'] = sum_c S[a][c] W_h[c'][c]: A = the rows (16 x D), B = W_h as stored ([n][k], k contiguous)
    float acc[4][4];
#pragma unroll
    for (int n = 0; n < 4; ++n) { acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f; }
    const int n0 = warp * 32;
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
        uint32_t af[3][4];
#pragma unroll
        for (int t = 0; t < 3; ++t)
            ldsm_x4(smem_u32(sA[t]) + swz<ROW_BYTES>(lane & 15, ks * 2 + (lane >> 4)), af[t][0], af[t][1], af[t][2], af[t][3]);
#pragma unroll
        for (int np = 0; np < 2; ++np) {
            uint32_t b0, b1, b2, b3;
            ldsm_x4(smem_u32(sW) + swz<ROW_BYTES>(n0 + np * 16 + (lane & 7) + ((lane >> 4) << 3), ks * 2 + ((lane >> 3) & 1)), b0, b1, b2, b3);
#pragma unroll
            for (int t = 0; t < 3; ++t) {
                mma_bf16(acc[2 * np], af[t][0], af[t][1], af[t][2], af[t][3], b0, b1);
                mma_bf16(acc[2 * np + 1], af[t][0], af[t][1], af[t][2], af[t][3], b2, b3);
            }
        }
    }
#pragma unroll
    for (int n = 0; n < 4; ++n) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const float x0 = acc[n][2 * half], x1 = acc[n][2 * half + 1];
            const uint32_t hp = pack_bf16(x0, x1);
            const float2 hf = unpack_bf16(hp);
            const size_t o = (item * D + a0 + (lane >> 2) + half * 8) * D + n0 + n * 8 + 2 * (lane & 3);
            *reinterpret_cast<uint32_t*>(sf_hi + o) = hp;
            *reinterpret_cast<uint32_t*>(sf_lo + o) = pack_bf16(x0 - hf.x, x1 - hf.y);
        }
    }
}
