// Linear-attention state kernels on the Blackwell tensor path (tcgen05.mma, accumulators in tensor memory, TMA loads):
//   k_absorb_tc5   Eq. 3, first half: per (batch, head) the token range is split over thread blocks, each writing
//                  its partial phi(K_ev)^T V_ev and sum_t phi(K_ev[t]) to scratch (k_reduce_fold adds them up)
//   k_readout_tc5  Eq. 4: (phi(Q) S') / (phi(Q).z + eps) + bias with S' = S W^T folded beforehand
// In both, the phi(.) operand never goes back to shared memory: the thread that owns a row of the A operand
// (TMEM lane = row) evaluates phi in fp32, splits it into bf16 hi + lo halves (~16 mantissa bits together) and
// stores them straight into tensor memory, from where the MMA reads A; the other operand comes from shared
// memory as TMA wrote it.  Accumulation is fp32.  Every wait is bounded (~1 s) and reports through the device
// status word; nothing traps.
#pragma once
#include "tc5_common.cuh"

// ------------------------------------------------------------------------------------------------------------
// Absorb.  A = phi(K)^T: M = key feature a (lane), K = token.  B = V tile [token][c] (N = c contiguous, MN-major).
// D[a][c] += sum_t phi(k_t)[a] v_t[c]  over the block's token tiles; z[a] += sum_t phi(k_t)[a] in the lane's register.
// ------------------------------------------------------------------------------------------------------------
template <int D>
struct AbsorbTc5 {
    static constexpr int TT = 64;                        // tokens per tile
    static constexpr int NST = 4;                        // K / V stages in flight
    static constexpr int SUB = D / 64;
    static constexpr int K_BYTES = TT * D * 2;           // row-major, not swizzled (read column-wise by the lanes)
    static constexpr int VSUB_BYTES = TT * 128;          // one 64-column sub-tile of V, 128-byte swizzle
    static constexpr int V_BYTES = SUB * VSUB_BYTES;
    static constexpr int OFF_K = 0, OFF_V = NST * K_BYTES, OFF_BAR = OFF_V + NST * V_BYTES;
    static constexpr int NQ = 4;                         // phi warps per TMEM lane quadrant: each converts TT / NQ tokens of a tile
    static constexpr int OFF_Z = OFF_BAR + 256;          // z partials of the warps of a quadrant, [NQ][D] floats
    static constexpr int SMEM_BYTES = OFF_Z + NQ * D * 4 + 1024;
    static constexpr int THREADS = 128 * NQ + 64;        // phi / epilogue warps, then one TMA warp and one MMA warp
    static constexpr int WARP_TMA = 4 * NQ, WARP_MMA = 4 * NQ + 1;
    static constexpr int OUT_STRIDE = D + 4;             // floats; padded row of the epilogue's staging tile (reuses the K / V stages)
    static_assert(D * OUT_STRIDE * 4 <= OFF_BAR, "staging tile must fit in the pipeline stages");
    static constexpr int TMEM_COLS = 256;                // D accumulator [0, D) ; A buffers at 128 + 64 b: hi 32 cols, lo 32 cols
    static constexpr int COL_A = 128;
    static constexpr int PART_FLOATS = D * D + D;
};


// phi(K) of one 64-token tile for one key feature (= TMEM lane) and one quarter of the tile's tokens: evaluated in fp32,
// split into bf16 hi + lo halves, stored as the A operand (M = feature, K = token) at tA (hi: 32 columns, lo: the next
// 32); the unrotated values are added to zacc.  k_tile: the tile in shared memory, row-major [token][D], not swizzled.
// Shared by the split kernel and the layer-batched kernel so that both form the same bits.
template <int D, bool ROPE, bool TAIL>
__device__ __forceinline__ void absorb_phi_tile_t(const uint8_t* k_tile, int nv, int tile_row0, int part, int a, uint32_t tA_buf,
                                                  const float* cos_k, const float* sin_k, int rope_rows, float2& zacc2) {
    typedef AbsorbTc5<D> C;
    constexpr int HT = C::TT / C::NQ;                       // tokens per thread and tile
    const uint8_t* kt = k_tile + (size_t)(part * HT) * D * 2 + a * 2;
    uint32_t hi[HT / 2], lo[HT / 2];
    constexpr float LOG2E = 1.4426950408889634f;
#pragma unroll
    for (int t = 0; t < HT; t += 2) {
        const float x0 = __uint_as_float((uint32_t)(*reinterpret_cast<const uint16_t*>(kt + (size_t)t * D * 2)) << 16);
        const float x1 = __uint_as_float((uint32_t)(*reinterpret_cast<const uint16_t*>(kt + (size_t)(t + 1) * D * 2)) << 16);
        // phi(x) = x > 0 ? x + 1 : exp(x) for the two tokens at once (packed fp32 add / multiply: one instruction each)
        const float2 xs = make_float2(x0, x1);
        const float2 lin = fadd2(xs, make_float2(1.f, 1.f));
        const float2 arg = ffma2(xs, make_float2(LOG2E, LOG2E), make_float2(0.f, 0.f));
        float f0 = x0 > 0.f ? lin.x : fast_exp2(arg.x), f1 = x1 > 0.f ? lin.y : fast_exp2(arg.y);
        if (TAIL) {                                 // only the tensor's last tile
            if (t >= nv) f0 = 0.f;
            if (t + 1 >= nv) f1 = 0.f;
        }
        zacc2 = fadd2(zacc2, make_float2(f0, f1));  // the normaliser keeps the unrotated values (even / odd tokens apart)
        if (ROPE) {
            // feature pairs (2i, 2i+1) sit in neighbouring lanes; the pair's angle belongs to the token
            const float g0 = __shfl_xor_sync(0xffffffffu, f0, 1), g1 = __shfl_xor_sync(0xffffffffu, f1, 1);
            const int tok = tile_row0 + part * HT + t;     // rows past the tables belong to masked tokens
            const size_t o0 = (size_t)min(tok, rope_rows - 1) * (D / 2) + (a >> 1);
            const size_t o1 = (size_t)min(tok + 1, rope_rows - 1) * (D / 2) + (a >> 1);
            const float c0 = __ldg(cos_k + o0), s0 = __ldg(sin_k + o0);
            const float c1 = __ldg(cos_k + o1), s1 = __ldg(sin_k + o1);
            f0 = (a & 1) ? fmaf(g0, s0, f0 * c0) : fmaf(-g0, s0, f0 * c0);
            f1 = (a & 1) ? fmaf(g1, s1, f1 * c1) : fmaf(-g1, s1, f1 * c1);
        }
        const uint32_t hp = pack_bf16(f0, f1);
        const float2 hf = unpack_bf16(hp);
        hi[t >> 1] = hp;
        lo[t >> 1] = pack_bf16(f0 - hf.x, f1 - hf.y);       // (the differences are exact: the bf16 rounding errors)
    }
    const uint32_t tA = tA_buf + part * (HT / 2);
    tc5::tmem_st8(tA, hi);
    tc5::tmem_st8(tA + 32, lo);
}
// zacc2: running sums of phi(K) over the thread's even and odd tokens; a split's sum is zacc2.x + zacc2.y.
template <int D, bool ROPE>
__device__ __forceinline__ void absorb_phi_tile(const uint8_t* k_tile, int n_tokens, int tile_row0, int part, int a, uint32_t tA_buf,
                                                const float* cos_k, const float* sin_k, int rope_rows, float2& zacc2) {
    typedef AbsorbTc5<D> C;
    constexpr int HT = C::TT / C::NQ;
    // rows past the end of the tensor read as zero: phi(0) = 1 must not count (only the tensor's last tile has any)
    const int nv = min(C::TT, n_tokens - tile_row0) - part * HT;
    if (nv >= HT) absorb_phi_tile_t<D, ROPE, false>(k_tile, nv, tile_row0, part, a, tA_buf, cos_k, sin_k, rope_rows, zacc2);
    else absorb_phi_tile_t<D, ROPE, true>(k_tile, nv, tile_row0, part, a, tA_buf, cos_k, sin_k, rope_rows, zacc2);
}

struct AbsorbTc5Params {
    const float* cos_k;       // rotation tables of Eq. 3, [rope_rows, D/2] each (used by the ROPE instantiation only)
    const float* sin_k;
    int rope_rows;
    int n_tokens;
    float* partials;          // [B*H, nsplit, D*D + D]
    int* dev_status;
};

// grid (nsplit, B*H).  tm_k: [D, n_tokens, B*H, 1] box {D, 64}, no swizzle.  tm_v: same tensor shape, box {64, 64}, 128B swizzle.
template <int D, bool ROPE>
__global__ void __launch_bounds__(AbsorbTc5<D>::THREADS, 1)
k_absorb_tc5(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, const AbsorbTc5Params p) {
    using namespace tc5;
    typedef AbsorbTc5<D> C;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t s_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* s_gen = smem_raw + (s_base - smem_u32(smem_raw));
    const uint32_t sK = s_base + C::OFF_K, sV = s_base + C::OFF_V, bar0 = s_base + C::OFF_BAR;
    const uint32_t bar_full = bar0, bar_kfree = bar0 + 32, bar_vfree = bar0 + 64, bar_afull = bar0 + 96, bar_afree = bar0 + 112,
                   bar_dfull = bar0 + 128, bar_z = bar0 + 136, bar_st = bar0 + 152;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(s_gen + C::OFF_BAR + 160);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(s_gen + C::OFF_BAR + 164);
    float* z_x = reinterpret_cast<float*>(s_gen + C::OFF_Z);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int split = blockIdx.x, nsplit = gridDim.x, bh = blockIdx.y;
    const int n_tiles = (p.n_tokens + C::TT - 1) / C::TT;
    const int tile_lo = (int)(((long long)n_tiles * split) / nsplit);
    const int tile_hi = (int)(((long long)n_tiles * (split + 1)) / nsplit);
    const int n_local = tile_hi - tile_lo;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::NST; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_kfree + 8 * s, C::NQ * D); mbar_init(bar_vfree + 8 * s, 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(bar_afull + 8 * s, C::NQ * D); mbar_init(bar_afree + 8 * s, 1); }
        mbar_init(bar_dfull, 1); mbar_init(bar_z, C::NQ * D); mbar_init(bar_st, 128 * C::NQ);
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
    pdl_wait();                 // (set-up above may overlap the tail of the kernel before this one in the stream)

    if (warp == C::WARP_TMA) {
        // ================================================================= TMA producer
        if (lane == 0) {
            bool ok = true;
            for (int i = 0; ok && i < n_local; ++i) {
                const int s = i % C::NST;
                const uint32_t par_free = ((i / C::NST) & 1) ^ 1;
                if (i >= C::NST) {
                    if (!(ok = mbar_wait<true>(bar_kfree + 8 * s, par_free, abort_flag, p.dev_status, 31))) break;
                    if (!(ok = mbar_wait<true>(bar_vfree + 8 * s, par_free, abort_flag, p.dev_status, 32))) break;
                }
                const int row0 = (tile_lo + i) * C::TT;
                mbar_expect_tx(bar_full + 8 * s, C::K_BYTES + C::V_BYTES);
                tma_load_4d(sK + s * C::K_BYTES, &tm_k, 0, row0, bh, 0, bar_full + 8 * s);
#pragma unroll
                for (int u = 0; u < C::SUB; ++u)
                    tma_load_4d(sV + s * C::V_BYTES + u * C::VSUB_BYTES, &tm_v, u * 64, row0, bh, 0, bar_full + 8 * s);
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
        for (int i = 0; ok && i < n_local; ++i) {
            const int s = i % C::NST, ab = i & 1;
            if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_afull + 8 * ab, (i >> 1) & 1, abort_flag, p.dev_status, 33)))) break;
            if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_full + 8 * s, (i / C::NST) & 1, abort_flag, p.dev_status, 34)))) break;
            fence_after_sync();
            if (elect_one()) {
                const uint32_t tA = tmem + C::COL_A + ab * 64;
                const uint64_t dv = dv0 + (uint64_t)((s * C::V_BYTES) >> 4);
#pragma unroll
                for (int ks = 0; ks < C::TT / 16; ++ks) {
                    const uint64_t db = dv + (uint64_t)(ks * (2048 >> 4));
                    mma_ts(tmem, tA + ks * 8, db, IDESC, i > 0 || ks > 0);          // hi half
                    mma_ts(tmem, tA + 32 + ks * 8, db, IDESC, true);                // lo half
                }
                mma_commit(bar_afree + 8 * ab);
                mma_commit(bar_vfree + 8 * s);
                if (i == n_local - 1) mma_commit(bar_dfull);
            }
            __syncwarp();
        }
    } else {
        // ================================================================= phi(K) into tensor memory, then the epilogue
        // NQ warps per TMEM lane quadrant: warps w, w + 4, ... own the same 32 key features (lanes) and convert
        // consecutive groups of TT / NQ tokens of a tile.
        const int part = warp >> 2;
        const int a = (warp & 3) * 32 + lane;                   // key feature = TMEM lane
        const bool active = a < D;
        const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        constexpr int HT = C::TT / C::NQ;                       // tokens per thread and tile
        bool ok = true;
        float2 zacc = make_float2(0.f, 0.f);
        // Warps whose lanes lie past the head dimension (the upper two quadrants at head_dim 64) have no part in the tile
        // loop and must stay out of it: they would wait on the stage barriers without ever arriving on the "free" ones, so
        // nothing would keep the pipeline from running more than a ring ahead of them, and a warp that falls NST tiles
        // behind waits on a phase parity that has come round again -- until its wait limit.  (`active` is warp-uniform.)
        for (int i = 0; ok && active && i < n_local; ++i) {
            const int s = i % C::NST, ab = i & 1;
            ok = __all_sync(0xffffffffu, mbar_wait(bar_full + 8 * s, (i / C::NST) & 1, abort_flag, p.dev_status, 35));
            if (!ok) break;
            if (i >= 2) {
                ok = __all_sync(0xffffffffu, mbar_wait(bar_afree + 8 * ab, ((i >> 1) & 1) ^ 1, abort_flag, p.dev_status, 36));
                if (!ok) break;
                fence_after_sync();
            }
            if (active) {
                absorb_phi_tile<D, ROPE>(s_gen + C::OFF_K + s * C::K_BYTES, p.n_tokens, (tile_lo + i) * C::TT, part, a,
                                         lane_base + C::COL_A + ab * 64, p.cos_k, p.sin_k, p.rope_rows, zacc);
                tmem_wait_st();
                fence_before_sync();
                mbar_arrive(bar_afull + 8 * ab);
                mbar_arrive(bar_kfree + 8 * s);
            }
        }
        // ---- epilogue: the accumulator goes through a padded staging tile in shared memory (the pipeline stages are
        // idle by now: every TMA copy has been consumed) so that the partial is written with coalesced stores
        pdl_trigger();          // the reduce/fold kernel may be launched now: it waits for this grid before it reads a partial
        if (ok && active) {
            z_x[part * D + a] = zacc.x + zacc.y;
            mbar_arrive(bar_z);
        }
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar_dfull, 0, abort_flag, p.dev_status, 37));
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar_z, 0, abort_flag, p.dev_status, 38));
        float* stage_out = reinterpret_cast<float*>(s_gen);
        if (ok && active) {
            fence_after_sync();
            constexpr int CW = D / C::NQ;                       // accumulator columns staged by this warp
            static_assert(CW % 16 == 0, "column share must be a multiple of 16");
#pragma unroll
            for (int c = 0; c < CW / 16; ++c) {
                const int col = part * CW + c * 16;
                uint32_t r[16];
                tmem_ld16(lane_base + col, r);
                tmem_wait_ld();
                float4* dst = reinterpret_cast<float4*>(stage_out + (size_t)a * C::OUT_STRIDE + col);
#pragma unroll
                for (int v = 0; v < 4; ++v)
                    dst[v] = make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]), __uint_as_float(r[4 * v + 2]),
                                         __uint_as_float(r[4 * v + 3]));
            }
        }
        // all phi warps (active or not) meet before the staged tile is read back
        mbar_arrive(bar_st);
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar_st, 0, abort_flag, p.dev_status, 39));
        if (ok) {
            float* part_out = p.partials + ((size_t)bh * nsplit + split) * C::PART_FLOATS;
            const int tid = threadIdx.x;                        // 0 .. 128 NQ - 1
            for (int e = tid; e < D * D / 4; e += 128 * C::NQ) {
                const int rrow = e / (D / 4), c4 = e - rrow * (D / 4);
                reinterpret_cast<float4*>(part_out)[e] = *reinterpret_cast<const float4*>(stage_out + (size_t)rrow * C::OUT_STRIDE + c4 * 4);
            }
            if (tid < D) {
                float zs = z_x[tid];
#pragma unroll
                for (int q = 1; q < C::NQ; ++q) zs += z_x[q * D + tid];
                part_out[D * D + tid] = zs;
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

// ------------------------------------------------------------------------------------------------------------
// Read-out.  Unit = (batch*head, tile of 128 query rows).  A = phi(Q): M = query row (lane), K = key feature.
// B = S' [a][c] (N = c contiguous, MN-major), hi and lo halves.  D = A_hi S'_hi + A_lo S'_hi + A_hi S'_lo.
// A thread block takes a contiguous run of units, so that S' is fetched once per (batch, head) it touches
// ("epoch"), into one of two buffers.
// ------------------------------------------------------------------------------------------------------------
template <int D>
struct ReadoutTc5 {
    static constexpr int ROWS = 128;
    static constexpr int NST = 2;                        // Q stages; S' {hi, lo} buffers likewise two
    static constexpr int SUB = D / 64;
    static constexpr int QSUB_BYTES = ROWS * 128, Q_BYTES = SUB * QSUB_BYTES;
    static constexpr int SSUB_BYTES = D * 128, S_BYTES = SUB * SSUB_BYTES;
    static constexpr int OFF_Q = 0, OFF_S = NST * Q_BYTES;   // S' buffer e at OFF_S + e * 2 * S_BYTES: hi then lo
    static constexpr int OFF_VEC = OFF_S + 2 * 2 * S_BYTES;  // per stage: z [D] floats, bias [D] floats
    static constexpr int OFF_DEN = OFF_VEC + NST * 2 * D * 4;   // per stage: denominator partials [2][128] floats
    static constexpr int OFF_BAR = OFF_DEN + NST * 2 * ROWS * 4;
    static constexpr int SMEM_BYTES = OFF_BAR + 256 + 1024;
    static constexpr int THREADS = 320;                  // warps 0-7: phi / epilogue (two per TMEM lane quadrant), warp 8: TMA, warp 9: MMA
    static constexpr int WARP_TMA = 8, WARP_MMA = 9;
    static constexpr int TMEM_COLS = 4 * D;              // D accumulators at D b ; A buffers at 2 D + D b: hi D/2 cols, lo D/2 cols
};

struct ReadoutTc5Params {
    const float* cos_q;       // rotation tables of Eq. 4's numerator, [T_c, D/2] each (ROPE instantiation only)
    const float* sin_q;
    const float* z;           // [B*H, D]
    const bf16* bias;         // [H, D] or nullptr
    int heads, Tc, Tm, n_units;
    float eps;
    bf16* out_bf16;           // exactly one of out_bf16 / out_f32 is non-null: [B*H, T_c, D]
    float* out_f32;
    bf16* out_lo;             // with out_bf16: the bf16 residual of the result (value = out_bf16 + out_lo to ~16 bits), or nullptr
    int* dev_status;
};

// CTA c processes units [c * upc, (c + 1) * upc), upc = ceil(n_units / gridDim.x).  tm_q: [D, T_c, B*H, 1] box {64, 128};
// tm_sh, tm_sl: [D, D, B*H, 1] box {64, D}; all 128B swizzle.
template <int D, bool ROPE>
__global__ void __launch_bounds__(ReadoutTc5<D>::THREADS, 1)
k_readout_tc5(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_sh,
              const __grid_constant__ CUtensorMap tm_sl, const ReadoutTc5Params p) {
    using namespace tc5;
    typedef ReadoutTc5<D> C;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t s_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* s_gen = smem_raw + (s_base - smem_u32(smem_raw));
    const uint32_t bar0 = s_base + C::OFF_BAR;
    const uint32_t bar_full = bar0, bar_qfree = bar0 + 16, bar_sfree = bar0 + 32, bar_afull = bar0 + 48, bar_afree = bar0 + 64,
                   bar_dfull = bar0 + 80, bar_dfree = bar0 + 96, bar_vec = bar0 + 112, bar_sfull = bar0 + 128;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(s_gen + C::OFF_BAR + 144);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(s_gen + C::OFF_BAR + 148);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int upc = (p.n_units + (int)gridDim.x - 1) / (int)gridDim.x;
    const int u0 = min((int)blockIdx.x * upc, p.n_units);
    const int my_units = min(upc, p.n_units - u0);

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar_full + 8 * s, 1); mbar_init(bar_qfree + 8 * s, 256); mbar_init(bar_sfree + 8 * s, 1);
            mbar_init(bar_afull + 8 * s, 256); mbar_init(bar_afree + 8 * s, 1); mbar_init(bar_dfull + 8 * s, 1);
            mbar_init(bar_dfree + 8 * s, 256); mbar_init(bar_vec + 8 * s, 256); mbar_init(bar_sfull + 8 * s, 1);
        }
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
        // ================================================================= TMA producer
        if (lane == 0) {
            bool ok = true;
            int epoch = -1, bh_prev = -1;
            for (int n = 0; ok && n < my_units; ++n) {
                const int u = u0 + n;
                const int bh = u / p.Tm, i = u - bh * p.Tm;
                const int s = n & 1;
                if (bh != bh_prev) {                 // new (batch, head): its folded state, hi and lo halves
                    bh_prev = bh; ++epoch;
                    const int e = epoch & 1;
                    if (epoch >= 2 && !(ok = mbar_wait<true>(bar_sfree + 8 * e, ((epoch >> 1) & 1) ^ 1, abort_flag, p.dev_status, 42))) break;
                    const uint32_t sb = s_base + C::OFF_S + e * 2 * C::S_BYTES;
                    mbar_expect_tx(bar_sfull + 8 * e, 2 * C::S_BYTES);
#pragma unroll
                    for (int v = 0; v < C::SUB; ++v) {
                        tma_load_4d(sb + v * C::SSUB_BYTES, &tm_sh, v * 64, 0, bh, 0, bar_sfull + 8 * e);
                        tma_load_4d(sb + C::S_BYTES + v * C::SSUB_BYTES, &tm_sl, v * 64, 0, bh, 0, bar_sfull + 8 * e);
                    }
                }
                if (n >= 2 && !(ok = mbar_wait<true>(bar_qfree + 8 * s, ((n >> 1) & 1) ^ 1, abort_flag, p.dev_status, 41))) break;
                const uint32_t st = s_base + C::OFF_Q + s * C::Q_BYTES;
                mbar_expect_tx(bar_full + 8 * s, C::Q_BYTES);
#pragma unroll
                for (int v = 0; v < C::SUB; ++v)
                    tma_load_4d(st + v * C::QSUB_BYTES, &tm_q, v * 64, i * C::ROWS, bh, 0, bar_full + 8 * s);
            }
            if (!ok) {
                const long long t0 = clock64();
                while (clock64() - t0 < 400000) {}
            }
        }
    } else if (warp == C::WARP_MMA) {
        // ================================================================= MMA issuer (warp-uniform, one elected lane issues)
        constexpr uint32_t IDESC = idesc_bf16(D, true);
        bool ok = true;
        int epoch = -1, bh_prev = -1;
        for (int n = 0; ok && n < my_units; ++n) {
            const int s = n & 1;
            const uint32_t par = (n >> 1) & 1;
            const int bh = (u0 + n) / p.Tm;
            if (bh != bh_prev) {
                bh_prev = bh; ++epoch;
                if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_sfull + 8 * (epoch & 1), (epoch >> 1) & 1, abort_flag, p.dev_status, 45)))) break;
            }
            const bool last_of_epoch = (n + 1 == my_units) || ((u0 + n + 1) / p.Tm != bh);
            if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_afull + 8 * s, par, abort_flag, p.dev_status, 43)))) break;
            if (n >= 2 && !(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_dfree + 8 * s, par ^ 1u, abort_flag, p.dev_status, 44)))) break;
            fence_after_sync();
            if (elect_one()) {
                const uint32_t tD = tmem + s * D, tA = tmem + 2 * D + s * D;
                const uint32_t sb = s_base + C::OFF_S + (epoch & 1) * 2 * C::S_BYTES;
                const uint64_t dsh = smem_desc_sw128(sb, C::SSUB_BYTES, 1024);
                const uint64_t dsl = smem_desc_sw128(sb + C::S_BYTES, C::SSUB_BYTES, 1024);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint64_t off = (uint64_t)(ks * (2048 >> 4));
                    mma_ts(tD, tA + ks * 8, dsh + off, IDESC, ks > 0);              // phi_hi S'_hi
                    mma_ts(tD, tA + D / 2 + ks * 8, dsh + off, IDESC, true);        // phi_lo S'_hi
                    mma_ts(tD, tA + ks * 8, dsl + off, IDESC, true);                // phi_hi S'_lo
                }
                mma_commit(bar_dfull + 8 * s);
                mma_commit(bar_afree + 8 * s);
                if (last_of_epoch) mma_commit(bar_sfree + 8 * (epoch & 1));
            }
            __syncwarp();
        }
    } else {
        // ================================================================= phi(Q) into tensor memory; epilogue one unit behind
        // Two warps per TMEM lane quadrant: warp w and w + 4 own the same 32 query rows (lanes); the lower one converts
        // key features [0, D/2) and stores output columns [0, D/2), the upper one the other halves.  Loops over 32-wide
        // chunks are kept rolled: the code stays small enough for the instruction cache.
        const int half = warp >> 2;
        const int row = (warp & 3) * 32 + lane;                 // query row of the tile = TMEM lane
        const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        constexpr int PASSES = D / 64;                          // 32-feature (and 32-column) passes per thread
        bool ok = true;
        auto convert = [&](int n) -> bool {                     // A operand of unit n; denominator partial of the half
            const int u = u0 + n;
            const int bh = u / p.Tm;
            const int s = n & 1;
            const uint32_t par = (n >> 1) & 1;
            const int r_tab = min((u - bh * p.Tm) * C::ROWS + row, p.Tc - 1);     // row of the rotation tables
            // z and bias of the unit's head, staged by these threads once every thread has left the epilogue that read
            // the stage's buffers last (two units ago)
            float* vec = reinterpret_cast<float*>(s_gen + C::OFF_VEC + s * 2 * D * 4);
            float* den_x = reinterpret_cast<float*>(s_gen + C::OFF_DEN + s * 2 * C::ROWS * 4);
            if (n >= 2 && !__all_sync(0xffffffffu, mbar_wait(bar_dfree + 8 * s, par ^ 1u, abort_flag, p.dev_status, 50))) return false;
            if (threadIdx.x < D) {
                vec[threadIdx.x] = p.z[(size_t)bh * D + threadIdx.x];
                vec[D + threadIdx.x] = p.bias ? __bfloat162float(p.bias[(size_t)(bh % p.heads) * D + threadIdx.x]) : 0.f;
            }
            mbar_arrive(bar_vec + 8 * s);
            if (!__all_sync(0xffffffffu, mbar_wait(bar_vec + 8 * s, par, abort_flag, p.dev_status, 46))) return false;
            if (!__all_sync(0xffffffffu, mbar_wait(bar_full + 8 * s, par, abort_flag, p.dev_status, 47))) return false;
            if (n >= 2) {
                if (!__all_sync(0xffffffffu, mbar_wait(bar_afree + 8 * s, par ^ 1u, abort_flag, p.dev_status, 48))) return false;
                fence_after_sync();
            }
            const uint8_t* qt = s_gen + C::OFF_Q + s * C::Q_BYTES + row * 128;
            const uint32_t tA = lane_base + 2 * D + s * D;
            float dsum = 0.f;
#pragma unroll 1
            for (int gi = 0; gi < PASSES; ++gi) {               // 32 features per pass: 16 packed hi + 16 packed lo registers
                const int g = half * PASSES + gi;
                uint32_t hi[16], lo[16];
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    const int chunk = g * 4 + cc;               // 16-byte chunk of the row (8 features)
                    const int sub = chunk >> 3, phys = (chunk & 7) ^ (row & 7);
                    const uint4 w = *reinterpret_cast<const uint4*>(qt + sub * C::QSUB_BYTES + phys * 16);
                    const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
                    float cs[4] = {1.f, 1.f, 1.f, 1.f}, sn[4] = {0.f, 0.f, 0.f, 0.f};
                    if (ROPE) {
                        const float4 c4 = __ldg(reinterpret_cast<const float4*>(p.cos_q + (size_t)r_tab * (D / 2)) + chunk);
                        const float4 s4 = __ldg(reinterpret_cast<const float4*>(p.sin_q + (size_t)r_tab * (D / 2)) + chunk);
                        cs[0] = c4.x; cs[1] = c4.y; cs[2] = c4.z; cs[3] = c4.w;
                        sn[0] = s4.x; sn[1] = s4.y; sn[2] = s4.z; sn[3] = s4.w;
                    }
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 x = unpack_bf16(ws[e]);
                        float f0 = phi_elu1(x.x), f1 = phi_elu1(x.y);
                        const int feat = chunk * 8 + 2 * e;
                        dsum = fmaf(f0, vec[feat], fmaf(f1, vec[feat + 1], dsum));     // denominator: unrotated
                        if (ROPE) {
                            const float r0 = fmaf(-f1, sn[e], f0 * cs[e]), r1 = fmaf(f0, sn[e], f1 * cs[e]);
                            f0 = r0; f1 = r1;
                        }
                        const uint32_t hp = pack_bf16(f0, f1);
                        const float2 hf = unpack_bf16(hp);
                        hi[cc * 4 + e] = hp;
                        lo[cc * 4 + e] = pack_bf16(f0 - hf.x, f1 - hf.y);
                    }
                }
                tmem_st16(tA + g * 16, hi);
                tmem_st16(tA + D / 2 + g * 16, lo);
            }
            den_x[half * C::ROWS + row] = dsum;
            tmem_wait_st();
            fence_before_sync();
            mbar_arrive(bar_afull + 8 * s);
            mbar_arrive(bar_qfree + 8 * s);
            return true;
        };
        auto epilogue = [&](int n) -> bool {
            const int u = u0 + n;
            const int bh = u / p.Tm, i = u - bh * p.Tm;
            const int s = n & 1;
            // the accumulator is complete; its MMAs were issued after every phi thread of the unit had arrived (and
            // published its denominator partial), so the partials of both halves are visible here
            if (!__all_sync(0xffffffffu, mbar_wait(bar_dfull + 8 * s, (n >> 1) & 1, abort_flag, p.dev_status, 49))) return false;
            fence_after_sync();
            const float* vec = reinterpret_cast<const float*>(s_gen + C::OFF_VEC + s * 2 * D * 4);
            const float* den_x = reinterpret_cast<const float*>(s_gen + C::OFF_DEN + s * 2 * C::ROWS * 4);
            const float inv = 1.f / (den_x[row] + den_x[C::ROWS + row] + p.eps);
            const int r_glob = i * C::ROWS + row;
            const bool valid = r_glob < p.Tc;
            const size_t g = ((size_t)bh * p.Tc + r_glob) * D;
#pragma unroll 1
            for (int ci = 0; ci < PASSES; ++ci) {
                const int col = half * (D / 2) + ci * 32;
                uint32_t r[32];
                tmem_ld32(lane_base + s * D + col, r);
                tmem_wait_ld();
                if (valid) {
                    float x[32];
#pragma unroll
                    for (int e = 0; e < 32; ++e) x[e] = fmaf(__uint_as_float(r[e]), inv, vec[D + col + e]);
                    if (p.out_f32) {
                        float4* dst = reinterpret_cast<float4*>(p.out_f32 + g + col);
#pragma unroll
                        for (int v = 0; v < 8; ++v) dst[v] = make_float4(x[4 * v], x[4 * v + 1], x[4 * v + 2], x[4 * v + 3]);
                    } else {
                        uint4* dst = reinterpret_cast<uint4*>(p.out_bf16 + g + col);
                        uint32_t hp[16];
#pragma unroll
                        for (int e = 0; e < 16; ++e) hp[e] = pack_bf16(x[2 * e], x[2 * e + 1]);
#pragma unroll
                        for (int v = 0; v < 4; ++v) dst[v] = make_uint4(hp[4 * v], hp[4 * v + 1], hp[4 * v + 2], hp[4 * v + 3]);
                        if (p.out_lo) {
                            uint4* dlo = reinterpret_cast<uint4*>(p.out_lo + g + col);
                            uint32_t lp[16];
#pragma unroll
                            for (int e = 0; e < 16; ++e) {
                                const float2 hf = unpack_bf16(hp[e]);
                                lp[e] = pack_bf16(x[2 * e] - hf.x, x[2 * e + 1] - hf.y);
                            }
#pragma unroll
                            for (int v = 0; v < 4; ++v) dlo[v] = make_uint4(lp[4 * v], lp[4 * v + 1], lp[4 * v + 2], lp[4 * v + 3]);
                        }
                    }
                }
            }
            fence_before_sync();
            mbar_arrive(bar_dfree + 8 * s);
            return true;
        };
        if (my_units > 0) ok = convert(0);
        for (int n = 0; ok && n < my_units; ++n) {
            if (n + 1 < my_units && !(ok = convert(n + 1))) break;
            ok = epilogue(n);
        }
    }
    fence_before_sync();
    __syncthreads();
    if (warp == C::WARP_MMA) {
        fence_after_sync();
        tmem_dealloc(tmem, C::TMEM_COLS);
    }
}
