// Block-sparse sliding-window attention (Eq. 6; Alg. 3 inner loops) on the Blackwell tensor path:
// TMA loads addressed by the kept-block index list, tcgen05.mma with S / P / O in tensor memory, fp32 softmax
// against a reference exponent fixed per query block.  Block size 128, head dim 64 or 128.  The HIST instantiation
// (head dim 128) also forms the history term of Eq. 4 and adds it (Eq. 7) before the one rounding to bf16.
//
// Persistent kernel, one CTA per SM; a CTA walks its (batch*head, query block) units and their kept key
// blocks as one stream of tiles t = 0, 1, ...
//   softmax warps   NG column groups of four warps; thread (group g, row r) owns columns [g*128/NG, (g+1)*128/NG)
//                   of S row r (TMEM lane = row) and the same share of the O columns.  At a unit's first tile the
//                   groups exchange their row maxima through shared memory; that maximum times 2^HEADROOM is the
//                   reference exponent m of the row for the whole unit (softmax does not depend on m; what m must do is
//                   keep exp2(S c - m) inside fp32, which the end of the unit checks).  After that tile the groups do not
//                   meet until the unit ends: no running maximum, no rescaling of O, row sums partial until then.
//   loader warp K   TMA: Q (one buffer, reloaded per unit), K tiles (ring of two at head dim 128, three at 64); HIST:
//                   per unit the lo tile of the head's folded state and a second copy of the Q tile
//   loader warp V   TMA: V tiles (ring of two)
//   MMA warp        TMEM allocation and tcgen05.mma issue.  S lives in three TMEM buffers and is issued two tiles
//                   ahead of the softmax (S_{t+2} before P_t V_t), so that neither the TMA latency of K nor the
//                   MMA issue chain sits on the softmax critical path.
//   S = Q K_t^T        A = Q (smem, K-major, 128B swizzle), B = K_t (smem, K-major)     -> TMEM cols 128*(t%3)
//   P = exp2(S*c - m)  bf16, written over the writing thread's own S columns (group g: columns 64 g .. 64 g + 31)
//   O += P V_t         A = P (TMEM, two pieces), B = V_t (smem, MN-major, 128B swizzle)  -> TMEM cols [384, 384+D)
//   HIST, unit end     A = (l / den) phi(Q) as bf16 hi + lo in the free S buffer (phi(Q) from the shared-memory copy of
//                      Q, den = phi(q).z + eps exchanged between the groups with the row sums l);
//                      O += A_hi S'_lo + A_hi S'_hi + A_lo S'_hi, S' = the folded state S W^T (hi tile loaded over the
//                      Q copy once it has been read); then O / l (+ bias) -> bf16 -> shared memory -> bulk tensor store
// Every wait is bounded (~1 s); on expiry the CTA raises the device status word and leaves through the
// common exit (drains its copies, frees its TMEM).
//
// Range of the fixed reference, and what happens outside it.  Alg. 3 carries a running row maximum so that no input
// overflows; here the reference is fixed after the first kept tile, which covers rows whose later tiles rise up to about
// 100 natural-log units above the first one.  A unit with a row beyond that (row sum not finite or above 2^100 at the
// unit's end -- a complete test: every P is a term of the row sum) is put on a list in shared memory, and when the
// thread block has finished its tile stream it computes those units again with the running maximum, rescaling l and O as
// Alg. 3 prints them (swa_redo_unit below: the warp-level code of k_swa_mma.cuh, plus the history term where this kernel
// forms it), overwriting the rows the fast path left.  The result is therefore the softmax of Eq. 6 for every finite input.
#pragma once
#include "tc5_common.cuh"
#include "k_swa_mma.cuh"


template <int D, int NG>
struct SwaTc5 {
    static constexpr int BLK = 128;
    static constexpr int GROUPS = NG;                  // softmax column groups (four warps each)
    static constexpr int GCOLS = BLK / NG;             // S columns per thread
    static constexpr int OCOLS = D / NG;               // O columns per thread
    static constexpr int SUB = D / 64;                 // 64-column (128-byte) sub-tiles per operand tile
    static constexpr int SUB_BYTES = BLK * 128;        // 16 KB
    static constexpr int TILE_BYTES = SUB * SUB_BYTES;
#ifndef HF_TC5_SKEW_CLK
#define HF_TC5_SKEW_CLK 500
#endif
    static constexpr long long SKEW_CLK = HF_TC5_SKEW_CLK;   // offset between the column groups, in clocks (see the softmax warps)
    static constexpr float HEADROOM = 60.f;           // log2 distance of the softmax reference above the first tile's row maximum
    static constexpr int KSTAGES = (D == 128) ? 2 : 3, VSTAGES = 2, SBUFS = 3;   // (a K tile is free again as soon as its S is done)
    // The history term (Eq. 4) can be formed inside this kernel at head_dim 128 with two column groups: the folded
    // state S W^T (bf16 hi and lo halves, one operand tile each) then sits in shared memory beside the K / V rings.
    static constexpr bool FUSE = (D == 128 && NG == 2);
    static constexpr int OFF_Q = 0, OFF_K = TILE_BYTES, OFF_V = OFF_K + KSTAGES * TILE_BYTES;
    static constexpr int OFF_H = OFF_V + VSTAGES * TILE_BYTES;
    static constexpr int OFF_BAR = OFF_H + (FUSE ? 2 * TILE_BYTES : 0);
    static constexpr int OFF_XM = OFF_BAR + 320;       // exchange between the column groups: [2][NG][128] floats
    static constexpr int USED_BYTES = OFF_XM + 2 * NG * BLK * 4;
    static constexpr int MAX_SMEM = 232448;            // 227 KB: the most one thread block can have
    // Slack for the manual 1024-byte alignment of the operand tiles (the kernel checks that it was enough); more than
    // half an SM's shared memory so that one CTA owns the SM (it allocates all 512 TMEM columns)
    static constexpr int WANT_BYTES = (USED_BYTES + 1024) > 120 * 1024 ? (USED_BYTES + 1024) : 120 * 1024;
    static constexpr int SMEM_BYTES = WANT_BYTES < MAX_SMEM ? WANT_BYTES : MAX_SMEM;
    static_assert(USED_BYTES <= MAX_SMEM, "shared memory layout does not fit");
    static constexpr int THREADS = 128 * NG + 96;
    static constexpr int WARP_LOAD_K = 4 * NG, WARP_LOAD_V = 4 * NG + 1, WARP_MMA = 4 * NG + 2;
    static constexpr int TMEM_COLS = 512;
    static constexpr int COL_O = SBUFS * BLK;          // S buffers at columns 0, 128, 256
};

struct Tc5Params {
    const int32_t* idx;      // [B*H, T_m, keep]
    int keep, Tc, n_b, n_cached, ring_head, P;   // P: physical ring slots (one more than the window holds); the sink slots follow them
    int n_sink;              // sink chunks held (logical chunks 0 .. n_sink - 1)
    int Tm, n_units;         // units = (batch*head, query block) pairs, unit u = bh * Tm + i
    float scale_log2;
    const float* hist;       // optional fp32 [B*H, T_c, D]: history term formed by another kernel, added in the epilogue
    // History term formed in the kernel (its HIST instantiation): q as the kernel's own tensor map sees it, z [B*H, D],
    // bias [H, D] or nullptr, eps of Eq. 4's denominator
    int heads;
    float eps;
    const bf16* q;
    const float* z;
    const bf16* bias;
    bf16* o;
    float* lse;
    int* dev_status;
    // for the units that are computed again with a running maximum: the window as plain pointers, and the folded state
    ChunkTable tab;
    const bf16* sf_hi;       // [B*H, D, D] bf16 hi / lo halves of S W^T (HIST only)
    const bf16* sf_lo;
};

// Ring position of item i in a ring of N stages: stage i % N, completed-phase parity (i / N) & 1, kept incrementally.
template <int N>
struct RingPos {
    int stage = 0;
    uint32_t phase = 0;
    __device__ __forceinline__ void advance() { if (++stage == N) { stage = 0; phase ^= 1u; } }
};


// One unit again, the way Alg. 3 prints it (running maximum m, rescaling of l and O), by threads 0 .. 255 of the thread
// block, after the tile stream has drained (shared memory and the exchange buffers are free by then).  HIST: the history
// term of Eq. 4 for the unit's rows is formed first, in fp32 on the CUDA cores, into a shared-memory tile that the
// attention epilogue adds (Eq. 7).  Slow and rare by design.
template <int D, bool HIST>
__device__ __noinline__ void swa_redo_unit(uint8_t* s_gen, const Tc5Params& p, int u) {
    typedef SwaMma<128, D> M;
    constexpr int BLK = 128;
    const int bh = u / p.Tm, i = u - bh * p.Tm;
    const int q0 = i * BLK, nq = min(BLK, p.Tc - q0);
    const int tid = threadIdx.x;
    const float* hist_rows = p.hist ? p.hist + ((size_t)bh * p.Tc + q0) * D : nullptr;
    asm volatile("bar.sync 1, 256;\n" ::: "memory");      // the previous unit's epilogue has read its history tile
    if constexpr (HIST) {
        constexpr int PS = D + 1;                                            // padded row of the phi(Q) tile
        float* phi_t = reinterpret_cast<float*>(s_gen + M::TILE_BYTES);     // [128][D + 1], in the K / V stages (not yet in use)
        float* den_t = phi_t + BLK * PS;                                    // [128]
        float* hist_t = reinterpret_cast<float*>(s_gen + M::SMEM_BYTES);    // [128][D], behind the attention tiles
        static_assert(M::TILE_BYTES + (BLK * PS + BLK) * 4 <= M::SMEM_BYTES, "phi(Q) tile must fit in the K / V stages");
        {   // phi(q) of the unit's rows (zero past the chunk's end): thread = (row, half of the features)
            const int row = tid >> 1, f0 = (tid & 1) * (D / 2);
            const bf16* src = p.q + ((size_t)bh * p.Tc + q0 + row) * D + f0;
            for (int c = 0; c < D / 2; c += 8) {
                uint4 w = make_uint4(0, 0, 0, 0);
                if (row < nq) w = __ldg(reinterpret_cast<const uint4*>(src + c));
                const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 x = unpack_bf16(ws[e]);
                    phi_t[row * PS + f0 + c + 2 * e] = row < nq ? phi_elu1(x.x) : 0.f;
                    phi_t[row * PS + f0 + c + 2 * e + 1] = row < nq ? phi_elu1(x.y) : 0.f;
                }
            }
        }
        asm volatile("bar.sync 1, 256;\n" ::: "memory");
        if (tid < BLK) {        // Eq. 4's denominator phi(q).z + eps, one row per thread
            float dsum = 0.f;
            const float* zr = p.z + (size_t)bh * D;
            for (int a = 0; a < D; ++a) dsum = fmaf(phi_t[tid * PS + a], __ldg(zr + a), dsum);
            den_t[tid] = dsum + p.eps;
        }
        {   // numerator phi(q) S' : thread = (output column, group of rows); S' = hi + lo halves of the folded state
            constexpr int GROUPS = 256 / D, RPT = BLK / GROUPS;
            const int c = tid % D, r0 = (tid / D) * RPT;
            const bf16* sh = p.sf_hi + (size_t)bh * D * D + c;
            const bf16* sl = p.sf_lo + (size_t)bh * D * D + c;
            float acc[RPT];
#pragma unroll
            for (int r = 0; r < RPT; ++r) acc[r] = 0.f;
            for (int a = 0; a < D; ++a) {
                const float sv = __bfloat162float(sh[(size_t)a * D]) + __bfloat162float(sl[(size_t)a * D]);
#pragma unroll
                for (int r = 0; r < RPT; ++r) acc[r] = fmaf(phi_t[(r0 + r) * PS + a], sv, acc[r]);
            }
            asm volatile("bar.sync 1, 256;\n" ::: "memory");      // denominators written
            const float b = p.bias ? __bfloat162float(p.bias[(size_t)(bh % p.heads) * D + c]) : 0.f;
#pragma unroll
            for (int r = 0; r < RPT; ++r) hist_t[(r0 + r) * D + c] = acc[r] / den_t[r0 + r] + b;
        }
        asm volatile("bar.sync 1, 256;\n" ::: "memory");          // tile complete; the K / V stages are free again
        hist_rows = hist_t;
    }
    if (tid == 0) atomicAdd(p.dev_status + 2, 1);                 // count of units that took this path
    swa_mma_unit<BLK, D>(s_gen, p.q, p.tab, p.idx + (size_t)u * p.keep, p.keep, p.Tc, p.n_b, p.scale_log2, hist_rows, p.o,
                         p.lse, p.dev_status, i, bh, u);
}

// Persistent: CTA c processes units c, c + gridDim.x, ...
// HIST: the history term is formed here (needs SwaTc5::FUSE and the tensor maps of S W^T); otherwise p.hist, if any, is added.
template <int D, int NG, bool HIST>
__global__ void __launch_bounds__(SwaTc5<D, NG>::THREADS, 1)
k_swa_tc5(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kring,
          const __grid_constant__ CUtensorMap tm_vring, const __grid_constant__ CUtensorMap tm_kcur,
          const __grid_constant__ CUtensorMap tm_vcur, const __grid_constant__ CUtensorMap tm_sh,
          const __grid_constant__ CUtensorMap tm_sl, const __grid_constant__ CUtensorMap tm_o,
          const __grid_constant__ Tc5Params p) {
    using namespace tc5;
    typedef SwaTc5<D, NG> C;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t s_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    if (s_base - smem_u32(smem_raw) + C::USED_BYTES > C::SMEM_BYTES) {   // the window started too far off a 1 KB boundary
        if (threadIdx.x == 0) { atomicOr(p.dev_status, HF_DEV_TIMEOUT_FLAG); atomicExch(p.dev_status + 1, 99); }
        return;
    }
    uint8_t* s_gen = smem_raw + (s_base - smem_u32(smem_raw));
    const uint32_t sQ = s_base + C::OFF_Q, sK = s_base + C::OFF_K, sV = s_base + C::OFF_V, sH = s_base + C::OFF_H;
    static_assert(!HIST || C::FUSE, "no room for the folded state in this configuration");
    constexpr bool fuse = HIST;
    const uint32_t bar0 = s_base + C::OFF_BAR;
    // barrier arrays are indexed by stage: address = base + 8 * stage
    const uint32_t bar_kf = bar0, bar_ke = bar0 + 24, bar_vf = bar0 + 48, bar_ve = bar0 + 64, bar_sf = bar0 + 80,
                   bar_pf = bar0 + 104, bar_pv = bar0 + 128, bar_mx = bar0 + 160, bar_qf = bar0 + 176, bar_qe = bar0 + 184,
                   bar_ep = bar0 + 192, bar_drain = bar0 + 200,
                   // history term: every thread has read the last tile's maxima / S W^T loaded / ... free again /
                   // phi(Q) operand written / the unit's accumulator complete
                   bar_rd = bar0 + 216, bar_hf = bar0 + 224, bar_he = bar0 + 232, bar_af = bar0 + 240, bar_ud = bar0 + 248,
                   bar_h2 = bar0 + 256;                    // ... and its hi tile loaded (after the copy of Q has been read)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(s_gen + C::OFF_BAR + 208);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(s_gen + C::OFF_BAR + 212);
    // units whose rows left the range of the fixed reference: count, last unit listed, up to REDO_CAP local unit numbers
    // (more than that: every unit of this thread block is computed again)
    constexpr int REDO_CAP = 8;
    int* redo_cnt = reinterpret_cast<int*>(s_gen + C::OFF_BAR + 264);
    int* redo_last = redo_cnt + 1;
    int* redo_list = redo_cnt + 2;
    static_assert(264 + (2 + REDO_CAP) * 4 <= 320, "the list must fit in front of the exchange buffers");
    static_assert(C::THREADS >= 256, "the second pass over a unit needs eight warps");
    float* x_max = reinterpret_cast<float*>(s_gen + C::OFF_XM);          // [2][NG][128]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int keep = p.keep;
    const int my_units = (p.n_units - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const int n_tiles = my_units * keep;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 3; ++s) { mbar_init(bar_kf + 8 * s, 1); mbar_init(bar_ke + 8 * s, 1); mbar_init(bar_sf + 8 * s, 1); mbar_init(bar_pf + 8 * s, 128 * NG); }
        for (int s = 0; s < 2; ++s) { mbar_init(bar_vf + 8 * s, 1); mbar_init(bar_ve + 8 * s, 1); mbar_init(bar_mx + 8 * s, 128 * NG); }
        for (int s = 0; s < 4; ++s) mbar_init(bar_pv + 8 * s, 1);
        mbar_init(bar_qf, 1); mbar_init(bar_qe, 1); mbar_init(bar_ep, 128 * NG); mbar_init(bar_drain, 1);
        mbar_init(bar_rd, 128 * NG); mbar_init(bar_hf, 1); mbar_init(bar_he, 4 * NG); mbar_init(bar_af, 128 * NG); mbar_init(bar_ud, 1); mbar_init(bar_h2, 1);
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
    // Everything above (barriers, tensor memory) may overlap the tail of the kernel before this one in the stream when the
    // launch allows it; the index list it wrote is read from here on.
    pdl_wait();
    // The next kernel in the stream may be made resident on SMs this grid has left (it waits itself) -- only where a thread
    // block of this kernel takes all of an SM's shared memory, so that no waiting block of the dependent grid ever sits
    // beside a working block of this one.
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
                if (ok && fuse && is_k) {
                    // For the history term at the unit's end: the lo tile of the head's folded state, and a second copy of
                    // the unit's Q tile where the hi tile will go (the softmax threads take phi(Q) from it; the Q buffer
                    // proper belongs to the next unit by then).  The buffer is free once the previous unit's output,
                    // which was staged in it, has been read by the bulk stores.
                    if (n >= 1 && !(ok = mbar_wait<true>(bar_he, (n - 1) & 1, abort_flag, p.dev_status, 13))) break;
                    mbar_expect_tx(bar_hf, 2 * C::TILE_BYTES);
#pragma unroll
                    for (int s = 0; s < C::SUB; ++s) {
                        tma_load_4d(sH + s * C::SUB_BYTES, &tm_q, s * 64, i * C::BLK, bh, 0, bar_hf);
                        tma_load_4d(sH + C::TILE_BYTES + s * C::SUB_BYTES, &tm_sl, s * 64, 0, bh, 0, bar_hf);
                    }
                }
            }
            if (!ok) {   // gave up: let the copies already in flight land before the CTA leaves
                const long long t0 = clock64();
                while (clock64() - t0 < 400000) {}
            }
        }
    } else if (warp == C::WARP_MMA) {
        // ================================================================= MMA issuer
        // The whole warp walks the loop (uniform control flow, so that descriptors and addresses can live in uniform
        // registers); one elected lane issues the tensor-core instructions.
        constexpr uint32_t IDESC_S = idesc_bf16(128, false);
        constexpr uint32_t IDESC_PV = idesc_bf16(D, true);
        constexpr uint32_t TILE_STEP = C::TILE_BYTES >> 4;      // descriptor address field counts 16-byte units
        const uint32_t tO = tmem + C::COL_O;
        const uint64_t dq0 = smem_desc_sw128(sQ, 16, 1024), dk0 = smem_desc_sw128(sK, 16, 1024);
        const uint64_t dv0 = smem_desc_sw128(sV, C::SUB_BYTES, 1024);
        const uint64_t dh0 = smem_desc_sw128(sH, C::SUB_BYTES, 1024);     // S W^T tiles: laid out like a V tile (rows = contraction index)
        const uint32_t q_lo = (uint32_t)dq0, k_lo = (uint32_t)dk0, v_lo = (uint32_t)dv0, h_lo = (uint32_t)dh0;
        const uint32_t qk_hi = (uint32_t)(dq0 >> 32), v_hi = (uint32_t)(dv0 >> 32);
        bool ok = true;
        int n_s = 0, j_s = 0;                         // unit and position in its list of the next S tile to issue
        RingPos<C::KSTAGES> rk;                       // K stage of the next S tile
        RingPos<C::SBUFS> rb;                         // ... and its S buffer
        auto issue_s = [&]() -> bool {                // S_t = Q K_t^T into S buffer t % 3
            if (j_s == 0 && !__all_sync(0xffffffffu, mbar_wait<true>(bar_qf, n_s & 1, abort_flag, p.dev_status, 4))) return false;
            if (!__all_sync(0xffffffffu, mbar_wait<true>(bar_kf + 8 * rk.stage, rk.phase, abort_flag, p.dev_status, 5))) return false;
            fence_after_sync();
            if (elect_one()) {
                mma_ss_tile<D>(tmem + rb.stage * C::BLK, q_lo, k_lo + rk.stage * TILE_STEP, qk_hi, IDESC_S);
                mma_commit(bar_sf + 8 * rb.stage);
                mma_commit(bar_ke + 8 * rk.stage);
                if (j_s == keep - 1) mma_commit(bar_qe);
            }
            __syncwarp();
            rk.advance();
            rb.advance();
            if (++j_s == keep) { j_s = 0; ++n_s; }
            return true;
        };
        if (n_tiles > 0) ok = issue_s();
        if (ok && n_tiles > 1) ok = issue_s();
        int j_pv = 0, n_pv = 0;                       // position of tile t in its unit's list; the unit
        RingPos<C::SBUFS> rp;                         // S buffer holding P_t
        RingPos<C::VSTAGES> rv;
        for (int t = 0; ok && t < n_tiles; ++t) {
            // With the history term formed here, the S buffer two tiles on takes the phi(Q) operand at a unit's last tile:
            // its S is issued after the history products instead of before this tile's P V.
            const bool last = fuse && (j_pv == keep - 1);
            if (t + 2 < n_tiles && !last && !(ok = issue_s())) break;
            if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_pf + 8 * rp.stage, rp.phase, abort_flag, p.dev_status, 6)))) break;
            if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_vf + 8 * rv.stage, rv.phase, abort_flag, p.dev_status, 7)))) break;
            fence_after_sync();
            if (elect_one()) {
                // P of keys 0..63 at the buffer's columns 0..31, of keys 64..127 where the second column group left them
                mma_ts_tile_split(tO, tmem + rp.stage * C::BLK, tmem + rp.stage * C::BLK + (NG > 1 ? C::GCOLS : 32),
                                  v_lo + rv.stage * TILE_STEP, v_hi, IDESC_PV, j_pv > 0);
                mma_commit(bar_pv + 8 * (t & 3));
                mma_commit(bar_ve + 8 * rv.stage);
            }
            __syncwarp();
            if (last) {
                // O += (l / den) phi(Q) S W^T: A = hi (64 columns) and lo (64 columns) halves in S buffer (t + 2) % 3,
                // B = the hi and lo tiles of S W^T; three products, the lo x lo one is below fp32 resolution
                if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_hf, n_pv & 1, abort_flag, p.dev_status, 14)))) break;
                if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_af, n_pv & 1, abort_flag, p.dev_status, 15)))) break;
                fence_after_sync();
                const int sb = rp.stage + 2 >= C::SBUFS ? rp.stage + 2 - C::SBUFS : rp.stage + 2;
                const uint32_t tA = tmem + sb * C::BLK;
                if (elect_one()) mma_ts_tile(tO, tA, h_lo + TILE_STEP, v_hi, IDESC_PV, true);         // hi x lo
                __syncwarp();
                // the hi tile was fetched over the copy of Q once every thread had taken its row from it
                if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_h2, n_pv & 1, abort_flag, p.dev_status, 20)))) break;
                fence_after_sync();
                if (elect_one()) {
                    mma_ts_tile(tO, tA, h_lo, v_hi, IDESC_PV, true);                                  // hi x hi
                    mma_ts_tile(tO, tA + D / 2, h_lo, v_hi, IDESC_PV, true);                          // lo x hi
                    mma_commit(bar_ud);
                }
                __syncwarp();
                if (t + 2 < n_tiles && !(ok = issue_s())) break;
            }
            rp.advance();
            rv.advance();
            if (++j_pv == keep) { j_pv = 0; ++n_pv; }
        }
        // drain: all MMAs issued by this warp have completed before TMEM is freed
        if (elect_one()) mma_commit(bar_drain);
        __syncwarp();
        {
            const long long t0 = clock64();
            while (!mbar_try_wait(bar_drain, 0) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
        }
    } else {
        // ================================================================= softmax / correction / epilogue
        const int grp = warp >> 2;                          // column group
        const int row = (warp & 3) * 32 + lane;             // query row of the tile = TMEM lane
        const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        const uint32_t tO = lane_base + C::COL_O + grp * C::OCOLS;
        constexpr int NC = C::GCOLS / 32;                   // 32-column register chunks of S per thread
        bool ok = true;
        int t = 0;
        RingPos<C::SBUFS> rs;                               // S buffer of tile t
        // P.V of tile i arrives on bar_pv[i & 3] as that barrier's completion number i >> 2.  When these threads wait for
        // tile t - 1 they have seen S of tile t - 1 (or later) land, which follows P.V of tile t - 4 in the tensor pipe,
        // so every earlier completion of that barrier (tiles t - 5, t - 9, ...) has happened; and P.V of tile t + 3
        // cannot be issued before they have arrived on its P.  The barrier is therefore in completion (t - 1) >> 2 or
        // one past it, and the parity test is exact.
        // All softmax threads test a unit's row sums between the same two block-wide exchanges, so listings of unit n all
        // come before any listing of unit n + 1: the exchange on redo_last lets exactly one thread list a unit.
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
            const int bh = u / p.Tm, i = u - bh * p.Tm;
            const int32_t* my_idx = p.idx + (size_t)u * keep;
            const int q0 = i * C::BLK;
            const int nq = min(C::BLK, p.Tc - q0);
            float m_used = -INFINITY, l_run = 0.f;          // l_run: this thread's share of the row sum
            // block index list read one tile ahead (off the critical path); an entry outside [0, T_n) -- the loader reads
            // block 0 for it and reports it -- is simply no tail here, so the loaded value is not touched until its tile comes
            int blk_next = __ldg(my_idx);
            if (fuse && n >= 1) {
                // The output tile of the previous unit was staged where S W^T lives: the loader may refill the buffer once
                // every warp's bulk store has read its part.  And that unit used both exchange buffers for its row sums and
                // denominators: every thread has read them once it has arrived with its phi(Q) operand.
                if (lane == 0) {
                    bulk_wait_read();
                    mbar_arrive(bar_he);
                }
                __syncwarp();
                ok = __all_sync(0xffffffffu, mbar_wait(bar_af, (n - 1) & 1, abort_flag, p.dev_status, 16));
                if (!ok) break;
            }
            for (int j = 0; j < keep; ++j, ++t) {
                // a chunk's last block may be short; found without an integer division (those run on the XU pipe and
                // would queue behind the other warp's exponentials)
                bool tail = false;
#pragma unroll
                for (int c = 1; c <= HF_MAX_CHUNKS; ++c) tail |= (blk_next + 1 == c * p.n_b);
                if (j + 1 < keep) blk_next = __ldg(my_idx + j + 1);
                const int nv = tail ? p.Tc - (p.n_b - 1) * C::BLK : C::BLK;
                const int st = t & 1;
                const uint32_t tS = lane_base + rs.stage * C::BLK;
                ok = __all_sync(0xffffffffu, mbar_wait(bar_sf + 8 * rs.stage, rs.phase, abort_flag, p.dev_status, 8));
                if (!ok) break;
                rs.advance();
                fence_after_sync();
                // ---- this thread's share of the S row in registers
                uint32_t r[NC][32];
#pragma unroll
                for (int c = 0; c < NC; ++c) tmem_ld32(tS + grp * C::GCOLS + c * 32, r[c]);
                tmem_wait_ld();
                if (nv < C::BLK) {
#pragma unroll
                    for (int c = 0; c < NC; ++c)
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (grp * C::GCOLS + c * 32 + e >= nv) r[c][e] = 0xff800000u;   // -inf
                }
                if (j == 0) {
                    // ---- the reference exponent of the row for the whole unit: the maximum of its first kept tile plus
                    // HEADROOM (2^60).  No running maximum, no rescaling and no exchange between the column groups after
                    // this.  P of the first tile is <= 2^-60; a later tile may rise above the first one by a factor of up to
                    // ~2^150 (about 100 natural-log units) before the row sum passes 2^100, which the end of the unit
                    // detects and reports (fp32 overflows at 2^128; rows that fall below the first tile lose nothing: what
                    // flushes to zero is 2^-66 of the largest term).  Floating point is scale invariant, so the result is
                    // the one the exact running maximum gives.
                    float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int c = 0; c < NC; ++c)
#pragma unroll
                        for (int e = 0; e < 32; e += 2)     // three-input maximum: two values per instruction
                            mx[(e >> 1) & 3] = fmax3(mx[(e >> 1) & 3], __uint_as_float(r[c][e]), __uint_as_float(r[c][e + 1]));
                    float mrow = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                    if (NG > 1) {
                        float* xm = x_max + (n & 1) * NG * C::BLK;
                        xm[grp * C::BLK + row] = mrow;
                        mbar_arrive(bar_mx + 8 * (n & 1));
                        ok = __all_sync(0xffffffffu, mbar_wait(bar_mx + 8 * (n & 1), (n >> 1) & 1, abort_flag, p.dev_status, 11));
                        if (!ok) break;
#pragma unroll
                        for (int g = 0; g < NG; ++g) mrow = fmaxf(mrow, xm[g * C::BLK + row]);
                        mbar_arrive(bar_rd);                // this thread is done with the buffer
                    }
                    m_used = fmaf(mrow, p.scale_log2, C::HEADROOM);
                    if (NG > 1 && grp > 0) {
                        // The exchange above has put the column groups in step.  The two warps that share a scheduler
                        // (same rows, different column groups) then run their exponentials at the same time and their
                        // waits at the same time, and the special-function unit idles through the latter; set back by part
                        // of a tile, one group's waits fall into the other's exponentials.  Nothing couples the groups
                        // until the end of the unit, so the offset stays.
                        const long long t_skew = clock64();
                        while (clock64() - t_skew < C::SKEW_CLK * grp) {}
                    }
                }
                // ---- P = exp2(S*c - m), row sum, bf16 pairs written over the thread's own S columns (group g: key columns
                // 64 g .. 64 g + 63 -> columns 64 g .. 64 g + 31 of the buffer; no group writes where another one reads)
                // (packed fp32: the scale-and-shift and the row sum handle two columns per instruction)
                float2 rsum[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                const float2 scale2 = make_float2(p.scale_log2, p.scale_log2), negm2 = make_float2(-m_used, -m_used);
#pragma unroll
                for (int c = 0; c < NC; ++c) {
                    uint32_t pk[16];
#pragma unroll
                    for (int e0 = 0; e0 < 32; e0 += 8) {    // four column pairs at a time, stage by stage: independent work side by side
                        float2 x[4], pe[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            x[u] = ffma2(make_float2(__uint_as_float(r[c][e0 + 2 * u]), __uint_as_float(r[c][e0 + 2 * u + 1])), scale2, negm2);
#pragma unroll
                        for (int u = 0; u < 4; ++u) pe[u] = make_float2(fast_exp2(x[u].x), fast_exp2(x[u].y));
#pragma unroll
                        for (int u = 0; u < 4; ++u) rsum[u] = fadd2(rsum[u], pe[u]);
#pragma unroll
                        for (int u = 0; u < 4; ++u) pk[(e0 >> 1) + u] = pack_bf16_alu(pe[u].x, pe[u].y);
                    }
                    tmem_st16(tS + grp * C::GCOLS + c * 16, pk);
                }
                l_run += ((rsum[0].x + rsum[0].y) + (rsum[1].x + rsum[1].y)) + ((rsum[2].x + rsum[2].y) + (rsum[3].x + rsum[3].y));
                tmem_wait_st();
                fence_before_sync();
                mbar_arrive(bar_pf + 8 * (rs.stage == 0 ? C::SBUFS - 1 : rs.stage - 1));
            }
            if (!ok) break;
            // ---- end of the unit.  The exchange buffers of the row maxima carry the groups' row sums (and, with the
            // history term formed here, their shares of Eq. 4's denominator) once every thread has read the last maxima.
            float inv;
            if (NG > 1) {
                ok = __all_sync(0xffffffffu, mbar_wait(bar_rd, n & 1, abort_flag, p.dev_status, 17));
                if (!ok) break;
            }
            float* x_l = x_max + (n & 1) * NG * C::BLK;           // this unit's buffer: next written two units on
            float* x_d = x_max + ((n + 1) & 1) * NG * C::BLK;     // the next unit's buffer: see the wait at a unit's start
            if constexpr (fuse) {
                // ---- history term (Eq. 4): A = (l / den) phi(q) as bf16 hi + lo, this group's 64 features of the row,
                // read from global memory (the Q tile in shared memory already belongs to the next unit)
                constexpr int FPT = D / NG;                         // features per thread
                const int feat0 = grp * FPT;
                uint4 qv[FPT / 8];
                {
                    ok = __all_sync(0xffffffffu, mbar_wait(bar_hf, n & 1, abort_flag, p.dev_status, 21));
                    if (!ok) break;
                    // this group's 64-column sub-tile of the copy, 128-byte swizzle (rows past the chunk's end: zero fill)
                    const uint8_t* qrow = s_gen + C::OFF_H + grp * C::SUB_BYTES + row * 128;
#pragma unroll
                    for (int c = 0; c < FPT / 8; ++c) qv[c] = *reinterpret_cast<const uint4*>(qrow + ((c ^ (row & 7)) << 4));
                }
                float f[FPT];
                float dsum = 0.f;
                const float4* zsrc = reinterpret_cast<const float4*>(p.z + (size_t)bh * D + feat0);
#pragma unroll
                for (int c = 0; c < FPT / 8; ++c) {
                    const float4 z0 = __ldg(zsrc + 2 * c), z1 = __ldg(zsrc + 2 * c + 1);
                    const float zz[8] = {z0.x, z0.y, z0.z, z0.w, z1.x, z1.y, z1.z, z1.w};
                    const uint32_t ws[4] = {qv[c].x, qv[c].y, qv[c].z, qv[c].w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 x = unpack_bf16(ws[e]);
                        const float f0 = phi_elu1(x.x), f1 = phi_elu1(x.y);
                        f[c * 8 + 2 * e] = f0; f[c * 8 + 2 * e + 1] = f1;
                        dsum = fmaf(f0, zz[2 * e], fmaf(f1, zz[2 * e + 1], dsum));
                    }
                }
                x_l[grp * C::BLK + row] = l_run;
                x_d[grp * C::BLK + row] = dsum;
                mbar_arrive(bar_ep);
                ok = __all_sync(0xffffffffu, mbar_wait(bar_ep, n & 1, abort_flag, p.dev_status, 12));
                if (!ok) break;
                if (warp == 0 && lane == 0) {
                    // every thread has taken its row of the Q copy (it arrived above only after that): the hi tile of the
                    // folded state can come in over it
                    mbar_expect_tx(bar_h2, C::TILE_BYTES);
#pragma unroll
                    for (int s = 0; s < C::SUB; ++s) tma_load_4d(sH + s * C::SUB_BYTES, &tm_sh, s * 64, 0, bh, 0, bar_h2);
                }
                float den = p.eps;
                l_run = 0.f;
#pragma unroll
                for (int g = 0; g < NG; ++g) { l_run += x_l[g * C::BLK + row]; den += x_d[g * C::BLK + row]; }
                inv = 1.f / l_run;
                if (!(l_run < 1e30f)) note_redo(n);     // overflow (or NaN): a later tile rose too far above the first one
                const float fac = l_run / den;                      // O is divided by l at the end: pre-multiply the history term
                // the S buffer two tiles on held P of the tile before the unit's last one: its P V must have read it
                if (t >= 2) {
                    ok = __all_sync(0xffffffffu, mbar_wait(bar_pv + 8 * ((t - 2) & 3), ((t - 2) >> 2) & 1, abort_flag, p.dev_status, 18));
                    if (!ok) break;
                    fence_after_sync();
                }
                const int sb = rs.stage + 1 >= C::SBUFS ? rs.stage + 1 - C::SBUFS : rs.stage + 1;   // rs: buffer of tile t; + 1 = (t_last + 2) % 3
                const uint32_t tA = lane_base + sb * C::BLK + feat0 / 2;
#pragma unroll
                for (int h = 0; h < FPT / 32; ++h) {
                    uint32_t hi[16], lo[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        const float a0 = f[h * 32 + 2 * e] * fac, a1 = f[h * 32 + 2 * e + 1] * fac;
                        const uint32_t hp = pack_bf16(a0, a1);
                        const float2 hf = unpack_bf16(hp);
                        hi[e] = hp;
                        lo[e] = pack_bf16(a0 - hf.x, a1 - hf.y);
                    }
                    tmem_st16(tA + h * 16, hi);
                    tmem_st16(tA + D / 2 + h * 16, lo);
                }
                tmem_wait_st();
                fence_before_sync();
                mbar_arrive(bar_af);
                // the unit's accumulator: its last P V and the three history products
                ok = __all_sync(0xffffffffu, mbar_wait(bar_ud, n & 1, abort_flag, p.dev_status, 19));
                if (!ok) break;
                fence_after_sync();
            } else {
                if (NG > 1) {
                    x_l[grp * C::BLK + row] = l_run;
                    mbar_arrive(bar_ep);
                    ok = __all_sync(0xffffffffu, mbar_wait(bar_ep, n & 1, abort_flag, p.dev_status, 12));
                    if (!ok) break;
                    l_run = x_l[row];
#pragma unroll
                    for (int g = 1; g < NG; ++g) l_run += x_l[g * C::BLK + row];
                }
                ok = wait_pv_prev(10);
                if (!ok) break;
                fence_after_sync();
                inv = 1.f / l_run;
                if (!(l_run < 1e30f)) note_redo(n);     // overflow (or NaN): a later tile rose too far above the first one
            }
            const bf16* bias_row = (fuse && p.bias) ? p.bias + (size_t)(bh % p.heads) * D : nullptr;
            const size_t g_row = (size_t)bh * p.Tc + q0 + row;
            if (grp == 0 && row < nq && p.lse) p.lse[g_row] = (m_used + log2f(l_run)) * 0.6931471805599453f;
            if constexpr (C::FUSE) {
                // Output through shared memory and one bulk tensor store per warp (32 rows x 64 columns): row-per-thread
                // global stores would touch 32 lines per instruction.  The staging tile is the S W^T buffer (free: the
                // history products have completed, or were never asked for); layout = the 128-byte swizzle of the map.
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
                        if (bias_row) {     // Eq. 4's Linear: its matrix is folded into the state, its bias is added here
                            const uint4 bw = __ldg(reinterpret_cast<const uint4*>(bias_row + grp * C::OCOLS + c * 32 + v * 8));
                            const float2 b0 = unpack_bf16(bw.x), b1 = unpack_bf16(bw.y), b2 = unpack_bf16(bw.z), b3 = unpack_bf16(bw.w);
                            x[0] += b0.x; x[1] += b0.y; x[2] += b1.x; x[3] += b1.y;
                            x[4] += b2.x; x[5] += b2.y; x[6] += b3.x; x[7] += b3.y;
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
            // the next unit's first P.V overwrites O: it is gated by p_full of that tile, which these threads
            // arrive on only after this epilogue
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
    // ---- second pass (rare): the listed units again, with the running maximum.  Every copy and tensor-core operation
    // of the tile stream has completed (the roles above drain before the barrier), so shared memory is free.
    const int n_redo = *redo_cnt;
    if (n_redo > 0 && *abort_flag == 0 && threadIdx.x < 256) {
        fence_proxy_async();                                  // the tile stream's bulk stores of these rows came first
        const int total = n_redo > REDO_CAP ? my_units : n_redo;
        for (int r = 0; r < total; ++r) {
            const int n = n_redo > REDO_CAP ? r : redo_list[r];
            swa_redo_unit<D, HIST>(s_gen, p, (int)blockIdx.x + n * (int)gridDim.x);
        }
    }
}
