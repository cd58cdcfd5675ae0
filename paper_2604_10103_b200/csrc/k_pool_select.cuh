// Block pooling (Eq. 5 "Mean"), cache append, block scores and the per-row top-K (Alg. 3, mask M_c).
//
// Canonical float32 order (the selection must be reproducible bit for bit):
//   block sum, per column: 16 chains, chain r adds tokens r, r+16, ... of the block in ascending order
//   from +0; the chains are then added in ascending r; mean = sum / float(n) with n the block's length.
//   score: 32 partials, partial l = sum over columns l, l+32, ... ascending of rounded products
//   (multiply and add rounded separately, never fused); partials folded as a butterfly +16, +8, +4, +2, +1.
#pragma once
#include "hf_common.cuh"

template <int VEC> struct VecLoad;
template <> struct VecLoad<8> {
    typedef uint4 T;
    static __device__ __forceinline__ void widen(const uint4& u, float* f) {
        float2 a = unpack_bf16(u.x), b = unpack_bf16(u.y), c = unpack_bf16(u.z), d = unpack_bf16(u.w);
        f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y; f[4] = c.x; f[5] = c.y; f[6] = d.x; f[7] = d.y;
    }
};
template <> struct VecLoad<4> {
    typedef uint2 T;
    static __device__ __forceinline__ void widen(const uint2& u, float* f) {
        float2 a = unpack_bf16(u.x), b = unpack_bf16(u.y);
        f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y;
    }
};

struct PoolJob {            // one tensor to pool (and optionally copy) per blockIdx.z
    const bf16* src;        // [B*H, T_c, d]
    bf16* copy_dst;         // same shape, or nullptr (may be src itself: every thread rewrites exactly what it read)
    float* pooled;          // [B*H, n_b, d] block means, or nullptr (copy only)
    // temporal rotation (ROT instantiation): frame f of the chunk is turned by rot_base + rot_per_frame * f index steps
    int rot_on, rot_base, rot_per_frame;
};
struct PoolJobs { PoolJob job[3]; };

// Relative temporal RoPE of the softmax branch (Eq. 8): pairs [first_pair, first_pair + n_pairs) of a token's features
// turn by (index steps) x (the pair's frequency); cosine and sine come from tables over integer steps 0 .. t0 (a backward
// turn uses the entry of |steps| with the sine negated).  The arithmetic order is fixed, because the rotated values feed
// the block selection: x0' = x0 c - x1 s, x1' = x0 s + x1 c, each product and each sum rounded separately in float32, the
// result rounded to bf16 (the cache and the attention operands are bf16).
struct TemporalRope {
    const float* cos_tab;   // [t0 + 1][n_pairs]
    const float* sin_tab;
    int first_pair, n_pairs, tokens_per_frame;
};

// One block of one tensor: copy (optional) and per-column mean in the canonical order.  256 threads: 16 threads per token
// row, 16 rows per pass.
template <int VEC, typename V>
__device__ __forceinline__ V rotate_vec(const V& u, int first_feature, int steps, const TemporalRope& tr) {
    float f[VEC];
    VecLoad<VEC>::widen(u, f);
    const int a = steps < 0 ? -steps : steps;
    uint32_t w[VEC / 2];
#pragma unroll
    for (int e = 0; e < VEC; e += 2) {
        const int pr = (first_feature + e) / 2 - tr.first_pair;
        float y0 = f[e], y1 = f[e + 1];
        if (pr >= 0 && pr < tr.n_pairs) {
            const float c = __ldg(tr.cos_tab + (size_t)a * tr.n_pairs + pr);
            float sn = __ldg(tr.sin_tab + (size_t)a * tr.n_pairs + pr);
            if (steps < 0) sn = -sn;
            y0 = __fsub_rn(__fmul_rn(f[e], c), __fmul_rn(f[e + 1], sn));
            y1 = __fadd_rn(__fmul_rn(f[e], sn), __fmul_rn(f[e + 1], c));
        }
        w[e / 2] = pack_bf16(y0, y1);
    }
    V out;
    if constexpr (VEC == 8) { out.x = w[0]; out.y = w[1]; out.z = w[2]; out.w = w[3]; }
    else { out.x = w[0]; out.y = w[1]; }
    return out;
}

template <int D, bool ROT>
__device__ __forceinline__ void pool_copy_block(const PoolJob& jb, int Tc, int blk, int n_b, int b_idx, int bh, const TemporalRope& tr) {
    constexpr int VEC = D / 16;
    typedef typename VecLoad<VEC>::T V;
    const int t0 = b_idx * blk;
    const int n = min(blk, Tc - t0);
    const int r = threadIdx.x >> 4, cv = threadIdx.x & 15;
    const size_t base = ((size_t)bh * Tc + t0) * D + cv * VEC;
    // Two batches of four rows: the loads of a batch first, then its copies, then its chain adds in token order.  (Four
    // 16-byte loads in flight per thread at six thread blocks per SM keep ~100 KB in flight per SM; eight would cost the
    // registers that the sixth block needs.)
    constexpr int MAXR = 8, BATCH = 4;            // blk <= 128 -> at most 8 rows per chain
    float acc[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
#pragma unroll
    for (int i0 = 0; i0 < MAXR; i0 += BATCH) {
        V u[BATCH];
#pragma unroll
        for (int i = 0; i < BATCH; ++i) {
            const int t = r + 16 * (i0 + i);
            if (t < n) {
                // (the rotating instantiation may work in place: plain loads there, the read-only path elsewhere)
                if (ROT) u[i] = *reinterpret_cast<const V*>(jb.src + base + (size_t)t * D);
                else u[i] = __ldg(reinterpret_cast<const V*>(jb.src + base + (size_t)t * D));
                if (ROT) {
                    if (jb.rot_on) u[i] = rotate_vec<VEC, V>(u[i], cv * VEC, jb.rot_base + jb.rot_per_frame * ((t0 + t) / tr.tokens_per_frame), tr);
                }
            }
        }
        if (jb.copy_dst) {
#pragma unroll
            for (int i = 0; i < BATCH; ++i) {
                const int t = r + 16 * (i0 + i);
                if (t < n) *reinterpret_cast<V*>(jb.copy_dst + base + (size_t)t * D) = u[i];
            }
        }
#pragma unroll
        for (int i = 0; i < BATCH; ++i) {
            if (r + 16 * (i0 + i) < n) {
                float f[VEC];
                VecLoad<VEC>::widen(u[i], f);
#pragma unroll
                for (int e = 0; e < VEC; ++e) acc[e] = __fadd_rn(acc[e], f[e]);
            }
        }
    }
    if (jb.pooled == nullptr) return;
    __shared__ float part[16][D];
#pragma unroll
    for (int e = 0; e < VEC; ++e) part[r][cv * VEC + e] = acc[e];
    __syncthreads();
    if (threadIdx.x < D) {
        float tot = part[0][threadIdx.x];
#pragma unroll
        for (int rr = 1; rr < 16; ++rr) tot = __fadd_rn(tot, part[rr][threadIdx.x]);
        jb.pooled[((size_t)bh * n_b + b_idx) * D + threadIdx.x] = __fdiv_rn(tot, (float)n);
    }
}

// grid (n_b, B*H, jobs), 256 threads.
template <int D>
__global__ void __launch_bounds__(256, 6) k_pool_copy(PoolJobs jobs, int Tc, int blk, int n_b) {
    pdl_wait();                 // launched under the tail of the kernel before it: that kernel's reads and writes are done from here on
    pdl_trigger();              // a dependent kernel (the selection) may be made resident; it waits for this grid itself
    const PoolJob jb = blockIdx.z == 0 ? jobs.job[0] : blockIdx.z == 1 ? jobs.job[1] : jobs.job[2];   // (no indexed copy of the parameter block)
    TemporalRope none = {nullptr, nullptr, 0, 0, 1};
    pool_copy_block<D, false>(jb, Tc, blk, n_b, blockIdx.x, blockIdx.y, none);
}
// The same with the temporal rotation applied to the jobs that ask for it (before the copy and the means).
template <int D>
__global__ void __launch_bounds__(256, 4) k_pool_copy_rot(PoolJobs jobs, int Tc, int blk, int n_b, TemporalRope tr) {
    pdl_wait();
    pdl_trigger();
    const PoolJob jb = blockIdx.z == 0 ? jobs.job[0] : blockIdx.z == 1 ? jobs.job[1] : jobs.job[2];
    pool_copy_block<D, true>(jb, Tc, blk, n_b, blockIdx.x, blockIdx.y, tr);
}

// The cache commit of several layers in one launch (Alg. 2 "KV.append" for every layer of the model): per layer the
// clean chunk's K (copied, block means stored) and V (copied) go to the ring slot slot[l] of that layer.
// grid (n_b, B*H, 2 * layers): blockIdx.z = 2 * layer + (0: K, 1: V).
struct PoolLayersParams {
    const bf16* k_src[64];      // per layer of the call: [B*H, T_c, d]
    const bf16* v_src[64];
    int slot[64];               // target slot within the layer's ring
    bf16* ring_k;               // first layer of the call: [layers][slots_per_layer][B*H, T_c, d]
    bf16* ring_v;
    float* pooled;              // [layers][slots_per_layer][B*H, n_b, d]
    size_t chunk_elems, pooled_elems;
    int slots_per_layer;
};
template <int D>
__global__ void __launch_bounds__(256, 6) k_pool_copy_layers(const __grid_constant__ PoolLayersParams p, int Tc, int blk, int n_b) {
    pdl_wait();
    pdl_trigger();
    const int lay = blockIdx.z >> 1;
    const bool is_v = blockIdx.z & 1;
    const size_t s = (size_t)lay * p.slots_per_layer + p.slot[lay];
    PoolJob jb;
    jb.src = is_v ? p.v_src[lay] : p.k_src[lay];
    jb.copy_dst = (is_v ? p.ring_v : p.ring_k) + s * p.chunk_elems;
    jb.pooled = is_v ? nullptr : p.pooled + s * p.pooled_elems;
    jb.rot_on = 0; jb.rot_base = 0; jb.rot_per_frame = 0;
    TemporalRope none = {nullptr, nullptr, 0, 0, 1};
    pool_copy_block<D, false>(jb, Tc, blk, n_b, blockIdx.x, blockIdx.y, none);
}

// A[i][j] = Mean(q_i) . Mean(k_j) in the canonical order, formed by one warp: 32 partials (partial l = columns l,
// l + 32, ... ascending, product and sum rounded separately; lane l holds partial l, so the loads of a key row are
// coalesced), then the butterfly p[l] + p[l ^ off], off = 16 .. 1: both partners get the same value (IEEE addition
// commutes), so lane 0 ends with the fold of the upper half onto the lower half level by level, bit for bit.
// grid (T_m, B*H), 256 threads.  One query-block row: T_n scores, top-K under the total order (score descending, block
// index ascending; by counting for short rows, by a bitonic sort of (score, index) keys for long ones), bit mask +
// ascending index list.
template <int D, bool WIDE>
__global__ void __launch_bounds__(256) k_select(ChunkTable tab, const float* __restrict__ pooled_q,
                                                int n_b, int Tm, int Tn, int keep, int mask_words,
                                                uint32_t* __restrict__ mask, int32_t* __restrict__ idx,
                                                uint32_t* __restrict__ mask_out, int32_t* __restrict__ idx_out,
                                                float* __restrict__ scores_out) {
    __shared__ float sc[HF_MAX_TN];
    __shared__ uint8_t keepf[HF_MAX_TN];
    __shared__ unsigned long long keys[HF_MAX_TN];
    const int i = blockIdx.x, bh = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const size_t row = (size_t)bh * Tm + i;
    pdl_trigger();              // the attention kernel may be made resident as blocks of this grid leave
    pdl_wait();                 // the pooled rows of the query and of the current chunk come from the kernel before
    // One warp per score, lane l = partial l.  All loads of a pass (the lane's columns of the query row and of sixteen key
    // rows) are issued before the first use: one trip to memory per pass, and one pass covers 128 key blocks.
    constexpr int NW = 8, PER = 16, M = D / 32;
    float qv[M];
#pragma unroll
    for (int m = 0; m < M; ++m) qv[m] = __ldg(pooled_q + row * D + lane + 32 * m);
    for (int base = 0; base < Tn; base += NW * PER) {
        float kv[PER][M];
#pragma unroll
        for (int u = 0; u < PER; ++u) {
            const int j = min(base + warp + NW * u, Tn - 1);
            const int c = j / n_b, jb = j - c * n_b;
            const float* kp = tab.pooled[c] + ((size_t)bh * n_b + jb) * D + lane;
#pragma unroll
            for (int m = 0; m < M; ++m) kv[u][m] = __ldg(kp + 32 * m);
        }
        if constexpr (WIDE) {
            // one butterfly per key row (the compiler keeps all loads of the pass in flight in front of them: ~80 registers)
#pragma unroll
            for (int u = 0; u < PER; ++u) {
                float p = __fmul_rn(qv[0], kv[u][0]);
#pragma unroll
                for (int m = 1; m < M; ++m) p = __fadd_rn(p, __fmul_rn(qv[m], kv[u][m]));
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) p = __fadd_rn(p, __shfl_xor_sync(0xffffffffu, p, off));
                const int j = base + warp + NW * u;
                if (lane == 0 && j < Tn) {
                    sc[j] = p;
                    if (scores_out) scores_out[row * Tn + j] = p;
                }
            }
        } else {
            // The sixteen butterflies side by side.  At the step with lane offset `off` a lane keeps the half of its rows
            // that its own bit of `off` names and hands the other half to its partner, which does the opposite: every sum
            // is still own partial + partner's partial (IEEE addition commutes, so both orders give the same bits), level
            // by level as in the one-row butterfly, with 8 + 4 + 2 + 1 + 1 shuffles instead of 16 x 5.  After the last
            // step lanes 2u and 2u + 1 both hold the score of row u.  (The compiler pairs this form's loads with their
            // products: ~40 registers, twice the resident thread blocks, more trips to memory per pass.)
            float pa[PER];
#pragma unroll
            for (int u = 0; u < PER; ++u) {
                float p = __fmul_rn(qv[0], kv[u][0]);
#pragma unroll
                for (int m = 1; m < M; ++m) p = __fadd_rn(p, __fmul_rn(qv[m], kv[u][m]));
                pa[u] = p;
            }
#pragma unroll
            for (int half = PER / 2, off = 16; half >= 1; half >>= 1, off >>= 1) {
                const bool upper = (lane & off) != 0;
#pragma unroll
                for (int x = 0; x < half; ++x) {
                    const float mine = upper ? pa[x + half] : pa[x];
                    const float theirs = upper ? pa[x] : pa[x + half];
                    pa[x] = __fadd_rn(mine, __shfl_xor_sync(0xffffffffu, theirs, off));
                }
            }
            static_assert(PER == 16, "one row per lane pair after four halvings");
            const float score = __fadd_rn(pa[0], __shfl_xor_sync(0xffffffffu, pa[0], 1));
            const int j = base + warp + NW * (lane >> 1);
            if ((lane & 1) == 0 && j < Tn) {
                sc[j] = score;
                if (scores_out) scores_out[row * Tn + j] = score;
            }
        }
    }
    __syncthreads();
    // Keep the `keep` best under a TOTAL order: score descending, then block index ascending; +0 and -0 tie; a NaN score (a
    // NaN anywhere in the query block or the key block) compares false both ways and would otherwise rank first everywhere:
    // here it ranks below every number, NaNs among themselves by block index, so that exactly `keep` blocks are kept whatever
    // the inputs hold.
    // 64-bit keys: an order-preserving image of the score (NaN lowest, -0 = +0), then the complement of the block index;
    // all keys of a row are distinct and "comes before" is "has the larger key"
    auto key_of = [](float s, int j) -> unsigned long long {
        uint32_t u = __float_as_uint(s);
        if (s != s) u = 0u;                                         // NaN: below -inf
        else {
            if (u == 0x80000000u) u = 0u;                           // -0 ties with +0
            u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);         // ascending integers = ascending floats
        }
        return ((unsigned long long)u << 32) | (unsigned long long)(0xffffffffu - (uint32_t)j);
    };
    if (Tn <= 128) {
        // short rows: count, for every block, the blocks that come before it.  Two threads per block, one for the even and
        // one for the odd competitors, four comparisons in flight each.
        for (int j = threadIdx.x; j < Tn; j += 256) keys[j] = key_of(sc[j], j);
        __syncthreads();
        {
            const int j = threadIdx.x >> 1, par = threadIdx.x & 1;
            int rank = 0;
            if (j < Tn) {
                const unsigned long long mine = keys[j];
                int r0 = 0, r1 = 0, r2 = 0, r3 = 0;
                int jj = par;
                for (; jj + 6 < Tn; jj += 8) {
                    r0 += keys[jj] > mine; r1 += keys[jj + 2] > mine; r2 += keys[jj + 4] > mine; r3 += keys[jj + 6] > mine;
                }
                for (; jj < Tn; jj += 2) r0 += keys[jj] > mine;
                rank = (r0 + r1) + (r2 + r3);
            }
            rank += __shfl_xor_sync(0xffffffffu, rank, 1);
            if (par == 0 && j < Tn) keepf[j] = rank < keep;
        }
    } else {
        // long rows (counting is quadratic in T_n): sort the keys in shared memory with a bitonic network and compare every
        // block with the keep-th key
        int n2 = 256;
        while (n2 < Tn) n2 <<= 1;
        for (int j = threadIdx.x; j < n2; j += 256) keys[j] = j < Tn ? key_of(sc[j], j) : 0ull;      // padding sorts last
        __syncthreads();
        for (int size = 2; size <= n2; size <<= 1) {
            for (int stride = size >> 1; stride > 0; stride >>= 1) {
                for (int x = threadIdx.x; x < (n2 >> 1); x += 256) {
                    const int lo = 2 * x - (x & (stride - 1)), hi = lo + stride;      // the pair (lo, lo + stride)
                    const bool descending = (lo & size) == 0;
                    const unsigned long long a = keys[lo], b = keys[hi];
                    if ((a < b) == descending) { keys[lo] = b; keys[hi] = a; }
                }
                __syncthreads();
            }
        }
        const unsigned long long kth = keys[keep - 1];
        for (int j = threadIdx.x; j < Tn; j += 256) keepf[j] = key_of(sc[j], j) >= kth;
    }
    __syncthreads();
    if (warp == 0) {
        int running = 0;
        for (int w = 0; w < mask_words; ++w) {
            const int j = w * 32 + lane;
            const bool f = (j < Tn) && keepf[j];
            const uint32_t word = __ballot_sync(0xffffffffu, f);
            if (lane == 0) {
                mask[row * mask_words + w] = word;
                if (mask_out) mask_out[row * mask_words + w] = word;
            }
            if (f) {
                const int pos = running + __popc(word & ((1u << lane) - 1u));
                if (pos < keep) {       // (always true under the total order above; the store never leaves the row)
                    idx[row * keep + pos] = j;
                    if (idx_out) idx_out[row * keep + pos] = j;
                }
            }
            running += __popc(word);
        }
    }
}
