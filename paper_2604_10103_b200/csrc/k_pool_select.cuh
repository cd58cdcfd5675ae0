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
    bf16* copy_dst;         // same shape, or nullptr
    float* pooled;          // [B*H, n_b, d] block means, or nullptr (copy only)
};
struct PoolJobs { PoolJob job[3]; };

// grid (n_b, B*H, jobs), 256 threads: 16 threads per token row, 16 rows per pass.
template <int D>
__global__ void __launch_bounds__(256) k_pool_copy(PoolJobs jobs, int Tc, int blk, int n_b) {
    constexpr int VEC = D / 16;
    typedef typename VecLoad<VEC>::T V;
    const PoolJob jb = jobs.job[blockIdx.z];
    const int b_idx = blockIdx.x, bh = blockIdx.y;
    const int t0 = b_idx * blk;
    const int n = min(blk, Tc - t0);
    const int r = threadIdx.x >> 4, cv = threadIdx.x & 15;
    const size_t base = ((size_t)bh * Tc + t0) * D + cv * VEC;
    // all loads of the thread first (up to 8 rows in flight), then the copies, then the chain adds in token order
    constexpr int MAXR = 8;                       // blk <= 128 -> at most 8 rows per chain
    V u[MAXR];
#pragma unroll
    for (int i = 0; i < MAXR; ++i) {
        const int t = r + 16 * i;
        if (t < n) u[i] = __ldg(reinterpret_cast<const V*>(jb.src + base + (size_t)t * D));
    }
    if (jb.copy_dst) {
#pragma unroll
        for (int i = 0; i < MAXR; ++i) {
            const int t = r + 16 * i;
            if (t < n) *reinterpret_cast<V*>(jb.copy_dst + base + (size_t)t * D) = u[i];
        }
    }
    float acc[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
#pragma unroll
    for (int i = 0; i < MAXR; ++i) {
        if (r + 16 * i < n) {
            float f[VEC];
            VecLoad<VEC>::widen(u[i], f);
#pragma unroll
            for (int e = 0; e < VEC; ++e) acc[e] = __fadd_rn(acc[e], f[e]);
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

// A[i][j] = Mean(q_i) . Mean(k_j) in the canonical order, formed by one thread: 32 partials (partial l = columns l,
// l + 32, ... ascending, product and sum rounded separately), then the butterfly.  The shuffle butterfly
// p[l] + p[l ^ off] gives both partners the same value (IEEE addition commutes), so folding the upper half onto the
// lower half level by level yields lane 0's result bit for bit.  sq: the pooled query row (shared memory), kp: the
// pooled key row.
template <int D>
__device__ __forceinline__ float canonical_score(const float* sq, const float4* __restrict__ kp) {
    float pl[32];
#pragma unroll
    for (int m = 0; m < D / 32; ++m) {
        float4 kv[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) kv[i] = __ldg(kp + m * 8 + i);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float kk[4] = {kv[i].x, kv[i].y, kv[i].z, kv[i].w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int l = 4 * i + e;
                const float pr = __fmul_rn(sq[l + 32 * m], kk[e]);
                pl[l] = (m == 0) ? pr : __fadd_rn(pl[l], pr);
            }
        }
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1)
#pragma unroll
        for (int l = 0; l < off; ++l) pl[l] = __fadd_rn(pl[l], pl[l + off]);
    return pl[0];
}

// grid (T_m, B*H), 128 threads.  One query-block row: T_n scores, rank-based top-K under the total order
// (score descending, block index ascending), bit mask + ascending index list.
template <int D>
__global__ void __launch_bounds__(128) k_select(ChunkTable tab, const float* __restrict__ pooled_q,
                                                int n_b, int Tm, int Tn, int keep, int mask_words,
                                                uint32_t* __restrict__ mask, int32_t* __restrict__ idx,
                                                uint32_t* __restrict__ mask_out, int32_t* __restrict__ idx_out,
                                                float* __restrict__ scores_out) {
    __shared__ float sq[D];
    __shared__ float sc[HF_MAX_TN];
    __shared__ uint8_t keepf[HF_MAX_TN];
    const int i = blockIdx.x, bh = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const size_t row = (size_t)bh * Tm + i;
    if (threadIdx.x < D) sq[threadIdx.x] = pooled_q[row * D + threadIdx.x];
    __syncthreads();
    // One thread per key block (see canonical_score).
    for (int j = threadIdx.x; j < Tn; j += 128) {
        const int c = j / n_b, jb = j - c * n_b;
        const float s = canonical_score<D>(sq, reinterpret_cast<const float4*>(tab.pooled[c] + ((size_t)bh * n_b + jb) * D));
        sc[j] = s;
        if (scores_out) scores_out[row * Tn + j] = s;
    }
    __syncthreads();
    for (int j = threadIdx.x; j < Tn; j += 128) {
        const float s = sc[j];
        int rank = 0;
        for (int jj = 0; jj < Tn; ++jj) {
            const float s2 = sc[jj];
            rank += (s2 > s) || (s2 == s && jj < j);
        }
        keepf[j] = rank < keep;
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
                idx[row * keep + pos] = j;
                if (idx_out) idx_out[row * keep + pos] = j;
            }
            running += __popc(word);
        }
    }
}
