// Eq. 4's "Linear" read as one projection over the model width: Y[t, :] = W_full X[t, :] + bias per token, X = the
// history read-out h = phi(q) S / (phi(q) . z + eps) of all heads side by side (head-major), W_full [H d, H d] bf16.
// X arrives as bf16 hi + lo halves [B*H, T_c, d] (written by the read-out kernel); the result goes out per head, as the
// fp32 history term the attention kernel adds in its epilogue, or rounded to bf16.
//
// Plain tiled GEMM on the tensor path: thread block = (128 tokens, one output head); the contraction runs over the input
// heads in 64-column steps: A = X tile [128 tokens x 64] (hi, then lo), B = W_full tile [d output rows x 64], both K-major
// with the 128-byte swizzle as TMA writes them; D [128 x d] fp32 in tensor memory = sum over steps of A_hi B^T + A_lo B^T.
// Warp 0 loads (four stages), warp 1 issues the MMAs, warps 2..5 read the accumulator out.  Every wait is bounded.
#pragma once
#include "tc5_common.cuh"

template <int D>
struct MergeFull {
    static constexpr int ROWS = 128, KB = 64;                // tokens per tile, contraction columns per step
    static constexpr int NST = 4;
    static constexpr int A_BYTES = ROWS * 128;               // one 64-column bf16 tile of X (hi or lo): 16 KB
    static constexpr int B_BYTES = D * 128;                  // d output rows x 64 columns of W_full
    static constexpr int STAGE_BYTES = 2 * A_BYTES + B_BYTES;
    static constexpr int OFF_BAR = NST * STAGE_BYTES;
    static constexpr int SMEM_BYTES = OFF_BAR + 128 + 1024;
    static constexpr int THREADS = 192;
    static constexpr int TMEM_COLS = D < 32 ? 32 : D;        // power of two >= 32
};

struct MergeFullParams {
    int heads, Tc, Tm;
    const bf16* bias;         // [H d] or nullptr
    float* out_f32;           // exactly one of the two is non-null: [B*H, T_c, D]
    bf16* out_bf16;
    int* dev_status;
};

// grid (T_m, H, B).  tm_xh, tm_xl: [D, T_c, B*H, 1] box {64, 128}; tm_w: [H d (in), H d (out)] box {64, D}; 128B swizzle.
template <int D>
__global__ void __launch_bounds__(MergeFull<D>::THREADS, 1)
k_merge_full(const __grid_constant__ CUtensorMap tm_xh, const __grid_constant__ CUtensorMap tm_xl,
             const __grid_constant__ CUtensorMap tm_w, const MergeFullParams p) {
    using namespace tc5;
    typedef MergeFull<D> C;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t s_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* s_gen = smem_raw + (s_base - smem_u32(smem_raw));
    const uint32_t bar0 = s_base + C::OFF_BAR;
    const uint32_t bar_full = bar0, bar_free = bar0 + 32, bar_done = bar0 + 64;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(s_gen + C::OFF_BAR + 72);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(s_gen + C::OFF_BAR + 76);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i = blockIdx.x, h_out = blockIdx.y, b = blockIdx.z;
    constexpr int SUB = D / 64;
    const int n_steps = p.heads * SUB;                       // 64-column steps of the contraction

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::NST; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_free + 8 * s, 1); }
        mbar_init(bar_done, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), C::TMEM_COLS);
        tmem_relinquish();
    }
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    pdl_wait();

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            for (int k = 0; ok && k < n_steps; ++k) {
                const int s = k % C::NST;
                if (k >= C::NST && !(ok = mbar_wait<true>(bar_free + 8 * s, ((k / C::NST) & 1) ^ 1u, abort_flag, p.dev_status, 61))) break;
                const int h_in = k / SUB, sub = k - h_in * SUB;
                const uint32_t st = s_base + s * C::STAGE_BYTES;
                mbar_expect_tx(bar_full + 8 * s, C::STAGE_BYTES);
                tma_load_4d(st, &tm_xh, sub * 64, i * C::ROWS, b * p.heads + h_in, 0, bar_full + 8 * s);
                tma_load_4d(st + C::A_BYTES, &tm_xl, sub * 64, i * C::ROWS, b * p.heads + h_in, 0, bar_full + 8 * s);
                tma_load_4d(st + 2 * C::A_BYTES, &tm_w, k * 64, h_out * D, 0, 0, bar_full + 8 * s);
            }
            if (!ok) {
                const long long t0 = clock64();
                while (clock64() - t0 < 400000) {}
            }
        }
    } else if (warp == 1) {
        constexpr uint32_t IDESC = idesc_bf16(D, false);
        bool ok = true;
        for (int k = 0; ok && k < n_steps; ++k) {
            const int s = k % C::NST;
            if (!(ok = __all_sync(0xffffffffu, mbar_wait<true>(bar_full + 8 * s, (k / C::NST) & 1, abort_flag, p.dev_status, 62)))) break;
            fence_after_sync();
            if (elect_one()) {
                const uint32_t st = s_base + s * C::STAGE_BYTES;
                const uint64_t da = smem_desc_sw128(st, 16, 1024), dl = smem_desc_sw128(st + C::A_BYTES, 16, 1024);
                const uint64_t db = smem_desc_sw128(st + 2 * C::A_BYTES, 16, 1024);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {            // 16 columns (32 bytes = 2 descriptor units) per step
                    mma_ss(tmem, da + 2 * ks, db + 2 * ks, IDESC, k > 0 || ks > 0);
                    mma_ss(tmem, dl + 2 * ks, db + 2 * ks, IDESC, true);
                }
                mma_commit(bar_free + 8 * s);
                if (k == n_steps - 1) mma_commit(bar_done);
            }
            __syncwarp();
        }
    } else {
        // ================================================================= epilogue: accumulator + bias -> global
        const int row = (warp & 3) * 32 + lane;                 // TMEM lane quadrant of the warp = warp id mod 4
        const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        bool ok = __all_sync(0xffffffffu, mbar_wait(bar_done, 0, abort_flag, p.dev_status, 63));
        if (ok) {
            fence_after_sync();
            const int t = i * C::ROWS + row;
            const size_t g = (((size_t)b * p.heads + h_out) * p.Tc + t) * D;
#pragma unroll 1
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(lane_base + c0, r);
                tmem_wait_ld();
                if (t < p.Tc) {
                    float x[32];
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        x[e] = __uint_as_float(r[e]) + (p.bias ? __bfloat162float(p.bias[h_out * D + c0 + e]) : 0.f);
                    if (p.out_f32) {
                        float4* dst = reinterpret_cast<float4*>(p.out_f32 + g + c0);
#pragma unroll
                        for (int v = 0; v < 8; ++v) dst[v] = make_float4(x[4 * v], x[4 * v + 1], x[4 * v + 2], x[4 * v + 3]);
                    } else {
                        uint4* dst = reinterpret_cast<uint4*>(p.out_bf16 + g + c0);
#pragma unroll
                        for (int v = 0; v < 4; ++v)
                            dst[v] = make_uint4(pack_bf16(x[8 * v], x[8 * v + 1]), pack_bf16(x[8 * v + 2], x[8 * v + 3]),
                                                pack_bf16(x[8 * v + 4], x[8 * v + 5]), pack_bf16(x[8 * v + 6], x[8 * v + 7]));
                    }
                }
            }
        }
    }
    fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        fence_after_sync();
        tmem_dealloc(tmem, C::TMEM_COLS);
    }
}
