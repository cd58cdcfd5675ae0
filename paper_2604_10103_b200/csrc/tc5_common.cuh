// Blackwell building blocks shared by the tcgen05 kernels: bounded mbarrier waits, TMA tile loads, tensor-memory
// allocation / load / store, MMA issue and commit, shared-memory and instruction descriptors.
#pragma once
#include <cuda.h>
#include "hf_common.cuh"

namespace tc5 {

constexpr long long WAIT_LIMIT_CYCLES = 2000000000LL;   // ~1 s

// ----------------------------------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Same test, but the hardware may park the thread for up to `ns` nanoseconds while the phase is pending: for the
// roles that wait long and often (loaders, MMA issuer) and would otherwise take issue slots from the softmax warps.
__device__ __forceinline__ bool mbar_try_wait_parked(uint32_t bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(ok) : "r"(bar), "r"(parity), "r"(ns) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the limit ran out or another role already gave up.  The polling loop is kept
// out of line: the common case is a barrier that has already flipped.  LIMIT: clock cycles before the wait gives up.
template <bool PARKED, long long LIMIT>
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* dev_status, int where) {
    const long long t0 = clock64();
    for (;;) {
        if (PARKED) {
#pragma unroll 1
            for (int i = 0; i < 8; ++i)
                if (mbar_try_wait_parked(bar, parity, 4000u)) return true;
        } else {
#pragma unroll 1
            for (int i = 0; i < 32; ++i)
                if (mbar_try_wait(bar, parity)) return true;
        }
        if (*abort_flag) return false;
        if (clock64() - t0 > LIMIT) {
            *abort_flag = 1;
            atomicOr(dev_status, HF_DEV_TIMEOUT_FLAG);
            atomicExch(dev_status + 1, where);
            return false;
        }
    }
}
template <bool PARKED = false, long long LIMIT = WAIT_LIMIT_CYCLES>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* dev_status, int where) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow<PARKED, LIMIT>(bar, parity, abort_flag, dev_status, where);
}

// ----------------------------------------------------------------------------------------- TMA
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];\n"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar) : "memory");
}

// Tile store shared -> global through a tensor map (bulk async-group completion).  The shared-memory writes that filled
// the tile must be followed by fence_proxy_async() in the writing threads before the issuing thread is signalled.
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];\n"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;\n" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;\n" ::: "memory"); }   // sources may be overwritten
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;\n" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }

// ----------------------------------------------------------------------------------------- tcgen05
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(taddr), "r"(ncols) : "memory");
}
// True in exactly one lane of a converged warp.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n .reg .pred P;\n elect.sync _|P, 0xffffffff;\n selp.u32 %0, 1, 0, P;\n}\n" : "=r"(pred));
    return pred != 0;
}
__device__ __forceinline__ void fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
// One tile's worth of MMAs in a single instruction stream: the descriptors of consecutive k-steps differ only in
// the address field (low word, 16-byte units), so each step is two adds, two moves and the MMA.
#define HF_SS_STEP(OFF, PRED)                                                                      \
    "add.u32 a, %1, " #OFF ";\n add.u32 b, %2, " #OFF ";\n mov.b64 da, {a, %3};\n mov.b64 db, {b, %3};\n" \
    "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, " PRED ";\n"
// D[tmem] = A[smem] * B[smem] over the whole head dimension (A, B K-major, 128-byte swizzle, 64-column sub-tiles
// SUB_BYTES = 16 KB apart).  a_lo / b_lo: low descriptor words of the tiles, hi: their common high word.
template <int D>
__device__ __forceinline__ void mma_ss_tile(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc) {
    if constexpr (D == 128) {
        asm volatile("{\n .reg .pred pt, pf;\n .reg .b64 da, db;\n .reg .b32 a, b;\n"
                     "setp.eq.u32 pt, %0, %0;\n setp.ne.u32 pf, %0, %0;\n"
                     HF_SS_STEP(0, "pf") HF_SS_STEP(2, "pt") HF_SS_STEP(4, "pt") HF_SS_STEP(6, "pt")
                     HF_SS_STEP(1024, "pt") HF_SS_STEP(1026, "pt") HF_SS_STEP(1028, "pt") HF_SS_STEP(1030, "pt")
                     "}\n" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc) : "memory");
    } else {
        asm volatile("{\n .reg .pred pt, pf;\n .reg .b64 da, db;\n .reg .b32 a, b;\n"
                     "setp.eq.u32 pt, %0, %0;\n setp.ne.u32 pf, %0, %0;\n"
                     HF_SS_STEP(0, "pf") HF_SS_STEP(2, "pt") HF_SS_STEP(4, "pt") HF_SS_STEP(6, "pt")
                     "}\n" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc) : "memory");
    }
}
#undef HF_SS_STEP
#define HF_TS_STEP(KS, PRED)                                                                       \
    "add.u32 a, %1, " #KS " * 8;\n add.u32 b, %2, " #KS " * 128;\n mov.b64 db, {b, %3};\n"          \
    "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], db, %4, " PRED ";\n"
// D[tmem] (+)= A[tmem] * B[smem] over 128 keys: A = bf16 P (8 columns per 16 keys), B = V tile, MN-major,
// 2048 bytes per 16 keys.  accumulate_first: whether the first step adds to D.
__device__ __forceinline__ void mma_ts_tile(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                            bool accumulate_first) {
    asm volatile("{\n .reg .pred pt, p0;\n .reg .b64 db;\n .reg .b32 a, b;\n"
                 "setp.eq.u32 pt, %0, %0;\n setp.ne.b32 p0, %5, 0;\n"
                 HF_TS_STEP(0, "p0") HF_TS_STEP(1, "pt") HF_TS_STEP(2, "pt") HF_TS_STEP(3, "pt")
                 HF_TS_STEP(4, "pt") HF_TS_STEP(5, "pt") HF_TS_STEP(6, "pt") HF_TS_STEP(7, "pt")
                 "}\n" ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"((uint32_t)accumulate_first) : "memory");
}
#undef HF_TS_STEP
// The same product with the A operand in two pieces: keys 0..63 at a_tmem (32 columns), keys 64..127 at a_tmem_hi.
#define HF_TS2_STEP(KS, AOP, AOFF, PRED)                                                            \
    "add.u32 a, " AOP ", " #AOFF " * 8;\n add.u32 b, %2, " #KS " * 128;\n mov.b64 db, {b, %3};\n" \
    "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], db, %4, " PRED ";\n"
__device__ __forceinline__ void mma_ts_tile_split(uint32_t d_tmem, uint32_t a_tmem, uint32_t a_tmem_hi, uint32_t b_lo, uint32_t b_hi,
                                                  uint32_t idesc, bool accumulate_first) {
    asm volatile("{\n .reg .pred pt, p0;\n .reg .b64 db;\n .reg .b32 a, b;\n"
                 "setp.eq.u32 pt, %0, %0;\n setp.ne.b32 p0, %5, 0;\n"
                 HF_TS2_STEP(0, "%1", 0, "p0") HF_TS2_STEP(1, "%1", 1, "pt") HF_TS2_STEP(2, "%1", 2, "pt") HF_TS2_STEP(3, "%1", 3, "pt")
                 HF_TS2_STEP(4, "%6", 0, "pt") HF_TS2_STEP(5, "%6", 1, "pt") HF_TS2_STEP(6, "%6", 2, "pt") HF_TS2_STEP(7, "%6", 3, "pt")
                 "}\n" ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"((uint32_t)accumulate_first), "r"(a_tmem_hi)
                 : "memory");
}
#undef HF_TS2_STEP
// 32 lanes x 32 consecutive 32-bit columns: thread t of the warp gets lane (base lane + t)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
                 "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
                 "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};\n"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                   "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
                   "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
                   "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
                 : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
                 "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};\n"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                   "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
                 : "memory");
}

__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};\n"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem], one k-step
// one MMA step, both operands from shared memory
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool accumulate) {
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate) : "memory");
}
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, bool accumulate) {
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate) : "memory");
}
// Shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1.
// lbo / sbo in bytes.  K-major operand: sbo = stride between 8-row groups (1024), lbo unused.
// MN-major operand: lbo = stride between 64-element groups along MN, sbo = stride between 8-row groups along K.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor, kind::f16: D = f32, A = B = bf16, M = 128.
__host__ __device__ constexpr uint32_t idesc_bf16(int n, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
}

}  // namespace tc5
