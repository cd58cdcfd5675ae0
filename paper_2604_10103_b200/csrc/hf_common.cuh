// Shared device/host definitions of libhf (CUDA path only; the CPU oracle shares nothing with this).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

typedef __nv_bfloat16 bf16;

#define HF_MAX_CHUNKS 8      // cached chunks + the current one
#define HF_MAX_TN 1024       // key blocks a selection row may span

// Window of one forward call in logical order: cached chunks oldest first, the current chunk last.
struct ChunkTable {
    const bf16* k[HF_MAX_CHUNKS];        // [B*H, T_c, d] each
    const bf16* v[HF_MAX_CHUNKS];
    const float* pooled[HF_MAX_CHUNKS];  // per-block K means [B*H, n_b, d]
    int n_chunks;
};

// Device status word layout (int[4]): [0] flags, [1] detail, [2] units the tcgen05 attention kernel computed a second
// time with a running maximum (a counter, not an error), [3] reserved.
enum { HF_DEV_TIMEOUT_FLAG = 1, HF_DEV_BAD_INDEX_FLAG = 2 };

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may start while its predecessor
// in the stream still runs (once every block of the predecessor has called pdl_trigger or exited); pdl_wait returns when the
// predecessor has completed and its writes are visible.  Both are no-ops for a kernel launched the ordinary way.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }

// A kept-block index read from a caller's list: inside [0, Tn) it is returned as it is; anything else is replaced by
// block 0 (so that every address formed from it stays inside the cache) and recorded in the status word.
__device__ __forceinline__ int checked_block(int j, int Tn, int* dev_status, int unit) {
    if ((unsigned)j < (unsigned)Tn) return j;
    if (dev_status) {
        atomicOr(dev_status, HF_DEV_BAD_INDEX_FLAG);
        atomicExch(dev_status + 1, unit);
    }
    return 0;
}

// ---------------------------------------------------------------------------------------------
// small PTX helpers (legacy tensor path: ldmatrix + mma.sync, cp.async)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    int sz = valid ? 16 : 0;   // size 0: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// D(16x8, f32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);   // .x = lo (low 16 bits), .y = hi
    return *reinterpret_cast<uint32_t*>(&t);
}
// The same packing on the integer pipe (two adds and a byte permute), for loops whose conversion unit is the busy one:
// round to nearest with ties away from zero, which differs from pack_bf16 only on exact ties.  Finite or infinite
// inputs (an infinity stays one; a NaN stays a NaN).
__device__ __forceinline__ uint32_t pack_bf16_alu(float lo, float hi) {
    return __byte_perm(__float_as_uint(lo) + 0x8000u, __float_as_uint(hi) + 0x8000u, 0x7632);
}
__device__ __forceinline__ float2 unpack_bf16(uint32_t u) {
    return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xFFFF0000u));
}
// Byte offset of the 16-byte chunk `chunk` of row `row` in a tile whose rows are ROW_BYTES long,
// chunks XOR-swizzled by the row so that ldmatrix reads are bank-conflict free.
template <int ROW_BYTES>
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
    return static_cast<uint32_t>(row * ROW_BYTES + ((chunk ^ (row & 7)) << 4));
}
__device__ __forceinline__ float fast_exp2(float x) {   // ex2.approx: 2 ulp, exp2(-inf) = +0
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}
// sm_100 packed fp32 arithmetic (two lanes per instruction) and the three-input maximum
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
    uint64_t rd;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(rd)
        : "l"(*reinterpret_cast<uint64_t*>(&a)), "l"(*reinterpret_cast<uint64_t*>(&b)), "l"(*reinterpret_cast<uint64_t*>(&c)));
    return *reinterpret_cast<float2*>(&rd);
}
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) {
    uint64_t rd;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(rd) : "l"(*reinterpret_cast<uint64_t*>(&a)), "l"(*reinterpret_cast<uint64_t*>(&b)));
    return *reinterpret_cast<float2*>(&rd);
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// phi(x) = elu(x) + 1.  The exponential is ex2.approx.ftz of x log2(e) (2 ulp; results below 2^-126 flush to zero, which
// is below anything the state or the read-out can resolve): the non-flushing form costs several more instructions
// per value, and the state update is bound by exactly these.
__device__ __forceinline__ float phi_elu1(float x) { return x > 0.f ? x + 1.f : fast_exp2(x * 1.4426950408889634f); }
