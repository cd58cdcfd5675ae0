// hf_state_absorb_noalloc: the state update (S += phi(K)^T V, z += sum phi(K)) for callers that must not
// allocate device memory.  The split partials that hf_state_absorb keeps in a buffer of its context live
// here in one file-scope device array instead.
#include "../../include/hf.h"
#include "hf_common.cuh"
#include "k_state_mma.cuh"

#include <cstdio>
#include <mutex>

extern "C" void hf_internal_set_error(const char* text);

namespace {

constexpr size_t NOALLOC_SCRATCH_BYTES = 16u << 20;     // 16 MiB, held by every device that loads the library
constexpr size_t NOALLOC_TICKET_BYTES = 4096;           // first 4 KiB: reserved for bookkeeping words
constexpr int NOALLOC_MAX_BH = 1024;
constexpr int NOALLOC_MAX_DEVICES = 64;

// Scratch shared by every call on a device: [reserved 4 KiB | split partials].  In host code this name is only a
// handle for cudaGetSymbolAddress; it is never passed to a kernel as a pointer.
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_SCRATCH_BYTES];

std::mutex g_setup_mutex;
unsigned char* g_scratch_addr[NOALLOC_MAX_DEVICES] = {};   // device address of g_noalloc_scratch, per device

hf_status nfail(hf_status s, const char* fmt, long long a = 0, long long b = 0) {
    char buf[256];
    snprintf(buf, sizeof(buf), fmt, a, b);
    hf_internal_set_error(buf);
    return s;
}

// Once per device, with that device current: resolve the device address of the scratch array and raise the
// kernels' dynamic shared-memory limit.  Neither step allocates.
hf_status setup_device(int dev, unsigned char** scratch) {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        void* ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
        if (e != cudaSuccess || ptr == nullptr) return nfail(HF_ERR_CUDA, "cudaGetSymbolAddress(scratch) failed with error %lld", (long long)e);
        e = cudaFuncSetAttribute(k_absorb_mma<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, AbsorbMma<64>::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(k_absorb_mma<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, AbsorbMma<128>::SMEM_BYTES);
        if (e != cudaSuccess) return nfail(HF_ERR_CUDA, "cudaFuncSetAttribute failed with error %lld", (long long)e);
        g_scratch_addr[dev] = static_cast<unsigned char*>(ptr);
    }
    *scratch = g_scratch_addr[dev];
    return HF_OK;
}

template <int D>
hf_status run(const bf16* k, const bf16* v, int bh, int n_tokens, float* S, float* z, unsigned char* scratch, cudaStream_t st) {
    typedef AbsorbMma<D> A;
    const size_t part_bytes = (size_t)A::PART_FLOATS * sizeof(float);
    const size_t room = (NOALLOC_SCRATCH_BYTES - NOALLOC_TICKET_BYTES) / part_bytes;   // partials that fit
    if ((size_t)bh > room)
        return nfail(HF_ERR_SHAPE, "batch_heads %lld exceeds the %lld partials the static scratch holds at this head_dim", bh, (long long)room);
    const int n_tiles = (n_tokens + A::TT - 1) / A::TT;
    int nsplit = (int)(room / (size_t)bh);
    if (nsplit > 32) nsplit = 32;
    if (nsplit > n_tiles) nsplit = n_tiles;
    float* partials = reinterpret_cast<float*>(scratch + NOALLOC_TICKET_BYTES);
    // the array keeps whatever the previous call left; every partial that is read below is first rewritten in full
    k_absorb_mma<D><<<dim3(nsplit, bh), A::THREADS, A::SMEM_BYTES, st>>>(k, v, n_tokens, partials);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) {
        k_reduce_fold<D><<<dim3(D / 16, bh), D, 0, st>>>(partials, nsplit, nsplit < 2 ? nsplit : 2, S, z, 1.f, nullptr, 1, bh, nullptr, nullptr, 0ull);
        e = cudaGetLastError();
    }
    if (e != cudaSuccess) return nfail(HF_ERR_CUDA, "kernel launch failed with error %lld", (long long)e);
    return HF_OK;
}

}  // namespace

extern "C" hf_status hf_state_absorb_noalloc(const void* k_ev, const void* v_ev, int batch_heads, int n_tokens, int head_dim,
                                             float* S, float* z, void* stream) {
    if (!k_ev || !v_ev || !S || !z) return nfail(HF_ERR_INVALID_ARG, "null pointer argument");
    if (((uintptr_t)k_ev | (uintptr_t)v_ev | (uintptr_t)S | (uintptr_t)z) & 15u) return nfail(HF_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    if (head_dim != 64 && head_dim != 128) return nfail(HF_ERR_SHAPE, "head_dim %lld not in {64, 128}", head_dim);
    if (n_tokens < 1) return nfail(HF_ERR_SHAPE, "n_tokens must be >= 1");
    if (batch_heads < 1 || batch_heads > NOALLOC_MAX_BH)
        return nfail(HF_ERR_SHAPE, "batch_heads %lld outside [1, %lld]", batch_heads, NOALLOC_MAX_BH);
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { cudaGetLastError(); return nfail(HF_ERR_CUDA, "cudaGetDevice failed with error %lld", (long long)e); }
    if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return nfail(HF_ERR_UNSUPPORTED, "device index %lld not supported", dev);
    unsigned char* scratch = nullptr;
    hf_status s = setup_device(dev, &scratch);
    if (s != HF_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    if (head_dim == 128)
        return run<128>((const bf16*)k_ev, (const bf16*)v_ev, batch_heads, n_tokens, S, z, scratch, st);
    return run<64>((const bf16*)k_ev, (const bf16*)v_ev, batch_heads, n_tokens, S, z, scratch, st);
}
