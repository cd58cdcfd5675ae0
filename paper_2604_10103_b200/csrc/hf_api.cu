// libhf host side: context, validation, ring bookkeeping (Alg. 2) and kernel dispatch.
#include "../../include/hf.h"
#include "hf_common.cuh"
#include "k_pool_select.cuh"
#include "k_swa_mma.cuh"
#include "k_swa_tc5.cuh"
#include "k_swa_tc5p.cuh"
#include "k_swa_tc5g.cuh"
#include "k_swa_bwd.cuh"
#include "k_readout_bwd.cuh"
#include "k_state_mma.cuh"
#include "k_state_tc5.cuh"
#include "k_state_items.cuh"
#include "k_merge_full.cuh"
#include "k_selftest.cuh"

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

namespace {

thread_local char g_err[512] = "";

hf_status fail(hf_status s, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return s;
}

#define HF_CUDA(call)                                                                                   \
    do {                                                                                                \
        cudaError_t e_ = (call);                                                                        \
        if (e_ != cudaSuccess) return fail(HF_ERR_CUDA, "%s: %s (%s:%d)", #call, cudaGetErrorString(e_), __FILE__, __LINE__); \
    } while (0)

struct LayerState {
    bf16* ring_k = nullptr;      // [P][B*H*T_c*d]
    bf16* ring_v = nullptr;
    float* pooled_k = nullptr;   // [P][B*H*n_b*d]
    float* S = nullptr;          // [B*H, d, d]
    float* z = nullptr;          // [B*H, d]
    bf16* sf_hi = nullptr;       // folded state S W^T, bf16 hi / lo halves
    bf16* sf_lo = nullptr;
    bf16* W = nullptr;           // [H, d, d]
    bf16* bias = nullptr;        // [H, d]
    bool has_w = false, has_bias = false;
    bf16* W_full = nullptr;      // [H d, H d]: the one-matrix reading of Eq. 4's Linear (HF_MERGE_FULL_WIDTH); bias then [H d]
    bool has_wfull = false;
    CUtensorMap tm_wfull;        // [H d (in, contiguous), H d (out)], box = 64 columns x d rows
    uint32_t* mask = nullptr;    // last selection [B*H, T_m, mask_words]
    int32_t* idx = nullptr;      // [B*H, T_m, keep]
    int n_cached = 0, head = 0;  // head = slot of the oldest cached chunk
    int n_sink = 0;              // sink chunks held (slots R, R + 1, ...)
    long long absorbed = 0;
    long long frames = 0;        // latent frames committed so far (sink chunks included): the stream position of Eq. 8
    unsigned long long cache_epoch = 0, sel_epoch = ~0ull;
    int sel_keep = 0;
    CUtensorMap tm_kring, tm_vring;   // 4-D maps over the whole ring [slot, B*H, T_c, d]
    CUtensorMap tm_sfhi, tm_sflo;     // folded state halves [B*H, d, d], box = 64 columns x d rows
};

}  // namespace

struct hf_ctx {
    hf_config cfg;
    int device = 0, sm_count = 0;
    int BH = 0, Tc = 0, n_b = 0, P = 0, R = 0, Tm = 0, max_Tn = 0, mask_words = 0, d = 0;
    int n_sink_max = 0;              // sink chunks of the configuration; ring (R = P + 1 slots: the window's P past chunks and a spare) and sink share one allocation
    size_t chunk_elems = 0, pooled_elems = 0;
    std::vector<LayerState> layers;
    // One allocation per kind for all layers (layer-major; the LayerState pointers point into them), so that a single
    // launch can address every layer: the layer-batched cache commit and state update.
    bf16* ring_k_all = nullptr;      // [layers][slots_per_layer][B*H*T_c*d]
    bf16* ring_v_all = nullptr;
    float* pooled_k_all = nullptr;   // [layers][slots_per_layer][B*H*n_b*d]
    float* S_all = nullptr;          // [layers][B*H, d, d]
    float* z_all = nullptr;          // [layers][B*H, d]
    bf16* sf_hi_all = nullptr;       // [layers][B*H, d, d]
    bf16* sf_lo_all = nullptr;
    bf16* W_all = nullptr;           // [layers][H, d, d] (HF_MERGE_PER_HEAD)
    bf16* bias_all = nullptr;        // [layers][H, d]
    int slots_per_layer = 0;         // ring slots + sink slots
    CUtensorMap tm_kall, tm_vall;    // the state-update kernels' views of all rings: [d, T_c, B*H, layers * slots_per_layer]
    float* pooled_q = nullptr;
    float* pooled_kcur = nullptr;
    float* hist = nullptr;           // fp32 [B*H, T_c, d]: history term handed to the attention epilogue
    bf16* x_hi = nullptr;            // full-width merge: the read-out h of all heads as bf16 hi + lo, [B*H, T_c, d] each
    bf16* x_lo = nullptr;
    uint32_t* union_entries = nullptr;   // small-block tcgen05 attention: merged kept lists [B*H * units, max tiles, G] ...
    int* union_tiles = nullptr;          // ... and tiles per unit
    int union_max_tiles = 0;
    float* bwd_delta = nullptr;          // backward pass: g . o_local per query row [B*H, T_c]
    float* partials = nullptr;       // absorb split partials
    float* partials_layers = nullptr;    // layer-batched state update: one partial per (layer, batch*head, group)
    size_t partials_layers_count = 0;
    int nsplit_max = 1;
    float z_scale = 1.f;             // 1 (z = sum of phi(K)) or 1 / tokens_per_frame (per-frame means)
    bf16* stage[4] = {nullptr, nullptr, nullptr, nullptr};   // q, k, v, o staging of the *_host calls
    int* dev_status = nullptr;
    float* rope_q[2] = {nullptr, nullptr};   // cos / sin tables [T_c, d/2] of Eq. 4's numerator (nullptr: no rotation)
    float* rope_k[2] = {nullptr, nullptr};   // ... of Eq. 3, applied to a chunk when it is absorbed
    bool has_rope_q = false, has_rope_k = false;
    // relative temporal RoPE of the softmax branch (Eq. 8): tables over index steps 0 .. t0, rotated copies of q / k_cur
    bool has_trope = false;
    int t0 = 0;
    TemporalRope trope = {nullptr, nullptr, 0, 0, 1};
    float* trope_tab[2] = {nullptr, nullptr};
    bf16* q_rot = nullptr;
    bf16* k_rot = nullptr;
    cudaStream_t side = nullptr;     // hf_hybrid_forward runs the history read-out here, beside pooling + selection
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    long long launches = 0;
    int swa_kernel = HF_SWA_MMA;
    void* encode_tiled = nullptr;    // cuTensorMapEncodeTiled, resolved through the runtime (no link against libcuda)
};

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

hf_status check_ptr(const void* p, const char* name) {
    if (p == nullptr) return fail(HF_ERR_INVALID_ARG, "%s is null", name);
    if (!aligned16(p)) return fail(HF_ERR_INVALID_ARG, "%s is not 16-byte aligned", name);
    return HF_OK;
}
hf_status check_layer(hf_ctx* c, int layer) {
    if (c == nullptr) return fail(HF_ERR_INVALID_ARG, "ctx is null");
    if (layer < 0 || layer >= c->cfg.layers) return fail(HF_ERR_INVALID_ARG, "layer %d outside [0, %d)", layer, c->cfg.layers);
    return HF_OK;
}
#define HF_TRY(expr) do { hf_status s_ = (expr); if (s_ != HF_OK) return s_; } while (0)

int keep_for(const hf_ctx* c, int Tn) {
    long long k = c->cfg.topk > 0 ? c->cfg.topk : ((long long)c->cfg.keep_permille * Tn + 999) / 1000;
    if (k < 1) k = 1;
    if (k > Tn) k = Tn;
    return (int)k;
}

hf_status validate(const hf_config& g) {
    if (g.batch < 1 || g.heads < 1 || g.layers < 1) return fail(HF_ERR_SHAPE, "batch, heads, layers must be >= 1");
    if (g.head_dim != 64 && g.head_dim != 128) return fail(HF_ERR_SHAPE, "head_dim %d not in {64, 128}", g.head_dim);
    if (g.block != 16 && g.block != 64 && g.block != 128) return fail(HF_ERR_SHAPE, "block %d not in {16, 64, 128}", g.block);
    if (g.tokens_per_frame < 1 || g.chunk_frames < 1) return fail(HF_ERR_SHAPE, "tokens_per_frame, chunk_frames must be >= 1");
    if (g.window_frames < g.chunk_frames || g.window_frames % g.chunk_frames != 0)
        return fail(HF_ERR_SHAPE, "window_frames must be a positive multiple of chunk_frames");
    if (g.window_frames / g.chunk_frames > HF_MAX_CHUNKS) return fail(HF_ERR_SHAPE, "window spans more than %d chunks", HF_MAX_CHUNKS);
    if (g.topk < 0 || (g.topk == 0 && (g.keep_permille < 1 || g.keep_permille > 1000)))
        return fail(HF_ERR_SHAPE, "need topk > 0 or keep_permille in [1, 1000]");
    if (g.phi != HF_PHI_ELU1) return fail(HF_ERR_UNSUPPORTED, "phi %d unsupported", g.phi);
    if (g.merge != HF_MERGE_IDENTITY && g.merge != HF_MERGE_PER_HEAD && g.merge != HF_MERGE_FULL_WIDTH)
        return fail(HF_ERR_UNSUPPORTED, "merge %d unsupported", g.merge);
    if (!(g.eps >= 0.f)) return fail(HF_ERR_SHAPE, "eps must be >= 0");
    if (g.swa_kernel < HF_SWA_AUTO || g.swa_kernel > HF_SWA_TCGEN05_PINGPONG) return fail(HF_ERR_UNSUPPORTED, "swa_kernel %d unknown", g.swa_kernel);
    if (g.z_mode != HF_Z_SUM && g.z_mode != HF_Z_FRAME_MEAN) return fail(HF_ERR_UNSUPPORTED, "z_mode %d unknown", g.z_mode);
    if (g.sink_frames < 0 || g.sink_frames % g.chunk_frames != 0) return fail(HF_ERR_SHAPE, "sink_frames must be a non-negative multiple of chunk_frames");
    if (g.sink_frames / g.chunk_frames + g.window_frames / g.chunk_frames > HF_MAX_CHUNKS)
        return fail(HF_ERR_SHAPE, "sink chunks + window chunks exceed %d", HF_MAX_CHUNKS);
    const long long Tc = (long long)g.tokens_per_frame * g.chunk_frames;
    const long long n_b = (Tc + g.block - 1) / g.block;
    if (Tc > (1 << 20)) return fail(HF_ERR_SHAPE, "chunk of %lld tokens too large", Tc);
    if (n_b * (g.window_frames / g.chunk_frames + g.sink_frames / g.chunk_frames) > HF_MAX_TN)
        return fail(HF_ERR_SHAPE, "window and sink span %lld key blocks, more than %d",
                    n_b * (g.window_frames / g.chunk_frames + g.sink_frames / g.chunk_frames), HF_MAX_TN);
    if ((long long)g.batch * g.heads > 65535) return fail(HF_ERR_SHAPE, "batch*heads exceeds 65535");
    return HF_OK;
}

template <typename T>
hf_status dmalloc(T** p, size_t count) {
    *p = nullptr;
    if (count == 0) return HF_OK;
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(p), count * sizeof(T));
    if (e == cudaErrorMemoryAllocation) { cudaGetLastError(); return fail(HF_ERR_NOMEM, "cudaMalloc of %zu bytes failed", count * sizeof(T)); }
    if (e != cudaSuccess) return fail(HF_ERR_CUDA, "cudaMalloc: %s", cudaGetErrorString(e));
    return HF_OK;
}

void free_all(hf_ctx* c) {
    for (auto& L : c->layers) { cudaFree(L.W_full); cudaFree(L.mask); cudaFree(L.idx); }
    cudaFree(c->ring_k_all); cudaFree(c->ring_v_all); cudaFree(c->pooled_k_all); cudaFree(c->S_all); cudaFree(c->z_all);
    cudaFree(c->sf_hi_all); cudaFree(c->sf_lo_all); cudaFree(c->W_all); cudaFree(c->bias_all);
    cudaFree(c->union_entries); cudaFree(c->union_tiles); cudaFree(c->bwd_delta); cudaFree(c->pooled_q); cudaFree(c->pooled_kcur); cudaFree(c->hist); cudaFree(c->partials); cudaFree(c->partials_layers); cudaFree(c->x_hi); cudaFree(c->x_lo);
    cudaFree(c->dev_status);
    cudaFree(c->rope_q[0]); cudaFree(c->rope_q[1]); cudaFree(c->rope_k[0]); cudaFree(c->rope_k[1]);
    cudaFree(c->trope_tab[0]); cudaFree(c->trope_tab[1]); cudaFree(c->q_rot); cudaFree(c->k_rot);
    if (c->ev_fork) cudaEventDestroy(c->ev_fork);
    if (c->ev_join) cudaEventDestroy(c->ev_join);
    if (c->side) cudaStreamDestroy(c->side);
    for (auto& s : c->stage) cudaFree(s);
}

template <int BLK, int D>
hf_status set_swa_attr() {
    HF_CUDA(cudaFuncSetAttribute(k_swa_mma<BLK, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, SwaMma<BLK, D>::SMEM_BYTES));
    return HF_OK;
}
template <int D>
hf_status set_state_attr() {
    HF_CUDA(cudaFuncSetAttribute(k_absorb_tc5<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, AbsorbTc5<D>::SMEM_BYTES));
    HF_CUDA(cudaFuncSetAttribute(k_absorb_tc5<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, AbsorbTc5<D>::SMEM_BYTES));
    HF_CUDA(cudaFuncSetAttribute(k_readout_tc5<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, ReadoutTc5<D>::SMEM_BYTES));
    HF_CUDA(cudaFuncSetAttribute(k_readout_tc5<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, ReadoutTc5<D>::SMEM_BYTES));
    HF_CUDA(cudaFuncSetAttribute(k_absorb_items<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, AbsorbItems<D>::SMEM_BYTES));
    HF_CUDA(cudaFuncSetAttribute(k_absorb_items<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, AbsorbItems<D>::SMEM_BYTES));
    return HF_OK;
}

#define HF_DISPATCH_D(c, FN, ...) ((c)->d == 128 ? FN<128>(__VA_ARGS__) : FN<64>(__VA_ARGS__))

// Launch configuration of a kernel that may start while the kernel before it in the stream still runs (programmatic
// dependent launch); the kernel calls pdl_wait() before it touches anything that kernel wrote.
struct PdlLaunch {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    PdlLaunch(dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool overlap) {
        memset(&cfg, 0, sizeof(cfg));
        cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = overlap ? 1 : 0;
    }
};

hf_status post_launch(hf_ctx* c, const char* what, int n = 1) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(HF_ERR_CUDA, "launch of %s failed: %s", what, cudaGetErrorString(e));
    c->launches += n;
    return HF_OK;
}

// ------------------------------------------------------------------------------------------- launches
template <int D>
hf_status launch_pool(hf_ctx* c, const PoolJobs& jobs, int njobs, cudaStream_t st) {
    dim3 grid(c->n_b, c->BH, njobs);
    PdlLaunch pl(grid, dim3(256), 0, st, true);
    bool rot = false;
    for (int i = 0; i < njobs; ++i) rot = rot || jobs.job[i].rot_on;
    if (rot) {
        HF_CUDA(cudaLaunchKernelEx(&pl.cfg, k_pool_copy_rot<D>, jobs, c->Tc, c->cfg.block, c->n_b, c->trope));
        return post_launch(c, "k_pool_copy_rot");
    }
    HF_CUDA(cudaLaunchKernelEx(&pl.cfg, k_pool_copy<D>, jobs, c->Tc, c->cfg.block, c->n_b));
    return post_launch(c, "k_pool_copy");
}

// Eq. 8: index of the last frame of the chunk that is generated when `frames` frames have been committed.
inline int trope_top(const hf_ctx* c, long long frames) {
    const long long last = frames + c->cfg.chunk_frames;
    return (int)(last < c->t0 ? last : c->t0);
}
// q and k_cur turned to the current chunk's indices, into the context's rotated copies (no pooling); k_cur may be null.
template <int D>
hf_status launch_rotate_inputs(hf_ctx* c, LayerState& L, const bf16* q, const bf16* k_cur, cudaStream_t st) {
    PoolJobs jobs;
    memset(&jobs, 0, sizeof(jobs));
    const int base = trope_top(c, L.frames) - c->cfg.chunk_frames + 1;
    int n = 0;
    if (q) { jobs.job[n].src = q; jobs.job[n].copy_dst = c->q_rot; jobs.job[n].rot_on = 1; jobs.job[n].rot_base = base; jobs.job[n].rot_per_frame = 1; ++n; }
    if (k_cur) { jobs.job[n].src = k_cur; jobs.job[n].copy_dst = c->k_rot; jobs.job[n].rot_on = 1; jobs.job[n].rot_base = base; jobs.job[n].rot_per_frame = 1; ++n; }
    return launch_pool<D>(c, jobs, n, st);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 4-D bf16 map [slots, B*H, rows, d] with a box of box_cols x box_rows, 128-byte swizzle (or none); rows past the end read as zero.
hf_status make_map_ex(hf_ctx* c, CUtensorMap* m, const void* base, long long rows, int slots, int box_cols, int box_rows, bool swizzle) {
    const cuuint64_t dims[4] = {(cuuint64_t)c->d, (cuuint64_t)rows, (cuuint64_t)c->BH, (cuuint64_t)slots};
    const cuuint64_t strides[3] = {(cuuint64_t)c->d * 2, (cuuint64_t)rows * c->d * 2, (cuuint64_t)c->BH * rows * c->d * 2};
    const cuuint32_t box[4] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows, 1, 1};
    const cuuint32_t es[4] = {1, 1, 1, 1};
    CUresult r = reinterpret_cast<EncodeTiledFn>(c->encode_tiled)(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims,
                                                                  strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                                  swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                                                                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(HF_ERR_CUDA, "cuTensorMapEncodeTiled failed with %d", (int)r);
    return HF_OK;
}
// [slots, B*H, T_c, d], box = 64 columns x 128 rows, 128-byte swizzle: the attention kernel's Q / K / V tiles.
hf_status make_map(hf_ctx* c, CUtensorMap* m, const void* base, int slots) {
    return make_map_ex(c, m, base, c->Tc, slots, 64, 128, true);
}

// Groups of consecutive splits in which the partial sums of an item are added up (part of the summation order, so a
// function of the split count alone -- see k_reduce_fold).
inline int absorb_groups(int nsplit) { return nsplit < 2 ? nsplit : 2; }

template <int D>
hf_status launch_fold(hf_ctx* c, LayerState& L, int nsplit, cudaStream_t st) {
    // after the partials kernel (nsplit > 0) the launch may overlap that kernel's epilogue; a fold on its own is ordinary
    PdlLaunch pl(dim3(D / 16, c->BH), dim3(D), 0, st, nsplit > 0);
    HF_CUDA(cudaLaunchKernelEx(&pl.cfg, k_reduce_fold<D>, (const float*)c->partials, nsplit, absorb_groups(nsplit), L.S, L.z, c->z_scale,
                               (const bf16*)(L.has_w ? L.W : nullptr), c->cfg.heads, c->BH, L.sf_hi, L.sf_lo, 1ull));
    return post_launch(c, "k_reduce_fold");
}

// on_side: both kernels go to the context's side stream, ordered after what `st` holds so far (the caller has
// independent work for `st` and joins with ev_join afterwards).
template <int D>
hf_status launch_absorb(hf_ctx* c, LayerState& L, const bf16* k, const bf16* v, int n_tokens, cudaStream_t st,
                        bool on_side = false) {
    typedef AbsorbTc5<D> A;
    const int n_tiles = (n_tokens + A::TT - 1) / A::TT;
    const int nsplit = n_tiles < c->nsplit_max ? n_tiles : c->nsplit_max;
    CUtensorMap tk, tv;
    HF_TRY(make_map_ex(c, &tk, k, n_tokens, 1, D, A::TT, false));
    HF_TRY(make_map_ex(c, &tv, v, n_tokens, 1, 64, A::TT, true));
    AbsorbTc5Params p;
    p.n_tokens = n_tokens; p.partials = c->partials; p.dev_status = c->dev_status;
    p.cos_k = c->rope_k[0]; p.sin_k = c->rope_k[1]; p.rope_rows = c->Tc;
    cudaStream_t run = st;
    if (on_side) {
        HF_CUDA(cudaEventRecord(c->ev_fork, st));
        HF_CUDA(cudaStreamWaitEvent(c->side, c->ev_fork, 0));
        run = c->side;
    }
    PdlLaunch pl(dim3(nsplit, c->BH), dim3(A::THREADS), A::SMEM_BYTES, run, !on_side);   // (an event wait sits before it on the side stream)
    if (c->has_rope_k) HF_CUDA(cudaLaunchKernelEx(&pl.cfg, k_absorb_tc5<D, true>, tk, tv, p));
    else HF_CUDA(cudaLaunchKernelEx(&pl.cfg, k_absorb_tc5<D, false>, tk, tv, p));
    HF_TRY(post_launch(c, "k_absorb_tc5"));
    HF_TRY(launch_fold<D>(c, L, nsplit, run));
    if (on_side) HF_CUDA(cudaEventRecord(c->ev_join, c->side));
    return HF_OK;
}

// Eq. 3 for n_layers layers (first_layer ..) in one persistent launch, then their folded states in a second, small one.
// tk / tv: the kernel's views of the tokens ([d, n_tokens, B*H, slots]); slot[l]: coordinate 3 of layer l of the call.
// The splits of an item's token range and their order are those of launch_absorb, so S and z get the same bits.
template <int D>
hf_status launch_absorb_layers(hf_ctx* c, int first_layer, int n_layers, const CUtensorMap& tk, const CUtensorMap& tv,
                               const int* slot, int n_tokens, cudaStream_t st) {
    typedef AbsorbItems<D> A;
    const size_t dd = (size_t)c->BH * D * D, dz = (size_t)c->BH * D;
    const int n_tiles = (n_tokens + A::TT - 1) / A::TT;
    AbsorbItemsParams p;
    memset(&p, 0, sizeof(p));
    p.n_tokens = n_tokens; p.BH = c->BH;
    p.nsplit = n_tiles < c->nsplit_max ? n_tiles : c->nsplit_max;
    p.ngroup = absorb_groups(p.nsplit);
    p.n_units = n_layers * c->BH * p.ngroup;
    // scratch for one partial per (item, group), grown on first use (never inside a later call of the same size)
    const size_t need = (size_t)n_layers * c->BH * p.ngroup * ((size_t)D * D + D);
    if (need > c->partials_layers_count) {
        HF_CUDA(cudaStreamSynchronize(st));
        cudaFree(c->partials_layers);
        c->partials_layers = nullptr; c->partials_layers_count = 0;
        HF_TRY(dmalloc(&c->partials_layers, need));
        c->partials_layers_count = need;
    }
    p.partials = c->partials_layers;
    for (int l = 0; l < n_layers; ++l) p.slot[l] = slot[l];
    p.cos_k = c->rope_k[0]; p.sin_k = c->rope_k[1]; p.rope_rows = c->Tc; p.dev_status = c->dev_status;
    const int grid = p.n_units < c->sm_count ? p.n_units : c->sm_count;
    PdlLaunch pl(dim3(grid), dim3(A::THREADS), A::SMEM_BYTES, st, false);
    if (c->has_rope_k) HF_CUDA(cudaLaunchKernelEx(&pl.cfg, k_absorb_items<D, true>, tk, tv, p));
    else HF_CUDA(cudaLaunchKernelEx(&pl.cfg, k_absorb_items<D, false>, tk, tv, p));
    HF_TRY(post_launch(c, "k_absorb_items"));
    unsigned long long has_w = 0;
    for (int l = 0; l < n_layers; ++l) if (c->layers[first_layer + l].has_w) has_w |= 1ull << l;
    PdlLaunch pf(dim3(D / 16, c->BH, n_layers), dim3(D), 0, st, true);
    HF_CUDA(cudaLaunchKernelEx(&pf.cfg, k_reduce_fold<D>, (const float*)c->partials_layers, p.ngroup, p.ngroup,
                               c->S_all + (size_t)first_layer * dd, c->z_all + (size_t)first_layer * dz, c->z_scale,
                               (const bf16*)(c->W_all ? c->W_all + (size_t)first_layer * c->cfg.heads * D * D : nullptr), c->cfg.heads,
                               c->BH, c->sf_hi_all + (size_t)first_layer * dd, c->sf_lo_all + (size_t)first_layer * dd, has_w));
    return post_launch(c, "k_reduce_fold (layers)");
}

template <int D>
hf_status launch_pool_layers(hf_ctx* c, const PoolLayersParams& p, int n_layers, cudaStream_t st) {
    PdlLaunch pl(dim3(c->n_b, c->BH, 2 * n_layers), dim3(256), 0, st, false);
    HF_CUDA(cudaLaunchKernelEx(&pl.cfg, k_pool_copy_layers<D>, p, c->Tc, c->cfg.block, c->n_b));
    return post_launch(c, "k_pool_copy_layers");
}

template <int D>
hf_status launch_readout(hf_ctx* c, LayerState& L, const bf16* q, bf16* out_bf16, float* out_f32, cudaStream_t st) {
    typedef ReadoutTc5<D> R;
    // Full-width reading of Eq. 4's Linear: the read-out leaves h = phi(q) S / (phi(q).z + eps) of every head as bf16 hi + lo
    // halves, and a second kernel applies the [H d, H d] matrix and the bias across the heads.
    const bool full = c->cfg.merge == HF_MERGE_FULL_WIDTH && L.has_wfull;
    CUtensorMap tq;
    HF_TRY(make_map(c, &tq, q, 1));
    ReadoutTc5Params p;
    p.cos_q = c->rope_q[0]; p.sin_q = c->rope_q[1];
    p.z = L.z; p.bias = (L.has_bias && !full) ? L.bias : nullptr; p.heads = c->cfg.heads; p.Tc = c->Tc;
    p.Tm = (c->Tc + R::ROWS - 1) / R::ROWS; p.n_units = p.Tm * c->BH; p.eps = c->cfg.eps;
    p.out_bf16 = full ? c->x_hi : out_bf16; p.out_f32 = full ? nullptr : out_f32; p.out_lo = full ? c->x_lo : nullptr;
    p.dev_status = c->dev_status;
    const int grid = p.n_units < c->sm_count ? p.n_units : c->sm_count;
    if (c->has_rope_q) k_readout_tc5<D, true><<<grid, R::THREADS, R::SMEM_BYTES, st>>>(tq, L.tm_sfhi, L.tm_sflo, p);
    else k_readout_tc5<D, false><<<grid, R::THREADS, R::SMEM_BYTES, st>>>(tq, L.tm_sfhi, L.tm_sflo, p);
    HF_TRY(post_launch(c, "k_readout_tc5"));
    if (!full) return HF_OK;
    typedef MergeFull<D> M;
    CUtensorMap txh, txl;
    HF_TRY(make_map(c, &txh, c->x_hi, 1));
    HF_TRY(make_map(c, &txl, c->x_lo, 1));
    MergeFullParams mp;
    mp.heads = c->cfg.heads; mp.Tc = c->Tc; mp.Tm = (c->Tc + M::ROWS - 1) / M::ROWS;
    mp.bias = L.has_bias ? L.bias : nullptr; mp.out_f32 = out_f32; mp.out_bf16 = out_f32 ? nullptr : out_bf16;
    mp.dev_status = c->dev_status;
    PdlLaunch pl(dim3(mp.Tm, c->cfg.heads, c->cfg.batch), dim3(M::THREADS), M::SMEM_BYTES, st, false);
    HF_CUDA(cudaLaunchKernelEx(&pl.cfg, k_merge_full<D>, txh, txl, L.tm_wfull, mp));
    return post_launch(c, "k_merge_full");
}

template <int D>
hf_status launch_readout_bwd(hf_ctx* c, LayerState& L, const bf16* q, const bf16* d_o, bf16* dq, cudaStream_t st) {
    typedef ReadoutBwd<D> R;
    HF_CUDA(cudaFuncSetAttribute(k_readout_bwd_dq<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, R::SMEM_BYTES));
    CUtensorMap tg;
    HF_TRY(make_map(c, &tg, d_o, 1));
    ReadoutBwdParams p;
    p.q = q; p.z = L.z; p.dq = dq; p.Tc = c->Tc; p.Tm = (c->Tc + R::ROWS - 1) / R::ROWS; p.n_units = p.Tm * c->BH;
    p.eps = c->cfg.eps; p.dev_status = c->dev_status;
    const int grid = p.n_units < c->sm_count ? p.n_units : c->sm_count;
    k_readout_bwd_dq<D><<<grid, R::THREADS, R::SMEM_BYTES, st>>>(tg, L.tm_sfhi, L.tm_sflo, p);
    return post_launch(c, "k_readout_bwd_dq");
}

ChunkTable make_table(hf_ctx* c, LayerState& L, const bf16* k_cur, const bf16* v_cur) {
    ChunkTable t;
    memset(&t, 0, sizeof(t));
    const int n_old = L.n_sink + L.n_cached;
    for (int i = 0; i < n_old; ++i) {       // sink chunks first, then the cached chunks oldest first
        const int slot = i < L.n_sink ? c->R + i : (L.head + i - L.n_sink) % c->R;
        t.k[i] = L.ring_k + (size_t)slot * c->chunk_elems;
        t.v[i] = L.ring_v + (size_t)slot * c->chunk_elems;
        t.pooled[i] = L.pooled_k + (size_t)slot * c->pooled_elems;
    }
    t.k[n_old] = k_cur;
    t.v[n_old] = v_cur;
    t.pooled[n_old] = c->pooled_kcur;
    t.n_chunks = n_old + 1;
    return t;
}

template <int D>
hf_status launch_select(hf_ctx* c, LayerState& L, const bf16* q, const bf16* k_cur,
                        uint32_t* mask_out, int32_t* idx_out, float* scores_out, cudaStream_t st) {
    PoolJobs jobs;
    memset(&jobs, 0, sizeof(jobs));
    jobs.job[0].src = q;     jobs.job[0].pooled = c->pooled_q;
    jobs.job[1].src = k_cur; jobs.job[1].pooled = c->pooled_kcur;
    if (c->has_trope) {     // the block means are those of the rotated tensors, which the attention kernel reads afterwards
        const int base = trope_top(c, L.frames) - c->cfg.chunk_frames + 1;
        jobs.job[0].copy_dst = c->q_rot; jobs.job[1].copy_dst = c->k_rot;
        for (int i = 0; i < 2; ++i) { jobs.job[i].rot_on = 1; jobs.job[i].rot_base = base; jobs.job[i].rot_per_frame = 1; }
    }
    HF_TRY(launch_pool<D>(c, jobs, 2, st));
    const int Tn = (L.n_sink + L.n_cached + 1) * c->n_b;
    const int keep = keep_for(c, Tn);
    ChunkTable tab = make_table(c, L, k_cur, nullptr);
    PdlLaunch pl(dim3(c->Tm, c->BH), dim3(256), 0, st, true);      // follows the pooling kernel launched above
    // Two forms of the scoring loop, same arithmetic: the wide one keeps a pass's loads in flight (80 registers, three
    // thread blocks per SM) and is ahead while the grid fits that; the narrow one (40 registers) fits twice the thread blocks.
    if (c->Tm * c->BH <= 3 * c->sm_count)
        HF_CUDA(cudaLaunchKernelEx(&pl.cfg, k_select<D, true>, tab, (const float*)c->pooled_q, c->n_b, c->Tm, Tn, keep, c->mask_words,
                                   L.mask, L.idx, mask_out, idx_out, scores_out));
    else
        HF_CUDA(cudaLaunchKernelEx(&pl.cfg, k_select<D, false>, tab, (const float*)c->pooled_q, c->n_b, c->Tm, Tn, keep, c->mask_words,
                                   L.mask, L.idx, mask_out, idx_out, scores_out));
    HF_TRY(post_launch(c, "k_select"));
    L.sel_epoch = L.cache_epoch;
    L.sel_keep = keep;
    return HF_OK;
}

template <int BLK, int D>
hf_status launch_swa_mma_t(hf_ctx* c, const bf16* q, const ChunkTable& tab, const int32_t* idx, int keep,
                           const float* hist, bf16* o, float* lse, cudaStream_t st) {
    typedef SwaMma<BLK, D> C;
    const float scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)D));
    k_swa_mma<BLK, D><<<dim3(c->Tm, c->BH), C::THREADS, C::SMEM_BYTES, st>>>(q, tab, idx, keep, c->Tc, c->n_b, scale_log2, hist, o, lse, c->dev_status);
    return post_launch(c, "k_swa_mma");
}


#ifndef HF_TC5_GROUPS
#define HF_TC5_GROUPS 2   // softmax column groups of the tcgen05 attention kernel at head_dim 64
#endif
#ifndef HF_TC5_GROUPS_128
#define HF_TC5_GROUPS_128 2   // ... and at head_dim 128
#endif
template <int D> struct Tc5Groups { static constexpr int N = (D == 128) ? HF_TC5_GROUPS_128 : HF_TC5_GROUPS; };

template <int D>
hf_status launch_swa_tc5_t(hf_ctx* c, LayerState& L, const bf16* q, const bf16* k_cur, const bf16* v_cur, const int32_t* idx,
                           int keep, const float* hist, bf16* o, float* lse, cudaStream_t st, bool fuse_history = false,
                           bool overlap_prev = false) {
    typedef SwaTc5<D, Tc5Groups<D>::N> C;
    CUtensorMap tq, tk, tv, to;
    HF_TRY(make_map(c, &tq, q, 1));
    HF_TRY(make_map(c, &tk, k_cur, 1));
    HF_TRY(make_map(c, &tv, v_cur, 1));
    HF_TRY(make_map_ex(c, &to, o, c->Tc, 1, 64, 32, true));      // output: one warp's 32 rows x 64 columns per store
    Tc5Params p;
    p.idx = idx; p.keep = keep; p.Tc = c->Tc; p.n_b = c->n_b; p.n_cached = L.n_cached; p.ring_head = L.head; p.n_sink = L.n_sink;
    p.P = c->R;
    p.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)D));
    p.hist = hist; p.o = o; p.lse = lse; p.dev_status = c->dev_status;
    p.heads = c->cfg.heads; p.eps = c->cfg.eps;
    p.q = q; p.z = L.z; p.bias = L.has_bias ? L.bias : nullptr;
    p.tab = make_table(c, L, k_cur, v_cur); p.sf_hi = L.sf_hi; p.sf_lo = L.sf_lo;
    const CUtensorMap& rk = c->R + c->n_sink_max > 0 ? L.tm_kring : tk;
    const CUtensorMap& rv = c->R + c->n_sink_max > 0 ? L.tm_vring : tv;
    p.Tm = c->Tm; p.n_units = c->Tm * c->BH;
    const int grid = p.n_units < c->sm_count ? p.n_units : c->sm_count;
    PdlLaunch pl(dim3(grid), dim3(C::THREADS), C::SMEM_BYTES, st, overlap_prev);
    if constexpr (C::FUSE) {
        if (fuse_history) {
            HF_CUDA(cudaLaunchKernelEx(&pl.cfg, k_swa_tc5<D, Tc5Groups<D>::N, true>, tq, rk, rv, tk, tv, L.tm_sfhi, L.tm_sflo, to, p));
            return post_launch(c, "k_swa_tc5 (history term inside)");
        }
    }
    if (fuse_history) return fail(HF_ERR_UNSUPPORTED, "the attention kernel of this configuration cannot form the history term");
    HF_CUDA(cudaLaunchKernelEx(&pl.cfg, k_swa_tc5<D, Tc5Groups<D>::N, false>, tq, rk, rv, tk, tv, L.tm_sfhi, L.tm_sflo, to, p));
    return post_launch(c, "k_swa_tc5");
}

#ifndef HF_TC5P_COLGROUPS
#define HF_TC5P_COLGROUPS 1   // column groups per tile group of the ping-pong attention kernel
#endif

template <int D>
hf_status launch_swa_tc5p_t(hf_ctx* c, LayerState& L, const bf16* q, const bf16* k_cur, const bf16* v_cur, const int32_t* idx,
                            int keep, const float* hist, bf16* o, float* lse, cudaStream_t st) {
    typedef SwaTc5P<D, HF_TC5P_COLGROUPS> C;
    CUtensorMap tq, tk, tv;
    HF_TRY(make_map(c, &tq, q, 1));
    HF_TRY(make_map(c, &tk, k_cur, 1));
    HF_TRY(make_map(c, &tv, v_cur, 1));
    Tc5Params p;
    p.idx = idx; p.keep = keep; p.Tc = c->Tc; p.n_b = c->n_b; p.n_cached = L.n_cached; p.ring_head = L.head; p.n_sink = L.n_sink;
    p.P = c->R;
    p.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)D));
    p.hist = hist; p.o = o; p.lse = lse; p.dev_status = c->dev_status;
    memset(&p.tab, 0, sizeof(p.tab)); p.sf_hi = nullptr; p.sf_lo = nullptr;
    const CUtensorMap& rk = c->R + c->n_sink_max > 0 ? L.tm_kring : tk;
    const CUtensorMap& rv = c->R + c->n_sink_max > 0 ? L.tm_vring : tv;
    p.Tm = c->Tm; p.n_units = c->Tm * c->BH;
    const int grid = p.n_units < c->sm_count ? p.n_units : c->sm_count;
    k_swa_tc5p<D, HF_TC5P_COLGROUPS><<<grid, C::THREADS, C::SMEM_BYTES, st>>>(tq, rk, rv, tk, tv, p);
    return post_launch(c, "k_swa_tc5p");
}

// Blocks of 16 or 64 tokens on the tcgen05 path: merge the kept lists of the query blocks that share a 128-row unit
// (k_union_tiles), then the attention kernel over 128-key tiles made of 128 / BLK key blocks each.
template <int D, int BLK>
hf_status launch_swa_tc5g_t(hf_ctx* c, LayerState& L, const bf16* q, const bf16* k_cur, const bf16* v_cur, const int32_t* idx,
                            int keep, const float* hist, bf16* o, float* lse, cudaStream_t st) {
    typedef SwaTc5<D, 2> C;
    constexpr int G = 128 / BLK;
    const int Tn = (L.n_sink + L.n_cached + 1) * c->n_b;
    const int Tmt = (c->Tc + 127) / 128;
    const int uni = G * keep < Tn ? G * keep : Tn;
    const int max_tiles = (uni + G - 1) / G;
    if (max_tiles > c->union_max_tiles) return fail(HF_ERR_SHAPE, "tile list of %d tiles exceeds the %d the context was sized for", max_tiles, c->union_max_tiles);
    PdlLaunch pu(dim3(Tmt, c->BH), dim3(256), 0, st, true);
    HF_CUDA(cudaLaunchKernelEx(&pu.cfg, k_union_tiles<BLK>, idx, keep, c->Tm, Tn, c->n_b, c->Tc, max_tiles, c->union_entries, c->union_tiles,
                               c->dev_status));
    HF_TRY(post_launch(c, "k_union_tiles"));
    CUtensorMap tq, tk, tv, to;
    HF_TRY(make_map(c, &tq, q, 1));
    HF_TRY(make_map_ex(c, &tk, k_cur, c->Tc, 1, 64, BLK, true));
    HF_TRY(make_map_ex(c, &tv, v_cur, c->Tc, 1, 64, BLK, true));
    HF_TRY(make_map_ex(c, &to, o, c->Tc, 1, 64, 32, true));
    Tc5GParams p;
    memset(&p, 0, sizeof(p));
    p.entries = c->union_entries; p.tiles = c->union_tiles; p.max_tiles = max_tiles;
    p.Tmt = Tmt; p.n_units = Tmt * c->BH;
    p.idx = idx; p.keep = keep; p.Tm = c->Tm;
    p.Tc = c->Tc; p.n_b = c->n_b; p.n_cached = L.n_cached; p.ring_head = L.head; p.P = c->R; p.n_sink = L.n_sink;
    p.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)D));
    p.hist = hist; p.q = q; p.o = o; p.lse = lse; p.dev_status = c->dev_status;
    p.tab = make_table(c, L, k_cur, v_cur);
    const CUtensorMap& rk = c->R + c->n_sink_max > 0 ? L.tm_kring : tk;
    const CUtensorMap& rv = c->R + c->n_sink_max > 0 ? L.tm_vring : tv;
    const int grid = p.n_units < c->sm_count ? p.n_units : c->sm_count;
    PdlLaunch pl(dim3(grid), dim3(C::THREADS), C::SMEM_BYTES, st, true);
    HF_CUDA(cudaLaunchKernelEx(&pl.cfg, k_swa_tc5g<D, BLK>, tq, rk, rv, tk, tv, to, p));
    return post_launch(c, "k_swa_tc5g");
}

hf_status launch_swa(hf_ctx* c, LayerState& L, const bf16* q, const bf16* k_cur, const bf16* v_cur, const int32_t* idx,
                     int keep, const float* hist, bf16* o, float* lse, cudaStream_t st) {
    if (c->swa_kernel == HF_SWA_TCGEN05 && c->cfg.block != 128) {
        const int b = c->cfg.block, d = c->d;
        if (b == 64 && d == 128) return launch_swa_tc5g_t<128, 64>(c, L, q, k_cur, v_cur, idx, keep, hist, o, lse, st);
        if (b == 64 && d == 64) return launch_swa_tc5g_t<64, 64>(c, L, q, k_cur, v_cur, idx, keep, hist, o, lse, st);
        if (b == 16 && d == 128) return launch_swa_tc5g_t<128, 16>(c, L, q, k_cur, v_cur, idx, keep, hist, o, lse, st);
        return launch_swa_tc5g_t<64, 16>(c, L, q, k_cur, v_cur, idx, keep, hist, o, lse, st);
    }
    if (c->swa_kernel == HF_SWA_TCGEN05_PINGPONG) {
        if (c->d == 128) return launch_swa_tc5p_t<128>(c, L, q, k_cur, v_cur, idx, keep, hist, o, lse, st);
        return launch_swa_tc5p_t<64>(c, L, q, k_cur, v_cur, idx, keep, hist, o, lse, st);
    }
    if (c->swa_kernel == HF_SWA_TCGEN05) {
        if (c->d == 128) return launch_swa_tc5_t<128>(c, L, q, k_cur, v_cur, idx, keep, hist, o, lse, st);
        return launch_swa_tc5_t<64>(c, L, q, k_cur, v_cur, idx, keep, hist, o, lse, st);
    }
    ChunkTable tab = make_table(c, L, k_cur, v_cur);
    const int b = c->cfg.block, d = c->d;
#define HF_SWA_CASE(B_, D_) if (b == B_ && d == D_) return launch_swa_mma_t<B_, D_>(c, q, tab, idx, keep, hist, o, lse, st)
    HF_SWA_CASE(16, 64); HF_SWA_CASE(16, 128); HF_SWA_CASE(64, 64); HF_SWA_CASE(64, 128); HF_SWA_CASE(128, 64); HF_SWA_CASE(128, 128);
#undef HF_SWA_CASE
    return fail(HF_ERR_UNSUPPORTED, "no attention kernel for block %d, head_dim %d", b, d);
}

template <int D>
hf_status launch_bwd_dq(hf_ctx* c, LayerState& L, const bf16* q, const bf16* k_cur, const bf16* v_cur, const int32_t* idx, int keep,
                               const bf16* o_local, const float* lse, const bf16* d_o, bf16* dq, cudaStream_t st) {
    typedef SwaBwd<D> C;
    if (c->bwd_delta == nullptr) HF_TRY(dmalloc(&c->bwd_delta, (size_t)c->BH * c->Tc));
    HF_CUDA(cudaFuncSetAttribute(k_swa_bwd_dq<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
    const long long rows = (long long)c->BH * c->Tc;
    k_rowdot<D><<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(d_o, o_local, c->bwd_delta, rows);
    HF_TRY(post_launch(c, "k_rowdot"));
    CUtensorMap tq, tdo, tk, tv;
    HF_TRY(make_map(c, &tq, q, 1));
    HF_TRY(make_map(c, &tdo, d_o, 1));
    HF_TRY(make_map(c, &tk, k_cur, 1));
    HF_TRY(make_map(c, &tv, v_cur, 1));
    SwaBwdParams p;
    memset(&p, 0, sizeof(p));
    p.idx = idx; p.keep = keep; p.Tc = c->Tc; p.n_b = c->n_b; p.n_cached = L.n_cached; p.ring_head = L.head; p.P = c->R; p.n_sink = L.n_sink;
    p.Tm = c->Tm; p.n_units = c->Tm * c->BH;
    p.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)D)); p.scale = (float)(1.0 / std::sqrt((double)D));
    p.lse = lse; p.delta = c->bwd_delta; p.dq = dq; p.dev_status = c->dev_status;
    const CUtensorMap& rk = c->R + c->n_sink_max > 0 ? L.tm_kring : tk;
    const CUtensorMap& rv = c->R + c->n_sink_max > 0 ? L.tm_vring : tv;
    const int grid = p.n_units < c->sm_count ? p.n_units : c->sm_count;
    PdlLaunch pl(dim3(grid), dim3(C::THREADS), C::SMEM_BYTES, st, false);
    HF_CUDA(cudaLaunchKernelEx(&pl.cfg, k_swa_bwd_dq<D>, tq, tdo, rk, rv, tk, tv, p));
    return post_launch(c, "k_swa_bwd_dq");
}

template <int D>
hf_status launch_bwd_dkv(hf_ctx* c, LayerState& L, const bf16* q, const bf16* k_cur, const bf16* v_cur, const bf16* o_local,
                         const float* lse, const bf16* d_o, bf16* dk, bf16* dv, cudaStream_t st) {
    typedef SwaBwdKV<D> C;
    if (c->bwd_delta == nullptr) HF_TRY(dmalloc(&c->bwd_delta, (size_t)c->BH * c->Tc));
    HF_CUDA(cudaFuncSetAttribute(k_swa_bwd_dkv<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
    const long long rows = (long long)c->BH * c->Tc;
    k_rowdot<D><<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(d_o, o_local, c->bwd_delta, rows);
    HF_TRY(post_launch(c, "k_rowdot"));
    CUtensorMap tq, tdo, tk, tv;
    HF_TRY(make_map(c, &tq, q, 1));
    HF_TRY(make_map(c, &tdo, d_o, 1));
    HF_TRY(make_map(c, &tk, k_cur, 1));
    HF_TRY(make_map(c, &tv, v_cur, 1));
    SwaBwdKVParams p;
    memset(&p, 0, sizeof(p));
    p.mask = L.mask; p.mask_words = c->mask_words; p.first_block = (L.n_sink + L.n_cached) * c->n_b;
    p.Tc = c->Tc; p.n_b = c->n_b; p.Tm = c->Tm; p.n_units = c->BH * c->n_b;
    p.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)D)); p.scale = (float)(1.0 / std::sqrt((double)D));
    p.lse = lse; p.delta = c->bwd_delta; p.dk = dk; p.dv = dv; p.dev_status = c->dev_status;
    const int grid = p.n_units < c->sm_count ? p.n_units : c->sm_count;
    PdlLaunch pl(dim3(grid), dim3(C::THREADS), C::SMEM_BYTES, st, false);
    HF_CUDA(cudaLaunchKernelEx(&pl.cfg, k_swa_bwd_dkv<D>, tq, tdo, tk, tv, p));
    return post_launch(c, "k_swa_bwd_dkv");
}

hf_status ensure_staging(hf_ctx* c) {
    for (int i = 0; i < 4; ++i)
        if (c->stage[i] == nullptr) HF_TRY(dmalloc(&c->stage[i], c->chunk_elems));
    return HF_OK;
}

}  // namespace

// =============================================================================================== C ABI
extern "C" {

const char* hf_status_string(hf_status s) {
    switch (s) {
        case HF_OK: return "HF_OK";
        case HF_ERR_INVALID_ARG: return "HF_ERR_INVALID_ARG";
        case HF_ERR_SHAPE: return "HF_ERR_SHAPE";
        case HF_ERR_STATE: return "HF_ERR_STATE";
        case HF_ERR_UNSUPPORTED: return "HF_ERR_UNSUPPORTED";
        case HF_ERR_NOMEM: return "HF_ERR_NOMEM";
        case HF_ERR_CUDA: return "HF_ERR_CUDA";
        case HF_ERR_DEVICE_TIMEOUT: return "HF_ERR_DEVICE_TIMEOUT";
    }
    return "HF_ERR_UNKNOWN";
}

const char* hf_last_error(void) { return g_err; }

// Library-internal (not part of the ABI): lets the other translation units of libhf record their error text.
void hf_internal_set_error(const char* text) {
    snprintf(g_err, sizeof(g_err), "%s", text ? text : "");
}

hf_status hf_create(const hf_config* cfg, int device, hf_ctx** out) {
    if (cfg == nullptr || out == nullptr) return fail(HF_ERR_INVALID_ARG, "cfg or out is null");
    *out = nullptr;
    HF_TRY(validate(*cfg));
    int count = 0;
    cudaError_t e = cudaGetDeviceCount(&count);
    if (e != cudaSuccess) { cudaGetLastError(); return fail(HF_ERR_CUDA, "cudaGetDeviceCount: %s", cudaGetErrorString(e)); }
    if (device < 0 || device >= count) return fail(HF_ERR_INVALID_ARG, "device %d outside [0, %d)", device, count);
    HF_CUDA(cudaSetDevice(device));
    hf_ctx* c = new (std::nothrow) hf_ctx();
    if (c == nullptr) return fail(HF_ERR_NOMEM, "host allocation failed");
    c->cfg = *cfg;
    c->device = device;
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, device);
    if (e != cudaSuccess) { delete c; return fail(HF_ERR_CUDA, "cudaGetDeviceProperties: %s", cudaGetErrorString(e)); }
    if (prop.major != 10) { delete c; return fail(HF_ERR_UNSUPPORTED, "device is sm_%d%d; this library is built for sm_100a only", prop.major, prop.minor); }
    c->sm_count = prop.multiProcessorCount;
    c->d = cfg->head_dim;
    c->BH = cfg->batch * cfg->heads;
    c->Tc = cfg->tokens_per_frame * cfg->chunk_frames;
    c->n_b = (c->Tc + cfg->block - 1) / cfg->block;
    c->Tm = c->n_b;
    c->P = cfg->window_frames / cfg->chunk_frames - 1;
    c->R = c->P > 0 ? c->P + 1 : 0;     // physical ring slots: one more than the window holds (see the cache commit)
    c->n_sink_max = cfg->sink_frames / cfg->chunk_frames;
    c->max_Tn = (c->P + c->n_sink_max + 1) * c->n_b;
    c->mask_words = (c->max_Tn + 31) / 32;
    c->chunk_elems = (size_t)c->BH * c->Tc * c->d;
    c->pooled_elems = (size_t)c->BH * c->n_b * c->d;
    c->z_scale = cfg->z_mode == HF_Z_FRAME_MEAN ? 1.f / (float)cfg->tokens_per_frame : 1.f;
    c->nsplit_max = c->sm_count / c->BH;          // one wave: the absorb kernel runs one thread block per SM
    if (c->nsplit_max > 32) c->nsplit_max = 32;
    if (c->nsplit_max < 1) c->nsplit_max = 1;
    if (cfg->swa_kernel == HF_SWA_TCGEN05_PINGPONG && cfg->block != 128) { delete c; return fail(HF_ERR_UNSUPPORTED, "the ping-pong attention kernel needs block == 128"); }
    c->swa_kernel = cfg->swa_kernel == HF_SWA_MMA ? HF_SWA_MMA
                    : (cfg->swa_kernel == HF_SWA_TCGEN05_PINGPONG ? HF_SWA_TCGEN05_PINGPONG : HF_SWA_TCGEN05);
    {
        cudaDriverEntryPointQueryResult qres;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &c->encode_tiled, cudaEnableDefault, &qres);
        if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || c->encode_tiled == nullptr) {
            delete c;
            return fail(HF_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
        }
    }

    hf_status s = HF_OK;
    c->layers.resize(cfg->layers);
    const size_t dd = (size_t)c->BH * c->d * c->d, dz = (size_t)c->BH * c->d;
    const size_t slots = (size_t)c->R + c->n_sink_max;          // per layer: ring slots, then sink slots
    const size_t nl = (size_t)cfg->layers, wd = (size_t)cfg->heads * c->d * c->d, bd = (size_t)cfg->heads * c->d;
    c->slots_per_layer = (int)slots;
    if (nl * slots > 0x7fffffffull) { delete c; return fail(HF_ERR_SHAPE, "layers x cache slots too large"); }
    if (s == HF_OK) s = dmalloc(&c->ring_k_all, nl * slots * c->chunk_elems);
    if (s == HF_OK) s = dmalloc(&c->ring_v_all, nl * slots * c->chunk_elems);
    if (s == HF_OK) s = dmalloc(&c->pooled_k_all, nl * slots * c->pooled_elems);
    if (s == HF_OK) s = dmalloc(&c->S_all, nl * dd);
    if (s == HF_OK) s = dmalloc(&c->z_all, nl * dz);
    if (s == HF_OK) s = dmalloc(&c->sf_hi_all, nl * dd);
    if (s == HF_OK) s = dmalloc(&c->sf_lo_all, nl * dd);
    if (s == HF_OK && cfg->merge == HF_MERGE_PER_HEAD) s = dmalloc(&c->W_all, nl * wd);
    if (s == HF_OK && cfg->merge != HF_MERGE_IDENTITY) s = dmalloc(&c->bias_all, nl * bd);
    if (s == HF_OK) {
        cudaMemset(c->S_all, 0, nl * dd * 4); cudaMemset(c->z_all, 0, nl * dz * 4);
        cudaMemset(c->sf_hi_all, 0, nl * dd * 2); cudaMemset(c->sf_lo_all, 0, nl * dd * 2);
    }
    if (s == HF_OK && slots > 0) s = make_map_ex(c, &c->tm_kall, c->ring_k_all, c->Tc, (int)(nl * slots), c->d, 64, false);
    if (s == HF_OK && slots > 0) s = make_map_ex(c, &c->tm_vall, c->ring_v_all, c->Tc, (int)(nl * slots), 64, 64, true);
    for (size_t li = 0; s == HF_OK && li < nl; ++li) {
        LayerState& L = c->layers[li];
        L.ring_k = slots ? c->ring_k_all + li * slots * c->chunk_elems : nullptr;
        L.ring_v = slots ? c->ring_v_all + li * slots * c->chunk_elems : nullptr;
        L.pooled_k = slots ? c->pooled_k_all + li * slots * c->pooled_elems : nullptr;
        L.S = c->S_all + li * dd; L.z = c->z_all + li * dz;
        L.sf_hi = c->sf_hi_all + li * dd; L.sf_lo = c->sf_lo_all + li * dd;
        L.W = c->W_all ? c->W_all + li * wd : nullptr;
        L.bias = c->bias_all ? c->bias_all + li * bd : nullptr;
        if (s == HF_OK && cfg->merge == HF_MERGE_FULL_WIDTH) {
            const size_t hd = (size_t)cfg->heads * c->d;
            s = dmalloc(&L.W_full, hd * hd);
            if (s == HF_OK) {
                const cuuint64_t dims[4] = {hd, hd, 1, 1};
                const cuuint64_t strides[3] = {hd * 2, hd * hd * 2, hd * hd * 2};
                const cuuint32_t box[4] = {64, (cuuint32_t)c->d, 1, 1};
                const cuuint32_t es[4] = {1, 1, 1, 1};
                CUresult r = reinterpret_cast<EncodeTiledFn>(c->encode_tiled)(&L.tm_wfull, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, L.W_full, dims,
                                                                              strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                                              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
                if (r != CUDA_SUCCESS) s = fail(HF_ERR_CUDA, "cuTensorMapEncodeTiled (merge matrix) failed with %d", (int)r);
            }
        }
        if (s == HF_OK) s = dmalloc(&L.mask, (size_t)c->BH * c->Tm * c->mask_words);
        if (s == HF_OK) s = dmalloc(&L.idx, (size_t)c->BH * c->Tm * c->max_Tn);
        // the attention kernels fetch key blocks: boxes of `block` rows
        if (s == HF_OK && slots > 0) s = make_map_ex(c, &L.tm_kring, L.ring_k, c->Tc, (int)slots, 64, cfg->block, true);
        if (s == HF_OK && slots > 0) s = make_map_ex(c, &L.tm_vring, L.ring_v, c->Tc, (int)slots, 64, cfg->block, true);
        if (s == HF_OK) s = make_map_ex(c, &L.tm_sfhi, L.sf_hi, c->d, 1, 64, c->d, true);
        if (s == HF_OK) s = make_map_ex(c, &L.tm_sflo, L.sf_lo, c->d, 1, 64, c->d, true);
    }
    if (s == HF_OK && cfg->block != 128) {
        const int G = 128 / cfg->block, Tmt = (c->Tc + 127) / 128;
        c->union_max_tiles = (c->max_Tn + G - 1) / G;
        s = dmalloc(&c->union_entries, (size_t)c->BH * Tmt * c->union_max_tiles * G);
        if (s == HF_OK) s = dmalloc(&c->union_tiles, (size_t)c->BH * Tmt);
    }
    if (s == HF_OK) s = dmalloc(&c->pooled_q, c->pooled_elems);
    if (s == HF_OK) s = dmalloc(&c->pooled_kcur, c->pooled_elems);
    if (s == HF_OK) s = dmalloc(&c->hist, c->chunk_elems);
    if (s == HF_OK && cfg->merge == HF_MERGE_FULL_WIDTH) s = dmalloc(&c->x_hi, c->chunk_elems);
    if (s == HF_OK && cfg->merge == HF_MERGE_FULL_WIDTH) s = dmalloc(&c->x_lo, c->chunk_elems);
    if (s == HF_OK && cfg->merge == HF_MERGE_FULL_WIDTH &&
        (cudaFuncSetAttribute(k_merge_full<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, MergeFull<64>::SMEM_BYTES) != cudaSuccess ||
         cudaFuncSetAttribute(k_merge_full<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, MergeFull<128>::SMEM_BYTES) != cudaSuccess))
        s = fail(HF_ERR_CUDA, "cudaFuncSetAttribute(k_merge_full) failed");
    if (s == HF_OK) s = dmalloc(&c->partials, (size_t)c->BH * c->nsplit_max * ((size_t)c->d * c->d + c->d));
    if (s == HF_OK) s = dmalloc(&c->dev_status, (size_t)8);     // status word [4] + self-test results [4]
    if (s == HF_OK && (cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) != cudaSuccess ||
                       cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
                       cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) != cudaSuccess))
        s = fail(HF_ERR_CUDA, "could not create the context's side stream / events");
    if (s == HF_OK) {
        cudaMemset(c->dev_status, 0, 32);
        s = set_swa_attr<16, 64>();
        if (s == HF_OK) s = set_swa_attr<16, 128>();
        if (s == HF_OK) s = set_swa_attr<64, 64>();
        if (s == HF_OK) s = set_swa_attr<64, 128>();
        if (s == HF_OK) s = set_swa_attr<128, 64>();
        if (s == HF_OK) s = set_swa_attr<128, 128>();
        if (s == HF_OK && cudaFuncSetAttribute(k_swa_tc5<64, Tc5Groups<64>::N, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SwaTc5<64, Tc5Groups<64>::N>::SMEM_BYTES) != cudaSuccess) s = fail(HF_ERR_CUDA, "cudaFuncSetAttribute(k_swa_tc5<64>) failed");
        if (s == HF_OK && cudaFuncSetAttribute(k_swa_tc5<128, Tc5Groups<128>::N, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SwaTc5<128, Tc5Groups<128>::N>::SMEM_BYTES) != cudaSuccess) s = fail(HF_ERR_CUDA, "cudaFuncSetAttribute(k_swa_tc5<128>) failed");
        if constexpr (SwaTc5<128, Tc5Groups<128>::N>::FUSE)
            if (s == HF_OK && cudaFuncSetAttribute(k_swa_tc5<128, Tc5Groups<128>::N, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SwaTc5<128, Tc5Groups<128>::N>::SMEM_BYTES) != cudaSuccess) s = fail(HF_ERR_CUDA, "cudaFuncSetAttribute(k_swa_tc5<128, history>) failed");
        if (s == HF_OK && cudaFuncSetAttribute(k_swa_tc5p<64, HF_TC5P_COLGROUPS>, cudaFuncAttributeMaxDynamicSharedMemorySize, SwaTc5P<64, HF_TC5P_COLGROUPS>::SMEM_BYTES) != cudaSuccess) s = fail(HF_ERR_CUDA, "cudaFuncSetAttribute(k_swa_tc5p<64>) failed");
        if (s == HF_OK && cudaFuncSetAttribute(k_swa_tc5p<128, HF_TC5P_COLGROUPS>, cudaFuncAttributeMaxDynamicSharedMemorySize, SwaTc5P<128, HF_TC5P_COLGROUPS>::SMEM_BYTES) != cudaSuccess) s = fail(HF_ERR_CUDA, "cudaFuncSetAttribute(k_swa_tc5p<128>) failed");
        if (s == HF_OK && (cudaFuncSetAttribute(k_swa_tc5g<64, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, SwaTc5<64, 2>::SMEM_BYTES) != cudaSuccess ||
                           cudaFuncSetAttribute(k_swa_tc5g<64, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, SwaTc5<64, 2>::SMEM_BYTES) != cudaSuccess ||
                           cudaFuncSetAttribute(k_swa_tc5g<128, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, SwaTc5<128, 2>::SMEM_BYTES) != cudaSuccess ||
                           cudaFuncSetAttribute(k_swa_tc5g<128, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, SwaTc5<128, 2>::SMEM_BYTES) != cudaSuccess))
            s = fail(HF_ERR_CUDA, "cudaFuncSetAttribute(k_swa_tc5g) failed");
        if (s == HF_OK) s = set_state_attr<64>();
        if (s == HF_OK) s = set_state_attr<128>();
    }
    if (s == HF_OK && cudaDeviceSynchronize() != cudaSuccess) s = fail(HF_ERR_CUDA, "device synchronize failed in hf_create");
    if (s != HF_OK) { free_all(c); delete c; return s; }
    *out = c;
    return HF_OK;
}

hf_status hf_destroy(hf_ctx* c) {
    if (c == nullptr) return fail(HF_ERR_INVALID_ARG, "ctx is null");
    cudaSetDevice(c->device);
    cudaDeviceSynchronize();
    free_all(c);
    delete c;
    return HF_OK;
}

hf_status hf_reset(hf_ctx* c, int layer, void* stream) {
    if (c == nullptr) return fail(HF_ERR_INVALID_ARG, "ctx is null");
    if (layer != -1) HF_TRY(check_layer(c, layer));
    cudaStream_t st = (cudaStream_t)stream;
    const size_t dd = (size_t)c->BH * c->d * c->d, dz = (size_t)c->BH * c->d;
    for (int l = 0; l < c->cfg.layers; ++l) {
        if (layer != -1 && l != layer) continue;
        LayerState& L = c->layers[l];
        HF_CUDA(cudaMemsetAsync(L.S, 0, dd * 4, st));
        HF_CUDA(cudaMemsetAsync(L.z, 0, dz * 4, st));
        HF_CUDA(cudaMemsetAsync(L.sf_hi, 0, dd * 2, st));
        HF_CUDA(cudaMemsetAsync(L.sf_lo, 0, dd * 2, st));
        L.n_cached = 0; L.head = 0; L.n_sink = 0; L.absorbed = 0; L.frames = 0; L.cache_epoch++; L.sel_epoch = ~0ull;
    }
    return HF_OK;
}

hf_status hf_set_merge_weights(hf_ctx* c, int layer, const void* W, const void* bias, void* stream) {
    HF_TRY(check_layer(c, layer));
    if (c->cfg.merge == HF_MERGE_IDENTITY) return fail(HF_ERR_STATE, "context was created with HF_MERGE_IDENTITY");
    HF_TRY(check_ptr(W, "W"));
    if (bias != nullptr) HF_TRY(check_ptr(bias, "bias"));
    cudaStream_t st = (cudaStream_t)stream;
    LayerState& L = c->layers[layer];
    if (c->cfg.merge == HF_MERGE_FULL_WIDTH) {      // one [H d, H d] matrix: applied by its own kernel after the read-out
        const size_t hd = (size_t)c->cfg.heads * c->d;
        HF_CUDA(cudaMemcpyAsync(L.W_full, W, hd * hd * 2, cudaMemcpyDeviceToDevice, st));
        if (bias) HF_CUDA(cudaMemcpyAsync(L.bias, bias, hd * 2, cudaMemcpyDeviceToDevice, st));
        L.has_wfull = true;
        L.has_bias = bias != nullptr;
        return HF_OK;
    }
    HF_CUDA(cudaMemcpyAsync(L.W, W, (size_t)c->cfg.heads * c->d * c->d * 2, cudaMemcpyDeviceToDevice, st));
    if (bias) HF_CUDA(cudaMemcpyAsync(L.bias, bias, (size_t)c->cfg.heads * c->d * 2, cudaMemcpyDeviceToDevice, st));
    L.has_w = true;
    L.has_bias = bias != nullptr;
    return HF_DISPATCH_D(c, launch_fold, c, L, 0, st);
}

hf_status hf_set_rope(hf_ctx* c, const float* cos_q, const float* sin_q, const float* cos_k, const float* sin_k, void* stream) {
    if (c == nullptr) return fail(HF_ERR_INVALID_ARG, "ctx is null");
    if ((cos_q == nullptr) != (sin_q == nullptr) || (cos_k == nullptr) != (sin_k == nullptr))
        return fail(HF_ERR_INVALID_ARG, "cos and sin tables come in pairs");
    const float* src[4] = {cos_q, sin_q, cos_k, sin_k};
    float** dst[4] = {&c->rope_q[0], &c->rope_q[1], &c->rope_k[0], &c->rope_k[1]};
    const size_t count = (size_t)c->Tc * (c->d / 2);
    cudaStream_t st = (cudaStream_t)stream;
    for (int i = 0; i < 4; ++i) {
        if (src[i] == nullptr) continue;
        HF_TRY(check_ptr(src[i], "rotation table"));
        if (*dst[i] == nullptr) HF_TRY(dmalloc(dst[i], count));
        HF_CUDA(cudaMemcpyAsync(*dst[i], src[i], count * sizeof(float), cudaMemcpyDeviceToDevice, st));
    }
    c->has_rope_q = cos_q != nullptr;
    c->has_rope_k = cos_k != nullptr;
    return HF_OK;
}

hf_status hf_set_temporal_rope(hf_ctx* c, int t0, int first_pair, int n_pairs, const float* cos_tab, const float* sin_tab, void* stream) {
    if (c == nullptr) return fail(HF_ERR_INVALID_ARG, "ctx is null");
    for (const LayerState& L : c->layers)
        if (L.frames != 0) return fail(HF_ERR_STATE, "the temporal rotation must be set before the first chunk is committed (or after hf_reset)");
    if (cos_tab == nullptr && sin_tab == nullptr) { c->has_trope = false; return HF_OK; }
    HF_TRY(check_ptr(cos_tab, "cos_tab"));
    HF_TRY(check_ptr(sin_tab, "sin_tab"));
    if (t0 < c->cfg.chunk_frames) return fail(HF_ERR_SHAPE, "t0 (%d) must be at least chunk_frames (%d)", t0, c->cfg.chunk_frames);
    if (first_pair < 0 || n_pairs < 1 || first_pair + n_pairs > c->d / 2)
        return fail(HF_ERR_SHAPE, "pairs [%d, %d) outside the head's %d feature pairs", first_pair, first_pair + n_pairs, c->d / 2);
    cudaStream_t st = (cudaStream_t)stream;
    const size_t count = (size_t)(t0 + 1) * n_pairs;
    HF_CUDA(cudaStreamSynchronize(st));
    const float* src[2] = {cos_tab, sin_tab};
    for (int i = 0; i < 2; ++i) {
        cudaFree(c->trope_tab[i]); c->trope_tab[i] = nullptr;
        HF_TRY(dmalloc(&c->trope_tab[i], count));
        HF_CUDA(cudaMemcpyAsync(c->trope_tab[i], src[i], count * sizeof(float), cudaMemcpyDeviceToDevice, st));
    }
    if (c->q_rot == nullptr) HF_TRY(dmalloc(&c->q_rot, c->chunk_elems));
    if (c->k_rot == nullptr) HF_TRY(dmalloc(&c->k_rot, c->chunk_elems));
    c->trope.cos_tab = c->trope_tab[0]; c->trope.sin_tab = c->trope_tab[1];
    c->trope.first_pair = first_pair; c->trope.n_pairs = n_pairs; c->trope.tokens_per_frame = c->cfg.tokens_per_frame;
    c->t0 = t0;
    c->has_trope = true;
    return HF_OK;
}

hf_status hf_state_absorb(hf_ctx* c, int layer, const void* k_ev, const void* v_ev, int n_tokens, void* stream) {
    HF_TRY(check_layer(c, layer));
    HF_TRY(check_ptr(k_ev, "k_ev"));
    HF_TRY(check_ptr(v_ev, "v_ev"));
    if (n_tokens < 1) return fail(HF_ERR_SHAPE, "n_tokens must be >= 1");
    if (c->has_rope_k && n_tokens > c->Tc)
        return fail(HF_ERR_SHAPE, "with rotation tables set, n_tokens may not exceed the chunk length (%d)", c->Tc);
    if (c->cfg.z_mode == HF_Z_FRAME_MEAN && n_tokens % c->cfg.tokens_per_frame != 0)
        return fail(HF_ERR_SHAPE, "with HF_Z_FRAME_MEAN n_tokens must be a multiple of tokens_per_frame (%d)", c->cfg.tokens_per_frame);
    LayerState& L = c->layers[layer];
    HF_TRY(HF_DISPATCH_D(c, launch_absorb, c, L, (const bf16*)k_ev, (const bf16*)v_ev, n_tokens, (cudaStream_t)stream));
    L.absorbed += n_tokens;
    return HF_OK;
}

hf_status hf_kv_append(hf_ctx* c, int layer, const void* k, const void* v, void* stream) {
    HF_TRY(check_layer(c, layer));
    HF_TRY(check_ptr(k, "k"));
    HF_TRY(check_ptr(v, "v"));
    LayerState& L = c->layers[layer];
    cudaStream_t st = (cudaStream_t)stream;
    // Relative temporal RoPE (Eq. 8): a key enters the cache turned to the index it has while the NEXT chunk is generated;
    // when the cap makes the window's indices slide, the chunks that stay are turned by the same amount, in place.
    const int cf = c->cfg.chunk_frames;
    const int top_now = c->has_trope ? trope_top(c, L.frames) : 0, top_next = c->has_trope ? trope_top(c, L.frames + cf) : 0;
    if (L.n_sink < c->n_sink_max) {   // the stream's first chunks are the attention sink: kept in slots of their own for good
        const int slot = c->R + L.n_sink;
        PoolJobs jobs;
        memset(&jobs, 0, sizeof(jobs));
        jobs.job[0].src = (const bf16*)k; jobs.job[0].copy_dst = L.ring_k + (size_t)slot * c->chunk_elems;
        jobs.job[0].pooled = L.pooled_k + (size_t)slot * c->pooled_elems;
        if (c->has_trope) { jobs.job[0].rot_on = 1; jobs.job[0].rot_base = top_now - cf + 1; jobs.job[0].rot_per_frame = 1; }   // its own indices, for good
        jobs.job[1].src = (const bf16*)v; jobs.job[1].copy_dst = L.ring_v + (size_t)slot * c->chunk_elems;
        HF_TRY(HF_DISPATCH_D(c, launch_pool, c, jobs, 2, st));
        L.n_sink++;
        L.frames += cf;
        L.cache_epoch++;
        return HF_OK;
    }
    if (c->P == 0) {   // window == chunk: a committed chunk leaves the window at once (as the window saw it: at its own indices)
        const bf16* ks = (const bf16*)k;
        if (c->has_trope) {
            PoolJobs jobs;
            memset(&jobs, 0, sizeof(jobs));
            jobs.job[0].src = ks; jobs.job[0].copy_dst = c->k_rot; jobs.job[0].rot_on = 1; jobs.job[0].rot_base = top_now - cf + 1; jobs.job[0].rot_per_frame = 1;
            HF_TRY(HF_DISPATCH_D(c, launch_pool, c, jobs, 1, st));
            ks = c->k_rot;
        }
        HF_TRY(HF_DISPATCH_D(c, launch_absorb, c, L, ks, (const bf16*)v, c->Tc, st));
        L.absorbed += c->Tc;
        L.frames += cf;
        L.cache_epoch++;
        return HF_OK;
    }
    // The ring has one slot more than the window holds, so the new chunk never lands on the chunk that leaves: the state
    // update (Eq. 3) of the evicted chunk runs on the side stream beside the copy of the new one (the copy kernel's thread
    // blocks fit on the SMs next to the absorb kernel's), and the call joins the two before it returns to the caller's
    // stream.  The state is still updated before anything can overwrite the evicted chunk: the slot it sits in is the
    // target of the NEXT commit, which is ordered after this call's join.
    const int slot = (L.head + L.n_cached) % c->R;
    bool evicted = false;
    if (L.n_cached == c->P) {
        HF_TRY(HF_DISPATCH_D(c, launch_absorb, c, L, L.ring_k + (size_t)L.head * c->chunk_elems,
                             L.ring_v + (size_t)L.head * c->chunk_elems, c->Tc, st, true));
        evicted = true;
        L.absorbed += c->Tc;
        L.head = (L.head + 1) % c->R;
    } else {
        L.n_cached++;
    }
    PoolJobs jobs;
    memset(&jobs, 0, sizeof(jobs));
    jobs.job[0].src = (const bf16*)k; jobs.job[0].copy_dst = L.ring_k + (size_t)slot * c->chunk_elems;
    jobs.job[0].pooled = L.pooled_k + (size_t)slot * c->pooled_elems;
    if (c->has_trope) { jobs.job[0].rot_on = 1; jobs.job[0].rot_base = top_next - 2 * cf + 1; jobs.job[0].rot_per_frame = 1; }
    jobs.job[1].src = (const bf16*)v; jobs.job[1].copy_dst = L.ring_v + (size_t)slot * c->chunk_elems;
    HF_TRY(HF_DISPATCH_D(c, launch_pool, c, jobs, 2, st));
    const int slide = c->has_trope ? top_next - top_now - cf : 0;       // 0 below the cap, then -chunk_frames
    if (slide != 0) {
        // the chunks that stay in the window (L.head is already past the one that left; the new chunk is not counted yet when
        // the window was still filling): their keys and block means, turned in place
        const int stay = evicted ? L.n_cached - 1 : L.n_cached - 1;
        for (int i = 0; i < stay; i += 3) {
            PoolJobs rj;
            memset(&rj, 0, sizeof(rj));
            int n = 0;
            for (; n < 3 && i + n < stay; ++n) {
                const int sl = (L.head + i + n) % c->R;
                bf16* kp = L.ring_k + (size_t)sl * c->chunk_elems;
                rj.job[n].src = kp; rj.job[n].copy_dst = kp; rj.job[n].pooled = L.pooled_k + (size_t)sl * c->pooled_elems;
                rj.job[n].rot_on = 1; rj.job[n].rot_base = slide; rj.job[n].rot_per_frame = 0;
            }
            HF_TRY(HF_DISPATCH_D(c, launch_pool, c, rj, n, st));
        }
    }
    if (evicted) HF_CUDA(cudaStreamWaitEvent(st, c->ev_join, 0));
    L.frames += cf;
    L.cache_epoch++;
    return HF_OK;
}

hf_status hf_state_absorb_layers(hf_ctx* c, int first_layer, int n_layers, const void* k_ev, const void* v_ev, int n_tokens,
                                 void* stream) {
    if (c == nullptr) return fail(HF_ERR_INVALID_ARG, "ctx is null");
    if (n_layers < 1 || first_layer < 0 || first_layer + n_layers > c->cfg.layers)
        return fail(HF_ERR_INVALID_ARG, "layers [%d, %d) outside [0, %d)", first_layer, first_layer + n_layers, c->cfg.layers);
    HF_TRY(check_ptr(k_ev, "k_ev"));
    HF_TRY(check_ptr(v_ev, "v_ev"));
    if (n_tokens < 1) return fail(HF_ERR_SHAPE, "n_tokens must be >= 1");
    if (c->has_rope_k && n_tokens > c->Tc)
        return fail(HF_ERR_SHAPE, "with rotation tables set, n_tokens may not exceed the chunk length (%d)", c->Tc);
    if (c->cfg.z_mode == HF_Z_FRAME_MEAN && n_tokens % c->cfg.tokens_per_frame != 0)
        return fail(HF_ERR_SHAPE, "with HF_Z_FRAME_MEAN n_tokens must be a multiple of tokens_per_frame (%d)", c->cfg.tokens_per_frame);
    cudaStream_t st = (cudaStream_t)stream;
    const size_t per_layer = (size_t)c->BH * n_tokens * c->d;
    // One persistent launch pays when there are at least as many (layer, batch*head) items as SMs; below that the
    // per-layer kernel, which cuts every item over several thread blocks, fills the device better.  Same bits either way.
    if ((long long)n_layers * c->BH < c->sm_count) {
        for (int l = 0; l < n_layers; ++l)
            HF_TRY(HF_DISPATCH_D(c, launch_absorb, c, c->layers[first_layer + l], (const bf16*)k_ev + l * per_layer,
                                 (const bf16*)v_ev + l * per_layer, n_tokens, st));
    } else {
        for (int l0 = 0; l0 < n_layers; l0 += HF_MAX_BATCH_LAYERS) {
            const int nl = n_layers - l0 < HF_MAX_BATCH_LAYERS ? n_layers - l0 : HF_MAX_BATCH_LAYERS;
            CUtensorMap tk, tv;
            HF_TRY(make_map_ex(c, &tk, (const bf16*)k_ev + l0 * per_layer, n_tokens, nl, c->d, 64, false));
            HF_TRY(make_map_ex(c, &tv, (const bf16*)v_ev + l0 * per_layer, n_tokens, nl, 64, 64, true));
            int slot[HF_MAX_BATCH_LAYERS];
            for (int l = 0; l < nl; ++l) slot[l] = l;
            HF_TRY(HF_DISPATCH_D(c, launch_absorb_layers, c, first_layer + l0, nl, tk, tv, slot, n_tokens, st));
        }
    }
    for (int l = 0; l < n_layers; ++l) c->layers[first_layer + l].absorbed += n_tokens;
    return HF_OK;
}

hf_status hf_kv_append_layers(hf_ctx* c, int first_layer, int n_layers, const void* const* k, const void* const* v, void* stream) {
    if (c == nullptr) return fail(HF_ERR_INVALID_ARG, "ctx is null");
    if (n_layers < 1 || first_layer < 0 || first_layer + n_layers > c->cfg.layers)
        return fail(HF_ERR_INVALID_ARG, "layers [%d, %d) outside [0, %d)", first_layer, first_layer + n_layers, c->cfg.layers);
    if (k == nullptr || v == nullptr) return fail(HF_ERR_INVALID_ARG, "pointer table is null");
    for (int l = 0; l < n_layers; ++l) {
        HF_TRY(check_ptr(k[l], "k[layer]"));
        HF_TRY(check_ptr(v[l], "v[layer]"));
    }
    cudaStream_t st = (cudaStream_t)stream;
    // The batched launches need every layer of the call in the same phase of Alg. 2's protocol (all still filling their
    // sink, all filling the window, or all evicting) and enough (layer, batch*head) items to fill the device; anything
    // else goes layer by layer.  The state gets the same bits either way.
    const LayerState& L0 = c->layers[first_layer];
    bool uniform = c->P > 0 && !c->has_trope && n_layers <= HF_MAX_BATCH_LAYERS && (long long)n_layers * c->BH >= c->sm_count;
    for (int l = 1; uniform && l < n_layers; ++l) {
        const LayerState& L = c->layers[first_layer + l];
        uniform = (L.n_sink < c->n_sink_max) == (L0.n_sink < c->n_sink_max) && (L.n_cached == c->P) == (L0.n_cached == c->P);
    }
    if (!uniform) {
        for (int l = 0; l < n_layers; ++l) HF_TRY(hf_kv_append(c, first_layer + l, k[l], v[l], stream));
        return HF_OK;
    }
    PoolLayersParams pp;
    memset(&pp, 0, sizeof(pp));
    pp.chunk_elems = c->chunk_elems; pp.pooled_elems = c->pooled_elems; pp.slots_per_layer = c->slots_per_layer;
    pp.ring_k = c->ring_k_all + (size_t)first_layer * c->slots_per_layer * c->chunk_elems;
    pp.ring_v = c->ring_v_all + (size_t)first_layer * c->slots_per_layer * c->chunk_elems;
    pp.pooled = c->pooled_k_all + (size_t)first_layer * c->slots_per_layer * c->pooled_elems;
    const bool sink = L0.n_sink < c->n_sink_max, evict = !sink && L0.n_cached == c->P;
    int ev_slot[HF_MAX_BATCH_LAYERS];
    for (int l = 0; l < n_layers; ++l) {
        LayerState& L = c->layers[first_layer + l];
        pp.k_src[l] = (const bf16*)k[l]; pp.v_src[l] = (const bf16*)v[l];
        pp.slot[l] = sink ? c->R + L.n_sink : (L.head + L.n_cached) % c->R;
        ev_slot[l] = (first_layer + l) * c->slots_per_layer + L.head;
    }
    if (evict) {
        // as in hf_kv_append: the state update of the chunks that leave runs on the side stream beside the copy of the new
        // ones (which go to the spare slots), and the call joins the two
        HF_CUDA(cudaEventRecord(c->ev_fork, st));
        HF_CUDA(cudaStreamWaitEvent(c->side, c->ev_fork, 0));
        HF_TRY(HF_DISPATCH_D(c, launch_absorb_layers, c, first_layer, n_layers, c->tm_kall, c->tm_vall, ev_slot, c->Tc, c->side));
        HF_CUDA(cudaEventRecord(c->ev_join, c->side));
    }
    HF_TRY(HF_DISPATCH_D(c, launch_pool_layers, c, pp, n_layers, st));
    if (evict) HF_CUDA(cudaStreamWaitEvent(st, c->ev_join, 0));
    for (int l = 0; l < n_layers; ++l) {
        LayerState& L = c->layers[first_layer + l];
        if (sink) L.n_sink++;
        else if (evict) { L.absorbed += c->Tc; L.head = (L.head + 1) % c->R; }
        else L.n_cached++;
        L.frames += c->cfg.chunk_frames;
        L.cache_epoch++;
    }
    return HF_OK;
}

hf_status hf_block_select(hf_ctx* c, int layer, const void* q, const void* k_cur, uint32_t* mask_out, int32_t* idx_out,
                          float* scores_out, void* stream) {
    HF_TRY(check_layer(c, layer));
    HF_TRY(check_ptr(q, "q"));
    HF_TRY(check_ptr(k_cur, "k_cur"));
    return HF_DISPATCH_D(c, launch_select, c, c->layers[layer], (const bf16*)q, (const bf16*)k_cur, mask_out, idx_out,
                         scores_out, (cudaStream_t)stream);
}

hf_status hf_sparse_swa(hf_ctx* c, int layer, const void* q, const void* k_cur, const void* v_cur, const int32_t* idx,
                        void* o_local, float* lse, void* stream) {
    HF_TRY(check_layer(c, layer));
    HF_TRY(check_ptr(q, "q"));
    HF_TRY(check_ptr(k_cur, "k_cur"));
    HF_TRY(check_ptr(v_cur, "v_cur"));
    HF_TRY(check_ptr(o_local, "o_local"));
    LayerState& L = c->layers[layer];
    const int keep = keep_for(c, (L.n_sink + L.n_cached + 1) * c->n_b);
    if (idx == nullptr) {
        if (L.sel_epoch != L.cache_epoch) return fail(HF_ERR_STATE, "no block selection for the current cache contents; call hf_block_select first");
        idx = L.idx;
    }
    if (c->has_trope) {     // the queries and the current chunk's keys at their Eq. 8 indices
        HF_TRY(HF_DISPATCH_D(c, launch_rotate_inputs, c, L, (const bf16*)q, (const bf16*)k_cur, (cudaStream_t)stream));
        q = c->q_rot; k_cur = c->k_rot;
    }
    return launch_swa(c, L, (const bf16*)q, (const bf16*)k_cur, (const bf16*)v_cur, idx, keep, nullptr, (bf16*)o_local, lse,
                      (cudaStream_t)stream);
}

hf_status hf_sparse_swa_backward_dq(hf_ctx* c, int layer, const void* q, const void* k_cur, const void* v_cur, const int32_t* idx,
                                    const void* o_local, const float* lse, const void* d_o, void* dq, void* stream) {
    HF_TRY(check_layer(c, layer));
    HF_TRY(check_ptr(q, "q")); HF_TRY(check_ptr(k_cur, "k_cur")); HF_TRY(check_ptr(v_cur, "v_cur"));
    HF_TRY(check_ptr(o_local, "o_local")); HF_TRY(check_ptr(lse, "lse")); HF_TRY(check_ptr(d_o, "d_o")); HF_TRY(check_ptr(dq, "dq"));
    if (c->cfg.block != 128) return fail(HF_ERR_UNSUPPORTED, "the backward kernel takes 128-token blocks");
    if (c->has_trope) return fail(HF_ERR_UNSUPPORTED, "the backward kernel does not rotate its inputs (temporal RoPE is set)");
    LayerState& L = c->layers[layer];
    const int keep = keep_for(c, (L.n_sink + L.n_cached + 1) * c->n_b);
    if (idx == nullptr) {
        if (L.sel_epoch != L.cache_epoch) return fail(HF_ERR_STATE, "no block selection for the current cache contents; call hf_block_select first");
        idx = L.idx;
    }
    return HF_DISPATCH_D(c, launch_bwd_dq, c, L, (const bf16*)q, (const bf16*)k_cur, (const bf16*)v_cur, idx, keep, (const bf16*)o_local, lse,
                         (const bf16*)d_o, (bf16*)dq, (cudaStream_t)stream);
}

hf_status hf_sparse_swa_backward_dkv(hf_ctx* c, int layer, const void* q, const void* k_cur, const void* v_cur, const void* o_local,
                                     const float* lse, const void* d_o, void* dk, void* dv, void* stream) {
    HF_TRY(check_layer(c, layer));
    HF_TRY(check_ptr(q, "q")); HF_TRY(check_ptr(k_cur, "k_cur")); HF_TRY(check_ptr(v_cur, "v_cur"));
    HF_TRY(check_ptr(o_local, "o_local")); HF_TRY(check_ptr(lse, "lse")); HF_TRY(check_ptr(d_o, "d_o"));
    HF_TRY(check_ptr(dk, "dk")); HF_TRY(check_ptr(dv, "dv"));
    if (c->cfg.block != 128) return fail(HF_ERR_UNSUPPORTED, "the backward kernels take 128-token blocks");
    if (c->has_trope) return fail(HF_ERR_UNSUPPORTED, "the backward kernels do not rotate their inputs (temporal RoPE is set)");
    LayerState& L = c->layers[layer];
    if (L.sel_epoch != L.cache_epoch) return fail(HF_ERR_STATE, "no block selection for the current cache contents; call hf_block_select first");
    return HF_DISPATCH_D(c, launch_bwd_dkv, c, L, (const bf16*)q, (const bf16*)k_cur, (const bf16*)v_cur, (const bf16*)o_local, lse,
                         (const bf16*)d_o, (bf16*)dk, (bf16*)dv, (cudaStream_t)stream);
}

hf_status hf_linear_attn(hf_ctx* c, int layer, const void* q, void* o_hist, void* stream) {
    HF_TRY(check_layer(c, layer));
    HF_TRY(check_ptr(q, "q"));
    HF_TRY(check_ptr(o_hist, "o_hist"));
    if (c->has_trope) {     // both branches see the queries with their temporal rotation
        HF_TRY(HF_DISPATCH_D(c, launch_rotate_inputs, c, c->layers[layer], (const bf16*)q, (const bf16*)nullptr, (cudaStream_t)stream));
        q = c->q_rot;
    }
    return HF_DISPATCH_D(c, launch_readout, c, c->layers[layer], (const bf16*)q, (bf16*)o_hist, (float*)nullptr, (cudaStream_t)stream);
}

hf_status hf_linear_attn_backward_dq(hf_ctx* c, int layer, const void* q, const void* d_o, void* dq, void* stream) {
    HF_TRY(check_layer(c, layer));
    HF_TRY(check_ptr(q, "q")); HF_TRY(check_ptr(d_o, "d_o")); HF_TRY(check_ptr(dq, "dq"));
    if (c->cfg.merge == HF_MERGE_FULL_WIDTH) return fail(HF_ERR_UNSUPPORTED, "the read-out's backward takes the per-head (or identity) merge");
    if (c->has_rope_q || c->has_trope) return fail(HF_ERR_UNSUPPORTED, "the read-out's backward does not rotate its inputs (a rotation is set)");
    return HF_DISPATCH_D(c, launch_readout_bwd, c, c->layers[layer], (const bf16*)q, (const bf16*)d_o, (bf16*)dq, (cudaStream_t)stream);
}

// Eq. 6 + Eq. 4 + Eq. 7 for a selection that is already made.  after_select: the call follows launch_select in the same
// stream directly, so the attention kernel may be launched under its tail.
static hf_status attend_merge(hf_ctx* c, LayerState& L, const bf16* q, const bf16* k, const bf16* v, const int32_t* idx, int keep,
                              bf16* o, cudaStream_t st, bool after_select) {
    // At head_dim 128 the tcgen05 attention kernel forms the history term itself (three more tensor-core products per
    // query block against the folded state, which it keeps in shared memory): no read-out kernel, no scratch buffer.
    // The rotated variant of Eq. 4 (numerator and denominator see different phi(Q)) keeps the separate read-out.
    if (c->swa_kernel == HF_SWA_TCGEN05 && c->d == 128 && c->cfg.block == 128 && SwaTc5<128, Tc5Groups<128>::N>::FUSE && !c->has_rope_q &&
        c->cfg.merge != HF_MERGE_FULL_WIDTH)
        return launch_swa_tc5_t<128>(c, L, q, k, v, idx, keep, nullptr, o, nullptr, st, true, after_select);
    // Otherwise the read-out kernel writes the history term to the context's scratch buffer and the attention kernel adds
    // it in its epilogue.
    HF_TRY(HF_DISPATCH_D(c, launch_readout, c, L, q, (bf16*)nullptr, c->hist, st));
    return launch_swa(c, L, q, k, v, idx, keep, c->hist, o, nullptr, st);
}

hf_status hf_sparse_swa_merged(hf_ctx* c, int layer, const void* q, const void* k_cur, const void* v_cur, const int32_t* idx,
                               void* o, void* stream) {
    HF_TRY(check_layer(c, layer));
    HF_TRY(check_ptr(q, "q"));
    HF_TRY(check_ptr(k_cur, "k_cur"));
    HF_TRY(check_ptr(v_cur, "v_cur"));
    HF_TRY(check_ptr(o, "o"));
    LayerState& L = c->layers[layer];
    const int keep = keep_for(c, (L.n_sink + L.n_cached + 1) * c->n_b);
    if (idx == nullptr) {
        if (L.sel_epoch != L.cache_epoch) return fail(HF_ERR_STATE, "no block selection for the current cache contents; call hf_block_select first");
        idx = L.idx;
    }
    if (c->has_trope) {
        HF_TRY(HF_DISPATCH_D(c, launch_rotate_inputs, c, L, (const bf16*)q, (const bf16*)k_cur, (cudaStream_t)stream));
        q = c->q_rot; k_cur = c->k_rot;
    }
    return attend_merge(c, L, (const bf16*)q, (const bf16*)k_cur, (const bf16*)v_cur, idx, keep, (bf16*)o, (cudaStream_t)stream, false);
}

hf_status hf_hybrid_forward(hf_ctx* c, int layer, const void* q, const void* k, const void* v, void* o, void* stream) {
    HF_TRY(check_layer(c, layer));
    HF_TRY(check_ptr(q, "q"));
    HF_TRY(check_ptr(k, "k"));
    HF_TRY(check_ptr(v, "v"));
    HF_TRY(check_ptr(o, "o"));
    LayerState& L = c->layers[layer];
    cudaStream_t st = (cudaStream_t)stream;
    const bool one_kernel = c->swa_kernel == HF_SWA_TCGEN05 && c->d == 128 && c->cfg.block == 128 && SwaTc5<128, Tc5Groups<128>::N>::FUSE &&
                            !c->has_rope_q && c->cfg.merge != HF_MERGE_FULL_WIDTH;
    if (one_kernel || c->has_trope) {
        // (with the temporal rotation the selection's pooling pass also writes the rotated q and k that everything after it
        // reads, so the history read-out cannot run beside it: one stream)
        HF_TRY(HF_DISPATCH_D(c, launch_select, c, L, (const bf16*)q, (const bf16*)k, (uint32_t*)nullptr, (int32_t*)nullptr, (float*)nullptr, st));
        if (c->has_trope) { q = c->q_rot; k = c->k_rot; }
        return attend_merge(c, L, (const bf16*)q, (const bf16*)k, (const bf16*)v, L.idx, L.sel_keep, (bf16*)o, st, one_kernel);
    }
    // Otherwise the history term depends on q and the state only: it runs on the context's side stream while pooling and
    // selection run on the caller's stream; the attention kernel, which adds it in its epilogue, waits for both.
    // (The fork event also orders this read-out after the previous call's attention kernel, which read the same
    // scratch buffer.)
    HF_CUDA(cudaEventRecord(c->ev_fork, st));
    HF_CUDA(cudaStreamWaitEvent(c->side, c->ev_fork, 0));
    HF_TRY(HF_DISPATCH_D(c, launch_readout, c, L, (const bf16*)q, (bf16*)nullptr, c->hist, c->side));
    HF_CUDA(cudaEventRecord(c->ev_join, c->side));
    HF_TRY(HF_DISPATCH_D(c, launch_select, c, L, (const bf16*)q, (const bf16*)k, (uint32_t*)nullptr, (int32_t*)nullptr, (float*)nullptr, st));
    HF_CUDA(cudaStreamWaitEvent(st, c->ev_join, 0));
    return launch_swa(c, L, (const bf16*)q, (const bf16*)k, (const bf16*)v, L.idx, L.sel_keep, c->hist, (bf16*)o, nullptr, st);
}

hf_status hf_hybrid_forward_host(hf_ctx* c, int layer, const void* q_host, const void* k_host, const void* v_host,
                                 void* o_host, void* stream) {
    HF_TRY(check_layer(c, layer));
    if (!q_host || !k_host || !v_host || !o_host) return fail(HF_ERR_INVALID_ARG, "host pointer is null");
    HF_TRY(ensure_staging(c));
    cudaStream_t st = (cudaStream_t)stream;
    const size_t bytes = c->chunk_elems * 2;
    HF_CUDA(cudaMemcpyAsync(c->stage[0], q_host, bytes, cudaMemcpyHostToDevice, st));
    HF_CUDA(cudaMemcpyAsync(c->stage[1], k_host, bytes, cudaMemcpyHostToDevice, st));
    HF_CUDA(cudaMemcpyAsync(c->stage[2], v_host, bytes, cudaMemcpyHostToDevice, st));
    HF_TRY(hf_hybrid_forward(c, layer, c->stage[0], c->stage[1], c->stage[2], c->stage[3], stream));
    HF_CUDA(cudaMemcpyAsync(o_host, c->stage[3], bytes, cudaMemcpyDeviceToHost, st));
    HF_CUDA(cudaStreamSynchronize(st));
    return HF_OK;
}

hf_status hf_kv_append_host(hf_ctx* c, int layer, const void* k_host, const void* v_host, void* stream) {
    HF_TRY(check_layer(c, layer));
    if (!k_host || !v_host) return fail(HF_ERR_INVALID_ARG, "host pointer is null");
    HF_TRY(ensure_staging(c));
    cudaStream_t st = (cudaStream_t)stream;
    const size_t bytes = c->chunk_elems * 2;
    HF_CUDA(cudaMemcpyAsync(c->stage[1], k_host, bytes, cudaMemcpyHostToDevice, st));
    HF_CUDA(cudaMemcpyAsync(c->stage[2], v_host, bytes, cudaMemcpyHostToDevice, st));
    HF_TRY(hf_kv_append(c, layer, c->stage[1], c->stage[2], stream));
    HF_CUDA(cudaStreamSynchronize(st));
    return HF_OK;
}

hf_status hf_get_state(hf_ctx* c, int layer, float* S, float* z, void* stream) {
    HF_TRY(check_layer(c, layer));
    LayerState& L = c->layers[layer];
    cudaStream_t st = (cudaStream_t)stream;
    if (S) HF_CUDA(cudaMemcpyAsync(S, L.S, (size_t)c->BH * c->d * c->d * 4, cudaMemcpyDeviceToDevice, st));
    if (z) HF_CUDA(cudaMemcpyAsync(z, L.z, (size_t)c->BH * c->d * 4, cudaMemcpyDeviceToDevice, st));
    return HF_OK;
}

// ---- checkpoint image: header, then per layer {counts, S, z, held chunks in logical order (K, V, pooled sums)}
namespace {
constexpr uint64_t IMAGE_MAGIC = 0x3145544154534648ull;   // "HFSTATE1"
constexpr uint32_t IMAGE_VERSION = 2;
struct ImageHeader {
    uint64_t magic;
    uint32_t version, header_bytes;
    int32_t batch, heads, head_dim, tokens_per_frame, chunk_frames, window_frames, block, layers, phi, z_mode, sink_frames, reserved;
    uint64_t total_bytes;
};
struct ImageLayer {
    int32_t n_sink, n_cached;
    int64_t absorbed;
    int64_t frames;
};
size_t image_chunk_bytes(const hf_ctx* c) { return 2 * c->chunk_elems * sizeof(bf16) + c->pooled_elems * sizeof(float); }
size_t image_state_bytes(const hf_ctx* c) { return ((size_t)c->BH * c->d * c->d + (size_t)c->BH * c->d) * sizeof(float); }
ImageHeader image_header(const hf_ctx* c) {
    ImageHeader h;
    memset(&h, 0, sizeof(h));
    h.magic = IMAGE_MAGIC; h.version = IMAGE_VERSION; h.header_bytes = (uint32_t)sizeof(ImageHeader);
    h.batch = c->cfg.batch; h.heads = c->cfg.heads; h.head_dim = c->cfg.head_dim; h.tokens_per_frame = c->cfg.tokens_per_frame;
    h.chunk_frames = c->cfg.chunk_frames; h.window_frames = c->cfg.window_frames; h.block = c->cfg.block;
    h.layers = c->cfg.layers; h.phi = c->cfg.phi; h.z_mode = c->cfg.z_mode; h.sink_frames = c->cfg.sink_frames;
    return h;
}
int held_slot(const hf_ctx* c, const LayerState& L, int i) {   // slot of the i-th held chunk in logical order
    return i < L.n_sink ? c->R + i : (L.head + i - L.n_sink) % c->R;
}
}  // namespace

hf_status hf_state_export(hf_ctx* c, void* host_buf, size_t* bytes) {
    if (c == nullptr || bytes == nullptr) return fail(HF_ERR_INVALID_ARG, "null argument");
    size_t need = sizeof(ImageHeader);
    for (const LayerState& L : c->layers)
        need += sizeof(ImageLayer) + image_state_bytes(c) + (size_t)(L.n_sink + L.n_cached) * image_chunk_bytes(c);
    if (host_buf == nullptr) { *bytes = need; return HF_OK; }
    if (*bytes < need) {
        const size_t have = *bytes;
        *bytes = need;
        return fail(HF_ERR_SHAPE, "image needs %zu bytes, buffer holds %zu", need, have);
    }
    HF_CUDA(cudaSetDevice(c->device));
    HF_CUDA(cudaDeviceSynchronize());
    uint8_t* out = (uint8_t*)host_buf;
    ImageHeader h = image_header(c);
    h.total_bytes = need;
    memcpy(out, &h, sizeof(h));
    out += sizeof(h);
    const size_t dd = (size_t)c->BH * c->d * c->d * sizeof(float), dz = (size_t)c->BH * c->d * sizeof(float);
    const size_t kv = c->chunk_elems * sizeof(bf16), pl = c->pooled_elems * sizeof(float);
    for (const LayerState& L : c->layers) {
        ImageLayer il;
        il.n_sink = L.n_sink; il.n_cached = L.n_cached; il.absorbed = L.absorbed; il.frames = L.frames;
        memcpy(out, &il, sizeof(il)); out += sizeof(il);
        HF_CUDA(cudaMemcpy(out, L.S, dd, cudaMemcpyDeviceToHost)); out += dd;
        HF_CUDA(cudaMemcpy(out, L.z, dz, cudaMemcpyDeviceToHost)); out += dz;
        for (int i = 0; i < L.n_sink + L.n_cached; ++i) {
            const int slot = held_slot(c, L, i);
            HF_CUDA(cudaMemcpy(out, L.ring_k + (size_t)slot * c->chunk_elems, kv, cudaMemcpyDeviceToHost)); out += kv;
            HF_CUDA(cudaMemcpy(out, L.ring_v + (size_t)slot * c->chunk_elems, kv, cudaMemcpyDeviceToHost)); out += kv;
            HF_CUDA(cudaMemcpy(out, L.pooled_k + (size_t)slot * c->pooled_elems, pl, cudaMemcpyDeviceToHost)); out += pl;
        }
    }
    *bytes = need;
    return HF_OK;
}

hf_status hf_state_import(hf_ctx* c, const void* host_buf, size_t bytes) {
    if (c == nullptr || host_buf == nullptr) return fail(HF_ERR_INVALID_ARG, "null argument");
    if (bytes < sizeof(ImageHeader)) return fail(HF_ERR_INVALID_ARG, "buffer is shorter than an image header");
    const uint8_t* in = (const uint8_t*)host_buf;
    ImageHeader h;
    memcpy(&h, in, sizeof(h));
    if (h.magic != IMAGE_MAGIC || h.version != IMAGE_VERSION || h.header_bytes != sizeof(ImageHeader))
        return fail(HF_ERR_INVALID_ARG, "buffer is not a state image of this library version");
    const ImageHeader mine = image_header(c);
    if (h.batch != mine.batch || h.heads != mine.heads || h.head_dim != mine.head_dim ||
        h.tokens_per_frame != mine.tokens_per_frame || h.chunk_frames != mine.chunk_frames ||
        h.window_frames != mine.window_frames || h.block != mine.block || h.layers != mine.layers || h.phi != mine.phi ||
        h.z_mode != mine.z_mode || h.sink_frames != mine.sink_frames)
        return fail(HF_ERR_SHAPE, "the image was written by a context with another configuration");
    if (h.total_bytes > bytes) return fail(HF_ERR_INVALID_ARG, "image is cut short: %zu of %zu bytes", bytes, (size_t)h.total_bytes);
    // first pass: every count in range and the sizes add up; nothing is touched before the image is known to be whole
    size_t off = sizeof(ImageHeader);
    for (int l = 0; l < c->cfg.layers; ++l) {
        if (off + sizeof(ImageLayer) > h.total_bytes) return fail(HF_ERR_INVALID_ARG, "image ends inside layer %d", l);
        ImageLayer il;
        memcpy(&il, in + off, sizeof(il));
        if (il.n_sink < 0 || il.n_sink > c->n_sink_max || il.n_cached < 0 || il.n_cached > c->P || il.absorbed < 0 || il.frames < 0 ||
            (il.n_cached > 0 && il.n_sink < c->n_sink_max))
            return fail(HF_ERR_INVALID_ARG, "layer %d of the image holds counts this configuration cannot have", l);
        off += sizeof(ImageLayer) + image_state_bytes(c) + (size_t)(il.n_sink + il.n_cached) * image_chunk_bytes(c);
    }
    if (off != h.total_bytes) return fail(HF_ERR_INVALID_ARG, "image size does not match its contents");
    HF_CUDA(cudaSetDevice(c->device));
    HF_CUDA(cudaDeviceSynchronize());
    const size_t dd = (size_t)c->BH * c->d * c->d * sizeof(float), dz = (size_t)c->BH * c->d * sizeof(float);
    const size_t kv = c->chunk_elems * sizeof(bf16), pl = c->pooled_elems * sizeof(float);
    in += sizeof(ImageHeader);
    for (LayerState& L : c->layers) {
        ImageLayer il;
        memcpy(&il, in, sizeof(il)); in += sizeof(il);
        HF_CUDA(cudaMemcpy(L.S, in, dd, cudaMemcpyHostToDevice)); in += dd;
        HF_CUDA(cudaMemcpy(L.z, in, dz, cudaMemcpyHostToDevice)); in += dz;
        L.n_sink = il.n_sink; L.n_cached = il.n_cached; L.head = 0; L.absorbed = il.absorbed; L.frames = il.frames;
        L.cache_epoch++; L.sel_epoch = ~0ull;
        for (int i = 0; i < L.n_sink + L.n_cached; ++i) {
            const int slot = held_slot(c, L, i);
            HF_CUDA(cudaMemcpy(L.ring_k + (size_t)slot * c->chunk_elems, in, kv, cudaMemcpyHostToDevice)); in += kv;
            HF_CUDA(cudaMemcpy(L.ring_v + (size_t)slot * c->chunk_elems, in, kv, cudaMemcpyHostToDevice)); in += kv;
            HF_CUDA(cudaMemcpy(L.pooled_k + (size_t)slot * c->pooled_elems, in, pl, cudaMemcpyHostToDevice)); in += pl;
        }
        HF_TRY(HF_DISPATCH_D(c, launch_fold, c, L, 0, (cudaStream_t)0));   // S W^T halves from the restored S
    }
    HF_CUDA(cudaDeviceSynchronize());
    return HF_OK;
}

hf_status hf_query(hf_ctx* c, int layer, int what, int64_t* value) {
    HF_TRY(check_layer(c, layer));
    if (value == nullptr) return fail(HF_ERR_INVALID_ARG, "value is null");
    LayerState& L = c->layers[layer];
    const int Tn = (L.n_sink + L.n_cached + 1) * c->n_b;
    switch (what) {
        case HF_Q_CACHED_CHUNKS: *value = L.n_cached; break;
        case HF_Q_KEY_BLOCKS: *value = Tn; break;
        case HF_Q_KEPT_BLOCKS: *value = keep_for(c, Tn); break;
        case HF_Q_ABSORBED_TOKENS: *value = L.absorbed; break;
        case HF_Q_QUERY_BLOCKS: *value = c->Tm; break;
        case HF_Q_MASK_WORDS: *value = c->mask_words; break;
        case HF_Q_SWA_KERNEL: *value = c->swa_kernel; break;
        case HF_Q_SINK_CHUNKS: *value = L.n_sink; break;
        default: return fail(HF_ERR_INVALID_ARG, "unknown query %d", what);
    }
    return HF_OK;
}

hf_status hf_get_device_status(hf_ctx* c, int* flags, int* detail) {
    if (c == nullptr) return fail(HF_ERR_INVALID_ARG, "ctx is null");
    int h[4] = {0, 0, 0, 0};
    HF_CUDA(cudaDeviceSynchronize());
    HF_CUDA(cudaMemcpy(h, c->dev_status, 16, cudaMemcpyDeviceToHost));
    if (flags) *flags = h[0];
    if (detail) *detail = h[1];
    if (h[0] != 0) {
        HF_CUDA(cudaMemset(c->dev_status, 0, 8));      // flags and detail; the counters behind them run on
        if (h[0] & HF_DEV_TIMEOUT_FLAG)
            return fail(HF_ERR_DEVICE_TIMEOUT, "a device-side wait ran out (flags %d, detail %d)", h[0], h[1]);
        return fail(HF_ERR_INVALID_ARG, "an index list held a block index outside [0, T_n) (unit %d); block 0 was read in its place",
                    h[1]);
    }
    return HF_OK;
}

hf_status hf_slow_path_units(hf_ctx* c, int64_t* units) {
    if (c == nullptr || units == nullptr) return fail(HF_ERR_INVALID_ARG, "null argument");
    int h[4] = {0, 0, 0, 0};
    HF_CUDA(cudaDeviceSynchronize());
    HF_CUDA(cudaMemcpy(h, c->dev_status, 16, cudaMemcpyDeviceToHost));
    *units = h[2];
    return HF_OK;
}

hf_status hf_selftest_wait_limit(hf_ctx* c, void* stream) {
    if (c == nullptr) return fail(HF_ERR_INVALID_ARG, "ctx is null");
    // the kernel's two result words go to the reserved half of the status buffer's second line
    k_selftest_wait<<<1, 32, 0, (cudaStream_t)stream>>>(c->dev_status, 77, c->dev_status + 4);
    return post_launch(c, "k_selftest_wait");
}

hf_status hf_launch_count(hf_ctx* c, int64_t* launches) {
    if (c == nullptr || launches == nullptr) return fail(HF_ERR_INVALID_ARG, "null argument");
    *launches = c->launches;
    return HF_OK;
}

}  // extern "C"
