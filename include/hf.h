/*
 * hf.h -- C ABI of libhf: hybrid attention for an autoregressive streaming video denoiser
 * (block-sparse sliding-window attention over a rolling KV cache + linear-attention history state).
 *
 * One hf_ctx lives on ONE CUDA device and owns, per layer: the rolling cache of the last
 * P = window_frames/chunk_frames - 1 clean chunks (K, V, pooled K), the linear state
 * S [B,H,d,d] / z [B,H,d] in fp32, the merge projection, the last block selection and scratch.
 * The caller owns q/k/v/o.  Unless a parameter says "host", every data pointer is a DEVICE pointer
 * on the context's device, 16-byte aligned, to a contiguous tensor laid out [B, H, T, d] (d fastest)
 * of bf16.  `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls enqueue
 * work on `stream` and return; only create / destroy / the *_host calls / hf_get_device_status
 * synchronise.  Every call returns an hf_status; an invalid argument never launches a kernel.
 * Nothing here throws, aborts or traps the device.
 *
 * Concurrency: ONE stream per context at a time.  The scratch buffers (pooled means, split partial sums, the history
 * term of the two-kernel forward path, the staging buffers of the *_host calls), the side stream and its two events
 * belong to the context, not to a layer: two calls on the same context whose work may overlap on the device -- two
 * streams, or two host threads -- race on them, even for different layers.  Calls on one stream, in any order of layers,
 * are safe; so are different contexts on different streams.  To change streams, synchronise the old one first.
 *
 * Logical key-block order seen by selection and attention: oldest cached chunk first, newest cached
 * chunk, then the current chunk.  Every chunk is cut into blocks of `block` tokens from its own first
 * token; a short last block is legal (its mean uses its own length).
 */
#ifndef HF_H_
#define HF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hf_ctx hf_ctx;

typedef enum {
    HF_OK = 0,
    HF_ERR_INVALID_ARG = 1,   /* null / misaligned pointer, bad layer index                   */
    HF_ERR_SHAPE = 2,         /* configuration or size outside what the kernels support       */
    HF_ERR_STATE = 3,         /* call order: e.g. attention with no selection available       */
    HF_ERR_UNSUPPORTED = 4,
    HF_ERR_NOMEM = 5,
    HF_ERR_CUDA = 6,          /* a CUDA runtime call failed (no device, launch error, ...)    */
    HF_ERR_DEVICE_TIMEOUT = 7 /* a bounded device-side wait ran out; see hf_get_device_status */
} hf_status;

enum { HF_PHI_ELU1 = 0 };                                /* phi(x) = elu(x) + 1                 */
enum { HF_MERGE_IDENTITY = 0, HF_MERGE_PER_HEAD = 1, HF_MERGE_FULL_WIDTH = 2 };   /* "Linear" of Eq. 4: none | W[H,d,d] | W[H d, H d] */
enum { HF_SWA_AUTO = 0, HF_SWA_MMA = 1, HF_SWA_TCGEN05 = 2, HF_SWA_TCGEN05_PINGPONG = 3 }; /* sparse-attention kernel choice */
enum { HF_Z_SUM = 0, HF_Z_FRAME_MEAN = 1 };              /* z of Eq. 3: sum of phi(K) rows | per-frame means */

typedef struct {
    int batch, heads, head_dim;      /* head_dim d in {64, 128}                                         */
    int tokens_per_frame;            /* tokens of one latent frame                                      */
    int chunk_frames;                /* latent frames per chunk; T_c = tokens_per_frame * chunk_frames  */
    int window_frames;               /* sliding window w in frames, counts the current chunk;
                                        a multiple of chunk_frames, at most 8 chunks                    */
    int block;                       /* b_q = b_kv in {16, 64, 128}                                     */
    int topk;                        /* > 0: key blocks kept per query block                            */
    int keep_permille;               /* used when topk == 0: k = ceil(keep_permille * T_n / 1000)       */
    int layers;                      /* independent layer states held by the context                    */
    int phi;                         /* HF_PHI_ELU1                                                     */
    float eps;                       /* added to the denominator phi(q).z of Eq. 4                      */
    int merge;                       /* HF_MERGE_IDENTITY | HF_MERGE_PER_HEAD | HF_MERGE_FULL_WIDTH     */
    int swa_kernel;                  /* HF_SWA_AUTO | HF_SWA_MMA | HF_SWA_TCGEN05 | HF_SWA_TCGEN05_PINGPONG */
    int z_mode;                      /* HF_Z_SUM: z += sum_t phi(K_ev[t]) (default).  HF_Z_FRAME_MEAN: Eq. 3 as printed,
                                        z += sum over evicted latent frames of the mean of phi(K) over the frame's
                                        tokens; absorbed token counts must then be multiples of tokens_per_frame      */
    int sink_frames;                 /* latent frames at the start of the stream kept visible for ever (attention sink):
                                        a multiple of chunk_frames; those first chunks go to slots of their own, as the oldest
                                        logical key blocks, and are never evicted nor folded into the state.  Sink chunks +
                                        window chunks may not exceed 8                                                   */
} hf_config;

/* Fields of hf_query(). */
enum {
    HF_Q_CACHED_CHUNKS = 0,   /* clean chunks now in the rolling cache of the layer (sink chunks not counted) */
    HF_Q_KEY_BLOCKS = 1,      /* T_n a forward would see now: (sink + cached + 1) * blocks per chunk   */
    HF_Q_KEPT_BLOCKS = 2,     /* k_eff = min(k, T_n) for that T_n                                      */
    HF_Q_ABSORBED_TOKENS = 3, /* tokens folded into (S, z) so far (per batch*head)                     */
    HF_Q_QUERY_BLOCKS = 4,    /* T_m = ceil(T_c / block)                                               */
    HF_Q_MASK_WORDS = 5,      /* uint32 words per mask row = ceil(max T_n / 32)                        */
    HF_Q_SWA_KERNEL = 6,      /* kernel hf_sparse_swa resolves to (HF_SWA_MMA | HF_SWA_TCGEN05 | ..._PINGPONG) */
    HF_Q_SINK_CHUNKS = 7      /* sink chunks held so far                                               */
};

/* Create a context on CUDA device `device` (allocates all persistent buffers, zero state).
 * Errors: HF_ERR_INVALID_ARG (null), HF_ERR_SHAPE (unsupported sizes), HF_ERR_CUDA, HF_ERR_NOMEM. */
hf_status hf_create(const hf_config* cfg, int device, hf_ctx** out);
hf_status hf_destroy(hf_ctx* ctx);

/* Empty the rolling cache and zero (S, z) of one layer (layer = -1: all layers). */
hf_status hf_reset(hf_ctx* ctx, int layer, void* stream);

/* Merge projection of the history branch ("Linear" in Eq. 4; the paper does not give its shape).
 *   HF_MERGE_PER_HEAD (default reading): one d x d matrix per head, y = W_h h + bias_h.  W: bf16 [H, d, d] row-major
 *     (row = output dim), bias: bf16 [H, d] or NULL.  The matrix is folded into the state (S W_h^T), so it costs nothing
 *     per call.
 *   HF_MERGE_FULL_WIDTH: one matrix over the model width, y = W x + bias with x = the read-outs of all heads side by
 *     side (head-major).  W: bf16 [H d, H d] row-major (row = output feature), bias: bf16 [H d] or NULL.  It couples the
 *     heads: the read-out kernel is followed by a projection kernel, and the attention kernel adds the result.
 * Copied into the context.  HF_ERR_STATE if the context was created with HF_MERGE_IDENTITY. */
hf_status hf_set_merge_weights(hf_ctx* ctx, int layer, const void* W, const void* bias, void* stream);

/* Rotation inside the linear branch (Eq. 3: RoPE(phi(K))^T V in the state; Eq. 4: RoPE(phi(Q)) in the numerator only, the
 * normaliser never rotates).  The rotation acts on feature pairs (2i, 2i+1); the angles are the caller's: device float
 * tables cos / sin [T_c, d/2], one row per token of a chunk, shared by batch, heads and layers (e.g. built from the
 * capped relative temporal index of Eq. 8 and the spatial coordinates).  cos_q / sin_q rotate the queries of every later
 * hf_linear_attn / hf_hybrid_forward; cos_k / sin_k rotate the keys of every chunk folded into the state from now on
 * (they are applied when the chunk is absorbed).  The tables are copied into the context.  A NULL pair switches that
 * rotation off (the default).  With key tables set, hf_state_absorb accepts at most T_c tokens per call. */
hf_status hf_set_rope(hf_ctx* ctx, const float* cos_q, const float* sin_q, const float* cos_k, const float* sin_k, void* stream);

/* Relative temporal RoPE of the softmax branch (Sec. 3.3, Eq. 8): the temporal index of the chunk being generated counts
 * up with the stream until it reaches t0 (21 in the paper) and stays there; the keys in the cache are re-indexed by their
 * offset to the current chunk.  With this set, q and k are passed to every call WITHOUT temporal rotation (their spatial
 * rotation is the caller's and never changes); the library turns feature pairs [first_pair, first_pair + n_pairs) -- pair p
 * = features (2p, 2p+1) -- of every token by (index of its frame) x (frequency of the pair):
 *   - the queries and the current chunk's keys of a forward call to Eq. 8's indices (the stream position is the number of
 *     frames committed to that layer so far), in the pooling pass that the selection needs anyway; both branches see the
 *     rotated queries;
 *   - a committed chunk's keys to the indices they have while the NEXT chunk is generated; once the cap is reached every
 *     commit turns the chunks that stay in the window back by chunk_frames index steps, in place (keys and block means);
 *     the chunk that leaves is folded into the state as the window last saw it; sink chunks keep their own indices.
 * The cache stores bf16, so each turn rounds once more (at most window/chunk roundings in a key's life).
 *   cos_tab, sin_tab   device float [t0 + 1, n_pairs]: cosine and sine of (index steps) x (frequency of the pair); copied.
 * Must be set while no chunk has been committed (HF_ERR_STATE otherwise); both tables NULL switches it off.
 * The order of the float32 operations of a turn is fixed (the rotated values decide the block selection): x0' = x0 c - x1 s,
 * x1' = x0 s + x1 c, products and sums rounded separately, result rounded to bf16. */
hf_status hf_set_temporal_rope(hf_ctx* ctx, int t0, int first_pair, int n_pairs, const float* cos_tab, const float* sin_tab,
                               void* stream);

/* Alg. 2, cache commit of a clean chunk: k, v bf16 [B,H,T_c,d].  If the cache already holds P chunks the oldest
 * is folded into the state (Eq. 3: S += phi(K_ev)^T V_ev, z += sum phi(K_ev)) and leaves the window; the chunk's
 * K, V are copied in and its per-block K means stored.  The ring has P + 1 slots per layer (a spare one), so the copy
 * of the new chunk and the state update of the old one run side by side; when the call's work is done in stream order
 * both have happened, and the evicted chunk's slot is not written before the next commit.  With P = 0 the chunk goes
 * straight into the state and nothing is cached.  Device memory per layer: (P + 1 + sink chunks) x 2 x B*H*T_c*d bf16. */
hf_status hf_kv_append(hf_ctx* ctx, int layer, const void* k, const void* v, void* stream);

/* Eq. 3 on caller-supplied tokens: k_ev, v_ev bf16 [B,H,n_tokens,d], any n_tokens >= 1. */
hf_status hf_state_absorb(hf_ctx* ctx, int layer, const void* k_ev, const void* v_ev, int n_tokens, void* stream);

/* Alg. 2's cache commit for layers first_layer .. first_layer + n_layers - 1 in one call.  In the sampler every layer
 * commits its clean chunk at the same moment ("if KV full: pop(0) -> update LN; KV.append", once per chunk), and one
 * layer's 28.75 MB at the 832x480 shape is too small a launch to use the memory system; here the chunks that leave are
 * folded into their layers' states by ONE persistent launch (Eq. 3; a thread block owns a (layer, batch*head) state for
 * the whole token range, so there are no partial sums and no second kernel to add them) and the new chunks are copied in
 * and pooled by one more.
 *   k, v   HOST arrays of n_layers DEVICE pointers, bf16 [B,H,T_c,d] each (entry l belongs to layer first_layer + l)
 * Every layer ends up exactly as after hf_kv_append(layer, k[l], v[l]): same cache contents and the same bits in S and
 * z (the token range is cut and summed in the same order).  Layers of the call that are in different phases of the
 * protocol (some still filling the window, some evicting), a window of one chunk, or too few (layer, batch*head) pairs
 * to fill the device are handled layer by layer inside the call. */
hf_status hf_kv_append_layers(hf_ctx* ctx, int first_layer, int n_layers, const void* const* k, const void* const* v, void* stream);

/* Eq. 3 on caller-supplied tokens for several layers at once: k_ev, v_ev device bf16 [n_layers, B, H, n_tokens, d]
 * (slice l goes into the state of layer first_layer + l).  Same result, bit for bit, as n_layers calls of
 * hf_state_absorb. */
hf_status hf_state_absorb_layers(hf_ctx* ctx, int first_layer, int n_layers, const void* k_ev, const void* v_ev, int n_tokens,
                                 void* stream);

/* Eq. 5 + top-K rule (Alg. 3: M_c[i,j] = 1 iff block j is among the K best of row i): block means of q and of
 * the window's keys (cached chunks + k_cur), scores in a fixed float32 operation order, per (batch, head, query
 * block) the k_eff highest scores kept, equal scores going to the lower block index.  The selection is kept in
 * the context for hf_sparse_swa and optionally written out:
 *   mask_out   uint32 [B,H,T_m,HF_Q_MASK_WORDS], bit (j & 31) of word (j >> 5) = block j kept;  or NULL
 *   idx_out    int32  [B,H,T_m,k_eff] kept block indices ascending;                            or NULL
 *   scores_out float  [B,H,T_m,T_n] raw scores A_ij;                                           or NULL */
hf_status hf_block_select(hf_ctx* ctx, int layer, const void* q, const void* k_cur,
                          uint32_t* mask_out, int32_t* idx_out, float* scores_out, void* stream);

/* Eq. 6 / Alg. 3 inner loops: o_local[r] = softmax_c(q_r . k_c / sqrt(d)) V over the tokens c of the kept key
 * blocks of r's query block.  idx: int32 [B,H,T_m,k_eff] ascending block indices, or NULL = the context's last
 * selection for this layer (HF_ERR_STATE if none or if the cache changed since).  o_local: bf16 [B,H,T_c,d].
 * lse: float [B,H,T_c] natural-log sum of exp of the scaled logits, or NULL.
 * The list lives on the device, so the host cannot look at it: the kernel checks every entry against [0, T_n), reads
 * block 0 in place of an entry outside it (no address is ever formed from such an entry) and sets flag 2 of the
 * device status word; the rows of that query block are then meaningless and hf_get_device_status reports
 * HF_ERR_INVALID_ARG. */
hf_status hf_sparse_swa(hf_ctx* ctx, int layer, const void* q, const void* k_cur, const void* v_cur,
                        const int32_t* idx, void* o_local, float* lse, void* stream);

/* Gradient of Eq. 6 with respect to the queries: the first piece of the backward pass that the training rollout needs
 * for the denoising step it runs with gradient (Alg. 1).  With p = softmax over the kept keys and g = dL/dO_local,
 *   dq_r = (1 / sqrt(d)) sum_c p_rc (g_r . v_c - g_r . o_local_r) k_c      (the block mask is the forward's, held fixed)
 *   q, k_cur, v_cur, idx   as for hf_sparse_swa (same cache contents, same selection)
 *   o_local bf16 [B,H,T_c,d], lse float [B,H,T_c]   what hf_sparse_swa returned for them
 *   d_o bf16 [B,H,T_c,d] = dL/dO_local;  dq bf16 [B,H,T_c,d] out
 * 128-token blocks only (HF_ERR_UNSUPPORTED otherwise, and with the temporal rotation set).  The history branch's share of
 * dq comes from hf_linear_attn_backward_dq. */
hf_status hf_sparse_swa_backward_dq(hf_ctx* ctx, int layer, const void* q, const void* k_cur, const void* v_cur, const int32_t* idx,
                                    const void* o_local, const float* lse, const void* d_o, void* dq, void* stream);

/* Gradients of Eq. 6 with respect to the CURRENT chunk's keys and values (the cached chunks come from earlier,
 * gradient-free passes of the rollout and receive none): with the notation above, for key token c of the current chunk
 *   dv_c = sum_r p_rc g_r,     dk_c = (1 / sqrt(d)) sum_r p_rc (g_r . v_c - g_r . o_local_r) q_r
 * over the query rows r whose query block keeps c's key block -- the context's last selection for this layer
 * (hf_block_select or hf_hybrid_forward; HF_ERR_STATE if the cache changed since).  Arguments as for
 * hf_sparse_swa_backward_dq; dk, dv bf16 [B,H,T_c,d] out (zero for a key block that no query block keeps). */
hf_status hf_sparse_swa_backward_dkv(hf_ctx* ctx, int layer, const void* q, const void* k_cur, const void* v_cur, const void* o_local,
                                     const float* lse, const void* d_o, void* dk, void* dv, void* stream);

/* Gradient of Eq. 4 (hf_linear_attn, per-head or identity merge, no rotation) with respect to the queries.  With
 * f = phi(q_r), den = f . z + eps, S' = S W^T and g_r = d_o[r] (the gradient with respect to o_hist[r], which by Eq. 7 is
 * the gradient with respect to the merged output):
 *   u = S' g_r,   df = (u - (f . u / den) z) / den,   dq[r] = df * phi'(q_r)   (phi' = 1 above zero, e^x otherwise).
 * S, z and the cached chunks come from earlier, gradient-free passes and receive nothing.  The total gradient of the
 * hybrid output with respect to q is this plus hf_sparse_swa_backward_dq's (the caller adds them).  q, d_o bf16
 * [B,H,T_c,d] device; dq bf16 [B,H,T_c,d] out.  HF_ERR_UNSUPPORTED with the full-width merge or a rotation set. */
hf_status hf_linear_attn_backward_dq(hf_ctx* ctx, int layer, const void* q, const void* d_o, void* dq, void* stream);

/* Eq. 4 without rotation: o_hist[r] = W (phi(q_r) S / (phi(q_r) . z + eps)) + bias, bf16 [B,H,T_c,d]. */
hf_status hf_linear_attn(hf_ctx* ctx, int layer, const void* q, void* o_hist, void* stream);

/* Eq. 6 + Eq. 4 + Eq. 7 for a selection that is already made (idx as for hf_sparse_swa; NULL = the context's last
 * selection): o = o_local + o_history, rounded once to bf16 [B,H,T_c,d].  hf_hybrid_forward is hf_block_select followed
 * by this call.  With 128-token blocks at head_dim 128 and no rotation tables it is ONE kernel: the attention kernel
 * forms the history term on the tensor cores at the end of each query block; otherwise the read-out kernel runs first
 * and the attention kernel adds its result. */
hf_status hf_sparse_swa_merged(hf_ctx* ctx, int layer, const void* q, const void* k_cur, const void* v_cur, const int32_t* idx,
                               void* o, void* stream);

/* Alg. 3 + Eq. 7 for one denoising step: selection, sparse attention and history read-out of q against the
 * cache + (k, v), o = o_local + o_history rounded once to bf16 [B,H,T_c,d]. */
hf_status hf_hybrid_forward(hf_ctx* ctx, int layer, const void* q, const void* k, const void* v, void* o, void* stream);

/* Same two calls for HOST buffers (pinned memory recommended): inputs are copied to staging buffers owned by the
 * context, the device path runs, o is copied back, and the call returns after the stream has drained. */
hf_status hf_hybrid_forward_host(hf_ctx* ctx, int layer, const void* q_host, const void* k_host, const void* v_host,
                                 void* o_host, void* stream);
hf_status hf_kv_append_host(hf_ctx* ctx, int layer, const void* k_host, const void* v_host, void* stream);

/* State update without any allocation.  (No counterpart in the paper: it is the arithmetic of hf_state_absorb,
 * offered for callers that cannot allocate.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a region whose memory plan is already
 * frozen (a serving loop that pre-sized its pools and must not perturb them), a callback or plugin that is not
 * allowed to touch the allocator or to create an hf_ctx (which allocates at creation), or a host thread that must
 * not take the allocator's implicit device-wide synchronisation.  hf_state_absorb splits the token range over
 * several thread blocks and needs global scratch for their partial sums; here that scratch is a fixed 16 MiB array
 * compiled into the library image, which every device that loads the library holds until the process exits.
 *
 * Computes, on the current device:  S[bh] += phi(k_ev[bh])^T v_ev[bh],  z[bh] += sum_t phi(k_ev[bh][t])
 *   k_ev, v_ev  device bf16 [batch_heads, n_tokens, head_dim], read only
 *   S           device float [batch_heads, head_dim, head_dim], updated in place (caller initialises it)
 *   z           device float [batch_heads, head_dim], updated in place
 * Limits: head_dim in {64, 128}; 1 <= batch_heads <= 1024 and batch_heads * (head_dim^2 + head_dim) * 4 bytes must
 * fit in 16 MiB - 4 KiB (253 batch*heads at head_dim 128, 1008 at head_dim 64); anything larger returns HF_ERR_SHAPE
 * and launches nothing.  All pointers 16-byte aligned (else HF_ERR_INVALID_ARG).
 * The first call on a device looks up the device address of the scratch array and sets a kernel attribute; make
 * that first call outside any stream capture.  No call here uses cudaMalloc, cudaFree or an allocating library routine.
 * All calls on a device share the one array (each call rewrites the part it reads, so nothing has to be cleared): two calls
 * whose kernels may overlap on the GPU -- different streams, or different threads -- race; keep them stream-ordered. */
hf_status hf_state_absorb_noalloc(const void* k_ev, const void* v_ev, int batch_heads, int n_tokens, int head_dim,
                                  float* S, float* z, void* stream);

/* Copy the state out: S float [B,H,d,d] (row = key feature, column = value dim), z float [B,H,d]; either may be NULL. */
hf_status hf_get_state(hf_ctx* ctx, int layer, float* S, float* z, void* stream);

/* Checkpoint of the whole streaming state of the method (the rolling cache and the linear state, which is all the
 * memory the method carries from chunk to chunk -- Sec. 3.3; Alg. 2's KV and LN), for every layer of the context, into
 * ONE host buffer: per layer the sink chunks and the cached clean chunks (K, V and their pooled block sums, oldest
 * first -- the physical rotation of the ring is not kept), S, z and the absorbed-token count.  Merge weights and
 * rotation tables are parameters, not state: they are not in the image.
 *   host_buf == NULL : *bytes receives the size the image would have now; nothing is copied.
 *   host_buf != NULL : *bytes holds the capacity of host_buf on entry and the bytes written on return;
 *                      HF_ERR_SHAPE (and the needed size in *bytes) if the capacity is too small.
 * Synchronises the device.  The image is only meaningful to hf_state_import of this library version. */
hf_status hf_state_export(hf_ctx* ctx, void* host_buf, size_t* bytes);

/* Load an image written by hf_state_export into a context created with the same configuration (every field that
 * fixes a shape or the arithmetic of the state must match: HF_ERR_SHAPE otherwise; HF_ERR_INVALID_ARG for a buffer
 * that is not an image or is cut short).  All layers are replaced; the folded state is rebuilt from S and the merge
 * weights the context holds at that moment (weights set later refold it again).  A stream that continues after the
 * import produces bit-for-bit what the uninterrupted stream produces.  Synchronises the device.  Nothing is changed
 * when the image is rejected. */
hf_status hf_state_import(hf_ctx* ctx, const void* host_buf, size_t bytes);

/* Host-side bookkeeping values (HF_Q_*). */
hf_status hf_query(hf_ctx* ctx, int layer, int what, int64_t* value);

/* Synchronises the device and reports the device status word.  Flag 1: a bounded wait inside a kernel ran out
 * (detail = where), HF_ERR_DEVICE_TIMEOUT.  Flag 2: a caller's index list held a block index outside [0, T_n)
 * (detail = batch*head and query block of the row, as one number), HF_ERR_INVALID_ARG.  In both cases the result of
 * that launch is invalid, the word is cleared and the context stays usable. */
hf_status hf_get_device_status(hf_ctx* ctx, int* flags, int* detail);

/* Alg. 3 keeps a running row maximum m (m_new = max(m, rowmax S)) and rescales l and O by e^{m - m_new}.  The tcgen05
 * attention kernel (HF_SWA_TCGEN05, what HF_SWA_AUTO resolves to) instead fixes a row's reference after its first kept
 * key block (softmax does not depend on the reference), which covers rows whose later blocks rise up to about 100
 * natural-log units above the first; a (batch*head, query block) unit with a row beyond that is computed a second time
 * inside the same launch with the running maximum, so o is the softmax of Eq. 6 for every finite input and no status has
 * to be polled.  This call synchronises the device and reports how many units have taken that second pass since the
 * context was created (a diagnostic: such units cost several times a normal one). */
hf_status hf_slow_path_units(hf_ctx* ctx, int64_t* units);

/* Self-test of the failure path all kernels share (no counterpart in the paper).  Every wait inside a kernel is bounded:
 * when its limit runs out the thread block raises flag 1 of the status word and leaves in the ordinary way.  This call
 * launches a one-warp kernel that waits, under a limit of about a millisecond, on a barrier nothing ever arrives on, so
 * the wait runs out by construction; the next hf_get_device_status must then report HF_ERR_DEVICE_TIMEOUT with detail 77
 * and clear the word, and the context must work as before.  Nothing in it can hang or fault the device. */
hf_status hf_selftest_wait_limit(hf_ctx* ctx, void* stream);

/* Number of kernels the library has launched since the context was created. */
hf_status hf_launch_count(hf_ctx* ctx, int64_t* launches);

const char* hf_status_string(hf_status s);
const char* hf_last_error(void);   /* text of the last failure on this thread ("" if none) */

#ifdef __cplusplus
}
#endif
#endif /* HF_H_ */
