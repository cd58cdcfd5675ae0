"""CPU oracle for the hybrid attention of Hybrid Forcing.  TEST INFRASTRUCTURE ONLY.

Plain, slow numpy (fp64) restatement of what the hot path computes, written from
the paper's definitions.  It shares nothing with the CUDA path and must never be
imported by the product: only tests, the smoke check and the bench's CPU-baseline
leg may call it.

Inputs are real-valued numpy arrays (the bf16 inputs widened exactly to fp64).
Nothing is rounded anywhere, except in the *canonical fp32 scorer* below, which
restates in IEEE float32 the exact operation order in which block means and
block scores are formed, because a floating-point score decides an integer
(which blocks are kept) and both sides must take that decision in one precision.

What follows which passage:
  phi                     activation of the linear branch (Eq. 3; unnamed there, elu+1 here)
  block_ranges            Alg. 3 "divide Q / K,V into blocks", one chunk at a time
  block_means, block_scores        Eq. 5 (mean of a query block times mean of a key block)
  block_means_f32, block_scores_f32   Eq. 5 in the canonical float32 order
  keep_count, select_blocks         top-K rule after Eq. 5 / Alg. 3 "M_c[i,j] = 1 if in TopK(P_c[i,:], K)"
  sparse_attention        Eq. 6 as its plain definition: softmax over the kept keys
  sparse_attention_blockwise  the same result as a mixture of per-block softmaxes (the identity behind Alg. 3's tiling)
  absorb                  Eq. 3 (state update) without the rotation
  absorb_frame_mean       Eq. 3 with H accumulated as printed: per evicted frame the mean of phi(K) over its tokens
  linear_readout          Eq. 4: Linear(phi(Q) L / (phi(Q) H)), optionally with RoPE(phi(Q)) in the numerator
  rotate_pairs, absorb_rope        the rotation of Eq. 3 / Eq. 4 on feature pairs (2i, 2i+1); angles are inputs
  relative_temporal_indices        Eq. 8 (capped relative temporal index)
  window_temporal_indices, rotate_temporal   Sec. 3.3: the indices of cached chunks follow their offset to the current chunk;
                          the temporal rotation of the softmax branch's queries and keys
  rotate_temporal_f32     the same rotation in the canonical float32 order with the bf16 rounding the cache applies
  HybridStream            Alg. 2 cache protocol (evict -> update state -> append) around Alg. 3, Eq. 7 sum
  sparse_attention_backward, linear_readout_backward, HybridStream.backward
                          gradients of Eq. 6 / Eq. 4 / Eq. 7 for the training rollout (Alg. 1: the sampled step is run with
                          gradient), with the block mask held fixed (the top-K choice is piecewise constant)

Readings taken where the paper is silent or inconsistent (all listed again in the
design notes): H is accumulated as the plain sum of phi(K) rows (so that Eq. 4 is a
normalised kernel average); no rotation inside the linear branch; phi = elu + 1;
"Linear" is a per-head d x d matrix plus optional bias, y = W x + b; the top-K is
per query-block row; ties go to the lower (older) block index; each chunk is cut
into blocks from its own first token, a short last block is averaged over its own
length; the denominator is phi(q).H + eps.

Parity unpinned (nothing in the paper fixes them, the authors' code is not
available): the choice of phi, the shape of "Linear", the sum-vs-mean reading of
H, the rounding of K = ratio * T_n, the blocking of ragged chunks, the tie rule,
the eps.  Everything else is pinned by tests against brute force, closed forms
and library routines.
"""
from __future__ import annotations

import math
import numpy as np

F32 = np.float32


# --------------------------------------------------------------------------- phi
def phi(x: np.ndarray) -> np.ndarray:
    """elu(x) + 1: x + 1 for x > 0, exp(x) otherwise (positive feature map of the linear branch)."""
    x = np.asarray(x, dtype=np.float64)
    return np.where(x > 0.0, x + 1.0, np.exp(np.minimum(x, 0.0)))


# --------------------------------------------------------------------------- blocks
def block_ranges(n_tokens: int, b: int):
    """[(start, stop)] of consecutive blocks of b tokens; the last may be short."""
    return [(s, min(s + b, n_tokens)) for s in range(0, n_tokens, b)]


def key_block_table(chunk_lengths, b: int):
    """Logical key blocks of a window made of chunks (oldest first, current chunk last).

    Each chunk is cut from its own token 0.  Returns [(chunk_index, start, stop)]."""
    table = []
    for c, n in enumerate(chunk_lengths):
        table += [(c, s, e) for (s, e) in block_ranges(n, b)]
    return table


# --------------------------------------------------------------------------- Eq. 5, fp64
def block_means(x: np.ndarray, b: int) -> np.ndarray:
    """x [T, d] -> [ceil(T/b), d]: mean over the tokens of each block (Eq. 5 "Mean")."""
    x = np.asarray(x, dtype=np.float64)
    return np.stack([x[s:e].mean(axis=0) for (s, e) in block_ranges(x.shape[0], b)])


def block_scores(q_means: np.ndarray, k_means: np.ndarray) -> np.ndarray:
    """A[i, j] = Mean(q_i) . Mean(k_j)  (Eq. 5)."""
    return np.asarray(q_means, np.float64) @ np.asarray(k_means, np.float64).T


def pooled_softmax(scores: np.ndarray, d: int) -> np.ndarray:
    """P_c = Softmax(pool(Q) pool(K)^T / sqrt(d)), row-wise (Alg. 3 form of the block score)."""
    s = np.asarray(scores, np.float64) / math.sqrt(d)
    s = s - s.max(axis=1, keepdims=True)
    e = np.exp(s)
    return e / e.sum(axis=1, keepdims=True)


# --------------------------------------------------------------------------- Eq. 5, canonical float32
def block_means_f32(x: np.ndarray, b: int) -> np.ndarray:
    """Block means in the canonical float32 order.

    x is float32 [T, d] (bf16 values widened exactly).  Per block and per column:
    16 running sums, chain r adding tokens r, r+16, r+32, ... of the block in
    ascending order starting from +0; the 16 chains are then added one after another
    in ascending r; the total is divided by float32(n), n the block's own length.
    Every operation is one IEEE float32 operation, round to nearest even."""
    x = np.asarray(x)
    assert x.dtype == np.float32 and x.ndim == 2
    d = x.shape[1]
    out = []
    for (s, e) in block_ranges(x.shape[0], b):
        chains = np.zeros((16, d), dtype=F32)
        for t0 in range(s, e, 16):
            rows = x[t0:min(t0 + 16, e)]
            chains[: rows.shape[0]] = chains[: rows.shape[0]] + rows
        total = chains[0].copy()
        for r in range(1, 16):
            total = total + chains[r]
        out.append(total / F32(e - s))
    out = np.stack(out)
    assert out.dtype == np.float32
    return out


def block_scores_f32(q_means: np.ndarray, k_means: np.ndarray) -> np.ndarray:
    """A[i, j] in the canonical float32 order.

    32 partial sums: partial l takes columns l, l+32, l+64, ... in ascending order,
    each term a rounded float32 product added by a rounded float32 add (no fused
    multiply-add), the first product taken as is.  The 32 partials are then folded
    as a butterfly: p[l] + p[l+16] for l < 16, then +8, +4, +2, +1."""
    qm = np.asarray(q_means)
    km = np.asarray(k_means)
    assert qm.dtype == np.float32 and km.dtype == np.float32
    d = qm.shape[1]
    assert d % 32 == 0
    prod = qm[:, None, :] * km[None, :, :]                  # float32 products
    prod = prod.reshape(qm.shape[0], km.shape[0], d // 32, 32)
    acc = prod[:, :, 0, :].copy()
    for m in range(1, d // 32):
        acc = acc + prod[:, :, m, :]
    width = 16
    while width >= 1:
        acc = acc[..., :width] + acc[..., width:2 * width]
        width //= 2
    assert acc.dtype == np.float32
    return acc[..., 0]


# --------------------------------------------------------------------------- top-K
def keep_count(topk: int, keep_permille: int, n_key_blocks: int) -> int:
    """Blocks kept per query-block row: topk if given, else ceil(permille/1000 * T_n); at least 1, at most T_n."""
    k = topk if topk > 0 else -(-keep_permille * n_key_blocks // 1000)
    return max(1, min(k, n_key_blocks))


def select_blocks(scores: np.ndarray, k: int) -> np.ndarray:
    """Binary mask M [T_m, T_n]: per row the k largest scores, equal scores going to the lower index."""
    scores = np.asarray(scores)
    mask = np.zeros(scores.shape, dtype=bool)
    for i in range(scores.shape[0]):
        order = sorted(range(scores.shape[1]), key=lambda j: (-float(scores[i, j]), j))
        mask[i, order[:k]] = True
    return mask


# --------------------------------------------------------------------------- Eq. 6
def sparse_attention(q, k_chunks, v_chunks, b: int, mask: np.ndarray, q_blocks=None) -> np.ndarray:
    """O_local by definition: every query row attends, with a softmax over q.k/sqrt(d), to exactly
    the key tokens of the key blocks its query block keeps (Eq. 6).

    q [T_c, d]; k_chunks / v_chunks: lists of [n_c, d] (oldest chunk first, current chunk last);
    mask [T_m, T_n] over the logical key blocks.  q_blocks: optional subset of query blocks to
    compute (other rows are returned as NaN)."""
    q = np.asarray(q, np.float64)
    d = q.shape[1]
    table = key_block_table([kc.shape[0] for kc in k_chunks], b)
    out = np.full(q.shape[:1] + (v_chunks[0].shape[1],), np.nan)
    for i, (qs, qe) in enumerate(block_ranges(q.shape[0], b)):
        if q_blocks is not None and i not in q_blocks:
            continue
        kept = [table[j] for j in range(len(table)) if mask[i, j]]
        ks = np.concatenate([np.asarray(k_chunks[c][s:e], np.float64) for (c, s, e) in kept])
        vs = np.concatenate([np.asarray(v_chunks[c][s:e], np.float64) for (c, s, e) in kept])
        s_ = q[qs:qe] @ ks.T / math.sqrt(d)
        s_ = s_ - s_.max(axis=1, keepdims=True)
        p = np.exp(s_)
        out[qs:qe] = (p @ vs) / p.sum(axis=1, keepdims=True)
    return out


def sparse_attention_blockwise(q, k_chunks, v_chunks, b: int, mask: np.ndarray) -> np.ndarray:
    """O_local a second way, as a witness for sparse_attention: every kept key block on its own first -- its softmax-weighted
    average of V rows and the log of its sum of exponentials -- then the blocks of a row combined with the weights
    exp(lse_block - lse_row).  This is the identity that lets Alg. 3 walk the kept blocks one tile at a time (a softmax
    over a union of blocks is the lse-weighted mixture of the per-block softmaxes); nothing is carried from block to block."""
    q = np.asarray(q, np.float64)
    d = q.shape[1]
    table = key_block_table([kc.shape[0] for kc in k_chunks], b)
    out = np.zeros((q.shape[0], v_chunks[0].shape[1]))
    for i, (qs, qe) in enumerate(block_ranges(q.shape[0], b)):
        qi = q[qs:qe]
        block_out, block_lse = [], []
        for j, (c, s, e) in enumerate(table):
            if not mask[i, j]:
                continue
            logits = qi @ np.asarray(k_chunks[c][s:e], np.float64).T / math.sqrt(d)
            top = logits.max(axis=1, keepdims=True)
            w = np.exp(logits - top)
            block_out.append((w @ np.asarray(v_chunks[c][s:e], np.float64)) / w.sum(axis=1, keepdims=True))
            block_lse.append(top[:, 0] + np.log(w.sum(axis=1)))
        lse = np.stack(block_lse)                               # [kept, rows]
        row_lse = lse.max(axis=0) + np.log(np.exp(lse - lse.max(axis=0)).sum(axis=0))
        share = np.exp(lse - row_lse)                           # sums to one over the kept blocks
        out[qs:qe] = sum(share[n][:, None] * block_out[n] for n in range(len(block_out)))
    return out


# --------------------------------------------------------------------------- Eq. 3 / Eq. 4
def absorb(S: np.ndarray, z: np.ndarray, k_ev, v_ev):
    """Fold evicted tokens into the state (Eq. 3): S += phi(K_ev)^T V_ev (rows: key feature, columns: value
    dim), z += sum over tokens of phi(K_ev)."""
    f = phi(k_ev)
    return S + f.T @ np.asarray(v_ev, np.float64), z + f.sum(axis=0)


def absorb_frame_mean(S: np.ndarray, z: np.ndarray, k_ev, v_ev, frame_tokens: int):
    """Eq. 3 read literally for H: S as in absorb(); z += sum over the evicted latent frames of the MEAN over that
    frame's tokens of phi(K) (the paper prints "mean" inside the sum).  k_ev must hold whole frames."""
    f = phi(k_ev)
    n = f.shape[0]
    assert n % frame_tokens == 0, "evicted tokens must be whole frames"
    zinc = np.zeros_like(z)
    for fr in range(n // frame_tokens):
        zinc = zinc + f[fr * frame_tokens:(fr + 1) * frame_tokens].mean(axis=0)
    return S + f.T @ np.asarray(v_ev, np.float64), z + zinc


def rotate_pairs(x, cos, sin) -> np.ndarray:
    """RoPE on feature pairs (2i, 2i+1): x [T, d], cos / sin [T, d/2] (one angle per token and pair).
    out[2i] = x[2i] cos_i - x[2i+1] sin_i,  out[2i+1] = x[2i] sin_i + x[2i+1] cos_i."""
    x = np.asarray(x, np.float64); cos = np.asarray(cos, np.float64); sin = np.asarray(sin, np.float64)
    out = np.empty_like(x)
    out[:, 0::2] = x[:, 0::2] * cos - x[:, 1::2] * sin
    out[:, 1::2] = x[:, 0::2] * sin + x[:, 1::2] * cos
    return out


def absorb_rope(S: np.ndarray, z: np.ndarray, k_ev, v_ev, cos_k, sin_k, frame_tokens=None):
    """Eq. 3 with its rotation: S += RoPE(phi(K_ev))^T V_ev; the normaliser keeps the unrotated phi(K_ev)
    (sum over tokens, or per-frame means when frame_tokens is given)."""
    f = phi(k_ev)
    S = S + rotate_pairs(f, cos_k, sin_k).T @ np.asarray(v_ev, np.float64)
    if frame_tokens is None:
        return S, z + f.sum(axis=0)
    _, z2 = absorb_frame_mean(np.zeros_like(S), z, k_ev, np.zeros_like(np.asarray(v_ev, np.float64)), frame_tokens)
    return S, z2


def relative_temporal_indices(i: int, t0: int):
    """Eq. 8: temporal RoPE indices of the three frames of the chunk that ends at (1-based) frame i, capped at the
    largest index T_0 the pretrained model has seen."""
    return [i - 2, i - 1, i] if i <= t0 else [t0 - 2, t0 - 1, t0]


def window_temporal_indices(cur_last_frame: int, chunk_last_frames, t0: int, chunk_frames: int):
    """Sec. 3.3 ("the temporal RoPE indices in the KV cache are updated based on the offsets to the current chunk"):
    the current chunk, whose last frame is the stream's (1-based) frame cur_last_frame, takes Eq. 8's indices; a cached
    chunk whose last frame was frame f keeps its distance to it: its last frame has index top - (cur_last_frame - f),
    top = min(cur_last_frame, T_0).  Returns (indices of the current chunk's frames, [indices per cached chunk])."""
    cur = relative_temporal_indices(cur_last_frame, t0) if chunk_frames == 3 else \
        [min(cur_last_frame, t0) - chunk_frames + 1 + i for i in range(chunk_frames)]
    top = cur[-1]
    cached = [[top - (cur_last_frame - f) - chunk_frames + 1 + i for i in range(chunk_frames)] for f in chunk_last_frames]
    return cur, cached


def temporal_tables(frame_indices, tokens_per_frame: int, d: int, first_pair: int, omegas):
    """cos / sin tables [T, d/2] of a chunk for rotate_pairs: pair first_pair + n turns by index * omegas[n], where index
    is the temporal index of the token's frame; every other pair is left alone (their rotation, by the spatial
    coordinates, is the caller's and does not change while a key sits in the cache)."""
    omegas = np.asarray(omegas, np.float64)
    idx = np.repeat(np.asarray(frame_indices, np.float64), tokens_per_frame)
    cos = np.ones((idx.shape[0], d // 2)); sin = np.zeros((idx.shape[0], d // 2))
    ang = idx[:, None] * omegas[None, :]
    cos[:, first_pair:first_pair + omegas.shape[0]] = np.cos(ang)
    sin[:, first_pair:first_pair + omegas.shape[0]] = np.sin(ang)
    return cos, sin


def rotate_temporal(x, frame_indices, tokens_per_frame: int, first_pair: int, omegas) -> np.ndarray:
    """Temporal RoPE of the softmax branch: x [T, d] (T = frames * tokens_per_frame), one index per frame."""
    cos, sin = temporal_tables(frame_indices, tokens_per_frame, np.asarray(x).shape[1], first_pair, omegas)
    return rotate_pairs(x, cos, sin)


def bf16_round_f32(x: np.ndarray) -> np.ndarray:
    """float32 -> nearest bf16 (ties to even) -> float32; finite input."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def rotate_temporal_f32(x: np.ndarray, frame_steps, tokens_per_frame: int, first_pair: int, cos_tab: np.ndarray,
                        sin_tab: np.ndarray) -> np.ndarray:
    """The rotation as the cache stores it (part of the bit-exact selection contract, like the float32 scorer): x float32
    [T, d] holding bf16 values; frame f turns by frame_steps[f] index steps (negative: backwards), the angle's cosine and
    sine taken from the float32 tables cos_tab / sin_tab [steps, pairs] at |steps| (sine negated for a backward turn);
    x0' = x0 c - x1 s and x1' = x0 s + x1 c with every product and the sum rounded separately in float32; the result
    rounded to bf16.  Pairs outside [first_pair, first_pair + pairs) pass through."""
    x = np.asarray(x)
    assert x.dtype == np.float32
    out = x.copy()
    n = cos_tab.shape[1]
    steps = np.repeat(np.asarray(frame_steps, np.int64), tokens_per_frame)
    c = cos_tab[np.abs(steps)].astype(F32)
    s_ = (sin_tab[np.abs(steps)] * np.where(steps < 0, F32(-1.0), F32(1.0))[:, None]).astype(F32)
    x0 = x[:, 2 * first_pair:2 * (first_pair + n):2]; x1 = x[:, 2 * first_pair + 1:2 * (first_pair + n):2]
    y0 = (x0 * c).astype(F32) - (x1 * s_).astype(F32)
    y1 = (x0 * s_).astype(F32) + (x1 * c).astype(F32)
    out[:, 2 * first_pair:2 * (first_pair + n):2] = bf16_round_f32(y0.astype(F32))
    out[:, 2 * first_pair + 1:2 * (first_pair + n):2] = bf16_round_f32(y1.astype(F32))
    return out


def linear_readout(q, S, z, W=None, bias=None, eps: float = 1e-6, cos_q=None, sin_q=None) -> np.ndarray:
    """O_history (Eq. 4): h = phi(q) S / (phi(q) . z + eps) per query row, then Linear: y = W h + bias.
    With cos_q / sin_q [T, d/2] the numerator uses RoPE(phi(q)) (Eq. 4 as printed); the denominator never rotates."""
    f = phi(q)
    fn = f if cos_q is None else rotate_pairs(f, cos_q, sin_q)      # Eq. 4: rotation in the numerator only
    h = (fn @ S) / (f @ z + eps)[:, None]
    if W is not None:
        h = h @ np.asarray(W, np.float64).T
    if bias is not None:
        h = h + np.asarray(bias, np.float64)[None, :]
    return h


def merge_full_width(h: np.ndarray, W_full, bias_full=None) -> np.ndarray:
    """Eq. 4's "Linear" read as ONE projection over the model width (the paper gives no shape; the per-head reading is the
    default): h [H, T, d] of one batch element, per token x = concat_h h[h, t, :] (head-major), y = W_full x + bias_full,
    W_full [H d, H d] (row = output feature), split back into heads.  Returns [H, T, d]."""
    H, T, d = h.shape
    x = np.transpose(np.asarray(h, np.float64), (1, 0, 2)).reshape(T, H * d)
    y = x @ np.asarray(W_full, np.float64).T
    if bias_full is not None:
        y = y + np.asarray(bias_full, np.float64)[None, :]
    return np.transpose(y.reshape(T, H, d), (1, 0, 2))


# --------------------------------------------------------------------------- gradients (Alg. 1: rollout step with gradient)
def phi_prime(x: np.ndarray) -> np.ndarray:
    """d/dx (elu(x) + 1): 1 for x > 0, exp(x) otherwise."""
    x = np.asarray(x, dtype=np.float64)
    return np.where(x > 0.0, 1.0, np.exp(np.minimum(x, 0.0)))


def sparse_attention_backward(q, k_chunks, v_chunks, b: int, mask: np.ndarray, d_out):
    """Gradients of O_local (Eq. 6) for a fixed block mask: given dL/dO_local [T_c, d] returns
    (dq [T_c, d], [dk per chunk], [dv per chunk]).  Per query block, with p = softmax(s) over the kept keys and
    s = q k^T / sqrt(d):  dv = p^T dO;  dp = dO v^T;  ds = p * (dp - rowsum(dp * p))  (Jacobian of the row softmax);
    dq = ds k / sqrt(d);  dk = ds^T q / sqrt(d).  Keys outside the kept blocks get no gradient from that query block."""
    q = np.asarray(q, np.float64); d_out = np.asarray(d_out, np.float64)
    d = q.shape[1]
    table = key_block_table([kc.shape[0] for kc in k_chunks], b)
    dq = np.zeros_like(q)
    dk = [np.zeros(np.asarray(kc).shape) for kc in k_chunks]
    dv = [np.zeros(np.asarray(vc).shape) for vc in v_chunks]
    for i, (qs, qe) in enumerate(block_ranges(q.shape[0], b)):
        kept = [table[j] for j in range(len(table)) if mask[i, j]]
        ks = np.concatenate([np.asarray(k_chunks[c][s:e], np.float64) for (c, s, e) in kept])
        vs = np.concatenate([np.asarray(v_chunks[c][s:e], np.float64) for (c, s, e) in kept])
        s_ = q[qs:qe] @ ks.T / math.sqrt(d)
        p = np.exp(s_ - s_.max(axis=1, keepdims=True))
        p = p / p.sum(axis=1, keepdims=True)
        g = d_out[qs:qe]
        dvs = p.T @ g
        dp = g @ vs.T
        ds = p * (dp - (dp * p).sum(axis=1, keepdims=True))
        dq[qs:qe] = ds @ ks / math.sqrt(d)
        dks = ds.T @ q[qs:qe] / math.sqrt(d)
        at = 0
        for (c, s, e) in kept:
            dk[c][s:e] += dks[at:at + e - s]
            dv[c][s:e] += dvs[at:at + e - s]
            at += e - s
    return dq, dk, dv


def linear_readout_backward(q, S, z, d_out, W=None, eps: float = 1e-6):
    """Gradients of O_history (Eq. 4, no rotation) given dL/dO_history [T, d]: returns (dq, dS, dz, dW, dbias).
    Forward: f = phi(q); num = f S; den = f . z + eps; h = num / den; y = W h + bias."""
    q = np.asarray(q, np.float64); g = np.asarray(d_out, np.float64)
    f = phi(q)
    num = f @ S
    den = f @ z + eps
    h = num / den[:, None]
    dbias = g.sum(axis=0)
    if W is not None:
        W = np.asarray(W, np.float64)
        dW = g.T @ h                    # y = h W^T
        dh = g @ W
    else:
        dW = None
        dh = g
    dnum = dh / den[:, None]
    dden = -(dh * num).sum(axis=1) / den ** 2
    df = dnum @ S.T + dden[:, None] * z[None, :]
    dS = f.T @ dnum
    dz = f.T @ dden
    return df * phi_prime(q), dS, dz, dW, dbias


# --------------------------------------------------------------------------- Alg. 2 + Alg. 3
class HybridStream:
    """Streaming state of one layer (all batches and heads) and the per-chunk forward.

    Alg. 2: the rolling cache holds the clean K/V of the last P = w/c - 1 chunks; a committed clean chunk
    is appended and whatever then exceeds P chunks is popped from the front and folded into (S, z) --
    the state is updated before the evicted K/V are dropped.  With P >= 1 this is the paper's
    "if full: pop(0), update state; append"; with P = 0 a committed chunk goes straight into the state.
    Sink (Eq. 1's first-frame term): the first sink_chunks committed chunks are kept outside that rotation, as the
    oldest logical key blocks of every later window; they are never evicted and never folded into the state.
    """

    def __init__(self, batch, heads, d, b, past_chunks, topk=0, keep_permille=0,
                 W=None, bias=None, eps=1e-6, z_frame_tokens=None, sink_chunks=0, rope_q=None, rope_k=None,
                 W_full=None, bias_full=None, temporal=None):
        self.B, self.H, self.d, self.b, self.P = batch, heads, d, b, past_chunks
        self.z_frame_tokens = z_frame_tokens     # None: z is the plain sum of phi(K); n: per-frame means of n tokens (Eq. 3 literal)
        self.topk, self.keep_permille, self.eps = topk, keep_permille, eps
        self.W = None if W is None else np.asarray(W, np.float64)        # [H, d, d]
        self.bias = None if bias is None else np.asarray(bias, np.float64)  # [H, d]
        # the full-width reading of "Linear" (one [H d, H d] matrix over all heads) replaces the per-head one
        self.W_full = None if W_full is None else np.asarray(W_full, np.float64)
        self.bias_full = None if bias_full is None else np.asarray(bias_full, np.float64)
        assert self.W_full is None or self.W is None
        self.rope_q, self.rope_k = rope_q, rope_k    # (cos, sin) tables [T_c, d/2] of the linear branch, or None
        self.sink_chunks = sink_chunks   # the first chunks of the stream stay visible for ever ("sink"): never evicted, never absorbed
        self.sink = []                                                   # list of (k, v) like self.past, oldest first
        self.past = []                                                   # list of (k [B,H,n,d], v) fp64
        self.S = np.zeros((batch, heads, d, d))
        self.z = np.zeros((batch, heads, d))
        self.absorbed_tokens = 0
        # Relative temporal RoPE of the softmax branch (Sec. 3.3, Eq. 8), or None.  dict(t0, first_pair, cos_tab, sin_tab
        # [steps, pairs] float32, tokens_per_frame, chunk_frames).  q, k then arrive WITHOUT temporal rotation.  The cache is a
        # bf16 store: a key enters it rotated to the index it will have while the NEXT chunk is generated, and is turned
        # further (and rounded to bf16 again) whenever the cap of Eq. 8 makes the window's indices slide; the queries and the
        # current chunk's keys are rotated to Eq. 8's indices and rounded to bf16 as well (they are the attention kernel's
        # bf16 operands).  All of it in the canonical float32 order (rotate_temporal_f32), because these values decide the
        # block selection.  Sink chunks keep the indices they had when they were generated.
        self.temporal = temporal
        self.frames_committed = 0

    # -- Alg. 2, cache commit
    def _turn(self, x, frame_steps):
        """x [B, H, T, d] -> rotated by frame_steps (one entry per frame) in the canonical order, as fp64 of bf16 values."""
        t = self.temporal
        out = np.empty(np.asarray(x).shape)
        for bi in range(self.B):
            for h in range(self.H):
                out[bi, h] = rotate_temporal_f32(np.asarray(x[bi, h], np.float64).astype(F32), frame_steps, t["tokens_per_frame"],
                                                 t["first_pair"], t["cos_tab"], t["sin_tab"])
        return out

    def current_indices(self):
        """Eq. 8 for the chunk being generated now."""
        t = self.temporal
        c = t["chunk_frames"]
        top = min(self.frames_committed + c, t["t0"])
        return [top - c + 1 + i for i in range(c)]

    def rotated_inputs(self, q, k_cur):
        """(q, k_cur) as the attention sees them: unchanged without temporal rotation, else turned to Eq. 8's indices."""
        if self.temporal is None:
            return q, k_cur
        idx = self.current_indices()
        return self._turn(q, idx), self._turn(k_cur, idx)

    def append(self, k_clean, v_clean):
        k_clean = np.asarray(k_clean, np.float64)
        if self.temporal is not None:
            t = self.temporal
            c, t0 = t["chunk_frames"], t["t0"]
            last = self.frames_committed + c                    # (1-based) number of this chunk's last frame
            top_now, top_next = min(last, t0), min(last + c, t0)
            self.frames_committed = last
            if len(self.sink) < self.sink_chunks or self.P == 0:
                # a sink chunk keeps its own indices for good; without a cache (window = one chunk) the chunk goes straight
                # into the state, as the window last saw it: at its own indices
                k_clean = self._turn(k_clean, [top_now - c + 1 + i for i in range(c)])
            else:
                # indices during the next chunk: this chunk sits c frames behind it; older chunks slide by the same amount
                k_clean = self._turn(k_clean, [top_next - 2 * c + 1 + i for i in range(c)])
                slide = top_next - top_now - c                  # 0 until the cap is reached, then -c
                if slide != 0:
                    # all but the chunk that is about to leave (it is folded into the state as the window last saw it)
                    keep_from = 1 if len(self.past) >= self.P else 0
                    for n in range(keep_from, len(self.past)):
                        self.past[n] = (self._turn(self.past[n][0], [slide] * c), self.past[n][1])
        if len(self.sink) < self.sink_chunks:
            self.sink.append((k_clean, np.asarray(v_clean, np.float64)))
            return
        self.past.append((k_clean, np.asarray(v_clean, np.float64)))
        while len(self.past) > self.P:
            k_ev, v_ev = self.past.pop(0)
            for bi in range(self.B):
                for h in range(self.H):
                    if self.rope_k is not None:
                        self.S[bi, h], self.z[bi, h] = absorb_rope(self.S[bi, h], self.z[bi, h], k_ev[bi, h], v_ev[bi, h],
                                                                   self.rope_k[0], self.rope_k[1], self.z_frame_tokens)
                    elif self.z_frame_tokens is None:
                        self.S[bi, h], self.z[bi, h] = absorb(self.S[bi, h], self.z[bi, h], k_ev[bi, h], v_ev[bi, h])
                    else:
                        self.S[bi, h], self.z[bi, h] = absorb_frame_mean(self.S[bi, h], self.z[bi, h], k_ev[bi, h],
                                                                         v_ev[bi, h], self.z_frame_tokens)
            self.absorbed_tokens += k_ev.shape[2]

    # -- Eq. 5 + top-K
    def n_key_blocks(self, n_cur: int) -> int:
        return sum(-(-kp.shape[2] // self.b) for kp, _ in self.sink + self.past) + -(-n_cur // self.b)

    def select(self, q, k_cur, exact: bool = False):
        """Masks [B, H, T_m, T_n].  exact=False: canonical float32 scores (the bit-exact contract);
        exact=True: fp64 scores (the ideal the canonical order approximates)."""
        B, H = self.B, self.H
        q, k_cur = self.rotated_inputs(q, k_cur)
        n_kb = self.n_key_blocks(k_cur.shape[2])
        k = keep_count(self.topk, self.keep_permille, n_kb)
        masks, scores = [], []
        for bi in range(B):
            for h in range(H):
                if exact:
                    qm = block_means(q[bi, h], self.b)
                    km = np.concatenate([block_means(kp[bi, h], self.b) for kp, _ in self.sink + self.past]
                                        + [block_means(k_cur[bi, h], self.b)])
                    a = block_scores(qm, km)
                else:
                    as32 = lambda x: np.asarray(x, np.float64).astype(F32)   # exact: values are bf16
                    qm = block_means_f32(as32(q[bi, h]), self.b)
                    km = np.concatenate([block_means_f32(as32(kp[bi, h]), self.b) for kp, _ in self.sink + self.past]
                                        + [block_means_f32(as32(k_cur[bi, h]), self.b)])
                    a = block_scores_f32(qm, km)
                scores.append(a)
                masks.append(select_blocks(a, k))
        shape = (B, H) + masks[0].shape
        return np.stack(masks).reshape(shape), np.stack(scores).reshape(shape)

    # -- Alg. 3 + Eq. 7
    def forward(self, q, k_cur, v_cur, mask=None, q_blocks=None, parts: bool = False):
        """O = O_local + O_history for the current chunk's queries against past chunks + the current chunk.
        mask: [B,H,T_m,T_n] (default: the canonical selection)."""
        q = np.asarray(q, np.float64); k_cur = np.asarray(k_cur, np.float64); v_cur = np.asarray(v_cur, np.float64)
        if mask is None:
            mask, _ = self.select(q, k_cur)
        q, k_cur = self.rotated_inputs(q, k_cur)        # (both branches see the queries with their temporal rotation)
        o_loc = np.empty_like(q); o_hist = np.empty_like(q)
        for bi in range(self.B):
            for h in range(self.H):
                kc = [kp[bi, h] for kp, _ in self.sink + self.past] + [k_cur[bi, h]]
                vc = [vp[bi, h] for _, vp in self.sink + self.past] + [v_cur[bi, h]]
                o_loc[bi, h] = sparse_attention(q[bi, h], kc, vc, self.b, mask[bi, h], q_blocks)
                o_hist[bi, h] = linear_readout(q[bi, h], self.S[bi, h], self.z[bi, h],
                                               None if self.W is None else self.W[h],
                                               None if self.bias is None else self.bias[h], self.eps,
                                               None if self.rope_q is None else self.rope_q[0],
                                               None if self.rope_q is None else self.rope_q[1])
            if self.W_full is not None:     # o_hist holds h = num / den so far (W, bias are None): project over all heads
                o_hist[bi] = merge_full_width(o_hist[bi], self.W_full, self.bias_full)
        if parts:
            return o_loc + o_hist, o_loc, o_hist
        return o_loc + o_hist

    # -- gradients of the forward above (Eq. 7: both branches receive dL/dO unchanged)
    def backward(self, q, k_cur, v_cur, d_out, mask=None):
        """dL/dO [B, H, T_c, d] -> dict(dq, dk_cur, dv_cur, dk_past, dv_past (lists per cached chunk, sink first), dS, dz,
        dW, dbias) for the per-head reading of "Linear", without rotation.  The block mask is held fixed."""
        assert self.temporal is None and self.rope_q is None and self.W_full is None
        q = np.asarray(q, np.float64); k_cur = np.asarray(k_cur, np.float64); v_cur = np.asarray(v_cur, np.float64)
        g = np.asarray(d_out, np.float64)
        if mask is None:
            mask, _ = self.select(q, k_cur)
        held = self.sink + self.past
        out = dict(dq=np.zeros_like(q), dk_cur=np.zeros_like(k_cur), dv_cur=np.zeros_like(v_cur),
                   dk_past=[np.zeros_like(kp) for kp, _ in held], dv_past=[np.zeros_like(vp) for _, vp in held],
                   dS=np.zeros_like(self.S), dz=np.zeros_like(self.z),
                   dW=None if self.W is None else np.zeros_like(self.W), dbias=np.zeros((self.H, self.d)))
        for bi in range(self.B):
            for h in range(self.H):
                kc = [kp[bi, h] for kp, _ in held] + [k_cur[bi, h]]
                vc = [vp[bi, h] for _, vp in held] + [v_cur[bi, h]]
                dq_l, dk_l, dv_l = sparse_attention_backward(q[bi, h], kc, vc, self.b, mask[bi, h], g[bi, h])
                dq_h, dS, dz, dW, db = linear_readout_backward(q[bi, h], self.S[bi, h], self.z[bi, h], g[bi, h],
                                                               None if self.W is None else self.W[h], self.eps)
                out["dq"][bi, h] = dq_l + dq_h
                out["dk_cur"][bi, h] = dk_l[-1]; out["dv_cur"][bi, h] = dv_l[-1]
                for n in range(len(held)):
                    out["dk_past"][n][bi, h] = dk_l[n]; out["dv_past"][n][bi, h] = dv_l[n]
                out["dS"][bi, h] = dS; out["dz"][bi, h] = dz
                out["dbias"][h] += db
                if dW is not None:
                    out["dW"][h] += dW
        return out
