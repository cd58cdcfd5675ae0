"""Seeded synthetic inputs and workload shapes.

This module serves both the CUDA path's tests/bench and the CPU oracle's tests.
It holds none of the method's arithmetic: only random draws, the bf16 bit
conversion of those draws, and the named workload shapes.

All tensors are handed around as ``numpy.uint16`` arrays holding bf16 bit
patterns ("bits"), so that the bytes the GPU sees and the bytes the oracle reads
are the same bytes.  Shapes are ``[B, H, T, d]`` (batch, heads, tokens, head dim).

Workloads: the paper measures on a trained Wan2.1-T2V-1.3B at 832x480
(Sec. 4.1); no weights or prompts exist here, so i.i.d. N(0,1) tensors of that
model's attention shapes stand in for it.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
import numpy as np

# tensor ids used in seeds
T_Q, T_K, T_V, T_KCLEAN, T_VCLEAN, T_W, T_BIAS, T_ANGLE_Q, T_ANGLE_K, T_DIR = range(10)


@dataclass(frozen=True)
class Workload:
    """Shape of one hybrid-attention layer stream (names follow Alg. 2 / Alg. 3)."""
    name: str
    batch: int
    heads: int
    head_dim: int            # d
    tokens_per_frame: int    # tokens in one latent frame
    chunk_frames: int        # latent frames per chunk
    window_frames: int       # sliding window w, counts the current chunk
    block: int               # b_q = b_kv
    topk: int                # >0: keep exactly this many key blocks per query block
    keep_permille: int       # used when topk == 0: k = ceil(permille * T_n_valid / 1000)
    layers: int = 1
    steps: int = 1           # denoising steps per chunk
    chunks: int = 1          # chunks streamed
    seed: int = 0
    eps: float = 1e-6

    @property
    def chunk_tokens(self) -> int:
        return self.tokens_per_frame * self.chunk_frames

    @property
    def past_chunks(self) -> int:
        """P: clean chunks the rolling cache holds besides the current chunk."""
        return self.window_frames // self.chunk_frames - 1

    @property
    def blocks_per_chunk(self) -> int:
        return -(-self.chunk_tokens // self.block)

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


def tiny() -> Workload:
    """Small case: 8x8 tokens per frame, 1-frame chunks, window 3, 16-token blocks, top-2."""
    return Workload("tiny", batch=1, heads=2, head_dim=64, tokens_per_frame=64, chunk_frames=1,
                    window_frames=3, block=16, topk=2, keep_permille=0, chunks=6, seed=1)


def layer_832x480() -> Workload:
    """One layer at the 832x480 latent shape: 1560 tokens/frame, 12 heads of 128."""
    return Workload("layer_832x480", batch=1, heads=12, head_dim=128, tokens_per_frame=1560,
                    chunk_frames=3, window_frames=9, block=128, topk=0, keep_permille=250,
                    chunks=5, seed=2)


def stream_832x480(chunks: int = 200) -> Workload:
    return layer_832x480().with_(name="stream_832x480", chunks=chunks, seed=3)


def full_depth_832x480(layers: int = 30, steps: int = 4, chunks: int = 20) -> Workload:
    return layer_832x480().with_(name="full_depth_832x480", layers=layers, steps=steps,
                                 chunks=chunks, seed=4)


def sweep_points():
    """The sweep grid: kept ratio x window x head_dim x block x batch."""
    pts = []
    for permille in (100, 250, 500, 1000):
        for window in (3, 9, 21):
            for d in (64, 128):
                for blk in (64, 128):
                    for batch in (1, 4):
                        pts.append(layer_832x480().with_(
                            name=f"sweep_k{permille}_w{window}_d{d}_b{blk}_B{batch}",
                            keep_permille=permille, window_frames=window, head_dim=d,
                            block=blk, batch=batch, seed=5))
    return pts


# ---------------------------------------------------------------------------
# bf16 bit conversion (format conversion only)
# ---------------------------------------------------------------------------

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round to nearest, ties to even); returns uint16 bits. Finite input."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(bits).astype(np.float64)


# ---------------------------------------------------------------------------
# seeded draws
# ---------------------------------------------------------------------------

def _rng(*key: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(np.random.SeedSequence([int(k) & 0xFFFFFFFF for k in key])))


def normal_bf16(shape, *key: int, scale: float = 1.0) -> np.ndarray:
    """N(0, scale^2) drawn in float32 and rounded to bf16; uint16 bits of ``shape``."""
    x = _rng(*key).standard_normal(size=shape, dtype=np.float32)
    if scale != 1.0:
        x = x * np.float32(scale)
    return f32_to_bf16_bits(x)


def qkv(w: Workload, layer: int, chunk: int, step: int):
    """(q, k, v) bits of one denoising step: each [B, H, T_c, d]."""
    shape = (w.batch, w.heads, w.chunk_tokens, w.head_dim)
    return tuple(normal_bf16(shape, w.seed, layer, chunk, step, t) for t in (T_Q, T_K, T_V))


def clean_kv(w: Workload, layer: int, chunk: int):
    """(k, v) bits of the clean (t = 0) pass whose K/V enter the rolling cache (Alg. 2)."""
    shape = (w.batch, w.heads, w.chunk_tokens, w.head_dim)
    return tuple(normal_bf16(shape, w.seed, layer, chunk, 0xC1EA, t) for t in (T_KCLEAN, T_VCLEAN))


def merge_weights(w: Workload, layer: int, with_bias: bool = True):
    """Random-init output projection of the history branch: W [H, d, d] ~ N(0, 1/d), bias [H, d] ~ N(0, 0.01)."""
    d = w.head_dim
    W = normal_bf16((w.heads, d, d), w.seed, layer, 0, 0, T_W, scale=d ** -0.5)
    b = normal_bf16((w.heads, d), w.seed, layer, 0, 0, T_BIAS, scale=0.1) if with_bias else None
    return W, b


def merge_weights_full(w: Workload, layer: int, with_bias: bool = True):
    """Random-init projection over the model width (the one-matrix reading of the history branch's Linear):
    W [H d, H d] ~ N(0, 1/(H d)), bias [H d] ~ N(0, 0.01)."""
    hd = w.heads * w.head_dim
    W = normal_bf16((hd, hd), w.seed, layer, 0, 1, T_W, scale=hd ** -0.5)
    b = normal_bf16((hd,), w.seed, layer, 0, 1, T_BIAS, scale=0.1) if with_bias else None
    return W, b


def rotation_tables(w: Workload, which: int):
    """(cos, sin) float32 tables [T_c, d/2] of seeded angles ~ U(0, 2 pi): stand-ins for the position angles a model
    would supply to the linear branch's rotation.  `which`: T_ANGLE_Q or T_ANGLE_K."""
    th = _rng(w.seed, 0, 0, 0, which).uniform(0.0, 2.0 * np.pi, size=(w.chunk_tokens, w.head_dim // 2))
    return np.cos(th).astype(np.float32), np.sin(th).astype(np.float32)


# ---------------------------------------------------------------------------
# structured draws: peaked attention rows (trained attention maps are concentrated; i.i.d. N(0,1) gives flat ones)
# ---------------------------------------------------------------------------

def direction(w: Workload, layer: int) -> np.ndarray:
    """One seeded N(0,1) vector per head, float32 [H, d]: queries and chosen key blocks are shifted along it, which
    moves the logits of those blocks by (q shift) * (k shift) * |u|^2 / sqrt(d) ~ (q shift) * (k shift) * sqrt(d)."""
    return _rng(w.seed, layer, 0, 0, T_DIR).standard_normal(size=(w.heads, w.head_dim), dtype=np.float32)


def shifted(bits: np.ndarray, u: np.ndarray, amount: float, tokens: slice = slice(None), scale: float = 1.0) -> np.ndarray:
    """bits [B, H, T, d] -> bf16 bits of (scale * x + amount * u[h]) on the token range `tokens`, x elsewhere."""
    x = bf16_bits_to_f32(bits).copy()
    x[:, :, tokens, :] = x[:, :, tokens, :] * np.float32(scale) + np.float32(amount) * u[None, :, None, :]
    return f32_to_bf16_bits(x)


def temporal_rope_tables(head_dim: int, t0: int, first_pair: int = 0, pairs: int | None = None, base: float = 10000.0):
    """Angle tables of the temporal rotary axis for integer index steps 0 .. t0: float32 (cos, sin) [t0 + 1, pairs] with the
    usual rotary frequencies base ** (-n / pairs), plus the frequencies themselves (float64).  `pairs` defaults to the
    share of the head's d/2 pairs that a (t, y, x) split gives the temporal axis (d/2 - 2 * (d/6))."""
    if pairs is None:
        pairs = head_dim // 2 - 2 * (head_dim // 6)
    om = base ** (-np.arange(pairs, dtype=np.float64) / pairs)
    n = np.arange(t0 + 1, dtype=np.float64)
    return np.cos(n[:, None] * om[None, :]).astype(np.float32), np.sin(n[:, None] * om[None, :]).astype(np.float32), om
