"""Test harness: drive the CUDA library and the CPU oracle over the same seeded stream and compare."""
from __future__ import annotations

import numpy as np

from oracle import hybrid_attention as oa
from paper_2604_10103_b200 import inputs as gen

# tolerances of the hot path (bf16 in, fp32 accumulate, bf16 out) against the fp64 oracle
MAX_ABS = 2e-2
REL_L2 = 5e-3
STATE_REL_L2 = 1e-4


def rel_l2(a, b):
    a = np.asarray(a, np.float64); b = np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def max_abs(a, b):
    return float(np.abs(np.asarray(a, np.float64) - np.asarray(b, np.float64)).max())


def temporal_setup(w: gen.Workload, t0: int, first_pair: int = 0, pairs=None):
    """The tables both sides get for the relative temporal RoPE (Eq. 8): (dict for the oracle, (cos, sin) float32)."""
    cos, sin, _ = gen.temporal_rope_tables(w.head_dim, t0, first_pair, pairs)
    return dict(t0=t0, first_pair=first_pair, cos_tab=cos, sin_tab=sin, tokens_per_frame=w.tokens_per_frame,
                chunk_frames=w.chunk_frames), (cos, sin)


def make_oracle(w: gen.Workload, layer: int = 0, merge: bool = True, bias: bool = True, z_frame_mean: bool = False,
                sink_chunks: int = 0, rope: bool = False, merge_full: bool = False, temporal=None):
    W = b = Wf = bf = None
    if merge_full:
        Wb, bb = gen.merge_weights_full(w, layer, with_bias=bias)
        Wf = gen.bf16_bits_to_f64(Wb)
        bf = None if bb is None else gen.bf16_bits_to_f64(bb)
    elif merge:
        Wb, bb = gen.merge_weights(w, layer, with_bias=bias)
        W = gen.bf16_bits_to_f64(Wb)
        b = None if bb is None else gen.bf16_bits_to_f64(bb)
    return oa.HybridStream(w.batch, w.heads, w.head_dim, w.block, w.past_chunks, topk=w.topk,
                           keep_permille=w.keep_permille, W=W, bias=b, eps=w.eps,
                           z_frame_tokens=w.tokens_per_frame if z_frame_mean else None, sink_chunks=sink_chunks,
                           rope_q=gen.rotation_tables(w, gen.T_ANGLE_Q) if rope else None,
                           rope_k=gen.rotation_tables(w, gen.T_ANGLE_K) if rope else None, W_full=Wf, bias_full=bf,
                           temporal=None if temporal is None else temporal_setup(w, *temporal)[0])


from paper_2604_10103_b200.binding import unpack_mask  # noqa: E402,F401


class GpuStream:
    """The library side of a one-layer stream (torch only for memory)."""

    def __init__(self, w: gen.Workload, layer: int = 0, merge: bool = True, bias: bool = True, swa_kernel: int = 0,
                 layers: int | None = None, z_frame_mean: bool = False, sink_chunks: int = 0, rope: bool = False,
                 merge_full: bool = False, temporal=None):
        import torch
        from paper_2604_10103_b200 import binding as hf
        self.torch, self.hf, self.w, self.layer = torch, hf, w, layer
        cfg = hf.make_config(w.with_(layers=layers or max(w.layers, layer + 1)),
                             merge=hf.HF_MERGE_FULL_WIDTH if merge_full else hf.HF_MERGE_PER_HEAD if merge else hf.HF_MERGE_IDENTITY,
                             swa_kernel=swa_kernel,
                             z_mode=hf.HF_Z_FRAME_MEAN if z_frame_mean else hf.HF_Z_SUM,
                             sink_frames=sink_chunks * w.chunk_frames)
        self.ctx = hf.Context(cfg)
        if merge_full:
            Wb, bb = gen.merge_weights_full(w, layer, with_bias=bias)
            self.ctx.hf_set_merge_weights(layer, hf.bits_to_cuda(Wb), None if bb is None else hf.bits_to_cuda(bb))
        elif merge:
            Wb, bb = gen.merge_weights(w, layer, with_bias=bias)
            self.ctx.hf_set_merge_weights(layer, hf.bits_to_cuda(Wb), None if bb is None else hf.bits_to_cuda(bb))
        if rope:
            to_dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
            cq, sq = gen.rotation_tables(w, gen.T_ANGLE_Q); ck, sk = gen.rotation_tables(w, gen.T_ANGLE_K)
            self.ctx.hf_set_rope(to_dev(cq), to_dev(sq), to_dev(ck), to_dev(sk))
            torch.cuda.synchronize()
        if temporal is not None:        # (t0, first_pair, pairs)
            t, (cos, sin) = temporal_setup(w, *temporal)
            to_dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
            self.ctx.hf_set_temporal_rope(t["t0"], t["first_pair"], cos.shape[1], to_dev(cos), to_dev(sin))
            torch.cuda.synchronize()
        self.shape = (w.batch, w.heads, w.chunk_tokens, w.head_dim)

    def up(self, bits):
        return self.hf.bits_to_cuda(bits)

    def f64(self, t):
        return gen.bf16_bits_to_f64(self.hf.cuda_to_bits(t))

    def select(self, q, k):
        torch, ctx, L = self.torch, self.ctx, self.layer
        tn = ctx.hf_query(L, self.hf.HF_Q_KEY_BLOCKS); keep = ctx.hf_query(L, self.hf.HF_Q_KEPT_BLOCKS)
        tm = ctx.hf_query(L, self.hf.HF_Q_QUERY_BLOCKS); mw = ctx.hf_query(L, self.hf.HF_Q_MASK_WORDS)
        B, H = self.w.batch, self.w.heads
        mask = torch.zeros((B, H, tm, mw), dtype=torch.int32, device="cuda")
        idx = torch.zeros((B, H, tm, keep), dtype=torch.int32, device="cuda")
        sc = torch.zeros((B, H, tm, tn), dtype=torch.float32, device="cuda")
        ctx.hf_block_select(L, q, k, mask, idx, sc)
        torch.cuda.synchronize()
        m = unpack_mask(mask.cpu().numpy().view(np.uint32), tn)
        return m, idx.cpu().numpy(), sc.cpu().numpy()

    def swa(self, q, k, v, idx=None, want_lse=False):
        torch = self.torch
        o = torch.empty(self.shape, dtype=torch.bfloat16, device="cuda")
        lse = torch.empty(self.shape[:3], dtype=torch.float32, device="cuda") if want_lse else None
        self.ctx.hf_sparse_swa(self.layer, q, k, v, o, idx=idx, lse=lse)
        torch.cuda.synchronize()
        return (self.f64(o), lse.cpu().numpy()) if want_lse else self.f64(o)

    def linear(self, q):
        o = self.torch.empty(self.shape, dtype=self.torch.bfloat16, device="cuda")
        self.ctx.hf_linear_attn(self.layer, q, o)
        self.torch.cuda.synchronize()
        return self.f64(o)

    def forward(self, q, k, v):
        o = self.torch.empty(self.shape, dtype=self.torch.bfloat16, device="cuda")
        self.ctx.hf_hybrid_forward(self.layer, q, k, v, o)
        self.torch.cuda.synchronize()
        return self.f64(o)

    def append(self, k, v):
        self.ctx.hf_kv_append(self.layer, k, v)

    def state(self):
        torch, w = self.torch, self.w
        S = torch.empty((w.batch, w.heads, w.head_dim, w.head_dim), dtype=torch.float32, device="cuda")
        z = torch.empty((w.batch, w.heads, w.head_dim), dtype=torch.float32, device="cuda")
        self.ctx.hf_get_state(self.layer, S, z)
        torch.cuda.synchronize()
        return S.cpu().numpy().astype(np.float64), z.cpu().numpy().astype(np.float64)

    def close(self):
        self.ctx.close()


def assert_close_out(got, ref, what=""):
    ok = ~np.isnan(ref)
    ma, rl = max_abs(got[ok], ref[ok]), rel_l2(got[ok], ref[ok])
    assert ma <= MAX_ABS and rl <= REL_L2, f"{what}: max-abs {ma:.3e} (<= {MAX_ABS}), rel-L2 {rl:.3e} (<= {REL_L2})"
    return ma, rl
