"""The layer-batched cache commit and state update (Alg. 2's "pop(0) -> update LN; KV.append" for all layers of the model
in one call) against the per-layer entry points -- bit for bit -- and against the CPU oracle."""
import numpy as np
import pytest

from paper_2604_10103_b200 import inputs as gen
from tests import harness as hz

pytestmark = pytest.mark.gpu

f64 = gen.bf16_bits_to_f64


def _ctx(w, **kw):
    from paper_2604_10103_b200 import binding as hf
    ctx = hf.Context(hf.make_config(w, **kw))
    for l in range(w.layers):
        Wb, bb = gen.merge_weights(w, l)
        ctx.hf_set_merge_weights(l, hf.bits_to_cuda(Wb), hf.bits_to_cuda(bb))
    return ctx


def _state(ctx, w, layer):
    import torch
    S = torch.empty((w.batch, w.heads, w.head_dim, w.head_dim), dtype=torch.float32, device="cuda")
    z = torch.empty((w.batch, w.heads, w.head_dim), dtype=torch.float32, device="cuda")
    ctx.hf_get_state(layer, S, z)
    torch.cuda.synchronize()
    return S.cpu().numpy(), z.cpu().numpy()


def _forward(ctx, w, layer, q, k, v):
    import torch
    from paper_2604_10103_b200 import binding as hf
    o = torch.empty_like(q)
    ctx.hf_hybrid_forward(layer, q, k, v, o)
    torch.cuda.synchronize()
    return hf.cuda_to_bits(o)


@pytest.mark.parametrize("d,tpf,sink,layers,heads", [
    (128, 200, 0, 14, 12),      # 168 (layer, head) items on 148 SMs: some thread blocks take two items; ragged tiles (200 = 3 x 64 + 8)
    (64, 333, 1, 20, 8),        # head_dim 64 (two idle lane quadrants), one sink chunk, 160 items
    (128, 1000, 0, 26, 6),      # 16 tiles per item: twelve splits of one or two tiles
])
def test_batched_commit_equals_per_layer_commits_bit_for_bit(d, tpf, sink, layers, heads):
    """Two contexts get the same stream, one through hf_kv_append layer by layer, one through hf_kv_append_layers: states
    equal bit for bit after every chunk, forwards equal bit for bit (cache contents and pooled means), bookkeeping equal,
    and two layers against the oracle."""
    from paper_2604_10103_b200 import binding as hf
    w = gen.Workload("layers", batch=1, heads=heads, head_dim=d, tokens_per_frame=tpf, chunk_frames=1, window_frames=3,
                     block=128, topk=0, keep_permille=500, layers=layers, seed=71)
    a = _ctx(w, sink_frames=sink); b = _ctx(w, sink_frames=sink)
    check_layers = [0, layers - 1]
    ora = {l: hz.make_oracle(w, layer=l, sink_chunks=sink) for l in check_layers}
    try:
        for c in range(sink + 5):
            kv = [gen.clean_kv(w, j, c) for j in range(3)]                   # three distinct tensors, cycled over the layers
            ks = [hf.bits_to_cuda(k) for k, _ in kv]; vs = [hf.bits_to_cuda(v) for _, v in kv]
            for l in range(layers):
                a.hf_kv_append(l, ks[l % 3], vs[l % 3])
            b.hf_kv_append_layers(0, [ks[l % 3] for l in range(layers)], [vs[l % 3] for l in range(layers)])
            for l in check_layers:
                ora[l].append(f64(kv[l % 3][0]), f64(kv[l % 3][1]))
            for l in range(layers):
                Sa, za = _state(a, w, l); Sb, zb = _state(b, w, l)
                assert np.array_equal(Sa, Sb) and np.array_equal(za, zb), f"chunk {c} layer {l}: states differ"
                for what in (hf.HF_Q_CACHED_CHUNKS, hf.HF_Q_ABSORBED_TOKENS, hf.HF_Q_SINK_CHUNKS, hf.HF_Q_KEY_BLOCKS):
                    assert a.hf_query(l, what) == b.hf_query(l, what)
            for l in check_layers:
                assert a.hf_query(l, hf.HF_Q_ABSORBED_TOKENS) == ora[l].absorbed_tokens
                if ora[l].absorbed_tokens:
                    Sb, zb = _state(b, w, l)
                    assert hz.rel_l2(Sb, ora[l].S) <= hz.STATE_REL_L2 and hz.rel_l2(zb, ora[l].z) <= hz.STATE_REL_L2
        assert ora[0].absorbed_tokens > 0
        qb, kb, vb = gen.qkv(w, 0, 9, 0)
        q, k, v = hf.bits_to_cuda(qb), hf.bits_to_cuda(kb), hf.bits_to_cuda(vb)
        for l in (0, layers // 2, layers - 1):
            oa, ob = _forward(a, w, l, q, k, v), _forward(b, w, l, q, k, v)
            assert np.array_equal(oa, ob), f"layer {l}: forwards differ"
        hz.assert_close_out(f64(_forward(b, w, 0, q, k, v)), ora[0].forward(f64(qb), f64(kb), f64(vb)), "forward after batched commits")
        assert a.hf_get_device_status() == (0, 0) and b.hf_get_device_status() == (0, 0)
    finally:
        a.close(); b.close()


@pytest.mark.parametrize("d,n,zmean,rope", [(128, 333, False, False), (64, 640, True, False), (128, 150, False, True)])
def test_batched_absorb_equals_per_layer_absorbs_bit_for_bit(d, n, zmean, rope):
    """hf_state_absorb_layers on [layers, B, H, n, d] tokens against one hf_state_absorb per layer (bit for bit) and the
    oracle's Eq. 3: token counts off the tile size, per-frame-mean normaliser, rotated keys."""
    import torch
    from oracle import hybrid_attention as oa
    from paper_2604_10103_b200 import binding as hf
    layers, B, H = 40, 2, 2
    w = gen.Workload("absl", batch=B, heads=H, head_dim=d, tokens_per_frame=n if not zmean else n // 2, chunk_frames=1 if not zmean else 2,
                     window_frames=2 if not zmean else 4, block=64, topk=1, keep_permille=0, layers=layers, seed=72)
    zm = hf.HF_Z_FRAME_MEAN if zmean else hf.HF_Z_SUM
    a = _ctx(w, z_mode=zm); b = _ctx(w, z_mode=zm)
    try:
        if rope:
            ck, sk = gen.rotation_tables(w, gen.T_ANGLE_K)
            to_dev = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda()
            for ctx in (a, b):
                ctx.hf_set_rope(None, None, to_dev(ck), to_dev(sk))
        for call in range(2):
            kb = gen.normal_bf16((layers, B, H, n, d), 72, call, 1); vb = gen.normal_bf16((layers, B, H, n, d), 72, call, 2)
            k, v = hf.bits_to_cuda(kb), hf.bits_to_cuda(vb)
            for l in range(layers):
                a.hf_state_absorb(l, k[l], v[l], n)
            b.hf_state_absorb_layers(0, layers, k, v, n)
            for l in range(layers):
                Sa, za = _state(a, w, l); Sb, zb = _state(b, w, l)
                assert np.array_equal(Sa, Sb) and np.array_equal(za, zb), f"call {call} layer {l}"
                assert b.hf_query(l, hf.HF_Q_ABSORBED_TOKENS) == (call + 1) * n
            if call == 0:
                for l in (0, layers - 1):
                    Sb, zb = _state(b, w, l)
                    for bi in range(B):
                        for h in range(H):
                            S0 = np.zeros((d, d)); z0 = np.zeros(d)
                            if rope:
                                Sr, zr = oa.absorb_rope(S0, z0, f64(kb)[l, bi, h], f64(vb)[l, bi, h], ck, sk)
                            elif zmean:
                                Sr, zr = oa.absorb_frame_mean(S0, z0, f64(kb)[l, bi, h], f64(vb)[l, bi, h], w.tokens_per_frame)
                            else:
                                Sr, zr = oa.absorb(S0, z0, f64(kb)[l, bi, h], f64(vb)[l, bi, h])
                            assert hz.rel_l2(Sb[bi, h], Sr) <= hz.STATE_REL_L2 and hz.rel_l2(zb[bi, h], zr) <= hz.STATE_REL_L2
        assert a.hf_get_device_status() == (0, 0) and b.hf_get_device_status() == (0, 0)
    finally:
        a.close(); b.close()


def test_layers_in_different_phases_and_small_calls_fall_back_to_the_per_layer_path():
    """Layer 0 is one chunk ahead of the others (it evicts while they still fill the window), and a call over two layers
    has too few items for the persistent launch: both must leave what per-layer commits leave."""
    from paper_2604_10103_b200 import binding as hf
    layers = 13
    w = gen.Workload("phases", batch=1, heads=12, head_dim=128, tokens_per_frame=130, chunk_frames=1, window_frames=3,
                     block=128, topk=0, keep_permille=500, layers=layers, seed=73)
    a = _ctx(w); b = _ctx(w)
    try:
        k0, v0 = (hf.bits_to_cuda(t) for t in gen.clean_kv(w, 0, 99))
        a.hf_kv_append(0, k0, v0); b.hf_kv_append(0, k0, v0)
        for c in range(4):
            k, v = (hf.bits_to_cuda(t) for t in gen.clean_kv(w, 0, c))
            for l in range(layers):
                a.hf_kv_append(l, k, v)
            if c < 3:       # c == 1: layer 0 evicts while the others still fill their window
                b.hf_kv_append_layers(0, [k] * layers, [v] * layers)
            else:
                b.hf_kv_append_layers(0, [k] * 2, [v] * 2)
                b.hf_kv_append_layers(2, [k] * (layers - 2), [v] * (layers - 2))
            for l in range(layers):
                Sa, za = _state(a, w, l); Sb, zb = _state(b, w, l)
                assert np.array_equal(Sa, Sb) and np.array_equal(za, zb), f"chunk {c} layer {l}"
                assert a.hf_query(l, hf.HF_Q_ABSORBED_TOKENS) == b.hf_query(l, hf.HF_Q_ABSORBED_TOKENS)
        with pytest.raises(hf.HFError, match="HF_ERR_INVALID_ARG"):
            b.hf_kv_append_layers(5, [k] * layers, [v] * layers)        # runs past the last layer
        assert b.hf_get_device_status() == (0, 0)
    finally:
        a.close(); b.close()


def test_batched_commit_at_the_832x480_shape_against_the_oracle():
    """30 layers x 12 heads of 4680 tokens: the shape the bench times.  Layers 0 and 29 against the oracle after the
    evictions of two chunks; all layers deterministic from run to run."""
    from paper_2604_10103_b200 import binding as hf
    w = gen.layer_832x480().with_(layers=30, seed=74)
    snaps = []
    for run in range(2):
        ctx = _ctx(w)
        try:
            ora = {l: hz.make_oracle(w, layer=l) for l in (0, 29)} if run == 0 else {}
            for c in range(4):
                kb, vb = gen.clean_kv(w, 0, c)
                k, v = hf.bits_to_cuda(kb), hf.bits_to_cuda(vb)
                ctx.hf_kv_append_layers(0, [k] * 30, [v] * 30)
                for l in ora:
                    ora[l].append(f64(kb), f64(vb))
            snaps.append([_state(ctx, w, l) for l in range(30)])
            for l in ora:
                S, z = snaps[-1][l]
                assert ora[l].absorbed_tokens == 2 * 4680 == ctx.hf_query(l, hf.HF_Q_ABSORBED_TOKENS)
                assert hz.rel_l2(S, ora[l].S) <= hz.STATE_REL_L2 and hz.rel_l2(z, ora[l].z) <= hz.STATE_REL_L2
            assert ctx.hf_get_device_status() == (0, 0)
        finally:
            ctx.close()
    for (S0, z0), (S1, z1) in zip(*snaps):
        assert np.array_equal(S0, S1) and np.array_equal(z0, z1)
