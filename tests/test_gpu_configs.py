"""GPU parity at the workload level: the long stream (state drift), the full-depth stack and a subset of the
sweep grid, all at the 832x480 latent shape (1560 tokens per latent frame, 3-frame chunks).  The oracle is
evaluated on sampled query blocks where a full evaluation would take minutes; masks are compared in full."""
import numpy as np
import pytest

from paper_2604_10103_b200 import inputs as gen
from tests import harness as hz

pytestmark = pytest.mark.gpu

f64 = gen.bf16_bits_to_f64


def check_forward(gpu, ora, w, layer, chunk, step, q_blocks, what):
    """Select + forward of one denoising step on both sides; masks in full, outputs on q_blocks."""
    qb, kb, vb = gen.qkv(w, layer, chunk, step)
    q, k, v = gpu.up(qb), gpu.up(kb), gpu.up(vb)
    m_gpu, _, sc_gpu = gpu.select(q, k)
    m_ref, sc_ref = ora.select(f64(qb), f64(kb))
    assert np.array_equal(sc_gpu, sc_ref), f"{what}: scores differ in {np.sum(sc_gpu != sc_ref)} places"
    assert np.array_equal(m_gpu, m_ref), f"{what}: masks differ"
    o_ref = ora.forward(f64(qb), f64(kb), f64(vb), mask=m_ref, q_blocks=q_blocks)
    return hz.assert_close_out(gpu.forward(q, k, v), o_ref, what)


def test_stream_200_chunks_state_drift():
    """200 consecutive chunks of one layer, one 3-frame chunk evicted into the state per chunk once the window is
    full: final (S, z) within rel-L2 1e-4 of the fp64 recurrence; outputs and masks checked every 25th chunk."""
    w = gen.stream_832x480(chunks=200)
    gpu = hz.GpuStream(w); ora = hz.make_oracle(w)
    try:
        worst = 0.0
        for c in range(w.chunks):
            if c % 25 == 24 or c == w.chunks - 1:
                _, rl = check_forward(gpu, ora, w, 0, c, 0, [0, 36], f"chunk {c}")
                worst = max(worst, rl)
                S, z = gpu.state()
                assert hz.rel_l2(S, ora.S) <= hz.STATE_REL_L2, f"chunk {c}: S rel-L2 {hz.rel_l2(S, ora.S):.3e}"
                assert hz.rel_l2(z, ora.z) <= hz.STATE_REL_L2
            kc, vc = gen.clean_kv(w, 0, c)
            gpu.append(gpu.up(kc), gpu.up(vc))
            ora.append(f64(kc), f64(vc))
        S, z = gpu.state()
        assert gpu.ctx.hf_query(0, gpu.hf.HF_Q_ABSORBED_TOKENS) == ora.absorbed_tokens == 198 * w.chunk_tokens
        assert hz.rel_l2(S, ora.S) <= hz.STATE_REL_L2, f"final S rel-L2 {hz.rel_l2(S, ora.S):.3e}"
        assert hz.rel_l2(z, ora.z) <= hz.STATE_REL_L2, f"final z rel-L2 {hz.rel_l2(z, ora.z):.3e}"
        assert gpu.ctx.hf_get_device_status() == (0, 0)
    finally:
        gpu.close()


def test_full_depth_stack_three_layers_verified():
    """30 layer states in one context, 4 denoising-step forwards and one cache commit per chunk; layers are
    independent, so three of them (first, middle, last) are followed by the oracle through 4 chunks and every
    step of the last chunk is compared."""
    w = gen.full_depth_832x480(layers=30, steps=4, chunks=4)
    layers = [0, 14, 29]
    from paper_2604_10103_b200 import binding as hf
    base = hz.GpuStream(w, layer=layers[0], layers=w.layers)      # one context holds all 30 layer states
    oras = {l: hz.make_oracle(w, layer=l) for l in layers}
    try:
        for l in layers[1:]:
            Wb, bb = gen.merge_weights(w, l)
            base.ctx.hf_set_merge_weights(l, hf.bits_to_cuda(Wb), hf.bits_to_cuda(bb))
        filler_k, filler_v = (base.up(t) for t in gen.clean_kv(w, 999, 0))
        for c in range(w.chunks):
            for l in range(w.layers):
                if l in layers:
                    base.layer = l
                    if c == w.chunks - 1:
                        for s in range(w.steps):
                            check_forward(base, oras[l], w, l, c, s, [5, 36], f"layer {l} chunk {c} step {s}")
                    kc, vc = gen.clean_kv(w, l, c)
                    base.ctx.hf_kv_append(l, base.up(kc), base.up(vc))
                    oras[l].append(f64(kc), f64(vc))
                else:       # the other layers only carry their share of the cache traffic
                    base.ctx.hf_kv_append(l, filler_k, filler_v)
        for l in layers:
            base.layer = l
            S, z = base.state()
            assert hz.rel_l2(S, oras[l].S) <= hz.STATE_REL_L2 and hz.rel_l2(z, oras[l].z) <= hz.STATE_REL_L2
            assert base.ctx.hf_query(l, hf.HF_Q_ABSORBED_TOKENS) == oras[l].absorbed_tokens
        assert base.ctx.hf_get_device_status() == (0, 0)
    finally:
        base.close()


SWEEP_SUBSET = [
    # keep permille, window frames, head_dim, block, batch
    (100, 3, 64, 64, 4),      # window == chunk: every committed chunk goes straight into the state
    (500, 21, 128, 128, 1),   # longest window: six cached chunks
    (1000, 9, 64, 128, 1),    # everything kept: dense attention over the window, head_dim 64 on the tcgen05 path
    (250, 9, 128, 64, 4),     # 64-token blocks (warp-level tensor path), batch 4
    (100, 9, 128, 128, 1),    # sparsest setting of the grid
]


@pytest.mark.parametrize("permille,window,d,blk,batch", SWEEP_SUBSET)
def test_sweep_subset(permille, window, d, blk, batch):
    w = gen.layer_832x480().with_(name="sweep", keep_permille=permille, window_frames=window, head_dim=d, block=blk,
                                  batch=batch, heads=12 if batch == 1 else 3, seed=5)
    gpu = hz.GpuStream(w); ora = hz.make_oracle(w)
    try:
        n_prime = w.past_chunks + 2            # window full and at least two chunks in the state
        for c in range(n_prime):
            kc, vc = gen.clean_kv(w, 0, c)
            gpu.append(gpu.up(kc), gpu.up(vc)); ora.append(f64(kc), f64(vc))
        last = w.blocks_per_chunk - 1
        check_forward(gpu, ora, w, 0, n_prime, 0, [1, last], f"sweep point {permille}/{window}/{d}/{blk}/{batch}")
        S, z = gpu.state()
        assert hz.rel_l2(S, ora.S) <= hz.STATE_REL_L2 and hz.rel_l2(z, ora.z) <= hz.STATE_REL_L2
        assert gpu.ctx.hf_get_device_status() == (0, 0)
    finally:
        gpu.close()


def test_full_width_merge_at_the_832x480_layer_shape():
    """The projection over the model width at full size (12 heads x 128 = 1536 features, 4680 tokens): history term of
    hf_linear_attn against the oracle after two evictions (the attention branch at this size is covered above)."""
    from oracle import hybrid_attention as oa
    w = gen.layer_832x480().with_(seed=53)
    gpu = hz.GpuStream(w, merge_full=True); ora = hz.make_oracle(w, merge_full=True)
    f64 = gen.bf16_bits_to_f64
    try:
        for c in range(4):
            kc, vc = gen.clean_kv(w, 0, c)
            gpu.append(gpu.up(kc), gpu.up(vc)); ora.append(f64(kc), f64(vc))
        assert ora.absorbed_tokens == 2 * w.chunk_tokens
        qb, _, _ = gen.qkv(w, 0, 4, 0)
        qf = f64(qb)
        h = np.stack([oa.linear_readout(qf[0, hh], ora.S[0, hh], ora.z[0, hh], None, None, ora.eps) for hh in range(w.heads)])
        ref = oa.merge_full_width(h, ora.W_full, ora.bias_full)[None]
        hz.assert_close_out(gpu.linear(gpu.up(qb)), ref, "O_history, full-width merge, 832x480 layer")
        S, z = gpu.state()
        assert hz.rel_l2(S, ora.S) <= hz.STATE_REL_L2 and hz.rel_l2(z, ora.z) <= hz.STATE_REL_L2
        assert gpu.ctx.hf_get_device_status() == (0, 0)
    finally:
        gpu.close()


def test_many_cache_commits_at_batch_4_leave_a_clean_status():
    """Back-to-back cache commits with evictions at batch 4 (48 batch*head pairs, 64-token blocks, head_dim 64): the
    absorb, reduce/fold and copy kernels of consecutive commits overlap on two streams; no bounded wait may run out, and
    the state must match a context that absorbed the same evicted chunks one call at a time."""
    import torch
    from paper_2604_10103_b200 import binding as hf
    w = gen.layer_832x480().with_(name="commits", batch=4, head_dim=64, block=64, layers=2, seed=59)
    ctx = hf.Context(hf.make_config(w)); ref = hf.Context(hf.make_config(w.with_(layers=1)))
    try:
        shape = (w.batch, w.heads, w.chunk_tokens, w.head_dim)
        g = torch.Generator(device="cuda"); g.manual_seed(59)
        chunks = [(torch.randn(shape, generator=g, device="cuda").to(torch.bfloat16),
                   torch.randn(shape, generator=g, device="cuda").to(torch.bfloat16)) for _ in range(3)]
        n = 24
        for r in range(n):
            kk, vv = chunks[r % 3]
            ctx.hf_kv_append(r % 2, kk, vv)
        assert ctx.hf_get_device_status() == (0, 0)
        # layer 0 saw commits r = 0, 2, 4, ...: all but the last two of them were evicted, in order
        evicted = [r for r in range(0, n, 2)][:-w.past_chunks]
        for r in evicted:
            kk, vv = chunks[r % 3]
            ref.hf_state_absorb(0, kk, vv, w.chunk_tokens)
        S = torch.empty((w.batch, w.heads, 64, 64), dtype=torch.float32, device="cuda"); z = torch.empty((w.batch, w.heads, 64), dtype=torch.float32, device="cuda")
        S2 = torch.empty_like(S); z2 = torch.empty_like(z)
        ctx.hf_get_state(0, S, z); ref.hf_get_state(0, S2, z2)
        torch.cuda.synchronize()
        assert torch.equal(S, S2) and torch.equal(z, z2)
        assert ctx.hf_query(0, hf.HF_Q_ABSORBED_TOKENS) == len(evicted) * w.chunk_tokens
        assert ref.hf_get_device_status() == (0, 0)
    finally:
        ctx.close(); ref.close()
