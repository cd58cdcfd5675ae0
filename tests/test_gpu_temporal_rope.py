"""Relative temporal RoPE of the softmax branch (Sec. 3.3, Eq. 8) inside the library: streams that cross the cap T_0,
against the oracle run the same way (bit-exact block scores and masks, outputs and state within tolerance)."""
import numpy as np
import pytest

from paper_2604_10103_b200 import inputs as gen
from tests import harness as hz

pytestmark = pytest.mark.gpu

f64 = gen.bf16_bits_to_f64


@pytest.mark.parametrize("d,b,tpf,cf,wf,sink,t0,first_pair,pairs,kernel,chunks", [
    (128, 128, 100, 3, 9, 0, 9, 0, None, 0, 8),     # one-kernel forward; the cap is reached with the third chunk; 300 = 2 x 128 + 44
    (128, 128, 100, 3, 9, 0, 21, 0, None, 0, 9),    # the paper's T_0 = 21: crossed with the eighth chunk
    (64, 16, 20, 3, 6, 1, 6, 4, 10, 0, 7),          # small blocks, a sink chunk, temporal pairs in the middle of the head
    (128, 64, 96, 1, 3, 0, 4, 0, 22, 0, 8),         # one-frame chunks
    (128, 128, 130, 2, 2, 0, 4, 0, None, 0, 5),     # window == chunk: nothing cached, chunks go straight to the state
    (64, 128, 150, 3, 6, 0, 6, 0, None, 3, 6),      # ping-pong kernel, head_dim 64
    (128, 128, 100, 3, 9, 0, 9, 0, None, 1, 6),     # warp-level kernel
])
def test_stream_across_the_cap(d, b, tpf, cf, wf, sink, t0, first_pair, pairs, kernel, chunks):
    w = gen.Workload("trope", batch=1, heads=2, head_dim=d, tokens_per_frame=tpf, chunk_frames=cf, window_frames=wf,
                     block=b, topk=0, keep_permille=500, seed=91)
    temporal = (t0, first_pair, pairs)
    gpu = hz.GpuStream(w, swa_kernel=kernel, sink_chunks=sink, temporal=temporal)
    ora = hz.make_oracle(w, sink_chunks=sink, temporal=temporal)
    try:
        for c in range(chunks):
            qb, kb, vb = gen.qkv(w, 0, c, 0)
            q, k, v = gpu.up(qb), gpu.up(kb), gpu.up(vb)
            m_gpu, _, sc_gpu = gpu.select(q, k)
            m_ref, sc_ref = ora.select(f64(qb), f64(kb))
            assert np.array_equal(sc_gpu, sc_ref), f"chunk {c}: {np.sum(sc_gpu != sc_ref)} scores differ"
            assert np.array_equal(m_gpu, m_ref), f"chunk {c}: masks differ"
            o_ref, ol_ref, oh_ref = ora.forward(f64(qb), f64(kb), f64(vb), mask=m_ref, parts=True)
            hz.assert_close_out(gpu.forward(q, k, v), o_ref, f"chunk {c} hybrid O")
            hz.assert_close_out(gpu.swa(q, k, v), ol_ref, f"chunk {c} O_local")
            hz.assert_close_out(gpu.linear(q), oh_ref, f"chunk {c} O_history")
            kc, vc = gen.clean_kv(w, 0, c)
            gpu.append(gpu.up(kc), gpu.up(vc)); ora.append(f64(kc), f64(vc))
            assert gpu.ctx.hf_query(0, gpu.hf.HF_Q_ABSORBED_TOKENS) == ora.absorbed_tokens
        assert ora.frames_committed + cf > t0, "the stream must have crossed the cap"
        S, z = gpu.state()
        if ora.absorbed_tokens:
            assert hz.rel_l2(S, ora.S) <= hz.STATE_REL_L2 and hz.rel_l2(z, ora.z) <= hz.STATE_REL_L2
        assert gpu.ctx.hf_get_device_status() == (0, 0)
    finally:
        gpu.close()


def test_the_rotation_matters_and_must_be_set_on_an_empty_stream():
    import torch
    w = gen.Workload("trope2", batch=1, heads=2, head_dim=128, tokens_per_frame=100, chunk_frames=3, window_frames=9,
                     block=128, topk=0, keep_permille=500, seed=92)
    plain = hz.GpuStream(w); rot = hz.GpuStream(w, temporal=(9, 0, None))
    try:
        for c in range(4):
            kc, vc = gen.clean_kv(w, 0, c)
            for g in (plain, rot):
                g.append(g.up(kc), g.up(vc))
        qb, kb, vb = gen.qkv(w, 0, 4, 0)
        a = plain.forward(plain.up(qb), plain.up(kb), plain.up(vb)); b = rot.forward(rot.up(qb), rot.up(kb), rot.up(vb))
        assert hz.rel_l2(a, b) > 0.05
        t, (cos, sin) = hz.temporal_setup(w, 9)
        with pytest.raises(plain.hf.HFError, match="HF_ERR_STATE"):
            plain.ctx.hf_set_temporal_rope(9, 0, cos.shape[1], torch.from_numpy(cos).cuda(), torch.from_numpy(sin).cuda())
        with pytest.raises(plain.hf.HFError, match="HF_ERR_SHAPE"):
            hz.GpuStream(w).ctx.hf_set_temporal_rope(9, 60, 22, torch.from_numpy(cos).cuda(), torch.from_numpy(sin).cuda())
    finally:
        plain.close(); rot.close()


def test_checkpoint_across_the_cap_continues_bit_for_bit():
    """The stream position is part of the image: a stream exported before the cap and continued in a fresh context gives the
    bits the uninterrupted stream gives, on both sides of the cap."""
    w = gen.Workload("trope3", batch=1, heads=2, head_dim=128, tokens_per_frame=100, chunk_frames=3, window_frames=9,
                     block=128, topk=0, keep_permille=500, seed=93)
    temporal = (12, 0, None)

    def run(ctx_stream, lo, hi, outs):
        for c in range(lo, hi):
            qb, kb, vb = gen.qkv(w, 0, c, 0)
            outs.append(ctx_stream.forward(ctx_stream.up(qb), ctx_stream.up(kb), ctx_stream.up(vb)))
            kc, vc = gen.clean_kv(w, 0, c)
            ctx_stream.append(ctx_stream.up(kc), ctx_stream.up(vc))

    whole = hz.GpuStream(w, temporal=temporal); first = hz.GpuStream(w, temporal=temporal); second = hz.GpuStream(w, temporal=temporal)
    try:
        a, b = [], []
        run(whole, 0, 8, a)
        run(first, 0, 3, b)
        second.ctx.hf_state_import(first.ctx.hf_state_export())
        run(second, 3, 8, b)
        for x, y in zip(a, b):
            assert np.array_equal(x, y)
        Sa, za = whole.state(); Sb, zb = second.state()
        assert np.array_equal(Sa, Sb) and np.array_equal(za, zb)
    finally:
        whole.close(); first.close(); second.close()
