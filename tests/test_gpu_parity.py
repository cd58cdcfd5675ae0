"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element,
on the same seeded bf16 inputs.  Masks bit-exact; outputs max-abs <= 2e-2 and rel-L2 <= 5e-3;
state rel-L2 <= 1e-4."""
import numpy as np
import pytest

from paper_2604_10103_b200 import inputs as gen
from tests import harness as hz

pytestmark = pytest.mark.gpu

f64 = gen.bf16_bits_to_f64


def stream_compare(w: gen.Workload, chunks: int, merge=True, bias=True, check_parts=True, q_blocks_for=None, swa_kernel=0):
    """Stream `chunks` chunks (one forward + one append each) on both sides; compare every call."""
    gpu = hz.GpuStream(w, merge=merge, bias=bias, swa_kernel=swa_kernel)
    ora = hz.make_oracle(w, merge=merge, bias=bias)
    worst = {"o": 0.0, "ol": 0.0, "oh": 0.0}
    try:
        for c in range(chunks):
            qb, kb, vb = gen.qkv(w, 0, c, 0)
            q, k, v = gpu.up(qb), gpu.up(kb), gpu.up(vb)
            qf, kf, vf = f64(qb), f64(kb), f64(vb)
            # Eq. 5 + top-K: bit-exact mask, ascending index list, scores equal to the canonical float32 scores
            m_gpu, idx_gpu, sc_gpu = gpu.select(q, k)
            m_ref, sc_ref = ora.select(qf, kf)
            assert sc_gpu.shape == sc_ref.shape
            assert np.array_equal(sc_gpu, sc_ref), f"chunk {c}: scores differ in {np.sum(sc_gpu != sc_ref)} places"
            assert np.array_equal(m_gpu, m_ref), f"chunk {c}: masks differ"
            keep = int(m_ref[0, 0, 0].sum())
            assert idx_gpu.shape[-1] == keep
            ref_idx = np.stack([np.flatnonzero(r) for r in m_ref.reshape(-1, m_ref.shape[-1])]).reshape(idx_gpu.shape)
            assert np.array_equal(idx_gpu, ref_idx)
            # Alg. 3 + Eq. 7
            qbl = None if q_blocks_for is None else q_blocks_for(c)
            if qbl is not None and len(qbl) == 0:
                gpu.forward(q, k, v)
            else:
                o_ref, ol_ref, oh_ref = ora.forward(qf, kf, vf, mask=m_ref, q_blocks=qbl, parts=True)
                worst["o"] = max(worst["o"], hz.assert_close_out(gpu.forward(q, k, v), o_ref, f"chunk {c} hybrid O")[1])
                if check_parts:
                    worst["ol"] = max(worst["ol"], hz.assert_close_out(gpu.swa(q, k, v), ol_ref, f"chunk {c} O_local")[1])
                    worst["oh"] = max(worst["oh"], hz.assert_close_out(gpu.linear(q), oh_ref, f"chunk {c} O_history")[1])
            # Alg. 2 cache commit
            kc, vc = gen.clean_kv(w, 0, c)
            gpu.append(gpu.up(kc), gpu.up(vc))
            ora.append(f64(kc), f64(vc))
            assert gpu.ctx.hf_query(0, gpu.hf.HF_Q_CACHED_CHUNKS) == len(ora.past)
            assert gpu.ctx.hf_query(0, gpu.hf.HF_Q_ABSORBED_TOKENS) == ora.absorbed_tokens
        S, z = gpu.state()
        if ora.absorbed_tokens:
            assert hz.rel_l2(S, ora.S) <= hz.STATE_REL_L2, f"S rel-L2 {hz.rel_l2(S, ora.S):.3e}"
            assert hz.rel_l2(z, ora.z) <= hz.STATE_REL_L2, f"z rel-L2 {hz.rel_l2(z, ora.z):.3e}"
        else:
            assert not S.any() and not z.any()
        assert gpu.ctx.hf_get_device_status() == (0, 0)
    finally:
        gpu.close()
    return worst


def test_tiny_config_stream():
    """Tiny case: 2 heads of 64, 64-token frames, window 3, 16-token blocks, top-2, 6 chunks (3 evictions seen)."""
    stream_compare(gen.tiny(), 6)


def test_tiny_identity_merge_and_no_bias():
    stream_compare(gen.tiny(), 5, merge=False)
    stream_compare(gen.tiny(), 5, merge=True, bias=False)


@pytest.mark.parametrize("d,b,tpf,cf,wf,B", [
    (64, 64, 100, 2, 6, 2),     # ragged 200-token chunks, 64-blocks, batch 2
    (128, 64, 150, 1, 3, 1),    # ragged, d=128
    (128, 128, 300, 1, 2, 1),   # several 128-tiles + 44-token tail, P = 1
    (64, 128, 129, 1, 3, 2),    # 1-token tail block
    (128, 16, 40, 1, 3, 1),     # 16-blocks with d=128, ragged
    (128, 128, 200, 1, 1, 1),   # window == chunk: P = 0, chunks go straight to the state
])
def test_ragged_shapes(d, b, tpf, cf, wf, B):
    w = gen.Workload("ragged", batch=B, heads=3, head_dim=d, tokens_per_frame=tpf, chunk_frames=cf, window_frames=wf,
                     block=b, topk=0, keep_permille=400, seed=11)
    stream_compare(w, wf // cf + 2)


def test_keep_everything_and_keep_one():
    w = gen.Workload("k_all", batch=1, heads=2, head_dim=64, tokens_per_frame=96, chunk_frames=1, window_frames=3,
                     block=16, topk=0, keep_permille=1000, seed=12)
    stream_compare(w, 4)
    stream_compare(w.with_(topk=1, keep_permille=0), 4)


def test_ties_go_to_the_lower_block_index():
    """q = 0 makes every score 0: the first k blocks must be kept, and O_local is the plain mean of their V rows."""
    import torch
    w = gen.tiny()
    gpu = hz.GpuStream(w)
    try:
        for c in range(3):
            kc, vc = gen.clean_kv(w, 0, c)
            gpu.append(gpu.up(kc), gpu.up(vc))
        _, kb, vb = gen.qkv(w, 0, 3, 0)
        q = torch.zeros(gpu.shape, dtype=torch.bfloat16, device="cuda")
        m, idx, sc = gpu.select(q, gpu.up(kb))
        assert not sc.any() and m[..., :2].all() and not m[..., 2:].any()
        assert (idx == np.array([0, 1])).all()
        o = gpu.swa(q, gpu.up(kb), gpu.up(vb))
        kc0, vc0 = gen.clean_kv(w, 0, 1)   # oldest cached chunk is chunk 1 (chunk 0 was evicted)
        ref = f64(vc0)[:, :, :32].mean(axis=2, keepdims=True)
        assert np.abs(o - ref).max() < 2e-3
    finally:
        gpu.close()


def test_selection_and_outputs_are_deterministic():
    w = gen.tiny().with_(seed=21)
    outs = []
    for _ in range(2):
        gpu = hz.GpuStream(w)
        try:
            for c in range(4):
                kc, vc = gen.clean_kv(w, 0, c)
                gpu.append(gpu.up(kc), gpu.up(vc))
            qb, kb, vb = gen.qkv(w, 0, 4, 0)
            o = gpu.forward(gpu.up(qb), gpu.up(kb), gpu.up(vb))
            S, z = gpu.state()
            outs.append((o, S, z))
        finally:
            gpu.close()
    for a, b in zip(outs[0], outs[1]):
        assert np.array_equal(a, b)


def test_state_absorb_arbitrary_token_counts():
    """hf_state_absorb on caller-supplied tokens (Eq. 3), including counts that are not a tile multiple."""
    from oracle import hybrid_attention as oa
    w = gen.Workload("abs", batch=2, heads=2, head_dim=128, tokens_per_frame=64, chunk_frames=1, window_frames=2,
                     block=64, topk=1, keep_permille=0, seed=13)
    gpu = hz.GpuStream(w, merge=False)
    try:
        S = np.zeros((2, 2, 128, 128)); z = np.zeros((2, 2, 128))
        for i, n in enumerate([1, 63, 64, 65, 1000]):
            kb = gen.normal_bf16((2, 2, n, 128), 13, i, 1); vb = gen.normal_bf16((2, 2, n, 128), 13, i, 2)
            gpu.ctx.hf_state_absorb(0, gpu.up(kb), gpu.up(vb), n)
            for b in range(2):
                for h in range(2):
                    S[b, h], z[b, h] = oa.absorb(S[b, h], z[b, h], f64(kb)[b, h], f64(vb)[b, h])
            Sg, zg = gpu.state()
            assert hz.rel_l2(Sg, S) <= hz.STATE_REL_L2 and hz.rel_l2(zg, z) <= hz.STATE_REL_L2
    finally:
        gpu.close()


def test_lse_output():
    w = gen.tiny().with_(seed=22)
    gpu = hz.GpuStream(w); ora = hz.make_oracle(w)
    try:
        qb, kb, vb = gen.qkv(w, 0, 0, 0)
        q, k, v = gpu.up(qb), gpu.up(kb), gpu.up(vb)
        m, idx, _ = gpu.select(q, k)
        o, lse = gpu.swa(q, k, v, want_lse=True)
        qf, kf = f64(qb), f64(kb)
        for h in range(2):
            for i in range(4):
                cols = np.concatenate([np.arange(j * 16, j * 16 + 16) for j in idx[0, h, i]])
                s = qf[0, h, i * 16:(i + 1) * 16] @ kf[0, h, cols].T / 8.0
                ref = np.log(np.exp(s).sum(axis=1))
                assert np.abs(lse[0, h, i * 16:(i + 1) * 16] - ref).max() < 1e-3
    finally:
        gpu.close()


def test_call_order_errors_do_not_launch():
    import torch
    w = gen.tiny()
    gpu = hz.GpuStream(w)
    try:
        qb, kb, vb = gen.qkv(w, 0, 0, 0)
        q, k, v = gpu.up(qb), gpu.up(kb), gpu.up(vb)
        o = torch.empty_like(q)
        n0 = gpu.ctx.hf_launch_count()
        with pytest.raises(gpu.hf.HFError, match="HF_ERR_STATE"):
            gpu.ctx.hf_sparse_swa(0, q, k, v, o)            # no selection yet
        with pytest.raises(gpu.hf.HFError, match="HF_ERR_INVALID_ARG"):
            gpu.ctx.hf_hybrid_forward(0, q, k, None, o)
        with pytest.raises(gpu.hf.HFError, match="HF_ERR_INVALID_ARG"):
            gpu.ctx.hf_hybrid_forward(5, q, k, v, o)
        with pytest.raises(gpu.hf.HFError, match="HF_ERR_INVALID_ARG"):
            gpu.ctx.hf_kv_append(0, k.view(-1)[1:], v)       # misaligned
        assert gpu.ctx.hf_launch_count() == n0
        gpu.select(q, k)
        gpu.ctx.hf_sparse_swa(0, q, k, v, o)
        gpu.append(k, v)
        with pytest.raises(gpu.hf.HFError, match="HF_ERR_STATE"):
            gpu.ctx.hf_sparse_swa(0, q, k, v, o)            # cache changed since the selection
    finally:
        gpu.close()


def test_layer_832x480_single_forward():
    """One layer at the 832x480 latent shape: prime with 4 clean chunks (2 evicted into the state), then check the
    forward of chunk 5 on every head for a sample of query blocks (first, a middle one, the ragged last)."""
    w = gen.layer_832x480()
    gpu = hz.GpuStream(w); ora = hz.make_oracle(w)
    try:
        for c in range(4):
            kc, vc = gen.clean_kv(w, 0, c)
            gpu.append(gpu.up(kc), gpu.up(vc)); ora.append(f64(kc), f64(vc))
        S, z = gpu.state()
        assert hz.rel_l2(S, ora.S) <= hz.STATE_REL_L2 and hz.rel_l2(z, ora.z) <= hz.STATE_REL_L2
        qb, kb, vb = gen.qkv(w, 0, 4, 0)
        q, k, v = gpu.up(qb), gpu.up(kb), gpu.up(vb)
        m_gpu, idx_gpu, sc_gpu = gpu.select(q, k)
        m_ref, sc_ref = ora.select(f64(qb), f64(kb))
        assert m_ref.shape == (1, 12, 37, 111) and int(m_ref[0, 0, 0].sum()) == 28
        assert np.array_equal(sc_gpu, sc_ref) and np.array_equal(m_gpu, m_ref)
        qbl = [0, 17, 36]
        o_ref, ol_ref, oh_ref = ora.forward(f64(qb), f64(kb), f64(vb), mask=m_ref, q_blocks=qbl, parts=True)
        hz.assert_close_out(gpu.forward(q, k, v), o_ref, "hybrid O")
        hz.assert_close_out(gpu.swa(q, k, v), ol_ref, "O_local")
        hz.assert_close_out(gpu.linear(q), oh_ref, "O_history")          # every row: max-abs and rel-L2
    finally:
        gpu.close()


def test_frame_mean_reading_of_the_state_denominator():
    """HF_Z_FRAME_MEAN: z accumulates per-frame means of phi(K) (Eq. 3 as printed); outputs and state against the oracle
    run the same way; a token count that is not whole frames is refused."""
    import torch
    w = gen.Workload("zmean", batch=1, heads=3, head_dim=128, tokens_per_frame=96, chunk_frames=2, window_frames=4,
                     block=64, topk=0, keep_permille=500, seed=14)
    gpu = hz.GpuStream(w, z_frame_mean=True); ora = hz.make_oracle(w, z_frame_mean=True)
    try:
        for c in range(4):
            kc, vc = gen.clean_kv(w, 0, c)
            gpu.append(gpu.up(kc), gpu.up(vc)); ora.append(f64(kc), f64(vc))
        S, z = gpu.state()
        assert hz.rel_l2(S, ora.S) <= hz.STATE_REL_L2 and hz.rel_l2(z, ora.z) <= hz.STATE_REL_L2
        qb, kb, vb = gen.qkv(w, 0, 4, 0)
        o_ref, _, oh_ref = ora.forward(f64(qb), f64(kb), f64(vb), parts=True)
        # with per-frame means the history term is T_f = 96 times larger (|O| up to ~10 here): the absolute bound is
        # widened by the bf16 half-ulp of the largest output, the relative bound stays
        o = gpu.forward(gpu.up(qb), gpu.up(kb), gpu.up(vb))
        assert hz.rel_l2(o, o_ref) <= hz.REL_L2
        assert hz.max_abs(o, o_ref) <= hz.MAX_ABS + 2.0 ** -8 * np.abs(o_ref).max()
        assert hz.rel_l2(gpu.linear(gpu.up(qb)), oh_ref) <= hz.REL_L2
        bad = torch.zeros((1, 3, 100, 128), dtype=torch.bfloat16, device="cuda")
        with pytest.raises(gpu.hf.HFError, match="HF_ERR_SHAPE"):
            gpu.ctx.hf_state_absorb(0, bad, bad, 100)
    finally:
        gpu.close()


@pytest.mark.parametrize("d,tpf,wf,permille", [
    (128, 300, 2, 400),     # several 128-tiles + 44-token tail, one cached chunk
    (64, 129, 3, 1000),     # head_dim 64, 1-token tail block, everything kept
    (128, 200, 1, 1000),    # window == chunk: two key blocks per row
    (128, 520, 3, 100),     # sparse: few tiles per row (odd counts leave one group with fewer tiles)
])
def test_pingpong_attention_kernel(d, tpf, wf, permille):
    """The tile-alternating tcgen05 kernel against the oracle (same stream as the other kernels), including rows whose
    kept list gives the two softmax groups unequal numbers of tiles."""
    from paper_2604_10103_b200 import binding as hf
    w = gen.Workload("pp", batch=2, heads=2, head_dim=d, tokens_per_frame=tpf, chunk_frames=1, window_frames=wf,
                     block=128, topk=0, keep_permille=permille, seed=15)
    stream_compare(w, wf + 2, swa_kernel=hf.HF_SWA_TCGEN05_PINGPONG)


def test_pingpong_single_kept_block_and_lse():
    """k = 1: the second softmax group has no tile at all and must drop out of the merge."""
    from paper_2604_10103_b200 import binding as hf
    w = gen.Workload("pp1", batch=1, heads=2, head_dim=128, tokens_per_frame=256, chunk_frames=1, window_frames=3,
                     block=128, topk=1, keep_permille=0, seed=16)
    stream_compare(w, 4, swa_kernel=hf.HF_SWA_TCGEN05_PINGPONG)


@pytest.mark.parametrize("d,b,tpf,wf,sink,kernel", [
    (128, 128, 300, 2, 1, 0),    # tcgen05 path, one sink chunk + one cached chunk
    (128, 128, 260, 3, 2, 3),    # ping-pong kernel, two sink chunks
    (64, 16, 64, 3, 1, 0),       # small blocks (warp-level tensor path)
    (128, 128, 200, 1, 1, 0),    # window == chunk: no rolling cache at all, only sink + current + state
])
def test_sink_chunks(d, b, tpf, wf, sink, kernel):
    """Attention sink: the first chunks of the stream stay visible as the oldest key blocks, are never evicted and
    never reach the state (cache bookkeeping, masks, outputs and state against the oracle run the same way)."""
    w = gen.Workload("sink", batch=1, heads=3, head_dim=d, tokens_per_frame=tpf, chunk_frames=1, window_frames=wf,
                     block=b, topk=0, keep_permille=500, seed=17)
    gpu = hz.GpuStream(w, sink_chunks=sink, swa_kernel=kernel); ora = hz.make_oracle(w, sink_chunks=sink)
    try:
        for c in range(sink + wf + 2):
            qb, kb, vb = gen.qkv(w, 0, c, 0)
            q, k, v = gpu.up(qb), gpu.up(kb), gpu.up(vb)
            m_gpu, _, sc_gpu = gpu.select(q, k)
            m_ref, sc_ref = ora.select(f64(qb), f64(kb))
            assert np.array_equal(sc_gpu, sc_ref) and np.array_equal(m_gpu, m_ref), f"chunk {c}"
            o_ref = ora.forward(f64(qb), f64(kb), f64(vb), mask=m_ref)
            hz.assert_close_out(gpu.forward(q, k, v), o_ref, f"chunk {c} hybrid O with sink")
            kc, vc = gen.clean_kv(w, 0, c)
            gpu.append(gpu.up(kc), gpu.up(vc)); ora.append(f64(kc), f64(vc))
            assert gpu.ctx.hf_query(0, gpu.hf.HF_Q_SINK_CHUNKS) == len(ora.sink)
            assert gpu.ctx.hf_query(0, gpu.hf.HF_Q_CACHED_CHUNKS) == len(ora.past)
            assert gpu.ctx.hf_query(0, gpu.hf.HF_Q_ABSORBED_TOKENS) == ora.absorbed_tokens
        S, z = gpu.state()
        assert ora.absorbed_tokens > 0
        assert hz.rel_l2(S, ora.S) <= hz.STATE_REL_L2 and hz.rel_l2(z, ora.z) <= hz.STATE_REL_L2
        assert gpu.ctx.hf_get_device_status() == (0, 0)
    finally:
        gpu.close()


@pytest.mark.parametrize("d,b,tpf,cf,wf,zmean", [
    (128, 128, 150, 2, 4, False),   # 300-token chunks (ragged tiles), one cached chunk
    (64, 64, 100, 1, 2, True),      # head_dim 64, per-frame-mean normaliser, odd tile tails
])
def test_rotation_inside_the_linear_branch(d, b, tpf, cf, wf, zmean):
    """hf_set_rope: RoPE(phi(K)) in the state (Eq. 3), RoPE(phi(Q)) in the numerator only (Eq. 4), seeded angle
    tables as inputs; state, read-out and hybrid output against the oracle run the same way."""
    w = gen.Workload("rope", batch=1, heads=3, head_dim=d, tokens_per_frame=tpf, chunk_frames=cf, window_frames=wf,
                     block=b, topk=0, keep_permille=500, seed=18)
    gpu = hz.GpuStream(w, rope=True, z_frame_mean=zmean); ora = hz.make_oracle(w, rope=True, z_frame_mean=zmean)
    try:
        for c in range(wf // cf + 2):
            kc, vc = gen.clean_kv(w, 0, c)
            gpu.append(gpu.up(kc), gpu.up(vc)); ora.append(f64(kc), f64(vc))
        assert ora.absorbed_tokens == 3 * w.chunk_tokens
        S, z = gpu.state()
        assert hz.rel_l2(S, ora.S) <= hz.STATE_REL_L2, f"S rel-L2 {hz.rel_l2(S, ora.S):.3e}"
        assert hz.rel_l2(z, ora.z) <= hz.STATE_REL_L2
        qb, kb, vb = gen.qkv(w, 0, 9, 0)
        o_ref, _, oh_ref = ora.forward(f64(qb), f64(kb), f64(vb), parts=True)
        assert hz.rel_l2(gpu.linear(gpu.up(qb)), oh_ref) <= hz.REL_L2
        o = gpu.forward(gpu.up(qb), gpu.up(kb), gpu.up(vb))
        assert hz.rel_l2(o, o_ref) <= hz.REL_L2
        assert hz.max_abs(o, o_ref) <= hz.MAX_ABS + 2.0 ** -8 * np.abs(o_ref).max()
        # the rotation matters: without the tables the state differs
        plain = hz.make_oracle(w, z_frame_mean=zmean)
        for c in range(wf // cf + 2):
            kc, vc = gen.clean_kv(w, 0, c)
            plain.append(f64(kc), f64(vc))
        assert hz.rel_l2(S, plain.S) > 0.1
    finally:
        gpu.close()


def test_maximum_number_of_key_blocks_per_row():
    """The largest selection row the library accepts: 8 chunks x 128 blocks = 1024 key blocks (16-token blocks)."""
    w = gen.Workload("maxtn", batch=1, heads=1, head_dim=64, tokens_per_frame=2048, chunk_frames=1, window_frames=8,
                     block=16, topk=0, keep_permille=30, seed=19)
    gpu = hz.GpuStream(w, merge=False); ora = hz.make_oracle(w, merge=False)
    try:
        for c in range(8):
            kc, vc = gen.clean_kv(w, 0, c)
            gpu.append(gpu.up(kc), gpu.up(vc)); ora.append(f64(kc), f64(vc))
        qb, kb, vb = gen.qkv(w, 0, 8, 0)
        q, k, v = gpu.up(qb), gpu.up(kb), gpu.up(vb)
        assert gpu.ctx.hf_query(0, gpu.hf.HF_Q_KEY_BLOCKS) == 1024 and gpu.ctx.hf_query(0, gpu.hf.HF_Q_KEPT_BLOCKS) == 31
        m_gpu, idx_gpu, sc_gpu = gpu.select(q, k)
        m_ref, sc_ref = ora.select(f64(qb), f64(kb))
        assert m_ref.shape == (1, 1, 128, 1024)
        assert np.array_equal(sc_gpu, sc_ref) and np.array_equal(m_gpu, m_ref)
        qbl = [0, 63, 127]
        o_ref = ora.forward(f64(qb), f64(kb), f64(vb), mask=m_ref, q_blocks=qbl)
        hz.assert_close_out(gpu.forward(q, k, v), o_ref, "1024 key blocks")
    finally:
        gpu.close()


def test_empty_token_range_is_refused_without_a_launch():
    import torch
    w = gen.tiny()
    gpu = hz.GpuStream(w)
    try:
        t = torch.zeros((1, 2, 64, 64), dtype=torch.bfloat16, device="cuda")
        n0 = gpu.ctx.hf_launch_count()
        with pytest.raises(gpu.hf.HFError, match="HF_ERR_SHAPE"):
            gpu.ctx.hf_state_absorb(0, t, t, 0)
        assert gpu.ctx.hf_launch_count() == n0
    finally:
        gpu.close()


@pytest.mark.parametrize("d,b,tpf,kernel", [(64, 16, 64, 0), (128, 128, 200, 0), (128, 128, 200, 3)])
def test_block_indices_outside_the_cache_are_caught_on_the_device(d, b, tpf, kernel):
    """An index list is device memory the host never sees: every kernel checks each entry against [0, T_n), reads block 0
    in its place and reports through the status word; the next call with a valid list is right again."""
    import torch
    w = gen.Workload("badidx", batch=1, heads=2, head_dim=d, tokens_per_frame=tpf, chunk_frames=1, window_frames=3,
                     block=b, topk=2, keep_permille=0, seed=23)
    gpu = hz.GpuStream(w, swa_kernel=kernel); ora = hz.make_oracle(w)
    try:
        for c in range(3):
            kc, vc = gen.clean_kv(w, 0, c)
            gpu.append(gpu.up(kc), gpu.up(vc)); ora.append(f64(kc), f64(vc))
        qb, kb, vb = gen.qkv(w, 0, 3, 0)
        q, k, v = gpu.up(qb), gpu.up(kb), gpu.up(vb)
        m_gpu, idx, _ = gpu.select(q, k)
        tn = gpu.ctx.hf_query(0, gpu.hf.HF_Q_KEY_BLOCKS)
        for bad in (tn, -1, 2 ** 30, -2 ** 31):
            wrong = idx.copy()
            wrong[0, 1, -1, 1] = bad
            gpu.swa(q, k, v, idx=torch.from_numpy(wrong).cuda())
            with pytest.raises(gpu.hf.HFError, match="HF_ERR_INVALID_ARG"):
                gpu.ctx.hf_get_device_status()
            assert gpu.ctx.hf_get_device_status() == (0, 0)      # the word was cleared
        m_ref, _ = ora.select(f64(qb), f64(kb))
        _, ol_ref, _ = ora.forward(f64(qb), f64(kb), f64(vb), mask=m_ref, parts=True)
        hz.assert_close_out(gpu.swa(q, k, v, idx=torch.from_numpy(idx).cuda()), ol_ref, "O_local after the refused lists")
        assert gpu.ctx.hf_get_device_status() == (0, 0)
    finally:
        gpu.close()


@pytest.mark.parametrize("d,b,tpf", [(128, 128, 200), (64, 16, 64)])
def test_attention_with_history_for_a_given_selection(d, b, tpf):
    """hf_sparse_swa_merged on the context's last selection gives the bits hf_hybrid_forward gives (one kernel at
    head_dim 128 with 128-token blocks, read-out + attention otherwise), and the oracle's output."""
    import torch
    w = gen.Workload("merged", batch=1, heads=2, head_dim=d, tokens_per_frame=tpf, chunk_frames=1, window_frames=3,
                     block=b, topk=2, keep_permille=0, seed=29)
    gpu = hz.GpuStream(w); ora = hz.make_oracle(w)
    try:
        for c in range(4):
            kc, vc = gen.clean_kv(w, 0, c)
            gpu.append(gpu.up(kc), gpu.up(vc)); ora.append(f64(kc), f64(vc))
        qb, kb, vb = gen.qkv(w, 0, 4, 0)
        q, k, v = gpu.up(qb), gpu.up(kb), gpu.up(vb)
        o_fwd = gpu.forward(q, k, v)
        m_gpu, idx, _ = gpu.select(q, k)
        o = torch.empty(gpu.shape, dtype=torch.bfloat16, device="cuda")
        gpu.ctx.hf_sparse_swa_merged(0, q, k, v, o)
        torch.cuda.synchronize()
        assert np.array_equal(gpu.f64(o), o_fwd)
        o2 = torch.empty_like(o)
        gpu.ctx.hf_sparse_swa_merged(0, q, k, v, o2, idx=torch.from_numpy(idx).cuda())
        torch.cuda.synchronize()
        assert np.array_equal(gpu.f64(o2), o_fwd)
        m_ref, _ = ora.select(f64(qb), f64(kb))
        hz.assert_close_out(o_fwd, ora.forward(f64(qb), f64(kb), f64(vb), mask=m_ref), "merged output")
        assert gpu.ctx.hf_get_device_status() == (0, 0)
    finally:
        gpu.close()


@pytest.mark.parametrize("topk,wf", [(1, 3), (2, 2), (3, 1)])
def test_one_kernel_forward_with_few_kept_blocks_and_several_units_per_cta(topk, wf):
    """The attention kernel with the history term inside, in the corners of its unit bookkeeping: one, two or three
    kept tiles per query block (the S buffer taken for the phi(Q) operand is then the previous unit's), more
    (head, query block) units than SMs, so that thread blocks walk several units, and a short last block."""
    w = gen.Workload("fewkept", batch=2, heads=8, head_dim=128, tokens_per_frame=1300, chunk_frames=1, window_frames=wf,
                     block=128, topk=topk, keep_permille=0, seed=31)
    assert w.batch * w.heads * w.blocks_per_chunk > 148
    stream_compare(w, wf + 2, check_parts=False)


def test_lse_output_of_the_tcgen05_kernel():
    """Natural-log sum of exponentials per query row from the fixed-reference kernel (reference exponent + log2 of the
    row sum, which is of the order 2^-60 there)."""
    w = gen.Workload("lse128", batch=1, heads=2, head_dim=128, tokens_per_frame=200, chunk_frames=1, window_frames=2,
                     block=128, topk=2, keep_permille=0, seed=43)
    gpu = hz.GpuStream(w)
    try:
        kc, vc = gen.clean_kv(w, 0, 0)
        gpu.append(gpu.up(kc), gpu.up(vc))
        qb, kb, vb = gen.qkv(w, 0, 1, 0)
        q, k, v = gpu.up(qb), gpu.up(kb), gpu.up(vb)
        m, idx, _ = gpu.select(q, k)
        o, lse = gpu.swa(q, k, v, want_lse=True)
        qf = f64(qb); keys = np.concatenate([f64(kc), f64(kb)], axis=2)       # logical order: cached chunk, current chunk
        nb = w.blocks_per_chunk
        for h in range(2):
            for i in range(nb):
                cols = []
                for j in idx[0, h, i]:
                    c, jb = divmod(int(j), nb)
                    lo = c * w.chunk_tokens + jb * 128
                    cols.append(np.arange(lo, min(lo + 128, (c + 1) * w.chunk_tokens)))
                cols = np.concatenate(cols)
                rows = slice(i * 128, min((i + 1) * 128, w.chunk_tokens))
                s = qf[0, h, rows] @ keys[0, h, cols].T / np.sqrt(128.0)
                ref = np.log(np.exp(s - s.max(axis=1, keepdims=True)).sum(axis=1)) + s.max(axis=1)
                assert np.abs(lse[0, h, rows] - ref).max() < 2e-3
    finally:
        gpu.close()


@pytest.mark.parametrize("d,b,tpf,heads,batch,bias", [(128, 128, 300, 3, 2, True), (64, 16, 64, 2, 1, True), (64, 128, 200, 4, 1, False)])
def test_full_width_merge_projection(d, b, tpf, heads, batch, bias):
    """Eq. 4's Linear read as one [H d, H d] matrix over all heads: read-out (bf16 hi + lo) -> projection kernel ->
    history term, against the oracle; hf_linear_attn alone and the whole forward, over a stream with evictions."""
    w = gen.Workload("fullw", batch=batch, heads=heads, head_dim=d, tokens_per_frame=tpf, chunk_frames=1, window_frames=2,
                     block=b, topk=0, keep_permille=500, seed=47)
    gpu = hz.GpuStream(w, merge_full=True, bias=bias); ora = hz.make_oracle(w, merge_full=True, bias=bias)
    try:
        for c in range(4):
            qb, kb, vb = gen.qkv(w, 0, c, 0)
            q, k, v = gpu.up(qb), gpu.up(kb), gpu.up(vb)
            m_gpu, _, _ = gpu.select(q, k)
            m_ref, _ = ora.select(f64(qb), f64(kb))
            assert np.array_equal(m_gpu, m_ref)
            o_ref, _, oh_ref = ora.forward(f64(qb), f64(kb), f64(vb), mask=m_ref, parts=True)
            hz.assert_close_out(gpu.forward(q, k, v), o_ref, f"chunk {c} hybrid O, full-width merge")
            hz.assert_close_out(gpu.linear(q), oh_ref, f"chunk {c} O_history, full-width merge")
            kc, vc = gen.clean_kv(w, 0, c)
            gpu.append(gpu.up(kc), gpu.up(vc)); ora.append(f64(kc), f64(vc))
        assert gpu.ctx.hf_get_device_status() == (0, 0)
    finally:
        gpu.close()
