"""Blocks of 16 and 64 tokens on the tcgen05 attention path (several query blocks share a 128-row tile, several key blocks
a 128-key tile, with per-(query block, key block) masking): against the oracle and against the warp-level kernel."""
import numpy as np
import pytest

from paper_2604_10103_b200 import inputs as gen
from tests import harness as hz
from tests.test_gpu_parity import stream_compare

pytestmark = pytest.mark.gpu

f64 = gen.bf16_bits_to_f64


def test_small_blocks_resolve_to_the_tcgen05_kernel():
    from paper_2604_10103_b200 import binding as hf
    for b in (16, 64, 128):
        w = gen.tiny().with_(block=b)
        ctx = hf.Context(hf.make_config(w))
        try:
            assert ctx.hf_query(0, hf.HF_Q_SWA_KERNEL) == hf.HF_SWA_TCGEN05
        finally:
            ctx.close()
    ctx = hf.Context(hf.make_config(gen.tiny(), swa_kernel=hf.HF_SWA_MMA))
    try:
        assert ctx.hf_query(0, hf.HF_Q_SWA_KERNEL) == hf.HF_SWA_MMA
    finally:
        ctx.close()


@pytest.mark.parametrize("d,b,tpf,cf,wf,B,H,permille", [
    (64, 16, 64, 1, 3, 1, 2, 170),       # the tiny configuration's shape (top-2 of 12)
    (128, 64, 1560, 1, 3, 1, 3, 250),    # 25 query blocks of 64 (24 full + 24 tokens): units of two query blocks, ragged last unit
    (64, 64, 1000, 1, 8, 2, 2, 100),     # seven cached chunks, sparse lists: tiles with a single useful block
    (128, 16, 300, 1, 3, 1, 2, 500),     # 19 query blocks of 16: last unit holds 3 of 8 row groups, 12-token tail block
    (64, 16, 520, 1, 2, 1, 3, 1000),     # everything kept: every tile fully used
    (128, 64, 200, 1, 1, 1, 2, 1000),    # window == chunk
])
def test_small_block_streams(d, b, tpf, cf, wf, B, H, permille):
    w = gen.Workload("smallblk", batch=B, heads=H, head_dim=d, tokens_per_frame=tpf, chunk_frames=cf, window_frames=wf,
                     block=b, topk=0, keep_permille=permille, seed=81)
    stream_compare(w, wf // cf + 2)


@pytest.mark.parametrize("d,b", [(128, 64), (64, 16)])
def test_more_units_than_sms_and_top1(d, b):
    """Several units per thread block (the tile counts differ from unit to unit), one kept block per query block."""
    w = gen.Workload("smallblk_many", batch=2, heads=6, head_dim=d, tokens_per_frame=2000, chunk_frames=1, window_frames=3,
                     block=b, topk=1, keep_permille=0, seed=82)
    assert w.batch * w.heads * -(-w.chunk_tokens // 128) > 148
    stream_compare(w, 4, check_parts=False)


def test_caller_supplied_lists_and_bad_indices():
    """hf_sparse_swa with the caller's own lists: equal to the warp-level kernel on the same lists; an index outside the
    window is caught by the list builder and reported."""
    import torch
    w = gen.Workload("smallblk_idx", batch=1, heads=2, head_dim=128, tokens_per_frame=400, chunk_frames=1, window_frames=3,
                     block=64, topk=3, keep_permille=0, seed=83)
    a = hz.GpuStream(w); b_ = hz.GpuStream(w, swa_kernel=1)
    try:
        for c in range(3):
            kc, vc = gen.clean_kv(w, 0, c)
            for g in (a, b_):
                g.append(g.up(kc), g.up(vc))
        qb, kb, vb = gen.qkv(w, 0, 3, 0)
        q, k, v = a.up(qb), a.up(kb), a.up(vb)
        tn = a.ctx.hf_query(0, a.hf.HF_Q_KEY_BLOCKS)
        rng = np.random.default_rng(5)
        idx = np.stack([np.sort(rng.choice(tn, size=3, replace=False)) for _ in range(2 * 7)]).reshape(1, 2, 7, 3).astype(np.int32)
        it = torch.from_numpy(idx).cuda()
        oa_ = a.swa(q, k, v, idx=it); ob = b_.swa(q, k, v, idx=it)
        assert hz.max_abs(oa_, ob) <= 2e-2 and hz.rel_l2(oa_, ob) <= 5e-3
        bad = idx.copy(); bad[0, 1, 3, 2] = tn
        a.swa(q, k, v, idx=torch.from_numpy(bad).cuda())
        with pytest.raises(a.hf.HFError, match="HF_ERR_INVALID_ARG"):
            a.ctx.hf_get_device_status()
        assert a.ctx.hf_get_device_status() == (0, 0)
    finally:
        a.close(); b_.close()
