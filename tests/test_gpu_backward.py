"""The backward pass (training rollout's step with gradient, Alg. 1): dq, and dk / dv of the current chunk, of the
block-sparse attention from the tcgen05 kernels against the oracle's gradients (themselves pinned by finite differences and
autograd)."""
import numpy as np
import pytest

from oracle import hybrid_attention as oa
from paper_2604_10103_b200 import inputs as gen
from tests import harness as hz

pytestmark = pytest.mark.gpu

f64 = gen.bf16_bits_to_f64


@pytest.mark.parametrize("d,tpf,wf,permille,heads,batch", [
    (128, 300, 3, 500, 2, 1),      # two cached chunks, 44-token tail blocks
    (64, 200, 2, 1000, 3, 2),      # head_dim 64, every block kept
    (128, 1300, 2, 150, 8, 2),     # more units than SMs (several units per thread block), sparse lists
])
def test_gradients_of_the_sparse_branch(d, tpf, wf, permille, heads, batch):
    import torch
    w = gen.Workload("bwd", batch=batch, heads=heads, head_dim=d, tokens_per_frame=tpf, chunk_frames=1, window_frames=wf,
                     block=128, topk=0, keep_permille=permille, seed=101)
    gpu = hz.GpuStream(w); ora = hz.make_oracle(w)
    try:
        for c in range(wf + 1):
            kc, vc = gen.clean_kv(w, 0, c)
            gpu.append(gpu.up(kc), gpu.up(vc)); ora.append(f64(kc), f64(vc))
        qb, kb, vb = gen.qkv(w, 0, wf + 1, 0)
        gb = gen.normal_bf16(qb.shape, 101, 7, 7)
        q, k, v, g = gpu.up(qb), gpu.up(kb), gpu.up(vb), gpu.up(gb)
        m_gpu, _, _ = gpu.select(q, k)
        m_ref, _ = ora.select(f64(qb), f64(kb))
        assert np.array_equal(m_gpu, m_ref)
        o = torch.empty(gpu.shape, dtype=torch.bfloat16, device="cuda")
        lse = torch.empty(gpu.shape[:3], dtype=torch.float32, device="cuda")
        gpu.ctx.hf_sparse_swa(0, q, k, v, o, lse=lse)
        dq = torch.empty_like(o)
        gpu.ctx.hf_sparse_swa_backward_dq(0, q, k, v, o, lse, g, dq)
        torch.cuda.synchronize()
        got = gpu.f64(dq)
        ref = np.empty_like(got)
        held = ora.sink + ora.past
        for bi in range(batch):
            for h in range(heads):
                kc_ = [kp[bi, h] for kp, _ in held] + [f64(kb)[bi, h]]
                vc_ = [vp[bi, h] for _, vp in held] + [f64(vb)[bi, h]]
                ref[bi, h] = oa.sparse_attention_backward(f64(qb)[bi, h], kc_, vc_, w.block, m_ref[bi, h], f64(gb)[bi, h])[0]
        rl = hz.rel_l2(got, ref); ma = hz.max_abs(got, ref)
        assert rl <= 1e-2 and ma <= 2e-2 * max(1.0, np.abs(ref).max()), f"dq: rel-L2 {rl:.3e}, max-abs {ma:.3e} (max |dq| {np.abs(ref).max():.3f})"
        # dk, dv of the current chunk (the transposed walk over the selection's bit mask)
        dk = torch.empty_like(o); dv = torch.empty_like(o)
        gpu.ctx.hf_sparse_swa_backward_dkv(0, q, k, v, o, lse, g, dk, dv)
        torch.cuda.synchronize()
        got_k, got_v = gpu.f64(dk), gpu.f64(dv)
        ref_k = np.empty_like(got_k); ref_v = np.empty_like(got_v)
        for bi in range(batch):
            for h in range(heads):
                kc_ = [kp[bi, h] for kp, _ in held] + [f64(kb)[bi, h]]
                vc_ = [vp[bi, h] for _, vp in held] + [f64(vb)[bi, h]]
                _, dks, dvs = oa.sparse_attention_backward(f64(qb)[bi, h], kc_, vc_, w.block, m_ref[bi, h], f64(gb)[bi, h])
                ref_k[bi, h] = dks[-1]; ref_v[bi, h] = dvs[-1]
        for name, a_, b_ in (("dk", got_k, ref_k), ("dv", got_v, ref_v)):
            rl = hz.rel_l2(a_, b_); ma = hz.max_abs(a_, b_)
            assert rl <= 1e-2 and ma <= 2e-2 * max(1.0, np.abs(b_).max()), f"{name}: rel-L2 {rl:.3e}, max-abs {ma:.3e} (max {np.abs(b_).max():.3f})"
        unkept = ~m_ref[..., -w.blocks_per_chunk:].any(axis=2)           # [B, H, n_b]: key blocks of the current chunk nobody keeps
        for bi, h, jb in zip(*np.nonzero(unkept)):
            assert not got_k[bi, h, jb * 128:(jb + 1) * 128].any() and not got_v[bi, h, jb * 128:(jb + 1) * 128].any()
        assert gpu.ctx.hf_get_device_status() == (0, 0)
    finally:
        gpu.close()


@pytest.mark.parametrize("d,tpf,heads,batch,merge", [
    (128, 300, 2, 1, True),        # per-head Linear folded into the state; 44-token tail tile
    (64, 200, 3, 2, True),         # head_dim 64
    (128, 1300, 8, 2, False),      # identity merge; several tiles per thread block, a new head in the middle of a range
])
def test_gradient_of_the_history_readout(d, tpf, heads, batch, merge):
    """dq of Eq. 4 (u = S' g on the tensor cores, then the quotient rule per row) against the oracle's read-out gradient."""
    import torch
    w = gen.Workload("bwdh", batch=batch, heads=heads, head_dim=d, tokens_per_frame=tpf, chunk_frames=1, window_frames=2,
                     block=128, topk=0, keep_permille=500, seed=103)
    gpu = hz.GpuStream(w, merge=merge); ora = hz.make_oracle(w, merge=merge)
    try:
        for c in range(4):                         # three chunks absorbed
            kc, vc = gen.clean_kv(w, 0, c)
            gpu.append(gpu.up(kc), gpu.up(vc)); ora.append(f64(kc), f64(vc))
        assert ora.absorbed_tokens == 3 * tpf
        qb, _, _ = gen.qkv(w, 0, 5, 0)
        gb = gen.normal_bf16(qb.shape, 103, 7, 7)
        q, g = gpu.up(qb), gpu.up(gb)
        dq = torch.empty_like(q)
        gpu.ctx.hf_linear_attn_backward_dq(0, q, g, dq)
        torch.cuda.synchronize()
        got = gpu.f64(dq)
        ref = np.empty_like(got)
        for bi in range(batch):
            for h in range(heads):
                ref[bi, h] = oa.linear_readout_backward(f64(qb)[bi, h], ora.S[bi, h], ora.z[bi, h], f64(gb)[bi, h],
                                                        W=None if ora.W is None else ora.W[h], eps=ora.eps)[0]
        rl = hz.rel_l2(got, ref); ma = hz.max_abs(got, ref)
        assert rl <= 1e-2 and ma <= 2e-2 * max(1.0, np.abs(ref).max()), f"dq_hist: rel-L2 {rl:.3e}, max-abs {ma:.3e} (max {np.abs(ref).max():.3e})"
        assert gpu.ctx.hf_get_device_status() == (0, 0)
    finally:
        gpu.close()
