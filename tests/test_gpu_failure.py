"""Failure detection on the device without a fault: a bounded wait that runs out must come back as a status, and the
context must stay usable."""
import numpy as np
import pytest

from paper_2604_10103_b200 import inputs as gen
from tests import harness as hz

pytestmark = pytest.mark.gpu

f64 = gen.bf16_bits_to_f64


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    """hf_selftest_wait_limit waits (about a millisecond) on a barrier nothing arrives on, through the same wait routine
    the kernels use: the status word must report the timeout with the kernel's location code, be cleared by the read,
    and a forward pass afterwards must match the oracle."""
    w = gen.Workload("wait", batch=1, heads=2, head_dim=128, tokens_per_frame=300, chunk_frames=1, window_frames=2,
                     block=128, topk=0, keep_permille=500, seed=61)
    gpu = hz.GpuStream(w); ora = hz.make_oracle(w)
    try:
        for c in range(3):
            kc, vc = gen.clean_kv(w, 0, c)
            gpu.append(gpu.up(kc), gpu.up(vc)); ora.append(f64(kc), f64(vc))
        assert gpu.ctx.hf_get_device_status() == (0, 0)
        for _ in range(2):
            gpu.ctx.hf_selftest_wait_limit()
            with pytest.raises(gpu.hf.HFError, match="HF_ERR_DEVICE_TIMEOUT") as e:
                gpu.ctx.hf_get_device_status()
            assert "detail 77" in str(e.value)
            assert gpu.ctx.hf_get_device_status() == (0, 0)          # cleared by the read
        qb, kb, vb = gen.qkv(w, 0, 3, 0)
        q, k, v = gpu.up(qb), gpu.up(kb), gpu.up(vb)
        m_gpu, _, _ = gpu.select(q, k)
        m_ref, _ = ora.select(f64(qb), f64(kb))
        assert np.array_equal(m_gpu, m_ref)
        hz.assert_close_out(gpu.forward(q, k, v), ora.forward(f64(qb), f64(kb), f64(vb), mask=m_ref), "forward after the timeout")
        S, z = gpu.state()
        assert hz.rel_l2(S, ora.S) <= hz.STATE_REL_L2
        assert gpu.ctx.hf_get_device_status() == (0, 0)
    finally:
        gpu.close()
