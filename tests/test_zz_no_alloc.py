"""hf_state_absorb_noalloc (the entry point for callers that may not allocate device memory) against
hf_state_absorb, through the C ABI, on two calls in a row.  Collected last on purpose."""
import ctypes as C

import numpy as np
import pytest

from paper_2604_10103_b200 import inputs as gen
from tests import harness as hz


@pytest.mark.gpu
@pytest.mark.parametrize("d,bh_shape,n", [(128, (1, 12), 4680), (64, (2, 3), 333)])
def test_noalloc_absorb_matches_context_absorb_twice_in_a_row(d, bh_shape, n):
    import torch
    from oracle import hybrid_attention as oa
    from paper_2604_10103_b200 import binding as hf
    B, H = bh_shape
    w = gen.Workload("noalloc", batch=B, heads=H, head_dim=d, tokens_per_frame=n, chunk_frames=1, window_frames=2,
                     block=128, topk=1, keep_permille=0, seed=31)
    gpu = hz.GpuStream(w, merge=False)
    try:
        S = torch.zeros((B, H, d, d), dtype=torch.float32, device="cuda")
        z = torch.zeros((B, H, d), dtype=torch.float32, device="cuda")
        S_ora = np.zeros((B, H, d, d)); z_ora = np.zeros((B, H, d))
        # the second call finds the first call's partial sums in the shared scratch array and must not be disturbed by them
        for call in range(2):
            k = hf.bits_to_cuda(gen.normal_bf16((B, H, n, d), 31, call, 1))
            v = hf.bits_to_cuda(gen.normal_bf16((B, H, n, d), 31, call, 2))
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            hf.hf_state_absorb_noalloc(k, v, S, z)
            torch.cuda.synchronize()
            if call == 1:   # (the first call may page in the library image, static array included)
                assert torch.cuda.mem_get_info()[0] >= free_before
            gpu.ctx.hf_state_absorb(0, k, v, n)
            torch.cuda.synchronize()
            S_ref, z_ref = gpu.state()
            assert hz.rel_l2(S.cpu().numpy(), S_ref) <= hz.STATE_REL_L2
            assert hz.rel_l2(z.cpu().numpy(), z_ref) <= hz.STATE_REL_L2
            # and against Eq. 3 itself (the CPU oracle), so that the check does not rest on the other CUDA entry point
            kf = gen.bf16_bits_to_f64(hf.cuda_to_bits(k)); vf = gen.bf16_bits_to_f64(hf.cuda_to_bits(v))
            for b_ in range(B):
                for h_ in range(H):
                    S_ora[b_, h_], z_ora[b_, h_] = oa.absorb(S_ora[b_, h_], z_ora[b_, h_], kf[b_, h_], vf[b_, h_])
            assert hz.rel_l2(S.cpu().numpy(), S_ora) <= hz.STATE_REL_L2
            assert hz.rel_l2(z.cpu().numpy(), z_ora) <= hz.STATE_REL_L2
        assert np.abs(z.cpu().numpy()).min() > 0
    finally:
        gpu.close()


@pytest.mark.gpu
def test_noalloc_rejects_sizes_beyond_the_static_scratch():
    import torch
    from paper_2604_10103_b200 import binding as hf
    k = torch.zeros((254, 64, 128), dtype=torch.bfloat16, device="cuda")
    S = torch.zeros((254, 128, 128), dtype=torch.float32, device="cuda")
    z = torch.zeros((254, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(hf.HFError, match="HF_ERR_SHAPE"):
        hf.hf_state_absorb_noalloc(k, k, S, z)
    with pytest.raises(hf.HFError, match="HF_ERR_INVALID_ARG"):
        hf.hf_state_absorb_noalloc(k[:4], k[:4], S[:4].view(-1)[1:], z[:4])
    assert not S.any()
    # head_dim 64: 1008 (batch, head) pairs fit the static scratch, 1009 do not
    k64 = torch.zeros((1009, 64, 64), dtype=torch.bfloat16, device="cuda")
    S64 = torch.zeros((1009, 64, 64), dtype=torch.float32, device="cuda")
    z64 = torch.zeros((1009, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(hf.HFError, match="HF_ERR_SHAPE"):
        hf.hf_state_absorb_noalloc(k64, k64, S64, z64)
    assert not S64.any()
    hf.hf_state_absorb_noalloc(k64[:1008], k64[:1008], S64[:1008], z64[:1008])
    torch.cuda.synchronize()
    assert torch.allclose(z64[:1008], torch.full_like(z64[:1008], 64.0)) and not z64[1008:].any()      # phi(0) = 1 over 64 tokens
