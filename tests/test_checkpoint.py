"""Checkpoint / resume of the streaming state (rolling cache + linear state, Alg. 2's KV and LN): a stream that is
exported, imported into a fresh context and continued gives bit-for-bit what the uninterrupted stream gives; images
that do not fit the context are refused with nothing changed.  Host-only argument checks run without a device."""
import ctypes as C

import numpy as np
import pytest

from paper_2604_10103_b200 import binding as hf, build as hfbuild, inputs as gen
from tests import harness as hz


def test_null_arguments_need_no_device():
    hfbuild.build()
    lib = hf.lib()
    n = C.c_size_t(0)
    assert lib.hf_state_export(None, None, C.byref(n)) == 1
    assert lib.hf_state_import(None, None, 0) == 1


def _run(w, chunks, split_at=None, sink_chunks=0, rope=False):
    """One forward + one append per chunk; with split_at the context is replaced by a fresh one that imports the
    image of the old one after that many chunks.  Returns every output, the final state and the image size."""
    gpu = hz.GpuStream(w, sink_chunks=sink_chunks, rope=rope)
    outs, image_bytes = [], 0
    try:
        for c in range(chunks):
            if split_at is not None and c == split_at:
                image = gpu.ctx.hf_state_export()
                image_bytes = image.nbytes
                gpu.close()
                gpu = hz.GpuStream(w, sink_chunks=sink_chunks, rope=rope)
                gpu.ctx.hf_state_import(image)
            qb, kb, vb = gen.qkv(w, 0, c, 0)
            outs.append(gpu.forward(gpu.up(qb), gpu.up(kb), gpu.up(vb)))
            kc, vc = gen.clean_kv(w, 0, c)
            gpu.append(gpu.up(kc), gpu.up(vc))
        S, z = gpu.state()
        counts = (gpu.ctx.hf_query(0, hf.HF_Q_CACHED_CHUNKS), gpu.ctx.hf_query(0, hf.HF_Q_ABSORBED_TOKENS),
                  gpu.ctx.hf_query(0, hf.HF_Q_SINK_CHUNKS))
        assert gpu.ctx.hf_get_device_status() == (0, 0)
    finally:
        gpu.close()
    return outs, S, z, counts, image_bytes


@pytest.mark.gpu
@pytest.mark.parametrize("split_at, sink, rope", [(10, 0, False), (1, 0, False), (5, 1, False), (7, 0, True)])
def test_resume_is_bit_for_bit(split_at, sink, rope):
    # 10 chunks, export, import into a fresh context, 10 more: the ring of the second context starts at slot 0, the
    # first one's had rotated, and nothing the caller can see may depend on that
    w = gen.tiny().with_(seed=77)
    chunks = 20
    whole = _run(w, chunks, None, sink, rope)
    resumed = _run(w, chunks, split_at, sink, rope)
    assert resumed[4] > 0
    for c, (a, b) in enumerate(zip(whole[0], resumed[0])):
        assert np.array_equal(a, b), f"chunk {c}: outputs differ after the resume"
    assert np.array_equal(whole[1], resumed[1]) and np.array_equal(whole[2], resumed[2])
    assert whole[3] == resumed[3]


@pytest.mark.gpu
def test_resume_with_ragged_blocks_and_several_layers():
    w = gen.tiny().with_(seed=5, tokens_per_frame=72, block=64, head_dim=128, heads=3, layers=2)
    import torch

    def stream(split_at):
        cfg = hf.make_config(w)
        ctx = hf.Context(cfg)
        outs = []
        shape = (w.batch, w.heads, w.chunk_tokens, w.head_dim)

        def weights(cx):
            for l in range(2):
                Wb, bb = gen.merge_weights(w, l)
                cx.hf_set_merge_weights(l, hf.bits_to_cuda(Wb), hf.bits_to_cuda(bb))
        weights(ctx)
        try:
            for c in range(8):
                if c == split_at:
                    image = ctx.hf_state_export()
                    ctx.close()
                    ctx = hf.Context(cfg)
                    ctx.hf_state_import(image)      # before the weights: setting them refolds the restored state
                    weights(ctx)
                for l in range(2):
                    qb, kb, vb = gen.qkv(w, l, c, 0)
                    o = torch.empty(shape, dtype=torch.bfloat16, device="cuda")
                    ctx.hf_hybrid_forward(l, hf.bits_to_cuda(qb), hf.bits_to_cuda(kb), hf.bits_to_cuda(vb), o)
                    torch.cuda.synchronize()
                    outs.append(hf.cuda_to_bits(o))
                    kc, vc = gen.clean_kv(w, l, c)
                    ctx.hf_kv_append(l, hf.bits_to_cuda(kc), hf.bits_to_cuda(vc))
            torch.cuda.synchronize()
        finally:
            ctx.close()
        return outs

    a, b = stream(None), stream(5)
    assert len(a) == len(b) == 16
    for i, (x, y) in enumerate(zip(a, b)):
        assert np.array_equal(x, y), f"call {i}"


@pytest.mark.gpu
def test_images_that_do_not_fit_are_refused_and_change_nothing():
    w = gen.tiny().with_(seed=3)
    gpu = hz.GpuStream(w)
    other = hz.GpuStream(w.with_(heads=w.heads + 1))
    try:
        for c in range(5):
            kc, vc = gen.clean_kv(w, 0, c)
            gpu.append(gpu.up(kc), gpu.up(vc))
        image = gpu.ctx.hf_state_export()
        S0, z0 = gpu.state()
        # size query, then a buffer that is too small: the needed size comes back, status HF_ERR_SHAPE
        n = C.c_size_t(0)
        assert hf.lib().hf_state_export(gpu.ctx._h, None, C.byref(n)) == 0 and n.value == image.nbytes
        small = np.empty(16, dtype=np.uint8)
        n = C.c_size_t(16)
        assert hf.lib().hf_state_export(gpu.ctx._h, C.c_void_p(small.ctypes.data), C.byref(n)) == 2 and n.value == image.nbytes
        # another configuration
        with pytest.raises(hf.HFError, match="HF_ERR_SHAPE"):
            other.ctx.hf_state_import(image)
        # not an image / cut short / inconsistent counts
        junk = image.copy(); junk[0] ^= 0xFF
        with pytest.raises(hf.HFError, match="HF_ERR_INVALID_ARG"):
            gpu.ctx.hf_state_import(junk)
        with pytest.raises(hf.HFError, match="HF_ERR_INVALID_ARG"):
            gpu.ctx.hf_state_import(np.ascontiguousarray(image[: image.nbytes // 2]))
        # the refusals left the context as it was
        S1, z1 = gpu.state()
        assert np.array_equal(S0, S1) and np.array_equal(z0, z1)
        assert gpu.ctx.hf_query(0, hf.HF_Q_CACHED_CHUNKS) == 2
        # and the image itself goes back in
        gpu.ctx.hf_reset()
        assert gpu.ctx.hf_query(0, hf.HF_Q_CACHED_CHUNKS) == 0
        gpu.ctx.hf_state_import(image)
        S2, z2 = gpu.state()
        assert np.array_equal(S0, S2) and np.array_equal(z0, z2)
        assert gpu.ctx.hf_query(0, hf.HF_Q_CACHED_CHUNKS) == 2
        assert gpu.ctx.hf_query(0, hf.HF_Q_ABSORBED_TOKENS) == 3 * w.chunk_tokens
    finally:
        gpu.close()
        other.close()
