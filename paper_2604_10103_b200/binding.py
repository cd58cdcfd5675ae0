"""ctypes binding of libhf.so: same names as the C ABI, argument marshalling only.

Tensors are torch CUDA tensors (bf16 unless noted); only their data pointers and the current
CUDA stream cross the boundary.  Every step of the path runs in the library's kernels; if the
library is missing this module raises -- there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libhf.so")

HF_OK = 0
STATUS_NAMES = ["HF_OK", "HF_ERR_INVALID_ARG", "HF_ERR_SHAPE", "HF_ERR_STATE", "HF_ERR_UNSUPPORTED",
                "HF_ERR_NOMEM", "HF_ERR_CUDA", "HF_ERR_DEVICE_TIMEOUT"]
HF_PHI_ELU1 = 0
HF_MERGE_IDENTITY, HF_MERGE_PER_HEAD, HF_MERGE_FULL_WIDTH = 0, 1, 2
HF_SWA_AUTO, HF_SWA_MMA, HF_SWA_TCGEN05, HF_SWA_TCGEN05_PINGPONG = 0, 1, 2, 3
HF_Z_SUM, HF_Z_FRAME_MEAN = 0, 1
(HF_Q_CACHED_CHUNKS, HF_Q_KEY_BLOCKS, HF_Q_KEPT_BLOCKS, HF_Q_ABSORBED_TOKENS, HF_Q_QUERY_BLOCKS,
 HF_Q_MASK_WORDS, HF_Q_SWA_KERNEL, HF_Q_SINK_CHUNKS) = range(8)

# every symbol include/hf.h declares
EXPORTS = [
    "hf_create", "hf_destroy", "hf_reset", "hf_set_merge_weights", "hf_kv_append", "hf_state_absorb",
    "hf_block_select", "hf_sparse_swa", "hf_linear_attn", "hf_hybrid_forward", "hf_hybrid_forward_host",
    "hf_kv_append_host", "hf_get_state", "hf_query", "hf_get_device_status", "hf_launch_count",
    "hf_status_string", "hf_last_error", "hf_state_absorb_noalloc", "hf_set_rope", "hf_state_export", "hf_state_import",
    "hf_sparse_swa_merged", "hf_slow_path_units", "hf_selftest_wait_limit", "hf_kv_append_layers", "hf_state_absorb_layers", "hf_set_temporal_rope", "hf_sparse_swa_backward_dq", "hf_sparse_swa_backward_dkv", "hf_linear_attn_backward_dq",
]


class hf_config(C.Structure):
    _fields_ = [("batch", C.c_int), ("heads", C.c_int), ("head_dim", C.c_int),
                ("tokens_per_frame", C.c_int), ("chunk_frames", C.c_int), ("window_frames", C.c_int),
                ("block", C.c_int), ("topk", C.c_int), ("keep_permille", C.c_int), ("layers", C.c_int),
                ("phi", C.c_int), ("eps", C.c_float), ("merge", C.c_int), ("swa_kernel", C.c_int), ("z_mode", C.c_int), ("sink_frames", C.c_int)]


class HFError(RuntimeError):
    def __init__(self, status: int, text: str):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{name}: {text}")


_lib = None


def lib() -> C.CDLL:
    """Load libhf.so (once).  Raises if it has not been built: the CUDA library is the only path."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2604_10103_b200.build` "
                           "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp, ip = C.c_void_p, C.c_int
    L.hf_create.argtypes = [C.POINTER(hf_config), ip, C.POINTER(vp)]
    L.hf_destroy.argtypes = [vp]
    L.hf_reset.argtypes = [vp, ip, vp]
    L.hf_set_merge_weights.argtypes = [vp, ip, vp, vp, vp]
    L.hf_set_rope.argtypes = [vp, vp, vp, vp, vp, vp]
    L.hf_set_temporal_rope.argtypes = [vp, ip, ip, ip, vp, vp, vp]
    L.hf_kv_append.argtypes = [vp, ip, vp, vp, vp]
    L.hf_state_absorb.argtypes = [vp, ip, vp, vp, ip, vp]
    L.hf_state_absorb_layers.argtypes = [vp, ip, ip, vp, vp, ip, vp]
    L.hf_kv_append_layers.argtypes = [vp, ip, ip, C.POINTER(vp), C.POINTER(vp), vp]
    L.hf_block_select.argtypes = [vp, ip, vp, vp, vp, vp, vp, vp]
    L.hf_sparse_swa.argtypes = [vp, ip, vp, vp, vp, vp, vp, vp, vp]
    L.hf_linear_attn.argtypes = [vp, ip, vp, vp, vp]
    L.hf_sparse_swa_backward_dq.argtypes = [vp, ip, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    L.hf_sparse_swa_backward_dkv.argtypes = [vp, ip, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    L.hf_linear_attn_backward_dq.argtypes = [vp, ip, vp, vp, vp, vp]
    L.hf_sparse_swa_merged.argtypes = [vp, ip, vp, vp, vp, vp, vp, vp]
    L.hf_hybrid_forward.argtypes = [vp, ip, vp, vp, vp, vp, vp]
    L.hf_hybrid_forward_host.argtypes = [vp, ip, vp, vp, vp, vp, vp]
    L.hf_kv_append_host.argtypes = [vp, ip, vp, vp, vp]
    L.hf_get_state.argtypes = [vp, ip, vp, vp, vp]
    L.hf_state_export.argtypes = [vp, vp, C.POINTER(C.c_size_t)]
    L.hf_state_import.argtypes = [vp, vp, C.c_size_t]
    L.hf_query.argtypes = [vp, ip, ip, C.POINTER(C.c_int64)]
    L.hf_get_device_status.argtypes = [vp, C.POINTER(ip), C.POINTER(ip)]
    L.hf_launch_count.argtypes = [vp, C.POINTER(C.c_int64)]
    L.hf_slow_path_units.argtypes = [vp, C.POINTER(C.c_int64)]
    L.hf_selftest_wait_limit.argtypes = [vp, vp]
    L.hf_state_absorb_noalloc.argtypes = [vp, vp, ip, ip, ip, vp, vp, vp]
    L.hf_status_string.argtypes = [ip]
    L.hf_status_string.restype = C.c_char_p
    L.hf_last_error.argtypes = []
    L.hf_last_error.restype = C.c_char_p
    for name in EXPORTS:
        if name not in ("hf_status_string", "hf_last_error"):
            getattr(L, name).restype = ip
    _lib = L
    return L


def _check(status: int):
    if status != HF_OK:
        raise HFError(status, lib().hf_last_error().decode())


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_config(w, merge: int = HF_MERGE_PER_HEAD, swa_kernel: int = HF_SWA_AUTO, z_mode: int = HF_Z_SUM,
                sink_frames: int = 0) -> hf_config:
    """hf_config from an inputs.Workload."""
    return hf_config(batch=w.batch, heads=w.heads, head_dim=w.head_dim, tokens_per_frame=w.tokens_per_frame,
                     chunk_frames=w.chunk_frames, window_frames=w.window_frames, block=w.block, topk=w.topk,
                     keep_permille=w.keep_permille, layers=w.layers, phi=HF_PHI_ELU1, eps=w.eps, merge=merge,
                     swa_kernel=swa_kernel, z_mode=z_mode, sink_frames=sink_frames)


class Context:
    """Owns one hf_ctx.  Methods mirror the C entry points one to one."""

    def __init__(self, cfg: hf_config, device: int = 0):
        self.cfg = cfg
        self._h = C.c_void_p()
        _check(lib().hf_create(C.byref(cfg), device, C.byref(self._h)))

    def close(self):
        if self._h:
            lib().hf_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- C ABI, one to one
    def hf_reset(self, layer=-1):
        _check(lib().hf_reset(self._h, layer, _stream()))

    def hf_set_merge_weights(self, layer, W, bias=None):
        _check(lib().hf_set_merge_weights(self._h, layer, _ptr(W), _ptr(bias), _stream()))

    def hf_set_rope(self, cos_q=None, sin_q=None, cos_k=None, sin_k=None):
        """float32 CUDA tensors [T_c, d/2] (or None) -- see include/hf.h."""
        _check(lib().hf_set_rope(self._h, _ptr(cos_q), _ptr(sin_q), _ptr(cos_k), _ptr(sin_k), _stream()))

    def hf_set_temporal_rope(self, t0, first_pair, n_pairs, cos_tab, sin_tab):
        """float32 CUDA tensors [t0 + 1, n_pairs] -- see include/hf.h."""
        _check(lib().hf_set_temporal_rope(self._h, t0, first_pair, n_pairs, _ptr(cos_tab), _ptr(sin_tab), _stream()))

    def hf_kv_append(self, layer, k, v):
        _check(lib().hf_kv_append(self._h, layer, _ptr(k), _ptr(v), _stream()))

    def hf_kv_append_layers(self, first_layer, ks, vs):
        """ks, vs: sequences of bf16 CUDA tensors [B,H,T_c,d], one per layer from first_layer on."""
        n = len(ks)
        ka = (C.c_void_p * n)(*[t.data_ptr() for t in ks])
        va = (C.c_void_p * n)(*[t.data_ptr() for t in vs])
        _check(lib().hf_kv_append_layers(self._h, first_layer, n, ka, va, _stream()))

    def hf_state_absorb_layers(self, first_layer, n_layers, k_ev, v_ev, n_tokens):
        """k_ev, v_ev: bf16 CUDA tensors [n_layers, B, H, n_tokens, d]."""
        _check(lib().hf_state_absorb_layers(self._h, first_layer, n_layers, _ptr(k_ev), _ptr(v_ev), n_tokens, _stream()))

    def hf_state_absorb(self, layer, k_ev, v_ev, n_tokens):
        _check(lib().hf_state_absorb(self._h, layer, _ptr(k_ev), _ptr(v_ev), n_tokens, _stream()))

    def hf_block_select(self, layer, q, k_cur, mask_out=None, idx_out=None, scores_out=None):
        _check(lib().hf_block_select(self._h, layer, _ptr(q), _ptr(k_cur), _ptr(mask_out), _ptr(idx_out),
                                     _ptr(scores_out), _stream()))

    def hf_sparse_swa(self, layer, q, k_cur, v_cur, o_local, idx=None, lse=None):
        _check(lib().hf_sparse_swa(self._h, layer, _ptr(q), _ptr(k_cur), _ptr(v_cur), _ptr(idx), _ptr(o_local),
                                   _ptr(lse), _stream()))

    def hf_sparse_swa_merged(self, layer, q, k_cur, v_cur, o, idx=None):
        _check(lib().hf_sparse_swa_merged(self._h, layer, _ptr(q), _ptr(k_cur), _ptr(v_cur), _ptr(idx), _ptr(o), _stream()))

    def hf_sparse_swa_backward_dq(self, layer, q, k_cur, v_cur, o_local, lse, d_o, dq, idx=None):
        _check(lib().hf_sparse_swa_backward_dq(self._h, layer, _ptr(q), _ptr(k_cur), _ptr(v_cur), _ptr(idx), _ptr(o_local), _ptr(lse),
                                               _ptr(d_o), _ptr(dq), _stream()))

    def hf_sparse_swa_backward_dkv(self, layer, q, k_cur, v_cur, o_local, lse, d_o, dk, dv):
        _check(lib().hf_sparse_swa_backward_dkv(self._h, layer, _ptr(q), _ptr(k_cur), _ptr(v_cur), _ptr(o_local), _ptr(lse), _ptr(d_o),
                                                _ptr(dk), _ptr(dv), _stream()))

    def hf_linear_attn_backward_dq(self, layer, q, d_o, dq):
        _check(lib().hf_linear_attn_backward_dq(self._h, layer, _ptr(q), _ptr(d_o), _ptr(dq), _stream()))

    def hf_linear_attn(self, layer, q, o_hist):
        _check(lib().hf_linear_attn(self._h, layer, _ptr(q), _ptr(o_hist), _stream()))

    def hf_hybrid_forward(self, layer, q, k, v, o):
        _check(lib().hf_hybrid_forward(self._h, layer, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _stream()))

    def hf_hybrid_forward_host(self, layer, q, k, v, o):
        """q, k, v, o: CPU tensors (pinned recommended)."""
        _check(lib().hf_hybrid_forward_host(self._h, layer, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _stream()))

    def hf_kv_append_host(self, layer, k, v):
        _check(lib().hf_kv_append_host(self._h, layer, _ptr(k), _ptr(v), _stream()))

    def hf_get_state(self, layer, S=None, z=None):
        _check(lib().hf_get_state(self._h, layer, _ptr(S), _ptr(z), _stream()))

    def hf_state_export(self):
        """The checkpoint image of all layers as a numpy uint8 array (size asked for first, then filled)."""
        import numpy as np
        n = C.c_size_t(0)
        _check(lib().hf_state_export(self._h, None, C.byref(n)))
        buf = np.empty(n.value, dtype=np.uint8)
        _check(lib().hf_state_export(self._h, C.c_void_p(buf.ctypes.data), C.byref(n)))
        return buf[:n.value]

    def hf_state_import(self, image):
        """image: contiguous numpy uint8 array written by hf_state_export."""
        _check(lib().hf_state_import(self._h, C.c_void_p(image.ctypes.data), image.nbytes))

    def hf_query(self, layer, what) -> int:
        v = C.c_int64()
        _check(lib().hf_query(self._h, layer, what, C.byref(v)))
        return v.value

    def hf_get_device_status(self):
        f, d = C.c_int(), C.c_int()
        _check(lib().hf_get_device_status(self._h, C.byref(f), C.byref(d)))
        return f.value, d.value

    def hf_selftest_wait_limit(self):
        _check(lib().hf_selftest_wait_limit(self._h, _stream()))

    def hf_slow_path_units(self) -> int:
        v = C.c_int64()
        _check(lib().hf_slow_path_units(self._h, C.byref(v)))
        return v.value

    def hf_launch_count(self) -> int:
        v = C.c_int64()
        _check(lib().hf_launch_count(self._h, C.byref(v)))
        return v.value


def hf_state_absorb_noalloc(k_ev, v_ev, S, z):
    """S += phi(k_ev)^T v_ev, z += sum phi(k_ev) without any allocation (see include/hf.h).
    k_ev, v_ev: bf16 CUDA tensors [..., n_tokens, d] (leading dims = batch*heads); S, z: float32, updated in place."""
    d = k_ev.shape[-1]
    n = k_ev.shape[-2]
    bh = k_ev.numel() // (n * d)
    _check(lib().hf_state_absorb_noalloc(_ptr(k_ev), _ptr(v_ev), bh, n, d, _ptr(S), _ptr(z), _stream()))


def bits_to_cuda(bits, device="cuda"):
    """numpy uint16 bf16 bits -> torch bf16 CUDA tensor holding the same bytes."""
    import numpy as np
    import torch
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device).view(torch.bfloat16)


def cuda_to_bits(t):
    """torch bf16 tensor -> numpy uint16 bits."""
    import numpy as np
    import torch
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def unpack_mask(words, n_blocks: int):
    """uint32 mask words [..., W] -> bool [..., n_blocks] (bit j & 31 of word j >> 5 = block j kept)."""
    import numpy as np
    words = np.asarray(words).view(np.uint32)
    bits = ((words[..., :, None] >> np.arange(32, dtype=np.uint32)) & 1).astype(bool)
    return bits.reshape(words.shape[:-1] + (-1,))[..., :n_blocks]
