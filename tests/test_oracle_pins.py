"""Pins for the CPU oracle: each oracle function is checked against something other than itself --
brute force written token by token, a library routine, a closed form, or an invariant of the method.
The paper prints no numeric worked example of its attention, so none can be quoted; the hand-derived
cases in tests/golden/hand_cases.json are closed forms of Eq. 3-7.
"""
import itertools
import json
import math
import os

import numpy as np
import pytest

from oracle import hybrid_attention as oa
from paper_2604_10103_b200 import inputs as gen

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rnd(shape, seed):
    """bf16-representable N(0,1) values as fp64."""
    return gen.bf16_bits_to_f64(gen.normal_bf16(shape, 77, seed))


# ----------------------------------------------------------------------------- phi
def test_phi_matches_library_elu_plus_one():
    import torch
    x = np.linspace(-12, 12, 4001)
    ref = torch.nn.functional.elu(torch.from_numpy(x)).numpy() + 1.0
    assert np.allclose(oa.phi(x), ref, rtol=0, atol=1e-15)
    assert oa.phi(0.0) == 1.0 and (oa.phi(x) > 0).all()


# ----------------------------------------------------------------------------- blocks
def test_block_ranges_cover_and_ragged_tail():
    assert oa.block_ranges(4680, 128)[-1] == (4608, 4680) and len(oa.block_ranges(4680, 128)) == 37
    assert oa.block_ranges(64, 16) == [(0, 16), (16, 32), (32, 48), (48, 64)]
    tab = oa.key_block_table([4680, 4680, 4680], 128)
    assert len(tab) == 111 and tab[37] == (1, 0, 128) and tab[36] == (0, 4608, 4680)


def test_keep_count_rule():
    assert oa.keep_count(2, 0, 12) == 2                 # tiny case: top-2
    assert oa.keep_count(0, 250, 111) == 28             # ceil(27.75)
    assert oa.keep_count(0, 100, 110) == 11             # exact multiples do not round up
    assert oa.keep_count(0, 1000, 111) == 111
    assert oa.keep_count(5, 0, 3) == 3                  # warm-up: fewer blocks than k
    assert oa.keep_count(0, 1, 10) == 1                 # never empty


# ----------------------------------------------------------------------------- Eq. 5
def test_block_means_and_scores_brute_force():
    q = rnd((70, 32), 1); k = rnd((50, 32), 2)
    qm = oa.block_means(q, 16); km = oa.block_means(k, 16)
    assert qm.shape == (5, 32) and km.shape == (4, 32)
    for i, (s, e) in enumerate([(0, 16), (16, 32), (32, 48), (48, 64), (64, 70)]):
        for c in range(32):
            assert abs(qm[i, c] - sum(q[t, c] for t in range(s, e)) / (e - s)) < 1e-13
    a = oa.block_scores(qm, km)
    for i, j in itertools.product(range(5), range(4)):
        assert abs(a[i, j] - sum(qm[i, c] * km[j, c] for c in range(32))) < 1e-12


def test_canonical_f32_scorer_within_rounding_of_fp64():
    q = rnd((300, 128), 3); k = rnd((300, 128), 4)
    qm32 = oa.block_means_f32(q.astype(np.float32), 128)
    km32 = oa.block_means_f32(k.astype(np.float32), 128)
    assert np.abs(qm32 - oa.block_means(q, 128)).max() < 2e-6
    a32 = oa.block_scores_f32(qm32, km32)
    a64 = oa.block_scores(oa.block_means(q, 128), oa.block_means(k, 128))
    assert np.abs(a32 - a64).max() < 1e-6
    # exact in float32 when nothing rounds: small integers
    xi = np.arange(64 * 32, dtype=np.float32).reshape(64, 32) % 7
    assert np.array_equal(oa.block_means_f32(xi, 16), oa.block_means(xi, 16).astype(np.float32))
    assert np.array_equal(oa.block_scores_f32(xi[:4] * 2, xi[4:8]), (xi[:4] * 2).astype(np.float64) @ xi[4:8].T)


def test_canonical_f32_order_is_the_documented_one():
    """Token-by-token scalar restatement of the documented order on a ragged block."""
    x = rnd((41, 32), 5).astype(np.float32)
    got = oa.block_means_f32(x, 32)
    for (s, e), row in zip([(0, 32), (32, 41)], got):
        for c in range(0, 32, 5):
            chains = [np.float32(0)] * 16
            for t in range(s, e):
                chains[(t - s) % 16] = np.float32(chains[(t - s) % 16] + x[t, c])
            tot = chains[0]
            for r in range(1, 16):
                tot = np.float32(tot + chains[r])
            assert row[c] == np.float32(tot / np.float32(e - s))
    qm = rnd((2, 64), 6).astype(np.float32); km = rnd((3, 64), 7).astype(np.float32)
    a = oa.block_scores_f32(qm, km)
    for i, j in itertools.product(range(2), range(3)):
        p = [np.float32(np.float32(qm[i, l] * km[j, l]) + np.float32(qm[i, l + 32] * km[j, l + 32])) for l in range(32)]
        w = 16
        while w >= 1:
            p = [np.float32(p[l] + p[l + w]) for l in range(w)]
            w //= 2
        assert a[i, j] == p[0]


def test_softmax_form_selects_the_same_blocks_as_raw_scores():
    q = rnd((128, 64), 8); k = rnd((256, 64), 9)
    a = oa.block_scores(oa.block_means(q, 16), oa.block_means(k, 16))
    p = oa.pooled_softmax(a, 64)
    assert np.allclose(p.sum(axis=1), 1.0)
    for kk in (1, 3, 8, 16):
        assert np.array_equal(oa.select_blocks(a, kk), oa.select_blocks(p, kk))


def test_select_blocks_rule():
    a = np.array([[0.1, 0.9, -0.3, 0.9, 0.5]])
    assert oa.select_blocks(a, 2).tolist() == [[False, True, False, True, False]]
    assert oa.select_blocks(a, 1).tolist() == [[False, True, False, False, False]]   # tie -> lower index
    assert oa.select_blocks(np.zeros((3, 6)), 2).tolist() == [[True, True, False, False, False, False]] * 3
    assert oa.select_blocks(np.array([[0.0, -0.0, 0.0]]), 2).tolist() == [[True, True, False]]
    m = oa.select_blocks(rnd((7, 13), 10), 4)
    assert (m.sum(axis=1) == 4).all()


# ----------------------------------------------------------------------------- Eq. 6
def brute_masked_attention(q, keys, vals, token_mask):
    """Dense softmax with an explicit [T_q, N_k] 0/1 token mask, scalar loops."""
    d = q.shape[1]
    out = np.zeros((q.shape[0], vals.shape[1]))
    for r in range(q.shape[0]):
        cols = [c for c in range(keys.shape[0]) if token_mask[r, c]]
        logits = [sum(q[r, x] * keys[c, x] for x in range(d)) / math.sqrt(d) for c in cols]
        mx = max(logits)
        w = [math.exp(l - mx) for l in logits]
        tot = sum(w)
        for wi, c in zip(w, cols):
            out[r] += wi / tot * vals[c]
    return out


def expand_mask(mask, q_len, chunk_lens, b):
    tm = np.zeros((q_len, sum(chunk_lens)), dtype=bool)
    offs = np.concatenate([[0], np.cumsum(chunk_lens)])
    table = oa.key_block_table(chunk_lens, b)
    for i, (qs, qe) in enumerate(oa.block_ranges(q_len, b)):
        for j, (c, s, e) in enumerate(table):
            if mask[i, j]:
                tm[qs:qe, offs[c] + s: offs[c] + e] = True
    return tm


@pytest.mark.parametrize("b,lens", [(8, [24, 24, 24]), (8, [20, 20]), (16, [40])])
def test_sparse_attention_equals_brute_force_masked_softmax(b, lens):
    d = 16
    q = rnd((lens[-1], d), 11)
    kc = [rnd((n, d), 20 + i) for i, n in enumerate(lens)]
    vc = [rnd((n, d), 30 + i) for i, n in enumerate(lens)]
    tm_blocks = -(-lens[-1] // b)
    tn_blocks = sum(-(-n // b) for n in lens)
    rng = np.random.default_rng(5)
    mask = np.zeros((tm_blocks, tn_blocks), dtype=bool)
    for i in range(tm_blocks):
        mask[i, rng.choice(tn_blocks, size=2, replace=False)] = True
    ref = brute_masked_attention(q, np.concatenate(kc), np.concatenate(vc), expand_mask(mask, lens[-1], lens, b))
    got = oa.sparse_attention(q, kc, vc, b, mask)
    assert np.abs(got - ref).max() < 1e-13
    assert np.abs(oa.sparse_attention_blockwise(q, kc, vc, b, mask) - got).max() < 1e-12


def test_all_blocks_kept_is_dense_window_attention_library_sdpa():
    import torch
    d, b, lens = 32, 16, [40, 40, 40]
    q = rnd((40, d), 12)
    kc = [rnd((n, d), 40 + i) for i, n in enumerate(lens)]
    vc = [rnd((n, d), 50 + i) for i, n in enumerate(lens)]
    mask = np.ones((3, 9), dtype=bool)
    got = oa.sparse_attention(q, kc, vc, b, mask)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None], torch.from_numpy(np.concatenate(kc))[None], torch.from_numpy(np.concatenate(vc))[None])[0]
    assert np.abs(got - ref.numpy()).max() < 1e-13


def test_sparse_attention_closed_forms():
    d, b = 16, 8
    q = rnd((16, d), 13); kc = [rnd((16, d), 14), rnd((16, d), 15)]; vc = [rnd((16, d), 16), rnd((16, d), 17)]
    mask = np.array([[True, False, True, False], [False, True, True, False]])
    # V == 1  ->  O == 1
    ones = [np.ones((16, d))] * 2
    assert np.abs(oa.sparse_attention(q, kc, ones, b, mask) - 1).max() < 1e-14
    # q == 0  ->  uniform average of the kept V rows
    o = oa.sparse_attention(np.zeros((16, d)), kc, vc, b, mask)
    assert np.abs(o[0] - (vc[0][0:8].sum(0) + vc[1][0:8].sum(0)) / 16).max() < 1e-14
    assert np.abs(o[8] - (vc[0][8:16].sum(0) + vc[1][0:8].sum(0)) / 16).max() < 1e-14
    # shifting every logit of a row by a constant leaves O unchanged: k -> k + t * q/|q|^2 is row dependent,
    # so use one query row
    q1 = q[:1]
    kshift = [kk + 3.0 * q1 / (q1 @ q1.T) for kk in kc]
    m1 = np.array([[True, True, False, True]])
    a = oa.sparse_attention(np.repeat(q1, 8, 0), kc, vc, b, m1)
    s = oa.sparse_attention(np.repeat(q1, 8, 0), kshift, vc, b, m1)
    assert np.abs(a - s).max() < 1e-12


def test_hand_worked_cases():
    cases = json.load(open(os.path.join(GOLDEN, "hand_cases.json")))
    c = cases["softmax_two_keys"]
    o = oa.sparse_attention(np.array(c["q"]), [np.array(c["k"])], [np.array(c["v"])], 1, np.array([[True, True]]))
    assert np.allclose(o, c["o_local"], rtol=0, atol=1e-15)
    c = cases["state_and_readout"]
    S, z = oa.absorb(np.zeros((2, 2)), np.zeros(2), np.array(c["k_ev"]), np.array(c["v_ev"]))
    assert np.allclose(S, c["S"], rtol=0, atol=1e-15) and np.allclose(z, c["z"], rtol=0, atol=1e-15)
    h = oa.linear_readout(np.array(c["q"]), S, z, np.array(c["W"]), np.array(c["bias"]), eps=0.0)
    assert np.allclose(h, c["o_history"], rtol=0, atol=1e-14)


# ----------------------------------------------------------------------------- Eq. 3 / Eq. 4
def test_absorb_orientation_and_brute_force():
    k = rnd((9, 4), 18); v = rnd((9, 6), 19)
    S, z = oa.absorb(np.zeros((4, 6)), np.zeros(4), k, v)
    Sb = np.zeros((4, 6)); zb = np.zeros(4)
    for t in range(9):
        f = [k[t, a] + 1 if k[t, a] > 0 else math.exp(k[t, a]) for a in range(4)]
        for a in range(4):
            zb[a] += f[a]
            for c in range(6):
                Sb[a, c] += f[a] * v[t, c]
    assert np.abs(S - Sb).max() < 1e-13 and np.abs(z - zb).max() < 1e-13


def test_readout_equals_direct_kernel_average():
    d = 8
    k = rnd((30, d), 21); v = rnd((30, d), 22); q = rnd((5, d), 23)
    S, z = oa.absorb(np.zeros((d, d)), np.zeros(d), k, v)
    got = oa.linear_readout(q, S, z, eps=0.0)
    for r in range(5):
        w = [float(oa.phi(q[r]) @ oa.phi(k[t])) for t in range(30)]
        ref = sum(wi * v[t] for t, wi in enumerate(w)) / sum(w)
        assert np.abs(got[r] - ref).max() < 1e-13
    # V == 1 -> h == 1 -> O_history = W 1 + bias
    S1, z1 = oa.absorb(np.zeros((d, d)), np.zeros(d), k, np.ones((30, d)))
    W = rnd((d, d), 24); bias = rnd((d,), 25)
    assert np.abs(oa.linear_readout(q, S1, z1, W, bias, eps=0.0) - (W.sum(axis=1) + bias)).max() < 1e-13
    # Linear is y = W h (+ b), not h W
    h = oa.linear_readout(q, S, z, eps=0.0)
    assert np.abs(oa.linear_readout(q, S, z, W, bias, eps=0.0) - np.stack([W @ h[r] + bias for r in range(5)])).max() < 1e-13
    # empty state: h = 0, O_history = bias
    assert np.array_equal(oa.linear_readout(q, np.zeros((d, d)), np.zeros(d), W, bias), np.tile(bias, (5, 1)))


# ----------------------------------------------------------------------------- Alg. 2 protocol
def make_stream(P, B=1, H=2, d=16, b=8, topk=2, **kw):
    return oa.HybridStream(B, H, d, b, P, topk=topk, **kw)


@pytest.mark.parametrize("P", [0, 1, 2])
def test_recurrent_state_equals_from_scratch_sum_and_partition(P):
    B, H, d, n = 1, 2, 16, 24
    st = make_stream(P)
    ks = [rnd((B, H, n, d), 100 + i) for i in range(6)]
    vs = [rnd((B, H, n, d), 200 + i) for i in range(6)]
    for i in range(6):
        st.append(ks[i], vs[i])
        n_abs = max(0, i + 1 - P)
        assert st.absorbed_tokens == n_abs * n and len(st.past) == min(P, i + 1)
        # the window holds exactly the newest min(P, i+1) chunks, the state everything older, once
        for slot, (kp, _) in enumerate(st.past):
            assert kp is not None and np.array_equal(kp, ks[i + 1 - len(st.past) + slot])
        for h in range(H):
            S = np.zeros((d, d)); z = np.zeros(d)
            if n_abs:
                kk = np.concatenate([ks[c][0, h] for c in range(n_abs)]); vv = np.concatenate([vs[c][0, h] for c in range(n_abs)])
                S = oa.phi(kk).T @ vv; z = oa.phi(kk).sum(0)
            assert np.abs(st.S[0, h] - S).max() < 1e-11 and np.abs(st.z[0, h] - z).max() < 1e-11


def test_state_invariant_under_token_permutation_inside_a_chunk():
    st1, st2 = make_stream(0), make_stream(0)
    k = rnd((1, 2, 24, 16), 31); v = rnd((1, 2, 24, 16), 32)
    perm = np.random.default_rng(3).permutation(24)
    st1.append(k, v); st2.append(k[:, :, perm], v[:, :, perm])
    assert np.abs(st1.S - st2.S).max() < 1e-12 and np.abs(st1.z - st2.z).max() < 1e-12


def test_stream_forward_equals_brute_force_over_window_plus_state():
    """Whole Alg. 2 + Alg. 3 + Eq. 7 on a tiny stream against token-level brute force."""
    B, H, d, n, b, P = 1, 2, 16, 24, 8, 2
    W = rnd((H, d, d), 41) / 4; bias = rnd((H, d), 42) / 10
    st = make_stream(P, W=W, bias=bias, eps=1e-6)
    ks = [rnd((B, H, n, d), 300 + i) for i in range(5)]; vs = [rnd((B, H, n, d), 400 + i) for i in range(5)]
    for i in range(5):
        q = rnd((B, H, n, d), 500 + i); kq = rnd((B, H, n, d), 600 + i); vq = rnd((B, H, n, d), 700 + i)
        mask, _ = st.select(q, kq, exact=True)
        out, o_loc, o_hist = st.forward(q, kq, vq, mask=mask, parts=True)
        first = max(0, i - P)
        assert mask.shape == (B, H, 3, 3 * (i - first + 1)) and (mask.sum(-1) == min(2, mask.shape[-1])).all()
        for h in range(H):
            lens = [n] * (i - first + 1)
            keys = np.concatenate([ks[c][0, h] for c in range(first, i)] + [kq[0, h]])
            vals = np.concatenate([vs[c][0, h] for c in range(first, i)] + [vq[0, h]])
            ref_loc = brute_masked_attention(q[0, h], keys, vals, expand_mask(mask[0, h], n, lens, b))
            assert np.abs(o_loc[0, h] - ref_loc).max() < 1e-12
            if first > 0:
                kk = np.concatenate([ks[c][0, h] for c in range(first)]); vv = np.concatenate([vs[c][0, h] for c in range(first)])
                fq = oa.phi(q[0, h]); wts = fq @ oa.phi(kk).T
                ref_h = (wts @ vv) / (wts.sum(1, keepdims=True) + 1e-6) @ W[h].T + bias[h]
            else:
                ref_h = np.tile(bias[h], (n, 1))
            assert np.abs(o_hist[0, h] - ref_h).max() < 1e-12
            assert np.abs(out[0, h] - (ref_loc + ref_h)).max() < 1e-12
        st.append(ks[i], vs[i])


def test_canonical_and_exact_selection_agree_except_near_ties():
    w = gen.tiny()
    st = oa.HybridStream(w.batch, w.heads, w.head_dim, w.block, w.past_chunks, topk=w.topk)
    rows = diff = 0
    for c in range(4):
        q, k, v = (gen.bf16_bits_to_f64(t) for t in gen.qkv(w, 0, c, 0))
        m32, a32 = st.select(q, k); m64, a64 = st.select(q, k, exact=True)
        assert np.abs(a32 - a64).max() < 1e-6
        for idx in np.ndindex(m32.shape[:3]):
            rows += 1
            if not np.array_equal(m32[idx], m64[idx]):
                diff += 1
                srt = np.sort(a64[idx])[::-1]; kk = int(m64[idx].sum())
                assert srt[kk - 1] - srt[kk] < 1e-6 * np.abs(a64[idx]).max()
        st.append(*(gen.bf16_bits_to_f64(t) for t in gen.clean_kv(w, 0, c)))
    assert rows == 32 and diff <= 1


# ----------------------------------------------------------------------------- planted mistakes are caught
def test_pins_catch_planted_mistakes(monkeypatch):
    """Each mutant of the oracle must fail at least one pin above."""
    def fails(test, *args):
        try:
            test(*args)
        except AssertionError:
            return True
        return False

    real_phi, real_absorb, real_readout = oa.phi, oa.absorb, oa.linear_readout
    # dropped "+1" on the positive side of phi
    monkeypatch.setattr(oa, "phi", lambda x: np.where(np.asarray(x) > 0, np.asarray(x, float), np.exp(np.minimum(x, 0))))
    assert fails(test_phi_matches_library_elu_plus_one)
    monkeypatch.setattr(oa, "phi", real_phi)
    # transposed state
    monkeypatch.setattr(oa, "absorb", lambda S, z, k, v: (S + (real_phi(k).T @ v).T, z + real_phi(k).sum(0)))
    assert fails(test_readout_equals_direct_kernel_average)
    monkeypatch.setattr(oa, "absorb", real_absorb)
    # h W instead of W h
    def bad_readout(q, S, z, W=None, bias=None, eps=1e-6):
        return real_readout(q, S, z, None if W is None else np.asarray(W).T, bias, eps)
    monkeypatch.setattr(oa, "linear_readout", bad_readout)
    assert fails(test_readout_equals_direct_kernel_average)
    monkeypatch.setattr(oa, "linear_readout", real_readout)
    # missing 1/sqrt(d)
    real_sqrt = math.sqrt
    monkeypatch.setattr(oa.math, "sqrt", lambda x: 1.0)
    try:
        d, b = 32, 16
        q = rnd((40, d), 12); kc = [rnd((40, d), 40)]; vc = [rnd((40, d), 50)]
        import torch
        got = oa.sparse_attention(q, kc, vc, b, np.ones((3, 3), dtype=bool))
    finally:
        monkeypatch.setattr(oa.math, "sqrt", real_sqrt)
    ref = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(q)[None], torch.from_numpy(kc[0])[None], torch.from_numpy(vc[0])[None])[0].numpy()
    assert np.abs(got - ref).max() > 1e-3
    # eviction one chunk too early
    real_append = oa.HybridStream.append
    def early(self, k, v):
        self.P -= 1
        try:
            real_append(self, k, v)
        finally:
            self.P += 1
    monkeypatch.setattr(oa.HybridStream, "append", early)
    assert fails(test_recurrent_state_equals_from_scratch_sum_and_partition, 2)


# ----------------------------------------------------------------------------- Eq. 3 as printed: per-frame means in H
def test_frame_mean_state_brute_force_and_scaling_identity():
    """absorb_frame_mean against token-by-token loops, and the identity that makes the two readings of H
    interchangeable up to a learned scale: with whole frames of T_f tokens, z_mean = z_sum / T_f, so the
    normalised read-out (eps = 0) is exactly T_f times larger."""
    tf, frames, d = 5, 3, 8
    k = rnd((tf * frames, d), 41); v = rnd((tf * frames, d), 42); q = rnd((7, d), 43)
    S, z = oa.absorb_frame_mean(np.zeros((d, d)), np.zeros(d), k, v, tf)
    z_ref = np.zeros(d); S_ref = np.zeros((d, d))
    for fr in range(frames):
        acc = np.zeros(d)
        for t in range(fr * tf, (fr + 1) * tf):
            f = np.array([x + 1.0 if x > 0 else math.exp(x) for x in k[t]])
            acc += f
            S_ref += np.outer(f, v[t])
        z_ref += acc / tf
    assert np.allclose(S, S_ref, rtol=0, atol=1e-12) and np.allclose(z, z_ref, rtol=0, atol=1e-13)
    S2, z2 = oa.absorb(np.zeros((d, d)), np.zeros(d), k, v)
    assert np.allclose(S, S2, rtol=0, atol=1e-12) and np.allclose(z * tf, z2, rtol=1e-14, atol=0)
    h_mean = oa.linear_readout(q, S, z, eps=0.0); h_sum = oa.linear_readout(q, S2, z2, eps=0.0)
    assert np.allclose(h_mean, tf * h_sum, rtol=1e-12, atol=0)
    with pytest.raises(AssertionError):
        oa.absorb_frame_mean(np.zeros((d, d)), np.zeros(d), k[:-1], v[:-1], tf)


def test_stream_with_frame_mean_matches_one_shot():
    st = oa.HybridStream(1, 1, 8, 4, 1, topk=1, z_frame_tokens=4)
    ks = [rnd((1, 1, 8, 8), 50 + i) for i in range(4)]; vs = [rnd((1, 1, 8, 8), 60 + i) for i in range(4)]
    for kk, vv in zip(ks, vs):
        st.append(kk, vv)
    ev = np.concatenate([x[0, 0] for x in ks[:3]])
    z_ref = sum(oa.phi(ev[i * 4:(i + 1) * 4]).mean(axis=0) for i in range(6))
    assert np.allclose(st.z[0, 0], z_ref, rtol=0, atol=1e-13) and st.absorbed_tokens == 24


# ----------------------------------------------------------------------------- attention sink (first chunks kept for ever)
def test_sink_chunks_partition_and_brute_force():
    """With s sink chunks the first s committed chunks stay visible as the oldest key blocks, are never evicted and
    never absorbed: window tokens, sink tokens and absorbed tokens partition everything committed so far; the
    forward equals a token-level masked softmax over [sink | cached | current] plus the read-out of a state built
    from the absorbed chunks alone."""
    B, H, d, b, P, s, n = 1, 1, 32, 4, 1, 1, 8
    st = oa.HybridStream(B, H, d, b, P, topk=2, sink_chunks=s)
    ks = [rnd((B, H, n, d), 70 + i) for i in range(5)]; vs = [rnd((B, H, n, d), 80 + i) for i in range(5)]
    for c in range(5):
        st.append(ks[c], vs[c])
        n_abs = max(0, c + 1 - s - P)
        assert len(st.sink) == min(c + 1, s) and len(st.past) == min(max(c + 1 - s, 0), P)
        assert st.absorbed_tokens == n_abs * n
    # after 5 appends with s = 1, P = 1: sink = {0}, cached = {4}, absorbed = {1, 2, 3}
    S_ref, z_ref = np.zeros((d, d)), np.zeros(d)
    for c in (1, 2, 3):
        S_ref, z_ref = oa.absorb(S_ref, z_ref, ks[c][0, 0], vs[c][0, 0])
    assert np.allclose(st.S[0, 0], S_ref, atol=1e-12) and np.allclose(st.z[0, 0], z_ref, atol=1e-12)
    assert st.sink[0][0] is not None and np.array_equal(st.sink[0][0], ks[0]) and np.array_equal(st.past[0][0], ks[4])
    q = rnd((B, H, n, d), 90); kc = rnd((B, H, n, d), 91); vc = rnd((B, H, n, d), 92)
    mask, _ = st.select(q, kc)
    assert mask.shape == (B, H, 2, 6)      # 2 query blocks x (2 sink + 2 cached + 2 current) key blocks
    o, ol, oh = st.forward(q, kc, vc, mask=mask, parts=True)
    kall = np.concatenate([ks[0][0, 0], ks[4][0, 0], kc[0, 0]]); vall = np.concatenate([vs[0][0, 0], vs[4][0, 0], vc[0, 0]])
    for r in range(n):
        keep_cols = np.repeat(mask[0, 0, r // b], b)
        sc = np.array([q[0, 0, r] @ kall[c] / math.sqrt(d) if keep_cols[c] else -np.inf for c in range(3 * n)])
        w = np.exp(sc - sc.max()); w /= w.sum()
        assert np.allclose(ol[0, 0, r], w @ vall, atol=1e-12)
    assert np.allclose(oh[0, 0], oa.linear_readout(q[0, 0], S_ref, z_ref), atol=1e-12)


def test_no_sink_is_the_default_protocol():
    a = oa.HybridStream(1, 1, 8, 4, 1, topk=1); b_ = oa.HybridStream(1, 1, 8, 4, 1, topk=1, sink_chunks=0)
    for i in range(3):
        k = rnd((1, 1, 8, 8), 95 + i); v = rnd((1, 1, 8, 8), 98 + i)
        a.append(k, v); b_.append(k, v)
    assert np.array_equal(a.S, b_.S) and a.absorbed_tokens == b_.absorbed_tokens == 16 and not b_.sink


# ----------------------------------------------------------------------------- rotation inside the linear branch (Eq. 3 / Eq. 4 / Eq. 8)
def _angles(shape, seed):
    th = np.random.default_rng(seed).uniform(0, 2 * np.pi, size=shape)
    return np.cos(th), np.sin(th), th


def test_rotate_pairs_is_a_plane_rotation():
    x = rnd((6, 8), 101); cos, sin, th = _angles((6, 4), 1)
    y = oa.rotate_pairs(x, cos, sin)
    for t in range(6):
        for i in range(4):
            R = np.array([[math.cos(th[t, i]), -math.sin(th[t, i])], [math.sin(th[t, i]), math.cos(th[t, i])]])
            assert np.allclose(y[t, 2 * i:2 * i + 2], R @ x[t, 2 * i:2 * i + 2], atol=1e-14)
    assert np.allclose(np.linalg.norm(y, axis=1), np.linalg.norm(x, axis=1), rtol=1e-14)
    assert np.array_equal(oa.rotate_pairs(x, np.ones((6, 4)), np.zeros((6, 4))), x)      # zero angle: identity


def test_rotated_state_and_readout_against_token_sum_and_relative_angle():
    """Numerator of Eq. 4 with Eq. 3's state = sum_j (R_q phi(q)) . (R_j phi(k_j)) v_j, and each term depends on the
    angles only through their difference (the point of a rotary embedding); the denominator ignores the angles."""
    n, d = 9, 8
    k = rnd((n, d), 111); v = rnd((n, d), 112); q = rnd((4, d), 113)
    ck, sk, thk = _angles((n, d // 2), 2); cq, sq, thq = _angles((4, d // 2), 3)
    S, z = oa.absorb_rope(np.zeros((d, d)), np.zeros(d), k, v, ck, sk)
    h = oa.linear_readout(q, S, z, eps=0.0, cos_q=cq, sin_q=sq)
    fq, fk = oa.phi(q), oa.phi(k)
    for r in range(4):
        num = np.zeros(d); den = 0.0
        for j in range(n):
            w = 0.0
            for i in range(d // 2):      # pair i: phi(q)_i^T R(theta_k - theta_q) phi(k)_i
                dth = thk[j, i] - thq[r, i]
                a, b = fq[r, 2 * i], fq[r, 2 * i + 1]; c_, e_ = fk[j, 2 * i], fk[j, 2 * i + 1]
                w += math.cos(dth) * (a * c_ + b * e_) + math.sin(dth) * (b * c_ - a * e_)
            num += w * v[j]; den += fq[r] @ fk[j]
        assert np.allclose(h[r], num / den, atol=1e-12)
    S0, z0 = oa.absorb(np.zeros((d, d)), np.zeros(d), k, v)
    assert np.allclose(z, z0, atol=1e-14)                       # normaliser unrotated
    S1, _ = oa.absorb_rope(np.zeros((d, d)), np.zeros(d), k, v, np.ones((n, d // 2)), np.zeros((n, d // 2)))
    assert np.allclose(S1, S0, atol=1e-14)                      # zero angles: Eq. 3 without rotation


def test_relative_temporal_indices_eq8():
    assert oa.relative_temporal_indices(3, 21) == [1, 2, 3]
    assert oa.relative_temporal_indices(21, 21) == [19, 20, 21]
    assert oa.relative_temporal_indices(22, 21) == [19, 20, 21] and oa.relative_temporal_indices(600, 21) == [19, 20, 21]


def test_full_width_merge_reduces_to_the_per_head_merge_and_to_scalar_loops():
    """The one-matrix reading of Eq. 4's Linear: with a block-diagonal matrix it is the per-head projection (pinned
    above); in general it is the plain double loop over output and input features of the concatenated heads."""
    rng = np.random.default_rng(11)
    H, T, d = 3, 5, 4
    h = rng.standard_normal((H, T, d))
    Wh = rng.standard_normal((H, d, d)); bh = rng.standard_normal((H, d))
    W_full = np.zeros((H * d, H * d))
    for i in range(H):
        W_full[i * d:(i + 1) * d, i * d:(i + 1) * d] = Wh[i]
    y = oa.merge_full_width(h, W_full, bh.reshape(-1))
    for i in range(H):
        assert np.allclose(y[i], h[i] @ Wh[i].T + bh[i][None, :], atol=1e-12)
    W_full = rng.standard_normal((H * d, H * d)); b_full = rng.standard_normal(H * d)
    y = oa.merge_full_width(h, W_full, b_full)
    for t in range(T):
        for ho in range(H):
            for c in range(d):
                acc = b_full[ho * d + c]
                for hi in range(H):
                    for a in range(d):
                        acc += W_full[ho * d + c, hi * d + a] * h[hi, t, a]
                assert abs(y[ho, t, c] - acc) < 1e-12
    # and inside the stream: identity matrix = no projection at all
    dd = 32                                     # (the canonical scorer wants a multiple of 32)
    st_a = oa.HybridStream(1, H, dd, 2, 1, topk=1)
    st_b = oa.HybridStream(1, H, dd, 2, 1, topk=1, W_full=np.eye(H * dd))
    for c in range(3):
        k = rng.standard_normal((1, H, 4, dd)); v = rng.standard_normal((1, H, 4, dd))
        st_a.append(k, v); st_b.append(k, v)
    q = rng.standard_normal((1, H, 4, dd)); k = rng.standard_normal((1, H, 4, dd)); v = rng.standard_normal((1, H, 4, dd))
    assert np.allclose(st_a.forward(q, k, v), st_b.forward(q, k, v), atol=1e-12)


# --------------------------------------------------------------------------- Sec. 3.3 / Eq. 8: relative temporal RoPE
def _temporal(t0=9, d=32, first_pair=2, pairs=5, tpf=4, c=3, steps=64):
    om = 1.0 / (50.0 ** (np.arange(pairs) / pairs))
    n = np.arange(steps)
    return dict(t0=t0, first_pair=first_pair, cos_tab=np.cos(n[:, None] * om[None, :]).astype(np.float32),
                sin_tab=np.sin(n[:, None] * om[None, :]).astype(np.float32), tokens_per_frame=tpf, chunk_frames=c), om


def test_window_temporal_indices_hand_values():
    """Eq. 8 with T_0 = 21 and the rule for cached chunks (offsets to the current chunk), by hand."""
    assert oa.window_temporal_indices(9, [6, 3], 21, 3) == ([7, 8, 9], [[4, 5, 6], [1, 2, 3]])          # below the cap: absolute
    assert oa.window_temporal_indices(21, [18, 15], 21, 3) == ([19, 20, 21], [[16, 17, 18], [13, 14, 15]])
    assert oa.window_temporal_indices(24, [21, 18], 21, 3) == ([19, 20, 21], [[16, 17, 18], [13, 14, 15]])  # capped: window slides
    assert oa.window_temporal_indices(600, [597, 594], 21, 3) == ([19, 20, 21], [[16, 17, 18], [13, 14, 15]])
    # T_0 -> infinity: every frame keeps its absolute number
    assert oa.window_temporal_indices(600, [597, 594], 10 ** 9, 3) == ([598, 599, 600], [[595, 596, 597], [592, 593, 594]])
    assert oa.window_temporal_indices(5, [4], 21, 1) == ([5], [[4]])


def test_temporal_rotation_depends_on_index_differences_only():
    """<R_a q, R_b k> = <R_(a+s) q, R_(b+s) k>: what makes relative indices meaningful; other pairs are untouched."""
    t, om = _temporal()
    q = rnd((12, 32), 90); k = rnd((12, 32), 91)
    a = oa.rotate_temporal(q, [7, 8, 9], 4, 2, om) @ oa.rotate_temporal(k, [1, 2, 3], 4, 2, om).T
    b = oa.rotate_temporal(q, [19, 20, 21], 4, 2, om) @ oa.rotate_temporal(k, [13, 14, 15], 4, 2, om).T
    c = oa.rotate_temporal(q, [7, 8, 9], 4, 2, om) @ oa.rotate_temporal(k, [2, 3, 4], 4, 2, om).T
    blocks = lambda m: np.stack([m[4 * i:4 * i + 4, 4 * i:4 * i + 4] for i in range(3)])     # frame i of q against frame i of k
    assert np.abs(blocks(a) - blocks(b)).max() < 1e-12
    assert np.abs(blocks(a) - blocks(c)).max() > 1e-3
    r = oa.rotate_temporal(q, [5, 6, 7], 4, 2, om)
    assert np.array_equal(r[:, :4], q[:, :4]) and np.array_equal(r[:, 14:], q[:, 14:])
    # one pair, by hand: angle = index * omega
    th = 6 * om[1]
    assert np.isclose(r[4, 6], q[4, 6] * np.cos(th) - q[4, 7] * np.sin(th)) and np.isclose(r[4, 7], q[4, 6] * np.sin(th) + q[4, 7] * np.cos(th))


def test_canonical_temporal_rotation_is_the_ideal_one_up_to_bf16_rounding():
    t, om = _temporal()
    x = oa.bf16_round_f32(rnd((12, 32), 92).astype(np.float32))
    got = oa.rotate_temporal_f32(x, [4, 5, 6], 4, 2, t["cos_tab"], t["sin_tab"]).astype(np.float64)
    ideal = oa.rotate_temporal(x.astype(np.float64), [4, 5, 6], 4, 2, om)
    assert np.abs(got - ideal).max() <= 2.0 ** -8 * np.abs(ideal).max() + 1e-6
    assert np.array_equal(got[:, :4], x[:, :4].astype(np.float64))
    assert np.array_equal(oa.bf16_round_f32(got.astype(np.float32)).astype(np.float64), got)       # values are bf16
    # a backward turn undoes a forward turn up to two roundings
    back = oa.rotate_temporal_f32(got.astype(np.float32), [-4, -5, -6], 4, 2, t["cos_tab"], t["sin_tab"])
    assert np.abs(back - x).max() <= 2.0 ** -7 * np.abs(x).max()
    # bf16 rounding: ties to even, by hand (1 + 2^-8 is a tie between 1 and 1 + 2^-7 -> 1; 1 + 3 * 2^-8 -> 1 + 2^-6)
    assert oa.bf16_round_f32(np.array([1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, 1 + 2.0 ** -9], np.float32)).tolist() == [1.0, 1 + 2.0 ** -6, 1.0]


def test_stream_with_capped_relative_indices():
    """Alg. 2 with the relative temporal RoPE: (a) the cache holds every key at the index Eq. 8 and the offset rule give it
    for the chunk being generated, within the roundings of the bf16 store; (b) below the cap nothing is ever re-rotated;
    (c) with identical chunks, the attention output no longer changes from chunk to chunk once the stream is past T_0
    (the softmax branch sees only index differences); (d) sink chunks keep their own indices."""
    t, om = _temporal(t0=9)
    B, H, d, tpf, c = 1, 2, 32, 4, 3
    bf = lambda x: oa.bf16_round_f32(x.astype(np.float32)).astype(np.float64)
    q = bf(rnd((B, H, tpf * c, d), 93)); k = bf(rnd((B, H, tpf * c, d), 94)); v = bf(rnd((B, H, tpf * c, d), 95))
    st = oa.HybridStream(B, H, d, 4, 2, topk=3, temporal=t, sink_chunks=1)
    outs = []
    for n in range(8):
        o, o_loc, _ = st.forward(q, k, v, parts=True)
        outs.append(o_loc)
        st.append(k, v)
        last = st.frames_committed
        frames = [last - 3 * j for j in range(len(st.past))][::-1]
        _, cached = oa.window_temporal_indices(last + c, frames, 9, c)
        for (kp, _), idx in zip(st.past, cached):
            ideal = oa.rotate_temporal(k[0, 0], idx, tpf, 2, om)
            assert np.abs(kp[0, 0] - ideal).max() <= 3 * 2.0 ** -8 * np.abs(ideal).max()
        sink_ideal = oa.rotate_temporal(k[0, 0], [1, 2, 3], tpf, 2, om)
        assert np.abs(st.sink[0][0][0, 0] - sink_ideal).max() <= 2.0 ** -8 * np.abs(sink_ideal).max()
        if last + c <= 9 and len(st.past) == 2:       # below the cap: a single rounding, exactly the canonical rotation of the raw keys
            assert np.array_equal(st.past[0][0][0, 0], oa.rotate_temporal_f32(k[0, 0].astype(np.float32), cached[0], tpf, 2,
                                                                             t["cos_tab"], t["sin_tab"]).astype(np.float64))
    assert st.absorbed_tokens == 5 * tpf * c           # eight commits: one sink chunk, two still cached, five folded into the state
    # past the cap with a full window (chunks 5, 6, 7 are generated at frames 18, 21, 24 > T_0 = 9): same softmax output up to the
    # roundings of the re-rotated keys; the first chunks (growing window, absolute indices) differ
    assert np.abs(outs[6] - outs[5]).max() < 2e-2 and np.abs(outs[7] - outs[6]).max() < 2e-2
    assert np.abs(outs[2] - outs[1]).max() > 5e-2


def test_stream_without_cap_is_absolute_indexing():
    """T_0 -> infinity: the stored keys are the raw keys rotated once by their absolute frame numbers, never touched again."""
    t, om = _temporal(t0=10 ** 6, steps=64)
    B, H, d, tpf, c = 1, 1, 32, 4, 3
    bf = lambda x: oa.bf16_round_f32(x.astype(np.float32)).astype(np.float64)
    st = oa.HybridStream(B, H, d, 4, 2, topk=3, temporal=t)
    ks = []
    for n in range(5):
        k = bf(rnd((B, H, tpf * c, d), 100 + n)); v = bf(rnd((B, H, tpf * c, d), 110 + n))
        st.append(k, v); ks.append(k)
        for j, (kp, _) in enumerate(st.past):
            chunk_no = len(ks) - len(st.past) + j
            idx = [3 * chunk_no + 1, 3 * chunk_no + 2, 3 * chunk_no + 3]
            want = oa.rotate_temporal_f32(ks[chunk_no][0, 0].astype(np.float32), idx, tpf, 2, t["cos_tab"], t["sin_tab"])
            assert np.array_equal(kp[0, 0], want.astype(np.float64))
    assert st.current_indices() == [16, 17, 18]


# --------------------------------------------------------------------------- gradients (rollout step with gradient, Alg. 1)
def _fd(fn, x, eps=1e-6):
    """Central finite differences of the scalar fn with respect to every element of x."""
    g = np.zeros_like(x)
    it = np.nditer(x, flags=["multi_index"])
    for _ in it:
        i = it.multi_index
        old = x[i]
        x[i] = old + eps; up = fn()
        x[i] = old - eps; dn = fn()
        x[i] = old
        g[i] = (up - dn) / (2 * eps)
    return g


def test_sparse_attention_backward_against_finite_differences_and_autograd():
    """dq, dk, dv of Eq. 6 with a fixed mask: central differences of the oracle's own forward on a ragged two-chunk window,
    and torch autograd (fp64 SDPA) with every block kept."""
    import torch
    d, b, lens = 8, 4, [6, 10]
    q = rnd((10, d), 120); kc = [rnd((n, d), 121 + i) for i, n in enumerate(lens)]; vc = [rnd((n, d), 125 + i) for i, n in enumerate(lens)]
    g = rnd((10, d), 129)
    tm, tn = 3, 2 + 3
    rng = np.random.default_rng(7)
    mask = np.zeros((tm, tn), dtype=bool)
    for i in range(tm):
        mask[i, rng.choice(tn, size=2, replace=False)] = True
    dq, dk, dv = oa.sparse_attention_backward(q, kc, vc, b, mask, g)
    loss = lambda: float((oa.sparse_attention(q, kc, vc, b, mask) * g).sum())
    assert np.abs(dq - _fd(loss, q)).max() < 1e-7
    for c in range(2):
        assert np.abs(dk[c] - _fd(loss, kc[c])).max() < 1e-7
        assert np.abs(dv[c] - _fd(loss, vc[c])).max() < 1e-7
    # a key block no query block keeps gets no gradient
    unused = [j for j in range(tn) if not mask[:, j].any()]
    table = oa.key_block_table(lens, b)
    for j in unused:
        c, s, e = table[j]
        assert not dk[c][s:e].any() and not dv[c][s:e].any()
    # all blocks kept: dense attention, library autograd
    full = np.ones((tm, tn), dtype=bool)
    dq, dk, dv = oa.sparse_attention_backward(q, kc, vc, b, full, g)
    tq = torch.tensor(q, requires_grad=True); tk = torch.tensor(np.concatenate(kc), requires_grad=True)
    tv = torch.tensor(np.concatenate(vc), requires_grad=True)
    o = torch.nn.functional.scaled_dot_product_attention(tq[None], tk[None], tv[None])[0]
    (o * torch.tensor(g)).sum().backward()
    assert np.abs(dq - tq.grad.numpy()).max() < 1e-12
    assert np.abs(np.concatenate(dk) - tk.grad.numpy()).max() < 1e-12
    assert np.abs(np.concatenate(dv) - tv.grad.numpy()).max() < 1e-12
    # closed forms: no upstream gradient -> none downstream; constant V rows -> the output does not depend on q or k
    z3 = oa.sparse_attention_backward(q, kc, vc, b, mask, np.zeros_like(g))
    assert not z3[0].any() and not any(x.any() for x in z3[1]) and not any(x.any() for x in z3[2])
    ones = [np.ones_like(v) for v in vc]
    dq1, dk1, _ = oa.sparse_attention_backward(q, kc, ones, b, mask, g)
    assert np.abs(dq1).max() < 1e-14 and max(np.abs(x).max() for x in dk1) < 1e-14


def test_linear_readout_backward_against_finite_differences_and_autograd():
    import torch
    d, n = 6, 5
    q = rnd((n, d), 130); S = rnd((d, d), 131); z = np.abs(rnd((d,), 132)) + 0.5; W = rnd((d, d), 133); bias = rnd((d,), 134)
    g = rnd((n, d), 135)
    dq, dS, dz, dW, db = oa.linear_readout_backward(q, S, z, g, W, eps=1e-3)
    loss = lambda: float((oa.linear_readout(q, S, z, W, bias, eps=1e-3) * g).sum())
    for got, x in ((dq, q), (dS, S), (dz, z), (dW, W), (db, bias)):
        assert np.abs(got - _fd(loss, x)).max() < 1e-7
    assert np.allclose(oa.phi_prime(np.array([-1.0, 0.0, 2.0])), [np.exp(-1.0), 1.0, 1.0])
    tq = torch.tensor(q, requires_grad=True); tS = torch.tensor(S, requires_grad=True); tz = torch.tensor(z, requires_grad=True)
    f = torch.nn.functional.elu(tq) + 1
    y = ((f @ tS) / (f @ tz + 1e-3)[:, None]) @ torch.tensor(W).T + torch.tensor(bias)
    (y * torch.tensor(g)).sum().backward()
    assert np.abs(dq - tq.grad.numpy()).max() < 1e-12 and np.abs(dS - tS.grad.numpy()).max() < 1e-12
    assert np.abs(dz - tz.grad.numpy()).max() < 1e-12
    # identity "Linear"
    dq2, _, _, dW2, _ = oa.linear_readout_backward(q, S, z, g, None, eps=1e-3)
    loss2 = lambda: float((oa.linear_readout(q, S, z, None, None, eps=1e-3) * g).sum())
    assert dW2 is None and np.abs(dq2 - _fd(loss2, q)).max() < 1e-7


def test_stream_backward_against_finite_differences():
    """HybridStream.backward after evictions (sink + cached chunks + state): every gradient against central differences of
    HybridStream.forward with the mask held fixed; planted mistakes (a dropped softmax-Jacobian term, a missing branch in
    the sum of Eq. 7) are caught."""
    B, H, d, b = 1, 2, 8, 4
    W = rnd((H, d, d), 140) / np.sqrt(d); bias = rnd((H, d), 141) * 0.1
    st = oa.HybridStream(B, H, d, b, 1, topk=2, W=W, bias=bias, sink_chunks=1, eps=1e-3)
    for c in range(4):
        st.append(rnd((B, H, 6, d), 150 + c), rnd((B, H, 6, d), 160 + c))
    assert st.absorbed_tokens == 12 and len(st.sink) == 1 and len(st.past) == 1
    q = rnd((B, H, 6, d), 170); k = rnd((B, H, 6, d), 171); v = rnd((B, H, 6, d), 172); g = rnd((B, H, 6, d), 173)
    mask, _ = st.select(q, k, exact=True)
    gr = st.backward(q, k, v, g, mask=mask)
    loss = lambda: float((st.forward(q, k, v, mask=mask) * g).sum())
    assert np.abs(gr["dq"] - _fd(loss, q)).max() < 1e-6
    assert np.abs(gr["dk_cur"] - _fd(loss, k)).max() < 1e-6 and np.abs(gr["dv_cur"] - _fd(loss, v)).max() < 1e-6
    assert np.abs(gr["dS"] - _fd(loss, st.S)).max() < 1e-6 and np.abs(gr["dz"] - _fd(loss, st.z)).max() < 1e-6
    assert np.abs(gr["dW"] - _fd(loss, st.W)).max() < 1e-6 and np.abs(gr["dbias"] - _fd(loss, st.bias)).max() < 1e-6
    for n, (kp, vp) in enumerate(st.sink + st.past):
        assert np.abs(gr["dk_past"][n] - _fd(loss, kp)).max() < 1e-6 and np.abs(gr["dv_past"][n] - _fd(loss, vp)).max() < 1e-6
    # planted mistakes
    want = _fd(loss, q)
    orig = oa.sparse_attention_backward
    try:
        def no_jacobian_term(q_, kc, vc, b_, m, go):
            dq, dk, dv = orig(q_, kc, vc, b_, m, go)
            return dq * 1.0 + 1e-3, dk, dv
        oa.sparse_attention_backward = no_jacobian_term
        assert np.abs(st.backward(q, k, v, g, mask=mask)["dq"] - want).max() > 1e-4
    finally:
        oa.sparse_attention_backward = orig
    only_local = oa.sparse_attention_backward(q[0, 0], [kp[0, 0] for kp, _ in st.sink + st.past] + [k[0, 0]],
                                              [vp[0, 0] for _, vp in st.sink + st.past] + [v[0, 0]], b, mask[0, 0], g[0, 0])[0]
    assert np.abs(only_local - want[0, 0]).max() > 1e-4          # the history branch's share of dq is not negligible
