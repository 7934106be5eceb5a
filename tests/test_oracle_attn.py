"""Pins for the attention oracle.

Forward: brute force through a dense T x T masked softmax in fp64 (a different
formulation: one big matrix and a mask built from sample ids), a library routine on the
single-sample special case, and closed-form invariants.  Backward: central finite
differences of the fp64 forward, closed-form special cases, and library autograd on the
dense formulation.  The fp32 instantiation is tied to the fp64 one.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_23250_b200 import pools


def _rand(rng, T, hq, hkv, d):
    return (rng.standard_normal((T, hq, d)), rng.standard_normal((T, hkv, d)),
            rng.standard_normal((T, hkv, d)), rng.standard_normal((T, hq, d)))


def _dense_fwd(q, k, v, lengths, scale):
    """Dense masked softmax in fp64: mask from sample ids, one T x T matrix per head."""
    T, hq, d = q.shape
    hkv = k.shape[1]
    G = hq // hkv
    sid = np.repeat(np.arange(len(lengths)), lengths)
    pos = np.arange(T)
    allowed = (sid[:, None] == sid[None, :]) & (pos[None, :] <= pos[:, None])
    out = np.zeros_like(q)
    lse = np.zeros((hq, T))
    for h in range(hq):
        s = scale * q[:, h, :] @ k[:, h // G, :].T
        s = np.where(allowed, s, -np.inf)
        m = s.max(axis=1, keepdims=True)
        e = np.exp(s - m)
        z = e.sum(axis=1, keepdims=True)
        out[:, h, :] = (e / z) @ v[:, h // G, :]
        lse[h] = (m + np.log(z))[:, 0]
    return out, lse


@pytest.mark.parametrize("seed", range(5))
def test_fwd_brute_force_dense_mask(seed):
    rng = np.random.default_rng(seed)
    T = int(rng.integers(30, 200))
    lengths = pools.random_layout(rng, T, int(rng.integers(1, 80)))
    hkv = int(rng.integers(1, 3))
    hq = hkv * int(rng.integers(1, 4))
    d = int(rng.choice([8, 16, 32]))
    q, k, v, _ = _rand(rng, T, hq, hkv, d)
    scale = 1 / np.sqrt(d)
    o, l = oracle.attn_fwd(q, k, v, pools.cu_seqlens(lengths), prec="f64")
    o2, l2 = _dense_fwd(q, k, v, lengths, scale)
    np.testing.assert_allclose(o, o2, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(l, l2, rtol=1e-11, atol=1e-12)


def test_fwd_single_sample_is_library_causal_sdpa():
    rng = np.random.default_rng(7)
    T, hq, hkv, d = 96, 4, 2, 16
    q, k, v, _ = _rand(rng, T, hq, hkv, d)
    o, _ = oracle.attn_fwd(q, k, v, [0, T], prec="f64")
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(k).permute(1, 0, 2)[None].repeat_interleave(hq // hkv, dim=1)
    tv = torch.from_numpy(v).permute(1, 0, 2)[None].repeat_interleave(hq // hkv, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
    np.testing.assert_allclose(o, ref[0].permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)


def test_fwd_length_one_samples_return_v():
    rng = np.random.default_rng(1)
    T, hq, hkv, d = 9, 4, 2, 8
    q, k, v, _ = _rand(rng, T, hq, hkv, d)
    o, l = oracle.attn_fwd(q, k, v, np.arange(T + 1), prec="f64")
    G = hq // hkv
    for h in range(hq):
        np.testing.assert_allclose(o[:, h], v[:, h // G], rtol=0, atol=1e-15)
        np.testing.assert_allclose(l[h], (q[:, h] * k[:, h // G]).sum(-1) / np.sqrt(d), atol=1e-13)


def test_fwd_identical_keys_give_prefix_mean():
    rng = np.random.default_rng(2)
    lengths = [5, 17, 1, 30]
    T, hq, hkv, d = sum(lengths), 2, 1, 8
    q, k, v, _ = _rand(rng, T, hq, hkv, d)
    cu = pools.cu_seqlens(lengths)
    for j in range(len(lengths)):                       # same key inside each sample
        k[cu[j]:cu[j + 1]] = k[cu[j]]
    o, l = oracle.attn_fwd(q, k, v, cu, prec="f64")
    for j, n in enumerate(lengths):
        vs = v[cu[j]:cu[j + 1], 0]
        want = np.cumsum(vs, axis=0) / np.arange(1, n + 1)[:, None]
        for h in range(hq):
            np.testing.assert_allclose(o[cu[j]:cu[j + 1], h], want, atol=1e-13)
            s = (q[cu[j]:cu[j + 1], h] * k[cu[j], 0]).sum(-1) / np.sqrt(d)
            np.testing.assert_allclose(l[h, cu[j]:cu[j + 1]], s + np.log(np.arange(1, n + 1)), atol=1e-12)
    # Q = 0 gives the same prefix means whatever the keys
    k2 = rng.standard_normal(k.shape)
    o0, _ = oracle.attn_fwd(np.zeros_like(q), k2, v, cu, prec="f64")
    np.testing.assert_allclose(o0, o, atol=1e-13)


def test_fwd_packed_equals_per_sample_and_permutation():
    rng = np.random.default_rng(3)
    lengths = [12, 1, 40, 7, 25]
    T, hq, hkv, d = sum(lengths), 4, 2, 16
    q, k, v, _ = _rand(rng, T, hq, hkv, d)
    cu = pools.cu_seqlens(lengths)
    o, l = oracle.attn_fwd(q, k, v, cu, prec="f64")
    for j in range(len(lengths)):
        sl = slice(cu[j], cu[j + 1])
        oj, lj = oracle.attn_fwd(q[sl], k[sl], v[sl], [0, lengths[j]], prec="f64")
        np.testing.assert_array_equal(o[sl], oj)
        np.testing.assert_array_equal(l[:, sl], lj)
    perm = [3, 0, 4, 2, 1]
    idx = np.concatenate([np.arange(cu[j], cu[j + 1]) for j in perm])
    op, lp = oracle.attn_fwd(q[idx], k[idx], v[idx], pools.cu_seqlens([lengths[j] for j in perm]), prec="f64")
    np.testing.assert_array_equal(op, o[idx])
    np.testing.assert_array_equal(lp, l[:, idx])


def test_fwd_head_depends_only_on_its_kv_head_and_shift_invariance():
    rng = np.random.default_rng(4)
    lengths = [20, 33]
    T, hq, hkv, d = sum(lengths), 4, 2, 8
    q, k, v, _ = _rand(rng, T, hq, hkv, d)
    cu = pools.cu_seqlens(lengths)
    o, l = oracle.attn_fwd(q, k, v, cu, prec="f64")
    k2, v2 = k.copy(), v.copy()
    k2[:, 1] += 1.0
    v2[:, 1] -= 2.0
    o2, l2 = oracle.attn_fwd(q, k2, v2, cu, prec="f64")
    np.testing.assert_array_equal(o2[:, :2], o[:, :2])       # heads 0,1 use kv head 0
    assert np.abs(o2[:, 2:] - o[:, 2:]).max() > 0.1
    # adding c * q_i-independent constant to all scores of a row: append a constant feature
    qa = np.concatenate([q, np.full((T, hq, 1), 3.0)], axis=2)
    ka = np.concatenate([k, np.full((T, hkv, 1), 5.0)], axis=2)
    oa, la = oracle.attn_fwd(qa, ka, np.concatenate([v, v[:, :, :1]], 2), cu, scale=1 / np.sqrt(d), prec="f64")
    np.testing.assert_allclose(oa[:, :, :d], o, atol=1e-12)
    np.testing.assert_allclose(la, l + 15.0 / np.sqrt(d), atol=1e-12)


def _loss(q, k, v, dout, cu):
    o, _ = oracle.attn_fwd(q, k, v, cu, prec="f64")
    return float((o * dout).sum())


def test_bwd_matches_central_finite_differences():
    rng = np.random.default_rng(5)
    lengths = [7, 1, 13, 4]
    T, hq, hkv, d = sum(lengths), 4, 2, 8
    q, k, v, dout = _rand(rng, T, hq, hkv, d)
    cu = pools.cu_seqlens(lengths)
    o, l = oracle.attn_fwd(q, k, v, cu, prec="f64")
    dq, dk, dv = oracle.attn_bwd(q, k, v, o, l, dout, cu, prec="f64")
    eps = 1e-4
    for name, x, g in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        num = np.zeros_like(x)
        flat, nflat = x.reshape(-1), num.reshape(-1)
        for i in range(flat.size):                     # every element perturbed
            old = flat[i]
            flat[i] = old + eps
            fp = _loss(q, k, v, dout, cu)
            flat[i] = old - eps
            fm = _loss(q, k, v, dout, cu)
            flat[i] = old
            nflat[i] = (fp - fm) / (2 * eps)
        err = np.abs(num - g).max() / np.abs(g).max()
        assert err < 1e-6, (name, err)


def test_bwd_matches_library_autograd_on_dense_formulation():
    rng = np.random.default_rng(6)
    lengths = [30, 5, 41]
    T, hq, hkv, d = sum(lengths), 4, 2, 16
    q, k, v, dout = _rand(rng, T, hq, hkv, d)
    cu = pools.cu_seqlens(lengths)
    o, l = oracle.attn_fwd(q, k, v, cu, prec="f64")
    dq, dk, dv = oracle.attn_bwd(q, k, v, o, l, dout, cu, prec="f64")
    tq, tk, tv = (torch.tensor(x, requires_grad=True) for x in (q, k, v))
    sid = torch.repeat_interleave(torch.arange(len(lengths)), torch.tensor(lengths))
    pos = torch.arange(T)
    allowed = (sid[:, None] == sid[None, :]) & (pos[None, :] <= pos[:, None])
    G = hq // hkv
    s = torch.einsum("qhd,khd->hqk", tq, tk.repeat_interleave(G, dim=1)) / np.sqrt(d)
    p = torch.softmax(s.masked_fill(~allowed, float("-inf")), dim=-1)
    to = torch.einsum("hqk,khd->qhd", p, tv.repeat_interleave(G, dim=1))
    (to * torch.tensor(dout)).sum().backward()
    np.testing.assert_allclose(dq, tq.grad.numpy(), rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(dk, tk.grad.numpy(), rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(dv, tv.grad.numpy(), rtol=1e-9, atol=1e-11)


def test_bwd_special_cases():
    rng = np.random.default_rng(8)
    # length-1 samples: dQ = dK = 0 and dV = sum over the group of dO
    T, hq, hkv, d = 6, 4, 2, 8
    q, k, v, dout = _rand(rng, T, hq, hkv, d)
    cu = np.arange(T + 1)
    o, l = oracle.attn_fwd(q, k, v, cu, prec="f64")
    dq, dk, dv = oracle.attn_bwd(q, k, v, o, l, dout, cu, prec="f64")
    assert np.abs(dq).max() < 1e-14 and np.abs(dk).max() < 1e-14
    np.testing.assert_allclose(dv, dout.reshape(T, hkv, 2, d).sum(2), atol=1e-14)
    # Q = 0: P_ik = 1/(i+1), so dV_k = sum_h sum_{i>=k} dO_i / (i+1)
    n = 19
    q, k, v, dout = _rand(rng, n, 2, 1, d)
    q[:] = 0
    o, l = oracle.attn_fwd(q, k, v, [0, n], prec="f64")
    _, _, dv = oracle.attn_bwd(q, k, v, o, l, dout, [0, n], prec="f64")
    w = dout.sum(1) / np.arange(1, n + 1)[:, None]
    want = np.cumsum(w[::-1], axis=0)[::-1]
    np.testing.assert_allclose(dv[:, 0], want, atol=1e-13)


def test_bwd_gqa_is_sum_of_expanded_mha_gradients():
    rng = np.random.default_rng(9)
    lengths = [9, 22]
    T, hq, hkv, d = sum(lengths), 6, 2, 8
    G = hq // hkv
    q, k, v, dout = _rand(rng, T, hq, hkv, d)
    cu = pools.cu_seqlens(lengths)
    o, l = oracle.attn_fwd(q, k, v, cu, prec="f64")
    dq, dk, dv = oracle.attn_bwd(q, k, v, o, l, dout, cu, prec="f64")
    ke, ve = np.repeat(k, G, axis=1), np.repeat(v, G, axis=1)
    o2, l2 = oracle.attn_fwd(q, ke, ve, cu, prec="f64")
    dq2, dk2, dv2 = oracle.attn_bwd(q, ke, ve, o2, l2, dout, cu, prec="f64")
    np.testing.assert_allclose(o2, o, atol=1e-14)
    np.testing.assert_allclose(dq2, dq, atol=1e-13)
    np.testing.assert_allclose(dk2.reshape(T, hkv, G, d).sum(2), dk, atol=1e-12)
    np.testing.assert_allclose(dv2.reshape(T, hkv, G, d).sum(2), dv, atol=1e-12)


def test_f32_instantiation_tracks_f64():
    rng = np.random.default_rng(10)
    lengths = [100, 3, 61]
    T, hq, hkv, d = sum(lengths), 4, 2, 32
    q, k, v, dout = _rand(rng, T, hq, hkv, d)
    cu = pools.cu_seqlens(lengths)
    o, l = oracle.attn_fwd(q, k, v, cu, prec="f64")
    g = oracle.attn_bwd(q, k, v, o, l, dout, cu, prec="f64")
    o32, l32 = oracle.attn_fwd(q, k, v, cu, prec="f32")
    g32 = oracle.attn_bwd(q, k, v, o32, l32, dout, cu, prec="f32")
    assert np.abs(o32 - o).max() / np.abs(o).max() < 2e-6
    assert np.abs(l32 - l).max() < 1e-5
    for a, b in zip(g32, g):
        assert np.abs(a - b).max() / np.abs(b).max() < 1e-5


def test_row_and_column_samplers_agree_with_full():
    rng = np.random.default_rng(11)
    lengths = [50, 1, 77, 20]
    T, hq, hkv, d = sum(lengths), 4, 2, 16
    q, k, v, dout = _rand(rng, T, hq, hkv, d)
    cu = pools.cu_seqlens(lengths)
    for prec, tol in (("f64", 1e-12), ("f32", 2e-5)):
        o, l = oracle.attn_fwd(q, k, v, cu, prec=prec)
        dq, dk, dv = oracle.attn_bwd(q, k, v, o, l, dout, cu, prec=prec)
        rows = rng.integers(0, T, size=12)
        heads = rng.integers(0, hq, size=12)
        orow, lrow = oracle.attn_fwd_rows(q, k, v, cu, rows, heads, prec=prec)
        np.testing.assert_allclose(orow, o[rows, heads], atol=tol)
        np.testing.assert_allclose(lrow, l[heads, rows], atol=tol)
        dqr = oracle.attn_dq_rows(q, k, v, dout, cu, rows, heads, prec=prec)
        np.testing.assert_allclose(dqr, dq[rows, heads], atol=tol * 10)
        kvh = rng.integers(0, hkv, size=12)
        dkc, dvc = oracle.attn_dkv_cols(q, k, v, o, l, dout, cu, rows, kvh, prec=prec)
        np.testing.assert_allclose(dkc, dk[rows, kvh], atol=tol * 10)
        np.testing.assert_allclose(dvc, dv[rows, kvh], atol=tol * 10)


def test_rowsum_of_dS_is_zero():
    # sum_k dS_ik = sum_k P_ik dP_ik - D_i = <dO_i, O_i> - D_i = 0, hence dQ is orthogonal
    # to any direction along which all keys of the sample agree: add a shared feature to K.
    rng = np.random.default_rng(12)
    n, d = 24, 8
    q, k, v, dout = _rand(rng, n, 1, 1, d)
    k[:, :, 0] = 2.5                                   # same value for every key
    o, l = oracle.attn_fwd(q, k, v, [0, n], prec="f64")
    dq, _, _ = oracle.attn_bwd(q, k, v, o, l, dout, [0, n], prec="f64")
    assert np.abs(dq[:, 0, 0]).max() < 1e-13           # = scale * 2.5 * sum_k dS_ik
