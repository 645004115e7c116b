"""Pins for the oracle's transformer arithmetic: a float64 library restatement,
closed forms and invariants.  None of them re-uses the oracle's own formulas."""
import dataclasses
import math

import numpy as np
import pytest
import torch

from oracle import hispec as orc
from paper_2510_01336_b200 import workload as wl
from tests.helpers import SMALL, oracle_for
from tests.ref_torch64 import exit_logits_all_positions


@pytest.mark.parametrize("shape,P", [(SMALL, 24), (wl.TINY, 20), (wl.MINI_GQA, 12)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_matches_float64_library_restatement(shape, P, dtype):
    w, m, hs = oracle_for(shape, dtype=dtype)
    toks = wl.make_tokens(shape, P).tolist()
    for L in (shape.L_d, shape.L_i, shape.L_f):
        out = hs.brute_force_exit(toks, L, list(range(P)))
        h64, z64 = exit_logits_all_positions(w, toks, L)
        rel = np.linalg.norm(out.hidden - h64.numpy(), axis=1) / np.linalg.norm(h64.numpy(), axis=1)
        assert rel.max() < 2e-5, (L, rel.max())
        assert np.abs(out.logits - z64.numpy()).max() < 2e-5
        # greedy ids agree wherever float64 has a clear winner
        top = torch.topk(z64, 2, dim=1)
        clear = (top.values[:, 0] - top.values[:, 1]) > 1e-4
        ids64 = top.indices[:, 0][clear].tolist()
        assert [i for i, c in zip(out.argmax_ids, clear.tolist()) if c] == ids64


def test_rmsnorm_unit_rms_and_gain():
    lib = orc._load()
    rng = np.random.default_rng(0)
    x = rng.standard_normal(300).astype(np.float32) * 7
    g = np.ones(300, np.float32)
    out = np.empty_like(x)
    lib.oracle_rmsnorm(orc._fp(x), orc._fp(g), 300, 0.0, orc._fp(out))
    assert abs(math.sqrt(float(np.mean(out.astype(np.float64) ** 2))) - 1.0) < 1e-6
    g2 = rng.standard_normal(300).astype(np.float32)
    out2 = np.empty_like(x)
    lib.oracle_rmsnorm(orc._fp(x), orc._fp(g2), 300, 0.0, orc._fp(out2))
    np.testing.assert_allclose(out2, out * g2, rtol=1e-6, atol=1e-7)
    # eps enters under the square root, added to the mean square
    one = np.full(4, 2.0, np.float32)
    o3 = np.empty_like(one)
    lib.oracle_rmsnorm(orc._fp(one), orc._fp(np.ones(4, np.float32)), 4, 5.0, orc._fp(o3))
    np.testing.assert_allclose(o3, 2.0 / 3.0, rtol=1e-6)


def test_rope_closed_forms():
    lib = orc._load()
    hd = 8
    v = np.zeros(hd, np.float32)
    v[0] = 1.0  # pair (0, 4) has frequency base^0 = 1: rotation by pos radians
    lib.oracle_rope(orc._fp(v), hd, 3, 10000.0)
    np.testing.assert_allclose(v[[0, 4]], [math.cos(3.0), math.sin(3.0)], atol=1e-7)
    assert np.all(v[[1, 2, 3, 5, 6, 7]] == 0)
    # pair (1, 5) has frequency base^(-2/hd)
    v = np.zeros(hd, np.float32)
    v[5] = 2.0
    lib.oracle_rope(orc._fp(v), hd, 7, 10000.0)
    th = 7 * 10000.0 ** (-2.0 / hd)
    np.testing.assert_allclose(v[[1, 5]], [-2 * math.sin(th), 2 * math.cos(th)], atol=1e-6)
    # position 0 is the identity; rotations preserve the norm and compose
    rng = np.random.default_rng(1)
    a = rng.standard_normal(64).astype(np.float32)
    b = a.copy()
    lib.oracle_rope(orc._fp(b), 64, 0, 500000.0)
    assert np.array_equal(a, b)
    lib.oracle_rope(orc._fp(b), 64, 12345, 500000.0)
    assert abs(np.linalg.norm(b) - np.linalg.norm(a)) < 1e-5
    # q(p).k(p') depends on p - p' only
    q, k = rng.standard_normal(64).astype(np.float32), rng.standard_normal(64).astype(np.float32)
    dots = []
    for shift in (0, 1000):
        qq, kk = q.copy(), k.copy()
        lib.oracle_rope(orc._fp(qq), 64, 17 + shift, 10000.0)
        lib.oracle_rope(orc._fp(kk), 64, 5 + shift, 10000.0)
        dots.append(float(qq.astype(np.float64) @ kk.astype(np.float64)))
    assert abs(dots[0] - dots[1]) < 1e-4


def test_bf16_rounding_is_nearest_even():
    rng = np.random.default_rng(2)
    x = np.concatenate([rng.standard_normal(4000).astype(np.float32) * 3,
                        np.array([1.00390625, 1.01171875, -1.00390625, 0.0, 3.3895314e38], np.float32)])
    ours = orc.round_bf16(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(ours, ref)
    assert ours[4000] == 1.0 and ours[4001] == np.float32(1.015625)  # ties go to the even mantissa


def test_single_key_attention_returns_v_and_zero_residual_branches():
    """With one position the softmax weight is 1: the attention output is v
    itself.  With Wo = Wdown = 0 every exit yields head . RMSNorm(E[x])."""
    shape = SMALL
    w = wl.make_weights(shape, dtype=torch.float32)
    for l in w.layers():
        w.wo[l].zero_()
        w.wdown[l].zero_()
    _, m, hs = oracle_for(shape, weights=w)
    toks = wl.make_tokens(shape, 6).tolist()
    out = hs.brute_force_exit(toks, shape.L_f, list(range(6)))
    emb = w.tok_emb[toks].double()
    expect = torch.nn.functional.rms_norm(emb, (shape.d_model,), None, shape.rms_eps) @ w.head.double().T
    np.testing.assert_allclose(out.logits, expect.numpy(), atol=1e-5)

    # one layer, one token, identity-like Wo: residual increment equals Wo v
    w2 = wl.make_weights(dataclasses.replace(shape, n_q_heads=2, n_kv_heads=2, head_dim=32), dtype=torch.float32)
    s2 = w2.shape
    w2.wdown[0].zero_()
    _, m2, hs2 = oracle_for(s2, weights=w2)
    x0 = m2.embed(toks[0])
    x = x0[None].copy()
    m2.forward(0, 1, x, 0, m2.new_cache(1))
    a = torch.nn.functional.rms_norm(torch.from_numpy(x0).double(), (s2.d_model,), None, s2.rms_eps)
    v = (w2.wqkv[0].double() @ a)[(s2.n_q_heads + s2.n_kv_heads) * s2.head_dim:]
    np.testing.assert_allclose(x[0] - x0, (w2.wo[0].double() @ v).numpy(), atol=1e-6)


def test_uniform_attention_when_queries_are_zero():
    """Wq = 0 makes every score 0: the attention output is the plain mean of
    the cached V rows of the matching KV head (softmax rows sum to one)."""
    shape = SMALL
    w = wl.make_weights(shape, dtype=torch.float32)
    hq, hkv, hd = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    w.wqkv[0][: hq * hd].zero_()
    w.wdown[0].zero_()
    _, m, hs = oracle_for(shape, weights=w)
    toks = wl.make_tokens(shape, 5).tolist()
    emb = np.stack([m.embed(t) for t in toks])
    x = emb.copy()
    cache = m.new_cache(5)
    m.forward(0, 1, x, 0, cache)
    vmean = cache.v[0].astype(np.float64).mean(axis=0)            # [hkv][hd], mean over the 5 positions
    o = np.repeat(vmean, hq // hkv, axis=0).reshape(-1)           # q head h uses kv head h // (hq/hkv)
    np.testing.assert_allclose(x[4] - emb[4], w.wo[0].double().numpy() @ o, atol=1e-6)


def test_argmax_lowest_id_on_ties():
    _, m, _ = oracle_for(SMALL)
    z = np.array([0.5, 2.0, 2.0, -1.0, 1.5], np.float32)
    i, t1, t2 = m.argmax(z)
    assert (i, t1, t2) == (1, 2.0, 2.0)
