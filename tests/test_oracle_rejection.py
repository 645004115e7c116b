"""Pins of the rejection-sampling oracle (App. G): the single-position lemma by exact enumeration, the
acceptance probability's closed form, special cases, and the two-stage composition by seeded Monte Carlo."""
import numpy as np

from oracle import rejection as rj


def _dist(rng, V, zeros=0):
    x = rng.random(V) ** 3
    if zeros:
        x[rng.choice(V, zeros, replace=False)] = 0.0
    return (x / x.sum()).astype(np.float32)


def test_softmax_and_inverse_cdf_definitions():
    z = np.array([0.0, np.log(2.0), np.log(5.0), -np.inf], dtype=np.float32)
    p = rj.softmax_f32(z)
    np.testing.assert_allclose(p, [1 / 8, 2 / 8, 5 / 8, 0.0], rtol=1e-6)
    np.testing.assert_allclose(rj.softmax_f32(z, temperature=0.5), np.array([1, 4, 25, 0]) / 30.0, rtol=1e-6)
    w = np.array([0.0, 1.0, 0.0, 3.0, 0.0])
    # cumulative bounds 0,1,1,4,4: u*4 in [0,1) -> 1, [1,4) -> 3
    assert [rj.sample_inverse_cdf(w, u) for u in (0.0, 0.2, 0.2499, 0.25, 0.5, 0.999999)] == [1, 1, 1, 3, 3, 3]


def test_single_position_lemma_by_exact_enumeration():
    """P(out = v) = p(v) min(1, q(v)/p(v)) + (1 - sum_w min(p(w), q(w))) res(v) must equal q(v): evaluated from
    the oracle's own pieces (ratio test, residual) with exact integration over u."""
    rng = np.random.default_rng(7)
    for V, zeros in ((5, 0), (8, 2), (16, 5)):
        p, q = _dist(rng, V, zeros), _dist(rng, V, zeros)
        out = np.zeros(V)
        for s in range(V):
            if p[s] == 0:
                continue
            # the stage keeps s exactly when u < min(1, q/p): probe the oracle just below and above the threshold
            thr = min(1.0, float(q[s]) / float(p[s]))
            for u, keep in ((max(thr - 1e-6, 0.0), thr > 0.0), (min(thr + 1e-6, 1.0), False)):
                if thr >= 1.0 and not keep:
                    continue
                res, a = rj.rejection_verify([s], p[None], q[None], [u], 0.5)
                assert (a == 1) == keep
            out[s] += p[s] * thr
            r = rj.residual(p, q).astype(np.float64)
            if r.sum() > 0:
                out += p[s] * (1.0 - thr) * r / r.sum()
        np.testing.assert_allclose(out, q, atol=2e-6)


def test_acceptance_probability_closed_form_and_special_cases():
    rng = np.random.default_rng(11)
    V, n = 12, 40000
    p, q = _dist(rng, V), _dist(rng, V)
    s = rng.choice(V, size=n, p=p / p.sum())
    u, us = rng.random(n), rng.random(n)
    kept, toks = 0, np.zeros(V)
    for i in range(n):
        res, a = rj.rejection_verify([int(s[i])], p[None], q[None], [u[i]], us[i])
        kept += a
        toks[res[0]] += 1
    expect = np.minimum(p, q).sum()            # P(accept) = sum_v min(p(v), q(v))
    assert abs(kept / n - expect) < 4 * np.sqrt(expect * (1 - expect) / n)
    assert np.all(np.abs(toks / n - q) < 4 * np.sqrt(q * (1 - q) / n) + 1e-3)      # output ~ q
    # p == q: everything is kept whatever u is; the bonus token comes from q's inverse CDF
    res, a = rj.rejection_verify([3, 1], np.stack([q, q]), np.stack([q, q, p]), [0.999999, 0.999999], 0.0)
    assert a == 2 and res[:2] == [3, 1] and res[2] == int(np.nonzero(p)[0][0])
    # q puts no mass on the draft token: always replaced, never by the same token
    q0 = q.copy(); q0[5] = 0; q0 /= q0.sum()
    res, a = rj.rejection_verify([5, 2], np.stack([p, p]), np.stack([q0, q0]), [0.0, 0.0], 0.3)
    assert a == 0 and len(res) == 1 and res[0] != 5
    # the first failure discards the rest of the block
    res, a = rj.rejection_verify([1, 2, 3], np.stack([p] * 3), np.stack([q] * 3), [0.0, 1.0, 0.0], 0.7)
    assert a == 1 and len(res) == 2 and res[0] == 1


def test_two_stage_composition_reproduces_the_final_distribution():
    """Draft from p_d, filter by p_i, filter again by p_f (App. G): the first emitted token must follow p_f.
    Context-free toy exits (the same three distributions at every position), blocks of 2, bonus rows on."""
    rng = np.random.default_rng(3)
    V, n = 6, 30000
    pd, pi, pf = _dist(rng, V), _dist(rng, V), _dist(rng, V)
    counts = np.zeros(V)
    second = np.zeros(V)
    for _ in range(n):
        S = [int(rng.choice(V, p=pd / pd.sum())) for _ in range(2)]
        Vl, _ = rj.rejection_verify(S, np.stack([pd] * 2), np.stack([pi] * 3), rng.random(2), rng.random())
        F, _ = rj.rejection_verify(Vl, np.stack([pi] * len(Vl)), np.stack([pf] * len(Vl)), rng.random(len(Vl)), rng.random())
        counts[F[0]] += 1
        if len(F) > 1:
            second[F[1]] += 1
    assert np.all(np.abs(counts / n - pf) < 4 * np.sqrt(pf * (1 - pf) / n) + 1e-3)
    m = second.sum()
    assert m > n / 4 and np.all(np.abs(second / m - pf) < 5 * np.sqrt(pf * (1 - pf) / m) + 2e-3)


def test_sampling_generation_at_low_temperature_is_greedy_decoding():
    """As the temperature goes to 0 every distribution becomes one-hot on its argmax: drafts are the greedy
    drafts, the ratio test keeps exactly the tokens the verifier's argmax agrees with, the residual is the
    verifier's argmax -- so sampling-based HiSpec must reproduce greedy auto-regressive decoding."""
    from paper_2510_01336_b200 import workload as wl
    from tests.helpers import oracle_for
    shape = wl.TINY
    scale = {l: 0.05 for l in range(shape.L_d, shape.L_f)}
    _, _, hs = oracle_for(shape, resid_scale=scale)
    prompt = wl.make_tokens(shape, 20).tolist()
    n_gen, N_d, rounds = 24, 3, 2
    uni = lambda sr: wl.make_uniforms(shape, sr, 1, rounds, N_d, rounds * (N_d + 1) + 2)
    ar = hs.ar_generate(prompt, n_gen)
    st = __import__("oracle.hispec", fromlist=["GenStats"]).GenStats()
    out = hs.hispec_generate_sampling(prompt, n_gen, N_d, rounds, uni, temperature=1e-3, stats=st)
    assert out == ar
    assert st.inter_accepted > 0 and st.target_accepted > 0
    # at temperature 1 the output differs from greedy (it is a sample) but every stage call keeps the state consistent
    out1 = hs.hispec_generate_sampling(prompt, n_gen, N_d, rounds, uni, temperature=1.0)
    assert len(out1) == n_gen and out1[0] == ar[0] and out1 != ar
