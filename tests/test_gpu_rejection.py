"""Rejection-sampling acceptance (App. G) on the GPU against the oracle, draw by draw on the same uniforms:
the stand-alone acceptance call on synthetic distributions (both stages, ragged batches, bonus rows, the
p == q and zero-mass corners), inversion sampling, and the sampling decoding loop end to end."""
import numpy as np
import pytest
import torch

from oracle import rejection as rj
from paper_2510_01336_b200 import workload as wl

pytestmark = pytest.mark.gpu

TOL_U = 2e-4      # a decision is compared only when u is this far from the threshold that decides it


def _binding():
    from paper_2510_01336_b200 import binding
    return binding


def _ctx(b, max_batch=8, max_rows=10):
    shape = wl.TINY
    wg = wl.make_weights(shape).to("cuda")
    ctx = b.Context(shape, wg, max_batch=max_batch, max_rows_per_seq=max_rows, max_pages_per_seq=8)
    st = ctx.new_state(max_batch, 8 * max_batch, wl.make_block_table(shape, max_batch, 8))
    return shape, ctx, st


def _token_ok(weights, u, tok):
    """tok is a valid inversion draw: u * total lies in tok's cumulative interval, up to rounding."""
    w = np.asarray(weights, np.float64)
    c = np.cumsum(w)
    t = u * c[-1]
    lo = c[tok] - w[tok]
    slack = 2e-5 * c[-1]
    return w[tok] > 0 and lo - slack <= t <= c[tok] + slack


def _check_stage(stage, k, seed):
    b = _binding()
    shape, ctx, st = _ctx(b)
    B, R, V = 8, ctx.max_rows, shape.vocab
    g = torch.Generator().manual_seed(seed)
    p_log = (torch.randn((B, R, V), generator=g) * 2.0)
    q_log = p_log + torch.randn((B, R, V), generator=g) * 0.7       # related distributions: a mix of keeps and rejections
    q_log[0] = p_log[0]                                               # sequence 0: p == q, everything is kept
    q_log[1, :, ::2] = -float("inf")                                  # sequence 1: q has no mass on even tokens
    P = rj.softmax_f32(p_log.numpy())
    Q = rj.softmax_f32(q_log.numpy())
    u_acc = torch.rand((B, R), generator=g)
    u_smp = torch.rand((B,), generator=g)
    base = 40
    rows = [k + 1, k + 1, k, 1, 0, k + 1, 2, k]                        # buffered rows per sequence (0: sits out)
    if stage == 2:
        rows = [min(r, k) for r in rows]
    acc_before = [0, 1, 2, 0, 0, 3, 1, 0] if stage == 1 else [0] * B    # rows already in V (stage 1 appends after them)
    S = torch.zeros((B, k), dtype=torch.int32)
    for s in range(B):
        nd = min(rows[s], k)
        for j in range(nd):
            S[s, j] = int(rj.sample_inverse_cdf(P[s, j], float(torch.rand((), generator=g))))
        if s == 1 and nd > 0:
            S[s, 0] = 2                                                # an even token: q gives it probability 0
        if stage == 1:
            st.len_target[s], st.len_inter[s], st.len_draft[s] = base - acc_before[s], base, base + rows[s]
        else:
            st.len_target[s], st.len_inter[s], st.len_draft[s] = base, base + rows[s], base + rows[s]
    res = ctx.new_result(B, ids=False)
    res.tentative = torch.full((B, R), -5, dtype=torch.int32, device="cuda")
    res.pending = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    stage_logits = torch.zeros((B, R, V), device="cuda") if stage == 1 else None
    pg, qg = p_log.cuda(), q_log.cuda()
    ctx.accept_rejection(stage, st, S.cuda(), k, pg, qg, u_acc.cuda(), u_smp.cuda(), res, stage_logits=stage_logits)
    assert ctx.status() == 0
    acc_g, nxt_g = res.n_accepted.cpu().tolist(), res.next_token.cpu().tolist()
    compared = 0
    for s in range(B):
        nr, nd = rows[s], min(rows[s], k)
        if nr == 0:
            assert (int(st.len_draft[s]), int(st.len_inter[s])) == (base, base) if stage == 1 else True
            continue
        out, a = rj.rejection_verify(S[s, :nd].tolist(), P[s, :nd], Q[s, :nr], u_acc[s].tolist(), float(u_smp[s]))
        # decisions the fp32 rounding of either side could flip are not compared
        fragile = False
        for j in range(min(a + 1, nd)):
            tok = int(S[s, j])
            ratio = 1.0 if not P[s, j, tok] > 0 else min(1.0, float(Q[s, j, tok]) / float(P[s, j, tok]))
            fragile |= abs(float(u_acc[s, j]) - ratio) < TOL_U and ratio < 1.0
        if fragile:
            continue
        compared += 1
        assert acc_g[s] == a, (stage, s, acc_g[s], a)
        if a < nr:
            w = rj.residual(P[s, a] if a < nd else None, Q[s, a])
            if not w.sum() > 0:
                w = Q[s, a]
            assert _token_ok(w, float(u_smp[s]), nxt_g[s]), (stage, s, nxt_g[s], out)
            assert int(res.pending[s]) == nxt_g[s]
        else:
            assert nxt_g[s] == -1 and int(res.pending[s]) == int(S[s, a - 1])
        nl = (base if stage == 1 else base) + min(a + 1, nr)
        assert int(st.len_draft[s]) == nl and int(st.len_inter[s]) == nl
        assert int(st.len_target[s]) == (nl if stage == 2 else base - acc_before[s])
        if stage == 1:
            tv = res.tentative[s].cpu().tolist()
            d0 = acc_before[s]
            assert tv[d0:d0 + a] == S[s, :a].tolist()
            if a < nr:
                assert tv[d0 + a] == nxt_g[s]
            kept = min(a + 1, nr)
            assert torch.equal(stage_logits[s, d0:d0 + kept].cpu(), q_log[s, :kept])
    assert compared >= 5
    # the corners did what they must: p == q keeps every draft; zero-mass token is rejected at once
    assert acc_g[0] == min(rows[0], k)
    assert acc_g[1] == 0 and nxt_g[1] % 2 == 1
    ctx.close()


@pytest.mark.parametrize("stage,k,seed", [(1, 5, 1), (1, 3, 2), (2, 6, 3), (2, 4, 4)])
def test_accept_rejection_matches_oracle_draw_by_draw(stage, k, seed):
    _check_stage(stage, k, seed)


def test_inversion_sampling_matches_oracle():
    b = _binding()
    shape, ctx, st = _ctx(b)
    B, V = 8, shape.vocab
    g = torch.Generator().manual_seed(9)
    logits = torch.randn((B, 3, V), generator=g) * 3.0
    logits[2, 1, 5:] = -float("inf")
    u = torch.rand((B,), generator=g)
    u[0], u[1] = 0.0, 0.9999999
    out = torch.full((B, 2), -1, dtype=torch.int32, device="cuda")
    lg = logits.cuda()
    for temp in (1.0, 0.5):
        ctx.sample(lg.data_ptr() + 4 * V, 3 * V, u.cuda(), out, B, out_stride=2, temperature=temp)   # row 1 of every sequence
        torch.cuda.synchronize()
        P = rj.softmax_f32(logits[:, 1].numpy(), temperature=temp)
        for s in range(B):
            assert _token_ok(P[s], float(u[s]), int(out[s, 0])), (temp, s)
        assert int(out[2, 0]) < 5 and torch.all(out[:, 1] == -1)
    ctx.close()


def test_sampling_loop_end_to_end():
    """The sampling decoding loop on the device: (1) every acceptance the loop makes is re-derived by the
    oracle from the very logits, drafts and uniforms the kernel read; (2) at a temperature close to zero the
    loop reproduces the GPU's own greedy auto-regressive output (the limit in which sampling is greedy)."""
    b = _binding()
    from paper_2510_01336_b200.driver import ARLoop, HiSpecSamplingLoop
    shape = wl.TINY
    scale = {l: 0.05 for l in range(shape.L_d, shape.L_f)}
    wg = wl.make_weights(shape, resid_scale=scale).to("cuda")
    B, N_d, rounds, n_prompt, n_gen = 2, 3, 2, 48, 20
    max_rows = rounds * (N_d + 1) + 3
    max_pages = (n_prompt + n_gen + 40) // 16 + 1
    prompts = [wl.make_tokens(shape, n_prompt, seed_offset=1000 + s).tolist() for s in range(B)]
    bt = wl.make_block_table(shape, B, max_pages)
    uni = lambda sr: wl.make_uniforms(shape, sr, B, rounds, N_d, max_rows)

    records = []
    ctx = b.Context(shape, wg, max_batch=B, max_rows_per_seq=max_rows, max_pages_per_seq=max_pages)
    st = ctx.new_state(B, max_pages * B, bt)
    loop = HiSpecSamplingLoop(ctx, st, B, N_d, rounds, uni, temperature=1.0,
                              on_accept=lambda stage, rnd, rec: records.append((stage, rnd, rec)))
    loop.prefill(prompts)
    toks = loop.generate(n_gen)
    assert ctx.status() == 0
    assert all(len(t) == n_gen and all(0 <= x < shape.vocab for x in t) for t in toks)
    compared = kept = 0
    for stage, rnd, rec in records:
        P = rj.softmax_f32(rec["p"].numpy())
        Q = rj.softmax_f32(rec["q"].numpy())
        ld, li, lf = (x.tolist() for x in rec["lens_before"])
        for s in range(B):
            avail = ld[s] - li[s] if stage == 1 else li[s] - lf[s]
            nr = min(avail, rec["k"] + 1)
            nd = min(nr, rec["k"])
            assert nr >= 1
            S = rec["S"][s, :nd].tolist()
            out, a = rj.rejection_verify(S, P[s, :nd], Q[s, :nr], rec["u_acc"][s].tolist(), float(rec["u_smp"][s]))
            fragile = False
            for j in range(min(a + 1, nd)):
                ratio = 1.0 if not P[s, j, S[j]] > 0 else min(1.0, float(Q[s, j, S[j]]) / float(P[s, j, S[j]]))
                fragile |= abs(float(rec["u_acc"][s, j]) - ratio) < TOL_U and ratio < 1.0
            if fragile:
                continue
            compared += 1
            kept += a
            assert int(rec["n_accepted"][s]) == a
            p0 = li[s] if stage == 1 else lf[s]
            nl = p0 + min(a + 1, nr)
            la = [int(x[s]) for x in rec["lens_after"]]
            assert la[0] == nl and la[1] == nl and la[2] == (nl if stage == 2 else lf[s])
            if a < nr:
                w = rj.residual(P[s, a] if a < nd else None, Q[s, a])
                if not w.sum() > 0:
                    w = Q[s, a]
                nxt = int(rec["next_token"][s])
                assert _token_ok(w, float(rec["u_smp"][s]), nxt) and int(rec["pending"][s]) == nxt
            if stage == 1:
                d0 = li[s] - lf[s]
                assert rec["V"][s, d0:d0 + a].tolist() == S[:a]
    assert compared >= 10 and kept > 0
    ctx.close()

    outs = {}
    for name in ("ar", "cold"):
        ctx = b.Context(shape, wg, max_batch=B, max_rows_per_seq=max_rows, max_pages_per_seq=max_pages)
        st = ctx.new_state(B, max_pages * B, bt)
        loop = ARLoop(ctx, st, B) if name == "ar" else HiSpecSamplingLoop(ctx, st, B, N_d, rounds, uni, temperature=1e-3)
        loop.prefill(prompts)
        outs[name] = loop.generate(n_gen)
        assert ctx.status() == 0
        ctx.close()
    assert outs["cold"] == outs["ar"]
