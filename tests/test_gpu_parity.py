"""GPU parity: every C-ABI call against the oracle's stage call on the same seeded
inputs, teacher-forced (the oracle's state is loaded before each call), through
libhispec.so.  Tolerances: exit hidden rows 1e-2 relative L2, logits 5e-2 max
abs, ids / accepted length / correction token bit-exact except where the
oracle's top-2 margin is below 0.1 (there the id must lie in the near-tie set and
the acceptance must follow the GPU's own ids)."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle.hispec import GenStats, HiSpecOracle, OracleModel
from paper_2510_01336_b200 import workload as wl
from tests import gpu_harness as gh
from tests.helpers import oracle_for

pytestmark = pytest.mark.gpu

FLAG_SETS = {"tcgen05": 0, "simt": 1, "tcgen05-plain": 2, "rowwarp-attn": 8, "multi-kernel": 16}


def _binding():
    from paper_2510_01336_b200 import binding
    return binding


class GpuObserver:
    """Runs every stage call of the oracle's decoding loop on the GPU as well, from the oracle's state."""

    def __init__(self, ctx, st, hs, page_size, max_rows):
        self.ctx, self.st, self.hs, self.ps, self.max_rows = ctx, st, hs, page_size, max_rows
        self.layers = list(range(hs.m.n_layers))
        self.calls = {"draft": 0, "verify_i": 0, "verify_t": 0}
        self.worst = {"rel_l2": 0.0, "logit_err": 0.0, "exempt": 0, "rows": 0}
        self.b = _binding()

    def before(self, kind, ost, seq_tokens, **kw):
        b = self.b
        gh.load_seq(self.st, 0, ost, self.ps, self.layers, self.max_rows)
        self.res = self.ctx.new_result(1, logits=True, hidden=True)
        self.kind, self.kw = kind, kw
        self.pre = (ost.len_d, ost.len_i, ost.len_f)
        dev = "cuda"
        if kind == "draft":
            self.out_tok = torch.full((1,), -5, dtype=torch.int32, device=dev)
            self.ctx.draft(self.st, torch.tensor([kw["token"]], dtype=torch.int32, device=dev), self.out_tok, self.res)
        else:
            S, R = kw["S"], kw["n_rows"]
            k = max(len(S), 1)
            dt = torch.zeros((1, k), dtype=torch.int32, device=dev)
            if S:
                dt[0, : len(S)] = torch.tensor(S, dtype=torch.int32)
            nd = torch.tensor([len(S)], dtype=torch.int32, device=dev)
            nr = torch.tensor([R], dtype=torch.int32, device=dev)
            fn = self.ctx.verify_intermediate if kind == "verify_i" else self.ctx.verify_target
            fn(self.st, dt, nd, nr, self.res)
        torch.cuda.synchronize()
        assert self.ctx.status() == 0

    def after(self, kind, ost, out):
        hs, st = self.hs, self.st
        R = 1 if kind == "draft" else self.kw["n_rows"]
        S = [] if kind == "draft" else self.kw["S"]
        s = gh.compare_exit(out, self.res, 0, R, S, check_accept=(kind != "draft"), tag=f"{kind}#{self.calls[kind]}")
        for k in ("rel_l2", "logit_err"):
            self.worst[k] = max(self.worst[k], s[k])
        self.worst["exempt"] += s["exempt"]
        self.worst["rows"] += R
        l0, l1, p0 = {"draft": (0, hs.L_d, self.pre[0]), "verify_i": (hs.L_d, hs.L_i, self.pre[1]),
                      "verify_t": (hs.L_i, hs.L_f, self.pre[2])}[kind]
        gh.compare_kv(st, 0, ost, self.ps, range(l0, l1), range(p0, p0 + R), tag=kind)
        if kind == "draft":
            gid = int(self.out_tok[0])
            assert gid == int(self.res.argmax_ids[0, 0])
            exp = (self.pre[0] + 1, self.pre[1], self.pre[2])
            row = st.h_draft[0, self.pre[0] - self.pre[1]].cpu().numpy()
            assert np.linalg.norm(row - out.hidden[0]) <= gh.HIDDEN_REL_L2 * np.linalg.norm(out.hidden[0])
        else:
            a = int(self.res.n_accepted[0])
            nl = p0 + min(a + 1, R)
            exp = (nl, nl, self.pre[2]) if kind == "verify_i" else (nl, nl, nl)
            if kind == "verify_i":
                base = self.pre[1] - self.pre[2]
                rows = st.h_inter[0, base: base + R].cpu().numpy()
                rel = np.linalg.norm(rows - out.hidden, axis=1) / np.linalg.norm(out.hidden, axis=1)
                assert rel.max() <= gh.HIDDEN_REL_L2
        got = (int(st.len_draft[0]), int(st.len_inter[0]), int(st.len_target[0]))
        assert got == exp, f"{kind}: lengths {got} != {exp}"
        self.calls[kind] += 1


def _tiny_setup(flags, n_prompt, n_gen, N_d, rounds, resid_scale=None):
    b = _binding()
    shape = wl.TINY
    w, m, hs = oracle_for(shape, kv_round=True, resid_scale=resid_scale)
    max_rows = rounds * (N_d + 1) + 2
    max_pages = (n_prompt + n_gen + max_rows + 2 + 15) // 16 + 1
    ctx = b.Context(shape, w.to("cuda"), page_size=16, max_batch=1, max_rows_per_seq=max_rows,
                    max_pages_per_seq=max_pages, flags=flags)
    bt = wl.make_block_table(shape, 1, max_pages, n_pages=max_pages + 5)
    st = ctx.new_state(1, max_pages + 5, bt)
    return shape, w, m, hs, ctx, st, max_rows


@pytest.mark.parametrize("flagname", ["simt", "tcgen05", "tcgen05-plain", "rowwarp-attn", "multi-kernel"])
def test_tiny_config_every_call(flagname):
    """cfg "tiny" as stated: prompt 128, k = 4 greedy drafts from the draft exit, target every 2
    rounds, 64 generated tokens -- every draft / verify-I / verify-T call compared."""
    n_gen = 64 if flagname == "tcgen05" else 12
    shape, w, m, hs, ctx, st, max_rows = _tiny_setup(FLAG_SETS[flagname], 128, n_gen, 4, 2)
    prompt = wl.make_tokens(shape, 128).tolist()
    obs = GpuObserver(ctx, st, hs, 16, max_rows)
    out = hs.hispec_generate(prompt, n_gen, 4, rounds=2, observer=obs, rows_cap=max_rows)
    assert len(out) == n_gen and min(obs.calls.values()) > 0
    print(f"\n[{flagname}] calls {obs.calls} worst rel-L2 {obs.worst['rel_l2']:.2e} logits {obs.worst['logit_err']:.2e} "
          f"exempt rows {obs.worst['exempt']}/{obs.worst['rows']}")
    ctx.close()


def test_tiny_accepting_drafts_and_target_bonus():
    """Weights whose deeper exits mostly agree with the shallower ones (Wo, Wdown of the layers above the draft
    exit scaled by 0.05), the paper's |V| >= N_i trigger and a bonus row at the target: accept, partial-accept
    and reject paths of both verifiers on the GPU."""
    scale = {l: 0.05 for l in range(wl.TINY.L_d, wl.TINY.L_f)}
    shape, w, m, hs, ctx, st, max_rows = _tiny_setup(0, 40, 30, 3, 3, resid_scale=scale)
    prompt = wl.make_tokens(shape, 40).tolist()
    ar = hs.ar_generate(prompt, 30)
    obs = GpuObserver(ctx, st, hs, 16, max_rows)
    stt = GenStats()
    out = hs.hispec_generate(prompt, 30, 3, N_i=4, bonus_target=True, observer=obs, stats=stt, rows_cap=max_rows)
    assert out == ar and stt.inter_accepted > 5 and stt.target_accepted > 5, stt
    assert stt.inter_accepted < stt.drafted
    ctx.close()


def test_tiny_prefill_and_free_running_lossless():
    """Prefill vs the oracle; then, free-running on the GPU alone, HiSpec's output must equal the GPU's own
    auto-regressive greedy output (the lossless guarantee, on the device arithmetic)."""
    b = _binding()
    from paper_2510_01336_b200.driver import ARLoop, HiSpecLoop
    shape = wl.TINY
    w, m, hs = oracle_for(shape, kv_round=True)
    wg = w.to("cuda")
    n_prompt, n_gen, N_d, rounds = 128, 64, 4, 2
    max_rows = rounds * (N_d + 1) + 3
    max_pages = (n_prompt + n_gen + 40) // 16 + 1
    prompt = wl.make_tokens(shape, n_prompt).tolist()

    ctx = b.Context(shape, wg, max_batch=1, max_rows_per_seq=max_rows, max_pages_per_seq=max_pages)
    bt = wl.make_block_table(shape, 1, max_pages)
    st = ctx.new_state(1, max_pages, bt)
    loop = HiSpecLoop(ctx, st, 1, N_d, rounds)
    first = loop.prefill([prompt])
    # oracle prefill: first token (margin rule), lengths, KV of every layer
    ost = hs.new_state(n_prompt + 8, 4)
    o = hs.prefill(ost, prompt)
    if o.top2[0, 0] - o.top2[0, 1] >= gh.MARGIN:
        assert first[0] == o.argmax_ids[0]
    assert (int(st.len_draft[0]), int(st.len_inter[0]), int(st.len_target[0])) == (n_prompt,) * 3
    bt_row = st.block_table[0].cpu()
    for l in range(shape.n_layers):
        g = gh.cache_from_pages(st.k_pages, bt_row, 16, l, 0, range(n_prompt))
        r = ost.cache.k[l, :n_prompt]
        assert np.linalg.norm(g - r) / np.linalg.norm(r) < 1e-2
    toks = loop.generate(n_gen)[0]
    assert ctx.status() == 0

    ctx2 = b.Context(shape, wg, max_batch=1, max_rows_per_seq=max_rows, max_pages_per_seq=max_pages)
    st2 = ctx2.new_state(1, max_pages, bt)
    ar = ARLoop(ctx2, st2, 1)
    ar.prefill([prompt])
    ar_toks = ar.generate(n_gen)[0]
    assert ctx2.status() == 0
    assert toks == ar_toks, "HiSpec on the GPU must reproduce the GPU's auto-regressive greedy output"
    assert loop.stats.committed >= n_gen - 1 and loop.stats.target_calls > 0
    ctx.close(); ctx2.close()


def test_tiny_dynamic_trigger_and_single_stage_loops_are_lossless():
    """The paper's dynamic trigger (|V| >= N_i) and Algorithm 1, free-running on the GPU with weights whose
    exits mostly agree: both must reproduce the GPU's own auto-regressive greedy output."""
    b = _binding()
    from paper_2510_01336_b200.driver import ARLoop, HiSpecDynamicLoop, SelfSpecLoop
    shape = wl.TINY
    scale = {l: 0.05 for l in range(shape.L_d, shape.L_f)}
    wg = wl.make_weights(shape, resid_scale=scale).to("cuda")
    n_prompt, n_gen, N_d, N_i = 64, 48, 2, 4
    max_rows, max_pages = 12, (n_prompt + n_gen + 40) // 16 + 1
    prompt = wl.make_tokens(shape, n_prompt).tolist()
    bt = wl.make_block_table(shape, 1, max_pages)
    outs = {}
    for name in ("ar", "dynamic", "selfspec"):
        ctx = b.Context(shape, wg, max_batch=1, max_rows_per_seq=max_rows, max_pages_per_seq=max_pages)
        st = ctx.new_state(1, max_pages, bt)
        loop = {"ar": lambda: ARLoop(ctx, st, 1), "dynamic": lambda: HiSpecDynamicLoop(ctx, st, 1, N_d, N_i),
                "selfspec": lambda: SelfSpecLoop(ctx, st, 1, N_d)}[name]()
        loop.prefill([prompt])
        outs[name] = loop.generate(n_gen)[0]
        assert ctx.status() == 0
        if name == "dynamic":
            assert loop.stats.inter_accepted > 5 and loop.stats.target_accepted > 5
            assert loop.stats.inter_calls > loop.stats.target_calls       # several rounds per target verification
        ctx.close()
    assert outs["dynamic"] == outs["ar"] and outs["selfspec"] == outs["ar"]


@pytest.mark.parametrize("flagname", ["tcgen05", "multi-kernel"])
def test_draft_block_equals_separate_draft_steps(flagname):
    """hispec_draft_block (all draft steps of a round in one call) against the same steps as separate calls:
    the same tokens, length counters, buffered exit rows and appended K/V, bit for bit."""
    b = _binding()
    shape = wl.TINY
    wg = wl.make_weights(shape).to("cuda")
    flags = {"tcgen05": 0, "multi-kernel": b.FLAG_MULTI_KERNEL}[flagname]
    B, N_d, n_prompt = 3, 4, 40
    max_rows, max_pages = 8, 6
    prompts = [wl.make_tokens(shape, n_prompt - 3 * s, seed_offset=1000 + s).tolist() for s in range(B)]
    bt = wl.make_block_table(shape, B, max_pages)
    outs = []
    for mode in ("separate", "block"):
        ctx = b.Context(shape, wg, max_batch=B, max_rows_per_seq=max_rows, max_pages_per_seq=max_pages, flags=flags)
        st = ctx.new_state(B, B * max_pages, bt)
        mx = max(len(p) for p in prompts)
        toks = torch.zeros((B, mx), dtype=torch.int32)
        for s_, p in enumerate(prompts):
            toks[s_, : len(p)] = torch.tensor(p, dtype=torch.int32)
        pending = torch.zeros(B, dtype=torch.int32, device="cuda")
        ctx.prefill(st, toks.cuda(), torch.tensor([len(p) for p in prompts], dtype=torch.int32).cuda(), pending)
        S = torch.full((B, N_d), -1, dtype=torch.int32, device="cuda")
        for rnd in range(2):      # two rounds in a row: the second starts from the first one's state
            if mode == "block":
                ctx.draft_block(st, pending, S, N_d, bonus=True)
            else:
                p_ = S.data_ptr()
                ctx.draft(st, pending, p_, batch=B, in_stride=1, out_stride=N_d)
                for j in range(1, N_d):
                    ctx.draft(st, p_ + 4 * (j - 1), p_ + 4 * j, batch=B, in_stride=N_d, out_stride=N_d)
                ctx.draft(st, p_ + 4 * (N_d - 1), None, batch=B, in_stride=N_d)
            if rnd == 0:          # accept nothing: prune the draft group back by hand to one token past the start
                S0 = S.clone()
                st.len_draft.copy_(st.len_inter + 1)
                pending = S0[:, 0].contiguous()
        assert ctx.status() == 0
        outs.append((S0.cpu(), S.cpu(), st.len_draft.cpu(), st.len_inter.cpu(), st.h_draft.cpu().clone(),
                     st.k_pages.cpu().clone(), st.v_pages.cpu().clone()))
        ctx.close()
    for x, y in zip(*outs):
        assert torch.equal(x, y)
    assert int(outs[0][2][0]) == len(prompts[0]) + 1 + N_d + 1


def test_tiny_chain_of_two_intermediate_verifiers_is_lossless():
    """Two intermediate verifiers (exits 1 < 2 < 3 < 4, App. K) composed from the three-exit calls: the output
    equals the GPU's own auto-regressive greedy output, and every level accepted something."""
    b = _binding()
    from paper_2510_01336_b200.driver import ARLoop, HiSpecChainLoop
    shape = wl.TINY
    scale = {l: 0.05 for l in range(1, shape.n_layers)}
    wg = wl.make_weights(shape, resid_scale=scale).to("cuda")
    B, n_prompt, n_gen, N_d, m1, m2 = 2, 48, 40, 2, 2, 2
    max_pages = (n_prompt + n_gen + 40) // 16 + 1
    prompts = [wl.make_tokens(shape, n_prompt - 5 * s, seed_offset=1000 + s).tolist() for s in range(B)]
    bt = wl.make_block_table(shape, B, max_pages)
    loop = HiSpecChainLoop(shape, wg, (1, 2, 3, 4), B, N_d, m1, m2, max_pages, bt)
    loop.prefill(prompts)
    toks = loop.generate(n_gen)
    assert loop.status() == 0
    acc1 = sum(int(r.n_accepted.sum()) for r in loop.res1)
    acc2 = sum(int(r.n_accepted.sum()) for r in loop.res2)
    assert acc1 > 0 and acc2 > 0 and loop.stats.target_accepted > 0
    assert loop.stats.inter_calls == loop.stats.super_rounds * (m1 * m2 + m2)
    loop.close()
    ctx = b.Context(shape, wg, max_batch=B, max_rows_per_seq=4, max_pages_per_seq=max_pages)
    st = ctx.new_state(B, int(bt.max()) + 1, bt)
    ar = ARLoop(ctx, st, B)
    ar.prefill(prompts)
    assert toks == ar.generate(n_gen)
    ctx.close()


def test_tiny_adaptive_parameters_loop_is_lossless():
    """Adaptive N_d / N_i (App. J) free-running on the GPU: the output equals the GPU's own auto-regressive
    greedy output, both parameters move, and the recorded schedule obeys the oracle's update rule."""
    b = _binding()
    from oracle import hispec as oh
    from paper_2510_01336_b200.driver import ARLoop, HiSpecAdaptiveLoop
    shape = wl.TINY
    scale = {l: 0.05 for l in range(shape.L_d, shape.L_f)}
    wg = wl.make_weights(shape, resid_scale=scale).to("cuda")
    n_prompt, n_gen = 64, 64
    max_rows, max_pages = 14, (n_prompt + n_gen + 40) // 16 + 1
    prompt = wl.make_tokens(shape, n_prompt).tolist()
    bt = wl.make_block_table(shape, 1, max_pages)
    ctx = b.Context(shape, wg, max_batch=1, max_rows_per_seq=max_rows, max_pages_per_seq=max_pages)
    st = ctx.new_state(1, max_pages, bt)
    loop = HiSpecAdaptiveLoop(ctx, st, 1, 2, 4)
    loop.prefill([prompt])
    toks = loop.generate(n_gen)[0]
    assert ctx.status() == 0
    ctx.close()
    ctx2 = b.Context(shape, wg, max_batch=1, max_rows_per_seq=max_rows, max_pages_per_seq=max_pages)
    st2 = ctx2.new_state(1, max_pages, bt)
    ar = ARLoop(ctx2, st2, 1)
    ar.prefill([prompt])
    assert toks == ar.generate(n_gen)[0]
    ctx2.close()
    n_d, n_i = 2, 4
    seen_d, seen_i = set(), set()
    for rec in loop.schedule:
        if rec[0] == "i":
            assert rec[1] == n_d and 0 <= rec[2] <= n_d
            seen_d.add(n_d)
            n_d = oh.adaptive_step(n_d, rec[2] / rec[1], oh.ADAPT_ND_PAPER)
        else:
            assert rec[1] == n_i and rec[2] >= 1 and rec[3] <= rec[2]
            seen_i.add(n_i)
            n_i = oh.adaptive_step(n_i, rec[3] / rec[2], oh.ADAPT_NI_PAPER)
    assert len(seen_d) > 1 and len(seen_i) > 1


@pytest.mark.parametrize("flagname,B", [("tcgen05", 3), ("simt", 3), ("rowwarp-attn", 3), ("multi-kernel", 3),
                                        ("tcgen05", 12), ("tcgen05", 16), ("tcgen05", 20), ("tcgen05", 30), ("tcgen05", 64)])
def test_batched_ragged_gqa_pages_permuted(flagname, B):
    """GQA 2:1, head_dim 128, odd sizes (d 320, ffn 400, vocab 1000): a batch of 3 sequences with different
    context lengths, ragged row counts and scattered pages against the oracle, one sequence at a time;
    then the same call with another page permutation must give bit-identical results."""
    b = _binding()
    shape = wl.MINI_GQA
    w, m, hs = oracle_for(shape, kv_round=True)
    # B = 12 and 16 give 96 and 128 padded rows (kernel-sequence path, one weight tile per CTA, one MMA over both
    # planes), B = 20 gives 160 (two weight tiles per activation tile), B = 30 gives 240 (one MMA per plane, separate
    # accumulators), B = 64 -- the largest batch of the persistent kernel's tables -- gives 512 (two row chunks of 256)
    N_d, max_rows, page = 4, 8, 16
    ctx_lens = ([37, 5, 64, 16, 33] * 13)[:B]
    n_rows = ([5, 3, 4, 1, 5] * 13)[:B]
    n_draft = ([4, 3, 4, 1, 4] * 13)[:B]
    max_pages = 8
    ctx = b.Context(shape, w.to("cuda"), page_size=page, max_batch=B, max_rows_per_seq=max_rows,
                    max_pages_per_seq=max_pages, flags=FLAG_SETS[flagname])
    outs, states = [], []
    drafts = []
    for s in range(B):
        prompt = wl.make_tokens(shape, ctx_lens[s], seed_offset=100 + s).tolist()
        ost = hs.new_state(ctx_lens[s] + 16, max_rows)
        pending = hs.prefill(ost, prompt).argmax_ids[0]
        ar = hs.ar_generate(prompt, 8)
        S = [ar[1 + j] if j < 2 else (ar[1 + j] + 7) % shape.vocab for j in range(n_draft[s])]
        u = pending
        for t in (S + [None])[: n_rows[s]]:
            hs.draft_step(ost, u)
            u = t
        drafts.append(S)
        states.append(ost)
    results = []
    for perm_seed in (3000, 3001):
        bt = wl.make_block_table(shape, B, max_pages, n_pages=B * max_pages + 7, seed_offset=perm_seed)
        st = ctx.new_state(B, B * max_pages + 7, bt)
        for s in range(B):
            gh.load_seq(st, s, states[s], page, range(shape.n_layers), max_rows)
        res = ctx.new_result(B, logits=True, hidden=True)
        dt = torch.zeros((B, N_d), dtype=torch.int32)
        for s in range(B):
            dt[s, : n_draft[s]] = torch.tensor(drafts[s], dtype=torch.int32)
        ctx.verify_intermediate(st, dt.cuda(), torch.tensor(n_draft, dtype=torch.int32).cuda(),
                                torch.tensor(n_rows, dtype=torch.int32).cuda(), res)
        torch.cuda.synchronize()
        assert ctx.status() == 0
        results.append((res, st))
    import copy
    res, st = results[0]
    for s in range(B):
        ost = copy.deepcopy(states[s])
        p0 = ost.len_i
        out = hs.verify_intermediate(ost, drafts[s], n_rows[s])
        gh.compare_exit(out, res, s, n_rows[s], drafts[s], check_accept=True, tag=f"seq{s}")
        gh.compare_kv(st, s, ost, page, range(hs.L_d, hs.L_i), range(p0, p0 + n_rows[s]), tag=f"seq{s}")
        assert int(st.len_inter[s]) == ost.len_i == int(st.len_draft[s])
    r2 = results[1][0]
    for name in ("n_accepted", "next_token", "argmax_ids", "logits", "hidden_out"):
        assert torch.equal(getattr(res, name), getattr(r2, name)), f"page permutation changed {name}"
    ctx.close()


def test_errors_and_status_word():
    """Host-detected errors return codes and enqueue nothing; device-detected faults set status bits and
    the call completes (no trap, no hang)."""
    b = _binding()
    shape = wl.TINY
    w = wl.make_weights(shape).to("cuda")
    ctx = b.Context(shape, w, max_batch=2, max_rows_per_seq=6, max_pages_per_seq=4)
    bt = wl.make_block_table(shape, 2, 4)
    st = ctx.new_state(2, 8, bt)
    res = ctx.new_result(2)
    i32 = lambda v: torch.tensor(v, dtype=torch.int32, device="cuda")
    dt = torch.zeros((2, 3), dtype=torch.int32, device="cuda")
    with pytest.raises(b.HiSpecError):   # k + 1 rows exceed max_rows_per_seq
        ctx.verify_intermediate(st, torch.zeros((2, 9), dtype=torch.int32, device="cuda"), i32([1, 1]), i32([1, 1]), res)
    with pytest.raises(b.HiSpecError):   # layer_end is not an exit
        ctx.draft(st, i32([1, 2]), layer_end=3)
    with pytest.raises(b.HiSpecError):   # batch over capacity
        ctx.draft(st, i32([1, 2, 3]))
    n0 = ctx.launch_count()
    # rows that were never buffered: STATE bit, lengths untouched
    ctx.verify_intermediate(st, dt, i32([2, 2]), i32([3, 3]), res)
    assert ctx.status() & b.ST_STATE
    assert st.len_draft.tolist() == [0, 0] and ctx.launch_count() > n0
    # a block-table entry outside the pool: BOUNDS bit, no fault
    st.block_table[1, 0] = 1000
    ctx.draft(st, i32([5, 6]))
    assert ctx.status() & b.ST_BOUNDS
    torch.cuda.synchronize()
    assert ctx.status() == 0
    ctx.close()


@pytest.mark.parametrize("flagname", ["tcgen05", "multi-kernel"])
def test_sequence_with_zero_rows_sits_out_and_all_empty_call(flagname):
    """n_rows[b] == 0 skips sequence b: its length counters and its K/V pages stay as they were while its neighbours
    are verified as usual; a call in which every sequence has zero rows changes nothing at all."""
    b = _binding()
    shape = wl.MINI_GQA
    w, m, hs = oracle_for(shape, kv_round=True)
    B, N_d, max_rows, page, max_pages = 3, 4, 8, 16, 8
    ctx_lens, buffered = [37, 21, 64], [5, 3, 4]
    n_rows, n_draft = [5, 0, 4], [4, 0, 4]
    ctx = b.Context(shape, w.to("cuda"), page_size=page, max_batch=B, max_rows_per_seq=max_rows,
                    max_pages_per_seq=max_pages, flags=FLAG_SETS[flagname])
    states, drafts = [], []
    for s in range(B):
        prompt = wl.make_tokens(shape, ctx_lens[s], seed_offset=200 + s).tolist()
        ost = hs.new_state(ctx_lens[s] + 16, max_rows)
        pending = hs.prefill(ost, prompt).argmax_ids[0]
        ar = hs.ar_generate(prompt, 8)
        S = [ar[1 + j] if j < 2 else (ar[1 + j] + 7) % shape.vocab for j in range(4)]
        u = pending
        for t in (S + [None])[: buffered[s]]:
            hs.draft_step(ost, u)
            u = t
        drafts.append(S)
        states.append(ost)
    bt = wl.make_block_table(shape, B, max_pages, n_pages=B * max_pages + 7, seed_offset=3100)
    st = ctx.new_state(B, B * max_pages + 7, bt)
    for s in range(B):
        gh.load_seq(st, s, states[s], page, range(shape.n_layers), max_rows)
    res = ctx.new_result(B, logits=True, hidden=True)
    dt = torch.zeros((B, N_d), dtype=torch.int32)
    for s in range(B):
        dt[s, : len(drafts[s])] = torch.tensor(drafts[s], dtype=torch.int32)
    i32 = lambda v: torch.tensor(v, dtype=torch.int32, device="cuda")
    # every sequence empty: nothing moves
    before = (st.len_draft.clone(), st.len_inter.clone(), st.len_target.clone(), st.k_pages.clone(), st.v_pages.clone())
    ctx.verify_intermediate(st, dt.cuda(), i32([0, 0, 0]), i32([0, 0, 0]), res)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    for x, y in zip(before, (st.len_draft, st.len_inter, st.len_target, st.k_pages, st.v_pages)):
        assert torch.equal(x, y)
    # the middle sequence sits out
    pages1 = st.block_table[1].long()
    k1, v1 = st.k_pages[:, pages1].clone(), st.v_pages[:, pages1].clone()
    ctx.verify_intermediate(st, dt.cuda(), i32(n_draft), i32(n_rows), res)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    import copy
    for s in (0, 2):
        ost = copy.deepcopy(states[s])
        p0 = ost.len_i
        out = hs.verify_intermediate(ost, drafts[s][: n_draft[s]], n_rows[s])
        gh.compare_exit(out, res, s, n_rows[s], drafts[s][: n_draft[s]], check_accept=True, tag=f"seq{s}")
        gh.compare_kv(st, s, ost, page, range(hs.L_d, hs.L_i), range(p0, p0 + n_rows[s]), tag=f"seq{s}")
        assert int(st.len_inter[s]) == ost.len_i == int(st.len_draft[s])
    assert int(st.len_draft[1]) == states[1].len_d and int(st.len_inter[1]) == states[1].len_i
    assert torch.equal(st.k_pages[:, pages1], k1) and torch.equal(st.v_pages[:, pages1], v1)
    ctx.close()


def test_largest_batch_of_the_persistent_kernel_draft_step(monkeypatch):
    """64 sequences (the persistent kernel's table size) with ragged contexts, one draft step each through layers
    [0, L_d) + exit head as ONE launch: token (margin rule), buffered exit row, appended K/V and length counters of
    every sequence against the oracle.  (With this toy model's weights the KV cache outweighs a layer, which would
    route the call to the kernel sequence: the switch that keeps it on the persistent kernel is set.)"""
    monkeypatch.setenv("HISPEC_FORCE_MEGA", "1")
    b = _binding()
    shape = wl.TINY
    w, m, hs = oracle_for(shape, kv_round=True)
    B, max_rows, page, max_pages = 64, 2, 16, 4
    ctx = b.Context(shape, w.to("cuda"), page_size=page, max_batch=B, max_rows_per_seq=max_rows, max_pages_per_seq=max_pages)
    st = ctx.new_state(B, B * max_pages + 5, wl.make_block_table(shape, B, max_pages, n_pages=B * max_pages + 5, seed_offset=3200))
    states, pend = [], []
    for s in range(B):
        n = 3 + (7 * s) % 40
        prompt = wl.make_tokens(shape, n, seed_offset=300 + s).tolist()
        ost = hs.new_state(n + 8, max_rows)
        pend.append(hs.prefill(ost, prompt).argmax_ids[0])
        states.append(ost)
        gh.load_seq(st, s, ost, page, range(shape.n_layers), max_rows)
    n0 = ctx.launch_count()
    tin = torch.tensor(pend, dtype=torch.int32, device="cuda")
    tout = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    ctx.draft(st, tin, tout)
    torch.cuda.synchronize()
    assert ctx.status() == 0 and ctx.launch_count() - n0 == 1
    got = tout.cpu().tolist()
    for s in range(B):
        ost = states[s]
        p0 = ost.len_d
        out = hs.draft_step(ost, pend[s])
        if float(out.top2[0, 0] - out.top2[0, 1]) >= gh.MARGIN:
            assert got[s] == out.argmax_ids[0], f"seq{s}: token"
        row = st.h_draft[s, 0].cpu().numpy()
        ref = ost.h_d[p0 - ost.len_i].astype(np.float64)
        assert np.linalg.norm(row - ref) <= gh.HIDDEN_REL_L2 * np.linalg.norm(ref), f"seq{s}: buffered exit row"
        gh.compare_kv(st, s, ost, page, range(0, hs.L_d), [p0], tag=f"seq{s}")
        assert (int(st.len_draft[s]), int(st.len_inter[s]), int(st.len_target[s])) == (ost.len_d, ost.len_i, ost.len_f)
    ctx.close()
