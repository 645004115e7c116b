"""Pins for the composition of the stages: the lossless guarantee of Sec. 3.1
(every emitted token is the argmax of L_f at its position, so HiSpec's output is
identical to auto-regressive greedy decoding), the special cases named in the
task statement, and the bookkeeping of the decoding loop."""
import numpy as np
import pytest

from oracle.hispec import GenStats
from paper_2510_01336_b200 import workload as wl
from tests.helpers import SMALL, oracle_for


def test_cached_ar_equals_definition():
    """Greedy decoding with a KV cache == a full cache-free forward pass per token."""
    _, m, hs = oracle_for(SMALL)
    prompt = wl.make_tokens(SMALL, 7).tolist()
    assert hs.ar_generate(prompt, 10) == hs.ar_generate_nocache(prompt, 10)


@pytest.mark.parametrize("seed", range(6))
def test_hispec_equals_ar_for_random_parameters(seed):
    rng = np.random.default_rng(seed)
    shape = SMALL
    _, m, _ = oracle_for(shape, kv_round=bool(seed % 2))
    from oracle.hispec import HiSpecOracle
    L_f = shape.n_layers
    L_d = int(rng.integers(1, L_f - 1))
    L_i = int(rng.integers(L_d + 1, L_f))
    hs = HiSpecOracle(m, L_d, L_i, L_f)
    prompt = wl.make_tokens(shape, int(rng.integers(3, 12)), seed_offset=seed).tolist()
    n_gen = 18
    ar = hs.ar_generate(prompt, n_gen)
    N_d = int(rng.integers(1, 5))
    trig = dict(N_i=int(rng.integers(1, 7))) if seed % 2 else dict(rounds=int(rng.integers(1, 4)))
    for bi in (True, False):
        for bt in (False, True):
            # real greedy drafts
            assert hs.hispec_generate(prompt, n_gen, N_d, bonus_inter=bi, bonus_target=bt, **trig) == ar
            # adversarial drafts: random ids -- the output must not depend on draft content
            adv = lambda pos, g: int(rng.integers(0, shape.vocab))
            assert hs.hispec_generate(prompt, n_gen, N_d, bonus_inter=bi, bonus_target=bt,
                                      draft_override=adv, **trig) == ar
    assert hs.selfspec_generate(prompt, n_gen, N_d) == ar          # Algorithm 1


def test_single_row_verify_is_one_ar_step():
    """k = 1 without a bonus row: verifying one draft token through [L_d, L_f)
    yields exactly the next auto-regressive token."""
    shape = SMALL
    _, m, hs = oracle_for(shape)
    prompt = wl.make_tokens(shape, 8).tolist()
    ar = hs.ar_generate(prompt, 6)
    st = hs.new_state(32, 4)
    pending = hs.prefill(st, prompt).argmax_ids[0]
    assert pending == ar[0]
    for step in range(1, 6):
        hs.draft_step(st, pending)                           # pending through [0, L_d)
        o = hs.verify_intermediate(st, [12345 % shape.vocab], 1, hs.L_d, hs.L_f)   # one row, exit at L_f
        nxt = o.argmax_ids[0]
        assert nxt == ar[step]
        assert o.n_accepted in (0, 1) and st.len_d == st.len_i == st.len_f == len(prompt) + step
        pending = nxt


def test_targets_own_greedy_tokens_are_all_accepted():
    """Drafts := the target's own greedy continuation => both stages of a model
    whose exits coincide accept all of them and the bonus is the next greedy token."""
    shape = SMALL
    _, m, hs = oracle_for(shape)
    prompt = wl.make_tokens(shape, 8).tolist()
    ar = hs.ar_generate(prompt, 12)
    st = hs.new_state(40, 8)
    pending = hs.prefill(st, prompt).argmax_ids[0]
    S = ar[1:5]
    u = pending
    for t in S + [None]:
        hs.draft_step(st, u)
        u = t
    # exit at L_f for this call => the verifier *is* the target
    o = hs.verify_intermediate(st, S, 5, hs.L_d, hs.L_f)
    assert o.n_accepted == 4 and o.next_token == ar[5] and o.argmax_ids == ar[1:6]
    # and through the two real stages: V := target-greedy tokens, verified by L_f
    st = hs.new_state(40, 8)
    pending = hs.prefill(st, prompt).argmax_ids[0]
    u = pending
    for t in S:
        hs.draft_step(st, u)
        u = t
    hs.verify_intermediate(st, S, 4)                          # fills h_i rows whatever L_i thinks
    st.len_d = st.len_i = st.len_f + 4                        # keep all 4 rows (V := S by construction)
    o = hs.verify_target(st, S, 4)
    assert o.n_accepted == 4 and o.next_token == -1 and o.argmax_ids == ar[1:5]
    assert st.len_d == st.len_i == st.len_f == len(prompt) + 4


def test_scripted_round_lengths_and_rows():
    """The narrated scenario (two of three drafts tentatively accepted, third
    rejected): lengths of the three layer groups and buffer rows after each call."""
    shape = SMALL
    _, m, hs = oracle_for(shape)
    prompt = wl.make_tokens(shape, 9).tolist()
    st = hs.new_state(40, 10)
    pending = hs.prefill(st, prompt).argmax_ids[0]             # n = 10 committed, lengths 9
    assert (st.len_d, st.len_i, st.len_f) == (9, 9, 9)
    # learn what L_i will say, then script drafts S1,S2 right and S3 wrong
    probe = hs.new_state(40, 10)
    hs.prefill(probe, prompt)
    vi = []
    u = pending
    for _ in range(3):
        hs.draft_step(probe, u)
        o = hs.verify_intermediate(probe, [], 1)
        u = o.argmax_ids[0]
        vi.append(u)
    S = [vi[0], vi[1], (vi[2] + 1) % shape.vocab]
    u = pending
    for t in S + [None]:
        hs.draft_step(st, u)
        u = t
    assert (st.len_d, st.len_i, st.len_f) == (13, 9, 9)
    o = hs.verify_intermediate(st, S, 4)
    assert o.n_accepted == 2 and o.next_token == vi[2]
    assert (st.len_d, st.len_i, st.len_f) == (12, 12, 9)       # rows for positions 9..11 kept
    assert st.len_i - st.len_f == 3                            # |V| = 3 rows in h_i


@pytest.mark.parametrize("alpha", [0.6, 0.83])
def test_acceptance_bookkeeping_matches_closed_form(alpha):
    """Single-stage check of the loop's counters: drafts correct i.i.d. with
    probability alpha against the verifier give a mean accepted length of
    alpha (1 - alpha^k) / (1 - alpha) per block of k."""
    shape = SMALL
    _, m, hs = oracle_for(shape)
    prompt = wl.make_tokens(shape, 5).tolist()
    n_gen, k = 400, 4
    ar = hs.ar_generate(prompt, n_gen + 8)
    rng = np.random.default_rng(11)
    st = GenStats()
    x = [ar[0]]
    state = hs.new_state(len(prompt) + n_gen + 16, k + 1)
    pending = hs.prefill(state, prompt).argmax_ids[0]
    blocks = acc = 0
    while len(x) < n_gen:
        S = []
        for j in range(k):
            pos = len(x) + j
            S.append(ar[pos] if rng.random() < alpha else (ar[pos] + 1) % shape.vocab)
        u = pending
        for t in S + [None]:
            hs.draft_step(state, u)
            u = t
        o = hs.verify_intermediate(state, S, k + 1, hs.L_d, hs.L_f)
        from oracle.hispec import leading_substring_verify
        F, a = leading_substring_verify(S, o.argmax_ids)
        assert F == ar[len(x): len(x) + len(F)]
        x += F
        pending = F[-1]
        blocks += 1
        acc += a
    mean = acc / blocks
    expect = alpha * (1 - alpha ** k) / (1 - alpha)
    se = 1.5 / np.sqrt(blocks)
    assert abs(mean - expect) < 4 * se, (mean, expect, blocks)


def test_chain_of_verifiers_is_lossless():
    """Several intermediate verifiers (App. K): whatever the chain, the output is greedy decoding from L_f; with
    one verifier level the chain is Algorithm 1, with two it is Algorithm 2 with a fixed number of rounds."""
    from paper_2510_01336_b200 import workload as wl
    from tests.helpers import oracle_for
    import dataclasses
    shape = dataclasses.replace(wl.MINI_GQA, L_d=1, L_i=3, L_f=6)
    scale = {l: 0.05 for l in range(1, 6)}
    _, _, hs = oracle_for(shape, resid_scale=scale)
    prompt = wl.make_tokens(shape, 12).tolist()
    n_gen = 20
    ar = hs.ar_generate(prompt, n_gen)
    sched = []
    assert hs.chain_generate(prompt, n_gen, [1, 2, 4, 6], 2, [2, 2], schedule=sched) == ar
    assert {lv for lv, _, _ in sched} == {1, 2, 3}
    assert sum(a for lv, _, a in sched if lv == 1) > 0 and sum(a for lv, _, a in sched if lv == 3) > 0
    assert hs.chain_generate(prompt, n_gen, [1, 3, 6], 2, [2]) == hs.hispec_generate(prompt, n_gen, 2, rounds=2)
    assert hs.chain_generate(prompt, n_gen, [1, 3, 6], 2, [2]) == ar
    assert hs.chain_generate(prompt, n_gen, [2, 6], 3, []) == ar
