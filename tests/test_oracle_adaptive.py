"""Adaptive N_d / N_i (App. J): the update rule against the cases its two equations fix, the loop's
losslessness under the policy, and the product's host rule against the oracle's."""
import itertools

import numpy as np
import pytest

from oracle import hispec as oh
from paper_2510_01336_b200 import workload as wl
from tests.helpers import oracle_for


def test_rule_cases_fixed_by_the_equations():
    nd, ni = oh.ADAPT_ND_PAPER, oh.ADAPT_NI_PAPER
    # thresholds and bounds printed in App. J
    assert (nd.tau_high, nd.tau_low, nd.n_min, nd.n_max) == (0.8, 0.5, 1, 3)
    assert (ni.tau_high, ni.tau_low, ni.n_min, ni.n_max) == (0.8, 0.3, 3, 8)
    # alpha >= tau_high: one more, capped at the maximum (">=" includes the threshold itself)
    assert oh.adaptive_step(2, 0.8, nd) == 3 and oh.adaptive_step(2, 1.0, nd) == 3
    assert oh.adaptive_step(3, 1.0, nd) == 3
    # alpha < tau_low: one less, floored at the minimum ("<" excludes the threshold itself)
    assert oh.adaptive_step(2, 0.49, nd) == 1 and oh.adaptive_step(1, 0.0, nd) == 1
    assert oh.adaptive_step(2, 0.5, nd) == 2
    # in between: unchanged
    assert oh.adaptive_step(2, 0.65, nd) == 2 and oh.adaptive_step(4, 0.3, ni) == 4
    assert oh.adaptive_step(4, 0.29, ni) == 3 and oh.adaptive_step(3, 0.0, ni) == 3
    assert oh.adaptive_step(7, 0.9, ni) == 8 and oh.adaptive_step(8, 0.9, ni) == 8


def test_rule_invariants_by_enumeration():
    for spec in (oh.ADAPT_ND_PAPER, oh.ADAPT_NI_PAPER, oh.AdaptiveSpec(0.7, 0.2, 2, 5)):
        for n in range(spec.n_min, spec.n_max + 1):
            prev = None
            for alpha in np.linspace(0.0, 1.0, 101):
                m = oh.adaptive_step(n, float(alpha), spec)
                assert spec.n_min <= m <= spec.n_max and abs(m - n) <= 1
                if prev is not None:
                    assert m >= prev          # monotone in the acceptance rate
                prev = m


def test_adaptive_generation_is_lossless_and_moves_the_parameters():
    """Whatever schedule the policy produces, the output is the target's greedy output (Sec. 3.3)."""
    shape = wl.TINY
    scale = {l: 0.05 for l in range(shape.L_d, shape.L_f)}
    _, _, hs = oracle_for(shape, resid_scale=scale)
    prompt = wl.make_tokens(shape, 24).tolist()
    n_gen = 40
    ar = hs.ar_generate(prompt, n_gen)
    sched = []
    out = hs.hispec_generate(prompt, n_gen, 2, N_i=4, adapt_nd=oh.ADAPT_ND_PAPER, adapt_ni=oh.ADAPT_NI_PAPER,
                             schedule=sched)
    assert out == ar
    nds = {rec[1] for rec in sched if rec[0] == "i"}
    nis = {rec[1] for rec in sched if rec[0] == "t"}
    assert len(nds) > 1 and len(nis) > 1, "with mostly-agreeing exits both parameters must have moved"
    assert nds <= {1, 2, 3} and nis <= set(range(3, 9))
    # the recorded schedule obeys the rule step by step
    n_d, n_i = 2, 4
    for rec in sched:
        if rec[0] == "i":
            assert rec[1] == n_d
            n_d = oh.adaptive_step(n_d, rec[2] / rec[1], oh.ADAPT_ND_PAPER)
        else:
            assert rec[1] == n_i and rec[2] >= 1
            n_i = oh.adaptive_step(n_i, rec[3] / rec[2], oh.ADAPT_NI_PAPER)
    # adversarial drafts: still lossless, and the parameters sink to their minima
    sched2 = []
    bad = hs.hispec_generate(prompt, 16, 2, N_i=4, adapt_nd=oh.ADAPT_ND_PAPER, adapt_ni=oh.ADAPT_NI_PAPER,
                             draft_override=lambda pos, tok: (tok + 1) % shape.vocab, schedule=sched2)
    assert bad == ar[:16]
    assert [rec[1] for rec in sched2 if rec[0] == "i"][-1] == 1


def test_product_rule_matches_oracle_rule():
    from paper_2510_01336_b200.driver import ND_RULE_PAPER, NI_RULE_PAPER, AdaptiveRule
    pairs = [(ND_RULE_PAPER, oh.ADAPT_ND_PAPER), (NI_RULE_PAPER, oh.ADAPT_NI_PAPER),
             (AdaptiveRule(0.6, 0.4, 2, 6), oh.AdaptiveSpec(0.6, 0.4, 2, 6))]
    for rule, spec in pairs:
        for n, k in itertools.product(range(spec.n_min, spec.n_max + 1), range(0, 13)):
            for d in (1, 2, 3, 4, 6, 12):
                if k <= d:
                    assert rule.next(n, k / d) == oh.adaptive_step(n, k / d, spec)
