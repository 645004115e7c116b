"""Pins for KV-cache and hidden-state reuse (Sec. 3.2): every stage call of the
cached path must equal, bit for bit, a brute-force recomputation of the whole
prefix with no cache and no buffered rows; the invariants of the shared state
hold after every call."""
import numpy as np
import pytest
import torch

from oracle.hispec import GenStats
from paper_2510_01336_b200 import workload as wl
from tests.helpers import SMALL, oracle_for


class BruteForceObserver:
    def __init__(self, hs):
        self.hs, self.calls, self.pending = hs, 0, None

    def before(self, kind, st, seq_tokens, **kw):
        hs = self.hs
        assert st.len_f <= st.len_i <= st.len_d
        if kind == "draft":
            pos, L = [st.len_d], hs.L_d
            assert seq_tokens[st.len_d] == kw["token"]
        elif kind == "verify_i":
            pos, L = list(range(st.len_i, st.len_i + kw["n_rows"])), hs.L_i
            assert st.len_d - st.len_i >= kw["n_rows"]
        else:
            pos, L = list(range(st.len_f, st.len_f + kw["n_rows"])), hs.L_f
            assert st.len_i - st.len_f >= kw["n_rows"]          # rows of V are all buffered
            assert kw["n_rows"] in (len(kw["S"]), len(kw["S"]) + 1)
        self.expect = hs.brute_force_exit(seq_tokens, L, pos)
        self.kind = kind

    def after(self, kind, st, out):
        assert np.array_equal(out.hidden, self.expect.hidden)
        assert np.array_equal(out.logits, self.expect.logits)
        assert out.argmax_ids == self.expect.argmax_ids
        if kind == "verify_t":
            assert st.len_d == st.len_i == st.len_f
        if kind == "verify_i":
            assert st.len_d == st.len_i
        self.calls += 1


@pytest.mark.parametrize("shape", [SMALL, wl.MINI_GQA])
@pytest.mark.parametrize("kv_round", [False, True])
@pytest.mark.parametrize("mode", [dict(N_i=4, bonus_inter=True, bonus_target=False),
                                  dict(rounds=2, bonus_inter=False, bonus_target=True),
                                  dict(N_i=3, bonus_inter=True, bonus_target=True)])
def test_cached_calls_equal_bruteforce(shape, kv_round, mode):
    _, m, hs = oracle_for(shape, kv_round=kv_round)
    prompt = wl.make_tokens(shape, 9).tolist()
    ar = hs.ar_generate(prompt, 40)
    # drafts that agree with the target most of the time, so that accept paths, partial
    # accepts and rejects all occur
    rng = np.random.default_rng(3)
    def override(pos, greedy):
        k = pos - len(prompt)
        return ar[k] if (k < len(ar) and rng.random() < 0.75) else greedy
    obs = BruteForceObserver(hs)
    st = GenStats()
    out = hs.hispec_generate(prompt, 14, 3, draft_override=override, observer=obs, stats=st, **mode)
    assert out == ar[:14]
    assert obs.calls > 10 and st.inter_accepted > 0 and st.flushed + st.target_accepted == st.target_checked


def test_tiny_config_cached_equals_bruteforce_on_real_drafts():
    """cfg "tiny": drafts come greedily from the draft exit (random weights: mostly rejected)."""
    shape = wl.TINY
    _, m, hs = oracle_for(shape, kv_round=True)
    prompt = wl.make_tokens(shape, 16).tolist()
    obs = BruteForceObserver(hs)
    out = hs.hispec_generate(prompt, 6, 4, rounds=2, observer=obs)
    assert out == hs.ar_generate(prompt, 6)
