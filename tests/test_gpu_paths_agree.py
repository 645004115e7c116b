"""The two GPU paths against each other on random call shapes.

The persistent kernel and the kernel sequence compute the same call with different partitions, tile shapes and
attention pipelines; the oracle-based tests pin each of them on chosen cases, this one sweeps seeded random batch
sizes, row counts (zero included) and context lengths (zero and page-boundary values included) and requires the two
to agree within the tolerances of the oracle comparison."""
import numpy as np
import pytest
import torch

from paper_2510_01336_b200 import workload as wl
from tests import gpu_harness as gh

pytestmark = pytest.mark.gpu


def _run(shape, flags, B, ctx_lens, n_rows, k_all, v_all, h_all, drafts, max_rows, max_pages, page, bt):
    from paper_2510_01336_b200 import binding
    layers = list(range(shape.L_i, shape.L_f))
    w = wl.make_weights(shape, device="cuda")
    ctx = binding.Context(shape, w, page_size=page, max_batch=B, max_rows_per_seq=max_rows, max_pages_per_seq=max_pages,
                          flags=flags)
    st = ctx.new_state(B, bt.numel() + 3, bt)
    for b in range(B):
        c = ctx_lens[b]
        for l in layers:
            if c:
                gh.load_dense_kv(st, b, l, k_all[l - shape.L_i, b, :c], v_all[l - shape.L_i, b, :c], page)
        st.h_inter[b] = h_all[b].cuda()
        st.len_target[b] = c
        st.len_inter[b] = c + n_rows[b]
        st.len_draft[b] = c + n_rows[b]
    res = ctx.new_result(B, logits=True, hidden=True)
    i32 = lambda v: torch.tensor(v, dtype=torch.int32, device="cuda")
    n0 = ctx.launch_count()
    ctx.verify_target(st, drafts.cuda().contiguous(), i32(n_rows), i32(n_rows), res, k=max_rows - 1)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    out = {"launches": ctx.launch_count() - n0, "hidden": res.hidden_out.cpu().numpy(), "logits": res.logits.cpu().numpy(),
           "ids": res.argmax_ids.cpu().numpy(), "top2": res.top2.cpu().numpy(), "acc": res.n_accepted.cpu().numpy(),
           "next": res.next_token.cpu().numpy(), "k": st.k_pages.float().cpu().numpy(), "v": st.v_pages.float().cpu().numpy(),
           "lens": (st.len_draft.cpu().numpy(), st.len_inter.cpu().numpy(), st.len_target.cpu().numpy())}
    ctx.close()
    return out


@pytest.mark.parametrize("seed", range(16))
def test_persistent_kernel_and_kernel_sequence_agree(seed, monkeypatch):
    from paper_2510_01336_b200 import binding
    monkeypatch.setenv("HISPEC_FORCE_MEGA", "1")   # toy weights: keep KV-heavy calls on the persistent kernel
    rng = np.random.default_rng(1000 + seed)
    shape = (wl.MINI_GQA, wl.TINY)[seed % 2]
    page, max_rows, max_pages = 16, 8, 8
    B = int(rng.integers(1, 9))   # up to 8 x 8 = 64 rows: the persistent kernel's range
    special = [0, 1, 15, 16, 17, 31, 32, 33, 100, 119]
    ctx_lens = [int(rng.choice(special)) if rng.random() < 0.5 else int(rng.integers(0, 120)) for _ in range(B)]
    n_rows = [int(rng.integers(0, max_rows)) for _ in range(B)]
    if sum(n_rows) == 0:
        n_rows[0] = 3
    layers = list(range(shape.L_i, shape.L_f))
    k_all, v_all, h_all = wl.make_random_state(shape, layers, [max(c, 1) for c in ctx_lens], max_rows, seed_offset=5000 + seed,
                                               hidden_std=3.0)
    drafts = wl.make_tokens(shape, B * (max_rows - 1), seed_offset=6000 + seed).reshape(B, max_rows - 1)
    bt = wl.make_block_table(shape, B, max_pages, n_pages=B * max_pages + 3, seed_offset=7000 + seed)
    args = (B, ctx_lens, n_rows, k_all, v_all, h_all, drafts, max_rows, max_pages, page, bt)
    a = _run(shape, 0, *args)
    s = _run(shape, binding.FLAG_MULTI_KERNEL, *args)
    assert a["launches"] == 1 and s["launches"] > 1, "the two runs must take different paths"
    for x, y in zip(a["lens"], s["lens"]):
        assert np.array_equal(x, y)
    for b in range(B):
        r = n_rows[b]
        if r == 0:
            continue
        ha, hs = a["hidden"][b, :r].astype(np.float64), s["hidden"][b, :r].astype(np.float64)
        rel = np.linalg.norm(ha - hs, axis=1) / np.linalg.norm(hs, axis=1)
        assert rel.max() <= gh.HIDDEN_REL_L2, f"seq{b}: hidden rows differ (rel-L2 {rel.max():.2e})"
        assert np.abs(a["logits"][b, :r] - s["logits"][b, :r]).max() <= gh.LOGITS_MAX_ABS
        same = True
        for j in range(r):
            margin = float(s["top2"][b, j, 0] - s["top2"][b, j, 1])
            if margin >= gh.MARGIN:
                assert a["ids"][b, j] == s["ids"][b, j], f"seq{b} row {j}: ids differ at margin {margin:.3f}"
            same = same and a["ids"][b, j] == s["ids"][b, j]
        if same:
            assert a["acc"][b] == s["acc"][b] and a["next"][b] == s["next"][b]
    # appended K/V (and everything else in the pools): equal up to one bf16 rounding step of nearly equal fp32 values
    for name in ("k", "v"):
        d = np.abs(a[name] - s[name])
        tol = np.abs(s[name]) * 2.0 ** -7 + 2e-2
        assert np.all(d <= tol), f"{name} pages differ"
