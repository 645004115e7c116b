"""GPU parity at the workloads' full layer shapes, in the launch configuration bench.py times.

A CPU prefill at these shapes would take hours, so the cached state of a stand-alone call is drawn
from a seed (K, V ~ N(0,1) as bf16, hidden rows ~ N(0, 3^2)) and handed, byte for byte, to both the
oracle and the GPU call; the oracle then computes that one call (a few to a few tens of GFLOP)."""
import numpy as np
import pytest
import torch

from oracle.hispec import HiSpecOracle, OracleModel
from paper_2510_01336_b200 import workload as wl
from tests import gpu_harness as gh

pytestmark = pytest.mark.gpu


def _run_case(shape, l0, l1, kind, ctx_lens, n_rows, n_draft, max_rows, flags=0, seed_offset=4000):
    from paper_2510_01336_b200 import binding
    B = len(ctx_lens)
    layers = list(range(l0, l1))
    w_gpu = wl.make_weights(shape, layers=layers, device="cuda", with_emb=False)
    w_cpu = w_gpu.to("cpu")
    m = OracleModel.from_weights(w_cpu, kv_round_bf16=True)
    hs = HiSpecOracle(m, shape.L_d, shape.L_i, shape.L_f)
    k_all, v_all, h_all = wl.make_random_state(shape, layers, ctx_lens, max_rows, seed_offset=seed_offset,
                                               hidden_std=3.0)
    page = 16
    max_pages = (max(ctx_lens) + max_rows + page - 1) // page + 1
    ctx = binding.Context(shape, w_gpu, page_size=page, max_batch=B, max_rows_per_seq=max_rows,
                          max_pages_per_seq=max_pages, flags=flags)
    bt = wl.make_block_table(shape, B, max_pages, n_pages=B * max_pages + 3)
    st = ctx.new_state(B, B * max_pages + 3, bt, first_layer=l0, n_pool_layers=len(layers))
    K = max(max(n_draft), 1)
    drafts = wl.make_tokens(shape, B * K, seed_offset=seed_offset + 1).reshape(B, K)
    osts = []
    for b in range(B):
        c = ctx_lens[b]
        ost = hs.new_state(c + max_rows + 1, max_rows)
        for i, l in enumerate(layers):
            ost.cache.k[l, :c] = k_all[i, b, :c].float().numpy()
            ost.cache.v[l, :c] = v_all[i, b, :c].float().numpy()
            gh.load_dense_kv(st, b, i, k_all[i, b, :c], v_all[i, b, :c], page)
        rows = h_all[b].numpy()
        if kind == "verify_i":
            ost.h_d[:] = rows
            ost.len_d, ost.len_i, ost.len_f = c + n_rows[b], c, c
            st.h_draft[b] = h_all[b].cuda()
        else:
            ost.h_i[:] = rows
            ost.len_d, ost.len_i, ost.len_f = c + n_rows[b], c + n_rows[b], c
            st.h_inter[b] = h_all[b].cuda()
        st.len_draft[b], st.len_inter[b], st.len_target[b] = ost.len_d, ost.len_i, ost.len_f
        osts.append(ost)
    res = ctx.new_result(B, logits=True, hidden=True)
    i32 = lambda v: torch.tensor(v, dtype=torch.int32, device="cuda")
    fn = ctx.verify_intermediate if kind == "verify_i" else ctx.verify_target
    fn(st, drafts.cuda().contiguous(), i32(n_draft), i32(n_rows), res)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    worst = {"rel_l2": 0.0, "logit_err": 0.0, "exempt": 0}
    for b in range(B):
        S = drafts[b, : n_draft[b]].tolist()
        p0 = ctx_lens[b]
        out = (hs.verify_intermediate if kind == "verify_i" else hs.verify_target)(osts[b], S, n_rows[b])
        s = gh.compare_exit(out, res, b, n_rows[b], S, check_accept=True, tag=f"{shape.name} {kind} seq{b}")
        # plain bf16 activations (a debug mode) perturb the deepest layer's K/V by more than the default slack
        gh.compare_kv(st, b, osts[b], page, [layers[0], layers[-1]], range(p0, p0 + n_rows[b]), tag=f"seq{b}",
                      slack=4.0 if flags & binding.FLAG_PLAIN_ACT else 1.0)
        for k in ("rel_l2", "logit_err"):
            worst[k] = max(worst[k], s[k])
        worst["exempt"] += s["exempt"]
        lens = (int(st.len_draft[b]), int(st.len_inter[b]), int(st.len_target[b]))
        assert lens == (osts[b].len_d, osts[b].len_i, osts[b].len_f) or s["exempt"] > 0
    print(f"\n[{shape.name} {kind} [{l0},{l1}) B={B}] rel-L2 {worst['rel_l2']:.2e} logits {worst['logit_err']:.2e} "
          f"exempt {worst['exempt']}")
    ctx.close()
    return worst


def test_llama3_8b_shape_verify_intermediate_batch1():
    """The benchmarked call: layers [8,16), batch 1, context 1024, k = 5 (6 rows)."""
    _run_case(wl.L3_8B, 8, 16, "verify_i", [1024], [6], [5], 13)


def test_llama3_8b_shape_verify_target_batch1():
    """Layers [16,32) on 12 accumulated rows, context 1024."""
    _run_case(wl.L3_8B, 16, 32, "verify_t", [1024], [12], [12], 13)


def test_llama3_8b_shape_serving_batch_ragged():
    """Serving-batch shape: ragged contexts (incl. one that is not a multiple of the page size and one of 4096),
    k = 8 (9 rows), ragged row counts, GQA 4:1."""
    _run_case(wl.L3_8B, 8, 16, "verify_i", [517, 1500, 4096], [9, 5, 8], [8, 4, 8], 9, seed_offset=4100)


def test_llama3_8b_shape_long_contexts_two_layers():
    """KV-heavy call (the cache a layer reads is a third of its weights): contexts up to 8192 next to one of a single
    page, so that the attention phase runs with its deepest page pipeline, several (sequence, KV head, key split)
    items per CTA and key splits that are empty for the short sequences."""
    import dataclasses
    shape = dataclasses.replace(wl.L3_8B, L_d=8, L_i=10, L_f=32)
    _run_case(shape, 8, 10, "verify_i", [8192, 3001, 16, 5000], [7, 7, 3, 6], [6, 6, 2, 6], 7, seed_offset=4500)


@pytest.mark.parametrize("multi_kernel", [False, True])
def test_llama3_8b_shape_target_rows_beyond_one_attention_tile_group(multi_kernel):
    """Target verification with 18 rows per sequence (padded to 19) at GQA 4:1: 76 stacked query rows per KV head, i.e. more than
    the 64 one attention item of the persistent kernel takes (two row groups there) and five 16-row warp tiles in
    one CTA of the stand-alone attention kernel."""
    import dataclasses
    from paper_2510_01336_b200 import binding
    shape = dataclasses.replace(wl.L3_8B, L_d=8, L_i=16, L_f=18)
    _run_case(shape, 16, 18, "verify_t", [700, 1300], [18, 11], [18, 11], 19, seed_offset=4700,
              flags=binding.FLAG_MULTI_KERNEL if multi_kernel else 0)


def test_llama2_13b_shape_two_layers():
    """Llama-2-13B layer shape (MHA, d 5120, ffn 13824, vocab 32000): two layers of the intermediate range,
    batch 2, context 2048, k = 6."""
    import dataclasses
    shape = dataclasses.replace(wl.L2_13B, L_d=10, L_i=12, L_f=40)
    _run_case(shape, 10, 12, "verify_i", [2048, 777], [7, 7], [6, 6], 7, seed_offset=4200)


def test_codellama_34b_shape_two_layers():
    """CodeLlama-34B layer shape (GQA 8:1, d 8192, ffn 22016): two layers of the intermediate range [7, 12),
    batch 1, context 1024, k = 5 with the bonus row."""
    import dataclasses
    shape = dataclasses.replace(wl.CL_34B, L_d=7, L_i=9, L_f=48)
    _run_case(shape, 7, 9, "verify_i", [1024], [6], [5], 7, seed_offset=4300)


def test_llama2_70b_shape_two_layers():
    """Llama-2-70B layer shape (GQA 8:1, d 8192, ffn 28672): two layers of the target range, batch 2, ragged."""
    import dataclasses
    shape = dataclasses.replace(wl.L2_70B, L_d=10, L_i=20, L_f=22)
    _run_case(shape, 20, 22, "verify_t", [600, 1023], [9, 4], [9, 4], 10, seed_offset=4400)


def test_llama3_8b_shape_plain_bf16_activations():
    """The same benchmarked call with plain bf16 tensor-core inputs (no hi/lo split): still inside the tolerances."""
    from paper_2510_01336_b200 import binding
    _run_case(wl.L3_8B, 8, 16, "verify_i", [1024], [6], [5], 13, flags=binding.FLAG_PLAIN_ACT)


def test_llama3_8b_shape_draft_steps_batch1():
    """The benchmarked draft calls, batch 1, context 1024, layers [0,8) + exit head L_d.
    (1) Six draft steps + the bonus row as ONE launch (hispec_draft_block): the oracle runs the steps free, one after
    the other; every step is compared (token, buffered exit row, appended K/V) until the first step whose greedy
    token differs, which must be one the oracle's own top-2 margin leaves open (< 0.1).
    (2) The same steps as single hispec_draft calls from the same start, each fed the ORACLE's token, so that all of
    them are compared whatever the margins are."""
    from paper_2510_01336_b200 import binding
    shape, n_steps, c, page, max_rows = wl.L3_8B, 6, 1024, 16, 13
    layers = list(range(0, shape.L_d))
    w_gpu = wl.make_weights(shape, layers=layers, device="cuda", with_emb=True)
    m = OracleModel.from_weights(w_gpu.to("cpu"), kv_round_bf16=True)
    hs = HiSpecOracle(m, shape.L_d, shape.L_i, shape.L_f)
    k_all, v_all, _ = wl.make_random_state(shape, layers, [c], max_rows, seed_offset=4600)
    max_pages = (c + max_rows + page - 1) // page + 1
    ctx = binding.Context(shape, w_gpu, page_size=page, max_batch=1, max_rows_per_seq=max_rows, max_pages_per_seq=max_pages)
    t0 = int(wl.make_tokens(shape, 1, seed_offset=4601)[0])

    def fresh():
        st = ctx.new_state(1, max_pages + 3, wl.make_block_table(shape, 1, max_pages, n_pages=max_pages + 3),
                           first_layer=0, n_pool_layers=len(layers))
        for i, l in enumerate(layers):
            gh.load_dense_kv(st, 0, i, k_all[i, 0, :c], v_all[i, 0, :c], page)
        st.len_draft.fill_(c); st.len_inter.fill_(c); st.len_target.fill_(c)
        return st

    # the oracle's free run
    ost = hs.new_state(c + max_rows + 1, max_rows)
    for i, l in enumerate(layers):
        ost.cache.k[l, :c] = k_all[i, 0, :c].float().numpy()
        ost.cache.v[l, :c] = v_all[i, 0, :c].float().numpy()
    ost.len_d = ost.len_i = ost.len_f = c
    inputs, ref_tok, ref_margin = [t0], [], []
    for j in range(n_steps + 1):
        out = hs.draft_step(ost, inputs[j])
        ref_tok.append(out.argmax_ids[0])
        ref_margin.append(float(out.top2[0][0] - out.top2[0][1]))
        inputs.append(out.argmax_ids[0])

    def check_step(st, j, tag):
        ref_row = ost.h_d[j].astype(np.float64)
        rel = float(np.linalg.norm(st.h_draft[0, j].cpu().numpy() - ref_row) / np.linalg.norm(ref_row))
        assert rel <= 1e-2, f"{tag} step {j}: buffered exit row rel-L2 {rel:.2e}"
        gh.compare_kv(st, 0, ost, page, [layers[0], layers[-1]], [c + j], tag=f"{tag} step {j}")
        return rel

    # (1) one launch, free running
    st = fresh()
    S = torch.full((1, n_steps), -1, dtype=torch.int32, device="cuda")
    ctx.draft_block(st, torch.tensor([t0], dtype=torch.int32, device="cuda"), S, n_steps, bonus=True)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    assert int(st.len_draft[0]) == c + n_steps + 1 and int(st.len_inter[0]) == c
    got, compared, worst = S[0].tolist(), 0, 0.0
    for j in range(n_steps + 1):          # the last step (bonus row) leaves no token
        worst = max(worst, check_step(st, j, "block"))
        compared += 1
        if j < n_steps and got[j] != ref_tok[j]:
            assert ref_margin[j] < 0.1, f"block step {j}: token {got[j]} != {ref_tok[j]} with margin {ref_margin[j]:.3f}"
            break
    assert compared >= 1
    # (2) single calls, inputs from the oracle
    st = fresh()
    exempt = 0
    for j in range(n_steps + 1):
        tin = torch.tensor([inputs[j]], dtype=torch.int32, device="cuda")
        tout = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        ctx.draft(st, tin, tout)
        torch.cuda.synchronize()
        worst = max(worst, check_step(st, j, "single"))
        if int(tout[0]) != ref_tok[j]:
            assert ref_margin[j] < 0.1, f"single step {j}: token {int(tout[0])} != {ref_tok[j]} with margin {ref_margin[j]:.3f}"
            exempt += 1
    assert ctx.status() == 0 and int(st.len_draft[0]) == c + n_steps + 1
    print(f"\n[{shape.name} draft [0,{shape.L_d}) x {n_steps}+1] block steps compared {compared}, single steps "
          f"{n_steps + 1} (exempt tokens {exempt}), worst row rel-L2 {worst:.2e}")
    ctx.close()


@pytest.mark.parametrize("seed", range(12))
def test_random_small_calls_against_the_oracle(seed, monkeypatch):
    """Seeded random calls on the two toy shapes (head_dim 64 MHA and head_dim 128 GQA): random batch size, ragged row
    counts, contexts that include zero, one and page-boundary lengths, either verification call, either GPU path --
    each compared with the oracle exactly as the full-size cases are."""
    import dataclasses
    from paper_2510_01336_b200 import binding
    monkeypatch.setenv("HISPEC_FORCE_MEGA", "1")   # toy weights: keep KV-heavy calls on the persistent kernel
    rng = np.random.default_rng(2000 + seed)
    shape = (wl.TINY, wl.MINI_GQA)[seed % 2]
    kind = ("verify_i", "verify_t")[(seed // 2) % 2]
    flags = (0, binding.FLAG_MULTI_KERNEL)[(seed // 4) % 2]
    max_rows = 8
    B = int(rng.integers(1, 7))
    special = [0, 1, 15, 16, 17, 32, 47, 48, 49, 100]
    ctx_lens = [int(rng.choice(special)) if rng.random() < 0.6 else int(rng.integers(0, 110)) for _ in range(B)]
    if max(ctx_lens) == 0:
        ctx_lens[0] = 33
    if kind == "verify_i":
        n_draft = [int(rng.integers(0, max_rows)) for _ in range(B)]
        n_rows = [d + int(rng.integers(0, 2)) if d else 1 for d in n_draft]      # with or without the bonus row
        n_rows = [min(r, max_rows) for r in n_rows]
        n_draft = [min(d, r) for d, r in zip(n_draft, n_rows)]
        l0, l1 = shape.L_d, shape.L_i
    else:
        n_rows = [int(rng.integers(1, max_rows)) for _ in range(B)]
        n_draft = list(n_rows)
        l0, l1 = shape.L_i, shape.L_f
    _run_case(shape, l0, l1, kind, ctx_lens, n_rows, n_draft, max_rows, flags=flags, seed_offset=8000 + 10 * seed)
