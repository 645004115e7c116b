"""Teacher-forced comparison of one C-ABI call with the oracle's stage call.

Before a call the oracle's state (KV cache as pages through a block table, length
counters, buffered hidden rows) is loaded onto the GPU; after it, everything the
call is specified to produce is compared: exit hidden rows, logits, greedy ids
(bit-exact unless the oracle's top-2 margin is below 0.1), accepted length,
correction token, the three length counters, the K/V entries appended and the
rows written to the hidden buffers.
"""
from __future__ import annotations

import numpy as np
import torch

from paper_2510_01336_b200 import binding

HIDDEN_REL_L2 = 1e-2   # per exit row, relative L2
LOGITS_MAX_ABS = 5e-2  # per logit
MARGIN = 0.1           # ids bit-exact unless the oracle's top-2 margin is below this


def pages_from_cache(cache_np: np.ndarray, block_table_row: torch.Tensor, page_size: int, pages: torch.Tensor,
                     layers, first_layer: int, upto: int):
    """Scatter an oracle cache [n_layers][cap][hkv][hd] (positions < upto) into the page pool."""
    for l in layers:
        src = torch.from_numpy(cache_np[l, :upto]).to(torch.bfloat16)  # exact: values are bf16-representable
        for lp in range((upto + page_size - 1) // page_size):
            n = min(page_size, upto - lp * page_size)
            blk = src[lp * page_size: lp * page_size + n].permute(1, 0, 2)  # [hkv][n][hd]
            pages[l - first_layer, int(block_table_row[lp]), :, :n] = blk.to(pages.device)


def cache_from_pages(pages: torch.Tensor, block_table_row: torch.Tensor, page_size: int, layer: int,
                     first_layer: int, positions) -> np.ndarray:
    out = []
    for p in positions:
        pg = int(block_table_row[p // page_size])
        out.append(pages[layer - first_layer, pg, :, p % page_size].float().cpu().numpy())
    return np.stack(out) if out else np.zeros((0,))


def load_seq(st: binding.KVState, b: int, ost, page_size: int, layers, max_rows: int):
    """Copy one oracle SeqState into slot b of the GPU state."""
    bt = st.block_table[b].cpu()
    upto = max(ost.len_d, ost.len_i, ost.len_f)
    pages_from_cache(ost.cache.k, bt, page_size, st.k_pages, layers, st.first_layer, upto)
    pages_from_cache(ost.cache.v, bt, page_size, st.v_pages, layers, st.first_layer, upto)
    st.len_draft[b], st.len_inter[b], st.len_target[b] = ost.len_d, ost.len_i, ost.len_f
    n = min(max_rows, ost.h_d.shape[0])
    st.h_draft[b, :n] = torch.from_numpy(ost.h_d[:n]).to(st.h_draft.device)
    st.h_inter[b, :n] = torch.from_numpy(ost.h_i[:n]).to(st.h_inter.device)


def compare_exit(out, res: binding.Result, b: int, n_rows: int, S, *, check_accept: bool, tag: str = ""):
    """Compare the oracle's ExitOut with row block b of a GPU Result. Returns stats."""
    stats = {"rel_l2": 0.0, "logit_err": 0.0, "exempt": 0, "rows": n_rows}
    ids = res.argmax_ids[b, :n_rows].cpu().tolist()
    if res.hidden_out is not None:
        h = res.hidden_out[b, :n_rows].cpu().numpy().astype(np.float64)
        ref = out.hidden.astype(np.float64)
        rel = np.linalg.norm(h - ref, axis=1) / np.linalg.norm(ref, axis=1)
        stats["rel_l2"] = float(rel.max()) if n_rows else 0.0
        assert stats["rel_l2"] <= HIDDEN_REL_L2, f"{tag} hidden rel-L2 {rel}"
    if res.logits is not None:
        z = res.logits[b, :n_rows].cpu().numpy()
        err = np.abs(z.astype(np.float64) - out.logits.astype(np.float64)).max() if n_rows else 0.0
        stats["logit_err"] = float(err)
        assert err <= LOGITS_MAX_ABS, f"{tag} logits max-abs {err}"
    exempt_before_accept = False
    for j in range(n_rows):
        margin = float(out.top2[j, 0] - out.top2[j, 1])
        if margin >= MARGIN:
            assert ids[j] == out.argmax_ids[j], f"{tag} row {j}: id {ids[j]} != {out.argmax_ids[j]} (margin {margin})"
        else:
            stats["exempt"] += 1
            # still inside the oracle's near-tie set
            assert out.logits[j, ids[j]] > out.top2[j, 0] - MARGIN, f"{tag} row {j}: id outside the near-tie set"
    if res.top2 is not None and n_rows:
        t2 = res.top2[b, :n_rows].cpu().numpy()
        assert np.abs(t2 - out.top2).max() <= LOGITS_MAX_ABS, f"{tag} top-2 values"
    if check_accept:
        # the acceptance rule applied to the GPU's own ids
        a = 0
        while a < len(S) and a < n_rows and int(S[a]) == ids[a]:
            a += 1
        nxt = ids[a] if a < n_rows else -1
        assert int(res.n_accepted[b]) == a and int(res.next_token[b]) == nxt, f"{tag} acceptance vs own ids"
        if ids == out.argmax_ids:
            assert a == out.n_accepted and nxt == out.next_token, f"{tag} acceptance vs oracle"
        stats["ids_equal"] = ids == out.argmax_ids
    return stats


def compare_kv(st: binding.KVState, b: int, ost, page_size: int, layers, positions, tag: str = "", slack: float = 1.0):
    """K/V appended by the call at `positions`: equal to the oracle's bf16-rounded entries up to one
    bf16 rounding step (the two sides round nearly equal fp32 values independently) plus 2 % of the
    entry's row RMS (bf16-rounded activations perturb small entries by more than their own ulp)."""
    bt = st.block_table[b].cpu()
    for l in layers:
        for pages, ref in ((st.k_pages, ost.cache.k), (st.v_pages, ost.cache.v)):
            g = cache_from_pages(pages, bt, page_size, l, st.first_layer, positions)
            r = ref[l, list(positions)]
            tol = np.abs(r) * 2.0 ** -7 + slack * 2e-2 * np.sqrt(np.mean(r.astype(np.float64) ** 2, axis=-1, keepdims=True))
            assert np.all(np.abs(g - r) <= tol), f"{tag} layer {l}: appended K/V differ"


def load_dense_kv(st: binding.KVState, b: int, layer_slot: int, k_dense: torch.Tensor, v_dense: torch.Tensor,
                  page_size: int):
    """Vectorised scatter of one layer's dense K/V [ctx][hkv][hd] (bf16) into sequence b's pages."""
    ctx_len = k_dense.shape[0]
    bt = st.block_table[b].long()
    n_full, rem = divmod(ctx_len, page_size)
    for pages, dense in ((st.k_pages, k_dense), (st.v_pages, v_dense)):
        dense = dense.to(pages.device)
        if n_full:
            blk = dense[: n_full * page_size].reshape(n_full, page_size, *dense.shape[1:]).permute(0, 2, 1, 3)
            pages[layer_slot, bt[:n_full]] = blk
        if rem:
            pages[layer_slot, bt[n_full], :, :rem] = dense[n_full * page_size:].permute(1, 0, 2)
