"""A small stand-alone case of the hot call for profilers: one intermediate-verification call
(layers [L_d, L_i) + exit head) of the Llama-3-8B-shaped model (or another shape, --shape) on seeded random
state, repeated a few times.  Device footprint ~5 GB at the default shape (8 layers of weights + head + a 1024-token KV pool): large against the
126 MB L2, small enough for a multi-pass ncu capture.

    python -m paper_2510_01336_b200.profile_case --calls 3
"""
from __future__ import annotations

import argparse

import torch

from . import binding, workload as wl


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--calls", type=int, default=3)
    ap.add_argument("--rows", type=int, default=6)
    ap.add_argument("--batch", type=int, default=1, help="sequences in the call (rows and context apply to each)")
    ap.add_argument("--ctx", type=int, default=1024)
    ap.add_argument("--flags", type=int, default=0)
    ap.add_argument("--shape", default="llama3-8b-shape", choices=sorted(wl.SHAPES),
                    help="model shape; the call covers its intermediate range [L_d, L_i)")
    args = ap.parse_args()
    shape = wl.SHAPES[args.shape]
    layers = list(range(shape.L_d, shape.L_i))
    w = wl.make_weights(shape, layers=layers, device="cuda", with_emb=False)
    B = args.batch
    max_rows = 13 if B == 1 else args.rows
    max_pages = (args.ctx + max_rows + 15) // 16 + 1
    ctx = binding.Context(shape, w, page_size=16, max_batch=B, max_rows_per_seq=max_rows, max_pages_per_seq=max_pages,
                          flags=args.flags)
    st = ctx.new_state(B, B * max_pages, wl.make_block_table(shape, B, max_pages), first_layer=shape.L_d,
                       n_pool_layers=len(layers))
    g = torch.Generator(device="cuda").manual_seed(shape.seed + 4000)
    st.k_pages.normal_(generator=g)
    st.v_pages.normal_(generator=g)
    st.h_draft.normal_(generator=g)
    res = ctx.new_result(B)
    i32 = lambda v: torch.tensor(v, dtype=torch.int32, device="cuda")
    drafts = torch.zeros((B, max(max_rows - 1, 1)), dtype=torch.int32, device="cuda")
    nd, nr = i32([args.rows - 1] * B), i32([args.rows] * B)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.calls + 1)]
    ev[0].record()
    for i in range(args.calls):
        st.len_draft.fill_(args.ctx + args.rows)
        st.len_inter.fill_(args.ctx)
        st.len_target.fill_(args.ctx)
        ctx.verify_intermediate(st, drafts, nd, nr, res, k=args.rows - 1)
        ev[i + 1].record()
    torch.cuda.synchronize()
    status = ctx.status()
    by = len(layers) * shape.layer_weight_bytes + shape.head_bytes + B * len(layers) * shape.kv_bytes_per_token_layer * (args.ctx + args.rows)
    for i in range(args.calls):
        ms = ev[i].elapsed_time(ev[i + 1])
        print(f"{shape.name} [{shape.L_d},{shape.L_i}) batch {B} rows {args.rows} ctx {args.ctx} call {i}: {ms * 1e3:.1f} us, "
              f"{by / 1e9:.2f} GB, {by / ms / 1e6:.0f} GB/s algorithmic, status {status}")
    ctx.close()


if __name__ == "__main__":
    main()
