#!/usr/bin/env python
"""Benchmark of the HiSpec verification path on B200.

One *step* is one super-round of Algorithm 2 on the Llama-3-8B-shaped early-exit
model (exits 8/16/32, batch 1, prompt 1024, k = N_d = 5, target verification after
every 2 intermediate rounds): 2 x [6 draft steps through layers [0,8) + one
intermediate verification of 6 rows through [8,16)] + one target verification of
the tentatively accepted rows through [16,32).  Every step of it runs in the
library's CUDA kernels, called through the C ABI.

  value   verified tokens/s: tokens committed after target verification divided by
          the device time of K steps, all inputs resident in HBM, no host round trip;
  e2e     the same metric through the public driver with host buffers: per step the
          host reads the step's result record (device -> pinned host) and the tokens
          are assembled on the host, and the next step's input -- the pending token, 4
          bytes -- is uploaded from pinned host memory; the prompt ids were uploaded the
          same way before the timed region;
  roofline  projections (the dominant kernel): weight bytes streamed / summed event
          time of the bracketed launches, against the measured HBM copy bandwidth;
  cpu_baseline  the fp32 CPU oracle timed on one super-round of the same shape.

`--impl reference` times the oracle alone (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "verified tokens/s per B200 (HiSpec, Llama-3-8B shape, batch 1, k=5)"
UNIT = "tokens/s"
N_PROMPT, N_D, ROUNDS = 1024, 5, 2
# dram__bytes_read.sum + dram__bytes_write.sum of one hispec_stage_kernel launch (a verify-I call of this
# workload: layers [8,16) + head, 6 rows, context 1024, 4.576 GB algorithmic) from the ncu capture summarised
# under profiles/.  The launches of a super-round differ in size (a block of 6 draft steps, a verify-I, a
# verify-T); their traffic is that ratio times their algorithmic bytes (traffic is the weight stream, read once).
ROOFLINE_TRAFFIC_BYTES_CAPTURED = 4.628e9
ROOFLINE_TRAFFIC_RATIO = ROOFLINE_TRAFFIC_BYTES_CAPTURED / 4.576e9


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            j = json.load(open(p))
            return float(j["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler(threading.Thread):
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.samples, self.stop_flag = index, [], False

    def run(self):
        while not self.stop_flag:
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                      "-i", str(self.index)], capture_output=True, text=True, timeout=5).stdout
                parts = [x.strip() for x in out.strip().split(",")]
                if len(parts) >= 6:
                    self.samples.append(parts)
            except Exception:
                pass
            time.sleep(0.05)

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        sm = sorted(int(float(s[0])) for s in self.samples)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(s[2 + i].lower().startswith("active") for s in self.samples)]
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": int(float(self.samples[0][1])), "reasons": reasons,
                "samples": len(sm)}


def algorithmic_bytes_super_round(shape, ctx_len: int) -> float:
    """What one super-round must move: weights of each call's layer range + head, KV read/write, hidden rows."""
    W, H, kvb = shape.layer_weight_bytes, shape.head_bytes, shape.kv_bytes_per_token_layer
    d4 = shape.d_model * 4
    draft = shape.L_d * W + H + shape.L_d * kvb * (ctx_len + 1) + d4
    vi = (shape.L_i - shape.L_d) * W + H + (shape.L_i - shape.L_d) * kvb * (ctx_len + N_D + 1) + 2 * (N_D + 1) * d4
    rows_t = ROUNDS * (N_D + 1)
    vt = (shape.L_f - shape.L_i) * W + H + (shape.L_f - shape.L_i) * kvb * (ctx_len + rows_t) + rows_t * d4
    return ROUNDS * ((N_D + 1) * draft + vi) + vt


def aggregate_replicas(ms_list, tok_list, world, device="cuda"):
    """Replicas only: whole-job time = max over ranks, whole-job tokens = sum over ranks."""
    if world <= 1:
        return list(ms_list), list(tok_list)
    import torch
    import torch.distributed as dist
    t = torch.tensor(ms_list, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    c = torch.tensor(tok_list, dtype=torch.float64, device=device)
    dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return t.tolist(), c.tolist()


def run_ours(args, rank, world, local_rank):
    import torch
    from paper_2510_01336_b200 import binding, workload as wl
    from paper_2510_01336_b200.driver import HiSpecLoop

    torch.cuda.set_device(local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    shape = wl.L3_8B
    t0 = time.time()
    w = wl.make_weights(shape, device="cuda")
    max_rows = ROUNDS * (N_D + 1) + 1
    n_super = args.warmup + 2 * args.steps + 16
    max_ctx = N_PROMPT + n_super * ROUNDS * (N_D + 1) + 64
    max_pages = (max_ctx + 15) // 16
    ctx = binding.Context(shape, w, page_size=16, max_batch=1, max_rows_per_seq=max_rows, max_pages_per_seq=max_pages)
    st = ctx.new_state(1, max_pages, wl.make_block_table(shape, 1, max_pages))
    loop = HiSpecLoop(ctx, st, 1, N_D, ROUNDS)
    prompt_host = wl.make_tokens(shape, N_PROMPT).pin_memory()
    loop.prefill([prompt_host.tolist()])
    setup_s = time.time() - t0
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    def timed(n_steps, host_roundtrip):
        l0 = int(st.len_target[0])
        n0 = ctx.launch_count()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        wall0 = time.perf_counter()
        e0.record(stream)
        for _ in range(n_steps):
            loop.enqueue_super_round()
            if host_roundtrip:
                loop.collect()
                loop.push_pending()
        e1.record(stream)
        barrier()
        wall = time.perf_counter() - wall0
        ms = e0.elapsed_time(e1)
        if host_roundtrip:
            ms = max(ms, wall * 1e3)
        toks = int(st.len_target[0]) - l0
        return ms, toks, ctx.launch_count() - n0

    for _ in range(max(args.warmup, 3)):
        loop.enqueue_super_round()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    # roofline of the dominant kernel (the persistent per-call kernel, one launch per stage call): every launch of
    # the timed region is bracketed by a pair of CUDA events on the launching stream
    ctx_len_roof = int(st.len_target[0])
    ctx.profile_enable(True)
    ctx.profile_read(20)
    ms, toks, launches = timed(args.steps, False)
    g_ms, g_wbytes, g_n = ctx.profile_read(20)
    ctx.profile_enable(False)
    sampler.stop_flag = True
    ms_e2e, toks_e2e, _ = timed(args.steps, True)
    status = ctx.status()
    peak, peak_kind = peaks()
    roof_bytes = args.steps * algorithmic_bytes_super_round(shape, ctx_len_roof)
    achieved = roof_bytes / (g_ms * 1e-3) / 1e9 if g_ms > 0 else 0.0

    (ms, ms_e2e), (toks, toks_e2e) = aggregate_replicas([ms, ms_e2e], [float(toks), float(toks_e2e)], world)
    if rank != 0:
        return
    ctx_len = N_PROMPT + args.warmup * 2
    step_bytes = algorithmic_bytes_super_round(shape, ctx_len)
    line = {
        "metric": METRIC, "value": toks / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "configs[1]: Llama-3-8B-shaped early-exit model, exits 8/16/32, batch 1, prompt 1024 "
                               "uniform-random tokens, k=5 greedy drafts, target every 2 intermediate rounds; "
                               "bf16 N(0,0.02) weights (literal: near-zero acceptance)",
                   "step": "one super-round: 2 x (6 draft steps as one call + verify-I) + verify-T", "replicas": world,
                   "l2": "inputs larger than L2 (each call streams >= 4.5 GB of weights)",
                   "activations": "bf16 hi+lo split", "tokens_committed": toks,
                   "algorithmic_gb_per_step": step_bytes / 1e9,
                   "step_hbm_gbs": step_bytes / 1e9 / (ms / args.steps * 1e-3), "device_status": status,
                   "setup_s": round(setup_s, 1)},
        "clocks": sampler.summary(),
        "e2e": {"value": toks_e2e / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 4,
                "d2h_bytes_per_step": 4 * (2 + max_rows + ROUNDS), "ms_per_step": ms_e2e / args.steps,
                "prompt_h2d_bytes": 4 * N_PROMPT},
        "gpu_launches": launches,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": ROOFLINE_TRAFFIC_RATIO * roof_bytes / max(g_n, 1),
                     "traffic_note": "ncu DRAM read+write of a verify-I launch (4.628 GB for 4.576 GB algorithmic), "
                                     "scaled to the average launch by algorithmic bytes",
                     "kernel": "hispec_stage_kernel (one launch = one block of draft steps, one verify-I or one verify-T call)",
                     "launches": g_n, "avg_launch_us": 1e3 * g_ms / max(g_n, 1),
                     "algorithmic_bytes_per_launch": roof_bytes / max(g_n, 1), "weight_bytes_per_launch": g_wbytes / max(g_n, 1),
                     "peak_source": f"of {peak_kind}", "frac_of_8TBs": achieved / 8000.0},
    }
    if not args.no_extras and world == 1:
        line["config"]["context_same_box"] = extras(shape, w, args)
    if not args.no_cpu_baseline and world == 1:
        del loop, ctx, st
        torch.cuda.empty_cache()
        line["cpu_baseline"] = cpu_super_round(shape, w, budget_steps=1)
    print(json.dumps(line), flush=True)


def extras(shape, w, args):
    """Context numbers on the same box (not the headline): plain auto-regressive decoding and Algorithm 1 on the
    literal weights, and HiSpec / Algorithm 1 / AR on acceptance-shaped weights (Wo, Wdown of the layers above the
    draft exit scaled by 0.05, so that the exits agree as trained early-exit checkpoints do)."""
    import torch
    from paper_2510_01336_b200 import binding, workload as wl
    from paper_2510_01336_b200.driver import ARLoop, HiSpecLoop, HiSpecSamplingLoop, SelfSpecLoop
    out = {}
    max_rows = ROUNDS * (N_D + 1) + 1
    max_pages = (N_PROMPT + 1024 + 15) // 16
    prompt = wl.make_tokens(shape, N_PROMPT).tolist()

    def timed_tokens(make_loop, run, weights):
        ctx = binding.Context(shape, weights, page_size=16, max_batch=1, max_rows_per_seq=max_rows, max_pages_per_seq=max_pages)
        st = ctx.new_state(1, max_pages, wl.make_block_table(shape, 1, max_pages))
        loop = make_loop(ctx, st)
        loop.prefill([prompt])
        l0 = int(st.len_target[0])
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        run(loop)
        e1.record()
        torch.cuda.synchronize()
        toks = int(st.len_target[0]) - l0
        stats = getattr(loop, "stats", None)
        ctx.close()
        return toks / (e0.elapsed_time(e1) * 1e-3), toks, stats

    def run_ar(loop):
        loop.generate(48)

    def run_hs(loop):
        for _ in range(12):
            loop.enqueue_super_round()

    def run_ss(loop):
        for _ in range(16):
            loop.enqueue_round()

    out["ar_tokens_per_s"] = round(timed_tokens(lambda c, s: ARLoop(c, s, 1), run_ar, w)[0], 1)
    out["selfspec_alg1_tokens_per_s"] = round(timed_tokens(lambda c, s: SelfSpecLoop(c, s, 1, N_D), run_ss, w)[0], 1)
    wg = wl.make_weights(shape, device="cuda", resid_scale={l: 0.05 for l in range(shape.L_d, shape.L_f)})
    tps, toks, stats = timed_tokens(lambda c, s: HiSpecLoop(c, s, 1, N_D, ROUNDS), run_hs, wg)
    ss = timed_tokens(lambda c, s: SelfSpecLoop(c, s, 1, N_D), run_ss, wg)
    ar = timed_tokens(lambda c, s: ARLoop(c, s, 1), run_ar, wg)[0]
    # the same loop with rejection-sampling acceptance at both stages (App. G), temperature 1
    uni = lambda sr: wl.make_uniforms(shape, sr, 1, ROUNDS, N_D, max_rows)
    rs = timed_tokens(lambda c, s: HiSpecSamplingLoop(c, s, 1, N_D, ROUNDS, uni), run_hs, wg)
    out["rejection_sampling_gamma0.05"] = {"hispec_tokens_per_s": round(rs[0], 1), "tokens_per_super_round": round(rs[1] / 12, 2),
                                           "over_greedy_hispec": round(rs[0] / tps, 2)}
    out["acceptance_shaped_gamma0.05"] = {"hispec_tokens_per_s": round(tps, 1), "tokens_per_super_round": round(toks / 12, 2),
                                          "selfspec_alg1_tokens_per_s": round(ss[0], 1), "tokens_per_alg1_round": round(ss[1] / 16, 2),
                                          "ar_tokens_per_s": round(ar, 1), "hispec_over_ar": round(tps / ar, 2),
                                          "hispec_over_alg1": round(tps / ss[0], 2)}
    del wg
    torch.cuda.empty_cache()
    return out


def cpu_super_round(shape, w_gpu, budget_steps: int):
    """The oracle, as it stands, timed on one super-round of the same shape from a synthetic cached state
    (K/V of all layers for 1024 positions drawn N(0,1): a CPU prefill of 1024 tokens would take hours)."""
    import numpy as np
    import torch
    from oracle import hispec as orc
    from paper_2510_01336_b200 import workload as wl

    w = w_gpu.to("cpu") if w_gpu is not None else wl.make_weights(shape)
    m = orc.OracleModel.from_weights(w, kv_round_bf16=True)
    hs = orc.HiSpecOracle(m, shape.L_d, shape.L_i, shape.L_f)
    rows = ROUNDS * (N_D + 1) + 1
    st = hs.new_state(N_PROMPT + 4 * rows, rows)
    rng = np.random.default_rng(shape.seed + 4000)
    for l in range(shape.n_layers):
        st.cache.k[l, :N_PROMPT] = rng.standard_normal(st.cache.k[l, :N_PROMPT].shape, dtype=np.float32)
        st.cache.v[l, :N_PROMPT] = rng.standard_normal(st.cache.v[l, :N_PROMPT].shape, dtype=np.float32)
    st.len_d = st.len_i = st.len_f = N_PROMPT
    pending = int(wl.make_tokens(shape, 1, seed_offset=5000)[0])
    times, committed = [], 0
    for _ in range(budget_steps):
        t0 = time.perf_counter()
        V = []
        for _r in range(ROUNDS):
            S, u = [], pending
            for j in range(N_D + 1):
                o = hs.draft_step(st, u)
                if j < N_D:
                    S.append(o.argmax_ids[0])
                    u = S[-1]
            o = hs.verify_intermediate(st, S, N_D + 1)
            Vh, _ = orc.leading_substring_verify(S, o.argmax_ids)
            V += Vh
            pending = V[-1]
        o = hs.verify_target(st, V, len(V))
        F, _ = orc.leading_substring_verify(V, o.argmax_ids)
        pending = F[-1]
        committed += len(F)
        times.append(time.perf_counter() - t0)
    total = sum(times)
    return {"value": committed / total, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
            "sample": f"{budget_steps} super-round(s) of the same shape (2 x (6 draft steps + verify-I of 6 rows) + "
                      f"verify-T) from a synthetic cached state of 1024 positions; {total:.1f} s of CPU work",
            "s_per_step": total / budget_steps}


def run_sweep(args):
    """Verify-step latency vs k (rows per sequence) x batch x context on the Llama-3-8B shape: one
    hispec_verify_intermediate call over [8, L_i) + exit head from seeded random state, median of 15 calls.
    Prints one JSON line per point (not the benchmark line)."""
    import torch
    from paper_2510_01336_b200 import binding, workload as wl
    import dataclasses
    torch.cuda.set_device(0)
    peak, peak_kind = peaks()
    free_b, _ = torch.cuda.mem_get_info()
    for L_i in ([16] if not args.sweep_all_li else [12, 16, 24]):
        shape = dataclasses.replace(wl.L3_8B, L_i=L_i)
        layers = list(range(shape.L_d, L_i))
        w = wl.make_weights(shape, layers=layers, device="cuda", with_emb=False)
        for B in (1, 4, 16, 64):
            for ctx_len in (512, 4096, 32768):
                kv_bytes = 2 * B * (ctx_len + 32) * len(layers) * shape.kv_bytes_per_token_layer // 2 * 1
                kv_bytes = B * (ctx_len + 32) * len(layers) * shape.kv_bytes_per_token_layer
                if kv_bytes > 0.8 * free_b:
                    print(json.dumps({"sweep": True, "L_i": L_i, "B": B, "ctx": ctx_len, "fits": False,
                                      "kv_gb": kv_bytes / 1e9}), flush=True)
                    continue
                max_pages = (ctx_len + 32 + 15) // 16
                ctxo = binding.Context(shape, w, page_size=16, max_batch=B, max_rows_per_seq=17, max_pages_per_seq=max_pages)
                st = ctxo.new_state(B, B * max_pages, wl.make_block_table(shape, B, max_pages), first_layer=shape.L_d,
                                    n_pool_layers=len(layers))
                g = torch.Generator(device="cuda").manual_seed(shape.seed + 4000)
                st.k_pages.normal_(generator=g)
                st.v_pages.normal_(generator=g)
                st.h_draft.normal_(generator=g)
                res = ctxo.new_result(B)
                for k in (1, 2, 4, 8, 16):
                    kd = max(k - 1, 1)
                    drafts = torch.zeros((B, kd), dtype=torch.int32, device="cuda")
                    nd = torch.full((B,), k - 1, dtype=torch.int32, device="cuda")
                    nr = torch.full((B,), k, dtype=torch.int32, device="cuda")
                    times = []
                    for it in range(18):
                        st.len_draft.fill_(ctx_len + k)
                        st.len_inter.fill_(ctx_len)
                        st.len_target.fill_(ctx_len)
                        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        e0.record()
                        ctxo.verify_intermediate(st, drafts, nd, nr, res, k=k - 1 if k > 1 else 0)
                        e1.record()
                        torch.cuda.synchronize()
                        if it >= 3:
                            times.append(e0.elapsed_time(e1))
                    times.sort()
                    ms = times[len(times) // 2]
                    T = B * k
                    by = (len(layers) * shape.layer_weight_bytes + shape.head_bytes +
                          B * len(layers) * shape.kv_bytes_per_token_layer * (ctx_len + k) + 2 * T * shape.d_model * 4)
                    fl = 2.0 * T * (len(layers) * shape.layer_params + shape.vocab * shape.d_model) + \
                        B * len(layers) * 4.0 * shape.n_q_heads * shape.head_dim * k * (ctx_len + (k + 1) / 2)
                    print(json.dumps({"sweep": True, "L_i": L_i, "B": B, "ctx": ctx_len, "k": k, "us": round(ms * 1e3, 1),
                                      "algorithmic_gb": round(by / 1e9, 3), "gbs": round(by / ms / 1e6, 0),
                                      "frac_of_measured_hbm": round(by / ms / 1e6 / peak, 3), "tflops": round(fl / ms / 1e9, 1),
                                      "status": ctxo.status()}), flush=True)
                ctxo.close()
                del st, ctxo
                torch.cuda.empty_cache()
        del w
        torch.cuda.empty_cache()


def run_configs(args):
    """The two serving configurations of the workload list beside the benchmarked one: per-call latency of the
    intermediate and the target verification on seeded random state (median of 15 calls), with the algorithmic
    bytes and flops of each call.  cfg3: Llama-3-8B shape, 16 sequences, contexts uniform in [512, 4096], k = 8
    (9 rows with the bonus row; the target checks 2 x 9 = 18 rows).  cfg4: Llama-2-13B shape, 8 sequences, context
    2048, k = 6 (7 rows; target 14).  One JSON line per call (not the benchmark line)."""
    import torch
    from paper_2510_01336_b200 import binding, workload as wl
    torch.cuda.set_device(0)
    peak, _ = peaks()
    cases = [("cfg3", wl.L3_8B, 16, 8, wl.make_prompt_lengths(wl.L3_8B, 16, 512, 4096)),
             ("cfg4", wl.L2_13B, 8, 6, [2048] * 8)]
    for name, shape, B, k, ctx_lens in cases:
        for call, l0, l1, R in (("verify_i", shape.L_d, shape.L_i, k + 1), ("verify_t", shape.L_i, shape.L_f, 2 * (k + 1))):
            layers = list(range(l0, l1))
            w = wl.make_weights(shape, layers=layers, device="cuda", with_emb=False)
            max_rows = 2 * (k + 1) + 1
            max_pages = (max(ctx_lens) + max_rows + 15) // 16 + 1
            ctxo = binding.Context(shape, w, page_size=16, max_batch=B, max_rows_per_seq=max_rows, max_pages_per_seq=max_pages)
            st = ctxo.new_state(B, B * max_pages, wl.make_block_table(shape, B, max_pages), first_layer=l0,
                                n_pool_layers=len(layers))
            g = torch.Generator(device="cuda").manual_seed(shape.seed + 4000)
            for t in (st.k_pages, st.v_pages, st.h_draft, st.h_inter):
                t.normal_(generator=g)
            res = ctxo.new_result(B)
            base = torch.tensor(ctx_lens, dtype=torch.int32, device="cuda")
            drafts = torch.zeros((B, max_rows - 1), dtype=torch.int32, device="cuda")
            nr = torch.full((B,), R, dtype=torch.int32, device="cuda")
            nd = torch.full((B,), R - 1 if call == "verify_i" else R, dtype=torch.int32, device="cuda")
            times = []
            for it in range(18):
                st.len_draft.copy_(base + R)
                st.len_inter.copy_(base + (R if call == "verify_t" else 0))
                st.len_target.copy_(base)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                # k of the call: rows are padded to k + 1 per sequence, so the tightest k that admits the rows
                (ctxo.verify_intermediate if call == "verify_i" else ctxo.verify_target)(st, drafts, nd, nr, res, k=R - 1 if call == "verify_i" else R)
                e1.record()
                torch.cuda.synchronize()
                if it >= 3:
                    times.append(e0.elapsed_time(e1))
            times.sort()
            ms = times[len(times) // 2]
            T = B * R
            by = (len(layers) * shape.layer_weight_bytes + shape.head_bytes +
                  sum(len(layers) * shape.kv_bytes_per_token_layer * (c + R) for c in ctx_lens) + 2 * T * shape.d_model * 4)
            fl = 2.0 * T * (len(layers) * shape.layer_params + shape.vocab * shape.d_model) + \
                sum(len(layers) * 4.0 * shape.n_q_heads * shape.head_dim * R * (c + (R + 1) / 2) for c in ctx_lens)
            print(json.dumps({"config": name, "shape": shape.name, "call": call, "layers": [l0, l1], "batch": B, "rows_per_seq": R,
                              "mean_ctx": round(sum(ctx_lens) / B), "us": round(ms * 1e3, 1),
                              "algorithmic_gb": round(by / 1e9, 3), "gbs": round(by / ms / 1e6, 0),
                              "frac_of_measured_hbm": round(by / ms / 1e6 / peak, 3), "tflops": round(fl / ms / 1e9, 1),
                              "status": ctxo.status()}), flush=True)
            ctxo.close()
            del st, ctxo, w
            torch.cuda.empty_cache()


def run_reference(args, rank, world):
    if rank != 0:
        return
    from paper_2510_01336_b200 import workload as wl
    shape = wl.L3_8B
    # sized so that the whole run stays within a few minutes: one super-round per step, at most 3 timed steps
    n = max(1, min(args.steps, 3))
    t0 = time.perf_counter()
    base = cpu_super_round(shape, None, budget_steps=n)
    line = {"impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": world,
            "steps": n, "warmup": 0, "ms_per_step": base["s_per_step"] * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "configs[1] shape; the CPU oracle on a bounded sample", "requested_steps": args.steps,
                       "wall_s": round(time.perf_counter() - t0, 1)},
            "cpu_baseline": {k: base[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the AR / Algorithm 1 / acceptance-shaped context numbers")
    ap.add_argument("--sweep", action="store_true", help="verify-step latency vs k / batch / context (not the bench line)")
    ap.add_argument("--sweep-all-li", action="store_true", help="sweep intermediate exits 12, 16, 24 instead of 16 only")
    ap.add_argument("--configs", action="store_true", help="per-call latency of the serving configurations cfg3 / cfg4 (not the bench line)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.sweep:
        if rank == 0:
            run_sweep(args)
    elif args.configs:
        if rank == 0:
            run_configs(args)
    elif args.impl == "reference":
        run_reference(args, rank, world)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
