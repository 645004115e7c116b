"""Host decoding loops over the C-ABI calls: HiSpec (Algorithm 2), single-stage
self-speculation (Algorithm 1) and plain auto-regressive decoding.

The loops only sequence calls and keep token lists; all arithmetic, the
acceptance rule and the pruning of the shared state run in the library's
kernels.  A super-round of HiSpec (m rounds of [N_d (+1) draft steps,
intermediate verification] followed by one target verification) is enqueued
without any host synchronisation: draft ids flow from one draft step to the
next and into the verifier through device memory, the list V of tentatively
accepted tokens is assembled by the intermediate verifier's acceptance kernel,
and the target verifier takes its row count from the length counters.  The
host reads back one small record per super-round.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, List, Optional

import torch

from . import binding


@dataclass
class LoopStats:
    super_rounds: int = 0
    draft_steps: int = 0
    inter_calls: int = 0
    target_calls: int = 0
    inter_accepted: int = 0
    target_checked: int = 0
    target_accepted: int = 0
    committed: int = 0


class HiSpecLoop:
    """Batch of sequences decoded in lockstep (every sequence runs the same phase; the
    acceptance outcome is per sequence)."""

    def __init__(self, ctx: binding.Context, st: binding.KVState, batch: int, N_d: int, rounds: int = 2,
                 bonus_inter: bool = True, device: str = "cuda", block_drafts: bool = True):
        per_round = N_d + (1 if bonus_inter else 0)
        assert per_round * rounds <= ctx.max_rows - 1, "hidden buffers too small: need rounds * (N_d + 1) + 1 rows"
        self.ctx, self.st, self.B, self.N_d, self.rounds, self.bonus = ctx, st, batch, N_d, rounds, bonus_inter
        self.block_drafts = block_drafts   # Generate(L_d, ., N_d) as one library call instead of N_d (+1)
        i32 = lambda *s: torch.zeros(s, dtype=torch.int32, device=device)
        self.pending = i32(batch)                      # token waiting to enter the draft layers
        self.S = i32(batch, N_d)                       # draft block of the current round
        self.res_i = [binding.Result(i32(batch), i32(batch)) for _ in range(rounds)]
        self.V = i32(batch, ctx.max_rows)              # tentatively accepted tokens (device-assembled)
        for r in self.res_i:
            r.tentative = self.V
            r.pending = self.pending
        self.res_t = binding.Result(i32(batch), i32(batch))
        self.res_t.pending = self.pending
        self.len_snapshot = i32(batch)
        # pinned host mirrors read once per super-round
        self.h_acc = torch.zeros(batch, dtype=torch.int32).pin_memory()
        self.h_next = torch.zeros(batch, dtype=torch.int32).pin_memory()
        self.h_V = torch.zeros((batch, ctx.max_rows), dtype=torch.int32).pin_memory()
        self.h_acc_i = torch.zeros((rounds, batch), dtype=torch.int32).pin_memory()
        self.h_nv = torch.zeros(batch, dtype=torch.int32).pin_memory()
        self.stats = LoopStats()
        self.tokens: List[List[int]] = [[] for _ in range(batch)]

    # -- prompt ---------------------------------------------------------------------------
    def prefill(self, prompts: List[List[int]]):
        B = self.B
        mx = max(len(p) for p in prompts)
        toks = torch.zeros((B, mx), dtype=torch.int32)
        for b, p in enumerate(prompts):
            toks[b, : len(p)] = torch.tensor(p, dtype=torch.int32)
        n = torch.tensor([len(p) for p in prompts], dtype=torch.int32)
        self.ctx.prefill(self.st, toks.cuda(), n.cuda(), self.pending)
        torch.cuda.synchronize()
        first = self.pending.cpu().tolist()
        for b in range(B):
            self.tokens[b] = [first[b]]
        return first

    # -- one super-round, enqueued without host synchronisation ---------------------------------
    def enqueue_super_round(self, stream=None):
        ctx, st, N_d, B = self.ctx, self.st, self.N_d, self.B
        S_ptr = self.S.data_ptr()
        for r in range(self.rounds):
            src = self.pending  # kept current by the acceptance kernel of the previous verification
            if self.block_drafts:
                # Generate(L_d, ., N_d) as one call: all draft steps (and the bonus step) inside one launch
                ctx.draft_block(st, src, self.S, N_d, bonus=self.bonus, stream=stream)
            else:
                # step j reads column j-1 of S (or the pending token) and writes column j
                for j in range(N_d):
                    if j == 0:
                        ctx.draft(st, src, S_ptr, batch=B, in_stride=1, out_stride=N_d, stream=stream)
                    else:
                        ctx.draft(st, S_ptr + 4 * (j - 1), S_ptr + 4 * j, batch=B, in_stride=N_d, out_stride=N_d,
                                  stream=stream)
                if self.bonus:  # push S_{N_d} through the draft layers so that L_i can emit v_{N_d+1}
                    ctx.draft(st, S_ptr + 4 * (N_d - 1), None, batch=B, in_stride=N_d, stream=stream)
            ctx.verify_intermediate(st, self.S, None, None, self.res_i[r], stream=stream, k=N_d)
            self.stats.draft_steps += N_d + (1 if self.bonus else 0)
            self.stats.inter_calls += 1
        # LeadingSubstringVerify(V, L_f, x): rows and |V| come from the length counters
        ctx.verify_target(st, self.V, None, None, self.res_t, stream=stream, k=ctx.max_rows - 1)
        self.stats.target_calls += 1
        self.stats.super_rounds += 1

    def collect(self, stream=None):
        """Read back the outcome of the last super-round and extend the token lists.
        Must follow enqueue_super_round; synchronises the stream."""
        s = stream if stream is not None else torch.cuda.current_stream()
        with torch.cuda.stream(s):
            self.h_acc.copy_(self.res_t.n_accepted, non_blocking=True)
            self.h_next.copy_(self.res_t.next_token, non_blocking=True)
            self.h_V.copy_(self.V, non_blocking=True)
            for r in range(self.rounds):
                self.h_acc_i[r].copy_(self.res_i[r].n_accepted, non_blocking=True)
        s.synchronize()
        new = []
        for b in range(self.B):
            a = int(self.h_acc[b])
            nxt = int(self.h_next[b])
            F = self.h_V[b, :a].tolist() + ([nxt] if nxt >= 0 else [])
            self.tokens[b] += F
            new.append(F)
            self.stats.target_accepted += a
            self.stats.committed += len(F)
            self.stats.inter_accepted += int(self.h_acc_i[:, b].sum())
        return new

    def push_pending(self, stream=None):
        """Host-driven serving loop: upload, from pinned host memory, the token the host read back last as the next
        draft input (4 bytes per sequence).  The acceptance kernel has left the same value on the device, so results
        do not change; a caller that edits the token on the host (a stop rule, a forced token) uses this hook.
        Must follow collect()."""
        if not bool((self.h_next >= 0).all()):
            return
        s = stream if stream is not None else torch.cuda.current_stream()
        with torch.cuda.stream(s):
            self.pending.copy_(self.h_next, non_blocking=True)

    def generate(self, n_gen: int) -> List[List[int]]:
        while min(len(t) for t in self.tokens) < n_gen:
            self.enqueue_super_round()
            self.collect()
        return [t[:n_gen] for t in self.tokens]


class HiSpecDynamicLoop(HiSpecLoop):
    """Algorithm 2 with the paper's dynamic trigger (Sec. 3.4): intermediate rounds continue until at
    least N_i tokens are tentatively accepted, then the target verifies them.  The host reads the accepted
    count after every intermediate verification (one small device-to-host copy per round) to decide."""

    def __init__(self, ctx, st, batch, N_d, N_i, device="cuda"):
        max_rounds = (ctx.max_rows - 1) // (N_d + 1)
        assert max_rounds >= 1 and N_i + N_d + 1 <= ctx.max_rows - 1, "hidden buffers too small for N_i + N_d + 1 rows"
        super().__init__(ctx, st, batch, N_d, rounds=max_rounds, bonus_inter=True, device=device)
        self.N_i = N_i
        self.h_len = torch.zeros((2, batch), dtype=torch.int32).pin_memory()

    def enqueue_super_round(self, stream=None):
        ctx, st, N_d, B = self.ctx, self.st, self.N_d, self.B
        S_ptr = self.S.data_ptr()
        s = stream if stream is not None else torch.cuda.current_stream()
        self.rounds_used = 0
        for r in range(self.rounds):
            for j in range(N_d):
                if j == 0:
                    ctx.draft(st, self.pending, S_ptr, batch=B, in_stride=1, out_stride=N_d, stream=stream)
                else:
                    ctx.draft(st, S_ptr + 4 * (j - 1), S_ptr + 4 * j, batch=B, in_stride=N_d, out_stride=N_d, stream=stream)
            ctx.draft(st, S_ptr + 4 * (N_d - 1), None, batch=B, in_stride=N_d, stream=stream)
            ctx.verify_intermediate(st, self.S, None, None, self.res_i[r], stream=stream, k=N_d)
            self.stats.draft_steps += N_d + 1
            self.stats.inter_calls += 1
            self.rounds_used += 1
            with torch.cuda.stream(s):
                self.h_len[0].copy_(st.len_inter, non_blocking=True)
                self.h_len[1].copy_(st.len_target, non_blocking=True)
            s.synchronize()
            if int((self.h_len[0] - self.h_len[1]).min()) >= self.N_i:   # every sequence has |V| >= N_i
                break
        ctx.verify_target(st, self.V, None, None, self.res_t, stream=stream, k=ctx.max_rows - 1)
        self.stats.target_calls += 1
        self.stats.super_rounds += 1

    def collect(self, stream=None):
        rounds, self.rounds = self.rounds, self.rounds_used
        try:
            return super().collect(stream)
        finally:
            self.rounds = rounds


@dataclass
class AdaptiveRule:
    """One adaptive hyper-parameter (App. J): the value moves up by one when the step's acceptance rate
    reaches tau_high, down by one when it falls below tau_low, and stays inside [n_min, n_max]."""
    tau_high: float
    tau_low: float
    n_min: int
    n_max: int

    def next(self, n: int, alpha: float) -> int:
        if alpha >= self.tau_high:
            return min(self.n_max, n + 1)
        if alpha < self.tau_low:
            return max(self.n_min, n - 1)
        return n


ND_RULE_PAPER = AdaptiveRule(0.8, 0.5, 1, 3)   # N_d from the intermediate verifier's acceptance rate
NI_RULE_PAPER = AdaptiveRule(0.8, 0.3, 3, 8)   # N_i from the final layer's acceptance rate


class HiSpecAdaptiveLoop(HiSpecDynamicLoop):
    """Algorithm 2 with the adaptive choice of N_d and N_i (App. J).  N_d is re-chosen after every
    intermediate verification, N_i after every target verification; with several sequences in the batch the
    acceptance rate of a step is the mean over the sequences.  The draft block keeps its widest layout
    (stride nd_rule.n_max), so a change of N_d moves no buffer."""

    def __init__(self, ctx, st, batch, N_d, N_i, nd_rule: Optional[AdaptiveRule] = ND_RULE_PAPER,
                 ni_rule: Optional[AdaptiveRule] = NI_RULE_PAPER, device="cuda"):
        nd_max = max(N_d, nd_rule.n_max if nd_rule else N_d)
        ni_max = max(N_i, ni_rule.n_max if ni_rule else N_i)
        super().__init__(ctx, st, batch, nd_max, ni_max, device=device)
        self.nd_rule, self.ni_rule = nd_rule, ni_rule
        self.N_d_cur, self.N_i_cur = N_d, N_i
        # every round commits at least one token to V, so N_i rounds always reach the trigger
        i32 = lambda *sh: torch.zeros(sh, dtype=torch.int32, device=device)
        while len(self.res_i) < ni_max:
            r = binding.Result(i32(batch), i32(batch))
            r.tentative, r.pending = self.V, self.pending
            self.res_i.append(r)
        self.rounds = len(self.res_i)
        self.h_acc_i = torch.zeros((self.rounds, batch), dtype=torch.int32).pin_memory()
        self.h_acc_round = torch.zeros(batch, dtype=torch.int32).pin_memory()
        self.schedule: List[tuple] = []            # ("i", N_d, accepted...) / ("t", N_i, |V|..., accepted...) per step

    def enqueue_super_round(self, stream=None):
        ctx, st, B, W = self.ctx, self.st, self.B, self.N_d      # W: stride of the draft block
        S_ptr = self.S.data_ptr()
        s = stream if stream is not None else torch.cuda.current_stream()
        self.rounds_used = 0
        self._inter_acc = 0
        for r in range(self.rounds):
            n_d = self.N_d_cur
            for j in range(n_d):
                if j == 0:
                    ctx.draft(st, self.pending, S_ptr, batch=B, in_stride=1, out_stride=W, stream=stream)
                else:
                    ctx.draft(st, S_ptr + 4 * (j - 1), S_ptr + 4 * j, batch=B, in_stride=W, out_stride=W, stream=stream)
            ctx.draft(st, S_ptr + 4 * (n_d - 1), None, batch=B, in_stride=W, stream=stream)
            ctx.verify_intermediate(st, self.S, None, None, self.res_i[r], stream=stream, k=n_d)
            self.stats.draft_steps += n_d + 1
            self.stats.inter_calls += 1
            self.rounds_used += 1
            with torch.cuda.stream(s):
                self.h_len[0].copy_(st.len_inter, non_blocking=True)
                self.h_len[1].copy_(st.len_target, non_blocking=True)
                self.h_acc_round.copy_(self.res_i[r].n_accepted, non_blocking=True)
            s.synchronize()
            acc = self.h_acc_round.tolist()
            self.schedule.append(("i", n_d, *acc))
            if self.nd_rule is not None:
                self.N_d_cur = self.nd_rule.next(n_d, sum(acc) / (B * n_d))
            n_v = self.h_len[0] - self.h_len[1]
            if int(n_v.min()) >= self.N_i_cur:   # every sequence has |V| >= N_i
                break
            if int(n_v.max()) + self.N_d_cur + 1 > ctx.max_rows - 1:   # no room for another round's rows
                break
        self._n_v = (self.h_len[0] - self.h_len[1]).tolist()
        ctx.verify_target(st, self.V, None, None, self.res_t, stream=stream, k=ctx.max_rows - 1)
        self.stats.target_calls += 1
        self.stats.super_rounds += 1

    def collect(self, stream=None):
        new = super().collect(stream)
        acc = self.h_acc.tolist()
        self.schedule.append(("t", self.N_i_cur, *self._n_v, *acc))
        if self.ni_rule is not None:
            self.N_i_cur = self.ni_rule.next(self.N_i_cur, sum(acc) / max(1, sum(self._n_v)))
        return new


class HiSpecSamplingLoop(HiSpecLoop):
    """Algorithm 2 with rejection-sampling acceptance at both stages (App. G): draft tokens are sampled
    from the draft exit, every verify call runs with deferred acceptance and writes its logits, and
    hispec_accept_rejection decides on the device.  A super-round is still enqueued without a host
    synchronisation; the uniforms it consumes are inputs (`uniforms(super_round) -> dict`, see
    workload.make_uniforms).  `on_accept(stage, round, record)` -- testing aid -- is called after every
    acceptance with copies of everything it read and wrote (this synchronises)."""

    def __init__(self, ctx, st, batch, N_d, rounds, uniforms: Callable[[int], dict], temperature: float = 1.0,
                 on_accept: Optional[Callable] = None, device="cuda"):
        super().__init__(ctx, st, batch, N_d, rounds, bonus_inter=True, device=device)
        V, R = ctx.shape.vocab, ctx.max_rows
        f = lambda: torch.zeros((batch, R, V), dtype=torch.float32, device=device)
        self.logits_d, self.logits_i, self.logits_t, self.logits_stage = f(), f(), f(), f()
        i32 = lambda *sh: torch.zeros(sh, dtype=torch.int32, device=device)
        # a draft step writes its logits to row 0 of the buffer it is given: step j gets the buffer shifted by j rows
        self.res_d = [binding.Result(i32(batch), i32(batch), logits=self.logits_d.data_ptr() + 4 * j * V) for j in range(N_d)]
        for r in self.res_i:
            r.logits, r.defer_accept = self.logits_i, True
        self.res_t.logits, self.res_t.defer_accept = self.logits_t, True
        self.uniforms, self.temperature, self.on_accept = uniforms, temperature, on_accept
        self.sr = 0

    def _record(self, stage, rnd, S, k, p, q, ua, us, res, lens_before):
        if self.on_accept is None:
            return
        torch.cuda.synchronize()
        st = self.st
        self.on_accept(stage, rnd, {
            "S": S.cpu().clone(), "k": k, "p": p.cpu().clone(), "q": q.cpu().clone(), "u_acc": ua.cpu().clone(),
            "u_smp": us.cpu().clone(), "n_accepted": res.n_accepted.cpu().clone(), "next_token": res.next_token.cpu().clone(),
            "lens_before": lens_before,
            "lens_after": (st.len_draft.cpu().clone(), st.len_inter.cpu().clone(), st.len_target.cpu().clone()),
            "V": self.V.cpu().clone(), "pending": self.pending.cpu().clone()})

    def _lens(self):
        if self.on_accept is None:
            return None
        torch.cuda.synchronize()
        st = self.st
        return (st.len_draft.cpu().clone(), st.len_inter.cpu().clone(), st.len_target.cpu().clone())

    def enqueue_super_round(self, stream=None):
        ctx, st, N_d, B, T = self.ctx, self.st, self.N_d, self.B, self.temperature
        Vc, R = ctx.shape.vocab, ctx.max_rows
        U = {k: v.cuda(non_blocking=True) for k, v in self.uniforms(self.sr).items()}
        self.sr += 1
        S_ptr = self.S.data_ptr()
        for r in range(self.rounds):
            for j in range(N_d):
                if j == 0:
                    ctx.draft(st, self.pending, None, res=self.res_d[j], batch=B, in_stride=1, stream=stream)
                else:
                    ctx.draft(st, S_ptr + 4 * (j - 1), None, res=self.res_d[j], batch=B, in_stride=N_d, stream=stream)
                ctx.sample(self.logits_d.data_ptr() + 4 * j * Vc, R * Vc, U["draft"][r, j], S_ptr + 4 * j, B,
                           out_stride=N_d, temperature=T, stream=stream)
            ctx.draft(st, S_ptr + 4 * (N_d - 1), None, batch=B, in_stride=N_d, stream=stream)
            ctx.verify_intermediate(st, self.S, None, None, self.res_i[r], stream=stream, k=N_d)
            lens = self._lens()
            ctx.accept_rejection(1, st, self.S, N_d, self.logits_d, self.logits_i, U["acc_i"][r], U["smp_i"][r],
                                 self.res_i[r], stage_logits=self.logits_stage, temperature=T, stream=stream)
            self._record(1, r, self.S, N_d, self.logits_d, self.logits_i, U["acc_i"][r], U["smp_i"][r], self.res_i[r], lens)
            self.stats.draft_steps += N_d + 1
            self.stats.inter_calls += 1
        ctx.verify_target(st, self.V, None, None, self.res_t, stream=stream, k=R - 1)
        lens = self._lens()
        ctx.accept_rejection(2, st, self.V, R - 1, self.logits_stage, self.logits_t, U["acc_t"], U["smp_t"], self.res_t,
                             temperature=T, stream=stream)
        self._record(2, 0, self.V, R - 1, self.logits_stage, self.logits_t, U["acc_t"], U["smp_t"], self.res_t, lens)
        self.stats.target_calls += 1
        self.stats.super_rounds += 1


class HiSpecChainLoop:
    """HiSpec with TWO intermediate verifiers, exits e0 < e1 < e2 < e3 (App. K, "multiple intermediate
    verifiers"), through the three-exit ABI: the library is given two overlapping views of the same state --
    view A = (e0, e1, e2) with the length counters (len0, len1, len2) and hidden buffers (h0, h1), view B =
    (e1, e2, e3) with (len1, len2, len3) and (h1, h2).  Drafts and the first verifier are view A's draft and
    intermediate-verification calls; the second verifier is view B's intermediate verification (rows from h1,
    exit rows appended to h2, its result list appended to V2); the target is view B's target verification.  A
    call of view B prunes len1..len3 but does not know layer group 0: a copy len1 -> len0 follows it.  One
    super-round = m2 x [ m1 x (N_d drafts + bonus, verify at e1), verify at e2 ], verify at e3; no host
    synchronisation inside."""

    def __init__(self, shape, weights, exits, batch: int, N_d: int, m1: int, m2: int, max_pages: int, block_table,
                 page_size: int = 16, device: str = "cuda"):
        e0, e1, e2, e3 = exits
        assert 0 < e0 < e1 < e2 < e3 <= shape.n_layers
        rows1 = m1 * (N_d + 1)                 # rows level 1 can accumulate before level 2 runs
        rows2 = m2 * rows1                     # ... level 2 before the target runs
        self.max_rows = rows2 + 2
        self.A = binding.Context(shape, weights, page_size=page_size, max_batch=batch, max_rows_per_seq=self.max_rows,
                                 max_pages_per_seq=max_pages, exits=(e0, e1, e2))
        self.Bc = binding.Context(shape, weights, page_size=page_size, max_batch=batch, max_rows_per_seq=self.max_rows,
                                  max_pages_per_seq=max_pages, exits=(e1, e2, e3))
        self.B, self.N_d, self.m1, self.m2 = batch, N_d, m1, m2
        stA = self.A.new_state(batch, int(block_table.max()) + 1, block_table)
        i32 = lambda *sh: torch.zeros(sh, dtype=torch.int32, device=device)
        f32 = lambda *sh: torch.zeros(sh, dtype=torch.float32, device=device)
        self.len = [stA.len_draft, stA.len_inter, stA.len_target, i32(batch)]      # len0..len3
        self.h = [stA.h_draft, stA.h_inter, f32(batch, self.max_rows, shape.d_model)]
        self.stA = stA
        self.stB = binding.KVState(stA.k_pages, stA.v_pages, stA.block_table, self.len[1], self.len[2], self.len[3],
                                   self.h[1], self.h[2], 0)
        self.pending = i32(batch)
        self.S = i32(batch, N_d)
        self.V1 = i32(batch, self.max_rows)
        self.V2 = i32(batch, self.max_rows)
        mk = lambda tent: binding.Result(i32(batch), i32(batch), tentative=tent, pending=self.pending)
        self.res1 = [mk(self.V1) for _ in range(m1 * m2)]
        self.res2 = [mk(self.V2) for _ in range(m2)]
        self.res3 = mk(None)
        self.h_acc = torch.zeros(batch, dtype=torch.int32).pin_memory()
        self.h_next = torch.zeros(batch, dtype=torch.int32).pin_memory()
        self.h_V2 = torch.zeros((batch, self.max_rows), dtype=torch.int32).pin_memory()
        self.tokens: List[List[int]] = [[] for _ in range(batch)]
        self.stats = LoopStats()

    def close(self):
        self.A.close(); self.Bc.close()

    def status(self) -> int:
        return self.A.status() | self.Bc.status()

    def prefill(self, prompts: List[List[int]]):
        B = self.B
        mx = max(len(p) for p in prompts)
        toks = torch.zeros((B, mx), dtype=torch.int32)
        for b, p in enumerate(prompts):
            toks[b, : len(p)] = torch.tensor(p, dtype=torch.int32)
        n = torch.tensor([len(p) for p in prompts], dtype=torch.int32).cuda()
        # view B's prefill runs the prompt through all layers [0, e3) and sets its three counters; group 0 follows
        self.Bc.prefill(self.stB, toks.cuda(), n, self.pending)
        self.len[0].copy_(self.len[1])
        torch.cuda.synchronize()
        first = self.pending.cpu().tolist()
        for b in range(B):
            self.tokens[b] = [first[b]]
        return first

    def enqueue_super_round(self, stream=None):
        A, Bc, N_d = self.A, self.Bc, self.N_d
        s = stream if stream is not None else torch.cuda.current_stream()
        r1 = 0
        for i2 in range(self.m2):
            for i1 in range(self.m1):
                A.draft_block(self.stA, self.pending, self.S, N_d, bonus=True, stream=stream)
                A.verify_intermediate(self.stA, self.S, None, None, self.res1[r1], stream=stream, k=N_d)
                r1 += 1
                self.stats.draft_steps += N_d + 1
                self.stats.inter_calls += 1
            # second verifier: LeadingSubstringVerify(V1, e2, .) on the rows level 1 has buffered
            Bc.verify_intermediate(self.stB, self.V1, None, None, self.res2[i2], stream=stream, k=self.max_rows - 1)
            with torch.cuda.stream(s):
                self.len[0].copy_(self.len[1])
            self.stats.inter_calls += 1
        Bc.verify_target(self.stB, self.V2, None, None, self.res3, stream=stream, k=self.max_rows - 1)
        with torch.cuda.stream(s):
            self.len[0].copy_(self.len[1])
        self.stats.target_calls += 1
        self.stats.super_rounds += 1

    def collect(self, stream=None):
        s = stream if stream is not None else torch.cuda.current_stream()
        with torch.cuda.stream(s):
            self.h_acc.copy_(self.res3.n_accepted, non_blocking=True)
            self.h_next.copy_(self.res3.next_token, non_blocking=True)
            self.h_V2.copy_(self.V2, non_blocking=True)
        s.synchronize()
        new = []
        for b in range(self.B):
            a, nxt = int(self.h_acc[b]), int(self.h_next[b])
            F = self.h_V2[b, :a].tolist() + ([nxt] if nxt >= 0 else [])
            self.tokens[b] += F
            new.append(F)
            self.stats.target_accepted += a
            self.stats.committed += len(F)
        return new

    def generate(self, n_gen: int) -> List[List[int]]:
        while min(len(t) for t in self.tokens) < n_gen:
            self.enqueue_super_round()
            self.collect()
        return [t[:n_gen] for t in self.tokens]


class SelfSpecLoop:
    """Algorithm 1 (single-stage self-speculation): N_d (+1) draft steps at L_d, then one verification of the
    block by the final layer -- hispec_verify_intermediate over [L_d, L_f) with the L_f exit."""

    def __init__(self, ctx: binding.Context, st: binding.KVState, batch: int, N_d: int, device: str = "cuda"):
        assert N_d + 1 <= ctx.max_rows
        self.ctx, self.st, self.B, self.N_d = ctx, st, batch, N_d
        i32 = lambda *s: torch.zeros(s, dtype=torch.int32, device=device)
        self.pending, self.S = i32(batch), i32(batch, N_d)
        self.res = binding.Result(i32(batch), i32(batch))
        self.res.pending = self.pending
        self.h = torch.zeros((2, batch), dtype=torch.int32).pin_memory()
        self.h_S = torch.zeros((batch, N_d), dtype=torch.int32).pin_memory()
        self.tokens: List[List[int]] = [[] for _ in range(batch)]

    def prefill(self, prompts: List[List[int]]):
        B = self.B
        mx = max(len(p) for p in prompts)
        toks = torch.zeros((B, mx), dtype=torch.int32)
        for b, p in enumerate(prompts):
            toks[b, : len(p)] = torch.tensor(p, dtype=torch.int32)
        n = torch.tensor([len(p) for p in prompts], dtype=torch.int32)
        self.ctx.prefill(self.st, toks.cuda(), n.cuda(), self.pending)
        torch.cuda.synchronize()
        self.tokens = [[t] for t in self.pending.cpu().tolist()]

    def enqueue_round(self, stream=None):
        ctx, st, N_d, B = self.ctx, self.st, self.N_d, self.B
        S_ptr = self.S.data_ptr()
        for j in range(N_d):
            if j == 0:
                ctx.draft(st, self.pending, S_ptr, batch=B, in_stride=1, out_stride=N_d, stream=stream)
            else:
                ctx.draft(st, S_ptr + 4 * (j - 1), S_ptr + 4 * j, batch=B, in_stride=N_d, out_stride=N_d, stream=stream)
        ctx.draft(st, S_ptr + 4 * (N_d - 1), None, batch=B, in_stride=N_d, stream=stream)
        ctx.verify_intermediate(st, self.S, None, None, self.res, layer_end=ctx.exits.L_f, stream=stream, k=N_d)

    def collect(self):
        self.h[0].copy_(self.res.n_accepted, non_blocking=True)
        self.h[1].copy_(self.res.next_token, non_blocking=True)
        self.h_S.copy_(self.S, non_blocking=True)
        torch.cuda.synchronize()
        for b in range(self.B):
            a, nxt = int(self.h[0, b]), int(self.h[1, b])
            self.tokens[b] += self.h_S[b, :a].tolist() + ([nxt] if nxt >= 0 else [])

    def generate(self, n_gen: int) -> List[List[int]]:
        while min(len(t) for t in self.tokens) < n_gen:
            self.enqueue_round()
            self.collect()
        return [t[:n_gen] for t in self.tokens]


class ARLoop:
    """Vanilla auto-regressive decoding: hispec_draft over [0, L_f) with the L_f exit, one row per step."""

    def __init__(self, ctx: binding.Context, st: binding.KVState, batch: int, device: str = "cuda"):
        self.ctx, self.st, self.B = ctx, st, batch
        self.buf = [torch.zeros(batch, dtype=torch.int32, device=device) for _ in range(2)]
        self.tokens: List[List[int]] = [[] for _ in range(batch)]

    def prefill(self, prompts: List[List[int]]):
        B = self.B
        mx = max(len(p) for p in prompts)
        toks = torch.zeros((B, mx), dtype=torch.int32)
        for b, p in enumerate(prompts):
            toks[b, : len(p)] = torch.tensor(p, dtype=torch.int32)
        n = torch.tensor([len(p) for p in prompts], dtype=torch.int32)
        self.ctx.prefill(self.st, toks.cuda(), n.cuda(), self.buf[0])
        torch.cuda.synchronize()
        first = self.buf[0].cpu().tolist()
        self.tokens = [[t] for t in first]
        return first

    def generate(self, n_gen: int, stream=None) -> List[List[int]]:
        hist = [self.buf[0].clone()]
        cur = 0
        for _ in range(n_gen - 1):
            self.ctx.draft(self.st, self.buf[cur], self.buf[1 - cur], layer_end=self.ctx.exits.L_f, stream=stream)
            cur = 1 - cur
            hist.append(self.buf[cur].clone())
        torch.cuda.synchronize()
        allt = torch.stack(hist, 1).cpu().tolist()
        self.tokens = [list(t) for t in allt]
        return self.tokens
