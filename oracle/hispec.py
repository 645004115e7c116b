"""CPU oracle for HiSpec (hierarchical speculative decoding) -- TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the bench's CPU-baseline leg may import this
module; the product (the CUDA library and its binding) never does, and this
module imports nothing from the product.

What is here, each part written from the paper:

* ``leading_substring_verify`` -- the function of that name in Algorithms 1
  and 2: v_k = argmax p_L(. | x, S_{1:k-1}); k* = first k with S_k != v_k, else
  |S|+1; result [S_{1:k*-1}, v_{k*}].
* ``OracleModel`` -- thin wrapper over the C arithmetic (hispec_oracle.c): one
  partial forward pass of the early-exit decoder and the shared exit head
  (Sec. 3.1).
* ``HiSpecOracle`` -- the three stage calls with the state of Sec. 3.2 (KV cache
  and hidden-state buffers shared by draft, intermediate verifier and target;
  expanded while drafting, pruned back after each verification), the decoding
  loops of Algorithm 1 (self-speculative), Algorithm 2 (HiSpec) and vanilla
  auto-regressive decoding, and a brute-force evaluation that recomputes the
  whole prefix with no cache and no hidden-state reuse.

Pins (see tests/test_oracle_*.py): the integer rule against exhaustive
enumeration; the arithmetic against a float64 restatement built from PyTorch
library routines plus closed forms and invariants; state reuse against the
brute-force recomputation (bit for bit); the composition against the lossless
guarantee (HiSpec output == auto-regressive greedy output from L_f).

Positions are 0-based.  With n committed tokens x_0..x_{n-1}, the three
layer groups A=[0,L_d), B=[L_d,L_i), C=[L_i,L_f) have valid KV length n-1 and
x_{n-1} is *pending* (it has been through no layer yet).
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass, field
from typing import Callable, List, Optional, Sequence, Tuple

import numpy as np

from . import build as _build

_c_float_p = ctypes.POINTER(ctypes.c_float)


class _CModel(ctypes.Structure):
    _fields_ = [
        ("n_layers", ctypes.c_int32), ("d_model", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
        ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("d_ffn", ctypes.c_int32),
        ("vocab", ctypes.c_int32), ("rope_base", ctypes.c_float), ("rms_eps", ctypes.c_float),
        ("weights_bf16", ctypes.c_int32), ("kv_round_bf16", ctypes.c_int32),
        ("tok_emb", ctypes.c_void_p),
        ("wqkv", ctypes.POINTER(ctypes.c_void_p)), ("wo", ctypes.POINTER(ctypes.c_void_p)),
        ("wgu", ctypes.POINTER(ctypes.c_void_p)), ("wdown", ctypes.POINTER(ctypes.c_void_p)),
        ("attn_norm", ctypes.POINTER(ctypes.c_void_p)), ("ffn_norm", ctypes.POINTER(ctypes.c_void_p)),
        ("final_norm", ctypes.c_void_p),
    ]


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_round_bf16.restype = ctypes.c_float
        lib.oracle_round_bf16.argtypes = [ctypes.c_float]
        lib.oracle_rmsnorm.argtypes = [_c_float_p, _c_float_p, ctypes.c_int, ctypes.c_float, _c_float_p]
        lib.oracle_rope.argtypes = [_c_float_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float]
        lib.oracle_embed.argtypes = [ctypes.POINTER(_CModel), ctypes.c_int32, _c_float_p]
        lib.oracle_layer.argtypes = [ctypes.POINTER(_CModel), ctypes.c_int, _c_float_p, ctypes.c_int,
                                     ctypes.c_int64, _c_float_p, _c_float_p]
        lib.oracle_forward.argtypes = [ctypes.POINTER(_CModel), ctypes.c_int, ctypes.c_int, _c_float_p,
                                       ctypes.c_int, ctypes.c_int64, _c_float_p, _c_float_p, ctypes.c_int64]
        lib.oracle_exit_logits.argtypes = [ctypes.POINTER(_CModel), ctypes.c_void_p, _c_float_p, _c_float_p]
        lib.oracle_argmax.restype = ctypes.c_int32
        lib.oracle_argmax.argtypes = [_c_float_p, ctypes.c_int, _c_float_p, _c_float_p]
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _fp(a: np.ndarray):
    assert a.dtype == np.float32 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_c_float_p)


def _as_matrix(t) -> Tuple[np.ndarray, bool]:
    """Accept a numpy fp32 / uint16(bf16 patterns) array or a CPU torch tensor
    (fp32 / bf16).  Returns (contiguous array, is_bf16)."""
    if isinstance(t, np.ndarray):
        a = np.ascontiguousarray(t)
    else:  # torch tensor, imported lazily so numpy-only callers work
        import torch
        t = t.detach().cpu().contiguous()
        if t.dtype == torch.bfloat16:
            a = t.view(torch.int16).numpy().view(np.uint16)
        else:
            a = t.to(torch.float32).numpy()
    if a.dtype == np.uint16:
        return a, True
    assert a.dtype == np.float32, a.dtype
    return a, False


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Element-wise fp32 -> bf16 (nearest even) -> fp32, through the C routine."""
    lib = _load()
    flat = np.ascontiguousarray(x, dtype=np.float32).ravel()
    return np.array([lib.oracle_round_bf16(float(v)) for v in flat], dtype=np.float32).reshape(np.shape(x))


def leading_substring_verify(S: Sequence[int], v: Sequence[int]) -> Tuple[List[int], int]:
    """LeadingSubstringVerify of Algorithms 1 and 2 as a pure integer function.

    S: the block to verify; v: the verifier's greedy tokens, v[k-1] = v_k =
    argmax p_L(. | x, S_{1:k-1}), for k = 1..len(v), len(v) in {|S|, |S|+1}.
    Returns ([S_1..S_{k*-1}, v_{k*}], k*-1): the accepted prefix followed by the
    verifier's token at the first mismatch, and the number of accepted tokens.
    When every S_k matches and v_{|S|+1} was not computed (len(v) == |S|), the
    result is S alone.
    """
    S = [int(t) for t in S]
    v = [int(t) for t in v]
    assert len(v) in (len(S), len(S) + 1)
    k_star = len(S) + 1
    for k in range(1, len(S) + 1):
        if S[k - 1] != v[k - 1]:
            k_star = k
            break
    out = S[: k_star - 1]
    if k_star <= len(v):
        out = out + [v[k_star - 1]]
    return out, k_star - 1


class OracleModel:
    """The early-exit decoder's weights bound to the C arithmetic."""

    def __init__(self, *, n_layers: int, d_model: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                 d_ffn: int, vocab: int, rope_base: float, rms_eps: float, tok_emb, head, final_norm,
                 wqkv: dict, wo: dict, wgu: dict, wdown: dict, attn_norm: dict, ffn_norm: dict,
                 kv_round_bf16: bool):
        self.lib = _load()
        self.n_layers, self.d_model, self.n_q_heads, self.n_kv_heads = n_layers, d_model, n_q_heads, n_kv_heads
        self.head_dim, self.d_ffn, self.vocab = head_dim, d_ffn, vocab
        self.kv_round_bf16 = bool(kv_round_bf16)
        self._keep = []
        kinds = set()

        def mat(t):
            if t is None:
                return None
            a, bf = _as_matrix(t)
            kinds.add(bf)
            self._keep.append(a)
            return a.ctypes.data

        def vec(t):
            a, bf = _as_matrix(t)
            assert not bf
            self._keep.append(a)
            return a.ctypes.data

        arr = lambda: (ctypes.c_void_p * n_layers)()
        self._wqkv, self._wo, self._wgu, self._wdown, self._an, self._fn = (arr() for _ in range(6))
        for l in range(n_layers):
            if l in wqkv:
                self._wqkv[l], self._wo[l] = mat(wqkv[l]), mat(wo[l])
                self._wgu[l], self._wdown[l] = mat(wgu[l]), mat(wdown[l])
                self._an[l], self._fn[l] = vec(attn_norm[l]), vec(ffn_norm[l])
        self.layers_present = sorted(wqkv.keys())
        emb = mat(tok_emb)
        self.head_ptr = mat(head)
        assert len(kinds) == 1, "all matrices must share one storage type"
        self.c = _CModel(n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab,
                         float(rope_base), float(rms_eps), int(kinds.pop()), int(self.kv_round_bf16), emb,
                         self._wqkv, self._wo, self._wgu, self._wdown, self._an, self._fn, vec(final_norm))

    @classmethod
    def from_weights(cls, w, kv_round_bf16: bool) -> "OracleModel":
        """`w`: any object with the attributes of the workload generator's
        weight container (shape, tok_emb, head, final_norm, per-layer dicts)."""
        s = w.shape
        return cls(n_layers=s.n_layers, d_model=s.d_model, n_q_heads=s.n_q_heads, n_kv_heads=s.n_kv_heads,
                   head_dim=s.head_dim, d_ffn=s.d_ffn, vocab=s.vocab, rope_base=s.rope_base, rms_eps=s.rms_eps,
                   tok_emb=w.tok_emb, head=w.head, final_norm=w.final_norm, wqkv=w.wqkv, wo=w.wo, wgu=w.wgu,
                   wdown=w.wdown, attn_norm=w.attn_norm, ffn_norm=w.ffn_norm, kv_round_bf16=kv_round_bf16)

    def embed(self, token: int) -> np.ndarray:
        out = np.empty(self.d_model, dtype=np.float32)
        self.lib.oracle_embed(ctypes.byref(self.c), int(token), _fp(out))
        return out

    def forward(self, l0: int, l1: int, x: np.ndarray, p0: int, cache: "KVCache") -> None:
        """Layers [l0,l1) on rows x[R][d] (in place) at positions p0.., appending K,V."""
        assert x.ndim == 2 and x.shape[1] == self.d_model
        assert all(l in self.layers_present for l in range(l0, l1)), "layer weights missing"
        assert p0 + x.shape[0] <= cache.capacity
        self.lib.oracle_forward(ctypes.byref(self.c), l0, l1, _fp(x), x.shape[0], int(p0), _fp(cache.k),
                                _fp(cache.v), cache.capacity)

    def exit_logits(self, h: np.ndarray) -> np.ndarray:
        """Shared final RMSNorm + shared LM head applied to one hidden row."""
        logits = np.empty(self.vocab, dtype=np.float32)
        self.lib.oracle_exit_logits(ctypes.byref(self.c), self.head_ptr, _fp(np.ascontiguousarray(h)), _fp(logits))
        return logits

    def argmax(self, logits: np.ndarray) -> Tuple[int, float, float]:
        t1, t2 = ctypes.c_float(), ctypes.c_float()
        i = self.lib.oracle_argmax(_fp(logits), logits.shape[0], ctypes.byref(t1), ctypes.byref(t2))
        return int(i), float(t1.value), float(t2.value)

    def new_cache(self, capacity: int) -> "KVCache":
        return KVCache(self.n_layers, capacity, self.n_kv_heads, self.head_dim)


class KVCache:
    """Contiguous per-sequence cache [n_layers][capacity][n_kv_heads][head_dim] fp32.
    (Pages and block tables are a storage matter of the GPU path: attention
    uses a sequence's valid entries only, whatever pages hold them -- Sec. 5.4.)"""

    def __init__(self, n_layers: int, capacity: int, n_kv_heads: int, head_dim: int):
        self.capacity = int(capacity)
        self.k = np.zeros((n_layers, capacity, n_kv_heads, head_dim), dtype=np.float32)
        self.v = np.zeros((n_layers, capacity, n_kv_heads, head_dim), dtype=np.float32)


@dataclass
class SeqState:
    """State of one sequence shared by the three stages (Sec. 3.2)."""

    cache: KVCache
    h_d: np.ndarray  # [rows_cap][d]: exit-L_d hidden rows awaiting intermediate verification
    h_i: np.ndarray  # [rows_cap][d]: exit-L_i hidden rows accumulated for the target
    len_d: int = 0   # valid KV length of layers [0, L_d)
    len_i: int = 0   # ... of [L_d, L_i)
    len_f: int = 0   # ... of [L_i, L_f)


@dataclass
class ExitOut:
    argmax_ids: List[int]
    logits: np.ndarray  # [R][vocab]
    hidden: np.ndarray  # [R][d] residual stream at the exit (before the final norm)
    top2: np.ndarray    # [R][2] largest and second largest logit
    n_accepted: int = 0
    next_token: int = -1


@dataclass
class GenStats:
    draft_steps: int = 0
    inter_calls: int = 0
    target_calls: int = 0
    drafted: int = 0
    inter_accepted: int = 0     # draft tokens accepted by L_i
    target_checked: int = 0     # tokens of V submitted to L_f
    target_accepted: int = 0    # tokens of V accepted by L_f
    flushed: int = 0            # tokens of V discarded after the first L_f mismatch
    committed: int = 0


@dataclass
class AdaptiveSpec:
    """Bounds and thresholds of one adaptive hyper-parameter (App. J)."""
    tau_high: float
    tau_low: float
    n_min: int
    n_max: int


# App. J: N_d follows the acceptance rate of the intermediate verifier (thresholds 0.8 / 0.5, bounds [1, 3]),
# N_i that of the final layer (thresholds 0.8 / 0.3, bounds [3, 8]).
ADAPT_ND_PAPER = AdaptiveSpec(0.8, 0.5, 1, 3)
ADAPT_NI_PAPER = AdaptiveSpec(0.8, 0.3, 3, 8)


def adaptive_step(n: int, alpha: float, spec: AdaptiveSpec) -> int:
    """Next value of N_d (or N_i) given this step's acceptance rate alpha (App. J, the two update equations):
    one more if alpha >= tau_high (capped at n_max), one less if alpha < tau_low (floored at n_min), else unchanged."""
    if alpha >= spec.tau_high:
        return min(spec.n_max, n + 1)
    if alpha < spec.tau_low:
        return max(spec.n_min, n - 1)
    return n


class HiSpecOracle:
    def __init__(self, model: OracleModel, L_d: int, L_i: int, L_f: int):
        assert 0 < L_d < L_i < L_f <= model.n_layers
        self.m, self.L_d, self.L_i, self.L_f = model, L_d, L_i, L_f

    # ------------------------------------------------------------------ state
    def new_state(self, capacity: int, rows_cap: int) -> SeqState:
        d = self.m.d_model
        return SeqState(self.m.new_cache(capacity), np.zeros((rows_cap, d), np.float32),
                        np.zeros((rows_cap, d), np.float32))

    def _exit(self, x: np.ndarray) -> ExitOut:
        R = x.shape[0]
        logits = np.stack([self.m.exit_logits(x[j]) for j in range(R)]) if R else np.zeros((0, self.m.vocab), np.float32)
        ids, top2 = [], np.zeros((R, 2), np.float32)
        for j in range(R):
            i, t1, t2 = self.m.argmax(logits[j])
            ids.append(i)
            top2[j] = (t1, t2)
        return ExitOut(ids, logits, x.copy(), top2)

    # ------------------------------------------------------------ stage calls
    def prefill(self, st: SeqState, tokens: Sequence[int]) -> ExitOut:
        """All prompt tokens through all L_f layers; the greedy token at the last
        prompt position (from the L_f exit) becomes the pending token."""
        assert st.len_d == st.len_i == st.len_f == 0
        x = np.stack([self.m.embed(t) for t in tokens])
        self.m.forward(0, self.L_f, x, 0, st.cache)
        st.len_d = st.len_i = st.len_f = len(tokens)
        return self._exit(x[-1:])

    def draft_step(self, st: SeqState, token: int, layer_end: Optional[int] = None) -> ExitOut:
        """One step of Generate(L_d, ., .): the token at position len_d through
        layers [0, L_d), its exit-L_d hidden row buffered for the intermediate
        verifier, greedy token from the exit head."""
        le = self.L_d if layer_end is None else layer_end
        x = self.m.embed(token)[None, :].copy()
        self.m.forward(0, le, x, st.len_d, st.cache)
        if le == self.L_d:
            st.h_d[st.len_d - st.len_i] = x[0]
        st.len_d += 1
        if le >= self.L_i:
            st.len_i += 1
        if le >= self.L_f:
            st.len_f += 1
        return self._exit(x)

    def _verify(self, st: SeqState, rows: np.ndarray, l0: int, l1: int, p0: int, S: Sequence[int]) -> ExitOut:
        x = rows.copy()
        self.m.forward(l0, l1, x, p0, st.cache)
        out = self._exit(x)
        R = x.shape[0]
        a = 0
        while a < len(S) and a < R and int(S[a]) == out.argmax_ids[a]:
            a += 1
        out.n_accepted = a
        out.next_token = out.argmax_ids[a] if a < R else -1
        return out

    def verify_intermediate(self, st: SeqState, S: Sequence[int], n_rows: int,
                            layer_begin: Optional[int] = None, layer_end: Optional[int] = None) -> ExitOut:
        """LeadingSubstringVerify(S, L_i, .) on the buffered exit-L_d rows: layers
        [L_d, L_i) over n_rows rows (n_rows = |S| or |S|+1), exit-L_i rows appended
        to h_i, then the groups [0,L_d) and [L_d,L_i) pruned to the accepted rows."""
        l0 = self.L_d if layer_begin is None else layer_begin
        l1 = self.L_i if layer_end is None else layer_end
        assert len(S) <= n_rows <= len(S) + 1 and st.len_d - st.len_i >= n_rows
        p0 = st.len_i
        out = self._verify(st, st.h_d[:n_rows], l0, l1, p0, S)
        base = st.len_i - st.len_f
        st.h_i[base: base + n_rows] = out.hidden
        new_len = p0 + min(out.n_accepted + 1, n_rows)
        st.len_d = st.len_i = new_len
        if l1 >= self.L_f:  # Algorithm 1 run through this call: the target is the verifier
            st.len_f = new_len
        return out

    def verify_target(self, st: SeqState, V: Sequence[int], n_rows: int) -> ExitOut:
        """LeadingSubstringVerify(V, L_f, x) on the accumulated exit-L_i rows: layers
        [L_i, L_f); afterwards all three groups are pruned to the accepted rows."""
        assert len(V) <= n_rows <= len(V) + 1 and st.len_i - st.len_f >= n_rows
        p0 = st.len_f
        out = self._verify(st, st.h_i[:n_rows], self.L_i, self.L_f, p0, V)
        st.len_d = st.len_i = st.len_f = p0 + min(out.n_accepted + 1, n_rows)
        return out

    # ------------------------------------------------ brute force (no reuse)
    def brute_force_exit(self, seq_tokens: Sequence[int], L: int, positions: Sequence[int]) -> ExitOut:
        """Exit-L results at `positions` by recomputing layers [0, L) over the
        whole token prefix from the embeddings: no cache, no buffered rows."""
        P = max(positions) + 1
        x = np.stack([self.m.embed(t) for t in seq_tokens[:P]])
        self.m.forward(0, L, x, 0, self.m.new_cache(P))
        return self._exit(x[list(positions)])

    # ------------------------------------------------------------ decoders
    def ar_generate_nocache(self, prompt: Sequence[int], n_gen: int) -> List[int]:
        """Vanilla generation by definition: x_{t+1} = argmax p_{L_f}(. | x_{1:t}),
        a full cache-free forward pass over the whole sequence per token."""
        x = [int(t) for t in prompt]
        for _ in range(n_gen):
            out = self.brute_force_exit(x, self.L_f, [len(x) - 1])
            x.append(out.argmax_ids[0])
        return x[len(prompt):]

    def ar_generate(self, prompt: Sequence[int], n_gen: int) -> List[int]:
        """The same greedy decoding with a KV cache (one row per step through [0, L_f))."""
        st = self.new_state(len(prompt) + n_gen + 1, 1)
        tok = self.prefill(st, prompt).argmax_ids[0]
        out = [tok]
        while len(out) < n_gen:
            tok = self.draft_step(st, tok, layer_end=self.L_f).argmax_ids[0]
            out.append(tok)
        return out[:n_gen]

    def selfspec_generate(self, prompt: Sequence[int], n_gen: int, N_d: int, bonus: bool = True,
                          stats: Optional[GenStats] = None) -> List[int]:
        """Algorithm 1: draft at L_d, verify every block at L_f."""
        stats = stats if stats is not None else GenStats()
        st = self.new_state(len(prompt) + n_gen + N_d + 2, N_d + 1)
        pending = self.prefill(st, prompt).argmax_ids[0]
        x = [pending]
        while len(x) < n_gen:
            S = self._generate(st, pending, N_d, bonus, stats)
            out = self.verify_intermediate(st, S, len(S) + (1 if bonus else 0), self.L_d, self.L_f)
            stats.inter_calls += 1
            F, a = leading_substring_verify(S, out.argmax_ids)
            x += F
            pending = F[-1]
        return x[:n_gen]

    def _generate(self, st: SeqState, pending: int, N_d: int, bonus: bool, stats: GenStats,
                  draft_override: Optional[Callable[[int, int], int]] = None) -> List[int]:
        """Generate(L_d, ., N_d): N_d sequential greedy draft steps; with `bonus`
        one more step pushes S_{N_d} through [0, L_d) so that the verifier can
        compute v_{N_d+1} (its own draft prediction is discarded)."""
        S, u = [], pending
        for j in range(N_d):
            tok = self.draft_step(st, u).argmax_ids[0]
            if draft_override is not None:
                tok = int(draft_override(st.len_d, tok))  # position the token will occupy, greedy draft
            S.append(tok)
            u = tok
            stats.draft_steps += 1
        if bonus:
            self.draft_step(st, u)
            stats.draft_steps += 1
        stats.drafted += N_d
        return S

    def hispec_generate(self, prompt: Sequence[int], n_gen: int, N_d: int, *, N_i: Optional[int] = None,
                        rounds: Optional[int] = None, bonus_inter: bool = True, bonus_target: bool = False,
                        draft_override: Optional[Callable[[int, int], int]] = None, observer=None,
                        stats: Optional[GenStats] = None, rows_cap: Optional[int] = None,
                        adapt_nd: Optional[AdaptiveSpec] = None, adapt_ni: Optional[AdaptiveSpec] = None,
                        schedule: Optional[list] = None) -> List[int]:
        """Algorithm 2.  The inner loop drafts and verifies at L_i until the
        trigger fires -- |V| >= N_i (the paper's dynamic policy, Sec. 3.4) or a
        fixed number of `rounds` -- then L_f verifies V.  Returns the n_gen
        generated tokens (the first is the prefill's greedy token).

        bonus_inter / bonus_target choose whether a stage computes v_{|S|+1}
        (needs the last block token pushed through the shallower layers first).
        `draft_override(position, greedy_token) -> token` replaces draft ids
        (adversarial or acceptance-shaped drafts); the output must not depend on it.
        `observer.before(kind, st, seq_tokens, **kw)` / `.after(kind, st, out)`
        see every stage call (kind in {"draft", "verify_i", "verify_t"}).
        `adapt_nd` / `adapt_ni` (App. J) re-choose N_d after every intermediate verification from its
        acceptance rate (accepted / drafted) and N_i after every target verification from its acceptance rate
        (accepted / |V|); `schedule` collects ("i", N_d, accepted) and ("t", N_i, |V|, accepted) records.
        """
        assert (N_i is None) != (rounds is None)
        assert adapt_ni is None or N_i is not None
        stats = stats if stats is not None else GenStats()
        nd_max = adapt_nd.n_max if adapt_nd else N_d
        ni_max = adapt_ni.n_max if adapt_ni else N_i
        per_round = max(N_d, nd_max) + 1
        cap_rows = rows_cap or ((rounds * per_round if rounds else max(N_i, ni_max) + per_round) + 2)
        st = self.new_state(len(prompt) + n_gen + cap_rows + 2, cap_rows)
        pending = self.prefill(st, prompt).argmax_ids[0]
        x = list(int(t) for t in prompt) + [pending]
        n0 = len(prompt)
        obs_b = (lambda *a, **k: None) if observer is None else observer.before
        obs_a = (lambda *a, **k: None) if observer is None else observer.after
        while len(x) - n0 < n_gen:
            V: List[int] = []
            r = 0
            while (len(V) < N_i) if rounds is None else (r < rounds):
                if observer is not None:
                    S = self._generate_observed(st, pending, N_d, bonus_inter, stats, draft_override, observer, x + V)
                else:
                    S = self._generate(st, pending, N_d, bonus_inter, stats, draft_override)
                R = len(S) + (1 if bonus_inter else 0)
                obs_b("verify_i", st, x + V + S, S=S, n_rows=R)
                out = self.verify_intermediate(st, S, R)
                obs_a("verify_i", st, out)
                stats.inter_calls += 1
                stats.inter_accepted += out.n_accepted
                Vhat, _ = leading_substring_verify(S, out.argmax_ids)
                V += Vhat
                pending = V[-1]
                r += 1
                if schedule is not None:
                    schedule.append(("i", N_d, int(out.n_accepted)))
                if adapt_nd is not None:
                    N_d = adaptive_step(N_d, out.n_accepted / len(S), adapt_nd)
            R = len(V)
            if bonus_target:  # catch V's last token up through [0, L_i) so that L_f can emit a bonus token
                obs_b("draft", st, x + V, token=pending)
                o = self.draft_step(st, pending)
                obs_a("draft", st, o)
                obs_b("verify_i", st, x + V, S=[], n_rows=1)
                o = self.verify_intermediate(st, [], 1)
                obs_a("verify_i", st, o)
                R += 1
            obs_b("verify_t", st, x + V, S=V, n_rows=R)
            out = self.verify_target(st, V, R)
            obs_a("verify_t", st, out)
            stats.target_calls += 1
            stats.target_checked += len(V)
            stats.target_accepted += out.n_accepted
            stats.flushed += len(V) - out.n_accepted
            F, _ = leading_substring_verify(V, out.argmax_ids)
            x += F
            pending = F[-1]
            if schedule is not None:
                schedule.append(("t", N_i, len(V), int(out.n_accepted)))
            if adapt_ni is not None:
                N_i = adaptive_step(N_i, out.n_accepted / len(V), adapt_ni)
        stats.committed = min(len(x) - n0, n_gen)
        return x[n0: n0 + n_gen]

    def hispec_generate_sampling(self, prompt: Sequence[int], n_gen: int, N_d: int, rounds: int,
                                 uniforms: Callable[[int], dict], temperature: float = 1.0, seq: int = 0,
                                 stats: Optional[GenStats] = None) -> List[int]:
        """Algorithm 2 with the rejection-sampling rule of App. G at both verification stages: drafts are
        drawn from p_{L_d}, the intermediate stage filters them into V (distributed as p_{L_i}), the target
        stage filters V (result distributed as p_{L_f}).  Fixed `rounds` per target verification, bonus row at
        the intermediate stage.  `uniforms(super_round)` returns the arrays documented in the workload
        generator (`draft`, `acc_i`, `smp_i`, `acc_t`, `smp_t`); `seq` selects the batch column.  The first
        generated token is the prefill's greedy token."""
        from . import rejection as rj
        stats = stats if stats is not None else GenStats()
        cap_rows = rounds * (N_d + 1) + 2
        st = self.new_state(len(prompt) + n_gen + cap_rows + 2, cap_rows)
        pending = self.prefill(st, prompt).argmax_ids[0]
        x = [int(t) for t in prompt] + [pending]
        n0, sr = len(prompt), 0
        while len(x) - n0 < n_gen:
            U = {k: np.asarray(v) for k, v in uniforms(sr).items()}
            sr += 1
            V: List[int] = []
            PV: List[np.ndarray] = []
            for r in range(rounds):
                S, P_rows, u = [], [], pending
                for j in range(N_d + 1):
                    o = self.draft_step(st, u)
                    stats.draft_steps += 1
                    if j < N_d:
                        p = rj.softmax_f32(o.logits[0], temperature)
                        u = rj.sample_inverse_cdf(p, float(U["draft"][r, j, seq]))
                        S.append(u)
                        P_rows.append(p)
                R = N_d + 1
                p0 = st.len_i
                out = self.verify_intermediate(st, S, R)       # rows, KV, exit rows; its greedy decision is replaced below
                Q = rj.softmax_f32(out.logits[:R], temperature)
                res, a = rj.rejection_verify(S, np.stack(P_rows), Q, U["acc_i"][r, seq], float(U["smp_i"][r, seq]))
                st.len_d = st.len_i = p0 + min(a + 1, R)
                V += res
                PV += [Q[j] for j in range(len(res))]
                pending = res[-1]
                stats.inter_calls += 1
                stats.inter_accepted += a
            R = len(V)
            p0 = st.len_f
            out = self.verify_target(st, V, R)
            Qf = rj.softmax_f32(out.logits[:R], temperature)
            F, a = rj.rejection_verify(V, np.stack(PV), Qf, U["acc_t"][seq], float(U["smp_t"][seq]))
            st.len_d = st.len_i = st.len_f = p0 + min(a + 1, R)
            x += F
            pending = F[-1]
            stats.target_calls += 1
            stats.target_checked += len(V)
            stats.target_accepted += a
        stats.committed = min(len(x) - n0, n_gen)
        return x[n0: n0 + n_gen]

    # ------------------------------------------------ several intermediate verifiers (App. K, future work)
    def chain_generate(self, prompt: Sequence[int], n_gen: int, exits: Sequence[int], N_d: int,
                       rounds: Sequence[int], schedule: Optional[list] = None) -> List[int]:
        """HiSpec with a chain of verifiers L_d = exits[0] < exits[1] < ... < exits[K] = L_f (App. K): level 1
        filters the draft blocks as in Algorithm 2; level l > 1 runs LeadingSubstringVerify on the list that
        level l - 1 has accumulated over rounds[l - 2] of its rounds; the last level is the target.  Every level
        keeps the exit rows of the level below (Sec. 3.2 applied per level) and every verification prunes all
        shallower layer groups.  len(rounds) == K - 1.  Written on the model primitives, with its own state, so
        that it does not lean on the three-exit stage calls; the output must equal greedy decoding from L_f."""
        K = len(exits) - 1
        assert K >= 1 and len(rounds) == K - 1 and list(exits) == sorted(set(exits)) and exits[-1] <= self.m.n_layers
        cap_rows = (N_d + 1) * int(np.prod([max(1, r) for r in rounds]) if rounds else 1) + 2
        cache = self.m.new_cache(len(prompt) + n_gen + 2 * cap_rows + 4)
        d = self.m.d_model
        H = [np.zeros((cap_rows, d), np.float32) for _ in range(K)]     # H[g]: exit rows of level g, relative to lens[g + 1]
        x0 = np.stack([self.m.embed(t) for t in prompt])
        self.m.forward(0, exits[-1], x0, 0, cache)
        lens = [len(prompt)] * (K + 1)                                   # lens[g]: valid KV length of layers [exits[g-1], exits[g])
        pending = self._exit(x0[-1:]).argmax_ids[0]
        x = [int(t) for t in prompt] + [pending]
        n0 = len(prompt)

        def verify(level: int, block: List[int], R: int) -> List[int]:
            p0 = lens[level]
            rows = H[level - 1][:R].copy()
            self.m.forward(exits[level - 1], exits[level], rows, p0, cache)
            if level < K:
                base = lens[level] - lens[level + 1]
                H[level][base: base + R] = rows
            ids = self._exit(rows).argmax_ids
            res, a = leading_substring_verify(block, ids[:R])
            for g in range(level + 1):
                lens[g] = p0 + min(a + 1, R)
            if schedule is not None:
                schedule.append((level, len(block), a))
            return res

        def produce(level: int) -> List[int]:
            """The list tentatively accepted at `level` after rounds[level - 1] of its rounds (level K: one round)."""
            nonlocal pending
            out: List[int] = []
            for _ in range(rounds[level - 1] if level < K else 1):
                if level == 1:
                    S, u = [], pending
                    for j in range(N_d + 1):                 # N_d drafts and the bonus step
                        row = self.m.embed(u)[None, :].copy()
                        self.m.forward(0, exits[0], row, lens[0], cache)
                        H[0][lens[0] - lens[1]] = row[0]
                        lens[0] += 1
                        if j < N_d:
                            u = self._exit(row).argmax_ids[0]
                            S.append(u)
                    res = verify(1, S, N_d + 1)
                else:
                    block = produce(level - 1)
                    res = verify(level, block, len(block))
                out += res
                pending = out[-1]
            return out

        while len(x) - n0 < n_gen:
            F = produce(K)
            x += F
            pending = F[-1]
        return x[n0: n0 + n_gen]

    def _generate_observed(self, st, pending, N_d, bonus, stats, draft_override, observer, ctx_tokens):
        S, u = [], pending
        for j in range(N_d + (1 if bonus else 0)):
            observer.before("draft", st, ctx_tokens + S, token=u)
            o = self.draft_step(st, u)
            observer.after("draft", st, o)
            stats.draft_steps += 1
            if j < N_d:
                tok = o.argmax_ids[0]
                if draft_override is not None:
                    tok = int(draft_override(st.len_d, tok))
                S.append(tok)
                u = tok
        stats.drafted += N_d
        return S
