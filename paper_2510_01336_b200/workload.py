"""Seeded synthetic inputs for the HiSpec verification path.

This module only *draws* inputs (weights, token ids, prompt lengths, page
permutations, random KV/hidden state for stand-alone call timing).  It holds
none of the method's arithmetic: no norm, projection, attention, argmax or
acceptance logic lives here, so both the CUDA path and the CPU oracle can be
fed from it without sharing any computation.

The paper evaluates trained early-exit Llama checkpoints on text datasets
(Sec. 4); neither is available offline, so every input is synthetic:
weights i.i.d. N(0, 0.02^2) rounded to bf16, token ids uniform over the
vocabulary, prompt lengths as the workload configuration states.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Sequence, Tuple

import torch


@dataclass(frozen=True)
class ModelShape:
    """Shape of an early-exit decoder (Sec. 3.1: exits L_d < L_i < L_f)."""

    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rope_base: float
    rms_eps: float = 1e-5
    L_d: int = 0
    L_i: int = 0
    L_f: int = 0
    seed: int = 20251001

    @property
    def qkv_rows(self) -> int:
        return (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim

    @property
    def layer_params(self) -> int:
        d, f = self.d_model, self.d_ffn
        return self.qkv_rows * d + d * self.n_q_heads * self.head_dim + 3 * f * d

    @property
    def layer_weight_bytes(self) -> int:
        return 2 * self.layer_params

    @property
    def head_bytes(self) -> int:
        return 2 * self.vocab * self.d_model

    @property
    def kv_bytes_per_token_layer(self) -> int:
        return 2 * 2 * self.n_kv_heads * self.head_dim


TINY = ModelShape("tiny", 4, 256, 4, 4, 64, 688, 4096, 10000.0, L_d=1, L_i=2, L_f=4, seed=20251001)
L3_8B = ModelShape("llama3-8b-shape", 32, 4096, 32, 8, 128, 14336, 128256, 500000.0,
                   L_d=8, L_i=16, L_f=32, seed=20251002)
L2_13B = ModelShape("llama2-13b-shape", 40, 5120, 40, 40, 128, 13824, 32000, 10000.0,
                    L_d=10, L_i=20, L_f=40, seed=20251004)
# The two larger models of the paper's tables, by layer shape (Table 1: CodeLlama-34B with exits 7/12/48,
# Llama-2-70B with exits 10/20/80): GQA 8:1, d 8192.
CL_34B = ModelShape("codellama-34b-shape", 48, 8192, 64, 8, 128, 22016, 32000, 1000000.0,
                    L_d=7, L_i=12, L_f=48, seed=20251006)
L2_70B = ModelShape("llama2-70b-shape", 80, 8192, 64, 8, 128, 28672, 32000, 10000.0,
                    L_d=10, L_i=20, L_f=80, seed=20251007)
# Small odd shapes for tests: GQA 2:1, K/M tails, head_dim 128.
MINI_GQA = ModelShape("mini-gqa", 6, 320, 4, 2, 128, 400, 1000, 10000.0, L_d=2, L_i=3, L_f=6, seed=77)

SHAPES = {s.name: s for s in (TINY, L3_8B, L2_13B, CL_34B, L2_70B, MINI_GQA)}

_KINDS = {"tok_emb": 1, "head": 2, "wqkv": 3, "wo": 4, "wgu": 5, "wdown": 6}


def _gen(seed: int, layer: int, kind: str, device: str) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1000003 + (layer + 1) * 64 + _KINDS[kind]) & 0x7FFFFFFFFFFFFFFF)
    return g


def _normal(shape: Tuple[int, ...], std: float, gen: torch.Generator, device: str,
            dtype: torch.dtype) -> torch.Tensor:
    """N(0, std^2) drawn in fp32 in row chunks (bounded transient memory)."""
    rows = shape[0]
    out = torch.empty(shape, dtype=dtype, device=device)
    chunk = max(1, (1 << 26) // max(1, shape[1]))
    for r0 in range(0, rows, chunk):
        r1 = min(rows, r0 + chunk)
        blk = torch.empty((r1 - r0,) + tuple(shape[1:]), dtype=torch.float32, device=device)
        blk.normal_(0.0, std, generator=gen)
        out[r0:r1] = blk.to(dtype)
    return out


@dataclass
class Weights:
    """Weights of the layers in `layers` plus embedding/head (any may be absent)."""

    shape: ModelShape
    dtype: torch.dtype
    tok_emb: Optional[torch.Tensor]
    head: Optional[torch.Tensor]
    final_norm: torch.Tensor
    wqkv: Dict[int, torch.Tensor] = field(default_factory=dict)
    wo: Dict[int, torch.Tensor] = field(default_factory=dict)
    wgu: Dict[int, torch.Tensor] = field(default_factory=dict)
    wdown: Dict[int, torch.Tensor] = field(default_factory=dict)
    attn_norm: Dict[int, torch.Tensor] = field(default_factory=dict)
    ffn_norm: Dict[int, torch.Tensor] = field(default_factory=dict)

    def layers(self) -> List[int]:
        return sorted(self.wqkv.keys())

    def to(self, device: str) -> "Weights":
        mv = lambda t: None if t is None else t.to(device)
        return Weights(self.shape, self.dtype, mv(self.tok_emb), mv(self.head), mv(self.final_norm),
                       {l: mv(t) for l, t in self.wqkv.items()}, {l: mv(t) for l, t in self.wo.items()},
                       {l: mv(t) for l, t in self.wgu.items()}, {l: mv(t) for l, t in self.wdown.items()},
                       {l: mv(t) for l, t in self.attn_norm.items()},
                       {l: mv(t) for l, t in self.ffn_norm.items()})

    def astype(self, dtype: torch.dtype) -> "Weights":
        """Same values in another storage type (bf16 -> fp32 is exact)."""
        cv = lambda t: None if t is None else t.to(dtype)
        return Weights(self.shape, dtype, cv(self.tok_emb), cv(self.head), self.final_norm,
                       {l: cv(t) for l, t in self.wqkv.items()}, {l: cv(t) for l, t in self.wo.items()},
                       {l: cv(t) for l, t in self.wgu.items()}, {l: cv(t) for l, t in self.wdown.items()},
                       dict(self.attn_norm), dict(self.ffn_norm))


def make_weights(shape: ModelShape, layers: Optional[Sequence[int]] = None, device: str = "cpu",
                 dtype: torch.dtype = torch.bfloat16, with_emb: bool = True, with_head: bool = True,
                 std: float = 0.02, resid_scale: Optional[Dict[int, float]] = None) -> Weights:
    """Every matrix i.i.d. N(0, std^2) from a per-matrix seed; norm gains 1.0.

    Matrices are row-major [out_features][in_features]:
      wqkv  [(hq + 2 hkv) * hd][d]   rows: all q heads, then k heads, then v heads
      wo    [d][hq * hd]
      wgu   [2 * ffn][d]             rows: gate, then up
      wdown [d][ffn]
      head / tok_emb [vocab][d]      (independent draws)
    `resid_scale[l]` multiplies wo and wdown of layer l (an acceptance-shaping
    knob for synthetic weights: small values make deeper exits agree with
    shallower ones); it is applied before rounding to `dtype`.
    A draw depends only on (shape.seed, layer, matrix kind, device type), so a
    subset of layers can be generated alone.
    """
    layers = list(range(shape.n_layers)) if layers is None else list(layers)
    d, f = shape.d_model, shape.d_ffn
    w = Weights(shape, dtype, None, None, torch.ones(d, dtype=torch.float32, device=device))
    if with_emb:
        w.tok_emb = _normal((shape.vocab, d), std, _gen(shape.seed, -1, "tok_emb", device), device, dtype)
    if with_head:
        w.head = _normal((shape.vocab, d), std, _gen(shape.seed, -1, "head", device), device, dtype)
    for l in layers:
        s = 1.0 if not resid_scale else float(resid_scale.get(l, 1.0))
        w.wqkv[l] = _normal((shape.qkv_rows, d), std, _gen(shape.seed, l, "wqkv", device), device, dtype)
        w.wo[l] = _normal((d, shape.n_q_heads * shape.head_dim), std * s,
                          _gen(shape.seed, l, "wo", device), device, dtype)
        w.wgu[l] = _normal((2 * f, d), std, _gen(shape.seed, l, "wgu", device), device, dtype)
        w.wdown[l] = _normal((d, f), std * s, _gen(shape.seed, l, "wdown", device), device, dtype)
        w.attn_norm[l] = torch.ones(d, dtype=torch.float32, device=device)
        w.ffn_norm[l] = torch.ones(d, dtype=torch.float32, device=device)
    return w


def make_tokens(shape: ModelShape, n: int, seed_offset: int = 1000) -> torch.Tensor:
    """`n` token ids i.i.d. uniform over the vocabulary (int32, CPU)."""
    g = torch.Generator().manual_seed(shape.seed + seed_offset)
    return torch.randint(0, shape.vocab, (n,), generator=g, dtype=torch.int64).to(torch.int32)


def make_uniforms(shape: ModelShape, super_round: int, batch: int, rounds: int, n_draft: int, max_rows: int,
                  seed_offset: int = 5000) -> dict:
    """The uniform random numbers one super-round of sampling-based decoding consumes (fp32, CPU, in [0,1)):
    `draft` [rounds][n_draft][batch] (one per sampled draft token), `acc_i` [rounds][batch][max_rows] and
    `smp_i` [rounds][batch] (accept tests and the replacement / bonus draw of each intermediate verification),
    `acc_t` [batch][max_rows] and `smp_t` [batch] (the same for the target verification)."""
    g = torch.Generator().manual_seed(shape.seed + seed_offset + 7919 * super_round)
    r = lambda *sh: torch.rand(sh, generator=g, dtype=torch.float32)
    return {"draft": r(rounds, n_draft, batch), "acc_i": r(rounds, batch, max_rows), "smp_i": r(rounds, batch),
            "acc_t": r(batch, max_rows), "smp_t": r(batch)}


def make_prompt_lengths(shape: ModelShape, batch: int, lo: int, hi: int, seed_offset: int = 2000) -> List[int]:
    """Per-sequence prompt lengths i.i.d. uniform integers in [lo, hi]."""
    g = torch.Generator().manual_seed(shape.seed + seed_offset)
    return torch.randint(lo, hi + 1, (batch,), generator=g).tolist()


def make_block_table(shape: ModelShape, batch: int, pages_per_seq: int, n_pages: Optional[int] = None,
                     seed_offset: int = 3000, permute: bool = True) -> torch.Tensor:
    """Physical page ids [batch][pages_per_seq]: a seeded permutation of the pool."""
    need = batch * pages_per_seq
    n_pages = need if n_pages is None else n_pages
    assert n_pages >= need
    if permute:
        g = torch.Generator().manual_seed(shape.seed + seed_offset)
        perm = torch.randperm(n_pages, generator=g)[:need]
    else:
        perm = torch.arange(need)
    return perm.to(torch.int32).reshape(batch, pages_per_seq).contiguous()


def make_random_state(shape: ModelShape, layers: Sequence[int], ctx: Sequence[int], rows: int,
                      device: str = "cpu", seed_offset: int = 4000,
                      hidden_std: float = 1.0) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """Stand-alone call state: K/V of `layers` for positions < ctx[b] and `rows`
    hidden rows per sequence, all i.i.d. normal (K, V ~ N(0,1) as bf16; hidden
    ~ N(0, hidden_std^2) fp32).  Returns (k, v, hidden) with
    k, v: [len(layers)][batch][max_ctx][hkv][hd] bf16 and hidden: [batch][rows][d].
    Used where a prefill through the oracle would take hours; timing and
    per-call parity do not depend on how the cached state came about.
    """
    g = torch.Generator(device=device).manual_seed(shape.seed + seed_offset)
    b, mc = len(ctx), max(ctx)
    kv_shape = (len(layers), b, mc, shape.n_kv_heads, shape.head_dim)
    k = torch.empty(kv_shape, dtype=torch.bfloat16, device=device)
    v = torch.empty(kv_shape, dtype=torch.bfloat16, device=device)
    for i in range(len(layers)):
        k[i] = torch.randn(kv_shape[1:], generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
        v[i] = torch.randn(kv_shape[1:], generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    h = torch.randn((b, rows, shape.d_model), generator=g, device=device, dtype=torch.float32) * hidden_std
    return k, v, h


def corrupt_drafts(tokens: torch.Tensor, vocab: int, alpha: float, seed: int) -> torch.Tensor:
    """Keep each draft id with probability alpha, else replace it by a different
    uniform id (acceptance-shaped drafts for synthetic weights)."""
    g = torch.Generator().manual_seed(seed)
    keep = torch.rand(tokens.shape, generator=g) < alpha
    shift = torch.randint(1, vocab, tokens.shape, generator=g, dtype=torch.int64)
    alt = ((tokens.to(torch.int64) + shift) % vocab).to(tokens.dtype)
    return torch.where(keep, tokens, alt)
