"""Float64 restatement of the early-exit decoder built from PyTorch *library*
routines (rms_norm, scaled_dot_product_attention, silu, matmul, complex
multiplication for the rotary embedding).  It exists only to pin the C oracle:
it is batched over all positions at once and formulated differently (complex
RoPE, library attention with a boolean causal mask, repeat_interleave for the
grouped KV heads), so a dropped term, wrong sign, transposed operand or wrong
head mapping in the oracle shows up as a disagreement."""
from __future__ import annotations

import torch
import torch.nn.functional as F


def exit_logits_all_positions(w, tokens, L: int) -> tuple:
    """Returns (hidden [P][d], logits [P][vocab]) at exit L for every position, float64."""
    s = w.shape
    f64 = lambda t: t.to(torch.float64)
    x = f64(w.tok_emb)[torch.as_tensor(tokens, dtype=torch.long)]  # [P][d]
    P = x.shape[0]
    hq, hkv, hd = s.n_q_heads, s.n_kv_heads, s.head_dim
    half = hd // 2
    inv_freq = torch.tensor(s.rope_base, dtype=torch.float64) ** (-torch.arange(half, dtype=torch.float64) * 2.0 / hd)
    ang = torch.arange(P, dtype=torch.float64)[:, None] * inv_freq[None, :]
    rot = torch.polar(torch.ones_like(ang), ang)  # e^{i pos theta}, [P][half]

    def rope(t):  # t: [P][h][hd]; pair (i, i+half) is one complex number
        c = torch.complex(t[..., :half], t[..., half:]) * rot[:, None, :]
        return torch.cat([c.real, c.imag], dim=-1)

    causal = torch.ones(P, P, dtype=torch.bool).tril()
    for l in range(L):
        a = F.rms_norm(x, (s.d_model,), f64(w.attn_norm[l]), s.rms_eps)
        qkv = a @ f64(w.wqkv[l]).T
        q = rope(qkv[:, : hq * hd].reshape(P, hq, hd))
        k = rope(qkv[:, hq * hd: (hq + hkv) * hd].reshape(P, hkv, hd))
        v = qkv[:, (hq + hkv) * hd:].reshape(P, hkv, hd)
        k = k.repeat_interleave(hq // hkv, dim=1)
        v = v.repeat_interleave(hq // hkv, dim=1)
        o = F.scaled_dot_product_attention(q.transpose(0, 1)[None], k.transpose(0, 1)[None],
                                           v.transpose(0, 1)[None], attn_mask=causal)[0]
        x = x + o.transpose(0, 1).reshape(P, hq * hd) @ f64(w.wo[l]).T
        m = F.rms_norm(x, (s.d_model,), f64(w.ffn_norm[l]), s.rms_eps)
        gu = m @ f64(w.wgu[l]).T
        x = x + (F.silu(gu[:, : s.d_ffn]) * gu[:, s.d_ffn:]) @ f64(w.wdown[l]).T
    z = F.rms_norm(x, (s.d_model,), f64(w.final_norm), s.rms_eps) @ f64(w.head).T
    return x, z
