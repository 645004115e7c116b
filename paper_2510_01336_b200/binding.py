"""Thin ctypes binding of libhispec.so (the C ABI declared in include/hispec.h).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  PyTorch supplies device memory and streams.  There is no fallback:
`load()` raises if the library has not been built, and every call raises on a
non-zero return code.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libhispec.so")

FLAG_SIMT_GEMM = 1
FLAG_PLAIN_ACT = 2
FLAG_NO_PDL = 4
FLAG_ROWWARP_ATTN = 8
FLAG_MULTI_KERNEL = 16

ST_BOUNDS, ST_STATE, ST_TIMEOUT = 1, 2, 4

EXPORTS = ["hispec_create", "hispec_destroy", "hispec_draft", "hispec_verify_intermediate", "hispec_verify_target",
           "hispec_prefill", "hispec_device_status", "hispec_launch_count", "hispec_strerror",
           "hispec_profile_enable", "hispec_profile_read", "hispec_last_error", "hispec_exit_argmax_noalloc",
           "hispec_debug_trace", "hispec_accept_rejection", "hispec_sample", "hispec_draft_block"]


class ModelDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab")] + \
               [("rope_base", ctypes.c_float), ("rms_eps", ctypes.c_float)] + \
               [(n, ctypes.c_int32) for n in ("page_size", "max_batch", "max_rows_per_seq", "max_pages_per_seq")] + \
               [("flags", ctypes.c_uint32)]


class CWeights(ctypes.Structure):
    _fields_ = [("tok_emb", ctypes.c_void_p)] + \
               [(n, ctypes.POINTER(ctypes.c_void_p)) for n in ("wqkv", "wo", "wgu", "wdown", "attn_norm", "ffn_norm")] + \
               [("final_norm", ctypes.c_void_p)]


class CExits(ctypes.Structure):
    _fields_ = [("L_d", ctypes.c_int32), ("L_i", ctypes.c_int32), ("L_f", ctypes.c_int32),
                ("head_d", ctypes.c_void_p), ("head_i", ctypes.c_void_p), ("head_f", ctypes.c_void_p)]


class CKv(ctypes.Structure):
    _fields_ = [("k_pages", ctypes.c_void_p), ("v_pages", ctypes.c_void_p), ("block_table", ctypes.c_void_p),
                ("len_draft", ctypes.c_void_p), ("len_inter", ctypes.c_void_p), ("len_target", ctypes.c_void_p),
                ("n_pages", ctypes.c_int64), ("first_layer", ctypes.c_int32), ("n_pool_layers", ctypes.c_int32)]


class CHidden(ctypes.Structure):
    _fields_ = [("h_draft", ctypes.c_void_p), ("h_inter", ctypes.c_void_p)]


class CResult(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("n_accepted", "next_token", "argmax_ids", "top2", "logits", "hidden_out",
                                               "tentative", "pending")] + [("defer_accept", ctypes.c_int32)]


_lib = None


def load() -> ctypes.CDLL:
    """Load libhispec.so; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2510_01336_b200.build` "
                               "(or __graft_entry__.build()) first; there is no non-CUDA path")
        lib = ctypes.CDLL(LIB_PATH)
        vp, i32 = ctypes.c_void_p, ctypes.c_int
        lib.hispec_create.argtypes = [ctypes.POINTER(ModelDesc), ctypes.POINTER(CWeights), ctypes.POINTER(vp)]
        lib.hispec_destroy.argtypes = [vp]
        lib.hispec_draft.argtypes = [vp, vp, i32, i32, ctypes.POINTER(CExits), ctypes.POINTER(CKv),
                                     ctypes.POINTER(CHidden), i32, vp, i32, vp, i32, ctypes.POINTER(CResult)]
        ver = [vp, vp, i32, i32, ctypes.POINTER(CExits), ctypes.POINTER(CKv), ctypes.POINTER(CHidden), i32, vp, i32, vp,
               vp, i32, ctypes.POINTER(CResult)]
        lib.hispec_verify_intermediate.argtypes = ver
        lib.hispec_verify_target.argtypes = ver
        lib.hispec_prefill.argtypes = [vp, vp, ctypes.POINTER(CExits), ctypes.POINTER(CKv), i32, vp, vp, i32, vp]
        lib.hispec_device_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint32)]
        lib.hispec_launch_count.argtypes = [vp]
        lib.hispec_launch_count.restype = ctypes.c_int64
        lib.hispec_strerror.argtypes = [i32]
        lib.hispec_strerror.restype = ctypes.c_char_p
        lib.hispec_profile_enable.argtypes = [vp, i32]
        lib.hispec_profile_read.argtypes = [vp, vp, i32, ctypes.POINTER(ctypes.c_double),
                                            ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_int64)]
        lib.hispec_last_error.restype = ctypes.c_char_p
        lib.hispec_exit_argmax_noalloc.argtypes = [vp, vp, vp, ctypes.c_float, i32, i32, vp, i32, vp, vp]
        lib.hispec_exit_argmax_noalloc.restype = ctypes.c_int
        lib.hispec_accept_rejection.argtypes = [vp, vp, i32, vp, vp, i32, vp, i32, i32, vp, vp, vp, vp, ctypes.c_float, vp, vp]
        lib.hispec_accept_rejection.restype = ctypes.c_int
        lib.hispec_sample.argtypes = [vp, vp, i32, vp, ctypes.c_int64, vp, ctypes.c_float, vp, i32]
        lib.hispec_sample.restype = ctypes.c_int
        lib.hispec_draft_block.argtypes = [vp, vp, i32, i32, ctypes.POINTER(CExits), ctypes.POINTER(CKv), ctypes.POINTER(CHidden),
                                           i32, vp, i32, vp, i32, i32, i32, ctypes.POINTER(CResult)]
        lib.hispec_draft_block.restype = ctypes.c_int
        for name in EXPORTS[:7] + EXPORTS[9:11]:
            getattr(lib, name).restype = ctypes.c_int
        _lib = lib
    return _lib


class HiSpecError(RuntimeError):
    pass


def _check(rc: int, what: str):
    if rc != 0:
        detail = load().hispec_last_error().decode() if rc == -3 else ""
        raise HiSpecError(f"{what}: {load().hispec_strerror(rc).decode()} ({rc}) {detail}")


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None or isinstance(t, int):   # an int is a raw device address (a row inside a larger buffer)
        return t
    assert t.is_cuda and t.is_contiguous()
    return t.data_ptr()


@dataclass
class KVState:
    """Caller-owned device state of a batch: pages, block table, length counters, hidden buffers."""

    k_pages: torch.Tensor      # [pool_layers][n_pages][hkv][page][hd] bf16
    v_pages: torch.Tensor
    block_table: torch.Tensor  # [batch][max_pages_per_seq] int32
    len_draft: torch.Tensor    # [batch] int32
    len_inter: torch.Tensor
    len_target: torch.Tensor
    h_draft: torch.Tensor      # [batch][max_rows][d] fp32
    h_inter: torch.Tensor
    first_layer: int = 0

    def c_kv(self) -> CKv:
        return CKv(_ptr(self.k_pages), _ptr(self.v_pages), _ptr(self.block_table), _ptr(self.len_draft),
                   _ptr(self.len_inter), _ptr(self.len_target), self.k_pages.shape[1], self.first_layer,
                   self.k_pages.shape[0])

    def c_hidden(self) -> CHidden:
        return CHidden(_ptr(self.h_draft), _ptr(self.h_inter))


@dataclass
class Result:
    n_accepted: torch.Tensor
    next_token: torch.Tensor
    argmax_ids: Optional[torch.Tensor] = None
    top2: Optional[torch.Tensor] = None
    logits: Optional[torch.Tensor] = None
    hidden_out: Optional[torch.Tensor] = None
    tentative: Optional[torch.Tensor] = None
    pending: Optional[torch.Tensor] = None
    defer_accept: bool = False

    def c(self) -> CResult:
        return CResult(_ptr(self.n_accepted), _ptr(self.next_token), _ptr(self.argmax_ids), _ptr(self.top2),
                       _ptr(self.logits), _ptr(self.hidden_out), _ptr(self.tentative), _ptr(self.pending),
                       1 if self.defer_accept else 0)


class Context:
    """Owns an hispec_ctx for one model (weights: the workload generator's container, on the GPU)."""

    def __init__(self, shape, weights, *, page_size: int = 16, max_batch: int = 1, max_rows_per_seq: int = 8,
                 max_pages_per_seq: int = 128, flags: int = 0, exits: Optional[Sequence[int]] = None):
        self.lib = load()
        self.shape, self.w = shape, weights
        self.page_size, self.max_batch = page_size, max_batch
        self.max_rows, self.max_pages = max_rows_per_seq, max_pages_per_seq
        L = shape.n_layers
        self._tabs = []

        def table(d):
            arr = (ctypes.c_void_p * L)()
            for l in range(L):
                arr[l] = _ptr(d[l]) if l in d else None
            self._tabs.append(arr)
            return arr

        for t in [weights.tok_emb, weights.final_norm] + list(weights.wqkv.values()):
            assert t is None or t.is_cuda, "weights must live on the GPU"
        self.desc = ModelDesc(L, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.d_ffn,
                              shape.vocab, shape.rope_base, shape.rms_eps, page_size, max_batch, max_rows_per_seq,
                              max_pages_per_seq, flags)
        emb = weights.tok_emb if weights.tok_emb is not None else weights.head
        cw = CWeights(_ptr(emb), table(weights.wqkv), table(weights.wo), table(weights.wgu), table(weights.wdown),
                      table(weights.attn_norm), table(weights.ffn_norm), _ptr(weights.final_norm))
        self.handle = ctypes.c_void_p()
        _check(self.lib.hispec_create(ctypes.byref(self.desc), ctypes.byref(cw), ctypes.byref(self.handle)), "hispec_create")
        ex = exits or (shape.L_d, shape.L_i, shape.L_f)
        self.set_exits(*ex)

    def set_exits(self, L_d: int, L_i: int, L_f: int, head_d=None, head_i=None, head_f=None):
        h = _ptr(self.w.head)
        self.exits = CExits(L_d, L_i, L_f, _ptr(head_d) if head_d is not None else h,
                            _ptr(head_i) if head_i is not None else h, _ptr(head_f) if head_f is not None else h)

    def close(self):
        if getattr(self, "handle", None) and self.handle.value:
            self.lib.hispec_destroy(self.handle)
            self.handle = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ helpers
    def new_state(self, batch: int, n_pages: int, block_table: torch.Tensor, first_layer: int = 0,
                  n_pool_layers: Optional[int] = None, device: str = "cuda") -> KVState:
        s = self.shape
        nl = s.n_layers if n_pool_layers is None else n_pool_layers
        kshape = (nl, n_pages, s.n_kv_heads, self.page_size, s.head_dim)
        z = lambda: torch.zeros(batch, dtype=torch.int32, device=device)
        return KVState(torch.zeros(kshape, dtype=torch.bfloat16, device=device),
                       torch.zeros(kshape, dtype=torch.bfloat16, device=device),
                       block_table.to(device=device, dtype=torch.int32).contiguous(), z(), z(), z(),
                       torch.zeros((batch, self.max_rows, s.d_model), dtype=torch.float32, device=device),
                       torch.zeros((batch, self.max_rows, s.d_model), dtype=torch.float32, device=device), first_layer)

    def new_result(self, batch: int, *, ids: bool = True, logits: bool = False, hidden: bool = False,
                   device: str = "cuda") -> Result:
        s = self.shape
        i = lambda *sh: torch.full(sh, -7, dtype=torch.int32, device=device)
        f = lambda *sh: torch.zeros(sh, dtype=torch.float32, device=device)
        return Result(i(batch), i(batch), i(batch, self.max_rows) if ids else None,
                      f(batch, self.max_rows, 2) if ids else None,
                      f(batch, self.max_rows, s.vocab) if logits else None,
                      f(batch, self.max_rows, s.d_model) if hidden else None)

    @staticmethod
    def _stream(stream) -> int:
        st = stream if stream is not None else torch.cuda.current_stream()
        return st.cuda_stream

    # ------------------------------------------------------------------ the ABI calls
    def draft(self, st: KVState, in_tokens, out_tokens=None, res: Optional[Result] = None,
              layer_end: Optional[int] = None, stream=None, batch: Optional[int] = None, in_stride: int = 1,
              out_stride: int = 1):
        """in_tokens / out_tokens: int32 device tensors, or raw device addresses (int) when a
        column of a [batch][k] block is addressed through the strides."""
        le = self.exits.L_d if layer_end is None else layer_end
        cres = res.c() if res is not None else None
        ip = in_tokens if isinstance(in_tokens, int) else _ptr(in_tokens)
        op = out_tokens if (out_tokens is None or isinstance(out_tokens, int)) else _ptr(out_tokens)
        b = batch if batch is not None else in_tokens.shape[0]
        _check(self.lib.hispec_draft(self.handle, self._stream(stream), 0, le, ctypes.byref(self.exits),
                                     ctypes.byref(st.c_kv()), ctypes.byref(st.c_hidden()), b, ip, in_stride, op,
                                     out_stride, ctypes.byref(cres) if cres else None), "hispec_draft")

    def draft_block(self, st: KVState, in_tokens, block: torch.Tensor, n_steps: int, bonus: bool = True,
                    res: Optional[Result] = None, layer_end: Optional[int] = None, stream=None, in_stride: int = 1):
        """Generate(L_d, ., n_steps) as one call: block [batch][stride >= n_steps] int32 receives the draft tokens."""
        le = self.exits.L_d if layer_end is None else layer_end
        cres = res.c() if res is not None else None
        batch, stride = block.shape
        _check(self.lib.hispec_draft_block(self.handle, self._stream(stream), 0, le, ctypes.byref(self.exits),
                                           ctypes.byref(st.c_kv()), ctypes.byref(st.c_hidden()), batch, _ptr(in_tokens),
                                           in_stride, _ptr(block), stride, n_steps, 1 if bonus else 0,
                                           ctypes.byref(cres) if cres else None), "hispec_draft_block")

    def _verify(self, fn, name, st, l0, l1, draft_tokens, n_draft, n_rows, res, stream, k=None):
        batch, stride = draft_tokens.shape
        k = stride if k is None else k
        _check(fn(self.handle, self._stream(stream), l0, l1, ctypes.byref(self.exits), ctypes.byref(st.c_kv()),
                  ctypes.byref(st.c_hidden()), batch, _ptr(draft_tokens), stride, _ptr(n_draft), _ptr(n_rows), k,
                  ctypes.byref(res.c())), name)

    def verify_intermediate(self, st: KVState, draft_tokens: torch.Tensor, n_draft: Optional[torch.Tensor],
                            n_rows: Optional[torch.Tensor], res: Result, layer_end: Optional[int] = None,
                            stream=None, k: Optional[int] = None):
        """draft_tokens [batch][stride] int32 (k defaults to the stride); n_draft / n_rows None
        = every buffered row."""
        le = self.exits.L_i if layer_end is None else layer_end
        self._verify(self.lib.hispec_verify_intermediate, "hispec_verify_intermediate", st, self.exits.L_d, le,
                     draft_tokens, n_draft, n_rows, res, stream, k)

    def verify_target(self, st: KVState, draft_tokens: torch.Tensor, n_draft: Optional[torch.Tensor],
                      n_rows: Optional[torch.Tensor], res: Result, stream=None, k: Optional[int] = None):
        self._verify(self.lib.hispec_verify_target, "hispec_verify_target", st, self.exits.L_i, self.exits.L_f,
                     draft_tokens, n_draft, n_rows, res, stream, k)

    def accept_rejection(self, stage: int, st: KVState, draft_tokens: torch.Tensor, k: int, p_logits, q_logits,
                         u_accept: torch.Tensor, u_sample: torch.Tensor, res: Result, stage_logits=None,
                         temperature: float = 1.0, stream=None):
        """Rejection-sampling acceptance for a verify call that ran with res.defer_accept (stage 1 =
        intermediate, 2 = target); p_logits / q_logits [batch][max_rows][vocab] fp32 tensors or raw addresses."""
        batch, stride = draft_tokens.shape
        pp = p_logits if isinstance(p_logits, int) else _ptr(p_logits)
        qp = q_logits if isinstance(q_logits, int) else _ptr(q_logits)
        _check(self.lib.hispec_accept_rejection(self.handle, self._stream(stream), stage, ctypes.byref(self.exits),
                                                ctypes.byref(st.c_kv()), batch, _ptr(draft_tokens), stride, k, pp, qp,
                                                _ptr(u_accept), _ptr(u_sample), temperature, _ptr(stage_logits),
                                                ctypes.byref(res.c())), "hispec_accept_rejection")

    def sample(self, logits, row_stride: int, u, out_tokens, batch: int, out_stride: int = 1,
               temperature: float = 1.0, stream=None):
        """One token per sequence from softmax(logits row / temperature) by inversion with u[b]."""
        lp = logits if isinstance(logits, int) else _ptr(logits)
        up = u if isinstance(u, int) else _ptr(u)
        op = out_tokens if isinstance(out_tokens, int) else _ptr(out_tokens)
        _check(self.lib.hispec_sample(self.handle, self._stream(stream), batch, lp, row_stride, up, temperature, op,
                                      out_stride), "hispec_sample")

    def prefill(self, st: KVState, tokens: torch.Tensor, n_tokens: torch.Tensor, first_token: torch.Tensor, stream=None):
        batch, max_tokens = tokens.shape
        _check(self.lib.hispec_prefill(self.handle, self._stream(stream), ctypes.byref(self.exits),
                                       ctypes.byref(st.c_kv()), batch, _ptr(tokens), _ptr(n_tokens), max_tokens,
                                       _ptr(first_token)), "hispec_prefill")

    def status(self, stream=None) -> int:
        out = ctypes.c_uint32(0)
        _check(self.lib.hispec_device_status(self.handle, self._stream(stream), ctypes.byref(out)), "hispec_device_status")
        return int(out.value)

    def profile_enable(self, on: bool):
        _check(self.lib.hispec_profile_enable(self.handle, 1 if on else 0), "hispec_profile_enable")

    def profile_read(self, kind: int, stream=None):
        """(milliseconds, weight bytes, launches) of the bracketed launches of `kind` since the last read."""
        ms, by, n = ctypes.c_double(), ctypes.c_double(), ctypes.c_int64()
        _check(self.lib.hispec_profile_read(self.handle, self._stream(stream), kind, ctypes.byref(ms),
                                            ctypes.byref(by), ctypes.byref(n)), "hispec_profile_read")
        return ms.value, by.value, n.value

    def launch_count(self) -> int:
        return int(self.lib.hispec_launch_count(self.handle))


def exit_argmax_noalloc(head: torch.Tensor, final_norm: torch.Tensor, rms_eps: float, hidden: torch.Tensor,
                        argmax_ids: torch.Tensor, top2: Optional[torch.Tensor] = None, stream=None) -> None:
    """Exit head + greedy token for hidden [n_rows][d] through the allocation-free entry point.
    Outputs are written into the caller's tensors; nothing is allocated here or in the library."""
    n_rows, d = hidden.shape
    st = stream if stream is not None else torch.cuda.current_stream()
    _check(load().hispec_exit_argmax_noalloc(st.cuda_stream, _ptr(head), _ptr(final_norm), float(rms_eps), d,
                                             head.shape[0], _ptr(hidden), n_rows, _ptr(argmax_ids), _ptr(top2)),
           "hispec_exit_argmax_noalloc")
