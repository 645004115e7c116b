"""Glue shared by the tests: builds oracle objects from generated workloads."""
from __future__ import annotations

import dataclasses

import numpy as np
import torch

from oracle.hispec import HiSpecOracle, OracleModel
from paper_2510_01336_b200 import workload as wl

SMALL = dataclasses.replace(wl.TINY, name="small", n_layers=4, d_model=64, n_q_heads=4, n_kv_heads=2,
                            head_dim=16, d_ffn=80, vocab=257, L_d=1, L_i=2, L_f=4, seed=5)


def oracle_for(shape, *, dtype=torch.bfloat16, kv_round=False, layers=None, weights=None, **kw):
    w = weights if weights is not None else wl.make_weights(shape, layers=layers, dtype=dtype, **kw)
    m = OracleModel.from_weights(w, kv_round_bf16=kv_round)
    return w, m, HiSpecOracle(m, shape.L_d, shape.L_i, shape.L_f)


def margin_ok(top2_row, thr=0.1):
    return float(top2_row[0] - top2_row[1]) >= thr
