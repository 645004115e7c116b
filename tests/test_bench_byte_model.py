"""The byte model behind bench.py's roofline figure, against hand arithmetic on the Llama-3-8B layer shape.

Per layer: Wqkv (32 + 2*8)*128 x 4096, Wo 4096 x 4096, Wgu 2*14336 x 4096, Wdown 4096 x 14336 = 218,103,808
bf16 parameters = 436.2 MB; exit head 128256 x 4096 = 1050.7 MB; K + V of one token in one layer
2 * 8 * 128 * 2 B = 4096 B."""
import bench
from paper_2510_01336_b200 import workload as wl


def test_layer_head_and_kv_bytes_of_the_benchmarked_shape():
    s = wl.L3_8B
    params = (32 + 2 * 8) * 128 * 4096 + 4096 * 4096 + 2 * 14336 * 4096 + 4096 * 14336
    assert params == 218_103_808
    assert s.layer_weight_bytes == 2 * params
    assert s.head_bytes == 2 * 128256 * 4096
    assert s.kv_bytes_per_token_layer == 4096


def test_super_round_bytes_are_the_sum_of_its_calls():
    """One super-round = 2 x (6 draft steps + one verify-I of 6 rows) + one verify-T of 12 rows (N_d = 5, two rounds)."""
    s, ctx = wl.L3_8B, 1024
    assert (bench.N_D, bench.ROUNDS) == (5, 2) and (s.L_d, s.L_i, s.L_f) == (8, 16, 32)
    W, H, kv, row = s.layer_weight_bytes, s.head_bytes, 4096, 4096 * 4
    draft = 8 * W + H + 8 * kv * (ctx + 1) + row                     # one row in, KV of ctx + 1 positions touched
    vi = 8 * W + H + 8 * kv * (ctx + 6) + 2 * 6 * row                # six rows read and six written
    vt = 16 * W + H + 16 * kv * (ctx + 12) + 12 * row
    total = 2 * (6 * draft + vi) + vt
    assert bench.algorithmic_bytes_super_round(s, ctx) == total
    # the per-call figures the documentation quotes
    assert abs(vi / 1e9 - 4.57) < 0.01 and abs(draft / 1e9 - 4.57) < 0.01 and abs(vt / 1e9 - 8.10) < 0.01
    # weights dominate: the KV cache and the rows are under 1 % at this context
    assert (total - (2 * (6 * (8 * W + H) + 8 * W + H) + 16 * W + H)) / total < 0.01
