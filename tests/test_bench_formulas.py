"""bench.py's algorithmic byte and flop counts against the sizes the workloads fix (no GPU):
the numbers every roofline fraction is a quotient of."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2402_09398_b200 import workloads as wl  # noqa: E402


def test_feature_map_bytes_are_the_weights_once_per_head_plus_rows():
    w = wl.CONFIGS[2]
    per_head = 2 * (128 * 512 + 512 * 8) * 2 + 8 * 8 * 2           # W1, W2 of phi and psi, W3 of psi, fp16
    assert per_head == 278_656                                       # Eq. 1, Eq. 2 with D = 128, R' = 512, R = 8
    assert bench.feature_map_bytes(w) == 1024 * per_head + 1024 * (2 * 256 + 2 * 32)
    w4 = wl.CONFIGS[4]
    assert bench.feature_map_bytes(w4) == 1600 * (2 * (128 * 512 + 512 * 16) * 2 + 16 * 16 * 2) + 6400 * (512 + 128)
    assert bench.feature_map_bytes(w, no_state=True) == 0


def test_step_bytes_of_the_batch_one_workload():
    w = wl.CONFIGS[2]
    n = 204
    per_instance = (n * (512 + 8 + 4)            # K and V rows, score read + write, position
                    + 3 * 256 + 512              # q, k, v in; fp32 out
                    + 2 * 256 + 8 + 4            # the new pair into its slot, its position and score, the count
                    + 8 * 128 * 4 + 32           # H, z read
                    + 2 * 32 + 32                # phi, psi read; psi into the slot's cache
                    + 8 * 128 * 4 + 32 + 32 + 256)   # H, z written; the victim's psi and v row
    assert bench.decode_bytes(w, n) == 1024 * per_instance
    assert bench.feature_map_bytes(w) + bench.decode_bytes(w, n) == 406_089_728
    assert bench.decode_bytes(w, n, out_bytes=2) == 1024 * (per_instance - 256)
    # the narrow roofline: kept K / V, accumulated scores and the low-rank state, read and written
    assert bench.kv_state_scores_bytes(w, n) == 1024 * (n * (512 + 8) + 2 * 8 * 128 * 4)
    assert bench.kv_state_scores_bytes(w, n, no_state=True) == 1024 * n * 520


def test_grouped_heads_share_the_slot_rows():
    w = wl.CONFIGS[3]
    g = w.with_(heads=w.heads // 8, group=8)
    n = 204
    assert g.instances * 8 == w.instances
    kv = lambda x: x.instances * n * 512
    assert kv(g) * 8 == kv(w)
    assert bench.decode_bytes(g, n) < bench.decode_bytes(w, n) / 4
    # phi per query head, psi per KV head
    assert bench.feature_map_bytes(g) - g.instances * (9 * 256 + 9 * 32) == 32 * 4 * (9 * (128 * 512 + 512 * 8) + 64) * 2


def test_prompt_phase_flops():
    w = wl.CONFIGS[5]
    fl = bench.prefill_flops(w)
    S = 32768
    assert fl["rowstat"] == fl["colsum"] == 256 * (S * (S + 1) // 2) * 2 * 128
    assert fl["psi"] == 256 * S * 2 * (128 * 512 + 512 * 16 + 16 * 16)
    assert fl["build"] == 256 * S * 2 * 16 * 128
