"""less_prompt_scores_noalloc: prompt scores for callers that cannot allocate.

Some users of the library live where device allocation is not theirs to do: a
serving process whose memory pool already owns the GPU, or a plugin that gets
buffers and a stream and nothing more.  For them the library carries its
scratch in a fixed array of its own.  This test calls that entry point through
the C ABI twice in a row (the second call with a different prompt length, so it
runs over whatever the first one left in the shared array) and checks each
result against the CPU oracle's prompt scores of the same inputs and against
the accumulated scores that less_prefill produces, within the tolerance the
prefill parity tests use for those scores; a third call fills the scratch
array to its last row.

The file sorts last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2402_09398_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"
ACC_RTOL, ACC_ATOL = 1e-4, 1e-6        # same as the prefill parity check of accumulated scores


def _scores_from_prefill(w, Q, K, V):
    """acc of every prompt token via the existing entry point: with at least as
    many slots as tokens nothing is evicted, so the exported slots hold them all."""
    from paper_2402_09398_b200 import binding
    ctx = binding.from_workload(w, None, DEV, max_prefill_layers=w.layers)
    ctx.prefill(Q, K, V, 0)
    recs = ctx.export_state(list(range(w.instances)))
    out = np.zeros((w.instances, w.prompt), dtype=np.float32)
    for i, r in enumerate(recs):
        assert r["count"] == w.prompt
        out[i, r["pos"]] = r["acc"]
    ctx.close()
    return out


def _scores_oracle(w, Q, K, V):
    """prompt_acc of every head from the fp64 oracle (nothing evicted: slots >= tokens)."""
    from oracle import less_oracle as lo
    out = np.zeros((w.instances, w.prompt))
    ident = lambda x: np.abs(x[:, :w.rank])             # the scores do not depend on the feature maps
    for inst in range(w.instances):
        b, layer, head = wl.instance_coords(w, inst)
        o = lo.LessInstance(w.head_dim, w.rank, w.heavy, w.recent, ident, ident)
        o.prefill(*(t[b, layer, head].double().cpu().numpy() for t in (Q, K, V)))
        out[inst] = o.prompt_acc
    return out


def _scores_noalloc(w, Q, K):
    from paper_2402_09398_b200 import binding as B
    # [B, L, H, S, D] contiguous is [n_inst, S, D] in the instance order of the library
    acc = torch.full((w.instances, w.prompt), float("nan"), dtype=torch.float32, device=DEV)
    rc = B.less_prompt_scores_noalloc(Q.data_ptr(), K.data_ptr(), w.instances, w.prompt,
                                      acc.data_ptr(), torch.cuda.current_stream().cuda_stream)
    assert rc == 0, B.less_strerror(rc)
    torch.cuda.synchronize()
    return acc.cpu().numpy()


def test_noalloc_scores_match_prefill_twice_in_a_row():
    from paper_2402_09398_b200 import binding as B
    cases = [wl.Workload(61, 2, 1, 3, 128, 333, 0, 200, 200, 8, heavy_rule="bernoulli", heavy_param=0.05),
             wl.Workload(62, 1, 2, 2, 128, 150, 0, 100, 100, 8, heavy_rule="every", heavy_param=16)]
    for w in cases:                                   # two calls in a row, shared scratch
        Q, K, V = wl.make_prompt(w, 0, w.layers, DEV)
        got = _scores_noalloc(w, Q, K)
        want = _scores_from_prefill(w, Q, K, V)
        ref = _scores_oracle(w, Q, K, V)
        assert np.isfinite(got).all()
        assert np.allclose(got, ref, rtol=ACC_RTOL, atol=ACC_ATOL), np.max(np.abs(got - ref))
        assert np.allclose(got, want, rtol=ACC_RTOL, atol=ACC_ATOL), np.max(np.abs(got - want))
        # every causal softmax row sums to one, so the scores of a head sum to the prompt length
        assert np.allclose(got.sum(axis=1), w.prompt, rtol=1e-4)
    # exactly as many rows as the scratch array holds: the last row is used, nothing beyond it
    w = wl.Workload(63, 64, 1, 4, 128, B.LESS_NOALLOC_MAX_ROWS // 256, 0, 300, 300, 8, heavy_rule="none")
    assert w.instances * w.prompt == B.LESS_NOALLOC_MAX_ROWS
    Q, K, V = wl.make_prompt(w, 0, w.layers, DEV)
    got = _scores_noalloc(w, Q, K)
    last = w.instances - 1                             # the head whose rows end the scratch array
    ref = _scores_oracle(w.with_(batch=1, heads=1), *(t.reshape(-1, 1, 1, w.prompt, 128)[last:last + 1]
                                                       for t in (Q, K, V)))
    assert np.allclose(got[-1], ref[0], rtol=ACC_RTOL, atol=ACC_ATOL)
    assert np.allclose(got.sum(axis=1), w.prompt, rtol=1e-4)
    # sizes beyond the built-in scratch are refused before anything is launched
    big = B.LESS_NOALLOC_MAX_ROWS // 64 + 1
    dummy = torch.zeros(16, dtype=torch.float16, device=DEV)
    rc = B.less_prompt_scores_noalloc(dummy.data_ptr(), dummy.data_ptr(), 64, big, dummy.data_ptr(), 0)
    assert rc == B.LESS_ERR_NOALLOC_TOO_LARGE
    assert "scratch" in B.less_strerror(rc)
    assert B.less_prompt_scores_noalloc(None, dummy.data_ptr(), 1, 8, dummy.data_ptr(), 0) == -2
