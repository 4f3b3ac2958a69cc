"""GPU parity at the full benchmark sizes, in the launch configurations bench.py times.

The contexts have the workloads' real shapes (all instances, all slots), so every
kernel runs with the grid, shared memory and tiling of the timed runs; the oracle
checks sampled (batch, layer, head) instances one by one: the prompt phase
(kept set, accumulated scores, cached psi, H, z) and teacher-forced decode steps
(output, feature maps, low-rank terms, eviction decision, score and state updates).
The long-prompt workloads prefill only the layers that hold sampled instances (the
prompt kernels' configuration depends on the layer group, not on how many groups
run); their other layers start empty, which does not change any launch.
"""
import numpy as np
import pytest
import torch

from paper_2402_09398_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _ctx(w, layers_per_call):
    from paper_2402_09398_b200 import binding
    W = wl.make_weights(w, DEV)
    ctx = binding.from_workload(w, W, DEV, max_prefill_layers=layers_per_call)
    return ctx, W


def _sample(w, n):
    """n instances spread over batch, layer and head, first and last included."""
    idx = sorted({int(round(i * (w.instances - 1) / (n - 1))) for i in range(n)}) if n > 1 else [0]
    return idx


def _check_prompt(ctx, w, W, instances):
    import harness
    worst = {}
    for inst in instances:
        b, layer, head = wl.instance_coords(w, inst)
        Q, K, V = wl.make_prompt(w, layer, 1, DEV)
        r = harness.check_prefill(ctx, w, _HeadView(W), Q, K, V, [inst], None, 0, None, layer_begin=layer)
        for k, v in r.items():
            worst[k] = max(worst.get(k, 0), v)
        del Q, K, V
    return worst


class _HeadView(dict):
    """Weights kept on the device; a head's matrices are copied out when asked for."""

    def __init__(self, W):
        super().__init__(W)

    def __getitem__(self, name):
        return _Lazy(dict.__getitem__(self, name))


class _Lazy:
    def __init__(self, t):
        self.t = t

    def __getitem__(self, idx):
        return self.t[idx].cpu()


def _decode_steps(ctx, w, W, instances, steps):
    import harness
    tf = harness.TeacherForced(ctx, w, _HeadView(W), instances)
    for s in range(steps):
        tf.step(*wl.make_decode_inputs(w, s, DEV))
    assert ctx.poll_status() == 0
    assert tf.exempt <= 0.02 * len(instances) * steps + 1
    return tf


@pytest.mark.parametrize("path", ["single_launch", "two_kernels"])
def test_cfg1_smallest_every_instance_every_step(path, monkeypatch):
    w = wl.CONFIGS[1]
    if path == "single_launch":             # what a workload of eight heads runs by default
        monkeypatch.delenv("LESS_SMALL_STEP", raising=False)
    ctx, W = _ctx(w, w.layers)
    Q, K, V = wl.make_prompt(w, 0, w.layers, DEV)
    ctx.prefill(Q, K, V, 0)
    inst = list(range(w.instances))
    print("cfg1 prompt", _check_prompt(ctx, w, W, inst))
    tf = _decode_steps(ctx, w, W, inst, w.steps)
    assert tf.evictions == w.steps * w.instances
    assert ctx.kernel_variant("decode").startswith("small_step_kernel") == (path == "single_launch")
    print("cfg1 decode", path, tf.worst, "exempt", tf.exempt)
    ctx.close()


def test_cfg2_llama7b_shape_sampled_instances():
    w = wl.CONFIGS[2]
    ctx, W = _ctx(w, w.layers)
    Q, K, V = wl.make_prompt(w, 0, w.layers, DEV)
    ctx.prefill(Q, K, V, 0)
    del Q, K, V
    inst = _sample(w, 6)
    print("cfg2 prompt", _check_prompt(ctx, w, W, inst))
    tf = _decode_steps(ctx, w, W, inst, 12)
    assert tf.evictions == 12 * len(inst)
    print("cfg2 decode", tf.worst, "exempt", tf.exempt)
    ctx.close()


def test_cfg3_batched_serving_sampled_instances():
    w = wl.CONFIGS[3]
    per_call = 2
    ctx, W = _ctx(w, per_call)
    for l0 in range(0, w.layers, per_call):
        Q, K, V = wl.make_prompt(w, l0, per_call, DEV)
        ctx.prefill(Q, K, V, l0)
        del Q, K, V
    inst = _sample(w, 6)
    print("cfg3 prompt", _check_prompt(ctx, w, W, inst))
    tf = _decode_steps(ctx, w, W, inst, 4)
    assert tf.evictions == 4 * len(inst)
    print("cfg3 decode", tf.worst, "exempt", tf.exempt)
    ctx.close()
    torch.cuda.empty_cache()


def test_cfg4_long_context_sampled_instances():
    w = wl.CONFIGS[4]
    ctx, W = _ctx(w, 1)
    inst = [wl.instance_index(w, 0, 0, 0), wl.instance_index(w, w.batch - 1, w.layers - 1, w.heads - 1)]
    for layer in (0, w.layers - 1):
        Q, K, V = wl.make_prompt(w, layer, 1, DEV)
        ctx.prefill(Q, K, V, layer)
        del Q, K, V
    print("cfg4 prompt", _check_prompt(ctx, w, W, inst))
    tf = _decode_steps(ctx, w, W, inst, 4)
    assert tf.evictions == 4 * len(inst)
    print("cfg4 decode", tf.worst, "exempt", tf.exempt)
    ctx.close()
    torch.cuda.empty_cache()


def test_cfg5_prefill_compression_one_layer_sampled_instance():
    """Prompt of 32 768 tokens: one whole layer (256 instances) goes through the prompt kernels;
    one instance is checked against the oracle (kept set, scores, cached psi, H, z)."""
    w = wl.CONFIGS[5]
    ctx, W = _ctx(w, 1)
    layer = 3
    Q, K, V = wl.make_prompt(w, layer, 1, DEV)
    ctx.prefill(Q, K, V, layer)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    del Q, K, V
    inst = [wl.instance_index(w, w.batch - 1, layer, 5)]
    r = _check_prompt(ctx, w, W, inst)
    print("cfg5 prompt", r)
    # bookkeeping of every instance of the layer: all slots filled, positions ascending, recent window kept
    some = [wl.instance_index(w, b, layer, h) for b in (0, 3, 7) for h in (0, 17, 31)]
    for rec in ctx.export_state(some):
        assert rec["count"] == w.slots
        pos = rec["pos"].astype(np.int64)
        assert np.all(np.diff(pos) > 0) and np.array_equal(pos[-w.recent:], np.arange(w.prompt - w.recent, w.prompt))
        assert np.isfinite(rec["H"]).all() and rec["z"].min() >= 0
    ctx.close()
    torch.cuda.empty_cache()


def test_maximum_slot_count_one_instance():
    """LESS_MAX_SLOTS = 32 768 slots in one instance: the decode kernel's largest shared-memory
    footprint and longest slot loops, with a prompt just longer than the cache so that the
    prompt selection and every decode step evict."""
    w = wl.Workload(50, 1, 1, 2, 128, 33000, 3, 16384, 16384, 8, heavy_rule="bernoulli", heavy_param=0.01)
    ctx, W = _ctx(w, 1)
    Q, K, V = wl.make_prompt(w, 0, 1, DEV)
    ctx.prefill(Q, K, V, 0)
    inst = [1]
    print("max slots prompt", _check_prompt(ctx, w, W, inst))
    tf = _decode_steps(ctx, w, W, inst, w.steps)
    assert tf.evictions == w.steps
    print("max slots decode", tf.worst)
    ctx.close()
    torch.cuda.empty_cache()


def test_cfg2_grouped_query_heads_sampled_instances():
    """The cfg2 shape with its 32 query heads per layer grouped over 4 KV heads (G = 8), in the
    launch configuration of `bench.py --group 8`: prompt phase and teacher-forced decode steps of
    sampled KV heads against the grouped oracle."""
    import harness
    w = wl.CONFIGS[2]
    w = w.with_(heads=w.heads // 8, group=8)
    ctx, W = _ctx(w, w.layers)
    Q, K, V = wl.make_prompt(w, 0, w.layers, DEV)
    ctx.prefill(Q, K, V, 0)
    assert ctx.poll_status() == 0
    inst = _sample(w, 4)
    Wc = {k: v.cpu() for k, v in W.items()}
    r = harness.check_prefill_group(ctx, w, Wc, Q.cpu(), K.cpu(), V.cpu(), inst)
    print("cfg2 grouped prompt", r)
    del Q, K, V
    tf = harness.GroupTeacherForced(ctx, w, Wc, inst)
    for s in range(8):
        tf.step(*wl.make_decode_inputs(w, s, DEV))
    assert ctx.poll_status() == 0 and tf.evictions == 8 * len(inst) and tf.exempt <= 1
    print("cfg2 grouped decode", tf.worst)
    ctx.close()
    torch.cuda.empty_cache()


def test_parallel_form_training_shape_sampled_instances():
    """The parallel form at the shape `bench.py --masked-form` times (batch 2, 32 heads, sequences
    of 4096, one layer per call): two whole instances against the oracle's S x S matrix."""
    from oracle import less_oracle as lo
    from paper_2402_09398_b200 import binding
    import harness
    S = 4096
    w = wl.CONFIGS[2].with_(batch=2, prompt=S, heavy=204, recent=204)
    W = wl.make_weights(w, DEV)
    ctx = binding.from_workload(w, W, DEV, max_prefill_layers=1, flags=binding.LESS_WITH_PARALLEL_FORM)
    layer = 7
    Q, K, V = wl.make_prompt(w, layer, 1, DEV)
    gen = torch.Generator(device=DEV).manual_seed(99)
    pos = torch.arange(S, device=DEV).expand(w.batch, 1, w.heads, S)
    eu = (pos + w.recent + torch.randint(0, 2 * w.slots, pos.shape, generator=gen, device=DEV)).to(torch.int32)
    # some keys stay for good: the first four (sinks) and a few in every eighth key tile, so that most
    # key tiles are dead (wholly discarded) for the later row blocks and some never are
    eu[:, :, :, :4] = 2**31 - 1
    eu[:, :, :, 1024::1024] = 2**31 - 1
    eu[:, :, :, 1500::1024] = 2**31 - 1
    eu = eu.contiguous()
    out = ctx.masked_attention(Q, K, V, eu, layer_begin=layer)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    for b, head in ((0, 3), (1, 31)):
        wts = [W[n][layer, head].double().cpu().numpy() for n in ("w_phi1", "w_phi2", "w_psi1", "w_psi2", "w_psi3")]
        phi_fn, psi_fn = lo.make_mlp_maps(*wts)
        ref, _ = lo.masked_parallel_attention(*(t[b, 0, head].double().cpu().numpy() for t in (Q, K, V)),
                                              eu[b, 0, head].cpu().numpy(), phi_fn, psi_fn)
        err = float(np.max(np.abs(out[b, 0, head].double().cpu().numpy() - ref)))
        print("parallel form 4096", b, head, err)
        assert err <= harness.OUT_TOL
    ctx.close()
    torch.cuda.empty_cache()


def test_parallel_form_long_sequences_sampled_rows():
    """Sequences of 16 384 (128 key tiles per row block): sampled rows of two instances against the
    oracle's rows, first and last rows and rows on both sides of tile boundaries included."""
    from oracle import less_oracle as lo
    from paper_2402_09398_b200 import binding
    import harness
    S = 16384
    w = wl.CONFIGS[2].with_(batch=1, heads=4, prompt=S, heavy=819, recent=819)
    W = wl.make_weights(w, DEV)
    ctx = binding.from_workload(w, W, DEV, max_prefill_layers=1, flags=binding.LESS_WITH_PARALLEL_FORM)
    layer = 30
    Q, K, V = wl.make_prompt(w, layer, 1, DEV)
    gen = torch.Generator(device=DEV).manual_seed(7)
    pos = torch.arange(S, device=DEV).expand(w.batch, 1, w.heads, S)
    eu = (pos + w.recent + torch.randint(0, 2 * w.slots, pos.shape, generator=gen, device=DEV)).to(torch.int32)
    eu[:, :, :, :4] = 2**31 - 1                          # sinks; every sixteenth key tile keeps two keys for good
    eu[:, :, :, 2048::2048] = 2**31 - 1
    eu[:, :, :, 2100::2048] = 2**31 - 1
    eu = eu.contiguous()
    out = ctx.masked_attention(Q, K, V, eu, layer_begin=layer)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    rows = [0, 1, 127, 128, 129, 4095, 4096, 8191, 12345, S - 129, S - 128, S - 2, S - 1]
    for head in (0, 3):
        wts = [W[n][layer, head].double().cpu().numpy() for n in ("w_phi1", "w_phi2", "w_psi1", "w_psi2", "w_psi3")]
        phi_fn, psi_fn = lo.make_mlp_maps(*wts)
        ref, _ = lo.masked_parallel_attention(*(t[0, 0, head].double().cpu().numpy() for t in (Q, K, V)),
                                              eu[0, 0, head].cpu().numpy(), phi_fn, psi_fn, rows=rows)
        err = float(np.max(np.abs(out[0, 0, head][rows].double().cpu().numpy() - ref)))
        print("parallel form 16384", head, err)
        assert err <= harness.OUT_TOL
    ctx.close()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("cfg,kw", [(2, {}), (4, {}), (3, dict(batch=16)), (3, dict(batch=16, heads=4, group=8))])
def test_back_to_back_steps_at_full_size_equal_serialised_ones(cfg, kw, monkeypatch):
    """24 steps with nothing between them, where a step's feature-map kernel comes up while the step before is
    still finishing, against a context that launches every kernel the ordinary way: every output and the
    sampled final state bit for bit."""
    monkeypatch.setenv("LESS_SMALL_STEP", "0")
    w = wl.CONFIGS[cfg].with_(**kw) if kw else wl.CONFIGS[cfg]
    from paper_2402_09398_b200 import binding
    W = wl.make_weights(w, DEV)
    ctx_o = binding.from_workload(w, W, DEV, max_prefill_layers=4)
    monkeypatch.setenv("LESS_NO_OVERLAP", "1")
    ctx_s = binding.from_workload(w, W, DEV, max_prefill_layers=4)
    monkeypatch.delenv("LESS_NO_OVERLAP")
    for l0 in range(0, w.layers, 4):
        Q, K, V = wl.make_prompt(w, l0, 4, DEV)
        ctx_o.prefill(Q, K, V, l0)
        ctx_s.prefill(Q, K, V, l0)
    del Q, K, V
    steps = 24
    inputs = [wl.make_decode_inputs(w, s, DEV) for s in range(steps)]
    torch.cuda.synchronize()
    outs = []
    for ctx in (ctx_o, ctx_s):
        bufs = [torch.empty(inputs[0][0].shape, dtype=torch.float32, device=DEV) for _ in range(steps)]
        for s in range(steps):
            ctx.decode_step(*inputs[s], out=bufs[s])
        torch.cuda.synchronize()
        assert ctx.poll_status() == 0
        outs.append(bufs)
    for s in range(steps):
        assert torch.equal(outs[0][s], outs[1][s]), s
    inst = list(range(0, w.instances, max(1, w.instances // 64)))
    for a, b in zip(ctx_o.export_state(inst), ctx_s.export_state(inst)):
        for key in ("pos", "acc", "K", "V", "psi", "H", "z"):
            assert np.array_equal(a[key], b[key]), key
    ctx_o.close(); ctx_s.close()

