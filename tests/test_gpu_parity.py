"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle
on the same seeded inputs."""
import os

import numpy as np
import pytest
import torch

from paper_2402_09398_b200 import workloads as wl

pytestmark = pytest.mark.gpu

DEV = "cuda"


def _setup(w, flags=0, psi_scale=None, max_prefill_layers=None, heavy=None, recent=None,
           max_prompt=None):
    from paper_2402_09398_b200 import binding
    W = wl.make_weights(w, DEV)
    ctx = binding.from_workload(w, W, DEV, max_prefill_layers=max_prefill_layers or w.layers,
                                flags=flags, psi_scale=psi_scale, heavy=heavy, recent=recent,
                                max_prompt=max_prompt)
    return ctx, {k: v.cpu() for k, v in W.items()}


def small(cfg_id=71, **kw):
    base = dict(batch=2, layers=2, heads=3, head_dim=128, prompt=300, steps=12, heavy=20, recent=20,
                rank=8, hidden=512, heavy_rule="bernoulli", heavy_param=0.05, weight_std=0.02)
    base.update(kw)
    return wl.Workload(cfg_id, **base)


def _prefill_all(ctx, w, with_out=True, prompt=None):
    Q, K, V = wl.make_prompt(w, 0, w.layers, DEV, prompt=prompt)
    out = torch.empty(Q.shape, dtype=torch.float32, device=DEV) if with_out else None
    ctx.prefill(Q, K, V, 0, attn_out=out)
    torch.cuda.synchronize()
    return Q, K, V, out


@pytest.mark.parametrize("variant", ["base", "rank16", "boosted", "ragged", "sparse_norm", "no_state",
                                     "scaled", "heavy0", "recent1", "hidden256", "long_prompt",
                                     "cuda_core_scoring", "lambda_masking", "lambda_no_state",
                                     "tiny_scalars", "huge_psi", "tova", "tova_no_state"])
def test_prefill_and_teacher_forced_decode(variant, monkeypatch):
    import harness
    flags, psi_scale = 0, None
    w = small()
    if variant == "rank16":
        w = small(72, rank=16, prompt=257)
    elif variant == "boosted":
        w = small(73, weight_std=0.2)           # low-rank mass is a large share of the denominator
    elif variant == "ragged":
        w = small(74, prompt=131, heavy=7, recent=9, batch=3, heads=2)
    elif variant == "sparse_norm":
        w, flags = small(75, weight_std=0.2), 1
    elif variant == "no_state":
        w, flags = small(76), 2
    elif variant == "scaled":
        w = small(77, weight_std=0.1)
        g = torch.Generator().manual_seed(5)
        psi_scale = 0.5 + 2.0 * torch.rand(w.layers, w.heads, 2, generator=g)
    elif variant == "heavy0":
        w = small(78, heavy=0, recent=24)
    elif variant == "recent1":
        w = small(79, heavy=30, recent=1)
    elif variant == "hidden256":
        w = small(80, hidden=256, weight_std=0.05)
    elif variant == "lambda_masking":       # first 4 tokens + sliding window, evicted pairs into H, z
        w, flags = small(58, heavy=4, recent=36, weight_std=0.1), 4
    elif variant == "lambda_no_state":
        w, flags = small(57, heavy=4, recent=21, prompt=211), 4 | 2
    elif variant == "tova":                 # lowest probability of the current query leaves, the new pair included
        w, flags = small(53, weight_std=0.1, steps=16), 8
    elif variant == "tova_no_state":
        w, flags = small(52, prompt=190, heavy=9, recent=8), 8 | 2
    elif variant == "tiny_scalars":         # the paper initialises psi's learnable scalars to 1e-4
        w = small(56, weight_std=0.1)
        psi_scale = torch.full((w.layers, w.heads, 2), 1e-4)
    elif variant == "huge_psi":             # psi of the order of 1e4: the fp16 operands must be rescaled
        w = small(55, weight_std=0.2)
        psi_scale = torch.full((w.layers, w.heads, 2), 40.0)
    elif variant == "long_prompt":          # several streamed 256-row tiles per scoring CTA, rings wrap
        w = small(60, prompt=1100, batch=1, heads=2, steps=4, heavy=50, recent=30)
    elif variant == "cuda_core_scoring":    # the prompt scoring kernels used when no tensor map can be made
        monkeypatch.setenv("LESS_SCORE_KERNEL", "plain")
        w = small(59, prompt=420)
    ctx, W = _setup(w, flags, psi_scale)
    Q, K, V, out = _prefill_all(ctx, w)
    inst = list(range(w.instances))
    summary = harness.check_prefill(ctx, w, W, Q, K, V, inst, out, flags, psi_scale)
    assert ctx.poll_status() == 0
    tf = harness.TeacherForced(ctx, w, W, inst, flags, psi_scale)
    for s in range(w.steps):
        q, k, v = wl.make_decode_inputs(w, s, DEV)
        tf.step(q, k, v)
    assert ctx.poll_status() == 0
    assert tf.evictions == w.steps * w.instances
    assert tf.exempt <= 0.02 * tf.evictions + 1
    if variant in ("boosted", "scaled"):
        assert tf.worst["lr_den"] > 0     # the low-rank path was really exercised and compared
    print(variant, summary, tf.worst, "exempt", tf.exempt)
    ctx.close()


@pytest.mark.parametrize("variant", ["one_row_eight_heads", "rank16_two_rows", "four_rows_hidden256",
                                     "hidden128_scaled", "sparse_norm", "lambda_masking", "tova", "from_empty",
                                     "by_size", "odd_slots", "more_slots_than_staged"])
def test_small_step_single_launch(variant, monkeypatch):
    """The single-launch step for workloads of a few heads (a cluster of CTAs per head computes phi(q_t)
    and psi(k_t), then one CTA per batch row runs Algorithm 1): every step against the oracle, started
    from the library's own pre-step state, with the feature maps compared too."""
    import harness
    monkeypatch.setenv("LESS_SMALL_STEP", "1")
    flags, psi_scale = 0, None
    w = small(40, batch=1, layers=1, heads=8, weight_std=0.1)
    if variant == "rank16_two_rows":
        w = small(41, rank=16, prompt=257, weight_std=0.2)
    elif variant == "four_rows_hidden256":
        w = small(42, batch=4, layers=1, heads=2, hidden=256, weight_std=0.1, prompt=131, heavy=7, recent=9)
    elif variant == "hidden128_scaled":
        w = small(43, batch=3, hidden=128, weight_std=0.2)
        g = torch.Generator().manual_seed(6)
        psi_scale = 0.5 + 2.0 * torch.rand(w.layers, w.heads, 2, generator=g)
    elif variant == "sparse_norm":
        w, flags = small(44, weight_std=0.2), 1
    elif variant == "lambda_masking":
        w, flags = small(45, heavy=4, recent=36, weight_std=0.1), 4
    elif variant == "tova":
        w, flags = small(46, weight_std=0.1, steps=16), 8
    elif variant == "from_empty":
        w = small(47, prompt=0, steps=30, heavy=5, recent=6, weight_std=0.2)
    elif variant == "by_size":              # no switch: few heads go this way by themselves
        monkeypatch.delenv("LESS_SMALL_STEP")
    elif variant == "odd_slots":            # 21 slots: the staged copies' sizes and offsets off the round numbers
        w = small(35, heavy=10, recent=11, weight_std=0.2)
    elif variant == "more_slots_than_staged":   # 170 slots: the K / V rows stream from the arena instead
        w = small(36, heavy=90, recent=80, prompt=400, steps=6, weight_std=0.2)
    ctx, W = _setup(w, flags, psi_scale, max_prompt=max(w.prompt, 16))
    inst = list(range(w.instances))
    if w.prompt:
        Q, K, V, out = _prefill_all(ctx, w)
        harness.check_prefill(ctx, w, W, Q, K, V, inst, out, flags, psi_scale)
    tf = harness.TeacherForced(ctx, w, W, inst, flags, psi_scale)
    for s in range(w.steps):
        tf.step(*wl.make_decode_inputs(w, s, DEV))
    assert ctx.kernel_variant("decode").startswith("small_step_kernel")
    assert ctx.poll_status() == 0
    assert tf.evictions == (w.steps * w.instances if w.prompt else (w.steps - w.slots) * w.instances)
    assert tf.exempt <= 0.02 * tf.evictions + 1
    n0 = ctx.launches
    ctx.decode_step(*wl.make_decode_inputs(w, w.steps, DEV))
    assert ctx.launches - n0 == 1 and ctx.poll_status() == 0  # one kernel per step
    print("small step", variant, tf.worst, "exempt", tf.exempt)
    ctx.close()


def test_small_step_shapes_it_does_not_take_use_the_two_kernels(monkeypatch):
    monkeypatch.setenv("LESS_SMALL_STEP", "1")
    import harness
    for kw, flags in ((dict(batch=5), 0), (dict(group=2), 0), (dict(), 2)):
        w = small(48, steps=3, weight_std=0.1, **kw)
        ctx, W = _setup(w, flags)
        _prefill_all(ctx, w, with_out=False)
        tf = (harness.GroupTeacherForced if w.group > 1 else harness.TeacherForced)(ctx, w, W, [0, w.instances - 1], flags)
        for s in range(w.steps):
            tf.step(*wl.make_decode_inputs(w, s, DEV))
        assert not ctx.kernel_variant("decode").startswith("small_step_kernel") and ctx.poll_status() == 0
        ctx.close()


@pytest.mark.parametrize("pinned", [True, False])
def test_small_step_host_entry_matches_the_device_entry(pinned, monkeypatch):
    """The single-launch step through less_decode_step_host: pinned q, k, v and the output are read /
    written in place by the kernel (asynchronous copies and plain loads over PCIe), pageable ones staged."""
    monkeypatch.setenv("LESS_SMALL_STEP", "1")
    test_host_buffer_entry_matches_device_entry(pinned, 1)


def test_small_step_captured_replays_like_direct_calls(monkeypatch):
    monkeypatch.setenv("LESS_SMALL_STEP", "1")
    test_captured_step_replays_like_direct_calls(3)


def test_short_prompt_fills_without_eviction_then_evicts():
    """prompt_len <= slots: everything is kept; decode appends until full."""
    import harness
    w = small(81, prompt=30, steps=25, heavy=20, recent=20)
    ctx, W = _setup(w)
    Q, K, V, out = _prefill_all(ctx, w)
    inst = list(range(w.instances))
    harness.check_prefill(ctx, w, W, Q, K, V, inst, out)
    tf = harness.TeacherForced(ctx, w, W, inst)
    for s in range(w.steps):
        tf.step(*wl.make_decode_inputs(w, s, DEV))
    # 30 prompt + 25 steps = 55 tokens, 40 slots -> 15 evictions per instance
    assert tf.evictions == 15 * w.instances
    assert ctx.poll_status() == 0
    ctx.close()


def test_decode_from_empty_context_and_reset():
    """No prefill at all: the cache fills from empty; the first output is v itself."""
    import harness
    w = small(82, prompt=0, steps=10, heavy=3, recent=3)
    ctx, W = _setup(w, max_prompt=16)
    inst = list(range(w.instances))
    tf = harness.TeacherForced(ctx, w, W, inst)
    q, k, v = wl.make_decode_inputs(w, 0, DEV)
    out = tf.step(q, k, v)
    assert torch.allclose(out, v.float(), atol=1e-6)      # softmax over one entry
    for s in range(1, w.steps):
        tf.step(*wl.make_decode_inputs(w, s, DEV))
    assert tf.evictions == (w.steps - 6) * w.instances
    ctx.reset()
    assert ctx.position == 0
    rec = ctx.export_state(inst[:2])
    assert rec[0]["count"] == 0 and not rec[0]["H"].any() and not rec[0]["z"].any()
    ctx.close()


def test_layer_groups_and_per_layer_prefill_agree():
    """Prefilling layer by layer, in groups, or all at once gives identical state."""
    w = small(83, layers=3, batch=1, heads=2, prompt=200)
    states = []
    for mode in ("all", "one", "two"):
        ctx, W = _setup(w, max_prefill_layers={"all": 3, "one": 1, "two": 2}[mode])
        if mode == "one":
            for layer in range(w.layers):
                Q, K, V = wl.make_prompt(w, layer, 1, DEV)
                ctx.prefill(Q, K, V, layer)
        else:
            Q, K, V = wl.make_prompt(w, 0, w.layers, DEV)
            ctx.prefill(Q, K, V, 0)
        states.append(ctx.export_state(list(range(w.instances))))
        ctx.close()
    for other in states[1:]:
        for a, b in zip(states[0], other):
            for key in ("pos", "acc", "K", "V", "psi", "H", "z"):
                assert np.array_equal(a[key], b[key]), key


def test_bit_identical_reruns():
    """Same inputs twice -> bit-identical outputs and state (no atomics, no races)."""
    w = small(84, steps=6)
    results = []
    for _ in range(2):
        ctx, W = _setup(w)
        _prefill_all(ctx, w, with_out=False)
        outs = [ctx.decode_step(*wl.make_decode_inputs(w, s, DEV)).cpu() for s in range(w.steps)]
        results.append((outs, ctx.export_state(list(range(w.instances)))))
        ctx.close()
    for a, b in zip(results[0][0], results[1][0]):
        assert torch.equal(a, b)
    for a, b in zip(results[0][1], results[1][1]):
        for key in ("pos", "acc", "K", "V", "psi", "H", "z"):
            assert np.array_equal(a[key], b[key]), key


def test_free_running_state_equals_sum_over_evicted_log():
    """End state after a free run: H, z against the plain sum over the positions the
    library itself evicted (prompt-phase evictions = positions not kept)."""
    import harness
    w = small(85, steps=40, weight_std=0.1)
    ctx, W = _setup(w)
    Q, K, V, _ = _prefill_all(ctx, w, with_out=False)
    inst = list(range(w.instances))
    pre = ctx.export_state(inst)
    evlog = {i: sorted(set(range(w.prompt)) - set(r["pos"].tolist())) for i, r in zip(inst, pre)}
    Kd, Vd = [], []
    ev = torch.empty(w.instances, dtype=torch.int32, device=DEV)
    for s in range(w.steps):
        q, k, v = wl.make_decode_inputs(w, s, DEV)
        ctx.decode_step(q, k, v, evicted_pos=ev)
        Kd.append(k.reshape(-1, w.head_dim).cpu())
        Vd.append(v.reshape(-1, w.head_dim).cpu())
        for i, p in enumerate(ev.cpu().tolist()):
            assert p >= 0
            evlog[i].append(p)
    post = ctx.export_state(inst)
    for i, r in zip(inst, post):
        b, layer, head = wl.instance_coords(w, i)
        Kh = torch.cat([K[b, layer, head].cpu()] + [kd[i][None] for kd in Kd]).double().numpy()
        Vh = torch.cat([V[b, layer, head].cpu()] + [vd[i][None] for vd in Vd]).double().numpy()
        assert len(set(evlog[i])) == len(evlog[i]) == w.prompt + w.steps - w.slots
        H, z = harness.brute_force_state(w, W, i, Kh, Vh, evlog[i])
        assert harness.rel_err(r["H"], H) <= 1e-3 and harness.rel_err(r["z"], z) <= 1e-3
        assert not (set(r["pos"].tolist()) & set(evlog[i]))
    ctx.close()


def test_crafted_tie_evicts_lowest_position():
    """Equal accumulated scores: the lowest position goes (imported state)."""
    w = small(86, batch=1, layers=1, heads=1, prompt=0, heavy=2, recent=2)
    ctx, W = _setup(w, max_prompt=8)
    D, R = w.head_dim, w.rank
    rec = {"count": 4, "t": 10, "pos": np.array([7, 3, 5, 9], dtype=np.int32),
           "acc": np.array([0.5, 0.5, 0.5, 0.1], dtype=np.float32),
           "K": np.zeros((4, D), dtype=np.float16),
           "V": np.arange(4 * D, dtype=np.float16).reshape(4, D) / 64,
           "psi": np.ones((4, R), dtype=np.float32), "H": np.zeros((R, D), dtype=np.float32),
           "z": np.zeros(R, dtype=np.float32)}
    ctx.import_state([0], [rec])
    assert ctx.position == 10
    z = torch.zeros(1, 1, 1, D, dtype=torch.float16, device=DEV)
    ev = torch.empty(1, dtype=torch.int32, device=DEV)
    ctx.decode_step(z, z, z + 1, evicted_pos=ev)
    assert int(ev.item()) == 3        # candidates pos <= 8: {7,3,5}, all tied -> lowest position
    post = ctx.export_state([0])[0]
    assert sorted(post["pos"].tolist()) == [5, 7, 9, 10]
    assert np.allclose(post["H"], np.outer(np.ones(R), rec["V"][1].astype(np.float32)))
    assert np.allclose(post["z"], 1.0)
    ctx.close()


def test_host_side_errors_on_gpu_box():
    from paper_2402_09398_b200 import binding as B
    w = small(87)
    ctx, W = _setup(w)
    Q, K, V = wl.make_prompt(w, 0, w.layers, DEV, prompt=w.prompt + 8)
    with pytest.raises(B.LessError) as e:
        ctx.prefill(Q, K, V, 0)
    assert e.value.code == -5                                  # prompt too long
    Q, K, V = wl.make_prompt(w, 0, w.layers, DEV)
    with pytest.raises(B.LessError) as e:
        ctx.prefill(Q, K, V, 1)
    assert e.value.code == -6                                  # layer range
    q, k, v = wl.make_decode_inputs(w, 0, DEV)
    rc = B.less_decode_step(ctx.ctx, q.data_ptr() + 2, k.data_ptr(), v.data_ptr(),
                            torch.empty(q.shape, device=DEV).data_ptr(), None, 0)
    assert rc == -3                                            # misaligned
    rc = B.less_decode_step(ctx.ctx, None, k.data_ptr(), v.data_ptr(), q.data_ptr(), None, 0)
    assert rc == -2
    assert ctx.poll_status() == 0
    ctx.close()


@pytest.mark.parametrize("batch,rank,hidden", [(1, 8, 512), (5, 16, 512), (17, 8, 256), (40, 16, 128),
                                               (64, 8, 512), (130, 16, 512)])
def test_feature_maps_over_batch_sizes(batch, rank, hidden):
    """phi(q_t), psi(k_t) and the step built on them for token tiles of every padded
    width (16, 32, 64, 128 tokens, and more than one tile)."""
    import harness
    w = small(88 + batch, batch=batch, layers=1, heads=2, prompt=40, steps=3, heavy=8, recent=8,
              rank=rank, hidden=hidden, weight_std=0.1)
    g = torch.Generator().manual_seed(batch)
    psi_scale = 0.5 + torch.rand(w.layers, w.heads, 2, generator=g)
    ctx, W = _setup(w, 0, psi_scale)
    Q, K, V, _ = _prefill_all(ctx, w, with_out=False)
    inst = list(range(w.instances))
    harness.check_prefill(ctx, w, W, Q, K, V, inst, None, 0, psi_scale)
    tf = harness.TeacherForced(ctx, w, W, inst, 0, psi_scale)
    for s in range(w.steps):
        tf.step(*wl.make_decode_inputs(w, s, DEV))
    assert ctx.poll_status() == 0
    assert tf.worst["lr_den"] > 0
    print(batch, rank, hidden, tf.worst)
    ctx.close()


@pytest.mark.parametrize("path", ["gemv", "plain"])
def test_cuda_core_feature_map_kernels(path, monkeypatch):
    """The streaming GEMV and the plain feature-map kernels (hidden widths the tensor-core
    kernel does not take fall back to them) against the oracle."""
    import harness
    monkeypatch.setenv("LESS_FEATURE_KERNEL", path)
    w = small(97, batch=3, layers=2, heads=2, prompt=60, steps=3, heavy=8, recent=8, weight_std=0.1)
    ctx, W = _setup(w)
    _prefill_all(ctx, w, with_out=False)
    tf = harness.TeacherForced(ctx, w, W, list(range(w.instances)))
    for s in range(w.steps):
        tf.step(*wl.make_decode_inputs(w, s, DEV))
    assert ctx.poll_status() == 0
    ctx.close()


@pytest.mark.parametrize("batch,rank", [(1, 8), (3, 16)])
def test_feature_maps_many_heads_per_cta(batch, rank):
    """More (layer, head, map) items than SMs: every persistent CTA of the feature-map kernel
    walks several items, so its rings and double buffers wrap."""
    import harness
    w = small(120 + rank, batch=batch, layers=5, heads=40, prompt=24, steps=2, heavy=6, recent=6,
              rank=rank, weight_std=0.1)
    ctx, W = _setup(w)
    _prefill_all(ctx, w, with_out=False)
    inst = list(range(0, w.instances, 3))
    tf = harness.TeacherForced(ctx, w, W, inst)
    for s in range(w.steps):
        tf.step(*wl.make_decode_inputs(w, s, DEV))
    assert ctx.poll_status() == 0
    ctx.close()


@pytest.mark.parametrize("overlap", [True, False])
def test_decode_many_instances_and_ragged_slots(overlap, monkeypatch):
    """More instances than one wave of CTAs and a slot count that is not a multiple of a row
    group, with the decode kernel launched as a programmatic dependent of the feature-map
    kernel (it overlaps the weight stream and waits for phi, psi on the device) and without."""
    import harness
    if not overlap:
        monkeypatch.setenv("LESS_NO_OVERLAP", "1")
    w = small(99, batch=4, layers=4, heads=25, prompt=150, steps=3, heavy=37, recent=40, weight_std=0.1)
    ctx, W = _setup(w)
    _prefill_all(ctx, w, with_out=False)
    tf = harness.TeacherForced(ctx, w, W, list(range(0, w.instances, 7)))
    for s in range(w.steps):
        tf.step(*wl.make_decode_inputs(w, s, DEV))
    assert ctx.poll_status() == 0
    ctx.close()


@pytest.mark.parametrize("batch,layers,heads,rank,ctas", [(4, 4, 80, 8, 0), (20, 2, 32, 16, 0), (70, 1, 19, 8, 0),
                                                          (20, 2, 32, 8, 16)])
def test_decode_follows_the_feature_kernel_head_by_head(batch, layers, heads, rank, ctas, monkeypatch):
    """More instances than can wait on the GPU at once (> 8 per SM), per-head counters switched on:
    behind the large-batch feature kernel the decode kernel starts as a programmatic dependent and
    every CTA waits only for the counters of its own head's phi and psi, CTAs numbered head-major
    (batches 20 and 70: one and two token tiles; a feature grid cut to 16 CTAs); behind the small-batch
    kernel (batch 4) the step stays serial.  Teacher-forced parity, then free-running steps back to
    back must equal, bit for bit, a context without the overlap."""
    import harness
    monkeypatch.setenv("LESS_HEAD_COUNTERS", "1")
    if ctas:
        monkeypatch.setenv("LESS_FEATURE_CTAS", str(ctas))
    w = small(130 + batch, batch=batch, layers=layers, heads=heads, prompt=40, steps=3, heavy=9, recent=9,
              rank=rank, weight_std=0.1)
    assert w.instances > 8 * 148
    ctx, W = _setup(w)
    assert "tc" in ctx.kernel_variant("feature_map") or ctx.kernel_variant("feature_map") == ""
    _prefill_all(ctx, w, with_out=False)
    tf = harness.TeacherForced(ctx, w, W, list(range(0, w.instances, 97)) + [w.instances - 1])
    for s in range(w.steps):
        tf.step(*wl.make_decode_inputs(w, s, DEV))
    assert ctx.poll_status() == 0
    assert ctx.kernel_variant("feature_map").startswith("feature_tc")
    monkeypatch.setenv("LESS_NO_OVERLAP", "1")
    ref, _ = _setup(w)
    monkeypatch.delenv("LESS_NO_OVERLAP")
    inst = list(range(0, w.instances, 53))
    ref.import_state(inst, ctx.export_state(inst))
    sub = torch.tensor(inst, device=DEV)
    ins = [wl.make_decode_inputs(w, 3 + s, DEV) for s in range(6)]
    outs_a = [ctx.decode_step(*x).clone() for x in ins]          # no synchronisation between the steps
    outs_b = [ref.decode_step(*x).clone() for x in ins]
    for a, b in zip(outs_a, outs_b):
        assert torch.equal(a.reshape(-1, w.head_dim)[sub], b.reshape(-1, w.head_dim)[sub])
    for a, b in zip(ctx.export_state(inst), ref.export_state(inst)):
        for key in ("pos", "acc", "K", "V", "psi", "H", "z"):
            assert np.array_equal(a[key], b[key]), key
    assert ctx.poll_status() == 0 and ref.poll_status() == 0
    ctx.close(); ref.close()


@pytest.mark.parametrize("group", [1, 4])
def test_fp16_output_flag(group):
    """LESS_OUT_F16: the attention output is the fp32 result rounded once to fp16 (tolerance: the
    2e-3 of fp32 outputs plus half an fp16 ulp of the value); cache and state do not depend on it."""
    import harness
    w = small(140 + group, steps=5, weight_std=0.1, group=group)
    ctx16, W = _setup(w, flags=32)
    ctx32, _ = _setup(w)
    for c in (ctx16, ctx32):
        _prefill_all(c, w, with_out=False)
    inst = list(range(w.instances))
    tf = (harness.GroupTeacherForced if group > 1 else harness.TeacherForced)(ctx16, w, W, inst, flags=32)
    for s in range(w.steps):
        q, k, v = wl.make_decode_inputs(w, s, DEV)
        o16 = tf.step(q, k, v)
        o32 = ctx32.decode_step(q, k, v)
        assert o16.dtype == torch.float16 and torch.equal(o16, o32.to(torch.float16))
    for a, b in zip(ctx16.export_state(inst), ctx32.export_state(inst)):
        for key in ("pos", "acc", "K", "V", "psi", "H", "z"):
            assert np.array_equal(a[key], b[key]), key
    # host entry: fp16 output written in place into pinned memory; q and k as one host block
    q, k, v = wl.make_decode_inputs(w, w.steps, DEV)
    ref = ctx32.decode_step(q, k, v).to(torch.float16).cpu()
    qk = torch.empty(q.numel() + k.numel(), dtype=torch.float16).pin_memory()
    hq, hk = qk[:q.numel()].view(q.shape), qk[q.numel():].view(k.shape)
    hq.copy_(q); hk.copy_(k)
    hv = v.cpu().pin_memory()
    hout = torch.zeros(ref.shape, dtype=torch.float16).pin_memory()
    ctx16.decode_step_host(hq, hk, hv, hout)
    assert torch.equal(hout, ref)
    assert ctx16.poll_status() == 0
    ctx16.close(); ctx32.close()


def test_bounded_wait_runs_out_and_the_context_reports_it():
    """A wait that nothing ever satisfies (a barrier without a producer, a limit of a few thousand
    polls) ends by itself: the kernel returns, the status word says which wait gave up, and a fresh
    context on the same GPU works normally afterwards.  Nothing here faults or waits without limit."""
    import harness
    from paper_2402_09398_b200 import binding
    w = small(150, batch=1, layers=1, heads=2, prompt=32, steps=2, heavy=6, recent=6)
    ctx, W = _setup(w)
    assert ctx.poll_status() == 0 and ctx.status_where() == 0
    assert ctx.selftest_wait_timeout(0) == -1 and ctx.selftest_wait_timeout(1 << 21) == -1
    assert ctx.selftest_wait_timeout(3000) == 0
    assert ctx.poll_status() == -7                       # LESS_ERR_DEVICE_TIMEOUT
    assert ctx.status_where() == 90
    assert "wait" in binding.less_strerror(-7)
    assert ctx.selftest_wait_timeout(3000) == 0          # a context that has given up skips the wait
    assert ctx.poll_status() == -7
    ctx.close()
    ctx, W = _setup(w)                                   # the GPU and the library are unaffected
    _prefill_all(ctx, w, with_out=False)
    tf = harness.TeacherForced(ctx, w, W, list(range(w.instances)))
    for s in range(w.steps):
        tf.step(*wl.make_decode_inputs(w, s, DEV))
    assert ctx.poll_status() == 0
    ctx.close()


@pytest.mark.parametrize("pinned,group", [(True, 1), (False, 1), (True, 4), (False, 2)])
def test_host_buffer_entry_matches_device_entry(pinned, group):
    """less_decode_step_host with pinned (read / written in place by the kernel) and pageable
    (staged and copied) host tensors gives bit-identical outputs and state to less_decode_step."""
    w = small(54, steps=5, weight_std=0.1, group=group)
    ctx_d, W = _setup(w)
    ctx_h, _ = _setup(w)
    for ctx in (ctx_d, ctx_h):
        _prefill_all(ctx, w, with_out=False)
    for s in range(w.steps):
        q, k, v = wl.make_decode_inputs(w, s, DEV)
        ref = ctx_d.decode_step(q, k, v).cpu()
        hq, hk, hv = (t.cpu() for t in (q, k, v))
        hout = torch.full(ref.shape, float("nan"), dtype=torch.float32)
        if pinned:
            hq, hk, hv, hout = (t.pin_memory() for t in (hq, hk, hv, hout))
        ctx_h.decode_step_host(hq, hk, hv, hout)
        assert torch.equal(hout, ref)
    inst = list(range(w.instances))
    for a, b in zip(ctx_d.export_state(inst), ctx_h.export_state(inst)):
        for key in ("pos", "acc", "K", "V", "psi", "H", "z"):
            assert np.array_equal(a[key], b[key]), key
    assert ctx_h.poll_status() == 0
    assert ctx_h.kernel_variant("decode").startswith("small_step") == (os.environ.get("LESS_SMALL_STEP") == "1")
    ctx_d.close(); ctx_h.close()


def test_host_entry_in_layer_segments_matches_the_device_entry():
    """A step large enough that the host entry launches it in layer segments (q, k of a segment copied
    on a stream of its own while the segment before computes): outputs and state bit-identical to the
    device entry's single launch, over several steps."""
    w = small(57, batch=16, layers=8, heads=64, prompt=24, steps=4, heavy=6, recent=6, weight_std=0.1)
    assert w.instances * w.head_dim * 2 * 2 >= 4 << 20
    ctx_d, W = _setup(w)
    ctx_h, _ = _setup(w)
    for ctx in (ctx_d, ctx_h):
        _prefill_all(ctx, w, with_out=False)
    for s in range(w.steps):
        q, k, v = wl.make_decode_inputs(w, s, DEV)
        ref = ctx_d.decode_step(q, k, v).cpu()
        hq, hk, hv = (t.cpu().pin_memory() for t in (q, k, v))
        hout = torch.full(ref.shape, float("nan"), dtype=torch.float32).pin_memory()
        ctx_h.decode_step_host(hq, hk, hv, hout)
        assert torch.equal(hout, ref)
    assert ctx_h.position == ctx_d.position
    inst = list(range(0, w.instances, 61))
    for a, b in zip(ctx_d.export_state(inst), ctx_h.export_state(inst)):
        for key in ("pos", "acc", "K", "V", "psi", "H", "z"):
            assert np.array_equal(a[key], b[key]), key
    assert ctx_h.poll_status() == 0
    ctx_d.close(); ctx_h.close()


def test_tova_new_token_can_evict_itself():
    """TOVA: a new key the query points away from has the lowest probability of its own step;
    it is absorbed into H, z at once and no slot changes (imported state)."""
    w = small(51, batch=1, layers=1, heads=1, prompt=0, heavy=2, recent=2, weight_std=0.1)
    ctx, W = _setup(w, flags=8, max_prompt=8)
    D, R = w.head_dim, w.rank
    K = np.zeros((4, D), dtype=np.float16)
    K[np.arange(4), np.arange(4)] = 3.0
    rec = {"count": 4, "t": 10, "pos": np.array([2, 5, 7, 9], dtype=np.int32),
           "acc": np.full(4, 0.25, dtype=np.float32), "K": K,
           "V": np.arange(4 * D, dtype=np.float16).reshape(4, D) / 64,
           "psi": np.ones((4, R), dtype=np.float32), "H": np.zeros((R, D), dtype=np.float32),
           "z": np.zeros(R, dtype=np.float32)}
    ctx.import_state([0], [rec])
    q = torch.ones(1, 1, 1, D, dtype=torch.float16, device=DEV)
    k = torch.full((1, 1, 1, D), -5.0, dtype=torch.float16, device=DEV)
    v = torch.full((1, 1, 1, D), 7.0, dtype=torch.float16, device=DEV)
    ev = torch.empty(1, dtype=torch.int32, device=DEV)
    ctx.decode_step(q, k, v, evicted_pos=ev)
    assert int(ev.item()) == 10                        # the new token's own position
    post = ctx.export_state([0])[0]
    assert post["pos"].tolist() == [2, 5, 7, 9] and post["count"] == 4
    assert np.array_equal(post["K"], K)
    _, psi_k = ctx.read_feature_maps()
    assert np.allclose(post["H"], np.outer(psi_k[0], np.full(D, 7.0)), rtol=1e-6)
    assert np.allclose(post["z"], psi_k[0], rtol=1e-6)
    ctx.close()


@pytest.mark.parametrize("batch", [1, 12])
def test_captured_step_replays_like_direct_calls(batch, group=1):
    """One decode step captured in a CUDA graph (fixed input / output buffers) and replayed: the
    position advances on the device, so every replay is the next step.  Outputs and state must be
    bit-identical to direct calls on a second context."""
    w = small(49, batch=batch, layers=2, heads=2, steps=7, weight_std=0.1, group=group)
    ctx_d, _ = _setup(w)
    ctx_g, _ = _setup(w)
    for ctx in (ctx_d, ctx_g):
        _prefill_all(ctx, w, with_out=False)
    q0, k0, v0 = wl.make_decode_inputs(w, 0, DEV)
    qb, kb, vb = q0.clone(), k0.clone(), v0.clone()
    ob = torch.empty(q0.shape, dtype=torch.float32, device=DEV)
    evb = torch.empty(w.instances, dtype=torch.int32, device=DEV)
    ref0 = ctx_d.decode_step(q0, k0, v0)
    assert torch.equal(ctx_g.decode_step(qb, kb, vb, out=ob, evicted_pos=evb), ref0)   # also the warm-up launch
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        ctx_g.decode_step(qb, kb, vb, out=ob, evicted_pos=evb)
    evd = torch.empty_like(evb)
    for s in range(1, w.steps):
        q, k, v = wl.make_decode_inputs(w, s, DEV)
        qb.copy_(q); kb.copy_(k); vb.copy_(v)
        graph.replay()
        ref = ctx_d.decode_step(q, k, v, evicted_pos=evd)
        assert torch.equal(ob, ref) and torch.equal(evb, evd), s
    assert ctx_g.poll_status() == 0 and ctx_d.poll_status() == 0
    assert ctx_g.position == ctx_d.position == w.prompt + w.steps
    inst = list(range(w.instances))
    for a, b in zip(ctx_d.export_state(inst), ctx_g.export_state(inst)):
        assert a["t"] == b["t"]
        for key in ("pos", "acc", "K", "V", "psi", "H", "z"):
            assert np.array_equal(a[key], b[key]), key
    ctx_d.close(); ctx_g.close()


@pytest.mark.parametrize("small_step", ["0", "1"])
def test_back_to_back_steps_equal_serialised_ones(small_step, monkeypatch):
    """Steps launched back to back, with nothing between them: each step's first kernel may start while the
    step before still runs (programmatic dependent launch).  Outputs of every step and the final state must be
    bit-identical to a context that launches every kernel the ordinary way (LESS_NO_OVERLAP)."""
    monkeypatch.setenv("LESS_SMALL_STEP", small_step)
    w = small(33, batch=2, layers=4, heads=12, steps=24, heavy=12, recent=12, weight_std=0.2)
    ctx_o, _ = _setup(w)
    monkeypatch.setenv("LESS_NO_OVERLAP", "1")
    ctx_s, _ = _setup(w)
    monkeypatch.delenv("LESS_NO_OVERLAP")
    for ctx in (ctx_o, ctx_s):
        _prefill_all(ctx, w, with_out=False)
    inputs = [wl.make_decode_inputs(w, s, DEV) for s in range(w.steps)]
    torch.cuda.synchronize()
    outs = {}
    for name, ctx in (("overlapped", ctx_o), ("serial", ctx_s)):
        bufs = [torch.empty(inputs[0][0].shape, dtype=torch.float32, device=DEV) for _ in range(w.steps)]
        for s in range(w.steps):
            ctx.decode_step(*inputs[s], out=bufs[s])
        torch.cuda.synchronize()
        outs[name] = bufs
        assert ctx.poll_status() == 0
    assert ctx_o.kernel_variant("decode").startswith("small_step") == (small_step == "1")
    for s in range(w.steps):
        assert torch.equal(outs["overlapped"][s], outs["serial"][s]), s
    inst = list(range(w.instances))
    for a, b in zip(ctx_o.export_state(inst), ctx_s.export_state(inst)):
        assert a["t"] == b["t"]
        for key in ("pos", "acc", "K", "V", "psi", "H", "z"):
            assert np.array_equal(a[key], b[key]), key
    ctx_o.close(); ctx_s.close()


def test_captured_step_replays_with_grouped_query_heads():
    test_captured_step_replays_like_direct_calls(3, group=4)


@pytest.mark.parametrize("kernel", ["rows", "mma"])
@pytest.mark.parametrize("group,rank,flags", [(2, 8, 0), (4, 16, 0), (8, 8, 0), (4, 8, 4), (2, 16, 1), (4, 8, 2)])
def test_grouped_query_heads_decode_from_empty(group, rank, flags, kernel, monkeypatch):
    """Section 3.2, multi-query attention: G query heads share one KV head's cache, scores and
    state; every step is checked against the grouped oracle (outputs of all G heads, per-head phi,
    aggregated H2O scores, the one eviction, Eq. 4 / Eq. 5)."""
    import harness
    monkeypatch.setenv("LESS_GROUP_KERNEL", kernel)     # both decode kernels for grouped heads
    w = small(60 + group, prompt=0, steps=30, heavy=9, recent=8, rank=rank, weight_std=0.1, group=group)
    ctx, W = _setup(w, flags=flags, max_prompt=16)
    inst = list(range(w.instances))
    tf = harness.GroupTeacherForced(ctx, w, W, inst, flags)
    for s in range(w.steps):
        q, k, v = wl.make_decode_inputs(w, s, DEV)
        assert q.shape[2] == w.heads * group
        out = tf.step(q, k, v)
        assert out.shape == q.shape
    assert tf.evictions == (w.steps - w.slots) * w.instances
    assert tf.exempt <= 2
    assert ctx.poll_status() == 0
    print("grouped decode", group, tf.worst)
    ctx.close()


@pytest.mark.parametrize("head_dim,group,rank,batch,flags", [(64, 71, 8, 1, 0), (64, 71, 16, 2, 0), (64, 1, 8, 3, 0),
                                                            (128, 3, 8, 2, 0), (64, 12, 16, 2, 4), (64, 5, 8, 2, 1),
                                                            (64, 6, 8, 2, 2), (64, 1, 8, 2, 8), (128, 71, 8, 1, 0)])
def test_general_shapes_decode_from_empty(head_dim, group, rank, batch, flags):
    """Head dimension 64 and any number of query heads per KV head, up to the multi-query shape the
    paper evaluates (Section 4: 71 query heads over one KV head of dimension 64): the general decode
    kernel, teacher-forced against the grouped oracle from an empty cache through filling, the first
    evictions and on; both policies, both normalisers, state off, TOVA with one head."""
    import harness
    w = small(160 + group, batch=batch, layers=2, heads=2, head_dim=head_dim, prompt=0, steps=26, heavy=5, recent=6,
              rank=rank, weight_std=0.1, group=group)
    ctx, W = _setup(w, flags=flags, max_prompt=64)
    ctx.reset()
    inst = list(range(w.instances))
    tf = (harness.GroupTeacherForced if group > 1 else harness.TeacherForced)(ctx, w, W, inst, flags=flags)
    for s in range(w.steps):
        tf.step(*wl.make_decode_inputs(w, s, DEV, prompt=0))
    assert tf.evictions > 0 and ctx.poll_status() == 0
    assert ctx.kernel_variant("decode").startswith("decode_group_loop_kernel")
    ctx.reset()                                          # prompt_len == 0 resets the layers
    rec = ctx.export_state(inst)
    assert all(r["count"] == 0 and not r["H"].any() and not r["z"].any() for r in rec) and ctx.position == 0
    ctx.close()


@pytest.mark.parametrize("head_dim,group,rank,prompt,flags", [(64, 71, 8, 150, 0), (64, 5, 16, 300, 0), (64, 1, 8, 131, 0),
                                                             (128, 3, 8, 257, 0), (64, 4, 8, 200, 4), (64, 1, 8, 140, 8),
                                                             (64, 6, 8, 200, 2), (64, 3, 16, 180, 1)])
def test_general_shapes_prompt_and_decode(head_dim, group, rank, prompt, flags):
    """The prompt phase of the general shapes (head dimension 64, any number of query heads per KV
    head) on the CUDA-core kernels: per-query-head attention output, column sums over the group's
    heads, selection, cached psi, H and z against the oracle; then teacher-forced decode steps on top."""
    import harness
    w = small(170 + group, batch=1, layers=2, heads=2, head_dim=head_dim, prompt=prompt, steps=6, heavy=20, recent=20,
              rank=rank, weight_std=0.1, group=group)
    if flags & 4:
        w = w.with_(heavy=4, recent=36)
    ctx, W = _setup(w, flags=flags)
    Q, K, V, out = _prefill_all(ctx, w)
    assert Q.shape[2] == w.heads * group and Q.shape[-1] == head_dim and ctx.poll_status() == 0
    assert ctx.kernel_variant("rowstat") in ("rowstat_kernel", "") and ctx.kernel_variant("psi") in ("psi_kernel", "")
    inst = list(range(w.instances))
    if group > 1:
        r = harness.check_prefill_group(ctx, w, W, Q, K, V, inst, out, flags)
        tf = harness.GroupTeacherForced(ctx, w, W, inst, flags)
    else:
        r = harness.check_prefill(ctx, w, W, Q, K, V, inst, out, flags)
        tf = harness.TeacherForced(ctx, w, W, inst, flags)
    assert r["exempt"] <= 2
    for s in range(w.steps):
        tf.step(*wl.make_decode_inputs(w, s, DEV))
    assert tf.evictions == w.steps * w.instances and ctx.poll_status() == 0
    ctx.close()


@pytest.mark.parametrize("group,rank,prompt,flags", [(2, 8, 300, 0), (4, 16, 513, 0), (8, 8, 131, 0),
                                                     (4, 8, 300, 4), (2, 8, 700, 1), (2, 16, 260, 2)])
def test_grouped_query_heads_prompt_and_decode(group, rank, prompt, flags):
    """Prompt phase with grouped query heads: per-query-head causal attention output, column sums
    aggregated over the group's heads (Section 3.2), one kept set and one H, z per KV head; then
    teacher-forced decode steps on top of it."""
    import harness
    w = small(40 + group, prompt=prompt, steps=8, heavy=20, recent=20, rank=rank, weight_std=0.1, group=group)
    if flags & 4:
        w = w.with_(heavy=4, recent=36)
    ctx, W = _setup(w, flags=flags)
    Q, K, V, out = _prefill_all(ctx, w)
    assert Q.shape[2] == w.heads * group and K.shape[2] == w.heads and out.shape == Q.shape
    assert ctx.poll_status() == 0
    inst = list(range(w.instances))
    r = harness.check_prefill_group(ctx, w, W, Q, K, V, inst, out, flags)
    assert r["exempt"] <= 2
    tf = harness.GroupTeacherForced(ctx, w, W, inst, flags)
    for s in range(w.steps):
        tf.step(*wl.make_decode_inputs(w, s, DEV))
    assert tf.evictions == w.steps * w.instances
    assert ctx.poll_status() == 0
    print("grouped prompt", group, r, tf.worst)
    ctx.close()


def test_grouped_query_heads_rejected_configurations(monkeypatch):
    from paper_2402_09398_b200 import binding
    w = small(39, group=129)
    W = wl.make_weights(w.with_(group=4), DEV)
    with pytest.raises(binding.LessError):
        binding.from_workload(w, W, DEV)                       # more query heads per KV head than the library takes
    with pytest.raises(binding.LessError):
        binding.from_workload(small(39, group=2), W, DEV, flags=8)   # TOVA stays per head
    with pytest.raises(binding.LessError):
        binding.from_workload(small(39, group=8, heavy=4000, recent=4000), W, DEV)   # scores of 8 heads x 8000 slots exceed shared memory


def test_grouped_query_heads_many_kv_heads_after_a_prompt():
    """Several KV heads per multiprocessor, ragged slot tiles (24 slots = one and a half 16-slot
    tiles of the default grouped decode kernel), on top of a prompt phase."""
    import harness
    w = small(38, batch=11, layers=3, heads=10, prompt=150, steps=4, heavy=12, recent=12, weight_std=0.1, group=4)
    assert w.instances > 2 * torch.cuda.get_device_properties(0).multi_processor_count
    ctx, W = _setup(w)
    _prefill_all(ctx, w, with_out=False)
    inst = list(range(0, w.instances, 7))
    tf = harness.GroupTeacherForced(ctx, w, W, inst)
    for s in range(w.steps):
        tf.step(*wl.make_decode_inputs(w, s, DEV))
    assert tf.evictions == w.steps * len(inst) and ctx.poll_status() == 0
    ctx.close()


# --------------------------------------------------------------------------- #
# The parallel form (Section 3.2, Inexpensive Training; Section 4.1)
# --------------------------------------------------------------------------- #
def _schedule(w, kind, S, seed):
    """exact_until [B, L, H, S] int32: 'random' = every key leaves a random number of steps after
    its own (a tenth never leave), 'never', 'at_once' (only the diagonal stays exact)."""
    g = torch.Generator().manual_seed(seed)
    shape = (w.batch, w.layers, w.heads, S)
    pos = torch.arange(S).expand(shape)
    if kind == "never":
        return torch.full(shape, 2**31 - 1, dtype=torch.int32)
    if kind == "at_once":
        return (pos + 1).to(torch.int32)
    if kind == "no_self":         # keys that are discarded before their own query attends (not what a policy
        # produces, but the definition covers it): even the diagonal entry is a kernel value for most rows
        return (pos - torch.randint(0, 50, shape, generator=g)).clamp(min=0).to(torch.int32)
    if kind == "banded":          # an H2O-like schedule: short lives, a few keys kept for good in two key tiles only
        eu = pos + 1 + torch.randint(0, 150, shape, generator=g)
        eu[..., :4] = 2**31 - 1
        eu[..., 700:703] = 2**31 - 1
        return eu.to(torch.int32)
    life = torch.randint(1, max(2, S // 3), shape, generator=g)
    eu = pos + life
    keep = torch.rand(shape, generator=g) < 0.1
    return torch.where(keep, torch.full_like(eu, 2**31 - 1), eu).to(torch.int32)


def _check_parallel_form(w, W, Q, K, V, eu, out, instances, psi_scale=None):
    from oracle import less_oracle as lo
    import harness
    worst = 0.0
    for inst in instances:
        b, layer, head = wl.instance_coords(w, inst)
        sc = None if psi_scale is None else psi_scale[layer, head].double().cpu().numpy()
        phi_fn, psi_fn = lo.make_mlp_maps(*harness.head_weights(W, layer, head), sc)
        ref, _ = lo.masked_parallel_attention(*(t[b, layer, head].double().cpu().numpy() for t in (Q, K, V)),
                                              eu[b, layer, head].cpu().numpy(), phi_fn, psi_fn)
        err = float(np.max(np.abs(out[b, layer, head].double().cpu().numpy() - ref)))
        worst = max(worst, err)
        assert err <= harness.OUT_TOL, f"inst {inst}: parallel form max-abs {err}"
    return worst


@pytest.mark.parametrize("kind,rank,S,std", [("random", 8, 300, 0.1), ("random", 16, 513, 0.2), ("never", 8, 131, 0.1),
                                             ("at_once", 16, 257, 0.2), ("random", 8, 128, 0.3), ("random", 16, 40, 0.1),
                                             ("banded", 8, 1500, 0.2), ("banded", 16, 1153, 0.3),
                                             ("no_self", 8, 700, 0.3)])
def test_parallel_form_against_the_oracle(kind, rank, S, std):
    from paper_2402_09398_b200 import binding
    w = small(30 + rank, prompt=S, rank=rank, weight_std=std)
    ctx, W = _setup(w, flags=binding.LESS_WITH_PARALLEL_FORM)
    Q, K, V = wl.make_prompt(w, 0, w.layers, DEV)
    eu = _schedule(w, kind, S, seed=S)
    out = ctx.masked_attention(Q, K, V, eu.to(DEV))
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    worst = _check_parallel_form(w, W, Q, K, V, eu, out, list(range(w.instances)))
    print("parallel form", kind, rank, S, worst)
    ctx.close()


def test_parallel_form_rows_equal_the_decode_steps():
    """The library against itself through the paper's identity: with the schedule its own sequential
    decode steps produced (evicted_pos), row i of the parallel form is the output of step i."""
    from paper_2402_09398_b200 import binding
    S = 150
    w = small(29, prompt=0, steps=S, heavy=12, recent=12, weight_std=0.2)
    ctx, W = _setup(w, flags=binding.LESS_WITH_PARALLEL_FORM, max_prompt=S)
    qs, ks, vs, outs = [], [], [], []
    eu = torch.full((w.batch, w.layers, w.heads, S), 2**31 - 1, dtype=torch.int32)
    ev = torch.empty(w.instances, dtype=torch.int32, device=DEV)
    for t in range(S):
        q, k, v = wl.make_decode_inputs(w, t, DEV)
        outs.append(ctx.decode_step(q, k, v, evicted_pos=ev).clone())
        e = ev.cpu().reshape(w.batch, w.layers, w.heads)
        idx = torch.nonzero(e >= 0, as_tuple=True)
        eu[idx[0], idx[1], idx[2], e[idx].long()] = t + 1
        qs.append(q); ks.append(k); vs.append(v)
    Q, K, V = (torch.stack(x, dim=3).contiguous() for x in (qs, ks, vs))
    seq = torch.stack(outs, dim=3)
    par = ctx.masked_attention(Q, K, V, eu.to(DEV))
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    assert (eu != 2**31 - 1).sum() == (S - w.slots) * w.instances
    err = float((par - seq).abs().max())
    print("parallel vs sequential", err)
    assert err <= 2e-3
    ctx.close()


@pytest.mark.parametrize("group,rank,S,kind", [(2, 8, 300, "random"), (4, 16, 257, "random"), (8, 8, 131, "banded"),
                                               (4, 8, 1153, "banded"), (2, 16, 128, "at_once")])
def test_parallel_form_with_grouped_query_heads(group, rank, S, kind):
    """Every query head of a group against the oracle's single-head parallel form on the KV head's
    K, V and schedule, with the query head's own Q rows and phi (Section 3.2, multi-query attention)."""
    from paper_2402_09398_b200 import binding
    from oracle import less_oracle as lo
    import harness
    w = small(60 + group + rank, prompt=S, rank=rank, weight_std=0.2, group=group, heads=2)
    ctx, W = _setup(w, flags=binding.LESS_WITH_PARALLEL_FORM)
    Q, K, V = wl.make_prompt(w, 0, w.layers, DEV)
    assert Q.shape[2] == w.heads * group
    eu = _schedule(w, kind, S, seed=S + group)
    out = ctx.masked_attention(Q, K, V, eu.to(DEV))
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0 and out.shape == Q.shape
    worst = 0.0
    for inst in range(w.instances):
        b, layer, head = wl.instance_coords(w, inst)
        psi_w = [W[n][layer, head].double().numpy() for n in ("w_psi1", "w_psi2", "w_psi3")]
        Kh, Vh = (t[b, layer, head].double().cpu().numpy() for t in (K, V))
        for g in range(group):
            hq = head * group + g
            phi_fn, psi_fn = lo.make_mlp_maps(W["w_phi1"][layer, hq].double().numpy(),
                                              W["w_phi2"][layer, hq].double().numpy(), *psi_w)
            ref, _ = lo.masked_parallel_attention(Q[b, layer, hq].double().cpu().numpy(), Kh, Vh,
                                                  eu[b, layer, head].numpy(), phi_fn, psi_fn)
            err = float(np.max(np.abs(out[b, layer, hq].double().cpu().numpy() - ref)))
            worst = max(worst, err)
            assert err <= harness.OUT_TOL, f"inst {inst} query head {g}: parallel form max-abs {err}"
    print("grouped parallel form", group, rank, S, kind, worst)
    ctx.close()


def test_grouped_parallel_form_rows_equal_the_decode_steps():
    """The identity of the single-head test with four query heads per KV head: the schedule comes
    from the grouped decode steps' own evictions."""
    from paper_2402_09398_b200 import binding
    S, G = 140, 4
    w = small(27, prompt=0, steps=S, heavy=12, recent=12, weight_std=0.2, group=G)
    ctx, W = _setup(w, flags=binding.LESS_WITH_PARALLEL_FORM, max_prompt=S)
    qs, ks, vs, outs = [], [], [], []
    eu = torch.full((w.batch, w.layers, w.heads, S), 2**31 - 1, dtype=torch.int32)
    ev = torch.empty(w.instances, dtype=torch.int32, device=DEV)
    for t in range(S):
        q, k, v = wl.make_decode_inputs(w, t, DEV)
        outs.append(ctx.decode_step(q, k, v, evicted_pos=ev).clone())
        e = ev.cpu().reshape(w.batch, w.layers, w.heads)
        idx = torch.nonzero(e >= 0, as_tuple=True)
        eu[idx[0], idx[1], idx[2], e[idx].long()] = t + 1
        qs.append(q); ks.append(k); vs.append(v)
    Q, K, V = (torch.stack(x, dim=3).contiguous() for x in (qs, ks, vs))
    assert Q.shape == (w.batch, w.layers, w.heads * G, S, w.head_dim)
    seq = torch.stack(outs, dim=3)
    par = ctx.masked_attention(Q, K, V, eu.to(DEV))
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    assert (eu != 2**31 - 1).sum() == (S - w.slots) * w.instances
    err = float((par - seq).abs().max())
    print("grouped parallel vs sequential", err)
    assert err <= 2e-3
    ctx.close()


def test_parallel_form_needs_its_flag_and_scaled_maps():
    from paper_2402_09398_b200 import binding
    w = small(28, prompt=200, weight_std=0.2)
    ctx, W = _setup(w)
    Q, K, V = wl.make_prompt(w, 0, w.layers, DEV)
    eu = _schedule(w, "random", 200, 1).to(DEV)
    with pytest.raises(binding.LessError):
        ctx.masked_attention(Q, K, V, eu)                 # workspace not reserved
    ctx.close()
    # psi of the order of 1e4 and of 1e-4: the operands' power-of-two scales and the row factor w_i
    for c in (40.0, 1e-4):
        ps = torch.full((w.layers, w.heads, 2), c)
        ctx, W = _setup(w, flags=binding.LESS_WITH_PARALLEL_FORM, psi_scale=ps)
        out = ctx.masked_attention(Q, K, V, eu)
        torch.cuda.synchronize()
        assert ctx.poll_status() == 0
        print("parallel form psi scale", c, _check_parallel_form(w, W, Q, K, V, eu.cpu(), out, [0, 5, w.instances - 1], ps))
        ctx.close()
