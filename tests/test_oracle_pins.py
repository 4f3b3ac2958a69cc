"""Pins of the fp64 oracle against what the paper and the mathematics fix.

None of these tests retypes the oracle's own formulae in its own style: each
compares it with a library routine (torch fp64 softmax / gelu / matmul), a
closed form, a brute-force replay kept in a different data structure, or a
number the paper prints (tests/golden/).
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import less_oracle as lo
from paper_2402_09398_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------- #
# helpers
# --------------------------------------------------------------------------- #
def tiny(cfg_id=91, S=24, T=12, heavy=3, recent=3, R=4, hidden=16, D=8, heads=2,
         rule="every", param=5, std=0.5):
    return wl.Workload(cfg_id, 1, 1, heads, D, S, T, heavy, recent, R, hidden=hidden,
                       heavy_rule=rule, heavy_param=param, weight_std=std)


def head_weights(W, layer, head):
    return [W[n][layer, head].double().numpy() for n in
            ("w_phi1", "w_phi2", "w_psi1", "w_psi2", "w_psi3")]


def torch_psi(k, w1, w2, w3):
    g = torch.nn.functional.gelu
    k, w1, w2, w3 = (torch.as_tensor(a, dtype=torch.float64) for a in (k, w1, w2, w3))
    return (g(g(k @ w1) @ w2) @ w3).abs()


def torch_phi(q, w1, w2):
    g = torch.nn.functional.gelu
    q, w1, w2 = (torch.as_tensor(a, dtype=torch.float64) for a in (q, w1, w2))
    return g(g(q @ w1) @ w2).abs()


def run_instance(w, head=0, score_norm="less", use_state=True, heavy=None, recent=None, policy="h2o"):
    """Oracle free run of one head of workload w; returns instance + history."""
    W = wl.make_weights(w)
    Q, K, V = wl.make_prompt(w, 0, 1)
    wts = head_weights(W, 0, head)
    phi_fn, psi_fn = lo.make_mlp_maps(*wts)
    inst = lo.LessInstance(w.head_dim, w.rank, w.heavy if heavy is None else heavy,
                           w.recent if recent is None else recent, phi_fn, psi_fn,
                           score_norm=score_norm, use_state=use_state, policy=policy)
    q_all = [Q[0, 0, head].double().numpy()]
    k_all = [K[0, 0, head].double().numpy()]
    v_all = [V[0, 0, head].double().numpy()]
    pre_out = inst.prefill(q_all[0], k_all[0], v_all[0])
    steps = []
    for s in range(w.steps):
        q, k, v = wl.make_decode_inputs(w, s)
        q, k, v = (a[0, 0, head].double().numpy() for a in (q, k, v))
        kept_before = inst.pos.copy()
        r = inst.decode(q, k, v)
        r["kept_before"] = kept_before
        r["q"], r["k"], r["v"] = q, k, v
        steps.append(r)
    Kh = np.vstack([k_all[0]] + [r["k"][None] for r in steps])
    Vh = np.vstack([v_all[0]] + [r["v"][None] for r in steps])
    return inst, pre_out, steps, (q_all[0], Kh, Vh), wts


# --------------------------------------------------------------------------- #
# P9: numbers the paper prints
# --------------------------------------------------------------------------- #
def test_table1_token_counts():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "table1_token_counts.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 6
    for _, max_len, pct, tokens in rows:
        n = lo.h2o_token_count(float(pct), int(max_len))
        assert n == int(tokens)
        assert n % 2 == 0


def test_budget_fraction_of_prompt():
    # 5 % + 5 % of 2048 must reproduce Table 1's 204 = 102 + 102 for that length
    assert 2 * lo.budget_from_fraction(0.05, 2048) == lo.h2o_token_count(10, 2048)
    assert lo.budget_from_fraction(0.02, 16384) == 327
    assert lo.budget_from_fraction(0.05, 32768) == 1638
    assert wl.CONFIGS[6].slots == lo.h2o_token_count(10, 2048)   # Table 1: Falcon at 10 % of its 2048 context
    for cid, w in wl.CONFIGS.items():      # the product's host logic agrees
        frac = {2: 0.05, 3: 0.10, 4: 0.02, 5: 0.05}.get(cid)      # 1: fixed slots; 6: the multi-query context shape
        if frac is not None:
            assert w.heavy == w.recent == lo.budget_from_fraction(frac, w.prompt)


def test_paper_sizes_pin_shapes():
    kv = {}
    for l in open(os.path.join(GOLDEN, "paper_sizes.txt")):
        if l.strip() and not l.startswith("#"):
            a, b = l.split()
            kv[a] = float(b)
    R, D, Rp = int(kv["state_rank"]), int(kv["head_dim"]), int(kv["hidden"])
    inst = lo.LessInstance(D, R, 4, 4, None, None)
    # H holds as many numbers as `state_equiv_tokens` cached (key,value) pairs
    assert inst.H.size == kv["state_equiv_tokens"] * 2 * D
    assert inst.H.shape == (R, D) and inst.z.shape == (R,)
    # per-head MLPs D -> R' -> R (-> R for psi): parameter fraction of 13B
    w = wl.Workload(99, 1, 1, 1, D, 4, 0, 1, 1, R, hidden=Rp)
    per_head = sum(t.numel() for t in wl.make_weights(w).values())
    assert per_head == 2 * (D * Rp + Rp * R) + R * R
    frac = per_head * kv["llama13b_layers"] * kv["llama13b_heads"] / kv["llama13b_params"]
    assert 0.015 < frac < kv["max_param_fraction"]


# --------------------------------------------------------------------------- #
# P6: feature maps against library routines
# --------------------------------------------------------------------------- #
def test_gelu_against_math_erf_and_torch():
    x = np.linspace(-6, 6, 241)
    ref = np.array([0.5 * v * (1 + math.erf(v / math.sqrt(2))) for v in x])
    assert np.max(np.abs(lo.gelu(x) - ref)) < 1e-15
    tref = torch.nn.functional.gelu(torch.tensor(x, dtype=torch.float64)).numpy()
    assert np.max(np.abs(lo.gelu(x) - tref)) < 1e-14
    assert lo.gelu(np.array([0.0]))[0] == 0.0
    assert abs(lo.gelu(np.array([1.0]))[0] - 0.8413447460685429) < 1e-15   # Phi(1)


def test_feature_maps_against_torch_and_nonneg():
    w = tiny(cfg_id=92, D=16, hidden=32, R=8, std=0.3)
    W = wl.make_weights(w)
    Q, K, _ = wl.make_prompt(w, 0, 1)
    for head in range(w.heads):
        p1, p2, s1, s2, s3 = head_weights(W, 0, head)
        q = Q[0, 0, head].double().numpy()
        k = K[0, 0, head].double().numpy()
        phi = lo.phi_map(q, p1, p2)
        psi = lo.psi_map(k, s1, s2, s3)
        assert phi.shape == (w.prompt, w.rank) and psi.shape == (w.prompt, w.rank)
        assert (phi >= 0).all() and (psi >= 0).all()             # absolute values (Eq. 1-2)
        assert np.allclose(phi, torch_phi(q, p1, p2).numpy(), rtol=1e-12, atol=1e-15)
        assert np.allclose(psi, torch_psi(k, s1, s2, s3).numpy(), rtol=1e-12, atol=1e-15)
        # phi and psi use different weights and psi has one more layer
        assert not np.allclose(phi, lo.phi_map(q, s1, s2))
        # W3 = 0 => psi == 0
        assert (lo.psi_map(k, s1, s2, np.zeros_like(s3)) == 0).all()
        # the learnable scalars multiply the activations after each GELU
        sc = np.array([0.5, 3.0])
        g = torch.nn.functional.gelu
        kt = torch.tensor(k)
        ref = ((3.0 * g((0.5 * g(kt @ torch.tensor(s1))) @ torch.tensor(s2))) @ torch.tensor(s3)).abs()
        assert np.allclose(lo.psi_map(k, s1, s2, s3, sc), ref.numpy(), rtol=1e-12, atol=1e-15)


def test_feature_map_hand_value():
    # 1-d closed form: phi(q) = |gelu(gelu(q*a)*b)|
    a, b, q = 0.7, -1.3, 2.0
    G = lambda x: 0.5 * x * (1 + math.erf(x / math.sqrt(2)))
    want = abs(G(G(q * a) * b))
    got = lo.phi_map(np.array([[q]]), np.array([[a]]), np.array([[b]]))[0, 0]
    assert abs(got - want) < 1e-15
    c = 0.9
    want_psi = abs(G(G(q * a) * b) * c)
    got_psi = lo.psi_map(np.array([[q]]), np.array([[a]]), np.array([[b]]), np.array([[c]]))[0, 0]
    assert abs(got_psi - want_psi) < 1e-15


# --------------------------------------------------------------------------- #
# P1: no eviction  ==  textbook attention (Section 3.1: prompt phase is regular
# attention; with budget >= sequence length nothing is ever discarded)
# --------------------------------------------------------------------------- #
def test_no_eviction_equals_full_attention():
    w = tiny(cfg_id=93, S=20, T=10, D=16)
    inst, pre_out, steps, (Qp, Kh, Vh), _ = run_instance(w, heavy=20, recent=20)
    Kt, Vt = torch.tensor(Kh), torch.tensor(Vh)
    # prompt: causal softmax
    s = torch.tensor(Qp) @ Kt[: w.prompt].T / math.sqrt(w.head_dim)
    s = s.masked_fill(torch.triu(torch.ones_like(s), 1).bool(), float("-inf"))
    ref = torch.softmax(s, dim=-1) @ Vt[: w.prompt]
    assert np.allclose(pre_out, ref.numpy(), rtol=1e-12, atol=1e-14)
    for i, r in enumerate(steps):
        n = w.prompt + i + 1
        p = torch.softmax(Kt[:n] @ torch.tensor(r["q"]) / math.sqrt(w.head_dim), dim=0)
        assert np.allclose(r["out"], (p @ Vt[:n]).numpy(), rtol=1e-12, atol=1e-14)
        assert r["evicted_pos"] == -1
    assert not inst.evicted and (inst.H == 0).all() and (inst.z == 0).all()
    assert list(inst.pos) == list(range(w.prompt + w.steps))


# --------------------------------------------------------------------------- #
# P2: state disabled  ==  softmax over the kept set only (pure H2O)
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("zero_by", ["flag", "w3"])
def test_state_off_equals_sparse_softmax(zero_by):
    w = tiny(cfg_id=94, S=30, T=15, D=16)
    if zero_by == "flag":
        inst, _, steps, (_, Kh, Vh), _ = run_instance(w, use_state=False)
    else:
        W = wl.make_weights(w)
        p1, p2, s1, s2, s3 = head_weights(W, 0, 0)
        phi_fn, psi_fn = lo.make_mlp_maps(p1, p2, s1, s2, np.zeros_like(s3))
        Q, K, V = wl.make_prompt(w, 0, 1)
        inst = lo.LessInstance(w.head_dim, w.rank, w.heavy, w.recent, phi_fn, psi_fn)
        inst.prefill(*(a[0, 0, 0].double().numpy() for a in (Q, K, V)))
        steps = []
        for s in range(w.steps):
            q, k, v = (a[0, 0, 0].double().numpy() for a in wl.make_decode_inputs(w, s))
            kb = inst.pos.copy()
            r = inst.decode(q, k, v)
            r.update(kept_before=kb, q=q, k=k, v=v)
            steps.append(r)
        Kh = np.vstack([K[0, 0, 0].double().numpy()] + [r["k"][None] for r in steps])
        Vh = np.vstack([V[0, 0, 0].double().numpy()] + [r["v"][None] for r in steps])
    assert inst.evicted, "the case must evict"
    for i, r in enumerate(steps):
        idx = list(r["kept_before"]) + [w.prompt + i]
        Ks, Vs = torch.tensor(Kh[idx]), torch.tensor(Vh[idx])
        p = torch.softmax(Ks @ torch.tensor(r["q"]) / math.sqrt(w.head_dim), dim=0)
        assert np.allclose(r["out"], (p @ Vs).numpy(), rtol=1e-12, atol=1e-14)
        assert np.allclose(r["p"], p.numpy(), rtol=1e-12, atol=1e-15)
    assert (inst.H == 0).all() and (inst.z == 0).all()


# --------------------------------------------------------------------------- #
# P3 / P8: Eq. 6 -- H, z equal the brute-force sums over the evicted log
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("norm", ["less", "sparse"])
def test_state_equals_sum_over_evicted_log(norm):
    w = tiny(cfg_id=95, S=40, T=25, heavy=4, recent=5, D=16, R=4)
    inst, _, steps, (_, Kh, Vh), wts = run_instance(w, score_norm=norm)
    ev = inst.evicted
    assert len(ev) == w.prompt + w.steps - inst.N                 # one per token beyond N
    assert len(set(ev)) == len(ev)
    psi = torch_psi(Kh[ev], *wts[2:])                             # library routine
    H_ref = psi.T @ torch.tensor(Vh[ev])
    z_ref = psi.sum(0)
    assert np.allclose(inst.H, H_ref.numpy(), rtol=1e-11, atol=1e-14)
    assert np.allclose(inst.z, z_ref.numpy(), rtol=1e-11, atol=1e-14)
    # bookkeeping: kept positions unique, contain the last `recent`, disjoint from evicted
    kept = list(inst.pos)
    t_end = w.prompt + w.steps
    assert len(set(kept)) == len(kept) == inst.N
    assert set(range(t_end - w.recent, t_end)) <= set(kept)
    assert not (set(kept) & set(ev)) and set(kept) | set(ev) == set(range(t_end))
    # cached rows are the rows of those positions
    assert np.array_equal(inst.K, Kh[kept]) and np.array_equal(inst.V, Vh[kept])
    # increments reported per step are rank one and add up
    dz = sum(r["dz"] for r in steps if r["dz"] is not None)
    pre_ev = [p for p in ev if p < w.prompt and p not in
              [r["evicted_pos"] for r in steps]]
    z_pre = torch_psi(Kh[pre_ev], *wts[2:]).sum(0).numpy()
    assert np.allclose(z_pre + dz, inst.z, rtol=1e-11, atol=1e-14)


def test_z_monotone_and_probabilities_sum_to_one():
    w = tiny(cfg_id=96, S=30, T=20, D=16, std=0.8)
    inst, _, steps, _, _ = run_instance(w)
    z_prev = None
    for r in steps:
        # P7: sparse probabilities plus the low-rank share make exactly one
        assert abs(r["p"].sum() + r["lr_den"] / r["den"] - 1.0) < 1e-13
        assert r["lr_den"] >= 0 and (r["p"] > 0).all()
    assert (inst.z >= 0).all()
    # prompt column sums: every row of the causal softmax sums to one
    assert abs(inst.prompt_acc.sum() - w.prompt) < 1e-10
    assert abs(inst.prompt_acc[-1] - 0) > 0 and inst.prompt_acc[0] >= 1.0   # column 0 gets row 0 entirely


# --------------------------------------------------------------------------- #
# P4: exhaustive replay on tiny inputs.  The replay below keeps the WHOLE
# history (every key/value, every probability row ever produced) and recomputes
# each accumulated score, H and z from scratch at every step; it never updates
# anything incrementally and never calls the oracle's step.
# --------------------------------------------------------------------------- #
def _replay(w, head, norm, use_state):
    W = wl.make_weights(w)
    p1, p2, s1, s2, s3 = (torch.tensor(a) for a in head_weights(W, 0, head))
    Q, K, V = (a[0, 0, head].double() for a in wl.make_prompt(w, 0, 1))
    S, D, N = w.prompt, w.head_dim, w.heavy + w.recent
    keys, vals = [K[i] for i in range(S)], [V[i] for i in range(S)]
    prob_rows = []                       # list of dict pos -> probability
    for i in range(S):
        sc = torch.stack([Q[i] @ keys[j] for j in range(i + 1)]) / math.sqrt(D)
        pr = torch.softmax(sc, 0)
        prob_rows.append({j: float(pr[j]) for j in range(i + 1)})
    total = lambda pos: sum(r.get(pos, 0.0) for r in prob_rows)
    kept, evicted = list(range(S)), []
    while len(kept) > N:                 # repeated argmin == one-shot selection
        cand = [p for p in kept if p < S - w.recent]
        vic = min(cand, key=lambda p: (total(p), p))
        kept.remove(vic)
        evicted.append(vic)
    outs, victims = [], []
    for step in range(w.steps):
        t = S + step
        q, k, v = (a[0, 0, head].double() for a in wl.make_decode_inputs(w, step))
        keys.append(k)
        vals.append(v)
        att = kept + [t]
        e = {p: math.exp(float(q @ keys[p]) / math.sqrt(D)) for p in att}
        num = sum(e[p] * vals[p] for p in att)
        den_sparse = sum(e.values())
        den = den_sparse
        if use_state and evicted:
            Ke = torch.stack([keys[p] for p in evicted])
            Ve = torch.stack([vals[p] for p in evicted])
            g = torch.nn.functional.gelu
            psi = (g(g(Ke @ s1) @ s2) @ s3).abs()
            phi = g(g(q[None] @ p1) @ p2).abs()[0]
            num = num + phi @ (psi.T @ Ve)
            den = den + float(phi @ psi.sum(0))
        outs.append((num / den).numpy())
        d = den if norm == "less" else den_sparse
        prob_rows.append({p: e[p] / d for p in att})
        kept = att
        vic = -1
        if len(kept) > N:
            cand = [p for p in kept if p <= t - w.recent]
            vic = min(cand, key=lambda p: (total(p), p))
            kept.remove(vic)
            evicted.append(vic)
        victims.append(vic)
    return outs, victims, kept, evicted


@pytest.mark.parametrize("norm,use_state", [("less", True), ("sparse", True), ("less", False)])
@pytest.mark.parametrize("geom", [(16, 12, 3, 3), (12, 10, 0, 4), (9, 8, 5, 1), (4, 9, 3, 3)])
def test_exhaustive_replay_matches(norm, use_state, geom):
    S, T, heavy, recent = geom
    w = tiny(cfg_id=97, S=S, T=T, heavy=heavy, recent=recent, D=8, R=4, hidden=16, std=0.9,
             rule="every", param=4)
    for head in range(w.heads):
        outs, victims, kept, evicted = _replay(w, head, norm, use_state)
        inst, _, steps, _, _ = run_instance(w, head=head, score_norm=norm, use_state=use_state)
        assert [r["evicted_pos"] for r in steps] == victims
        assert sorted(inst.pos) == sorted(kept)
        assert sorted(inst.evicted) == sorted(evicted)
        for r, o in zip(steps, outs):
            assert np.allclose(r["out"], o, rtol=1e-10, atol=1e-13)


def test_tie_break_lowest_position():
    # identical keys and values => identical accumulated scores for equal-age
    # columns is impossible (older columns collect more rows), so build ties
    # directly through an imported state.
    D, R = 4, 2
    phi_fn = lambda x: np.ones((x.shape[0], R))
    psi_fn = lambda x: np.ones((x.shape[0], R))
    inst = lo.LessInstance(D, R, 2, 2, phi_fn, psi_fn)
    pos = np.array([7, 3, 5, 9])
    K = np.zeros((4, D))
    V = np.arange(16.0).reshape(4, D)
    acc = np.array([0.5, 0.5, 0.5, 0.1])          # pos 9 has the lowest score but is recent
    inst.import_state(pos, K, V, acc, np.zeros((R, D)), np.zeros(R), t=10)
    r = inst.decode(np.zeros(D), np.zeros(D), np.ones(D))
    # candidates: pos <= 10 - 2 = 8 -> {7,3,5}, all tied after adding equal p => lowest position
    assert r["evicted_pos"] == 3
    assert r["tie_gap"] == 0.0
    assert np.allclose(inst.H, np.outer(np.ones(R), V[1]))
    assert sorted(inst.pos) == [5, 7, 9, 10]


# --------------------------------------------------------------------------- #
# P5: ideal kernel identity (Section 3.1, after Eq. 2): if phi(q) psi(k)^T equals
# exp(q k^T / sqrt(D)) for all q, k, LESS returns the ORIGINAL attention, for any
# eviction pattern.  psi = one-hot over tokens, phi(q)_j = exp(q.k_j / sqrt(D)).
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("norm", ["less", "sparse"])
def test_ideal_kernel_recovers_full_attention(norm):
    w = tiny(cfg_id=98, S=14, T=10, heavy=2, recent=3, D=8)
    Q, K, V = (a[0, 0, 0].double().numpy() for a in wl.make_prompt(w, 0, 1))
    dec = [tuple(a[0, 0, 0].double().numpy() for a in wl.make_decode_inputs(w, s))
           for s in range(w.steps)]
    Kall = np.vstack([K] + [d[1][None] for d in dec])
    Vall = np.vstack([V] + [d[2][None] for d in dec])
    n_tok = Kall.shape[0]

    def psi_fn(x):
        out = np.zeros((x.shape[0], n_tok))
        for r, row in enumerate(x):
            j = int(np.nonzero((Kall == row).all(axis=1))[0][0])
            out[r, j] = 1.0
        return out

    def phi_fn(x):
        return np.exp(x @ Kall.T / math.sqrt(w.head_dim))

    inst = lo.LessInstance(w.head_dim, n_tok, w.heavy, w.recent, phi_fn, psi_fn, score_norm=norm)
    inst.prefill(Q, K, V)
    for s, (q, k, v) in enumerate(dec):
        r = inst.decode(q, k, v)
        n = w.prompt + s + 1
        p = torch.softmax(torch.tensor(Kall[:n] @ q) / math.sqrt(w.head_dim), 0)
        ref = (p @ torch.tensor(Vall[:n])).numpy()
        assert np.allclose(r["out"], ref, rtol=1e-11, atol=1e-13)
    assert len(inst.evicted) == n_tok - inst.N


def test_hellinger_closed_forms():
    assert lo.hellinger([1, 0], [0, 1]) == pytest.approx(1.0)
    assert lo.hellinger([0.25, 0.75], [0.25, 0.75]) == 0.0
    assert lo.hellinger([1, 0], [0.5, 0.5]) == pytest.approx(math.sqrt(1 - math.sqrt(0.5)))


# --------------------------------------------------------------------------- #
# The pins must be sharp: plausible mistakes planted in the oracle (on the CPU)
# have to break at least one of the checks above.
# --------------------------------------------------------------------------- #
class _Mutant(lo.LessInstance):
    kind = ""

    def decode(self, q, k, v):
        if self.kind == "drop_z":
            z = self.z.copy()
            self.z = np.zeros_like(z)
            r = super().decode(q, k, v)
            self.z = z + (self.z)          # keep accumulating what decode added
            return r
        if self.kind == "recent_off_by_one":
            self.recent += 1
            try:
                return super().decode(q, k, v)
            finally:
                self.recent -= 1
        if self.kind == "no_sqrt_d":
            return super().decode(np.asarray(q, dtype=np.float64) * math.sqrt(self.D), k, v)
        return super().decode(q, k, v)


@pytest.mark.parametrize("kind", ["drop_z", "recent_off_by_one", "no_sqrt_d"])
def test_planted_mistakes_are_caught(kind):
    w = tiny(cfg_id=97, S=16, T=12, heavy=3, recent=3, D=8, R=4, hidden=16, std=0.9,
             rule="every", param=4)
    W = wl.make_weights(w)
    wts = head_weights(W, 0, 0)
    phi_fn, psi_fn = lo.make_mlp_maps(*wts)
    outs, victims, kept, evicted = _replay(w, 0, "less", True)
    m = _Mutant(w.head_dim, w.rank, w.heavy, w.recent, phi_fn, psi_fn)
    m.kind = kind
    Q, K, V = (a[0, 0, 0].double().numpy() for a in wl.make_prompt(w, 0, 1))
    m.prefill(Q, K, V)
    bad = False
    for s in range(w.steps):
        q, k, v = (a[0, 0, 0].double().numpy() for a in wl.make_decode_inputs(w, s))
        r = m.decode(q, k, v)
        if r["evicted_pos"] != victims[s] or not np.allclose(r["out"], outs[s], rtol=1e-10, atol=1e-13):
            bad = True
    assert bad, f"mutant {kind} slipped through the replay pin"


# --------------------------------------------------------------------------- #
# Lambda-masking as the sparse policy (Section 4: the first tokens plus the most recent ones)
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("use_state", [True, False])
def test_lambda_masking_closed_forms(use_state):
    """The kept set has a closed form at every step; with the state off the output is the
    softmax over exactly that set (the streaming pattern), with it on H and z are the plain sums
    over every other position (Eq. 6) and the step obeys Eq. 3 with those sums."""
    sinks, window = 4, 7
    w = tiny(cfg_id=96, S=33, T=14, heavy=sinks, recent=window, D=16, R=4)
    inst, _, steps, (_, Kh, Vh), wts = run_instance(w, use_state=use_state, policy="lambda")
    Kt, Vt = torch.tensor(Kh), torch.tensor(Vh)
    for i, r in enumerate(steps):
        t = w.prompt + i                                             # position of the new token
        kept = list(range(sinks)) + list(range(t - window, t))      # sinks + the `window` latest cached tokens
        assert list(r["kept_before"]) == kept
        assert r["evicted_pos"] == t - window                        # the oldest token of the window leaves
        idx = kept + [t]
        e = torch.exp(Kt[idx] @ torch.tensor(r["q"]) / math.sqrt(w.head_dim))
        if not use_state:
            p = e / e.sum()
            assert np.allclose(r["out"], (p @ Vt[idx]).numpy(), rtol=1e-12, atol=1e-14)
        else:
            gone = [j for j in range(t) if j not in kept]
            psi = torch_psi(Kh[gone], *wts[2:])
            phi = torch_phi(r["q"][None], *wts[:2])[0]
            num = phi @ (psi.T @ Vt[gone]) + e @ Vt[idx]
            den = phi @ psi.sum(0) + e.sum()
            assert np.allclose(r["out"], (num / den).numpy(), rtol=1e-10, atol=1e-13)
    t_end = w.prompt + w.steps
    assert list(inst.pos) == list(range(sinks)) + list(range(t_end - window, t_end))
    assert sorted(inst.evicted) == list(range(sinks, t_end - window))
    if not use_state:
        assert (inst.H == 0).all() and (inst.z == 0).all()


def test_lambda_masking_short_context_and_budget_that_holds_everything():
    w = tiny(cfg_id=97, S=6, T=9, heavy=2, recent=5, D=16, R=4)    # 7 slots, prompt of 6: fills, then slides
    inst, _, steps, _, _ = run_instance(w, policy="lambda")
    assert [r["evicted_pos"] for r in steps] == [-1] + list(range(2, 10))
    w = tiny(cfg_id=98, S=12, T=5, D=16)
    a, _, sa, _, _ = run_instance(w, heavy=4, recent=30, policy="lambda")
    b, _, sb, _, _ = run_instance(w, heavy=30, recent=30, policy="h2o")
    for x, y in zip(sa, sb):                                         # nothing evicted: the policy cannot matter
        assert np.array_equal(x["out"], y["out"]) and x["evicted_pos"] == -1


# --------------------------------------------------------------------------- #
# TOVA as the sparse policy (named in Section 4; the rule is the cited work's: the entry with the
# lowest attention probability of the current query leaves, the newest included)
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("use_state", [True, False])
def test_tova_against_an_independent_replay(use_state):
    """A replay kept as a plain python set of positions, with torch softmax for the probabilities,
    must choose the same victims; the outputs obey Eq. 3 with torch-computed Eq. 6 sums."""
    w = tiny(cfg_id=99, S=26, T=16, heavy=3, recent=4, D=16, R=4)
    N = w.heavy + w.recent
    inst, _, steps, (Qp, Kh, Vh), wts = run_instance(w, use_state=use_state, policy="tova")
    Kt, Vt = torch.tensor(Kh), torch.tensor(Vh)
    # prompt: the last prompt query's causal softmax row ranks the prompt tokens
    p_last = torch.softmax(Kt[: w.prompt] @ torch.tensor(Qp[-1]) / math.sqrt(w.head_dim), dim=0).numpy()
    order = sorted(range(w.prompt), key=lambda j: (p_last[j], j))
    kept = set(range(w.prompt)) - set(order[: w.prompt - N])
    gone = set(order[: w.prompt - N])
    new_token_evicted = 0
    for i, r in enumerate(steps):
        t = w.prompt + i
        assert sorted(kept) == list(r["kept_before"])
        idx = sorted(kept) + [t]
        e = torch.exp(Kt[idx] @ torch.tensor(r["q"]) / math.sqrt(w.head_dim))
        if use_state and gone:
            g = sorted(gone)
            psi = torch_psi(Kh[g], *wts[2:])
            phi = torch_phi(r["q"][None], *wts[:2])[0]
            num, den = phi @ (psi.T @ Vt[g]) + e @ Vt[idx], phi @ psi.sum(0) + e.sum()
        else:
            num, den = e @ Vt[idx], e.sum()
        assert np.allclose(r["out"], (num / den).numpy(), rtol=1e-10, atol=1e-13)
        prob = (e / den).numpy()
        victim = min(zip(prob, idx))[1]                     # lowest probability, then lowest position
        assert r["evicted_pos"] == victim
        new_token_evicted += victim == t
        kept = (kept | {t}) - {victim}
        gone.add(victim)
    assert sorted(kept) == list(inst.pos) and sorted(gone) == sorted(inst.evicted)
    assert len(kept) == N
    if not use_state:
        assert (inst.H == 0).all() and (inst.z == 0).all()


def test_tova_can_evict_the_new_token_itself():
    """A new key that the query points away from gets the lowest probability of its own step:
    it never enters the cache and is absorbed into H, z at once."""
    D, R = 8, 2
    phi = lambda x: np.abs(x[:, :R])
    psi = lambda x: np.abs(x[:, :R]) + 1.0
    inst = lo.LessInstance(D, R, 2, 2, phi, psi, policy="tova")
    K = np.eye(D)[:4] * 3.0
    V = np.arange(4 * D, dtype=np.float64).reshape(4, D)
    inst.prefill(np.ones((4, D)), K, V)
    assert list(inst.pos) == [0, 1, 2, 3]
    q = np.ones(D)
    k_new, v_new = -5.0 * np.ones(D), np.full(D, 7.0)
    r = inst.decode(q, k_new, v_new)
    assert r["evicted_pos"] == 4 and list(inst.pos) == [0, 1, 2, 3]
    assert np.allclose(inst.H, np.outer(psi(k_new[None])[0], v_new)) and np.allclose(inst.z, psi(k_new[None])[0])


# --------------------------------------------------------------------------- #
# Grouped query heads (Section 3.2: H2O scores aggregated across the query heads of a KV head)
# --------------------------------------------------------------------------- #
def _group_case(G, cfg_id=100, S=28, T=12, heavy=3, recent=4, D=16, R=4, policy="h2o", use_state=True,
                score_norm="less"):
    w = tiny(cfg_id=cfg_id, S=S, T=T, heavy=heavy, recent=recent, D=D, R=R, heads=G + 1)
    W = wl.make_weights(w)
    Q, K, V = wl.make_prompt(w, 0, 1)
    phis = [lo.make_mlp_maps(*head_weights(W, 0, g))[0] for g in range(G)]      # phi of query head g
    psi_w = head_weights(W, 0, G)                                               # psi of the KV head
    psi_fn = lo.make_mlp_maps(*psi_w)[1]
    grp = lo.LessGroup(D, R, heavy, recent, phis, psi_fn, score_norm=score_norm, use_state=use_state, policy=policy)
    Qg = np.stack([Q[0, 0, g].double().numpy() for g in range(G)])
    Kk, Vv = K[0, 0, G].double().numpy(), V[0, 0, G].double().numpy()
    return w, W, grp, Qg, Kk, Vv, psi_w


GROUP_MODES = [(policy, norm, state) for policy in ("h2o", "lambda") for norm in ("less", "sparse")
               for state in (True, False)]


@pytest.mark.parametrize("policy,norm,state", GROUP_MODES)
def test_group_of_one_is_the_single_head_instance(policy, norm, state):
    """G = 1 reduces the grouped recursion to LessInstance in every mode the grouped CUDA kernels
    are compared against: both policies, both normalisers of the H2O scores, state on and off."""
    w, W, grp, Qg, Kk, Vv, psi_w = _group_case(1, policy=policy, use_state=state, score_norm=norm)
    one = lo.LessInstance(16, 4, 3, 4, grp.phi_fns[0], grp.psi_fn, score_norm=norm, use_state=state, policy=policy)
    assert np.array_equal(grp.prefill(Qg, Kk, Vv)[0], one.prefill(Qg[0], Kk, Vv))
    assert list(grp.pos) == list(one.pos) and np.array_equal(grp.acc, one.acc)
    for s in range(w.steps):
        q, k, v = (a[0, 0].double().numpy() for a in wl.make_decode_inputs(w, s))
        a, b = grp.decode(q[:1], k[1], v[1]), one.decode(q[0], k[1], v[1])
        assert np.array_equal(a["out"][0], b["out"]) and a["evicted_pos"] == b["evicted_pos"]
        assert np.array_equal(grp.acc, one.acc)
    assert np.array_equal(grp.H, one.H) and np.array_equal(grp.z, one.z) and list(grp.pos) == list(one.pos)
    if not state:
        assert not grp.H.any() and not grp.z.any()


@pytest.mark.parametrize("policy,norm,state", GROUP_MODES)
@pytest.mark.parametrize("G", [2, 4])
def test_group_scores_are_summed_over_heads_and_state_is_shared(G, policy, norm, state):
    """Independent replay with torch, in every mode: each head's output is Eq. 3 over the shared
    kept set and the shared Eq. 6 sums (zero with the state off); H2O's victim is the minimum of
    the head-summed accumulated probabilities - each head's probability under its own normaliser,
    Eq. 3's or the sparse-only one - kept here in a dict by position and rebuilt every step;
    Lambda-masking's kept set is its closed form, the first `heavy` positions plus the window."""
    w, W, grp, Qg, Kk, Vv, psi_w = _group_case(G, cfg_id=101, policy=policy, use_state=state, score_norm=norm)
    heavy, recent, N = 3, 4, 7
    grp.prefill(Qg, Kk, Vv)
    Kt, Vt = [torch.tensor(Kk)], [torch.tensor(Vv)]
    S = w.prompt
    if policy == "h2o":
        # prompt scores: sum over heads of the causal softmax column sums
        score = np.zeros(S)
        for g in range(G):
            s = torch.tensor(Qg[g]) @ Kt[0].T / math.sqrt(16)
            s = s.masked_fill(torch.triu(torch.ones_like(s), 1).bool(), float("-inf"))
            score += torch.softmax(s, dim=-1).sum(0).numpy()
        cand = sorted(range(S - recent), key=lambda j: (score[j], j))
        gone = set(cand[: S - N])
    else:
        score = np.zeros(S)
        gone = set(range(heavy, S - recent))
    kept = set(range(S)) - gone
    hist = {j: score[j] for j in kept}
    assert sorted(kept) == list(grp.pos)
    phi_w = [head_weights(W, 0, g)[:2] for g in range(G)]
    for i in range(w.steps):
        q, k, v = (a[0, 0].double().numpy() for a in wl.make_decode_inputs(w, i))
        t = S + i
        Kt.append(torch.tensor(k[G])[None]); Vt.append(torch.tensor(v[G])[None])
        Kall, Vall = torch.cat(Kt), torch.cat(Vt)
        r = grp.decode(q[:G], k[G], v[G])
        idx = sorted(kept) + [t]
        g_idx = sorted(gone)
        if state:
            psi = torch_psi(Kall[g_idx].numpy(), *psi_w[2:])
            Hs, zs = psi.T @ Vall[g_idx], psi.sum(0)
            assert np.allclose(r["lr_num"][0], (torch_phi(q[0][None], *phi_w[0])[0] @ Hs).numpy(), rtol=1e-9, atol=1e-13)
        else:
            Hs, zs = torch.zeros(4, 16, dtype=torch.float64), torch.zeros(4, dtype=torch.float64)
            assert not grp.H.any() and not grp.z.any()
        psum = np.zeros(len(idx))
        for g in range(G):
            e = torch.exp(Kall[idx] @ torch.tensor(q[g]) / math.sqrt(16))
            phi = torch_phi(q[g][None], *phi_w[g])[0]
            den = phi @ zs + e.sum()
            assert np.allclose(r["out"][g], ((phi @ Hs + e @ Vall[idx]) / den).numpy(), rtol=1e-10, atol=1e-13)
            psum += (e / (den if norm == "less" else e.sum())).numpy()
        assert np.allclose(r["p"], psum, rtol=1e-10, atol=1e-14)
        if policy == "h2o":
            for j, pj in zip(idx, psum):
                hist[j] = hist.get(j, 0.0) + pj
            victim = min((hist[j], j) for j in idx if j <= t - recent)[1]
            del hist[victim]
        else:
            victim = min(j for j in idx if j >= heavy)
            assert victim == t - recent                # closed form: the window slides by one
        assert r["evicted_pos"] == victim
        kept = (kept | {t}) - {victim}
        gone.add(victim)
        if policy == "lambda":
            assert kept == set(range(heavy)) | set(range(t - recent + 1, t + 1))
    assert sorted(kept) == list(grp.pos)
    if policy == "h2o":
        assert np.allclose(grp.acc, [hist[j] for j in sorted(kept)], rtol=1e-10, atol=1e-14)


def test_group_sparse_normaliser_differs_only_through_the_low_rank_mass():
    """A planted slip - the sparse normaliser applied where Eq. 3's belongs - changes the
    accumulated scores exactly when z != 0: with the state off the two modes agree bit for bit,
    with it on they must differ."""
    runs = {}
    for norm in ("less", "sparse"):
        for state in (True, False):
            w, W, grp, Qg, Kk, Vv, _ = _group_case(2, cfg_id=102, use_state=state, score_norm=norm)
            grp.prefill(Qg, Kk, Vv)
            for i in range(w.steps):
                q, k, v = (a[0, 0].double().numpy() for a in wl.make_decode_inputs(w, i))
                grp.decode(q[:2], k[2], v[2])
            runs[norm, state] = (list(grp.pos), grp.acc.copy())
    assert runs["less", False][0] == runs["sparse", False][0]
    assert np.array_equal(runs["less", False][1], runs["sparse", False][1])
    common = sorted(set(runs["less", True][0]) & set(runs["sparse", True][0]))
    a = np.array([runs["less", True][1][runs["less", True][0].index(j)] for j in common])
    b = np.array([runs["sparse", True][1][runs["sparse", True][0].index(j)] for j in common])
    assert np.all(b >= a) and np.any(b > a)            # the sparse normaliser is the smaller one


# --------------------------------------------------------------------------- #
# The parallel form (Section 3.2, Inexpensive Training; Section 4.1): the whole causal attention
# matrix at once, entries the sparse policy dropped replaced by phi(q_i) psi(k_j)^T
# --------------------------------------------------------------------------- #
def _sequence_case(cfg_id, S=40, heavy=3, recent=4, D=16, R=4, policy="h2o"):
    w = tiny(cfg_id=cfg_id, S=S, T=0, heavy=heavy, recent=recent, D=D, R=R, heads=1, std=0.4)
    W = wl.make_weights(w)
    Q, K, V = (t[0, 0, 0].double().numpy() for t in wl.make_prompt(w, 0, 1))
    phi_fn, psi_fn = lo.make_mlp_maps(*head_weights(W, 0, 0))
    return w, Q, K, V, phi_fn, psi_fn


@pytest.mark.parametrize("policy", ["h2o", "lambda", "tova"])
def test_parallel_form_rows_are_the_sequential_steps(policy):
    """Row i of the parallel form is Algorithm 1's output at step i when the mask is the schedule
    the sequential run produced: the two share nothing but the feature maps (the sequential run
    keeps H, z by Eq. 4 / Eq. 5 and a slot cache; the parallel form builds the S x S matrix)."""
    w, Q, K, V, phi_fn, psi_fn = _sequence_case(110, policy=policy)
    S = Q.shape[0]
    inst = lo.LessInstance(w.head_dim, w.rank, w.heavy, w.recent, phi_fn, psi_fn, policy=policy)
    outs, ev = [], []
    for t in range(S):
        r = inst.decode(Q[t], K[t], V[t])
        outs.append(r["out"])
        ev.append(r["evicted_pos"])
    eu = lo.eviction_schedule(ev, 0, S)
    assert (eu != lo.NEVER).sum() == S - inst.N and np.all(eu > np.arange(S))
    out, P = lo.masked_parallel_attention(Q, K, V, eu, phi_fn, psi_fn)
    assert np.allclose(P.sum(axis=1), 1.0) and np.all(np.triu(P, 1) == 0)
    assert np.allclose(out, np.stack(outs), rtol=1e-10, atol=1e-12)


def test_parallel_form_with_nothing_evicted_is_causal_softmax():
    w, Q, K, V, phi_fn, psi_fn = _sequence_case(111)
    S, D = Q.shape
    out, P = lo.masked_parallel_attention(Q, K, V, np.full(S, lo.NEVER), phi_fn, psi_fn)
    ref = torch.nn.functional.scaled_dot_product_attention(
        *(torch.as_tensor(a)[None, None] for a in (Q, K, V)), is_causal=True)[0, 0].numpy()
    assert np.allclose(out, ref, rtol=1e-10, atol=1e-12)


def test_parallel_form_with_everything_evicted_at_once_is_linear_attention():
    """exact_until[j] = j + 1: only the diagonal is exact, the rest of a row is the kernel
    phi(q_i) psi(k_j)^T; closed form with prefix sums (Eq. 6 for every prefix)."""
    w, Q, K, V, phi_fn, psi_fn = _sequence_case(112)
    S, D = Q.shape
    out, _ = lo.masked_parallel_attention(Q, K, V, np.arange(S) + 1, phi_fn, psi_fn)
    tQ, tK, tV = (torch.as_tensor(a) for a in (Q, K, V))
    phi, psi = torch.as_tensor(phi_fn(Q)), torch.as_tensor(psi_fn(K))
    Hpre = torch.cumsum(psi[:, :, None] * tV[:, None, :], dim=0) - psi[:, :, None] * tV[:, None, :]   # sum over j < i
    zpre = torch.cumsum(psi, dim=0) - psi
    d = torch.exp((tQ * tK).sum(1) / math.sqrt(D))
    num = d[:, None] * tV + torch.einsum("ir,ird->id", phi, Hpre)
    den = d + (phi * zpre).sum(1)
    assert np.allclose(out, (num / den[:, None]).numpy(), rtol=1e-10, atol=1e-12)


def test_parallel_form_mask_boundary_is_strict():
    """Key j is exact for query i = exact_until[j] - 1 and low-rank for i = exact_until[j]."""
    w, Q, K, V, phi_fn, psi_fn = _sequence_case(113, S=12)
    S, D = Q.shape
    eu = np.full(S, lo.NEVER)
    eu[2] = 7
    _, P = lo.masked_parallel_attention(Q, K, V, eu, phi_fn, psi_fn)
    e = np.exp(Q @ K.T / math.sqrt(D))
    low = phi_fn(Q) @ psi_fn(K).T
    for i, want in ((6, e[6, 2]), (7, low[7, 2])):
        row = np.where(np.arange(S) <= i, e[i], 0.0)
        if i >= 7:
            row[2] = low[i, 2]
        assert np.isclose(P[i, 2], want / row.sum(), rtol=1e-12)


def test_parallel_form_row_subset_equals_the_full_matrix_rows():
    w, Q, K, V, phi_fn, psi_fn = _sequence_case(114, S=30)
    eu = np.arange(30) + 1 + (np.arange(30) * 7) % 11
    out, P = lo.masked_parallel_attention(Q, K, V, eu, phi_fn, psi_fn)
    rows = [0, 3, 17, 29]
    out_r, P_r = lo.masked_parallel_attention(Q, K, V, eu, phi_fn, psi_fn, rows=rows)
    assert np.array_equal(out_r, out[rows]) or np.allclose(out_r, out[rows], rtol=1e-13, atol=0)
    assert np.allclose(P_r, P[rows], rtol=1e-13, atol=0)
