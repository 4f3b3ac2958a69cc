"""Shared machinery of the GPU parity tests: builds oracle instances for chosen
(batch, layer, head) instances and compares the library's results with them.

Tolerances (fp16 inputs, fp32 accumulation on the GPU, fp64 in the oracle):
  outputs            max-abs <= 2e-3 (fp16 outputs: plus half an fp16 ulp of the value, 2^-11 |x|)
  H, z, dH, dz       norm-wise relative <= 1e-3
  phi, psi           norm-wise relative <= 1e-3
  accumulated score  relative <= 2e-5 (+1e-7 absolute)
  kept / evicted     exact, except decisions whose two lowest keys differ by
                     less than 1e-4 relative (counted and reported)
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import less_oracle as lo
from paper_2402_09398_b200 import workloads as wl

OUT_TOL = 2e-3
REL_TOL = 1e-3
ACC_RTOL, ACC_ATOL = 2e-5, 1e-7
TIE_BAND = 1e-4


def rel_err(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    nb = np.linalg.norm(b)
    if nb == 0:
        return float(np.linalg.norm(a))
    return float(np.linalg.norm(a - b) / nb)


def head_weights(W, layer, head):
    return [W[n][layer, head].double().cpu().numpy() for n in
            ("w_phi1", "w_phi2", "w_psi1", "w_psi2", "w_psi3")]


def make_oracle(w, W, inst, flags=0, psi_scale=None, heavy=None, recent=None):
    b, layer, head = wl.instance_coords(w, inst)
    sc = None if psi_scale is None else psi_scale[layer, head].double().cpu().numpy()
    phi_fn, psi_fn = lo.make_mlp_maps(*head_weights(W, layer, head), sc)
    return lo.LessInstance(w.head_dim, w.rank, w.heavy if heavy is None else heavy,
                           w.recent if recent is None else recent, phi_fn, psi_fn,
                           score_norm="sparse" if flags & 1 else "less",
                           use_state=not (flags & 2), policy="lambda" if flags & 4 else ("tova" if flags & 8 else "h2o"))


def check_prefill(ctx, w, W, Q, K, V, instances, attn_out=None, flags=0, psi_scale=None,
                  layer_begin=0, heavy=None, recent=None):
    """Compare the library's post-prefill state of `instances` with the oracle's.
    Q, K, V: the tensors given to less_prefill, [B, Lc, H, S, D].  Returns a
    summary dict; raises AssertionError on a mismatch."""
    recs = ctx.export_state(instances)
    S = Q.shape[3]
    exempt = 0
    worst = {"out": 0.0, "H": 0.0, "z": 0.0, "acc": 0.0, "psi": 0.0}
    for inst, rec in zip(instances, recs):
        b, layer, head = wl.instance_coords(w, inst)
        lj = layer - layer_begin
        q, k, v = (t[b, lj, head].double().cpu().numpy() for t in (Q, K, V))
        orc = make_oracle(w, W, inst, flags, psi_scale, heavy, recent)
        out = orc.prefill(q, k, v)
        assert rec["t"] == S and rec["count"] == min(S, orc.N), (inst, rec["count"])
        if attn_out is not None:
            err = np.max(np.abs(attn_out[b, lj, head].double().cpu().numpy() - out)) if S else 0.0
            worst["out"] = max(worst["out"], float(err))
            assert err <= OUT_TOL, f"inst {inst}: prompt attention max-abs {err}"
        gpu_pos = rec["pos"].astype(np.int64)
        assert len(set(gpu_pos.tolist())) == len(gpu_pos), "duplicate positions in slots"
        assert np.all(np.diff(gpu_pos) > 0), "prefill slots must ascend in position"
        kept_o, kept_g = set(orc.pos.tolist()), set(gpu_pos.tolist())
        if kept_o != kept_g:
            # only candidates within the tie band of the threshold may differ
            acc_o = orc.prompt_acc
            cand = np.arange(S - orc.recent)
            thr = np.sort(acc_o[cand])[::-1][orc.heavy - 1] if orc.heavy > 0 else np.inf
            diff = kept_o ^ kept_g
            for pz in diff:
                assert pz < S - orc.recent, f"inst {inst}: recent token {pz} mis-kept"
                assert abs(acc_o[pz] - thr) <= TIE_BAND * abs(thr), \
                    f"inst {inst}: pos {pz} acc {acc_o[pz]} vs threshold {thr}"
            exempt += len(diff)
            assert len(kept_g) == len(kept_o)
        # rows and scores of the tokens both kept
        Kh, Vh = K[b, lj, head].cpu().numpy(), V[b, lj, head].cpu().numpy()
        assert np.array_equal(rec["K"], Kh[gpu_pos]) and np.array_equal(rec["V"], Vh[gpu_pos])
        acc_ref = orc.prompt_acc[gpu_pos]
        aerr = np.max(np.abs(rec["acc"] - acc_ref) / (np.abs(acc_ref) + 1e-30)) if len(gpu_pos) else 0.0
        worst["acc"] = max(worst["acc"], float(aerr))
        assert np.allclose(rec["acc"], acc_ref, rtol=1e-4, atol=1e-6), f"inst {inst}: acc rel {aerr}"
        if kept_o == kept_g and not (flags & 2):
            eH, ez = rel_err(rec["H"], orc.H), rel_err(rec["z"], orc.z)
            worst["H"], worst["z"] = max(worst["H"], eH), max(worst["z"], ez)
            assert eH <= REL_TOL and ez <= REL_TOL, f"inst {inst}: H rel {eH}, z rel {ez}"
            assert np.max(np.abs(rec["H"] - orc.H)) <= REL_TOL * max(np.max(np.abs(orc.H)), 1e-30)
        if flags & 2:
            assert not rec["H"].any() and not rec["z"].any()
        elif len(gpu_pos):
            psi_ref = orc.psi_fn(Kh[gpu_pos].astype(np.float64))
            ep = rel_err(rec["psi"], psi_ref)
            worst["psi"] = max(worst["psi"], ep)
            assert ep <= REL_TOL, f"inst {inst}: cached psi rel {ep}"
    return {"exempt": exempt, **worst}


class TeacherForced:
    """Runs decode steps on the library and checks each against one oracle step
    started from the library's own pre-step state."""

    def __init__(self, ctx, w, W, instances, flags=0, psi_scale=None, heavy=None, recent=None):
        self.ctx, self.w, self.instances, self.flags = ctx, w, list(instances), flags
        self.oracles = [make_oracle(w, W, i, flags, psi_scale, heavy, recent) for i in instances]
        self.exempt = 0
        self.evictions = 0
        self.worst = {"out": 0.0, "dH": 0.0, "dz": 0.0, "acc": 0.0, "phi": 0.0, "psi": 0.0,
                      "lr_num": 0.0, "lr_den": 0.0}
        dev = ctx.device
        self.evicted = torch.empty(ctx.instances, dtype=torch.int32, device=dev)
        self.f16_out = bool(flags & 32)

    def step(self, q, k, v):
        ctx, w = self.ctx, self.w
        pre = ctx.export_state(self.instances)
        out = ctx.decode_step(q, k, v, evicted_pos=self.evicted)
        post = ctx.export_state(self.instances)
        ev = self.evicted.cpu().numpy()
        out_h = out.reshape(-1, w.head_dim).cpu().numpy()
        phi_g, psi_g = ctx.read_feature_maps()
        qh = q.reshape(-1, w.head_dim).cpu().numpy().astype(np.float64)
        kh = k.reshape(-1, w.head_dim).cpu().numpy().astype(np.float64)
        vh = v.reshape(-1, w.head_dim).cpu().numpy().astype(np.float64)
        use_state = not (self.flags & 2)
        for inst, orc, a, b in zip(self.instances, self.oracles, pre, post):
            orc.import_state(a["pos"], a["K"], a["V"], a["acc"], a["H"], a["z"], a["t"])
            r = orc.decode(qh[inst], kh[inst], vh[inst])
            err = float(np.max(np.abs(out_h[inst] - r["out"])))
            self.worst["out"] = max(self.worst["out"], err)
            tol = OUT_TOL + (2.0 ** -11 * np.abs(r["out"]) if self.f16_out else 0.0)
            assert np.all(np.abs(out_h[inst] - r["out"]) <= tol), f"inst {inst} t={a['t']}: out max-abs {err}"
            if use_state:
                e1 = rel_err(phi_g[inst], orc.phi_fn(qh[inst][None])[0])
                e2 = rel_err(psi_g[inst], orc.psi_fn(kh[inst][None])[0])
                self.worst["phi"], self.worst["psi"] = max(self.worst["phi"], e1), max(self.worst["psi"], e2)
                assert e1 <= REL_TOL and e2 <= REL_TOL, f"inst {inst}: phi rel {e1}, psi rel {e2}"
                # the low-rank terms on their own (they are a small share of the output)
                lr_num_g = phi_g[inst].astype(np.float64) @ a["H"].astype(np.float64)
                lr_den_g = float(phi_g[inst].astype(np.float64) @ a["z"].astype(np.float64))
                if np.linalg.norm(r["lr_num"]) > 0:
                    e3 = rel_err(lr_num_g, r["lr_num"])
                    e4 = abs(lr_den_g - r["lr_den"]) / max(abs(r["lr_den"]), 1e-300)
                    self.worst["lr_num"] = max(self.worst["lr_num"], e3)
                    self.worst["lr_den"] = max(self.worst["lr_den"], e4)
                    assert e3 <= REL_TOL and e4 <= REL_TOL
            # eviction decision
            gpu_vic = int(ev[inst])
            exempt = False
            if gpu_vic != r["evicted_pos"]:
                assert r["tie_gap"] is not None and r["tie_gap"] < TIE_BAND, \
                    f"inst {inst} t={a['t']}: evicted {gpu_vic}, oracle {r['evicted_pos']}, gap {r['tie_gap']}"
                self.exempt += 1
                exempt = True
            if gpu_vic >= 0:
                self.evictions += 1
            assert b["t"] == a["t"] + 1
            # post-step bookkeeping: positions, rows, scores
            gpos = b["pos"].astype(np.int64)
            assert len(set(gpos.tolist())) == len(gpos)
            if not exempt:
                assert set(gpos.tolist()) == set(orc.pos.tolist()), f"inst {inst}: kept sets differ"
                order_g, order_o = np.argsort(gpos), np.argsort(orc.pos)
                assert np.array_equal(b["K"][order_g].astype(np.float64), orc.K[order_o])
                assert np.array_equal(b["V"][order_g].astype(np.float64), orc.V[order_o])
                acc_g, acc_o = b["acc"][order_g], orc.acc[order_o]
                aerr = float(np.max(np.abs(acc_g - acc_o) / (np.abs(acc_o) + 1e-30)))
                self.worst["acc"] = max(self.worst["acc"], aerr)
                assert np.allclose(acc_g, acc_o, rtol=ACC_RTOL, atol=ACC_ATOL), f"inst {inst}: acc rel {aerr}"
                if use_state and r["dH"] is not None:
                    dH_g = b["H"].astype(np.float64) - a["H"].astype(np.float64)
                    dz_g = b["z"].astype(np.float64) - a["z"].astype(np.float64)
                    # increments are compared against the increment, with the rounding of
                    # adding them into an fp32 H of norm |H| allowed for
                    slack_H = 2e-7 * np.linalg.norm(a["H"]) / max(np.linalg.norm(r["dH"]), 1e-300)
                    slack_z = 2e-7 * np.linalg.norm(a["z"]) / max(np.linalg.norm(r["dz"]), 1e-300)
                    eH, ez = rel_err(dH_g, r["dH"]), rel_err(dz_g, r["dz"])
                    self.worst["dH"] = max(self.worst["dH"], eH)
                    self.worst["dz"] = max(self.worst["dz"], ez)
                    assert eH <= REL_TOL + slack_H, f"inst {inst}: dH rel {eH}"
                    assert ez <= REL_TOL + slack_z, f"inst {inst}: dz rel {ez}"
                elif use_state:
                    assert np.array_equal(a["H"], b["H"]) and np.array_equal(a["z"], b["z"])
            if self.flags & 2:
                assert not b["H"].any() and not b["z"].any()
        return out


def brute_force_state(w, W, inst, K_hist, V_hist, evicted_positions, psi_scale=None):
    """Eq. 6: H, z as plain sums over a list of evicted positions."""
    orc = make_oracle(w, W, inst, 0, psi_scale)
    ev = np.asarray(sorted(evicted_positions), dtype=np.int64)
    if ev.size == 0:
        return np.zeros((w.rank, w.head_dim)), np.zeros(w.rank)
    psi = orc.psi_fn(K_hist[ev])
    return psi.T @ V_hist[ev], psi.sum(axis=0)


# --------------------------------------------------------------------------- #
# grouped query heads over one KV head (Section 3.2, multi-query attention)
# --------------------------------------------------------------------------- #
def make_group_oracle(w, W, inst, flags=0, psi_scale=None):
    b, layer, head = wl.instance_coords(w, inst)
    G = w.group
    sc = None if psi_scale is None else psi_scale[layer, head].double().cpu().numpy()
    psi_w = [W[n][layer, head].double().cpu().numpy() for n in ("w_psi1", "w_psi2", "w_psi3")]
    phi_fns = []
    for g in range(G):
        w1, w2 = (W[n][layer, head * G + g].double().cpu().numpy() for n in ("w_phi1", "w_phi2"))
        phi_fns.append(lo.make_mlp_maps(w1, w2, *psi_w, sc)[0])
    psi_fn = lo.make_mlp_maps(W["w_phi1"][layer, head * G].double().cpu().numpy(),
                              W["w_phi2"][layer, head * G].double().cpu().numpy(), *psi_w, sc)[1]
    return lo.LessGroup(w.head_dim, w.rank, w.heavy, w.recent, phi_fns, psi_fn,
                        score_norm="sparse" if flags & 1 else "less", use_state=not (flags & 2),
                        policy="lambda" if flags & 4 else "h2o")


def check_prefill_group(ctx, w, W, Q, K, V, instances, attn_out=None, flags=0, psi_scale=None, layer_begin=0):
    """Grouped version of check_prefill: Q [B, Lc, H*G, S, D], K, V [B, Lc, H, S, D];
    attn_out [B, Lc, H*G, S, D]."""
    recs = ctx.export_state(instances)
    S, G = Q.shape[3], w.group
    exempt = 0
    worst = {"out": 0.0, "H": 0.0, "z": 0.0, "acc": 0.0}
    for inst, rec in zip(instances, recs):
        b, layer, head = wl.instance_coords(w, inst)
        lj = layer - layer_begin
        q = Q[b, lj, head * G:(head + 1) * G].double().cpu().numpy()
        k, v = (t[b, lj, head].double().cpu().numpy() for t in (K, V))
        orc = make_group_oracle(w, W, inst, flags, psi_scale)
        out = orc.prefill(q, k, v)
        assert rec["t"] == S and rec["count"] == min(S, orc.N), (inst, rec["count"])
        if attn_out is not None and S:
            err = float(np.max(np.abs(attn_out[b, lj, head * G:(head + 1) * G].double().cpu().numpy() - out)))
            worst["out"] = max(worst["out"], err)
            assert err <= OUT_TOL, f"inst {inst}: prompt attention max-abs {err}"
        gpu_pos = rec["pos"].astype(np.int64)
        assert np.all(np.diff(gpu_pos) > 0), "prefill slots must ascend in position"
        kept_o, kept_g = set(orc.pos.tolist()), set(gpu_pos.tolist())
        if kept_o != kept_g:
            acc_o = orc.prompt_acc
            cand = np.arange(S - orc.recent)
            thr = np.sort(acc_o[cand])[::-1][orc.heavy - 1] if orc.heavy > 0 else np.inf
            diff = kept_o ^ kept_g
            for pz in diff:
                assert pz < S - orc.recent, f"inst {inst}: recent token {pz} mis-kept"
                assert abs(acc_o[pz] - thr) <= TIE_BAND * abs(thr), f"inst {inst}: pos {pz}"
            exempt += len(diff)
            assert len(kept_g) == len(kept_o)
        Kh, Vh = K[b, lj, head].cpu().numpy(), V[b, lj, head].cpu().numpy()
        assert np.array_equal(rec["K"], Kh[gpu_pos]) and np.array_equal(rec["V"], Vh[gpu_pos])
        acc_ref = orc.prompt_acc[gpu_pos]
        aerr = np.max(np.abs(rec["acc"] - acc_ref) / (np.abs(acc_ref) + 1e-30)) if len(gpu_pos) else 0.0
        worst["acc"] = max(worst["acc"], float(aerr))
        assert np.allclose(rec["acc"], acc_ref, rtol=1e-4, atol=1e-6), f"inst {inst}: acc rel {aerr}"
        if kept_o == kept_g and not (flags & 2):
            eH, ez = rel_err(rec["H"], orc.H), rel_err(rec["z"], orc.z)
            worst["H"], worst["z"] = max(worst["H"], eH), max(worst["z"], ez)
            assert eH <= REL_TOL and ez <= REL_TOL, f"inst {inst}: H rel {eH}, z rel {ez}"
    return {"exempt": exempt, **worst}


class GroupTeacherForced:
    """TeacherForced for G query heads per KV head: every step of the library is checked
    against one LessGroup step started from the library's own pre-step state."""

    def __init__(self, ctx, w, W, instances, flags=0, psi_scale=None):
        self.ctx, self.w, self.instances, self.flags = ctx, w, list(instances), flags
        self.oracles = [make_group_oracle(w, W, i, flags, psi_scale) for i in instances]
        self.exempt = 0
        self.evictions = 0
        self.worst = {"out": 0.0, "dH": 0.0, "dz": 0.0, "acc": 0.0, "phi": 0.0, "psi": 0.0}
        self.evicted = torch.empty(ctx.instances, dtype=torch.int32, device=ctx.device)
        self.f16_out = bool(flags & 32)

    def step(self, q, k, v):
        ctx, w, G, D = self.ctx, self.w, self.w.group, self.w.head_dim
        pre = ctx.export_state(self.instances)
        out = ctx.decode_step(q, k, v, evicted_pos=self.evicted)
        post = ctx.export_state(self.instances)
        ev = self.evicted.cpu().numpy()
        out_h = out.reshape(-1, G, D).cpu().numpy()
        phi_g, psi_g = ctx.read_feature_maps()
        phi_g = phi_g.reshape(-1, G, w.rank)
        qh = q.reshape(-1, G, D).cpu().numpy().astype(np.float64)
        kh = k.reshape(-1, D).cpu().numpy().astype(np.float64)
        vh = v.reshape(-1, D).cpu().numpy().astype(np.float64)
        use_state = not (self.flags & 2)
        for inst, orc, a, b in zip(self.instances, self.oracles, pre, post):
            orc.import_state(a["pos"], a["K"], a["V"], a["acc"], a["H"], a["z"], a["t"])
            r = orc.decode(qh[inst], kh[inst], vh[inst])
            err = float(np.max(np.abs(out_h[inst] - r["out"])))
            self.worst["out"] = max(self.worst["out"], err)
            tol = OUT_TOL + (2.0 ** -11 * np.abs(r["out"]) if self.f16_out else 0.0)
            assert np.all(np.abs(out_h[inst] - r["out"]) <= tol), f"inst {inst} t={a['t']}: out max-abs {err}"
            if use_state:
                for g in range(G):
                    e1 = rel_err(phi_g[inst, g], orc.phi_fns[g](qh[inst, g][None])[0])
                    self.worst["phi"] = max(self.worst["phi"], e1)
                    assert e1 <= REL_TOL, f"inst {inst} head {g}: phi rel {e1}"
                e2 = rel_err(psi_g[inst], orc.psi_fn(kh[inst][None])[0])
                self.worst["psi"] = max(self.worst["psi"], e2)
                assert e2 <= REL_TOL, f"inst {inst}: psi rel {e2}"
            gpu_vic = int(ev[inst])
            exempt = False
            if gpu_vic != r["evicted_pos"]:
                assert r["tie_gap"] is not None and r["tie_gap"] < TIE_BAND, \
                    f"inst {inst} t={a['t']}: evicted {gpu_vic}, oracle {r['evicted_pos']}, gap {r['tie_gap']}"
                self.exempt += 1
                exempt = True
            if gpu_vic >= 0:
                self.evictions += 1
            assert b["t"] == a["t"] + 1
            gpos = b["pos"].astype(np.int64)
            assert len(set(gpos.tolist())) == len(gpos)
            if not exempt:
                assert set(gpos.tolist()) == set(orc.pos.tolist()), f"inst {inst}: kept sets differ"
                order_g, order_o = np.argsort(gpos), np.argsort(orc.pos)
                assert np.array_equal(b["K"][order_g].astype(np.float64), orc.K[order_o])
                assert np.array_equal(b["V"][order_g].astype(np.float64), orc.V[order_o])
                acc_g, acc_o = b["acc"][order_g], orc.acc[order_o]
                aerr = float(np.max(np.abs(acc_g - acc_o) / (np.abs(acc_o) + 1e-30)))
                self.worst["acc"] = max(self.worst["acc"], aerr)
                assert np.allclose(acc_g, acc_o, rtol=ACC_RTOL, atol=ACC_ATOL), f"inst {inst}: acc rel {aerr}"
                if use_state and r["dH"] is not None:
                    dH_g = b["H"].astype(np.float64) - a["H"].astype(np.float64)
                    dz_g = b["z"].astype(np.float64) - a["z"].astype(np.float64)
                    slack_H = 2e-7 * np.linalg.norm(a["H"]) / max(np.linalg.norm(r["dH"]), 1e-300)
                    slack_z = 2e-7 * np.linalg.norm(a["z"]) / max(np.linalg.norm(r["dz"]), 1e-300)
                    eH, ez = rel_err(dH_g, r["dH"]), rel_err(dz_g, r["dz"])
                    self.worst["dH"], self.worst["dz"] = max(self.worst["dH"], eH), max(self.worst["dz"], ez)
                    assert eH <= REL_TOL + slack_H and ez <= REL_TOL + slack_z, f"inst {inst}: dH {eH} dz {ez}"
                elif use_state:
                    assert np.array_equal(a["H"], b["H"]) and np.array_equal(a["z"], b["z"])
        return out
