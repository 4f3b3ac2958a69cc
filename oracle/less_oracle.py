"""fp64 CPU oracle of one LESS head instance (arxiv 2402.09398).

TEST INFRASTRUCTURE ONLY: nothing in the product package may import this file.
It shares no code with the CUDA path.  Everything is numpy in float64 on the
exact fp16 input values widened to double; there is no blocking or fusion
beyond what the equations state (the prompt phase walks the causal attention
matrix in row blocks only to bound memory; each row is the plain softmax).

One object = one (batch, layer, head) instance, because every instance of the
method is independent of every other.

Paper passages followed:
  * Eq. 1 / Eq. 2   feature maps phi, psi (per-head MLPs, GELU, absolute value)
  * Eq. 3           attention synthesis, ONE normalisation over sparse + low-rank
  * Eq. 4 / Eq. 5   H, z absorb every discarded (k, v)
  * Eq. 6           expanded recursion (used by the tests as an invariant)
  * Algorithm 1     order inside a generation step
  * Section 2.1 / Section 4  H2O policy: accumulated attention probabilities,
                    equal heavy/recent split, even-floored token counts (Table 1)
  * Section 3.1     the prompt phase is regular attention (H_0 = 0, z_0 = 0)
  * Section 4       Lambda-masking as the sparse policy: the first tokens plus the most recent ones;
                    TOVA is named there without a definition (the rule of the cited work is used)
  * Section 3.2 (Inexpensive Training), Section 4.1   the parallel form used for training and for the
                    language-modelling evaluation: the whole causal attention matrix at once, entries
                    the sparse policy does not keep replaced by phi(q_i) psi(k_j)^T

Readings where the paper is silent (none of them is fixed by a printed number,
so they are "parity unpinned" by the paper and fixed by the design notes that
come with this code): exact erf GELU without biases; the learnable psi scalars sit after each
GELU of psi; the accumulated probabilities use Eq. 3's full denominator (flag
for the sparse-only one); the new token's own probability seeds its score and
the diagonal counts in the prompt column sums; "recent" = the `recent` highest
positions including the current token; ties evict the lowest position; the
prompt is scored in one shot and the policy applied once at its end.
"""
from __future__ import annotations

import math
from typing import Callable, Optional

import numpy as np
from scipy.special import erf as _erf

_SQRT2 = math.sqrt(2.0)


# --------------------------------------------------------------------------- #
# Feature maps (Eq. 1, Eq. 2)
# --------------------------------------------------------------------------- #
def gelu(x: np.ndarray) -> np.ndarray:
    """Exact GELU, x * Phi(x) (Section 3.2: all nonlinearities are GELUs)."""
    x = np.asarray(x, dtype=np.float64)
    return 0.5 * x * (1.0 + _erf(x / _SQRT2))


def phi_map(q: np.ndarray, w1: np.ndarray, w2: np.ndarray) -> np.ndarray:
    """Eq. 1: phi(q) = | gelu( gelu(q W1) W2 ) |, W1 [D,R'], W2 [R',R]."""
    q = np.asarray(q, dtype=np.float64)
    return np.abs(gelu(gelu(q @ w1.astype(np.float64)) @ w2.astype(np.float64)))


def psi_map(k: np.ndarray, w1: np.ndarray, w2: np.ndarray, w3: np.ndarray,
            scale: Optional[np.ndarray] = None) -> np.ndarray:
    """Eq. 2: psi(k) = | gelu( gelu(k W1) W2 ) W3 |, W3 [R,R].

    `scale` = the two learnable scalars Section 3.2 places inside psi, read as
    one multiplier after each GELU; None means both are 1.
    """
    k = np.asarray(k, dtype=np.float64)
    c1, c2 = (1.0, 1.0) if scale is None else (float(scale[0]), float(scale[1]))
    h1 = c1 * gelu(k @ w1.astype(np.float64))
    h2 = c2 * gelu(h1 @ w2.astype(np.float64))
    return np.abs(h2 @ w3.astype(np.float64))


# --------------------------------------------------------------------------- #
# Budgets (Section 4, Table 1)
# --------------------------------------------------------------------------- #
def h2o_token_count(percent: float, max_len: int) -> int:
    """Tokens cached at `percent` % of the model's max context, rounded down
    to the nearest even number so H2O splits evenly (Section 4, Table 1)."""
    n = int(math.floor(percent * max_len / 100.0 + 1e-9))
    return n - (n % 2)


def budget_from_fraction(frac: float, prompt_len: int) -> int:
    """Slots for one half (heavy or recent) when a workload states the budget
    as a fraction of the prompt length: floor(frac * S)."""
    return int(math.floor(frac * prompt_len + 1e-9))


# --------------------------------------------------------------------------- #
# One head instance
# --------------------------------------------------------------------------- #
class LessInstance:
    """State of one (batch, layer, head): kept entries, H, z, evicted log."""

    def __init__(self, head_dim: int, rank: int, heavy: int, recent: int,
                 phi_fn: Callable[[np.ndarray], np.ndarray],
                 psi_fn: Callable[[np.ndarray], np.ndarray],
                 score_norm: str = "less", use_state: bool = True, policy: str = "h2o"):
        if recent < 1 or heavy < 0:
            raise ValueError("need recent >= 1 and heavy >= 0")
        if policy not in ("h2o", "lambda", "tova"):
            raise ValueError("policy is 'h2o', 'lambda' or 'tova'")
        # 'lambda' = Lambda-masking (Section 4: a handful of first positions plus the recent window
        # are cached): `heavy` counts the first tokens that are always kept, `recent` the window;
        # accumulated scores play no role in it.
        # 'tova' = the third policy Section 4 names.  The paper gives no definition of it; this is
        # the published rule of the work it cites, per head: whenever the cache overflows, the
        # entry with the lowest attention probability OF THE CURRENT QUERY leaves, the newest one
        # included and no window protected; `heavy + recent` only sets the slot count.  Under the
        # one-shot reading of the prompt phase the current query at its end is the last prompt token.
        self.policy = policy
        if score_norm not in ("less", "sparse"):
            raise ValueError("score_norm is 'less' or 'sparse'")
        self.D, self.R = int(head_dim), int(rank)
        self.heavy, self.recent = int(heavy), int(recent)
        self.N = self.heavy + self.recent
        self.phi_fn, self.psi_fn = phi_fn, psi_fn
        self.score_norm, self.use_state = score_norm, bool(use_state)
        self.reset()

    # -- state ------------------------------------------------------------- #
    def reset(self) -> None:
        D, R = self.D, self.R
        self.pos = np.zeros(0, dtype=np.int64)
        self.K = np.zeros((0, D))
        self.V = np.zeros((0, D))
        self.acc = np.zeros(0)
        self.H = np.zeros((R, D))          # H_0 = 0 (Section 2.2)
        self.z = np.zeros(R)               # z_0 = 0
        self.t = 0                         # tokens seen so far
        self.evicted = []                  # positions, in eviction order

    def import_state(self, pos, K, V, acc, H, z, t) -> None:
        """Teacher forcing: take over a state produced elsewhere."""
        self.pos = np.asarray(pos, dtype=np.int64).copy()
        self.K = np.asarray(K, dtype=np.float64).copy()
        self.V = np.asarray(V, dtype=np.float64).copy()
        self.acc = np.asarray(acc, dtype=np.float64).copy()
        self.H = np.asarray(H, dtype=np.float64).copy()
        self.z = np.asarray(z, dtype=np.float64).copy()
        self.t = int(t)

    # -- prompt phase ------------------------------------------------------ #
    def prefill(self, Q: np.ndarray, K: np.ndarray, V: np.ndarray,
                row_block: int = 512) -> np.ndarray:
        """Prompt phase (Section 3.1: regular attention), then the policy once.

        Returns the causal attention output [S, D].  Afterwards the instance
        holds min(S, N) kept entries with their accumulated scores, and H, z
        hold the bulk form of Eq. 4 / Eq. 5 over the discarded set D_1.
        """
        self.reset()
        Q = np.asarray(Q, dtype=np.float64)
        K = np.asarray(K, dtype=np.float64)
        V = np.asarray(V, dtype=np.float64)
        S, D = Q.shape
        out = np.zeros((S, D))
        acc = np.zeros(S)
        inv_sqrt_d = 1.0 / math.sqrt(D)
        for r0 in range(0, S, row_block):
            r1 = min(S, r0 + row_block)
            s = (Q[r0:r1] @ K[:r1].T) * inv_sqrt_d            # rows r0..r1-1, cols 0..r1-1
            col = np.arange(r1)[None, :]
            row = np.arange(r0, r1)[:, None]
            s = np.where(col <= row, s, -np.inf)              # causal
            s = s - s.max(axis=1, keepdims=True)
            e = np.exp(s)
            P = e / e.sum(axis=1, keepdims=True)              # softmax rows
            out[r0:r1] = P @ V[:r1]
            acc[:r1] += P.sum(axis=0)                         # H2O: column sums, diagonal included
            if r1 == S:
                last_row = P[-1].copy()                       # TOVA: the last query's probabilities
        self.t = S
        pos = np.arange(S, dtype=np.int64)
        if self.policy == "lambda":
            acc = np.zeros(S)                                 # the policy keeps no scores
        elif self.policy == "tova":
            acc = last_row                                    # attention of the last prompt query
        if S <= self.N:
            keep = pos
            evict = pos[:0]
        else:
            if self.policy == "lambda":
                evict = pos[self.heavy: S - self.recent]      # everything between the first tokens and the window
            elif self.policy == "tova":
                order = np.lexsort((pos, acc))                # key (p, pos) ascending, nothing protected
                evict = np.sort(pos[order[: S - self.N]])
            else:
                cand = pos[: S - self.recent]                 # recent window is protected
                order = np.lexsort((cand, acc[cand]))         # key (acc, pos) ascending
                evict = np.sort(cand[order[: S - self.N]])
            keep_mask = np.ones(S, dtype=bool)
            keep_mask[evict] = False
            keep = pos[keep_mask]
        self.pos = keep.copy()
        self.K, self.V, self.acc = K[keep].copy(), V[keep].copy(), acc[keep].copy()
        if evict.size and self.use_state:
            psi = self.psi_fn(K[evict])                       # [n_ev, R]
            self.H = psi.T @ V[evict]                         # Eq. 4 summed over D_1
            self.z = psi.sum(axis=0)                          # Eq. 5 summed over D_1
        self.evicted = [int(p) for p in evict]
        self.prompt_acc = acc
        return out

    # -- one generation step (Algorithm 1) --------------------------------- #
    def decode(self, q: np.ndarray, k: np.ndarray, v: np.ndarray) -> dict:
        q = np.asarray(q, dtype=np.float64)
        k = np.asarray(k, dtype=np.float64)
        v = np.asarray(v, dtype=np.float64)
        t = self.t
        # K', V' = cached entries with the new pair appended (Algorithm 1)
        Kp = np.vstack([self.K, k[None, :]])
        Vp = np.vstack([self.V, v[None, :]])
        s = (Kp @ q) / math.sqrt(self.D)
        e = np.exp(s)                                          # Eq. 3, literal (fp64 range)
        phi_q = self.phi_fn(q[None, :])[0]
        lr_num = phi_q @ self.H                                # phi(q) H_t
        lr_den = float(phi_q @ self.z)                         # phi(q) z_t^T
        num = lr_num + e @ Vp
        den_sparse = float(e.sum())
        den = lr_den + den_sparse
        out = num / den
        # H2O: accumulate this step's attention probabilities
        p = e / (den if self.score_norm == "less" else den_sparse)
        if self.policy == "tova":
            acc = p.copy()                                     # TOVA scores = this query's probabilities
        else:
            acc = np.concatenate([self.acc + p[:-1], p[-1:]])
        pos = np.concatenate([self.pos, np.array([t], dtype=np.int64)])
        evicted_pos, gap, dH, dz = -1, None, None, None
        if pos.size > self.N:
            if self.policy == "lambda":
                cand = np.nonzero(pos >= self.heavy)[0]       # never one of the first tokens
                order = np.argsort(pos[cand])                 # the oldest of the others leaves the window
            elif self.policy == "tova":
                cand = np.arange(pos.size)                    # every entry, the new pair included
                order = np.lexsort((pos, acc))
            else:
                cand = np.nonzero(pos <= t - self.recent)[0]
                order = np.lexsort((pos[cand], acc[cand]))    # (acc, pos) ascending
            vic = int(cand[order[0]])
            if cand.size > 1 and self.policy != "lambda":
                a0, a1 = acc[cand[order[0]]], acc[cand[order[1]]]
                gap = abs(a1 - a0) / max(abs(a0), abs(a1), 1e-300)
            evicted_pos = int(pos[vic])
            if self.use_state:
                psi = self.psi_fn(Kp[vic][None, :])[0]
                dH = np.outer(psi, Vp[vic])                    # Eq. 4
                dz = psi                                       # Eq. 5
                self.H = self.H + dH
                self.z = self.z + dz
            self.evicted.append(evicted_pos)
            keep = np.ones(pos.size, dtype=bool)
            keep[vic] = False
            pos, acc, Kp, Vp = pos[keep], acc[keep], Kp[keep], Vp[keep]
        self.pos, self.acc, self.K, self.V = pos, acc, Kp, Vp
        self.t = t + 1
        return {"out": out, "evicted_pos": evicted_pos, "tie_gap": gap,
                "p": p, "den": den, "lr_num": lr_num, "lr_den": lr_den,
                "dH": dH, "dz": dz}


class LessGroup:
    """One KV head shared by G query heads (multi-query / grouped-query attention).

    Section 3.2 extends H2O to multi-query attention by summing the attention scores of all query
    heads before it decides which pair to evict.  Reading taken here: the cache
    (kept K, V), the accumulated scores and the low-rank state H, z belong to the KV head (psi
    acts on keys, so H = sum psi(k)^T v does not depend on the query head); every query head g has
    its own phi_g and its own Eq. 3 over the shared cache and state; the H2O score of an entry
    grows by the sum over g of the probabilities p_{g,i}; one entry is evicted per step for all G
    heads.  Policies: 'h2o' and 'lambda' (TOVA is left per head).  With G = 1 this is LessInstance.
    """

    def __init__(self, head_dim, rank, heavy, recent, phi_fns, psi_fn, score_norm="less",
                 use_state=True, policy="h2o"):
        if policy not in ("h2o", "lambda"):
            raise ValueError("grouped heads support the 'h2o' and 'lambda' policies")
        self.G = len(phi_fns)
        self.phi_fns = list(phi_fns)
        # bookkeeping (slots, scores, state, eviction) is that of a single instance
        self.core = LessInstance(head_dim, rank, heavy, recent, phi_fns[0], psi_fn, score_norm, use_state, policy)

    # the shared state, as LessInstance exposes it
    def __getattr__(self, name):
        if name in ("pos", "K", "V", "acc", "H", "z", "t", "evicted", "N", "heavy", "recent", "prompt_acc",
                    "psi_fn", "import_state"):
            return getattr(self.core, name)
        raise AttributeError(name)

    def prefill(self, Q, K, V, row_block=512):
        """Q [G, S, D]; K, V [S, D].  Returns the G causal attention outputs [G, S, D]."""
        c = self.core
        Q = np.asarray(Q, dtype=np.float64)
        K = np.asarray(K, dtype=np.float64)
        V = np.asarray(V, dtype=np.float64)
        G, S, D = Q.shape
        c.reset()
        out = np.zeros((G, S, D))
        acc = np.zeros(S)
        for g in range(G):
            for r0 in range(0, S, row_block):
                r1 = min(S, r0 + row_block)
                s = (Q[g, r0:r1] @ K[:r1].T) / math.sqrt(D)
                s = np.where(np.arange(r1)[None, :] <= np.arange(r0, r1)[:, None], s, -np.inf)
                e = np.exp(s - s.max(axis=1, keepdims=True))
                P = e / e.sum(axis=1, keepdims=True)
                out[g, r0:r1] = P @ V[:r1]
                acc[:r1] += P.sum(axis=0)                     # summed over rows and over the G heads
        c.t = S
        pos = np.arange(S, dtype=np.int64)
        if c.policy == "lambda":
            acc = np.zeros(S)
        if S <= c.N:
            keep, evict = pos, pos[:0]
        else:
            if c.policy == "lambda":
                evict = pos[c.heavy: S - c.recent]
            else:
                cand = pos[: S - c.recent]
                order = np.lexsort((cand, acc[cand]))
                evict = np.sort(cand[order[: S - c.N]])
            mask = np.ones(S, dtype=bool)
            mask[evict] = False
            keep = pos[mask]
        c.pos, c.K, c.V, c.acc = keep.copy(), K[keep].copy(), V[keep].copy(), acc[keep].copy()
        if evict.size and c.use_state:
            psi = c.psi_fn(K[evict])
            c.H, c.z = psi.T @ V[evict], psi.sum(axis=0)
        c.evicted = [int(p) for p in evict]
        c.prompt_acc = acc
        return out

    def decode(self, q, k, v):
        """q [G, D]; k, v [D].  One step for the G query heads of this KV head."""
        c = self.core
        q = np.asarray(q, dtype=np.float64)
        k = np.asarray(k, dtype=np.float64)
        v = np.asarray(v, dtype=np.float64)
        t = c.t
        Kp, Vp = np.vstack([c.K, k[None]]), np.vstack([c.V, v[None]])
        outs, p_sum, lr_nums, lr_dens = [], np.zeros(Kp.shape[0]), [], []
        for g in range(self.G):
            e = np.exp((Kp @ q[g]) / math.sqrt(c.D))                 # Eq. 3 for head g
            phi = self.phi_fns[g](q[g][None])[0]
            lr_num, lr_den = phi @ c.H, float(phi @ c.z)
            den_sparse = float(e.sum())
            den = lr_den + den_sparse
            outs.append((lr_num + e @ Vp) / den)
            p_sum += e / (den if c.score_norm == "less" else den_sparse)
            lr_nums.append(lr_num)
            lr_dens.append(lr_den)
        acc = np.concatenate([c.acc + p_sum[:-1], p_sum[-1:]])       # aggregated over the heads
        pos = np.concatenate([c.pos, np.array([t], dtype=np.int64)])
        evicted_pos, gap, dH, dz = -1, None, None, None
        if pos.size > c.N:
            if c.policy == "lambda":
                cand = np.nonzero(pos >= c.heavy)[0]
                order = np.argsort(pos[cand])
            else:
                cand = np.nonzero(pos <= t - c.recent)[0]
                order = np.lexsort((pos[cand], acc[cand]))
            vic = int(cand[order[0]])
            if cand.size > 1 and c.policy == "h2o":
                a0, a1 = acc[cand[order[0]]], acc[cand[order[1]]]
                gap = abs(a1 - a0) / max(abs(a0), abs(a1), 1e-300)
            evicted_pos = int(pos[vic])
            if c.use_state:
                psi = c.psi_fn(Kp[vic][None])[0]
                dH, dz = np.outer(psi, Vp[vic]), psi
                c.H, c.z = c.H + dH, c.z + dz
            c.evicted.append(evicted_pos)
            keep = np.ones(pos.size, dtype=bool)
            keep[vic] = False
            pos, acc, Kp, Vp = pos[keep], acc[keep], Kp[keep], Vp[keep]
        c.pos, c.acc, c.K, c.V = pos, acc, Kp, Vp
        c.t = t + 1
        return {"out": np.stack(outs), "evicted_pos": evicted_pos, "tie_gap": gap, "p": p_sum,
                "lr_num": np.stack(lr_nums), "lr_den": np.array(lr_dens), "dH": dH, "dz": dz}


def make_mlp_maps(w_phi1, w_phi2, w_psi1, w_psi2, w_psi3, psi_scale=None):
    """phi/psi callables of one head from its weight matrices."""
    def phi_fn(x):
        return phi_map(x, w_phi1, w_phi2)

    def psi_fn(x):
        return psi_map(x, w_psi1, w_psi2, w_psi3, psi_scale)
    return phi_fn, psi_fn


def hellinger(p: np.ndarray, q: np.ndarray) -> float:
    """Eq. 7: || sqrt(p) - sqrt(q) ||_2 / sqrt(2)."""
    p = np.asarray(p, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    return float(np.linalg.norm(np.sqrt(p) - np.sqrt(q)) / _SQRT2)


NEVER = np.iinfo(np.int32).max


def masked_parallel_attention(Q, K, V, exact_until, phi_fn, psi_fn, rows=None):
    """The parallel form (Section 3.2, Inexpensive Training; Section 4.1): every row of the causal
    attention matrix at once.  Entry (i, j), j <= i, is exp(q_i . k_j / sqrt(D)) while key j is still
    in the sparse cache when query i attends, i.e. i < exact_until[j], and phi(q_i) psi(k_j)^T from
    then on (Section 3.2: the kernel functions supply what the sparse cache no longer holds); each
    row is normalised once, as in Eq. 3:

        out_i = sum_j A_ij v_j / sum_j A_ij.

    The sparse policies here discard a pair once and for all, so one integer per key describes the
    mask: exact_until[j] = 1 + (the step at whose end j was evicted), NEVER if it stays.
    Q, K, V: [S, D]; returns (out [S, D], A / row sums [S, S]).  With `rows` (query positions) only
    those rows are formed: out [len(rows), D], P [len(rows), S]; the rows do not depend on each other."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    eu = np.asarray(exact_until, dtype=np.int64)
    S, D = Q.shape
    qi = np.arange(S) if rows is None else np.asarray(rows, dtype=np.int64)
    i = qi[:, None]
    j = np.arange(S)[None, :]
    causal = j <= i
    exact = causal & (i < eu[None, :])
    A_exact = np.exp((Q[qi] @ K.T) / math.sqrt(D))
    A_low = phi_fn(Q[qi]) @ psi_fn(K).T
    A = np.where(exact, A_exact, np.where(causal, A_low, 0.0))
    P = A / A.sum(axis=1, keepdims=True)
    return P @ V, P


def eviction_schedule(evicted_positions, first_step, S):
    """exact_until of a sequence of S tokens from the list of positions a sequential run evicted:
    evicted_positions[n] is the position discarded at the end of step first_step + n (-1 = none)."""
    eu = np.full(S, NEVER, dtype=np.int64)
    for n, pos in enumerate(evicted_positions):
        if pos >= 0:
            eu[pos] = first_step + n + 1
    return eu
