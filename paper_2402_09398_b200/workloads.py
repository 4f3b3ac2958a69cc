"""Seeded synthetic inputs for the LESS hot path.

This module holds NO arithmetic of the method: only shapes, seeds and random
draws.  It serves both the CUDA path and the CPU oracle, so that both see the
same fp16 bits.  The five named workloads follow the benchmark configurations
(Llama-2 attention shapes, N(0,1) fp16 Q/K/V, a sparse set of keys scaled x4 to
create heavy hitters, feature-map weights ~ N(0, 0.02^2)); they stand in for
the padded synthetic prompts the paper measures with (Section 4.3).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Dict, Optional, Tuple

import torch

# kinds of random stream; seed = (cfg_id * 1000 + kind) * 100003 + index
_Q, _K, _V, _W, _MASK, _DQ, _DK, _DV, _DMASK = range(9)


@dataclass(frozen=True)
class Workload:
    cfg_id: int
    batch: int
    layers: int
    heads: int
    head_dim: int
    prompt: int            # S
    steps: int             # T decode steps
    heavy: int
    recent: int
    rank: int              # R
    hidden: int = 512      # R' (Section 3.2)
    heavy_rule: str = "none"      # "every" | "bernoulli" | "none"
    heavy_param: float = 0.0      # period (every) or probability (bernoulli)
    sink_prefix: int = 0          # first tokens whose keys are scaled too
    key_boost: float = 4.0
    weight_std: float = 0.02
    group: int = 1                # query heads per KV head (`heads` counts KV heads)

    @property
    def instances(self) -> int:
        return self.batch * self.layers * self.heads

    @property
    def slots(self) -> int:
        return self.heavy + self.recent

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


def _half_budget(frac: float, prompt: int) -> int:
    return int(math.floor(frac * prompt + 1e-9))


CONFIGS: Dict[int, Workload] = {
    1: Workload(1, 1, 1, 8, 128, 256, 32, 32, 32, 8, heavy_rule="every", heavy_param=64),
    2: Workload(2, 1, 32, 32, 128, 2048, 256, _half_budget(0.05, 2048), _half_budget(0.05, 2048), 8,
                heavy_rule="bernoulli", heavy_param=0.01),
    3: Workload(3, 64, 32, 32, 128, 1024, 128, _half_budget(0.10, 1024), _half_budget(0.10, 1024), 8,
                heavy_rule="bernoulli", heavy_param=0.01),
    4: Workload(4, 4, 40, 40, 128, 16384, 512, _half_budget(0.02, 16384), _half_budget(0.02, 16384), 16,
                heavy_rule="bernoulli", heavy_param=0.005, sink_prefix=4),
    5: Workload(5, 8, 32, 32, 128, 32768, 0, _half_budget(0.05, 32768), _half_budget(0.05, 32768), 16,
                heavy_rule="none"),
    # context shape, not one of the five benchmark configurations: the multi-query model the paper
    # evaluates (Section 4: 32 layers, 71 query heads over one KV head of dimension 64, context 2048
    # -> 102 + 102 slots at 10 %), batch 64, decoding from an empty cache
    6: Workload(6, 64, 32, 1, 64, 0, 128, 102, 102, 8, heavy_rule="bernoulli", heavy_param=0.01, group=71),
}


def _gen(device, cfg_id: int, kind: int, index: int = 0) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((cfg_id * 1000 + kind) * 100003 + index)
    return g


def _randn_half(shape, g, device, std: float = 1.0) -> torch.Tensor:
    x = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    if std != 1.0:
        x.mul_(std)
    return x.to(torch.float16)


def make_weights(w: Workload, device="cpu") -> Dict[str, torch.Tensor]:
    """Per-head feature-map weights, fp16, row-major:
    w_phi1/w_psi1 [L,H,D,R'], w_phi2/w_psi2 [L,H,R',R], w_psi3 [L,H,R,R]; with grouped
    query heads the phi weights have one set per query head: [L, H*group, ...]."""
    L, H, D, Rp, R = w.layers, w.heads, w.head_dim, w.hidden, w.rank
    Hq = H * w.group
    shapes = {"w_phi1": (L, Hq, D, Rp), "w_phi2": (L, Hq, Rp, R),
              "w_psi1": (L, H, D, Rp), "w_psi2": (L, H, Rp, R), "w_psi3": (L, H, R, R)}
    out = {}
    for i, (name, shape) in enumerate(shapes.items()):
        out[name] = _randn_half(shape, _gen(device, w.cfg_id, _W, i), device, w.weight_std)
    return out


def _boost_mask(w: Workload, shape_prefix: Tuple[int, ...], positions: torch.Tensor,
                g: torch.Generator, device) -> Optional[torch.Tensor]:
    """Boolean mask [*shape_prefix, len(positions)] of keys that get scaled."""
    n = positions.numel()
    if w.heavy_rule == "every":
        m = (positions % int(w.heavy_param) == 0).expand(*shape_prefix, n).clone()
    elif w.heavy_rule == "bernoulli":
        m = torch.rand(*shape_prefix, n, generator=g, device=device) < w.heavy_param
    elif w.heavy_rule == "none":
        m = torch.zeros(*shape_prefix, n, dtype=torch.bool, device=device)
    else:
        raise ValueError(w.heavy_rule)
    if w.sink_prefix:
        m = m | (positions < w.sink_prefix)
    return m


def make_prompt(w: Workload, layer_begin: int, layer_count: int, device="cpu",
                prompt: Optional[int] = None):
    """Prompt Q, K, V, fp16 [B, layer_count, H, S, D], generated layer by layer
    so that a layer's bits do not depend on how the layers are grouped.  With grouped query
    heads Q is [B, layer_count, H*group, S, D]."""
    S = w.prompt if prompt is None else prompt
    B, H, D = w.batch, w.heads, w.head_dim
    Hq = H * w.group
    Q = torch.empty((B, layer_count, Hq, S, D), dtype=torch.float16, device=device)
    K = torch.empty((B, layer_count, H, S, D), dtype=torch.float16, device=device)
    V = torch.empty_like(K)
    positions = torch.arange(S, device=device)
    for j in range(layer_count):
        layer = layer_begin + j
        Q[:, j] = _randn_half((B, Hq, S, D), _gen(device, w.cfg_id, _Q, layer), device)
        k = torch.randn((B, H, S, D), generator=_gen(device, w.cfg_id, _K, layer),
                        device=device, dtype=torch.float32)
        m = _boost_mask(w, (B, H), positions, _gen(device, w.cfg_id, _MASK, layer), device)
        k = torch.where(m[..., None], k * w.key_boost, k)
        K[:, j] = k.to(torch.float16)
        V[:, j] = _randn_half((B, H, S, D), _gen(device, w.cfg_id, _V, layer), device)
    return Q, K, V


def make_decode_inputs(w: Workload, step: int, device="cpu", prompt: Optional[int] = None):
    """q, k, v of decode step `step` (absolute position prompt+step), fp16 [B,L,H,D]
    (q [B,L,H*group,D] with grouped query heads)."""
    S = w.prompt if prompt is None else prompt
    shape = (w.batch, w.layers, w.heads, w.head_dim)
    q = _randn_half((w.batch, w.layers, w.heads * w.group, w.head_dim),
                    _gen(device, w.cfg_id, _DQ, step), device)
    k = torch.randn(shape, generator=_gen(device, w.cfg_id, _DK, step), device=device,
                    dtype=torch.float32)
    pos = torch.tensor([S + step], device=device)
    m = _boost_mask(w, shape[:3], pos, _gen(device, w.cfg_id, _DMASK, step), device)
    k = torch.where(m, k * w.key_boost, k).to(torch.float16)
    v = _randn_half(shape, _gen(device, w.cfg_id, _DV, step), device)
    return q, k, v


def instance_index(w: Workload, b: int, layer: int, head: int) -> int:
    """Flat index of (b, layer, head) in the [B, L, H] order every buffer uses."""
    return (b * w.layers + layer) * w.heads + head


def instance_coords(w: Workload, inst: int) -> Tuple[int, int, int]:
    head = inst % w.heads
    layer = (inst // w.heads) % w.layers
    b = inst // (w.heads * w.layers)
    return b, layer, head
