"""Seeded synthetic inputs shaped like the MoE workloads the hot path is measured on.

This module only *draws inputs* (weights, activations, router logits, bit-width
assignments, channel-cache pools, significant-channel sets, switch events).  It
holds none of the method's arithmetic: no quantization, routing, packing or FFN
code lives here, so both the CPU oracle's tests and the CUDA path can be fed the
same buffers without sharing any computation.

Recipe (stand-in for the trained MoEs and text datasets the paper evaluates on,
which are not needed for a throughput/parity study of the layer):

* weights  = bf16_rne(N(0, 0.02^2)); per expert ``max(1, round(0.01*d))`` input
  channels (the same set for W_gate and W_up) are multiplied by 20 *before* the
  bf16 rounding (outlier channels); W_down has no outliers.
* x        = bf16_rne(N(0, 1)).
* logits   = fp32 N(0, 1) + bias_e,  bias_e = -1.2 * ln(rank_e)  (Zipf(1.2)
  popularity; rank 1 = most popular) or no bias.
* cache pool per expert = the outlier channels + seeded random others up to
  P = 2*S, sorted; initial significant set = all outliers + seeded random pool
  members up to S, sorted.

Every tensor has its own ``numpy.random.SeedSequence([BASE_SEED, config, layer,
tensor_id, expert])`` stream, so tensors can be generated independently and in
any order.
"""
from __future__ import annotations

import dataclasses
import math
from concurrent.futures import ThreadPoolExecutor
from typing import List, Optional

import numpy as np
import torch

BASE_SEED = 250321135

# tensor ids of the per-stream seeds
_T_X, _T_LOGITS, _T_OUTLIER, _T_POOL, _T_SIG, _T_BITS, _T_SWITCH, _T_ROUTER = 0, 1, 2, 3, 4, 5, 6, 7
_T_POOL_DOWN, _T_SIG_DOWN = 8, 9
_T_WGATE, _T_WUP, _T_WDOWN = 10, 11, 12


@dataclasses.dataclass(frozen=True)
class MoEConfig:
    """Shape and recipe of one synthetic MoE layer workload."""

    name: str
    config_id: int
    d_model: int
    d_ff: int
    n_experts: int
    top_k: int
    group_size: int
    max_sig: int            # S: capacity of a significant-channel set
    cache_size: int         # P: cached candidate channels per expert
    tokens: tuple           # token counts the workload is run at
    n_shared: int = 0
    zipf: Optional[str] = None   # None | "desc" (rank = E - e) | "asc" (rank = e + 1)
    n_layers: int = 1

    @property
    def n_total(self) -> int:
        return self.n_experts + self.n_shared

    @property
    def n_outlier(self) -> int:
        return max(1, int(round(0.01 * self.d_model)))


CONFIGS = {
    "tiny": MoEConfig("tiny", 1, 512, 1024, 8, 2, 128, 32, 64, (64,), zipf="desc"),
    "decode": MoEConfig("decode", 2, 4096, 14336, 8, 2, 128, 64, 128, (1, 8, 32, 64)),
    "prefill": MoEConfig("prefill", 3, 4096, 14336, 8, 2, 128, 128, 256, (4096,), zipf="desc"),
    "finegrained": MoEConfig("finegrained", 4, 2048, 1408, 64, 6, 64, 32, 64, (2048,),
                             n_shared=2, zipf="asc"),
    "switch": MoEConfig("switch", 5, 4096, 14336, 8, 2, 128, 64, 128, (16,), n_layers=16),
}


def scaled(cfg: MoEConfig, **kw) -> MoEConfig:
    """A copy of ``cfg`` with some fields replaced (used for reduced-size test cases)."""
    return dataclasses.replace(cfg, **kw)


def _rng(cfg: MoEConfig, layer: int, tensor_id: int, expert: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(
        np.random.SeedSequence([BASE_SEED, cfg.config_id, layer, tensor_id, expert])))


def bits_assignment(cfg: MoEConfig, layer: int = 0) -> np.ndarray:
    """Base bit-width of every expert (routed, then shared), int32 [E + E_s]."""
    E = cfg.n_experts
    if cfg.config_id == 1:
        base = [2, 3, 4, 4, 4, 4, 8, 8]
        bits = [base[e % 8] for e in range(E)]
    elif cfg.config_id in (2, 5):
        base = [2, 2, 2, 3, 3, 4, 4, 8]
        bits = [base[e % 8] for e in range(E)]
        _rng(cfg, layer, _T_BITS).shuffle(bits)
    elif cfg.config_id == 3:
        base = [3, 3, 3, 3, 4, 4, 4, 8]
        bits = [base[e % 8] for e in range(E)]
    else:  # fine-grained: by popularity rank (rank = e + 1): 1/4 at 4-bit, 3/8 at 3-bit, 3/8 at 2-bit
        n4 = E // 4
        n3 = (3 * E) // 8
        bits = [4] * n4 + [3] * n3 + [2] * (E - n4 - n3)
    bits = list(bits) + [8] * cfg.n_shared
    return np.asarray(bits, dtype=np.int32)


def popularity_bias(cfg: MoEConfig) -> np.ndarray:
    """Per-expert additive router bias, float64 [E]."""
    E = cfg.n_experts
    if cfg.zipf is None:
        return np.zeros(E)
    e = np.arange(E)
    rank = (E - e) if cfg.zipf == "desc" else (e + 1)
    return -1.2 * np.log(rank.astype(np.float64))


def outlier_channels(cfg: MoEConfig, layer: int, expert: int) -> np.ndarray:
    perm = _rng(cfg, layer, _T_OUTLIER, expert).permutation(cfg.d_model)
    return np.sort(perm[: cfg.n_outlier]).astype(np.int32)


def _normal_bf16(rng: np.random.Generator, shape, std: float, scale_cols=None) -> torch.Tensor:
    a = rng.standard_normal(size=shape, dtype=np.float32)
    a *= np.float32(std)
    if scale_cols is not None and len(scale_cols):
        a[:, scale_cols] *= np.float32(20.0)
    return torch.from_numpy(a).to(torch.bfloat16)


def expert_weights(cfg: MoEConfig, layer: int, expert: int):
    """(w_gate [f,d], w_up [f,d], w_down [d,f]) bf16 CPU tensors of one expert."""
    d, f = cfg.d_model, cfg.d_ff
    out = outlier_channels(cfg, layer, expert) if expert < cfg.n_experts else None
    wg = _normal_bf16(_rng(cfg, layer, _T_WGATE, expert), (f, d), 0.02, out)
    wu = _normal_bf16(_rng(cfg, layer, _T_WUP, expert), (f, d), 0.02, out)
    wd = _normal_bf16(_rng(cfg, layer, _T_WDOWN, expert), (d, f), 0.02, None)
    return wg, wu, wd


def layer_weights(cfg: MoEConfig, layer: int = 0, threads: int = 8):
    """(w_gate [E+Es,f,d], w_up [E+Es,f,d], w_down [E+Es,d,f]) bf16 CPU tensors."""
    n = cfg.n_total
    d, f = cfg.d_model, cfg.d_ff
    wg = torch.empty((n, f, d), dtype=torch.bfloat16)
    wu = torch.empty((n, f, d), dtype=torch.bfloat16)
    wd = torch.empty((n, d, f), dtype=torch.bfloat16)

    def one(e):
        g, u, dn = expert_weights(cfg, layer, e)
        wg[e], wu[e], wd[e] = g, u, dn

    if threads > 1 and n > 1:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(one, range(n)))
    else:
        for e in range(n):
            one(e)
    return wg, wu, wd


def activations(cfg: MoEConfig, T: int, layer: int = 0, step: int = 0) -> torch.Tensor:
    """x bf16 [T, d]."""
    a = _rng(cfg, layer, _T_X, step).standard_normal(size=(T, cfg.d_model), dtype=np.float32)
    return torch.from_numpy(a).to(torch.bfloat16)


def router_logits(cfg: MoEConfig, T: int, layer: int = 0, step: int = 0) -> torch.Tensor:
    """Router logits fp32 [T, E] (an *input* of the layer)."""
    a = _rng(cfg, layer, _T_LOGITS, step).standard_normal(size=(T, cfg.n_experts), dtype=np.float32)
    a = a.astype(np.float64) + popularity_bias(cfg)[None, :]
    return torch.from_numpy(a.astype(np.float32))


def router_weights(cfg: MoEConfig, layer: int = 0):
    """Router weight bf16 [E, d] ~ N(0, 1/d) (unit-variance scores for unit-variance inputs) and bias fp32 [E] =
    the config's popularity bias: inputs of the fused router GEMM."""
    w = _rng(cfg, layer, _T_ROUTER, 0).standard_normal(size=(cfg.n_experts, cfg.d_model), dtype=np.float32)
    w *= np.float32(1.0 / np.sqrt(cfg.d_model))
    return torch.from_numpy(w).to(torch.bfloat16), torch.from_numpy(popularity_bias(cfg).astype(np.float32))


def cache_pool(cfg: MoEConfig, layer: int = 0) -> np.ndarray:
    """Cached candidate channels per routed expert, int32 [E, P], each row sorted, unique."""
    out = np.empty((cfg.n_experts, cfg.cache_size), dtype=np.int32)
    for e in range(cfg.n_experts):
        o = outlier_channels(cfg, layer, e)[: cfg.cache_size]
        rest = np.setdiff1d(np.arange(cfg.d_model, dtype=np.int32), o)
        extra = _rng(cfg, layer, _T_POOL, e).permutation(rest)[: cfg.cache_size - len(o)]
        out[e] = np.sort(np.concatenate([o, extra]).astype(np.int32))
    return out


def cache_pool_down(cfg: MoEConfig, size: int, layer: int = 0) -> np.ndarray:
    """Cached hidden units (input channels of W_down) per routed expert, int32 [E, size], each row sorted, unique."""
    out = np.empty((cfg.n_experts, size), dtype=np.int32)
    for e in range(cfg.n_experts):
        out[e] = np.sort(_rng(cfg, layer, _T_POOL_DOWN, e).permutation(cfg.d_ff)[:size].astype(np.int32))
    return out


def sig_sets_down(cfg: MoEConfig, pool_down: np.ndarray, n_sig: int, layer: int = 0, event: int = 0) -> List[np.ndarray]:
    """A significant set of n_sig cached hidden units per routed expert (a different draw per event)."""
    return [np.sort(_rng(cfg, layer, _T_SIG_DOWN, e * 4096 + event).permutation(pool_down[e])[:n_sig].astype(np.int32))
            for e in range(cfg.n_experts)]


def initial_sig_sets(cfg: MoEConfig, pool: np.ndarray, layer: int = 0) -> List[np.ndarray]:
    """Initial significant set of every routed expert: all outliers + random pool members up to S."""
    sets = []
    for e in range(cfg.n_experts):
        o = np.intersect1d(outlier_channels(cfg, layer, e), pool[e])[: cfg.max_sig]
        rest = np.setdiff1d(pool[e], o)
        extra = _rng(cfg, layer, _T_SIG, e).permutation(rest)[: cfg.max_sig - len(o)]
        sets.append(np.sort(np.concatenate([o, extra]).astype(np.int32)))
    return sets


def switch_event(cfg: MoEConfig, pool: np.ndarray, current: List[np.ndarray], layer: int,
                 event: int, frac: float = 0.25) -> List[np.ndarray]:
    """New significant sets: ``frac`` of each expert's set is swapped for pool members not in it."""
    new = []
    for e in range(cfg.n_experts):
        rng = _rng(cfg, layer, _T_SWITCH, e * 4096 + event)
        cur = np.asarray(current[e], dtype=np.int32)
        n_swap = min(int(round(frac * len(cur))), len(pool[e]) - len(cur))
        keep = rng.permutation(cur)[n_swap:] if n_swap > 0 else cur
        cand = np.setdiff1d(pool[e], cur)
        enter = rng.permutation(cand)[:n_swap]
        new.append(np.sort(np.concatenate([keep, enter]).astype(np.int32)))
    return new


def sig_arrays(cfg: MoEConfig, sets: List[np.ndarray]):
    """Pack a list of per-expert index sets into (sig_idx int32 [E,S] padded with -1, sig_cnt int32 [E])."""
    idx = np.full((cfg.n_experts, cfg.max_sig), -1, dtype=np.int32)
    cnt = np.zeros((cfg.n_experts,), dtype=np.int32)
    for e, s in enumerate(sets):
        idx[e, : len(s)] = s
        cnt[e] = len(s)
    return idx, cnt


def expected_mean_bits(cfg: MoEConfig, layer: int = 0) -> float:
    return float(np.mean(bits_assignment(cfg, layer)[: cfg.n_experts]))


def _self_check() -> None:  # pragma: no cover - manual sanity helper
    for c in CONFIGS.values():
        b = bits_assignment(c)
        assert len(b) == c.n_total and math.isfinite(expected_mean_bits(c))
