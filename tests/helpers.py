"""Shared test helpers: build the same layer in the oracle and in the CUDA library."""
import numpy as np
import torch

import oracle
from paper_2503_21135_b200 import workloads as wl


def make_inputs(cfg, layer=0):
    wg, wu, wd = wl.layer_weights(cfg, layer)
    bits = wl.bits_assignment(cfg, layer)
    pool = wl.cache_pool(cfg, layer)
    sets = wl.initial_sig_sets(cfg, pool, layer)
    return wg, wu, wd, bits, pool, sets


def make_oracle_layer(cfg, wg, wu, wd, bits, renormalize=True, experts=None):
    return oracle.OracleLayer(oracle.as_u16(wg), oracle.as_u16(wu), oracle.as_u16(wd), bits, cfg.group_size,
                              cfg.n_experts, cfg.top_k, renormalize=renormalize, experts=experts)


def make_gpu_layer(cfg, wg, wu, wd, bits, pool, max_tokens=None, renormalize=True, workspace=None):
    from paper_2503_21135_b200 import binding

    layer = binding.DynamoLayer.from_config(cfg, max_tokens=max_tokens, renormalize=renormalize, workspace=workspace)
    layer.pack_experts(wg.cuda(), wu.cuda(), wd.cuda(), bits, pool)
    torch.cuda.synchronize()
    return layer


def rel_err(y_gpu: np.ndarray, y_ref: np.ndarray) -> float:
    """max |gpu - oracle| / RMS(oracle)."""
    rms = float(np.sqrt(np.mean(np.square(y_ref))))
    return float(np.max(np.abs(y_gpu.astype(np.float64) - y_ref))) / max(rms, 1e-300)


def stratified_tokens(idx: np.ndarray, E: int, n: int, seed: int = 0, all_of_two_least: bool = False) -> np.ndarray:
    """A seeded subset of at least n tokens that touches every expert: the tokens of the two least-loaded experts
    (all of them if asked, else capped at n/4 each), one token of every other expert, then a uniform sample."""
    T = idx.shape[0]
    rng = np.random.default_rng(seed)
    counts = np.bincount(idx.ravel(), minlength=E)
    chosen = set()
    order = np.argsort(counts, kind="stable")
    for e in order[:2]:
        toks = np.flatnonzero((idx == e).any(axis=1))
        if not all_of_two_least:
            toks = toks[: max(1, n // 4)]
        chosen.update(int(t) for t in toks)
    for e in range(E):
        toks = np.flatnonzero((idx == e).any(axis=1))
        if len(toks):
            chosen.add(int(toks[rng.integers(len(toks))]))
    rest = rng.permutation(T)
    for t in rest:
        if len(chosen) >= n:
            break
        chosen.add(int(t))
    return np.array(sorted(chosen), dtype=np.int32)
