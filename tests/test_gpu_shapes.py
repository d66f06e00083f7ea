"""GPU parity on odd layer shapes and degenerate settings, every token against the oracle: dimensions that are the
smallest multiples the layout allows, top-k at its maximum, a cache pool that is not a multiple of 32, no channel
cache at all, only 8-bit experts, 6-bit experts, a shared expert, empty experts, token counts of 0 and 1."""
import numpy as np
import pytest
import torch

import oracle
from helpers import make_gpu_layer, make_oracle_layer, rel_err
from paper_2503_21135_b200 import binding
from paper_2503_21135_b200 import workloads as wl

pytestmark = pytest.mark.gpu
TOL = 1e-2
BASE = wl.CONFIGS["tiny"]

CASES = {
    # d, f, E, k, G, shared, S, P, bits of the routed experts, token counts
    "odd_dims_shared_g64": dict(d_model=768, d_ff=384, n_experts=5, top_k=3, group_size=64, n_shared=1, max_sig=16,
                                cache_size=32, bits=[2, 3, 4, 8, 3], tokens=(1, 7, 70)),
    "smallest_all_8bit_no_cache": dict(d_model=256, d_ff=128, n_experts=3, top_k=1, group_size=128, n_shared=0, max_sig=0,
                                       cache_size=0, bits=[8, 8, 8], tokens=(1, 33)),
    "low_bits_no_cache": dict(d_model=256, d_ff=256, n_experts=4, top_k=2, group_size=64, n_shared=0, max_sig=0,
                              cache_size=0, bits=[2, 3, 4, 2], tokens=(5, 90)),
    "topk8_pool_not_multiple_of_32": dict(d_model=1024, d_ff=640, n_experts=16, top_k=8, group_size=64, n_shared=0,
                                          max_sig=48, cache_size=48, bits=[2, 3, 4, 8] * 4, tokens=(3, 130)),
    # INT6 as the base width of whole experts (Section IV-A: INT2/4/6/8), at both group sizes, with and without cache
    "int6_base_g128": dict(d_model=1024, d_ff=512, n_experts=8, top_k=2, group_size=128, n_shared=0, max_sig=32,
                           cache_size=64, bits=[2, 3, 4, 6, 6, 4, 8, 6], tokens=(1, 7, 40, 200)),
    "int6_base_g64_shared": dict(d_model=768, d_ff=384, n_experts=4, top_k=2, group_size=64, n_shared=1, max_sig=16,
                                 cache_size=32, bits=[6, 6, 6, 2], tokens=(3, 150)),
    "int6_only_no_cache": dict(d_model=256, d_ff=128, n_experts=2, top_k=1, group_size=128, n_shared=0, max_sig=0,
                               cache_size=0, bits=[6, 6], tokens=(1, 90)),
    "one_expert": dict(d_model=512, d_ff=256, n_experts=1, top_k=1, group_size=128, n_shared=0, max_sig=8, cache_size=40,
                       bits=[3], tokens=(2, 100)),
}


@pytest.mark.parametrize("name", list(CASES))
def test_shape(name):
    c = dict(CASES[name])
    bits_routed, tokens = c.pop("bits"), c.pop("tokens")
    cfg = wl.scaled(BASE, name=name, tokens=tokens, zipf="desc", **c)
    wg, wu, wd = wl.layer_weights(cfg)
    bits = np.array(list(bits_routed) + [8] * cfg.n_shared, np.int32)
    pool = wl.cache_pool(cfg)
    assert pool.shape == (cfg.n_experts, cfg.cache_size)
    gpu = make_gpu_layer(cfg, wg, wu, wd, bits, pool, max_tokens=max(tokens))
    ora = make_oracle_layer(cfg, wg, wu, wd, bits)
    sets = wl.initial_sig_sets(cfg, pool)
    gpu.set_channel_switch(sets)
    ora.set_channel_switch(sets)
    # codes of every expert's gate matrix, and of all three matrices of the 6-bit experts, bit for bit
    for e in range(cfg.n_experts + cfg.n_shared):
        for mat in ((binding.MAT_GATE, binding.MAT_UP, binding.MAT_DOWN) if bits[e] == 6 else (binding.MAT_GATE,)):
            q, s, m = gpu.export_codes(e, mat)
            assert torch.equal(q.cpu(), torch.from_numpy(ora.base[e][mat].q)), (e, mat)
            assert np.array_equal(s.cpu().numpy().view(np.uint16), ora.base[e][mat].s)
            assert np.array_equal(m.cpu().numpy().view(np.uint16), ora.base[e][mat].m)
    for step, T in enumerate(tokens):
        x, lg = wl.activations(cfg, T, step=step), wl.router_logits(cfg, T, step=step)
        y, dbg = gpu.forward(x.cuda(), lg.cuda(), binding.F32, debug=True)
        torch.cuda.synchronize()
        assert gpu.poll_status() == 0
        out = ora.forward(oracle.as_u16(x), lg.numpy())
        assert np.array_equal(dbg["idx"].cpu().numpy(), out["idx"])
        assert np.array_equal(dbg["offsets"].cpu().numpy(), out["offsets"])
        assert np.array_equal(dbg["perm"].cpu().numpy(), out["perm"])
        err = rel_err(y.cpu().numpy(), out["y"])
        assert err <= TOL, (name, T, err)
        yb = gpu.forward(x.cuda(), lg.cuda(), binding.BF16)
        assert torch.equal(yb, y.to(torch.bfloat16))
    # no tokens: a no-op that leaves the output alone
    y0 = torch.full((4, cfg.d_model), 7.0, device="cuda")
    gpu.forward(torch.empty((0, cfg.d_model), dtype=torch.bfloat16, device="cuda"),
                torch.empty((0, cfg.n_experts), dtype=torch.float32, device="cuda"), binding.F32, y=y0[:0])
    assert torch.all(y0 == 7.0)
    # an empty set everywhere equals the base layer; with a pool, the full set changes something
    empty = [np.array([], np.int32)] * cfg.n_experts
    gpu.set_channel_switch(empty)
    ora.set_channel_switch(empty)
    T = tokens[-1]
    x, lg = wl.activations(cfg, T, step=9), wl.router_logits(cfg, T, step=9)
    y = gpu.forward(x.cuda(), lg.cuda(), binding.F32)
    assert rel_err(y.cpu().numpy(), ora.forward(oracle.as_u16(x), lg.numpy())["y"]) <= TOL
