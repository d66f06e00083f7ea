"""The allocation-free routing entry point against the regular forward's routing outputs and the CPU oracle.

Callers that may not allocate device memory (stream capture in progress, framework plugins with a
fixed buffer set, real-time loops) use dynamo_route_permute_static; it must give exactly what
dynamo_moe_forward reports for the same logits, and exactly the oracle's top-k and permutation, call
after call, although all calls share one scratch array inside the library.  This file sorts last so that a stop-at-first-failure run has
already executed every other test."""
import numpy as np
import pytest
import torch

import oracle
from helpers import make_gpu_layer, make_inputs
from paper_2503_21135_b200 import binding
from paper_2503_21135_b200 import workloads as wl

pytestmark = pytest.mark.gpu
CFG = wl.CONFIGS["tiny"]


def _static_route(lg, k, E, renorm=1):
    T = lg.shape[0]
    dev = lg.device
    idx = torch.full((T, k), -7, dtype=torch.int32, device=dev)
    w = torch.full((T, k), -7.0, dtype=torch.float32, device=dev)
    off = torch.full((E + 1,), -7, dtype=torch.int32, device=dev)
    perm = torch.full((T * k,), -7, dtype=torch.int32, device=dev)
    st = binding.dynamo_route_permute_static(lg.data_ptr(), T, E, k, renorm, idx.data_ptr(), w.data_ptr(),
                                             off.data_ptr(), perm.data_ptr(),
                                             torch.cuda.current_stream().cuda_stream)
    assert st == 0
    return idx, w, off, perm


def test_static_route_matches_forward_twice_in_a_row():
    wg, wu, wd, bits, pool, sets = make_inputs(CFG)
    gpu = make_gpu_layer(CFG, wg, wu, wd, bits, pool, max_tokens=256)
    # two calls in a row with different sizes: the second must not see the first one's leftovers
    for T, step in ((200, 11), (37, 12)):
        x = wl.activations(CFG, T, step=step).cuda()
        lg = wl.router_logits(CFG, T, step=step).cuda()
        _, dbg = gpu.forward(x, lg, binding.F32, debug=True)
        idx, w, off, perm = _static_route(lg, CFG.top_k, CFG.n_experts)
        torch.cuda.synchronize()
        assert torch.equal(idx, dbg["idx"])
        assert torch.equal(off, dbg["offsets"])
        assert torch.equal(perm, dbg["perm"])
        assert float((w - dbg["w"]).abs().max()) <= 1e-6
        # and directly against the oracle: indices, offsets and permutation bit-exact, weights to 1e-6
        ref_idx, ref_w = oracle.route(lg.cpu().numpy(), CFG.top_k)
        ref_off, ref_perm = oracle.permute(ref_idx, CFG.n_experts)
        assert np.array_equal(idx.cpu().numpy(), ref_idx)
        assert np.array_equal(off.cpu().numpy(), ref_off)
        assert np.array_equal(perm.cpu().numpy(), ref_perm)
        assert float(np.max(np.abs(w.cpu().numpy() - ref_w))) <= 1e-6


def test_static_route_limits():
    lg = torch.zeros((4, 8), dtype=torch.float32, device="cuda")
    args = (lg.data_ptr(), lg.data_ptr(), lg.data_ptr(), lg.data_ptr(), None)
    f = binding.dynamo_route_permute_static
    assert f(lg.data_ptr(), 32768 // 2 + 1, 8, 2, 1, *args) == 10      # beyond the fixed scratch
    assert f(lg.data_ptr(), 4, 300, 2, 1, *args) == 2
    assert f(lg.data_ptr(), 4, 8, 9, 1, *args) == 2
    assert f(None, 4, 8, 2, 1, *args) == 1
    assert f(lg.data_ptr(), 0, 8, 2, 1, *args) == 0
