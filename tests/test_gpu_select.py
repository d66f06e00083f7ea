"""GPU parity of the runtime selection of significant channels (Sections IV-B, V-A): the activation statistics
accumulated during forwards are compared bit for bit with the oracle's (same float32 order), the selected sets
exactly, and the forward after the device-side switch against the oracle with those sets."""
import numpy as np
import pytest
import torch

import oracle
from helpers import make_gpu_layer, make_inputs, make_oracle_layer, rel_err
from paper_2503_21135_b200 import binding
from paper_2503_21135_b200 import workloads as wl

pytestmark = pytest.mark.gpu
TOL = 1e-2
CFG = wl.CONFIGS["tiny"]


@pytest.fixture(scope="module")
def tiny():
    wg, wu, wd, bits, pool, sets = make_inputs(CFG)
    ora = make_oracle_layer(CFG, wg, wu, wd, bits)
    gpu = make_gpu_layer(CFG, wg, wu, wd, bits, pool, max_tokens=256)
    gpu.set_channel_switch(sets)
    ora.set_channel_switch(sets)
    return dict(ora=ora, gpu=gpu, bits=bits, pool=pool, sets=sets)


def test_stats_selection_and_forward_follow_the_oracle(tiny):
    gpu, ora, pool, bits = tiny["gpu"], tiny["ora"], tiny["pool"], tiny["bits"]
    E, P = CFG.n_experts, CFG.cache_size
    switchable = [int(b) < 8 for b in bits[:E]]
    gpu.select_significant(0, reset=True)                      # start from zero statistics, empty sets
    assert torch.count_nonzero(gpu.channel_stats()) == 0
    stats = np.zeros((E, P), np.float32)
    gpu.set_stats_collection(True)
    try:
        for T, step in ((64, 21), (7, 22), (200, 23)):
            x, lg = wl.activations(CFG, T, step=step), wl.router_logits(CFG, T, step=step)
            launches = gpu.kernel_launches()
            gpu.forward(x.cuda(), lg.cuda(), binding.F32)
            assert gpu.kernel_launches() - launches in (7, 9)  # one kernel more than without collection
            idx, _ = oracle.route(lg.numpy(), CFG.top_k)
            stats = oracle.channel_stats_update(stats, oracle.as_u16(x), idx, pool)
            got = gpu.channel_stats().cpu().numpy()
            assert np.array_equal(got.view(np.uint32), stats.view(np.uint32))      # bit for bit
    finally:
        gpu.set_stats_collection(False)
    # collection off: a forward leaves the statistics alone
    x, lg = wl.activations(CFG, 32, step=24), wl.router_logits(CFG, 32, step=24)
    gpu.forward(x.cuda(), lg.cuda(), binding.F32)
    assert np.array_equal(gpu.channel_stats().cpu().numpy(), stats)
    # selection on the device == the oracle's rule on the same numbers
    n_sel = CFG.max_sig // 2
    ref_sets = oracle.select_significant(stats, pool, n_sel, switchable)
    got_sets = gpu.select_significant(n_sel, reset=True)
    assert len(got_sets) == E
    for e in range(E):
        assert got_sets[e].tolist() == ref_sets[e].tolist(), e
    assert torch.count_nonzero(gpu.channel_stats()) == 0       # reset
    # the tables the kernel wrote serve the forward exactly like a host-driven switch to those sets
    ora.set_channel_switch(ref_sets)
    y = gpu.forward(x.cuda(), lg.cuda(), binding.F32)
    torch.cuda.synchronize()
    assert gpu.poll_status() == 0
    ref = ora.forward(oracle.as_u16(x), lg.numpy())
    assert rel_err(y.cpu().numpy(), ref["y"]) <= TOL
    gpu.set_channel_switch(ref_sets)
    assert torch.equal(gpu.forward(x.cuda(), lg.cuda(), binding.F32), y)
    # the host mirror follows: the active 8-bit export lists exactly the selected channels
    for e in range(E):
        if not switchable[e]:
            continue
        q, _, _ = gpu.export_codes(e, binding.MAT_UP, binding.CODES_HI_ACTIVE)
        expect = np.zeros_like(ora.hi[e][1].q)
        expect[:, ref_sets[e]] = ora.hi[e][1].q[:, ref_sets[e]]
        assert np.array_equal(q.cpu().numpy(), expect)
    # restore the fixture's sets
    gpu.set_channel_switch(tiny["sets"])
    ora.set_channel_switch(tiny["sets"])


def test_selection_tracks_a_change_of_the_data(tiny):
    """New data whose large activations sit on other cached channels moves the selection onto them."""
    gpu, pool, bits = tiny["gpu"], tiny["pool"], tiny["bits"]
    E = CFG.n_experts
    gpu.select_significant(0, reset=True)
    x = wl.activations(CFG, 128, step=31).clone()
    lg = wl.router_logits(CFG, 128, step=31)
    boosted = {e: pool[e][-3:] for e in range(E)}              # the three highest cached channels of every expert
    for e in range(E):
        x[:, boosted[e].tolist()] *= 50
    gpu.set_stats_collection(True)
    gpu.forward(x.cuda(), lg.cuda(), binding.F32)
    gpu.set_stats_collection(False)
    idx, _ = oracle.route(lg.numpy(), CFG.top_k)
    sets = gpu.select_significant(8, reset=True)
    for e in range(E):
        if int(bits[e]) >= 8:
            assert len(sets[e]) == 0
        elif (idx == e).any():
            assert set(boosted[e].tolist()) <= set(sets[e].tolist()), e
    gpu.set_channel_switch(tiny["sets"])


def test_selection_errors(tiny):
    gpu = tiny["gpu"]
    st = binding.load().dynamo_select_significant(gpu.ctx, CFG.max_sig + 1, 0, None, None, None)
    assert st == binding.STATUS_NAMES.index("ERR_SHAPE")
    st = binding.load().dynamo_select_significant(None, 1, 0, None, None, None)
    assert st == binding.STATUS_NAMES.index("ERR_NULL")
