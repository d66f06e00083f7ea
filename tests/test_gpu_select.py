"""GPU parity of the runtime selection of significant channels (Sections IV-B, V-A).  The statistic decides an integer
selection and the kernel accumulates it in fp32 while the oracle sums in float64, so parity is a three-part rule:
(1) the GPU's statistics lie within the fp32 accumulation bound of the oracle's; (2) GIVEN the GPU's statistics the
selected sets are exactly what the oracle's ranking rule picks from those numbers; (3) wherever no two exact
statistics that the ranking has to tell apart are closer than the bound, the sets equal the ones picked from the
exact statistics.  The forward after the device-side switch is then compared with the oracle given those sets."""
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
    stats = np.zeros((E, P), np.float64)
    n_add = np.zeros((E,), np.int64)           # additions behind every statistic of the expert
    gpu.set_stats_collection(True)
    try:
        for T, step in ((64, 21), (7, 22), (200, 23)):
            x, lg = wl.activations(CFG, T, step=step), wl.router_logits(CFG, T, step=step)
            launches = gpu.kernel_launches()
            gpu.forward(x.cuda(), lg.cuda(), binding.F32)
            assert gpu.kernel_launches() - launches in (5, 7, 9)  # one kernel more than without collection
            idx, _ = oracle.route(lg.numpy(), CFG.top_k)
            stats = oracle.channel_stats_update(stats, oracle.as_u16(x), idx, pool)
            n_add += np.bincount(idx.ravel(), minlength=E) + 1
            got = gpu.channel_stats().cpu().numpy().astype(np.float64)
            # (1) fp32 accumulation of n non-negative terms: |fl(sum) - sum| <= n * 2^-24 * sum
            bound = n_add[:, None] * 2.0 ** -24 * stats
            assert np.all(np.abs(got - stats) <= bound), float(np.max(np.abs(got - stats) - bound))
    finally:
        gpu.set_stats_collection(False)
    # collection off: a forward leaves the statistics alone
    x, lg = wl.activations(CFG, 32, step=24), wl.router_logits(CFG, 32, step=24)
    gpu.forward(x.cuda(), lg.cuda(), binding.F32)
    gpu_stats = gpu.channel_stats().cpu().numpy()
    assert np.array_equal(gpu_stats.astype(np.float64), got)
    n_sel = CFG.max_sig // 2
    # (2) selection on the device == the oracle's rule on the GPU's own numbers
    ref_sets = oracle.select_significant(gpu_stats, pool, n_sel, switchable)
    got_sets = gpu.select_significant(n_sel, reset=True)
    assert len(got_sets) == E
    for e in range(E):
        assert got_sets[e].tolist() == ref_sets[e].tolist(), e
    # (3) where the exact statistics the ranking must tell apart are further apart than twice the bound, the
    # selection from the exact statistics is the same
    exact_sets = oracle.select_significant(stats, pool, n_sel, switchable)
    n_decided = 0
    for e in range(E):
        if not switchable[e]:
            continue
        top = np.sort(stats[e])[::-1][: n_sel + 1]
        gap = np.min(-np.diff(top)) if len(top) > 1 else np.inf
        if gap > 2 * np.max(n_add[e] * 2.0 ** -24 * stats[e]):
            assert got_sets[e].tolist() == exact_sets[e].tolist(), e
            n_decided += 1
    assert n_decided >= 1          # continuous data: ties at this scale are rare
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


def test_selection_enqueued_without_waiting_takes_effect_in_stream_order(tiny):
    """forward, select (no wait), forward, with no host synchronisation in between: the second forward runs on the
    selected sets; the sets reach the host afterwards through dynamo_sync_sets."""
    gpu = tiny["gpu"]
    x, lg = wl.activations(CFG, 48, step=33).cuda(), wl.router_logits(CFG, 48, step=33).cuda()
    gpu.select_significant(0, reset=True)
    gpu.set_stats_collection(True)
    gpu.forward(x, lg, binding.F32)
    gpu.set_stats_collection(False)
    stats = gpu.channel_stats().clone()
    torch.cuda.synchronize()
    y_before = torch.empty((48, CFG.d_model), dtype=torch.float32, device="cuda")
    y_after = torch.empty_like(y_before)
    gpu.forward(x, lg, binding.F32, y=y_before)
    assert gpu.select_significant(6, reset=False, wait=False) is None
    gpu.forward(x, lg, binding.F32, y=y_after)
    sets = gpu.sync_sets()
    torch.cuda.synchronize()
    ref_sets = oracle.select_significant(stats.cpu().numpy(), tiny["pool"], 6, [int(b) < 8 for b in tiny["bits"][:CFG.n_experts]])
    for e in range(CFG.n_experts):
        assert sets[e].tolist() == ref_sets[e].tolist(), e
    gpu.set_channel_switch([np.array([], np.int32)] * CFG.n_experts)
    assert torch.equal(gpu.forward(x, lg, binding.F32), y_before)
    gpu.set_channel_switch(ref_sets)
    assert torch.equal(gpu.forward(x, lg, binding.F32), y_after)
    assert not torch.equal(y_before, y_after)
    assert [s.tolist() for s in gpu.sync_sets()] == [s.tolist() for s in ref_sets]   # whoever installed them
    gpu.set_channel_switch(tiny["sets"])


def test_selection_errors(tiny):
    gpu = tiny["gpu"]
    st = binding.load().dynamo_select_significant(gpu.ctx, CFG.max_sig + 1, 0, None, None, None)
    assert st == binding.STATUS_NAMES.index("ERR_SHAPE")
    st = binding.load().dynamo_select_significant(None, 1, 0, None, None, None)
    assert st == binding.STATUS_NAMES.index("ERR_NULL")
