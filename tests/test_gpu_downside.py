"""GPU parity for significant channels on the d_ff side (Section IV-B applied to W_down's input channels): 8-bit codes
and parameters of the cached hidden units bit-exact against the oracle, forwards on every FFN kernel within the output
tolerance, state = last set installed, other target precisions, the requantize-from-cache switch mode, error cases."""
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
P2, S2 = 96, 48
ERR = binding.STATUS_NAMES.index


def _u16(t):
    return t.cpu().numpy().view(np.uint16)


@pytest.fixture(scope="module")
def lay():
    wg, wu, wd, bits, pool, sets = make_inputs(CFG)
    ora = make_oracle_layer(CFG, wg, wu, wd, bits)
    gpu = make_gpu_layer(CFG, wg, wu, wd, bits, pool, max_tokens=256)
    gpu.set_channel_switch(sets)
    ora.set_channel_switch(sets)
    pool_d = wl.cache_pool_down(CFG, P2)
    ora.enable_down_side(oracle.as_u16(wd))
    gpu.pack_down_cache(wd.cuda(), bits, pool_d, S2)
    torch.cuda.synchronize()
    return dict(bits=bits, pool_d=pool_d, ora=ora, gpu=gpu, wd=wd)


def _forward(lay, T, step):
    x, lg = wl.activations(CFG, T, step=step), wl.router_logits(CFG, T, step=step)
    y = lay["gpu"].forward(x.cuda(), lg.cuda(), binding.F32)
    torch.cuda.synchronize()
    assert lay["gpu"].poll_status() == 0
    ref = lay["ora"].forward(oracle.as_u16(x), lg.numpy())["y"]
    return y, ref


def _install(lay, sets):
    lay["gpu"].set_channel_switch_down(sets)
    lay["ora"].set_channel_switch_down(sets)


def test_down_pool_codes_bit_exact(lay):
    gpu, ora, pool_d = lay["gpu"], lay["ora"], lay["pool_d"]
    sets = wl.sig_sets_down(CFG, pool_d, S2)
    _install(lay, sets)
    for e in range(CFG.n_experts):
        if lay["bits"][e] >= 8:
            with pytest.raises(binding.DynamoError):
                gpu.export_codes(e, binding.MAT_DOWN, binding.CODES_HI_POOL)
            continue
        ref = ora.hi_down[e]
        for which, cols in ((binding.CODES_HI_POOL, pool_d[e]), (binding.CODES_HI_ACTIVE, sets[e])):
            q, s, m = gpu.export_codes(e, binding.MAT_DOWN, which)
            expect = np.zeros_like(ref.q)
            expect[:, cols] = ref.q[:, cols]
            assert np.array_equal(q.cpu().numpy(), expect), (e, which)
            assert np.array_equal(_u16(s), ref.s) and np.array_equal(_u16(m), ref.m), (e, which)
    _install(lay, [np.array([], np.int32)] * CFG.n_experts)


@pytest.mark.parametrize("T", [1, 8, 40, 200])
def test_forward_with_down_side_sets(lay, T):
    # T <= 64: every expert on the streaming kernel; 200: loaded experts on the tcgen05 pair kernel
    y0, ref0 = _forward(lay, T, step=T)
    assert rel_err(y0.cpu().numpy(), ref0) <= TOL
    sets = wl.sig_sets_down(CFG, lay["pool_d"], S2, event=T)
    _install(lay, sets)
    y1, ref1 = _forward(lay, T, step=T)
    assert rel_err(y1.cpu().numpy(), ref1) <= TOL
    # the correction itself is resolved: GPU and oracle agree on what the sets change, far below the change
    dg, dr = (y1 - y0).cpu().numpy().astype(np.float64), ref1 - ref0
    assert np.max(np.abs(dr)) > 0
    assert np.max(np.abs(dg - dr)) <= 0.05 * np.max(np.abs(dr)) + 1e-3 * np.sqrt(np.mean(ref1 ** 2))
    # state depends only on the last set installed; the empty set is the base forward, bit for bit
    _install(lay, wl.sig_sets_down(CFG, lay["pool_d"], 7, event=99))
    _install(lay, sets)
    assert torch.equal(_forward(lay, T, step=T)[0], y1)
    _install(lay, [np.array([], np.int32)] * CFG.n_experts)
    assert torch.equal(_forward(lay, T, step=T)[0], y0)


def test_all_cached_units_on_both_kernels(lay):
    gpu = lay["gpu"]
    sets = [p[:S2] for p in lay["pool_d"]]
    _install(lay, sets)
    try:
        for T, step in ((200, 3), (33, 4)):     # tcgen05 kernel for the popular experts; streaming kernel only
            y, ref = _forward(lay, T, step=step)
            assert rel_err(y.cpu().numpy(), ref) <= TOL
    finally:
        _install(lay, [np.array([], np.int32)] * CFG.n_experts)


@pytest.mark.parametrize("target", [6, 4, 3, 2, "mixed"])
def test_down_side_target_precision(lay, target):
    """Section IV-B on the d_ff side: the significant hidden units requantized to another precision, higher or lower."""
    gpu, ora, pool_d = lay["gpu"], lay["ora"], lay["pool_d"]
    E = CFG.n_experts
    hb = [6, 2, 4, 3, 8, 6, 4, 2][:E] if target == "mixed" else [target] * E
    sets = wl.sig_sets_down(CFG, pool_d, S2, event=3)
    _install(lay, sets)
    y8 = {T: _forward(lay, T, step=50 + T)[0] for T in (40, 200)}
    try:
        gpu.set_channel_precision_down(hb)
        ora.set_channel_precision_down(hb, oracle.as_u16(lay["wd"]))
        for e in range(E):
            if lay["bits"][e] >= 8:
                continue
            ref = ora.hi_down[e]
            q, s, m = gpu.export_codes(e, binding.MAT_DOWN, binding.CODES_HI_POOL)
            expect = np.zeros_like(ref.q)
            expect[:, pool_d[e]] = ref.q[:, pool_d[e]]
            assert np.array_equal(q.cpu().numpy(), expect), e
            assert int(expect.max()) <= 2 ** hb[e] - 1
            assert np.array_equal(_u16(s), ref.s) and np.array_equal(_u16(m), ref.m), e
        for T in (40, 200):                      # streaming kernel only; tcgen05 kernel for the popular experts
            y, ref = _forward(lay, T, step=50 + T)
            assert rel_err(y.cpu().numpy(), ref) <= TOL
        # a target equal to the base bit-width: every difference is zero, the forward is the base forward bit for bit
        gpu.set_channel_precision_down([int(b) if b < 8 else 8 for b in lay["bits"][:E]])
        y_same = _forward_gpu_only(lay, 40, 90)
        _install(lay, [np.array([], np.int32)] * E)
        assert torch.equal(_forward_gpu_only(lay, 40, 90), y_same)
        _install(lay, sets)
    finally:
        gpu.set_channel_precision_down([8] * E)
        ora.set_channel_precision_down([8] * E, oracle.as_u16(lay["wd"]))
    for T in (40, 200):                          # back at 8: the packed state, bit for bit
        assert torch.equal(_forward(lay, T, step=50 + T)[0], y8[T])
    _install(lay, [np.array([], np.int32)] * E)


def _forward_gpu_only(lay, T, step):
    x, lg = wl.activations(CFG, T, step=step), wl.router_logits(CFG, T, step=step)
    y = lay["gpu"].forward(x.cuda(), lg.cuda(), binding.F32)
    torch.cuda.synchronize()
    assert lay["gpu"].poll_status() == 0
    return y


def test_down_side_requant_mode_reaches_the_same_state(lay):
    """Switch mode "requantize from the cache" on the d_ff side: codes and differences of a new set are re-derived
    from the bf16 channel cache at the current target precision; the state equals the one SELECT mode reaches."""
    gpu, ora, pool_d = lay["gpu"], lay["ora"], lay["pool_d"]
    E = CFG.n_experts
    hb = [4, 6, 3, 6, 8, 2, 4, 6][:E]
    sets = [wl.sig_sets_down(CFG, pool_d, S2, event=ev) for ev in (5, 6)]
    try:
        gpu.set_channel_precision_down(hb)
        ora.set_channel_precision_down(hb, oracle.as_u16(lay["wd"]))
        outs = {}
        for mode in (binding.SWITCH_SELECT, binding.SWITCH_REQUANT):
            gpu.set_switch_mode(mode)
            n0 = gpu.kernel_launches()
            for st in sets:                       # two events in a row: the state depends on the last one only
                _install(lay, st)
            if mode == binding.SWITCH_REQUANT:
                assert gpu.kernel_launches() - n0 == 2      # one requantization launch per event
            else:
                assert gpu.kernel_launches() - n0 == 0      # table writes only
            codes = [tuple(t.clone() for t in gpu.export_codes(e, binding.MAT_DOWN, binding.CODES_HI_ACTIVE))
                     for e in range(E) if lay["bits"][e] < 8]
            y, ref = _forward(lay, 40, step=61)
            assert rel_err(y.cpu().numpy(), ref) <= TOL
            outs[mode] = (codes, y)
        for (qa, sa, ma), (qb, sb, mb) in zip(outs[binding.SWITCH_SELECT][0], outs[binding.SWITCH_REQUANT][0]):
            assert torch.equal(qa, qb) and torch.equal(sa, sb) and torch.equal(ma, mb)
        assert torch.equal(outs[binding.SWITCH_SELECT][1], outs[binding.SWITCH_REQUANT][1])
        e0 = next(e for e in range(E) if lay["bits"][e] < 8)
        q, _, _ = gpu.export_codes(e0, binding.MAT_DOWN, binding.CODES_HI_ACTIVE)
        expect = np.zeros_like(ora.hi_down[e0].q)
        expect[:, sets[1][e0]] = ora.hi_down[e0].q[:, sets[1][e0]]
        assert np.array_equal(q.cpu().numpy(), expect)
    finally:
        gpu.set_switch_mode(binding.SWITCH_SELECT)
        gpu.set_channel_precision_down([8] * E)
        ora.set_channel_precision_down([8] * E, oracle.as_u16(lay["wd"]))
        _install(lay, [np.array([], np.int32)] * E)


def test_down_side_precision_errors(lay):
    gpu = lay["gpu"]
    E = CFG.n_experts
    with pytest.raises(binding.DynamoError) as ei:
        gpu.set_channel_precision_down([5] * E)
    assert ei.value.status == ERR("ERR_BITS")
    fresh = binding.DynamoLayer.from_config(CFG, max_tokens=16)
    with pytest.raises(binding.DynamoError) as ei:
        fresh.set_channel_precision_down([8] * E)
    assert ei.value.status == ERR("ERR_STATE")


def test_switch_enqueued_between_two_forwards_takes_effect_between_them(lay):
    """No host synchronisation anywhere in the sequence forward, switch, forward, switch back, forward: every
    forward must see exactly the set installed before it in stream order."""
    gpu = lay["gpu"]
    T = 24
    x, lg = wl.activations(CFG, T, step=41).cuda(), wl.router_logits(CFG, T, step=41).cuda()
    empty = [np.array([], np.int32)] * CFG.n_experts
    sets = wl.sig_sets_down(CFG, lay["pool_d"], S2)
    gpu.set_channel_switch_down(empty)
    y_empty = gpu.forward(x, lg, binding.F32).clone()
    gpu.set_channel_switch_down(sets)
    y_sets = gpu.forward(x, lg, binding.F32).clone()
    torch.cuda.synchronize()
    assert not torch.equal(y_empty, y_sets)
    outs = [torch.empty_like(y_empty) for _ in range(3)]
    gpu.set_channel_switch_down(empty)
    gpu.forward(x, lg, binding.F32, y=outs[0])
    gpu.set_channel_switch_down(sets)          # enqueued behind the first forward, ahead of the second
    gpu.forward(x, lg, binding.F32, y=outs[1])
    gpu.set_channel_switch_down(empty)
    gpu.forward(x, lg, binding.F32, y=outs[2])
    torch.cuda.synchronize()
    assert torch.equal(outs[0], y_empty) and torch.equal(outs[1], y_sets) and torch.equal(outs[2], y_empty)
    lay["ora"].set_channel_switch_down(empty)


def test_down_side_errors_leave_state(lay):
    gpu, pool_d = lay["gpu"], lay["pool_d"]
    E = CFG.n_experts
    sets = wl.sig_sets_down(CFG, pool_d, 5)
    _install(lay, sets)
    y, _ = _forward(lay, 16, step=7)
    not_cached = np.setdiff1d(np.arange(CFG.d_ff), pool_d[0])[:1]
    for bad, code in ((not_cached, "ERR_NOT_CACHED"), (np.array([CFG.d_ff]), "ERR_INDEX_RANGE"),
                      (np.array([pool_d[0][0], pool_d[0][0]]), "ERR_INDEX_DUP"), (pool_d[0][: S2 + 1], "ERR_INDEX_RANGE")):
        s = list(sets)
        s[0] = bad
        with pytest.raises(binding.DynamoError) as ei:
            gpu.set_channel_switch_down(s)
        assert ei.value.status == ERR(code), code
    assert torch.equal(_forward(lay, 16, step=7)[0], y)
    fresh = binding.DynamoLayer.from_config(CFG, max_tokens=16)
    fresh.max_sig_down = S2
    with pytest.raises(binding.DynamoError) as ei:
        fresh.set_channel_switch_down(sets)
    assert ei.value.status == ERR("ERR_STATE")
    unsorted = pool_d.copy()
    unsorted[1, [0, 1]] = unsorted[1, [1, 0]]
    with pytest.raises(binding.DynamoError) as ei:
        gpu.pack_down_cache(lay["wd"].cuda(), lay["bits"], unsorted, S2)
    assert ei.value.status == ERR("ERR_INDEX_DUP")
    assert torch.equal(_forward(lay, 16, step=7)[0], y)      # the failed re-pack left the cache in place
    _install(lay, [np.array([], np.int32)] * E)
