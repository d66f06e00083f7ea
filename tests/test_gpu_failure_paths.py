"""Failure and guard paths on the GPU, none of which faults, traps or hangs the device:
a bounded wait that really runs out (a debug kernel waits, with a short limit, on a barrier nobody arrives at),
activations beyond the fp16 operand range (clamped and reported), and the guard blocks between the regions of
the weights arena and the workspace after a sweep of shapes and state changes."""
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
ERR = {n: i for i, n in enumerate(binding.STATUS_NAMES)}


@pytest.fixture(scope="module")
def tiny():
    wg, wu, wd, bits, pool, sets = make_inputs(CFG)
    ora = make_oracle_layer(CFG, wg, wu, wd, bits)
    gpu = make_gpu_layer(CFG, wg, wu, wd, bits, pool, max_tokens=256)
    gpu.set_channel_switch(sets)
    ora.set_channel_switch(sets)
    return dict(ora=ora, gpu=gpu, bits=bits, pool=pool, sets=sets)


def test_expired_wait_is_reported_blocks_forwards_and_clears(tiny):
    gpu, ora = tiny["gpu"], tiny["ora"]
    T = 40
    x, lg = wl.activations(CFG, T, step=71), wl.router_logits(CFG, T, step=71)
    ref = ora.forward(oracle.as_u16(x), lg.numpy())["y"]
    y = gpu.forward(x.cuda(), lg.cuda(), binding.F32)
    assert gpu.poll_status() == 0
    assert rel_err(y.cpu().numpy(), ref) <= TOL
    # a wait with a 2 ms limit on a barrier nobody arrives at: the kernel returns by itself
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    gpu.debug_expire_wait(2_000_000)
    t1.record()
    torch.cuda.synchronize()
    assert 1.0 <= t0.elapsed_time(t1) < 500.0          # it did wait, and it gave up long before the 1 s default
    # while the status is set a forward starts nothing: its output buffer keeps what it held
    sentinel = torch.full((T, CFG.d_model), 123.0, dtype=torch.float32, device="cuda")
    gpu.forward(x.cuda(), lg.cuda(), binding.F32, y=sentinel)
    torch.cuda.synchronize()
    assert bool((sentinel == 123.0).all())
    assert gpu.poll_status() == ERR["ERR_TIMEOUT"]
    assert gpu.poll_status() == 0                       # reading clears it
    y2 = gpu.forward(x.cuda(), lg.cuda(), binding.F32)
    assert gpu.poll_status() == 0
    assert torch.equal(y2, y)
    # argument errors of the debug call itself
    lib = binding.load()
    assert lib.dynamo_debug_expire_wait(gpu.ctx, 10, None) == ERR["ERR_ARG"]
    assert lib.dynamo_debug_expire_wait(None, 2_000_000, None) == ERR["ERR_NULL"]


def test_activation_beyond_the_operand_range_is_clamped_and_reported(tiny):
    gpu, ora = tiny["gpu"], tiny["ora"]
    T = 24
    x, lg = wl.activations(CFG, T, step=72).clone(), wl.router_logits(CFG, T, step=72)
    assert gpu.poll_status() == 0
    x[3, 17] = 5000.0                                   # 4992 in bf16: above the limit of 4080
    x[9, 300] = -float("inf")
    y = gpu.forward(x.cuda(), lg.cuda(), binding.F32)
    assert gpu.poll_status() == ERR["ERR_RANGE"]
    assert gpu.poll_status() == 0
    assert np.isfinite(y.cpu().numpy()).all()
    # defined outcome: exactly the forward of the clamped input (4080 is a bf16 value)
    xc = x.clone()
    xc[3, 17] = 4080.0
    xc[9, 300] = -4080.0
    assert float(xc[3, 17]) == 4080.0
    yc = gpu.forward(xc.cuda(), lg.cuda(), binding.F32)
    assert torch.equal(y, yc)
    gpu.poll_status()                                   # (a hidden value may itself have been clamped: cleared here)
    # inside the range nothing is reported and the oracle agrees: one large channel on a token of its own, small
    # enough that the hidden values h = silu(g) * u (which grow with its square) stay below the limit as well
    x2 = wl.activations(CFG, T, step=73).clone()
    x2[0, :] = 0
    x2[0, 5] = 64.0
    y2 = gpu.forward(x2.cuda(), lg.cuda(), binding.F32)
    assert gpu.poll_status() == 0
    ref = ora.forward(oracle.as_u16(x2), lg.numpy())["y"]
    assert rel_err(y2.cpu().numpy(), ref) <= TOL


def test_guard_blocks_intact_after_a_sweep_of_shapes_and_state_changes(tiny):
    gpu, pool, sets = tiny["gpu"], tiny["pool"], tiny["sets"]
    assert gpu.debug_check_guards() == 0
    for T in (1, 7, 8, 9, 24, 25, 33, 64, 129, 200, 256):
        x, lg = wl.activations(CFG, T, step=80 + T), wl.router_logits(CFG, T, step=80 + T)
        gpu.forward(x.cuda(), lg.cuda(), binding.F32)
        gpu.forward(x.cuda(), lg.cuda(), binding.BF16)
    for ev in range(3):
        new = wl.switch_event(CFG, pool, sets, 0, ev)
        for mode in (binding.SWITCH_REQUANT, binding.SWITCH_SELECT):
            gpu.set_switch_mode(mode)
            gpu.set_channel_switch(new)
    gpu.set_channel_precision([6] * CFG.n_experts)
    gpu.set_channel_precision([8] * CFG.n_experts)
    gpu.set_channel_switch(sets)
    gpu.set_stats_collection(True)
    x, lg = wl.activations(CFG, 64, step=99), wl.router_logits(CFG, 64, step=99)
    gpu.forward(x.cuda(), lg.cuda(), binding.F32)
    gpu.set_stats_collection(False)
    gpu.select_significant(CFG.max_sig // 2, reset=True)
    gpu.set_channel_switch(sets)
    assert gpu.poll_status() == 0
    assert gpu.debug_check_guards() == 0
    assert binding.load().dynamo_debug_check_guards(gpu.ctx, None, None) == ERR["ERR_NULL"]
