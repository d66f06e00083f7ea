"""GPU parity at the full decode shape (config 2: Mixtral-8x7B-shaped layer, batch 1/8/32/64), in the
launch configuration the benchmark times.  Codes and params of every expert are compared bit-exactly
on all elements; outputs element by element against the float64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from helpers import make_gpu_layer, make_inputs, make_oracle_layer, rel_err
from paper_2503_21135_b200 import binding
from paper_2503_21135_b200 import workloads as wl

pytestmark = pytest.mark.gpu
TOL = 1e-2
CFG = wl.CONFIGS["decode"]


@pytest.fixture(scope="module")
def layer():
    wg, wu, wd, bits, pool, sets = make_inputs(CFG)
    gpu = make_gpu_layer(CFG, wg, wu, wd, bits, pool, max_tokens=64)
    ora = make_oracle_layer(CFG, wg, wu, wd, bits)
    gpu.set_channel_switch(sets)
    ora.set_channel_switch(sets)
    return dict(gpu=gpu, ora=ora, bits=bits, pool=pool, sets=sets)


def test_bits_recipe():
    bits = wl.bits_assignment(CFG)
    assert sorted(bits.tolist()) == [2, 2, 2, 3, 3, 4, 4, 8] and abs(np.mean(bits) - 3.5) < 1e-12


def test_all_codes_bit_exact(layer):
    gpu, ora = layer["gpu"], layer["ora"]
    for e in range(CFG.n_total):
        for mat in range(3):
            q, s, m = gpu.export_codes(e, mat)
            ref = ora.base[e][mat]
            assert torch.equal(q.cpu(), torch.from_numpy(ref.q)), (e, mat)
            assert np.array_equal(s.cpu().numpy().view(np.uint16), ref.s), (e, mat)
            assert np.array_equal(m.cpu().numpy().view(np.uint16), ref.m), (e, mat)
        if layer["bits"][e] < 8:
            for mat in range(2):
                q, s, m = gpu.export_codes(e, mat, binding.CODES_HI_ACTIVE)
                ref = ora.hi[e][mat]
                cols = layer["sets"][e]
                assert torch.equal(q.cpu()[:, cols], torch.from_numpy(ref.q[:, cols]))
                assert int(q.sum()) == int(ref.q[:, cols].astype(np.int64).sum())
                assert np.array_equal(s.cpu().numpy().view(np.uint16), ref.s)
                assert np.array_equal(m.cpu().numpy().view(np.uint16), ref.m)


@pytest.mark.parametrize("T", [1, 8, 32, 64])
def test_forward_parity(layer, T):
    gpu, ora = layer["gpu"], layer["ora"]
    x, lg = wl.activations(CFG, T, step=T), wl.router_logits(CFG, T, step=T)
    y, dbg = gpu.forward(x.cuda(), lg.cuda(), binding.F32, debug=True)
    torch.cuda.synchronize()
    assert gpu.poll_status() == 0
    ref = ora.forward(oracle.as_u16(x), lg.numpy())
    assert np.array_equal(dbg["idx"].cpu().numpy(), ref["idx"])
    assert np.array_equal(dbg["offsets"].cpu().numpy(), ref["offsets"])
    assert np.array_equal(dbg["perm"].cpu().numpy(), ref["perm"])
    assert np.max(np.abs(dbg["w"].cpu().numpy().astype(np.float64) - ref["w"])) <= 1e-6
    err = rel_err(y.cpu().numpy(), ref["y"])
    print(f"decode T={T}: max|gpu-oracle|/rms = {err:.3e}")
    assert err <= TOL, err


def test_stream_bytes_accounting(layer):
    gpu = layer["gpu"]
    d, f, G = CFG.d_model, CFG.d_ff, CFG.group_size
    for e in range(CFG.n_total):
        b = int(layer["bits"][e])
        base = 3 * d * f * b // 8 + 3 * d * f // G * 4
        hi = 2 * f * len(layer["sets"][e]) * 2 if (e < CFG.n_experts and b < 8) else 0
        assert gpu.stream_bytes(e) == base + hi
