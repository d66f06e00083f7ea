"""GPU parity for a variable target precision of the significant channels (Section IV-B: the replaced channels
are requantized to the precision the new data calls for, INT6 among the candidates): codes and parameters of the
channel cache bit-exact against the oracle's uniform b-bit quantization, the forward within the output
tolerance, and the state a function of the last precision installed."""
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


def _u16(t):
    return t.cpu().numpy().view(np.uint16)


@pytest.fixture(scope="module")
def lay():
    wg, wu, wd, bits, pool, sets = make_inputs(CFG)
    ora = make_oracle_layer(CFG, wg, wu, wd, bits)
    gpu = make_gpu_layer(CFG, wg, wu, wd, bits, pool, max_tokens=256)
    gpu.set_channel_switch(sets)
    ora.set_channel_switch(sets)
    return dict(ug=oracle.as_u16(wg), uu=oracle.as_u16(wu), bits=bits, pool=pool, sets=sets, ora=ora, gpu=gpu)


def _pool_state(gpu, bits):
    out = []
    for e in range(CFG.n_experts):
        if bits[e] < 8:
            for mat in (binding.MAT_GATE, binding.MAT_UP):
                out += [t.clone() for t in gpu.export_codes(e, mat, binding.CODES_HI_POOL)]
    return out


def _check_pool(lay):
    gpu, ora, pool = lay["gpu"], lay["ora"], lay["pool"]
    for e in range(CFG.n_experts):
        if lay["bits"][e] >= 8:
            continue
        for mat in (binding.MAT_GATE, binding.MAT_UP):
            q, s, m = gpu.export_codes(e, mat, binding.CODES_HI_POOL)
            ref = ora.hi[e][mat]
            expect = np.zeros_like(ref.q)
            expect[:, pool[e]] = ref.q[:, pool[e]]
            assert np.array_equal(q.cpu().numpy(), expect), (e, mat)
            assert np.array_equal(_u16(s), ref.s) and np.array_equal(_u16(m), ref.m), (e, mat)


def _check_forward(lay, T, step):
    x, lg = wl.activations(CFG, T, step=step), wl.router_logits(CFG, T, step=step)
    y = lay["gpu"].forward(x.cuda(), lg.cuda(), binding.F32)
    torch.cuda.synchronize()
    assert lay["gpu"].poll_status() == 0
    ref = lay["ora"].forward(oracle.as_u16(x), lg.numpy())["y"]
    assert rel_err(y.cpu().numpy(), ref) <= TOL
    return y


@pytest.mark.parametrize("hb", [6, 4, 3, 2])
def test_uniform_target_precision(lay, hb):
    gpu, ora = lay["gpu"], lay["ora"]
    E = CFG.n_experts
    before = _pool_state(gpu, lay["bits"])
    y8 = _check_forward(lay, 40, step=1).clone()
    gpu.set_channel_precision([hb] * E)
    ora.set_channel_precision([hb] * E, lay["ug"], lay["uu"])
    _check_pool(lay)
    q = gpu.export_codes(0, binding.MAT_GATE, binding.CODES_HI_POOL)[0]
    assert int(q.max()) <= 2 ** hb - 1
    y = _check_forward(lay, 40, step=1)              # streaming path
    assert not torch.equal(y, y8)
    _check_forward(lay, 200, step=2)                 # tensor-core path for the loaded experts
    # back to 8 bits: the cache is exactly what pack wrote
    gpu.set_channel_precision([8] * E)
    ora.set_channel_precision([8] * E, lay["ug"], lay["uu"])
    after = _pool_state(gpu, lay["bits"])
    assert all(torch.equal(a, b) for a, b in zip(before, after))
    assert torch.equal(_check_forward(lay, 40, step=1), y8)


def test_mixed_target_precision_and_switches(lay):
    gpu, ora, pool = lay["gpu"], lay["ora"], lay["pool"]
    E = CFG.n_experts
    hb = [(6, 4, 8, 3)[e % 4] for e in range(E)]
    gpu.set_channel_precision(hb)
    ora.set_channel_precision(hb, lay["ug"], lay["uu"])
    _check_pool(lay)
    _check_forward(lay, 33, step=3)
    # a switch event at the new precision, in both switch modes
    new = wl.switch_event(CFG, pool, lay["sets"], 0, 0)
    ora.set_channel_switch(new)
    for mode in (binding.SWITCH_SELECT, binding.SWITCH_REQUANT):
        gpu.set_switch_mode(mode)
        gpu.set_channel_switch(lay["sets"])
        gpu.set_channel_switch(new)
        _check_pool(lay)
        _check_forward(lay, 33, step=4)
        for e in range(E):
            if lay["bits"][e] >= 8:
                continue
            qa = gpu.export_codes(e, binding.MAT_UP, binding.CODES_HI_ACTIVE)[0].cpu().numpy()
            ref = ora.hi[e][1]
            expect = np.zeros_like(ref.q)
            expect[:, new[e]] = ref.q[:, new[e]]
            assert np.array_equal(qa, expect)
    gpu.set_switch_mode(binding.SWITCH_SELECT)
    # installing the same vector again launches nothing and changes nothing
    n0 = gpu.kernel_launches()
    gpu.set_channel_precision(hb)
    assert gpu.kernel_launches() == n0
    gpu.set_channel_switch(lay["sets"])
    ora.set_channel_switch(lay["sets"])
    gpu.set_channel_precision([8] * E)
    ora.set_channel_precision([8] * E, lay["ug"], lay["uu"])


def test_precision_errors_leave_state(lay):
    gpu = lay["gpu"]
    E = CFG.n_experts
    x, lg = wl.activations(CFG, 8, step=6).cuda(), wl.router_logits(CFG, 8, step=6).cuda()
    y0 = gpu.forward(x, lg).clone()
    for bad in (5, 7, 0, 16, -1):
        hb = [6] * E
        hb[E - 1] = bad
        with pytest.raises(binding.DynamoError) as ei:
            gpu.set_channel_precision(hb)
        assert ei.value.status == binding.STATUS_NAMES.index("ERR_BITS")
    assert torch.equal(gpu.forward(x, lg), y0)
    fresh = binding.DynamoLayer.from_config(CFG, max_tokens=16)
    with pytest.raises(binding.DynamoError) as ei:
        fresh.set_channel_precision([8] * E)
    assert ei.value.status == binding.STATUS_NAMES.index("ERR_STATE")


def test_recluster_on_new_data_sets_the_target_precision(lay):
    # Section IV-B loop: expert loads measured on the data at hand -> Algorithm 1 -> per-expert target precision of the
    # cached channels (higher or lower than before), on both sides
    gpu, ora = lay["gpu"], lay["ora"]
    E = CFG.n_experts
    x, lg = wl.activations(CFG, 256, step=9), wl.router_logits(CFG, 256, step=9)
    _, dbg = gpu.forward(x.cuda(), lg.cuda(), binding.F32, debug=True)
    counts = np.diff(dbg["offsets"].cpu().numpy()).astype(np.float64)
    assert counts.sum() == 256 * CFG.top_k
    share = counts / counts.sum()
    got = binding.assign_bits(share, [8, 6, 4, 3], token_share=share, overlap=0.05)
    U0 = oracle.assign.initial_memberships(share.tolist(), 4, 2.0)
    V, U, _, _ = oracle.assign.fuzzy_cmeans(share[:, None].tolist(), U0)
    ref_bits, _ = oracle.assign.assign_bits(V, U, [8, 6, 4, 3], overlap=0.05)
    assert got["bits"].tolist() == ref_bits and len(set(ref_bits)) >= 2
    gpu.set_channel_precision(got["bits"])
    ora.set_channel_precision(ref_bits, lay["ug"], lay["uu"])
    _check_pool(lay)
    _check_forward(lay, 64, step=10)
    gpu.set_channel_precision([8] * E)
    ora.set_channel_precision([8] * E, lay["ug"], lay["uu"])
