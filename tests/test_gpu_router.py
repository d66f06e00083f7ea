"""GPU parity of the forward with the router GEMM + top-k fused in front (Section II-A gating network).

The scores are accumulated in fp32 on the GPU and in float64 in the oracle, so the comparison has two parts:
(1) the scores agree within the fp32 accumulation bound; (2) GIVEN the GPU's own fp32 scores, selection,
permutation and output are exactly what the oracle computes from those scores (indices bit-exact).  A third check
compares the selection with the one from exact scores wherever the exact margins exceed the bound."""
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
    w_r, bias = wl.router_weights(CFG)
    return dict(ora=ora, gpu=gpu, w_r=w_r, bias=bias)


def _score_bound(x, w_r):
    """fp32 accumulation bound per score: (additions on the longest path) * 2^-24 * sum |x_c w_ec|, doubled."""
    n = x.shape[1] // 256 + 5 + 7   # terms per lane, butterfly levels, partials added
    return 2.0 * n * 2.0 ** -24 * (np.abs(x.double().numpy()) @ np.abs(w_r.double().numpy()).T)


@pytest.mark.parametrize("T", [1, 7, 64, 200])
@pytest.mark.parametrize("with_bias", [True, False])
def test_router_forward_parity(tiny, T, with_bias):
    gpu, ora, w_r = tiny["gpu"], tiny["ora"], tiny["w_r"]
    bias = tiny["bias"] if with_bias else None
    x = wl.activations(CFG, T, step=900 + T)
    y, lg, dbg = gpu.forward_router(x.cuda(), w_r.cuda(), None if bias is None else bias.cuda(), binding.F32,
                                    want_logits=True, debug=True)
    torch.cuda.synchronize()
    assert gpu.poll_status() == 0
    lg = lg.cpu().numpy()
    # (1) scores against the float64 oracle within the accumulation bound
    ref_scores = oracle.router_scores(oracle.as_u16(x), oracle.as_u16(w_r), None if bias is None else bias.numpy())
    bound = _score_bound(x, w_r) + 1e-7
    assert np.all(np.abs(lg.astype(np.float64) - ref_scores) <= bound)
    # (2) given the GPU's scores: selection, permutation, output as the oracle computes them
    ref = ora.forward(oracle.as_u16(x), lg)
    assert np.array_equal(dbg["idx"].cpu().numpy(), ref["idx"])
    assert np.array_equal(dbg["offsets"].cpu().numpy(), ref["offsets"])
    assert np.array_equal(dbg["perm"].cpu().numpy(), ref["perm"])
    assert np.max(np.abs(dbg["w"].cpu().numpy().astype(np.float64) - ref["w"])) <= 1e-6
    assert rel_err(y.cpu().numpy(), ref["y"]) <= TOL
    # and identical to the forward that is handed those scores
    y2 = gpu.forward(x.cuda(), torch.from_numpy(lg).cuda(), binding.F32)
    assert torch.equal(y2, y)
    # (3) against the selection from EXACT scores, wherever no two scores of a token are closer than the bound
    idx_exact, _ = oracle.route(ref_scores.astype(np.float32), CFG.top_k)
    srt = np.sort(ref_scores, axis=1)
    clear = np.min(np.diff(srt, axis=1), axis=1) > 2 * bound.max(axis=1) + 2.0 ** -20 * np.abs(srt).max(axis=1)
    assert clear.mean() > 0.9
    assert np.array_equal(dbg["idx"].cpu().numpy()[clear], idx_exact[clear])


def test_router_forward_errors(tiny):
    gpu, w_r = tiny["gpu"], tiny["w_r"].cuda()
    x = wl.activations(CFG, 4, step=1).cuda()
    y = torch.empty((4, CFG.d_model), dtype=torch.float32, device="cuda")
    st = binding.dynamo_moe_forward_router(gpu.ctx, x.data_ptr(), None, None, 4, y.data_ptr(), binding.F32, None, None, None)
    assert st == binding.STATUS_NAMES.index("ERR_NULL")
    st = binding.dynamo_moe_forward_router(gpu.ctx, x.data_ptr(), w_r.data_ptr() + 2, None, 4, y.data_ptr(), binding.F32,
                                           None, None, None)
    assert st == binding.STATUS_NAMES.index("ERR_ALIGN")
    st = binding.dynamo_moe_forward_router(gpu.ctx, x.data_ptr(), w_r.data_ptr(), None, 10 ** 6, y.data_ptr(), binding.F32,
                                           None, None, None)
    assert st == binding.STATUS_NAMES.index("ERR_TOKENS")
