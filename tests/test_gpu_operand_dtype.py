"""Operand precision of the tensor-core products (Section V-B dequantizes to FP16; bf16 is the other common choice).
Codes and bf16 inputs are exact in both formats, so the formats differ only in the rounding of the hidden
activations.  Checked here on both FFN kernels: fp16 operands meet the output tolerance against the oracle; bf16
operands are explained by a float64 model that rounds the hidden activations to bf16, and their error against the
exact oracle is measured (it is the reason fp16 is the default)."""
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


def _bf16_rne(a: np.ndarray) -> np.ndarray:
    return torch.from_numpy(a.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()


def _model_with_bf16_hidden(ora, x_u16, logits):
    """The layer in float64 from the oracle's dense weights, hidden activations rounded to bf16."""
    x = np.array([[oracle.bf16_bits_to_f64(int(b)) for b in row] for row in x_u16])
    idx, w = oracle.route(logits, ora.k, ora.renormalize)
    y = np.zeros((x.shape[0], ora.d))
    for e in range(ora.E):
        toks, slots = np.nonzero(idx == e)
        if len(toks) == 0:
            continue
        wg, wu, wd = ora.effective_weights(e)
        g, u = x[toks] @ wg.T, x[toks] @ wu.T
        h = _bf16_rne(g / (1.0 + np.exp(-g)) * u)
        y[toks] += w[toks, slots][:, None] * (h @ wd.T)
    return y


@pytest.mark.parametrize("T", [8, 40, 200])     # streaming kernel only; both kernels at 200
def test_fp16_and_bf16_operands(T, record_property):
    wg, wu, wd, bits, pool, sets = make_inputs(CFG)
    ora = make_oracle_layer(CFG, wg, wu, wd, bits)
    gpu = make_gpu_layer(CFG, wg, wu, wd, bits, pool, max_tokens=256)
    gpu.set_channel_switch(sets)
    ora.set_channel_switch(sets)
    x, lg = wl.activations(CFG, T, step=5), wl.router_logits(CFG, T, step=5)
    ref = ora.forward(oracle.as_u16(x), lg.numpy())["y"]
    y16 = gpu.forward(x.cuda(), lg.cuda(), binding.F32).cpu().numpy()
    gpu.set_operand_dtype(binding.OPERAND_BF16)
    yb = gpu.forward(x.cuda(), lg.cuda(), binding.F32).cpu().numpy()
    gpu.set_operand_dtype(binding.OPERAND_FP16)
    y16_again = gpu.forward(x.cuda(), lg.cuda(), binding.F32).cpu().numpy()
    assert gpu.poll_status() == 0
    e16, eb = rel_err(y16, ref), rel_err(yb, ref)
    model = _model_with_bf16_hidden(ora, oracle.as_u16(x), lg.numpy())
    eb_model = rel_err(yb, model)
    record_property("fp16_operands_vs_oracle", e16)
    record_property("bf16_operands_vs_oracle", eb)
    print(f"T={T}: fp16 operands {e16:.2e}, bf16 operands {eb:.2e} against the oracle; "
          f"bf16 operands against the bf16-hidden model {eb_model:.2e}")
    assert e16 <= TOL
    assert np.array_equal(y16, y16_again)              # the setting is a switch, not a state change
    # The bf16 setting computes what it says: the model explains most of its distance from the exact result.  (Not
    # all of it: a hidden value that the kernel's fp32 sums put on the other side of a bf16 rounding boundary moves by
    # a whole bf16 step against the model, and the more tokens there are, the larger the worst such element.)
    rms = lambda a: float(np.sqrt(np.mean(np.square(a))))
    print(f"      rms(bf16 - model) / rms(bf16 - oracle) = {rms(yb - model) / rms(yb - ref):.3f}")
    assert eb_model < eb and rms(yb - model) <= 0.8 * rms(yb - ref)
    if T <= 8:
        assert eb_model <= 2e-3
    assert eb > e16 and eb <= 6e-2                     # and is less exact than fp16 operands
    lib = binding.load()
    assert lib.dynamo_set_operand_dtype(gpu.ctx, 7) == binding.STATUS_NAMES.index("ERR_ARG")
    assert lib.dynamo_set_operand_dtype(None, 0) == binding.STATUS_NAMES.index("ERR_NULL")
