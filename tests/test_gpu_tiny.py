"""GPU parity on the tiny layer (config 1): the CUDA path through the C-ABI against the CPU oracle.

Integer work (codes, params, routing indices, permutation) is bit-exact; the fp32 output must satisfy
max|gpu - oracle| / RMS(oracle) <= 1e-2, and the bf16 output must be the bf16 rounding of the fp32 one."""
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
    return dict(wg=wg, wu=wu, wd=wd, bits=bits, pool=pool, sets=sets, ora=ora, gpu=gpu)


def _u16(t):
    return t.cpu().numpy().view(np.uint16)


def test_packed_codes_and_params_bit_exact(tiny):
    gpu, ora = tiny["gpu"], tiny["ora"]
    for e in range(CFG.n_total):
        for mat in (binding.MAT_GATE, binding.MAT_UP, binding.MAT_DOWN):
            q, s, m = gpu.export_codes(e, mat, binding.CODES_BASE)
            ref = ora.base[e][mat]
            assert np.array_equal(q.cpu().numpy(), ref.q), (e, mat)
            assert np.array_equal(_u16(s), ref.s) and np.array_equal(_u16(m), ref.m), (e, mat)


def test_hi_pool_codes_bit_exact(tiny):
    gpu, ora, pool = tiny["gpu"], tiny["ora"], tiny["pool"]
    for e in range(CFG.n_experts):
        if tiny["bits"][e] >= 8:
            with pytest.raises(binding.DynamoError):
                gpu.export_codes(e, binding.MAT_GATE, binding.CODES_HI_POOL)
            continue
        for mat in (binding.MAT_GATE, binding.MAT_UP):
            q, s, m = gpu.export_codes(e, mat, binding.CODES_HI_POOL)
            ref = ora.hi[e][mat]
            expect = np.zeros_like(ref.q)
            expect[:, pool[e]] = ref.q[:, pool[e]]
            assert np.array_equal(q.cpu().numpy(), expect)
            assert np.array_equal(_u16(s), ref.s) and np.array_equal(_u16(m), ref.m)


def _forward_both(tiny, T, sets, step=0, renorm=True):
    gpu, ora = tiny["gpu"], tiny["ora"]
    x = wl.activations(CFG, T, step=step)
    lg = wl.router_logits(CFG, T, step=step)
    gpu.set_channel_switch(sets)
    ora.set_channel_switch(sets)
    y, dbg = gpu.forward(x.cuda(), lg.cuda(), binding.F32, debug=True)
    torch.cuda.synchronize()
    assert gpu.poll_status() == 0
    ref = ora.forward(oracle.as_u16(x), lg.numpy())
    return y.cpu().numpy(), {k: v.cpu().numpy() for k, v in dbg.items()}, ref, x, lg


@pytest.mark.parametrize("T", [64, 1, 7, 8, 9, 17, 33, 129])
def test_forward_parity_and_routing(tiny, T):
    y, dbg, ref, _, _ = _forward_both(tiny, T, tiny["sets"], step=T)
    assert np.array_equal(dbg["idx"], ref["idx"])
    assert np.array_equal(dbg["offsets"], ref["offsets"])
    assert np.array_equal(dbg["perm"], ref["perm"])
    assert np.max(np.abs(dbg["w"].astype(np.float64) - ref["w"])) <= 1e-6
    err = rel_err(y, ref["y"])
    assert err <= TOL, err


@pytest.mark.parametrize("T", [40, 64, 200])
def test_tensor_core_and_streaming_kernels_agree_with_the_oracle(tiny, T):
    """The same tokens through either FFN kernel: experts above 8 rows on the tcgen05 kernel, then
    every expert on the streaming kernel (large experts as 32-token chunks)."""
    gpu = tiny["gpu"]
    out = {}
    try:
        for rows in (8, 0):
            gpu.set_tc_min_rows(rows)
            y, _, ref, _, _ = _forward_both(tiny, T, tiny["sets"], step=300 + T)
            assert rel_err(y, ref["y"]) <= TOL, (rows, rel_err(y, ref["y"]))
            out[rows] = y
    finally:
        gpu.set_tc_min_rows(32)
    assert np.max(np.abs(out[8] - out[0])) <= TOL * np.sqrt(np.mean(out[0].astype(np.float64) ** 2))
    launches = []
    for rows in (8, 0):   # the two settings really take different paths: 8 vs 6 kernels per forward
        gpu.set_tc_min_rows(rows)
        n0 = gpu.kernel_launches()
        _forward_both(tiny, T, tiny["sets"], step=300 + T)
        launches.append(gpu.kernel_launches() - n0)
    gpu.set_tc_min_rows(32)
    assert launches[0] - launches[1] == 2, launches


def test_empty_sets_and_bf16_output(tiny):
    empty = [np.zeros((0,), np.int32)] * CFG.n_experts
    y, _, ref, x, lg = _forward_both(tiny, 64, empty, step=1)
    assert rel_err(y, ref["y"]) <= TOL
    yb = tiny["gpu"].forward(x.cuda(), lg.cuda(), binding.BF16)
    torch.cuda.synchronize()
    assert torch.equal(yb.cpu(), torch.from_numpy(y).to(torch.bfloat16))


def test_significant_channels_change_the_output_as_in_the_oracle(tiny):
    empty = [np.zeros((0,), np.int32)] * CFG.n_experts
    y0, _, r0, _, _ = _forward_both(tiny, 64, empty, step=2)
    y1, _, r1, _, _ = _forward_both(tiny, 64, tiny["sets"], step=2)
    d_gpu, d_ref = y1.astype(np.float64) - y0, r1["y"] - r0["y"]
    assert np.max(np.abs(d_ref)) > 0
    # the correction itself (not just the total) follows the oracle
    assert np.max(np.abs(d_gpu - d_ref)) <= TOL * np.sqrt(np.mean(r1["y"] ** 2))
    assert np.linalg.norm(d_gpu - d_ref) <= 0.05 * np.linalg.norm(d_ref)


def test_switch_is_path_independent_and_leaves_base_untouched(tiny):
    gpu, pool = tiny["gpu"], tiny["pool"]
    before = [gpu.export_codes(e, binding.MAT_GATE)[0].clone() for e in range(CFG.n_experts)]
    a = tiny["sets"]
    b = wl.switch_event(CFG, pool, a, 0, 0)
    assert any(not np.array_equal(x, y) for x, y in zip(a, b))
    x = wl.activations(CFG, 32, step=3).cuda()
    lg = wl.router_logits(CFG, 32, step=3).cuda()
    gpu.set_channel_switch(b)
    yb = gpu.forward(x, lg).clone()
    gpu.set_channel_switch(a)
    gpu.set_channel_switch(b)
    assert torch.equal(gpu.forward(x, lg), yb)
    for e in range(CFG.n_experts):
        assert torch.equal(gpu.export_codes(e, binding.MAT_GATE)[0], before[e])
    # active export lists exactly the installed set
    for e in range(CFG.n_experts):
        if tiny["bits"][e] >= 8:
            continue
        q, _, _ = gpu.export_codes(e, binding.MAT_UP, binding.CODES_HI_ACTIVE)
        ref = tiny["ora"].hi[e][1]
        expect = np.zeros_like(ref.q)
        expect[:, b[e]] = ref.q[:, b[e]]
        assert np.array_equal(q.cpu().numpy(), expect)


def test_requant_mode_matches_select_mode(tiny):
    gpu, pool = tiny["gpu"], tiny["pool"]
    a = tiny["sets"]
    b = wl.switch_event(CFG, pool, a, 0, 1)
    x = wl.activations(CFG, 16, step=4).cuda()
    lg = wl.router_logits(CFG, 16, step=4).cuda()
    gpu.set_switch_mode(binding.SWITCH_SELECT)
    gpu.set_channel_switch(a)
    gpu.set_channel_switch(b)
    y_sel = gpu.forward(x, lg).clone()
    q_sel = gpu.export_codes(0, binding.MAT_GATE, binding.CODES_HI_POOL)[0].clone()
    gpu.set_switch_mode(binding.SWITCH_REQUANT)
    gpu.set_channel_switch(a)
    gpu.set_channel_switch(b)
    assert torch.equal(gpu.forward(x, lg), y_sel)
    assert torch.equal(gpu.export_codes(0, binding.MAT_GATE, binding.CODES_HI_POOL)[0], q_sel)
    gpu.set_switch_mode(binding.SWITCH_SELECT)


def test_rejected_switch_keeps_previous_state(tiny):
    gpu, pool = tiny["gpu"], tiny["pool"]
    gpu.set_channel_switch(tiny["sets"])
    x = wl.activations(CFG, 8, step=5).cuda()
    lg = wl.router_logits(CFG, 8, step=5).cuda()
    y = gpu.forward(x, lg).clone()
    not_cached = np.setdiff1d(np.arange(CFG.d_model), pool[0])[:1]
    for bad, code in ((not_cached, 8), (np.array([CFG.d_model]), 6), (np.array([pool[0][0], pool[0][0]]), 7)):
        sets = list(tiny["sets"])
        sets[0] = bad.astype(np.int32)
        with pytest.raises(binding.DynamoError) as ei:
            gpu.set_channel_switch(sets)
        assert ei.value.status == code
    assert torch.equal(gpu.forward(x, lg), y)


def test_token_count_errors_and_empty_batch(tiny):
    gpu = tiny["gpu"]
    x = wl.activations(CFG, 4).cuda()
    lg = wl.router_logits(CFG, 4).cuda()
    assert binding.dynamo_moe_forward(gpu.ctx, x.data_ptr(), lg.data_ptr(), 0, 0, binding.F32, None, None) == 0
    assert binding.dynamo_moe_forward(gpu.ctx, x.data_ptr(), lg.data_ptr(), -1, 0, binding.F32, None, None) == 10
    assert binding.dynamo_moe_forward(gpu.ctx, x.data_ptr(), lg.data_ptr(), 257, 0, binding.F32, None, None) == 10


def test_host_buffer_entry_point_matches_device_one(tiny):
    gpu = tiny["gpu"]
    gpu.set_channel_switch(tiny["sets"])
    x = wl.activations(CFG, 64, step=6)
    lg = wl.router_logits(CFG, 64, step=6)
    y_dev = gpu.forward(x.cuda(), lg.cuda()).cpu()
    y_host = torch.empty((64, CFG.d_model), dtype=torch.float32).pin_memory()
    gpu.forward_host(x.pin_memory(), lg.pin_memory(), y_host)
    assert torch.equal(y_host, y_dev)


def test_all_channels_switched_equals_uniform_8bit():
    # identity: with every input channel significant, a low-bit expert's gate/up equal its 8-bit quantization
    cfg = wl.scaled(CFG, max_sig=256, cache_size=256, d_model=256, d_ff=256, n_experts=4, tokens=(16,))
    wg, wu, wd = wl.layer_weights(cfg)
    pool = np.tile(np.arange(256, dtype=np.int32), (4, 1))
    low = make_gpu_layer(cfg, wg, wu, wd, np.array([2, 3, 4, 4], np.int32), pool)
    hi = make_gpu_layer(cfg, wg, wu, wd, np.array([8, 8, 8, 8], np.int32), pool)
    low.set_channel_switch([np.arange(256, dtype=np.int32)] * 4)
    for e in range(4):
        for mat in (binding.MAT_GATE, binding.MAT_UP):
            a = low.export_codes(e, mat, binding.CODES_HI_ACTIVE)
            b = hi.export_codes(e, mat, binding.CODES_BASE)
            assert all(torch.equal(u, v) for u, v in zip(a, b))
    # outputs: oracle with all channels switched vs GPU
    ora = make_oracle_layer(cfg, wg, wu, wd, [2, 3, 4, 4])
    ora.set_channel_switch([np.arange(256)] * 4)
    x, lg = wl.activations(cfg, 16), wl.router_logits(cfg, 16)
    y = low.forward(x.cuda(), lg.cuda()).cpu().numpy()
    assert rel_err(y, ora.forward(oracle.as_u16(x), lg.numpy())["y"]) <= TOL


def test_forward_can_be_captured_in_a_cuda_graph(tiny):
    # a forward allocates nothing, synchronises nothing and zeroes its own work counters on the device, so a decode
    # step can be captured once and replayed; inputs are read from the captured buffers at replay time
    gpu = tiny["gpu"]
    gpu.set_channel_switch(tiny["sets"])
    T = 24
    x = wl.activations(CFG, T, step=11).cuda()
    lg = wl.router_logits(CFG, T, step=11).cuda()
    y_ref = gpu.forward(x, lg, binding.F32).clone()
    xs, ls = torch.zeros_like(x), torch.zeros_like(lg)
    ys = torch.empty((T, CFG.d_model), dtype=torch.float32, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        gpu.forward(xs, ls, binding.F32, y=ys)                 # warm-up on the capture stream
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    n0 = gpu.kernel_launches()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        gpu.forward(xs, ls, binding.F32, y=ys)
    per_forward = gpu.kernel_launches() - n0
    assert per_forward in (4, 6)       # small batches fuse routing, permutation and gather into one launch
    xs.copy_(x)
    ls.copy_(lg)
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(ys, y_ref)
    x2 = wl.activations(CFG, T, step=12).cuda()
    lg2 = wl.router_logits(CFG, T, step=12).cuda()
    xs.copy_(x2)
    ls.copy_(lg2)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(ys, gpu.forward(x2, lg2, binding.F32))
    assert gpu.poll_status() == 0


def test_misaligned_input_or_output_is_rejected(tiny):
    # x and y are read and written with 16-byte vectors: an address off by one element is an argument error
    gpu = tiny["gpu"]
    x = wl.activations(CFG, 5, step=13).cuda()
    lg = wl.router_logits(CFG, 5, step=13).cuda()
    y = torch.empty((5, CFG.d_model), dtype=torch.float32, device="cuda")
    ok = binding.dynamo_moe_forward(gpu.ctx, x.data_ptr(), lg.data_ptr(), 4, y.data_ptr(), binding.F32, None, None)
    assert ok == 0
    for xp, yp in ((x.data_ptr() + 2, y.data_ptr()), (x.data_ptr(), y.data_ptr() + 4)):
        st = binding.dynamo_moe_forward(gpu.ctx, xp, lg.data_ptr(), 4, yp, binding.F32, None, None)
        assert st == binding.STATUS_NAMES.index("ERR_ALIGN")
    torch.cuda.synchronize()
    assert gpu.poll_status() == 0
