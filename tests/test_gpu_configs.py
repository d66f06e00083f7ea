"""GPU parity at the full sizes of the prefill (config 3), fine-grained (config 4) and switch-stress
(config 5) workloads.  Routing, permutation and sampled codes are compared bit-exactly in full; the FFN
output is compared on a seeded, expert-stratified token subset that the float64 oracle can compute in
seconds (the subset rule: all experts touched, the two least-loaded experts over-sampled)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import make_gpu_layer, make_inputs, make_oracle_layer, rel_err, stratified_tokens
from paper_2503_21135_b200 import binding
from paper_2503_21135_b200 import workloads as wl

pytestmark = pytest.mark.gpu
TOL = 1e-2


def _check_forward(cfg, gpu, ora, T, n_sample, step=0, layer=0, all_of_two_least=False):
    x, lg = wl.activations(cfg, T, layer, step), wl.router_logits(cfg, T, layer, step)
    y, dbg = gpu.forward(x.cuda(), lg.cuda(), binding.F32, debug=True)
    torch.cuda.synchronize()
    assert gpu.poll_status() == 0
    idx, w = oracle.route(lg.numpy(), cfg.top_k)
    offsets, perm = oracle.permute(idx, cfg.n_experts)
    assert np.array_equal(dbg["idx"].cpu().numpy(), idx)
    assert np.array_equal(dbg["offsets"].cpu().numpy(), offsets)
    assert np.array_equal(dbg["perm"].cpu().numpy(), perm)
    assert np.max(np.abs(dbg["w"].cpu().numpy().astype(np.float64) - w)) <= 1e-6
    toks = (stratified_tokens(idx, cfg.n_experts, n_sample, seed=step, all_of_two_least=all_of_two_least)
            if n_sample < T else np.arange(T, dtype=np.int32))
    ref = ora.forward(oracle.as_u16(x), lg.numpy(), tokens=toks)["y"][toks]
    got = y.cpu().numpy()[toks]
    assert np.all(np.isfinite(y.cpu().numpy()))
    err = rel_err(got, ref)
    print(f"{cfg.name} T={T} sample={len(toks)}: max|gpu-oracle|/rms = {err:.3e}")
    assert err <= TOL, err
    return idx


def test_prefill_config():
    cfg = wl.CONFIGS["prefill"]
    wg, wu, wd, bits, pool, sets = make_inputs(cfg)
    assert bits.tolist() == [3, 3, 3, 3, 4, 4, 4, 8]
    gpu = make_gpu_layer(cfg, wg, wu, wd, bits, pool, max_tokens=8192)
    ora = make_oracle_layer(cfg, wg, wu, wd, bits)
    gpu.set_channel_switch(sets)
    ora.set_channel_switch(sets)
    # sampled codes: one expert per bit-width
    for e in (0, 4, 7):
        q, s, m = gpu.export_codes(e, binding.MAT_DOWN)
        assert torch.equal(q.cpu(), torch.from_numpy(ora.base[e][2].q))
        assert np.array_equal(s.cpu().numpy().view(np.uint16), ora.base[e][2].s)
    # the bench size: at least 512 stratified tokens, among them ALL tokens of the two least-loaded experts (every
    # row of their token tiles, ragged last tile included, is compared with the oracle)
    idx = _check_forward(cfg, gpu, ora, 4096, 512, all_of_two_least=True)
    counts = np.bincount(idx.ravel(), minlength=8)
    assert counts[7] == counts.max() and counts[7] > 2 * counts[0]        # Zipf skew: expert 7 most loaded
    # a ragged token count that leaves partial 32-token chunks in every expert
    _check_forward(cfg, gpu, ora, 1000, 48, step=1)
    # twice the bench size: 16384 expert rows, activation buffers of half a gigabyte (offsets beyond 2^29)
    _check_forward(cfg, gpu, ora, 8192, 40, step=5)
    # significant hidden units on the d_ff side at full size (P2 = 128 cached, 64 significant per expert):
    # prefill (tcgen05 pair kernel wrote h as operand tiles) and a decode-sized batch (streaming layout)
    pool_d = wl.cache_pool_down(cfg, 128)
    sets_d = wl.sig_sets_down(cfg, pool_d, 64)
    gpu.pack_down_cache(wd.cuda(), bits, pool_d, 64)
    ora.enable_down_side(oracle.as_u16(wd))
    gpu.set_channel_switch_down(sets_d)
    ora.set_channel_switch_down(sets_d)
    q, s, m = gpu.export_codes(0, binding.MAT_DOWN, binding.CODES_HI_ACTIVE)
    expect = np.zeros_like(ora.hi_down[0].q)
    expect[:, sets_d[0]] = ora.hi_down[0].q[:, sets_d[0]]
    assert torch.equal(q.cpu(), torch.from_numpy(expect))
    assert np.array_equal(s.cpu().numpy().view(np.uint16), ora.hi_down[0].s)
    _check_forward(cfg, gpu, ora, 4096, 64, step=2)
    _check_forward(cfg, gpu, ora, 64, 64, step=3)
    # the arithmetic order is fixed (static tiles, MMAs in k order, K splits summed in order), so repeated forwards
    # must agree bit for bit: a race between the roles of the tensor-core kernel would show up here
    x, lg = wl.activations(cfg, 4096, 0, 7).cuda(), wl.router_logits(cfg, 4096, 0, 7).cuda()
    y0 = gpu.forward(x, lg, binding.F32).clone()
    for _ in range(25):
        assert torch.equal(gpu.forward(x, lg, binding.F32), y0)
    assert gpu.poll_status() == 0


def test_finegrained_config_with_shared_experts():
    cfg = wl.CONFIGS["finegrained"]
    wg, wu, wd, bits, pool, sets = make_inputs(cfg)
    assert sorted(bits[:64].tolist(), reverse=True) == [4] * 16 + [3] * 24 + [2] * 24 and bits[64:].tolist() == [8, 8]
    gpu = make_gpu_layer(cfg, wg, wu, wd, bits, pool, max_tokens=2048)
    ora = make_oracle_layer(cfg, wg, wu, wd, bits)
    gpu.set_channel_switch(sets)
    ora.set_channel_switch(sets)
    for e in (0, 20, 50, 65):
        for mat in (binding.MAT_GATE, binding.MAT_DOWN):
            q, s, m = gpu.export_codes(e, mat)
            assert torch.equal(q.cpu(), torch.from_numpy(ora.base[e][mat].q))
            assert np.array_equal(m.cpu().numpy().view(np.uint16), ora.base[e][mat].m)
    idx = _check_forward(cfg, gpu, ora, 2048, 80)
    counts = np.bincount(idx.ravel(), minlength=64)
    assert counts.min() <= 8 and counts.max() >= 1000                     # from decode-like to prefill-like experts
    _check_forward(cfg, gpu, ora, 37, 37, step=2)
    # router GEMM + top-k fused in front (E = 64: two 32-expert register groups, k = 6, shared experts behind)
    w_r, bias = wl.router_weights(cfg)
    x = wl.activations(cfg, 300, 0, 5)
    y, lg, dbg = gpu.forward_router(x.cuda(), w_r.cuda(), bias.cuda(), binding.F32, want_logits=True, debug=True)
    torch.cuda.synchronize()
    assert gpu.poll_status() == 0
    lg = lg.cpu().numpy()
    ref_scores = oracle.router_scores(oracle.as_u16(x), oracle.as_u16(w_r), bias.numpy())
    bound = 2.0 * (cfg.d_model // 256 + 12) * 2.0 ** -24 * (np.abs(x.double().numpy()) @ np.abs(w_r.double().numpy()).T)
    assert np.all(np.abs(lg.astype(np.float64) - ref_scores) <= bound + 1e-7)
    idx_r, w_rt = oracle.route(lg, cfg.top_k)
    assert np.array_equal(dbg["idx"].cpu().numpy(), idx_r)
    assert np.max(np.abs(dbg["w"].cpu().numpy().astype(np.float64) - w_rt)) <= 1e-6
    assert torch.equal(gpu.forward(x.cuda(), torch.from_numpy(lg).cuda(), binding.F32), y)
    # significant hidden units on the d_ff side with G = 64 groups, 64 routed + 2 shared experts (the shared ones
    # and the 8-bit ones keep no set): codes of one 2-bit and one 4-bit expert, then a ragged forward
    pool_d = wl.cache_pool_down(cfg, 64)
    sets_d = wl.sig_sets_down(cfg, pool_d, 32)
    gpu.pack_down_cache(wd.cuda(), bits, pool_d, 32)
    ora.enable_down_side(oracle.as_u16(wd))
    gpu.set_channel_switch_down(sets_d)
    ora.set_channel_switch_down(sets_d)
    for e in (int(np.flatnonzero(bits[:64] == 2)[0]), int(np.flatnonzero(bits[:64] == 4)[0])):
        q, s_, m_ = gpu.export_codes(e, binding.MAT_DOWN, binding.CODES_HI_ACTIVE)
        expect = np.zeros_like(ora.hi_down[e].q)
        expect[:, sets_d[e]] = ora.hi_down[e].q[:, sets_d[e]]
        assert torch.equal(q.cpu(), torch.from_numpy(expect))
        assert np.array_equal(s_.cpu().numpy().view(np.uint16), ora.hi_down[e].s)
        assert np.array_equal(m_.cpu().numpy().view(np.uint16), ora.hi_down[e].m)
    _check_forward(cfg, gpu, ora, 300, 60, step=6)


def test_switch_stress_stack():
    """Config 5: the 16-layer stack at decode batch 16.  Every layer is compared with the oracle at step 0 and after
    the first switch event (one call for the whole stack); layers 0 and 1 also after the next two events.  The
    oracle of a layer is built, asked for its reference outputs and dropped (sixteen of them do not fit the host)."""
    cfg = wl.CONFIGS["switch"]
    n_layers, T = cfg.n_layers, 16
    assert n_layers == 16
    gpus, pools, cur, ws = [], [], [], None
    refs = {}          # (layer, event index or -1) -> dict(idx, perm, y)
    keep = {}          # oracle layers of the two layers followed further
    new_sets = []
    for l in range(n_layers):
        wg, wu, wd, bits, pool, sets = make_inputs(cfg, layer=l)
        g = make_gpu_layer(cfg, wg, wu, wd, bits, pool, max_tokens=T, workspace=ws)
        ws = g.workspace
        gpus.append(g)
        pools.append(pool)
        cur.append(sets)
        new = wl.switch_event(cfg, pool, sets, l, 0)
        for e in range(cfg.n_experts):
            assert len(np.setdiff1d(new[e], sets[e])) == 16               # 25 % of 64 swapped
        new_sets.append(new)
        need = set()
        for step in (0, 8):
            idx, _ = oracle.route(wl.router_logits(cfg, T, l, step).numpy(), cfg.top_k)
            need |= set(int(e) for e in idx.ravel())
        ora = make_oracle_layer(cfg, wg, wu, wd, bits, experts=sorted(need) if l >= 2 else None)
        for tag, s_, step in ((-1, sets, 0), (0, new, 8)):
            ora.set_channel_switch(s_)
            x, lg = wl.activations(cfg, T, l, step), wl.router_logits(cfg, T, l, step)
            refs[(l, tag)] = ora.forward(oracle.as_u16(x), lg.numpy())
        if l < 2:
            keep[l] = ora
        del ora, wg, wu, wd

    def check(l, tag, step):
        x, lg = wl.activations(cfg, T, l, step), wl.router_logits(cfg, T, l, step)
        y, dbg = gpus[l].forward(x.cuda(), lg.cuda(), binding.F32, debug=True)
        torch.cuda.synchronize()
        assert gpus[l].poll_status() == 0
        ref = refs[(l, tag)]
        assert np.array_equal(dbg["idx"].cpu().numpy(), ref["idx"])
        assert np.array_equal(dbg["perm"].cpu().numpy(), ref["perm"])
        err = rel_err(y.cpu().numpy(), ref["y"])
        assert err <= TOL, (l, tag, err)

    binding.set_channel_switch_many(gpus, cur)
    for l in range(n_layers):
        check(l, -1, 0)
    binding.set_channel_switch_many(gpus, new_sets)                        # one upload + one launch for the stack
    cur = new_sets
    for l in range(n_layers):
        check(l, 0, 8)
    step = 8
    for event in (1, 2):
        step += 8
        new = [wl.switch_event(cfg, pools[l], cur[l], l, event) for l in range(n_layers)]
        binding.set_channel_switch_many(gpus, new)
        cur = new
        for l in (0, 1):
            keep[l].set_channel_switch(new[l])
            x, lg = wl.activations(cfg, T, l, step), wl.router_logits(cfg, T, l, step)
            refs[(l, event)] = keep[l].forward(oracle.as_u16(x), lg.numpy())
            check(l, event, step)
    # all-or-nothing: one bad layer rejects the whole event and nothing changes
    x, lg = wl.activations(cfg, T, 0, 99).cuda(), wl.router_logits(cfg, T, 0, 99).cuda()
    y0 = gpus[0].forward(x, lg).clone()
    bad = [list(s) for s in cur]
    bad[n_layers - 1][3] = np.array([int(np.setdiff1d(np.arange(cfg.d_model), pools[n_layers - 1][3])[0])], np.int32)
    with pytest.raises(binding.DynamoError) as ei:
        binding.set_channel_switch_many(gpus, bad)
    assert ei.value.status == 8
    assert torch.equal(gpus[0].forward(x, lg), y0)
