"""Pins for the CPU oracle: every function is checked against something other than itself
(a library routine, a closed form, an invariant, brute force on tiny inputs)."""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2503_21135_b200 import workloads as wl


def bf16_bits(a: np.ndarray) -> np.ndarray:
    return oracle.as_u16(torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16))


def f16_to_f64(bits: np.ndarray) -> np.ndarray:
    return np.asarray(bits, dtype=np.uint16).view(np.float16).astype(np.float64)


# ---- number formats ----------------------------------------------------------------------

def test_f16_decode_all_patterns_matches_numpy():
    L = oracle.lib()
    for h in range(0, 65536, 1):
        ref = float(np.uint16(h).view(np.float16).astype(np.float64))
        got = L.orc_f16_to_f64(h)
        assert (np.isnan(ref) and np.isnan(got)) or ref == got, h


def test_f64_to_f16_single_rounding_matches_numpy():
    # numpy converts float64 -> float16 directly (one rounding, ties to even): a library pin.
    L = oracle.lib()
    pos = np.arange(0, 0x7c00, dtype=np.uint16).view(np.float16).astype(np.float64)
    mids = (pos[:-1] + pos[1:]) / 2.0                      # exact halves: the tie rule decides
    cases = [pos, mids, np.nextafter(mids, np.inf), np.nextafter(mids, -np.inf),
             np.array([65504.0, 65519.99, 65520.0, 65536.0, 1e6, 2.0 ** -25, 2.0 ** -26, 0.0, 5e-324])]
    rng = np.random.default_rng(1)
    cases.append(rng.standard_normal(20000) * np.exp(rng.uniform(-20, 12, 20000)))
    with np.errstate(over="ignore"):
        for arr in cases:
            for sign in (1.0, -1.0):
                v = arr * sign
                ref = v.astype(np.float16).view(np.uint16)
                got = np.array([L.orc_f64_to_f16(float(z)) for z in v], dtype=np.uint16)
                assert np.array_equal(ref, got)


def test_f64_to_f16_avoids_double_rounding():
    # 1 + 2^-11 + 2^-30 is just above a tie: via float32 it would first round to the tie and
    # then to even (1.0); one rounding gives the next fp16 up.
    v = 1.0 + 2.0 ** -11 + 2.0 ** -30
    assert oracle.f64_to_f16_bits(v) == 0x3c01
    assert oracle.f64_to_f16_bits(1.0 + 2.0 ** -11) == 0x3c00  # exact tie -> even


def test_bf16_decode_matches_torch():
    bits = np.arange(0, 65536, 7, dtype=np.uint16)
    ref = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    got = np.array([oracle.bf16_bits_to_f64(int(b)) for b in bits])
    ok = (ref == got) | (np.isnan(ref) & np.isnan(got))
    assert ok.all()


# ---- C1 quantizer ------------------------------------------------------------------------

@pytest.mark.parametrize("bits", [2, 3, 4, 6, 8])
@pytest.mark.parametrize("G", [64, 128])
def test_quantizer_bruteforce_nearest_level(bits, G):
    rng = np.random.default_rng(100 + bits + G)
    N, K = 6, 2 * G
    w = rng.standard_normal((N, K)) * 0.02
    w[:, 5] *= 20
    wb = bf16_bits(w)
    wv = torch.from_numpy(wb.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    q, s, m = oracle.quantize(wb, G, bits)
    L = 2 ** bits - 1
    sv, mv = f16_to_f64(s), f16_to_f64(m)
    assert q.max() <= L
    for n in range(N):
        for g in range(K // G):
            grp = wv[n, g * G:(g + 1) * G]
            lo, hi = grp.min(), grp.max()
            # parameters: fp16 of the range / L and of the minimum (library conversion)
            assert s[n, g] == np.float64((hi - lo) / L).astype(np.float16).view(np.uint16)
            assert m[n, g] == np.float64(lo).astype(np.float16).view(np.uint16)
            levels = sv[n, g] * np.arange(L + 1) + mv[n, g]
            for i, v in enumerate(grp):
                dist = np.abs(v - levels)
                best = np.flatnonzero(dist == dist.min())
                code = q[n, g * G + i]
                if len(best) == 1:
                    assert code == best[0]
                else:  # exact tie between two neighbouring levels -> the even one
                    assert code in best and code % 2 == 0
                # error bound: half a step inside the covered range, clamp overshoot outside
                bound = sv[n, g] / 2 + abs(lo - mv[n, g]) + L * abs(sv[n, g] - (hi - lo) / L) + 1e-300
                assert abs(v - levels[code]) <= bound


@pytest.mark.parametrize("bits", [2, 3, 4, 6, 8])
def test_quantizer_lossless_construction_and_ties(bits):
    # group = m + j*s with s a power of two and m fp16-exact  =>  q = j and s*q+m = w exactly
    G, L = 64, 2 ** bits - 1
    rng = np.random.default_rng(bits)
    j = rng.integers(0, L + 1, size=(3, 2 * G))
    j[:, 0], j[:, 1] = 0, L
    j[:, G], j[:, G + 1] = 0, L
    s0, m0 = 2.0 ** -6, -0.25
    w = m0 + j * s0
    wb = bf16_bits(w)
    assert np.array_equal(torch.from_numpy(wb.view(np.int16)).view(torch.bfloat16).double().numpy(), w)
    q, s, m = oracle.quantize(wb, G, bits)
    assert np.array_equal(q, j.astype(np.uint8))
    assert np.all(f16_to_f64(s) == s0) and np.all(f16_to_f64(m) == m0)
    assert np.array_equal(oracle.dequantize(q, s, m, G), w)


def test_quantizer_exact_half_goes_to_even():
    # levels 0, 1, 2, 3 (s = 1, m = 0, bits = 2); 0.5 -> 0, 1.5 -> 2, 2.5 -> 2
    G = 64
    w = np.zeros((1, G))
    w[0, :6] = [0.0, 3.0, 0.5, 1.5, 2.5, 1.0]
    q, s, m = oracle.quantize(bf16_bits(w), G, 2)
    assert f16_to_f64(s)[0, 0] == 1.0 and f16_to_f64(m)[0, 0] == 0.0
    assert list(q[0, :6]) == [0, 3, 0, 2, 2, 1]


def test_quantizer_constant_group():
    G = 128
    w = np.full((2, G), 0.375)
    q, s, m = oracle.quantize(bf16_bits(w), G, 4)
    assert np.all(q == 0) and np.all(f16_to_f64(s) == 1.0) and np.all(f16_to_f64(m) == 0.375)
    assert np.all(oracle.dequantize(q, s, m, G) == 0.375)


def test_dequantize_matches_numpy_formula():
    rng = np.random.default_rng(5)
    wb = bf16_bits(rng.standard_normal((8, 256)) * 0.02)
    q, s, m = oracle.quantize(wb, 128, 3)
    ref = np.repeat(f16_to_f64(s), 128, axis=1) * q + np.repeat(f16_to_f64(m), 128, axis=1)
    assert np.array_equal(oracle.dequantize(q, s, m, 128), ref)


# ---- C2 packing --------------------------------------------------------------------------

@pytest.mark.parametrize("bits", [2, 3, 4, 6, 8])
@pytest.mark.parametrize("K", [32, 33, 64, 100, 128, 384])
def test_pack_roundtrip(bits, K):
    rng = np.random.default_rng(bits * 1000 + K)
    L = 2 ** bits - 1
    pats = [rng.integers(0, L + 1, size=(5, K)), np.full((2, K), L), np.tile(np.array([0, L]), (1, K))[:, :K]]
    for q in pats:
        q = q.astype(np.uint8)
        words = oracle.pack_rows(q, bits)
        assert words.shape[1] == -(-K * bits // 32)
        assert np.array_equal(oracle.unpack_rows(words, K, bits), q)


def test_pack_bit_positions_hand_example():
    # hand-worked fixture: code k sits at bits [3k, 3k+3) of a little-endian stream
    fx = {}
    for line in open(os.path.join(os.path.dirname(__file__), "golden", "pack_3bit_words.txt")):
        if line.strip() and not line.startswith("#"):
            key, *vals = line.split()
            fx[key] = vals
    bits = int(fx["bits"][0])
    q = np.array([[int(v) for v in fx["codes"]]], dtype=np.uint8)
    expect = [int(v, 16) for v in fx["words"]]
    words = oracle.pack_rows(q, bits)
    assert [int(w) for w in words[0]] == expect
    stream = sum(int(c) << (bits * k) for k, c in enumerate(q[0]))
    assert expect[0] == stream & 0xFFFFFFFF and expect[1] == stream >> 32


def test_groups_stay_word_aligned():
    for G, bits in itertools.product((64, 128), (2, 3, 4, 6, 8)):
        assert (G * bits) % 32 == 0


# ---- C3 routing --------------------------------------------------------------------------

def test_route_matches_stable_sort_and_softmax():
    from scipy.special import softmax

    rng = np.random.default_rng(7)
    T, E, k = 200, 8, 2
    logits = rng.standard_normal((T, E)).astype(np.float32)
    logits[3, :] = 0.25                      # all equal -> idx 0..k-1, w = 1/k
    logits[4, [1, 5]] = 9.0                  # tie at the top -> lower index first
    idx, w = oracle.route(logits, k, True)
    order = np.argsort(-logits.astype(np.float64), axis=1, kind="stable")[:, :k]
    assert np.array_equal(idx, order.astype(np.int32))
    p = softmax(logits.astype(np.float64), axis=1)
    pk = np.take_along_axis(p, order, axis=1)
    assert np.allclose(w, pk / pk.sum(1, keepdims=True), rtol=1e-13, atol=0)
    assert np.allclose(w.sum(1), 1.0, atol=1e-14)
    assert list(idx[3]) == [0, 1] and np.allclose(w[3], 0.5)
    assert list(idx[4]) == [1, 5]
    idx2, w2 = oracle.route(logits, k, False)
    assert np.array_equal(idx2, idx) and np.allclose(w2, pk, rtol=1e-13)
    # k = E: weights are the softmax itself (library routine), in descending-logit order
    idx3, w3 = oracle.route(logits, E, True)
    assert np.allclose(np.take_along_axis(p, idx3.astype(np.int64), axis=1), w3, rtol=1e-13)
    # adding a per-row constant (exactly representable shift) changes nothing
    idx4, w4 = oracle.route(logits + np.float32(4.0), k, True)
    assert np.array_equal(idx4, idx) and np.allclose(w4, w, rtol=1e-6)


# ---- C4 permutation ----------------------------------------------------------------------

@pytest.mark.parametrize("T,E,k", [(1, 8, 2), (64, 8, 2), (300, 64, 6), (5, 4, 4)])
def test_permute_matches_python_sorted(T, E, k):
    rng = np.random.default_rng(T + E)
    logits = (rng.standard_normal((T, E)) + wl.popularity_bias(wl.CONFIGS["finegrained"])[:E]).astype(np.float32)
    idx, _ = oracle.route(logits, k, True)
    offsets, perm = oracle.permute(idx, E)
    ref = sorted(range(T * k), key=lambda i: (idx[i // k][i % k], i // k))
    assert list(perm) == ref
    assert sorted(perm.tolist()) == list(range(T * k))                  # bijection
    counts = np.bincount(idx.ravel(), minlength=E)
    assert np.array_equal(np.diff(offsets), counts) and offsets[0] == 0
    for e in range(E):
        toks = perm[offsets[e]:offsets[e + 1]] // k
        assert np.all(np.diff(toks) > 0)                                # ascending, no repeats


# ---- C5 / C6 FFN and switch semantics ----------------------------------------------------

def _tiny_layer(seed=0, E=4, k=2, d=128, f=192, G=64, bits=(2, 3, 4, 8), n_shared=0, T=9):
    rng = np.random.default_rng(seed)
    n = E + n_shared
    wg = rng.standard_normal((n, f, d)) * 0.02
    wu = rng.standard_normal((n, f, d)) * 0.02
    wd = rng.standard_normal((n, d, f)) * 0.02
    wg[:, :, 3] *= 20
    wu[:, :, 3] *= 20
    x = bf16_bits(rng.standard_normal((T, d)))
    logits = rng.standard_normal((T, E)).astype(np.float32)
    allbits = list(bits)[:E] + [8] * n_shared
    layer = oracle.OracleLayer(bf16_bits(wg), bf16_bits(wu), bf16_bits(wd), allbits, G, E, k)
    return layer, x, logits, (wg, wu, wd)


def _numpy_eff(layer, e):
    """Effective weights rebuilt independently of the C dequantizer."""
    G = layer.G
    mats = []
    for i, qm in enumerate(layer.base[e]):
        w = np.repeat(f16_to_f64(qm.s), G, axis=1) * qm.q + np.repeat(f16_to_f64(qm.m), G, axis=1)
        if i < 2 and e < layer.E and layer.hi[e] is not None and len(layer.sig[e]):
            h = layer.hi[e][i]
            w8 = np.repeat(f16_to_f64(h.s), G, axis=1) * h.q + np.repeat(f16_to_f64(h.m), G, axis=1)
            w[:, layer.sig[e]] = w8[:, layer.sig[e]]
        if i == 2 and e < layer.E and layer.hi_down[e] is not None and len(layer.sig_down[e]):
            h = layer.hi_down[e]
            w8 = np.repeat(f16_to_f64(h.s), G, axis=1) * h.q + np.repeat(f16_to_f64(h.m), G, axis=1)
            w[:, layer.sig_down[e]] = w8[:, layer.sig_down[e]]
        mats.append(w)
    return mats


def _dense_token_major(layer, x_u16, logits):
    """Brute force: loop tokens -> their k experts -> dense matmul with the effective weights."""
    xv = torch.from_numpy(x_u16.view(np.int16)).view(torch.bfloat16).double().numpy()
    T = xv.shape[0]
    order = np.argsort(-logits.astype(np.float64), axis=1, kind="stable")[:, :layer.k]
    z = logits.astype(np.float64)
    p = np.exp(z - z.max(1, keepdims=True))
    p /= p.sum(1, keepdims=True)
    eff = {e: _numpy_eff(layer, e) for e in range(layer.n_total)}
    y = np.zeros((T, layer.d))
    for t in range(T):
        pk = p[t, order[t]]
        pk = pk / pk.sum() if layer.renormalize else pk
        for j, e in enumerate(order[t]):
            g, u, dn = eff[int(e)]
            a, b = g @ xv[t], u @ xv[t]
            y[t] += pk[j] * (dn @ (a / (1 + np.exp(-a)) * b))
        for e in range(layer.E, layer.n_total):
            g, u, dn = eff[e]
            a, b = g @ xv[t], u @ xv[t]
            y[t] += dn @ (a / (1 + np.exp(-a)) * b)
    return y


@pytest.mark.parametrize("n_shared", [0, 2])
def test_forward_matches_dense_bruteforce(n_shared):
    layer, x, logits, _ = _tiny_layer(seed=11, n_shared=n_shared)
    layer.set_channel_switch([np.array([3, 7, 64, 100]), np.array([], np.int32), np.array([3]), np.array([1, 2])])
    out = layer.forward(x, logits)
    ref = _dense_token_major(layer, x, logits)
    assert np.max(np.abs(out["y"] - ref)) <= 1e-12 * np.max(np.abs(ref))
    # the effective weights the C FFN uses equal the numpy reconstruction
    for e in range(layer.n_total):
        for a, b in zip(layer.effective_weights(e), _numpy_eff(layer, e)):
            assert np.array_equal(a, b)


def test_lossless_8bit_reduces_to_plain_swiglu_mlp():
    # weights built as m + j*s per group (s power of two) are reproduced exactly by the 8-bit
    # quantizer, so the layer must equal an unquantized float64 SwiGLU MLP (torch matmul).
    rng = np.random.default_rng(3)
    d, f, G, T = 128, 128, 64, 5

    def lossless(N, K):
        j = rng.integers(0, 256, size=(N, K))
        j[:, 0::G], j[:, 1::G] = 0, 255
        return -0.5 + j * 2.0 ** -8

    wg, wu, wd = lossless(f, d), lossless(f, d), lossless(d, f)
    layer = oracle.OracleLayer(bf16_bits(wg)[None], bf16_bits(wu)[None], bf16_bits(wd)[None], [8], G, 1, 1)
    x = bf16_bits(rng.standard_normal((T, d)))
    out = layer.forward(x, np.zeros((T, 1), np.float32))
    xt = torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).double()
    a, b = xt @ torch.from_numpy(wg).T, xt @ torch.from_numpy(wu).T
    ref = (torch.nn.functional.silu(a) * b) @ torch.from_numpy(wd).T
    assert np.allclose(out["y"], ref.numpy(), rtol=1e-12, atol=1e-12)
    assert np.all(out["w"] == 1.0)


def test_zero_input_gives_zero():
    layer, x, logits, _ = _tiny_layer(seed=2)
    out = layer.forward(np.zeros_like(x), logits)
    assert np.all(out["y"] == 0.0)


def test_all_channels_switched_equals_uniform_8bit():
    layer, x, logits, (wg, wu, wd) = _tiny_layer(seed=5, bits=(2, 3, 4, 4))
    ref = oracle.OracleLayer(bf16_bits(wg), bf16_bits(wu), bf16_bits(wd), [8, 8, 8, 8], layer.G, 4, 2)
    # gate/up fully at 8-bit; W_down stays at base bits in both (set it equal for the comparison)
    for e in range(4):
        assert all(np.array_equal(layer.hi[e][i].q, ref.base[e][i].q) and
                   np.array_equal(layer.hi[e][i].s, ref.base[e][i].s) and
                   np.array_equal(layer.hi[e][i].m, ref.base[e][i].m) for i in (0, 1))
        ref.base[e] = (ref.base[e][0], ref.base[e][1], layer.base[e][2])
    layer.set_channel_switch([np.arange(layer.d)] * 4)
    assert np.array_equal(layer.forward(x, logits)["y"], ref.forward(x, logits)["y"])


@pytest.mark.parametrize("hb", [3, 4, 6])
def test_channel_precision_all_switched_equals_uniform_target(hb):
    # with every channel significant and target precision hb, gate/up are the expert's uniform hb-bit
    # quantization; a target equal to the base bit-width changes nothing; going back to 8 restores the state
    layer, x, logits, (wg, wu, wd) = _tiny_layer(seed=5, bits=(2, 3, 2, 8))
    ug, uu = bf16_bits(wg), bf16_bits(wu)
    layer.set_channel_switch([np.arange(0, layer.d, 3)] * 4)
    y8 = layer.forward(x, logits)["y"]
    layer.set_channel_precision([hb] * 4, ug, uu)
    ref = oracle.OracleLayer(ug, uu, bf16_bits(wd), [hb, hb, hb, 8], layer.G, 4, 2)
    for e in range(3):
        ref.base[e] = (ref.base[e][0], ref.base[e][1], layer.base[e][2])
    assert layer.hi[3] is None                                   # the 8-bit expert has no switch
    layer.set_channel_switch([np.arange(layer.d)] * 4)
    assert np.array_equal(layer.forward(x, logits)["y"], ref.forward(x, logits)["y"])
    if hb == 3:                                                  # expert 1 is 3-bit already: mask has no effect on it
        g0, u0, _ = layer.effective_weights(1)
        layer.set_channel_switch([np.array([], np.int32)] * 4)
        g1, u1, _ = layer.effective_weights(1)
        assert np.array_equal(g0, g1) and np.array_equal(u0, u1)
    layer.set_channel_precision([8] * 4, ug, uu)
    layer.set_channel_switch([np.arange(0, layer.d, 3)] * 4)
    assert np.array_equal(layer.forward(x, logits)["y"], y8)


def test_down_side_set_brute_force_and_identities():
    # significant INPUT channels of W_down (indices in [0, f)): the forward equals the token-major brute force on
    # independently rebuilt effective weights; all channels switched on both sides = the uniform 8-bit layer;
    # the empty set is the base; the 8-bit expert ignores its set
    layer, x, logits, (wg, wu, wd) = _tiny_layer(seed=12, bits=(2, 3, 4, 8))
    base = layer.forward(x, logits)["y"]
    layer.enable_down_side(bf16_bits(wd))
    assert layer.hi_down[3] is None and layer.hi_down[0] is not None
    assert np.array_equal(layer.forward(x, logits)["y"], base)
    layer.set_channel_switch([np.array([3, 7, 64]), np.array([], np.int32), np.array([3]), np.array([1])])
    layer.set_channel_switch_down([np.array([0, 5, 191]), np.array([64, 65]), np.array([], np.int32), np.array([2, 9])])
    out = layer.forward(x, logits)["y"]
    ref = _dense_token_major(layer, x, logits)
    assert np.max(np.abs(out - ref)) <= 1e-12 * np.max(np.abs(ref))
    assert not np.array_equal(out, base)
    for e in range(4):
        for a, b in zip(layer.effective_weights(e), _numpy_eff(layer, e)):
            assert np.array_equal(a, b)
    _, _, d0 = layer.effective_weights(0)
    changed = np.nonzero(np.any(d0 != oracle.dequantize(*[getattr(layer.base[0][2], k) for k in "qsm"], layer.G), axis=0))[0]
    assert set(changed.tolist()) <= {0, 5, 191} and len(changed) >= 2       # only the listed columns move
    # everything switched on both sides == uniform 8-bit layer
    ref8 = oracle.OracleLayer(bf16_bits(wg), bf16_bits(wu), bf16_bits(wd), [8, 8, 8, 8], layer.G, 4, 2)
    layer.set_channel_switch([np.arange(layer.d)] * 4)
    layer.set_channel_switch_down([np.arange(layer.f)] * 4)
    assert np.array_equal(layer.forward(x, logits)["y"], ref8.forward(x, logits)["y"])
    layer.set_channel_switch([np.array([], np.int32)] * 4)
    layer.set_channel_switch_down([np.array([], np.int32)] * 4)
    assert np.array_equal(layer.forward(x, logits)["y"], base)


@pytest.mark.parametrize("hb", [3, 4, 6])
def test_down_side_precision_all_switched_equals_uniform_target(hb):
    # every hidden unit significant at target hb: W_down is the expert's uniform hb-bit quantization (gate/up stay
    # at their base); a target equal to the base bit-width changes nothing; going back to 8 restores the state
    layer, x, logits, (wg, wu, wd) = _tiny_layer(seed=15, bits=(2, 3, 2, 8))
    ud = bf16_bits(wd)
    layer.enable_down_side(ud)
    some = [np.arange(0, layer.f, 5)] * 4
    layer.set_channel_switch_down(some)
    y8 = layer.forward(x, logits)["y"]
    layer.set_channel_precision_down([hb] * 4, ud)
    assert layer.hi_down[3] is None                              # the 8-bit expert has no switch
    ref = oracle.OracleLayer(bf16_bits(wg), bf16_bits(wu), ud, [hb, hb, hb, 8], layer.G, 4, 2)
    for e in range(3):
        ref.base[e] = (layer.base[e][0], layer.base[e][1], ref.base[e][2])
    layer.set_channel_switch_down([np.arange(layer.f)] * 4)
    assert np.array_equal(layer.forward(x, logits)["y"], ref.forward(x, logits)["y"])
    if hb == 3:                                                  # expert 1 is 3-bit already: its set has no effect
        _, _, d0 = layer.effective_weights(1)
        layer.set_channel_switch_down([np.array([], np.int32)] * 4)
        _, _, d1 = layer.effective_weights(1)
        assert np.array_equal(d0, d1)
    layer.set_channel_precision_down([8] * 4, ud)
    layer.set_channel_switch_down(some)
    assert np.array_equal(layer.forward(x, logits)["y"], y8)


def test_empty_set_is_base_and_8bit_expert_ignores_mask():
    layer, x, logits, _ = _tiny_layer(seed=6)           # expert 3 is 8-bit
    base = layer.forward(x, logits)["y"]
    layer.set_channel_switch([np.array([], np.int32)] * 3 + [np.arange(50)])
    assert np.array_equal(layer.forward(x, logits)["y"], base)
    layer.set_channel_switch([np.array([3, 9])] * 4)
    changed = layer.forward(x, logits)["y"]
    assert not np.array_equal(changed, base)
    # path independence: the state depends only on the last set installed
    layer.set_channel_switch([np.array([1])] * 4)
    layer.set_channel_switch([np.array([3, 9])] * 4)
    assert np.array_equal(layer.forward(x, logits)["y"], changed)


def test_significant_channels_reduce_error_on_outliers():
    # serving the outlier channel at 8-bit must bring a 2-bit expert closer to the unquantized MLP
    layer, x, logits, (wg, wu, wd) = _tiny_layer(seed=8, E=1, k=1, bits=(2,), T=16)
    xt = torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).double().numpy()
    r = lambda w: torch.from_numpy(w).to(torch.bfloat16).double().numpy()
    a, b = xt @ r(wg[0]).T, xt @ r(wu[0]).T
    h_ref = a / (1 + np.exp(-a)) * b
    def h_err():
        g, u, _ = layer.effective_weights(0)
        a2, b2 = xt @ g.T, xt @ u.T
        return np.linalg.norm(a2 / (1 + np.exp(-a2)) * b2 - h_ref)
    e0 = h_err()
    layer.set_channel_switch([np.array([3])])
    assert h_err() < e0


# ---- router scores (Section II-A gating network; a "next" row of the scope table) --------------

def test_router_scores_match_library_matmul_and_closed_forms():
    rng = np.random.default_rng(77)
    T, d, E = 9, 512, 8
    x = bf16_bits(rng.standard_normal((T, d)))
    w = bf16_bits(rng.standard_normal((E, d)) / np.sqrt(d))
    b = rng.standard_normal(E).astype(np.float32)
    xv = torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    wv = torch.from_numpy(w.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    s = oracle.router_scores(x, w, b)
    ref = xv @ wv.T + b.astype(np.float64)                       # library routine, float64
    assert np.max(np.abs(s - ref)) <= 1e-12 * np.max(np.abs(ref))
    assert np.array_equal(oracle.router_scores(x, w, None), s - b.astype(np.float64)[None, :]) or \
        np.max(np.abs(oracle.router_scores(x, w, None) - (s - b.astype(np.float64)[None, :]))) <= 1e-14
    # one-hot rows pick single input channels exactly; zero weights leave the bias
    onehot = np.zeros((E, d))
    cols = rng.permutation(d)[:E]
    onehot[np.arange(E), cols] = 1.0
    assert np.array_equal(oracle.router_scores(x, bf16_bits(onehot), None), xv[:, cols])
    assert np.array_equal(oracle.router_scores(x, bf16_bits(np.zeros((E, d))), b), np.tile(b.astype(np.float64), (T, 1)))
    # a transposed operand or a dropped bias would fail this hand-worked case: x = (1, 2, -3, 0.5),
    # w0 = (1, 0, 0, 0), w1 = (0.5, 0.5, 0.5, 0.5), bias = (0, 1)  ->  (1, 0.25 + 1)
    xs = bf16_bits(np.array([[1.0, 2.0, -3.0, 0.5]]))
    ws = bf16_bits(np.array([[1.0, 0.0, 0.0, 0.0], [0.5, 0.5, 0.5, 0.5]]))
    assert oracle.router_scores(xs, ws, np.array([0.0, 1.0], np.float32)).tolist() == [[1.0, 1.25]]


# ---- runtime selection of the significant channels ---------------------------------------------

def test_channel_stats_closed_forms():
    rng = np.random.default_rng(5)
    T, d, E, k, P = 40, 64, 4, 2, 8
    idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    pool = np.stack([np.sort(rng.permutation(d)[:P]) for _ in range(E)]).astype(np.int32)
    # |x| = 1 everywhere: the statistic is the number of tokens routed to the expert
    ones = bf16_bits(np.where(rng.random((T, d)) < 0.5, 1.0, -1.0))
    s = oracle.channel_stats_update(np.zeros((E, P)), ones, idx, pool)
    assert s.dtype == np.float64
    assert np.array_equal(s, np.tile(np.bincount(idx.ravel(), minlength=E).astype(np.float64)[:, None], (1, P)))
    # x zero outside one channel: only that channel (where cached) accumulates, by the routed tokens' |x|
    xz = np.zeros((T, d))
    xz[:, pool[1, 3]] = rng.integers(1, 5, size=T) * np.where(rng.random(T) < 0.5, 1.0, -1.0)
    s = oracle.channel_stats_update(np.zeros((E, P)), bf16_bits(xz), idx, pool)
    for e in range(E):
        toks = (idx == e).any(axis=1)
        expect = np.where(pool[e] == pool[1, 3], np.abs(xz[toks, pool[1, 3]]).sum(), 0.0)
        assert np.array_equal(s[e], expect)
    # two updates add: running total = first + second
    s2 = oracle.channel_stats_update(s, bf16_bits(xz), idx, pool)
    assert np.array_equal(s2, 2 * s)
    # exact sums: 2^24 + 1 + 1 keeps both ones, and the result does not depend on the order of the tokens
    big = np.zeros((3, d))
    big[0, pool[0, 0]], big[1, pool[0, 0]], big[2, pool[0, 0]] = 2.0 ** 24, 1.0, -1.0
    routed = np.zeros((3, 1), np.int32)
    s3 = oracle.channel_stats_update(np.zeros((E, P)), bf16_bits(big), routed, pool)
    assert s3[0, 0] == 2.0 ** 24 + 2
    assert np.array_equal(oracle.channel_stats_update(np.zeros((E, P)), bf16_bits(big[::-1].copy()), routed, pool), s3)
    # random data against a library routine: a masked matrix product of |x|
    xr = bf16_bits(rng.standard_normal((T, d)))
    xa = np.abs((xr.astype(np.uint32) << 16).view(np.float32)).astype(np.float64)
    s4 = oracle.channel_stats_update(np.zeros((E, P)), xr, idx, pool)
    member = np.stack([(idx == e).any(axis=1) for e in range(E)]).astype(np.float64)       # [E, T]
    full = member @ xa                                                                     # [E, d]
    assert np.allclose(s4, np.take_along_axis(full, pool.astype(np.int64), axis=1), rtol=1e-13, atol=0)


def test_select_significant_rank_rule():
    pool = np.array([[2, 5, 9, 11, 30, 31], [0, 1, 2, 3, 4, 5]], np.int32)
    stats = np.array([[1.0, 7.0, 7.0, 0.0, 3.0, 9.0], [0.0, 0.0, 0.0, 0.0, 0.0, 0.0]], np.float32)
    sets = oracle.select_significant(stats, pool, 4, [True, True])
    # hand-ranked: 9.0 (ch 31), then the tie 7.0 -> lower channel first (5 before 9), then 3.0 (ch 30)
    assert sets[0].tolist() == [31, 5, 9, 30]
    assert sets[1].tolist() == [0, 1, 2, 3]                             # all equal: lowest channels
    assert oracle.select_significant(stats, pool, 4, [False, True])[0].tolist() == []
    assert len(oracle.select_significant(stats, pool, 10, [True, True])[0]) == 6   # never more than the pool holds
    # distinct values: equals a library argsort; and nothing left out beats anything selected
    rng = np.random.default_rng(3)
    st = rng.permutation(64).astype(np.float32).reshape(1, 64)
    pl = np.arange(64, dtype=np.int32).reshape(1, 64) * 3
    got = oracle.select_significant(st, pl, 10, [True])[0]
    assert got.tolist() == (pl[0][np.argsort(-st[0], kind="stable")[:10]]).tolist()
    assert st[0][np.isin(pl[0], got)].min() > st[0][~np.isin(pl[0], got)].max()
