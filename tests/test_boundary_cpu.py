"""Host-side checks of the C-ABI that need no GPU: the library loads, exports every symbol the
header declares, and rejects bad arguments before touching the device."""
import os
import re

import numpy as np
import pytest

from paper_2503_21135_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return binding.load()


def _desc(**kw):
    base = dict(d_model=512, d_ff=1024, n_experts=8, n_shared=0, top_k=2, group_size=128, max_sig=32,
                cache_size=64, max_tokens=64, renormalize=1)
    base.update(kw)
    return binding.LayerDesc(**base)


def test_header_symbols_are_exported(lib):
    text = open(os.path.join(ROOT, "include", "dynamo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(dynamo_[a-z_]+)\s*\(", text))
    assert names == set(binding.EXPORTED)
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings(lib):
    assert binding.status_str(0) == "ok"
    assert "cache" in binding.status_str(8)


def test_create_rejects_bad_shapes(lib):
    for kw in (dict(d_model=500), dict(d_ff=1000), dict(group_size=32), dict(top_k=0), dict(top_k=9),
               dict(n_experts=0), dict(max_sig=80, cache_size=64), dict(max_tokens=0), dict(n_experts=1, top_k=2)):
        st, h = binding.dynamo_create(_desc(**kw))
        assert st == 2 and not h, kw
    st, h = binding.dynamo_create(_desc())
    assert st == 0 and h
    assert binding.dynamo_destroy(h) == 0
    assert binding.dynamo_destroy(None) == 1


def test_arena_bytes_and_bits_validation(lib):
    d = _desc()
    bits = np.array([2, 3, 4, 4, 4, 4, 8, 8], np.int32)
    st, wb, sb = binding.dynamo_arena_bytes(d, bits)
    assert st == 0
    # packed codes alone: 3*d*f*b/8 per expert; the arena must hold at least that and stay within 2x
    codes = sum(3 * 512 * 1024 * int(b) // 8 for b in bits)
    assert codes < wb < 2.5 * codes
    assert sb > 0
    bad = bits.copy()
    bad[0] = 5
    assert binding.dynamo_arena_bytes(d, bad)[0] == 3
    assert binding.dynamo_arena_bytes(d, None)[0] == 1
    # shared experts must be 8-bit
    ds = _desc(n_shared=1)
    assert binding.dynamo_arena_bytes(ds, np.array(list(bits) + [4], np.int32))[0] == 3
    assert binding.dynamo_arena_bytes(ds, np.array(list(bits) + [8], np.int32))[0] == 0


def test_cache_share_of_weight_storage(lib):
    # The channel cache of ~1 % of the channels costs about 1 % of the 16-bit weight storage
    # (the paper's 152.8 MB = 1.02 % figure is this ratio): P/d of the gate/up originals.
    d = _desc(d_model=4096, d_ff=14336, max_sig=41, cache_size=41)
    cache = 2 * 41 * 14336 * 2
    full = 3 * 4096 * 14336 * 2
    assert abs(cache / full - (2 / 3) * 41 / 4096) < 1e-12 and cache / full < 0.0102


def test_calls_before_pack_are_state_errors(lib):
    st, h = binding.dynamo_create(_desc())
    assert st == 0
    idx = np.zeros((8, 32), np.int32)
    cnt = np.zeros((8,), np.int32)
    assert binding.dynamo_set_channel_switch(h, idx, cnt, None) == 9
    assert binding.dynamo_moe_forward(h, 1, 1, 4, 1, binding.F32, None, None) == 9
    assert binding.dynamo_moe_forward_host(h, 1, 1, 4, 1, binding.F32, None) == 9
    assert binding.dynamo_export_codes(h, 0, 0, 1, 1, 1, 0, None) == 9
    assert binding.dynamo_expert_stream_bytes(h, 0)[0] == 9
    assert binding.dynamo_poll_status(h, None) == 9
    assert binding.dynamo_set_switch_mode(h, 7) == 2
    assert binding.dynamo_set_switch_mode(h, binding.SWITCH_REQUANT) == 0
    assert binding.dynamo_kernel_launches(h) == 0
    binding.dynamo_destroy(h)


def test_pack_argument_errors_detected_before_any_launch(lib):
    st, h = binding.dynamo_create(_desc())
    bits = np.array([2, 3, 4, 4, 4, 4, 8, 8], np.int32)
    pool = np.tile(np.arange(64, dtype=np.int32), (8, 1))
    ok_ptr = 256 * 1000
    args = dict(w=ok_ptr, arena=ok_ptr, nbytes=1 << 40)
    call = lambda **k: binding.dynamo_pack_experts(
        h, k.get("wg", args["w"]), args["w"], args["w"], k.get("bits", bits), k.get("pool", pool),
        k.get("arena", args["arena"]), k.get("nbytes", args["nbytes"]), args["arena"], args["nbytes"], None)
    assert call(wg=None) == 1
    bad = bits.copy(); bad[3] = 5
    assert call(bits=bad) == 3
    six = bits.copy(); six[3] = 6                      # INT6 is a base width
    assert binding.dynamo_arena_bytes(_desc(), six)[0] == 0
    p2 = pool.copy(); p2[2, 5] = p2[2, 4]
    assert call(pool=p2) == 7
    p3 = pool.copy(); p3[1, 63] = 512
    assert call(pool=p3) == 6
    assert call(arena=ok_ptr + 8) == 4
    assert call(nbytes=1024) == 5
    assert binding.dynamo_kernel_launches(h) == 0
    binding.dynamo_destroy(h)
