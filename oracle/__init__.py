"""CPU oracle of the DynaMo quantized-MoE hot path.  TEST INFRASTRUCTURE ONLY.

A thin ctypes wrapper over ``dynamo_oracle.c`` (plain C, float64) plus the few
steps that are clearer in numpy (the weighted combine, the layer bookkeeping).
Nothing in here is imported by the CUDA library or its Python binding; only the
tests, the smoke check and the benchmark's CPU-baseline leg may import it.

What follows the paper: expert-level uniform mixed-precision quantization
(Section IV-A), channel cache + channel-level switching (Sections IV-B, V-A),
packing of low-bit codes into 32-bit words and dequantize-then-multiply
(Section V-B), Top-K expert selection and one-to-many dispatch (Section II-A).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dynamo_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None

HI_BITS = 8


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (IEEE double, no FMA contraction, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", "-std=c11",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.check_call(cmd)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB)
        u8p, u16p, u32p = (ctypes.POINTER(ctypes.c_uint8), ctypes.POINTER(ctypes.c_uint16),
                           ctypes.POINTER(ctypes.c_uint32))
        i32p, f32p, f64p = (ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_float),
                            ctypes.POINTER(ctypes.c_double))
        i64, ci = ctypes.c_int64, ctypes.c_int
        L.orc_bf16_to_f64.restype = ctypes.c_double
        L.orc_bf16_to_f64.argtypes = [ctypes.c_uint16]
        L.orc_f16_to_f64.restype = ctypes.c_double
        L.orc_f16_to_f64.argtypes = [ctypes.c_uint16]
        L.orc_f64_to_f16.restype = ctypes.c_uint16
        L.orc_f64_to_f16.argtypes = [ctypes.c_double]
        L.orc_quantize.restype = None
        L.orc_quantize.argtypes = [u16p, i64, i64, ci, ci, u8p, u16p, u16p]
        L.orc_dequantize.restype = None
        L.orc_dequantize.argtypes = [u8p, u16p, u16p, i64, i64, ci, f64p]
        L.orc_packed_words.restype = i64
        L.orc_packed_words.argtypes = [i64, ci]
        L.orc_pack_rows.restype = None
        L.orc_pack_rows.argtypes = [u8p, i64, i64, ci, u32p]
        L.orc_unpack_rows.restype = None
        L.orc_unpack_rows.argtypes = [u32p, i64, i64, ci, u8p]
        L.orc_router_scores.restype = None
        L.orc_router_scores.argtypes = [u16p, u16p, f32p, i64, i64, ci, f64p]
        L.orc_route.restype = None
        L.orc_route.argtypes = [f32p, i64, ci, ci, ci, i32p, f64p]
        L.orc_permute.restype = None
        L.orc_permute.argtypes = [i32p, i64, ci, ci, i32p, i32p]
        L.orc_expert_ffn.restype = None
        L.orc_expert_ffn.argtypes = ([u16p, i32p, i64, i64, i64, ci] + [u8p, u16p, u16p] * 5 + [u8p] +
                                     [u8p, u16p, u16p] + [u8p, f64p])
        L.orc_threads.restype = ci
        L.orc_set_threads.argtypes = [ci]
        _lib = L
    return _lib


def _p(a: Optional[np.ndarray], ct):
    if a is None:
        return ctypes.cast(None, ctypes.POINTER(ct))
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.POINTER(ct))


def threads() -> int:
    return int(lib().orc_threads())


def set_threads(n: int) -> None:
    lib().orc_set_threads(int(n))


# ---- scalar conversions (exposed for the pins) -----------------------------------------

def f64_to_f16_bits(x: float) -> int:
    return int(lib().orc_f64_to_f16(float(x)))


def f16_bits_to_f64(h: int) -> float:
    return float(lib().orc_f16_to_f64(int(h)))


def bf16_bits_to_f64(h: int) -> float:
    return float(lib().orc_bf16_to_f64(int(h)))


def as_u16(t) -> np.ndarray:
    """bf16 torch tensor (CPU) -> numpy uint16 bit patterns, same shape."""
    import torch

    assert t.dtype == torch.bfloat16
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


# ---- C1 / C2 -------------------------------------------------------------------------------

def quantize(w_u16: np.ndarray, G: int, bits: int):
    """Group-wise asymmetric uniform quantizer.  w_u16 [N,K] bf16 bits -> (q u8 [N,K], s, m u16 [N,K/G])."""
    w_u16 = np.ascontiguousarray(w_u16, dtype=np.uint16)
    N, K = w_u16.shape
    assert K % G == 0 and bits in (2, 3, 4, 6, 8)
    q = np.empty((N, K), np.uint8)
    s = np.empty((N, K // G), np.uint16)
    m = np.empty((N, K // G), np.uint16)
    lib().orc_quantize(_p(w_u16, ctypes.c_uint16), N, K, G, bits, _p(q, ctypes.c_uint8),
                       _p(s, ctypes.c_uint16), _p(m, ctypes.c_uint16))
    return q, s, m


def dequantize(q: np.ndarray, s: np.ndarray, m: np.ndarray, G: int) -> np.ndarray:
    N, K = q.shape
    out = np.empty((N, K), np.float64)
    lib().orc_dequantize(_p(np.ascontiguousarray(q), ctypes.c_uint8), _p(np.ascontiguousarray(s), ctypes.c_uint16),
                         _p(np.ascontiguousarray(m), ctypes.c_uint16), N, K, G, _p(out, ctypes.c_double))
    return out


def pack_rows(q: np.ndarray, bits: int) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.uint8)
    N, K = q.shape
    nw = int(lib().orc_packed_words(K, bits))
    out = np.empty((N, nw), np.uint32)
    lib().orc_pack_rows(_p(q, ctypes.c_uint8), N, K, bits, _p(out, ctypes.c_uint32))
    return out


def unpack_rows(words: np.ndarray, K: int, bits: int) -> np.ndarray:
    words = np.ascontiguousarray(words, dtype=np.uint32)
    N = words.shape[0]
    q = np.empty((N, K), np.uint8)
    lib().orc_unpack_rows(_p(words, ctypes.c_uint32), N, K, bits, _p(q, ctypes.c_uint8))
    return q


# ---- C3 / C4 -------------------------------------------------------------------------------

def router_scores(x_u16: np.ndarray, w_u16: np.ndarray, bias: Optional[np.ndarray] = None) -> np.ndarray:
    """Router scores float64 [T, E] = x . w_r^T + bias from bf16 bit patterns (Section II-A)."""
    x_u16 = np.ascontiguousarray(x_u16, dtype=np.uint16)
    w_u16 = np.ascontiguousarray(w_u16, dtype=np.uint16)
    T, d = x_u16.shape
    E = w_u16.shape[0]
    assert w_u16.shape[1] == d
    b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    out = np.empty((T, E), dtype=np.float64)
    lib().orc_router_scores(_p(x_u16, ctypes.c_uint16), _p(w_u16, ctypes.c_uint16), _p(b, ctypes.c_float), T, d, E,
                            _p(out, ctypes.c_double))
    return out


def route(logits: np.ndarray, k: int, renormalize: bool = True):
    """Top-k routing.  logits fp32 [T,E] -> (idx int32 [T,k], w float64 [T,k])."""
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    T, E = logits.shape
    idx = np.empty((T, k), np.int32)
    w = np.empty((T, k), np.float64)
    lib().orc_route(_p(logits, ctypes.c_float), T, E, k, int(bool(renormalize)), _p(idx, ctypes.c_int32),
                    _p(w, ctypes.c_double))
    return idx, w


def permute(idx: np.ndarray, E: int):
    """Stable counting sort of the (token, slot) pairs by expert -> (offsets int32 [E+1], perm int32 [T*k])."""
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    T, k = idx.shape
    offsets = np.empty((E + 1,), np.int32)
    perm = np.empty((T * k,), np.int32)
    lib().orc_permute(_p(idx, ctypes.c_int32), T, k, E, _p(offsets, ctypes.c_int32), _p(perm, ctypes.c_int32))
    return offsets, perm


# ---- C5 / C6: a layer ----------------------------------------------------------------------

class QuantMatrix:
    """Codes and fp16 parameters of one quantized matrix."""

    __slots__ = ("q", "s", "m")

    def __init__(self, q, s, m):
        self.q, self.s, self.m = q, s, m


class OracleLayer:
    """One MoE layer in the oracle: quantized experts, significant sets, forward.

    ``w_gate``/``w_up``: uint16 (bf16 bits) [E+Es, f, d]; ``w_down``: [E+Es, d, f].
    ``bits``: base bit-width per expert.  The 8-bit ("hi") quantization of W_gate and
    W_up is kept for every routed expert with base bits < 8: a significant channel takes
    the value it has in that uniform 8-bit quantization.  The same holds on the d_ff side
    (``set_channel_switch_down``): a significant INPUT channel c of W_down, c in [0, f),
    takes column c of the uniform 8-bit quantization of W_down.
    """

    def __init__(self, w_gate, w_up, w_down, bits: Sequence[int], G: int, n_experts: int, top_k: int,
                 renormalize: bool = True, experts: Optional[Sequence[int]] = None):
        self.G, self.E, self.k = int(G), int(n_experts), int(top_k)
        self.n_total = w_gate.shape[0]
        self.f, self.d = w_gate.shape[1], w_gate.shape[2]
        self.bits = [int(b) for b in bits]
        self.renormalize = bool(renormalize)
        self.base: List[Optional[tuple]] = [None] * self.n_total
        self.hi: List[Optional[tuple]] = [None] * self.n_total
        todo = range(self.n_total) if experts is None else experts
        for e in todo:
            b = self.bits[e]
            self.base[e] = tuple(QuantMatrix(*quantize(w[e], G, b)) for w in (w_gate, w_up, w_down))
            if e < self.E and b < HI_BITS:
                self.hi[e] = tuple(QuantMatrix(*quantize(w[e], G, HI_BITS)) for w in (w_gate, w_up))
        self.sig: List[np.ndarray] = [np.zeros((0,), np.int32) for _ in range(self.E)]
        self.hi_down: List[Optional[QuantMatrix]] = [None] * self.n_total
        self.sig_down: List[np.ndarray] = [np.zeros((0,), np.int32) for _ in range(self.E)]

    def enable_down_side(self, w_down) -> None:
        """Keep the uniform 8-bit quantization of W_down for every routed expert with base bits < 8
        (Section IV-B applied to the channels of the second projection: its input channels are the d_ff
        hidden units).  w_down: the original bf16 bit patterns [E+Es, d, f]."""
        for e in range(self.E):
            if self.base[e] is not None and self.bits[e] < HI_BITS:
                self.hi_down[e] = QuantMatrix(*quantize(w_down[e], self.G, HI_BITS))

    def set_channel_precision_down(self, hi_bits: Sequence[int], w_down) -> None:
        """Precision the significant hidden units are served at, per routed expert (Section IV-B, as
        ``set_channel_precision`` but for the input channels of W_down): a significant hidden unit of expert e
        takes the column it has in the expert's uniform hi_bits[e]-bit quantization of the ORIGINAL W_down
        (same groups, same quantizer).  w_down: the original bf16 bit patterns [E+Es, d, f]."""
        assert len(hi_bits) == self.E
        for e in range(self.E):
            if self.hi_down[e] is not None:
                self.hi_down[e] = QuantMatrix(*quantize(w_down[e], self.G, int(hi_bits[e])))

    def set_channel_switch_down(self, sets: Sequence[np.ndarray]) -> None:
        """Install the significant set of W_down's input channels (indices in [0, f)) of every routed expert."""
        assert len(sets) == self.E
        self.sig_down = [np.unique(np.asarray(s, dtype=np.int32)) for s in sets]

    def mask_down(self, e: int) -> Optional[np.ndarray]:
        if e >= self.E or self.hi_down[e] is None or len(self.sig_down[e]) == 0:
            return None
        mk = np.zeros((self.f,), np.uint8)
        mk[self.sig_down[e]] = 1
        return mk

    def set_channel_precision(self, hi_bits: Sequence[int], w_gate, w_up) -> None:
        """Precision the significant channels are served at, per routed expert (Section IV-B: the replaced
        channels are requantized to the precision the new data calls for): a significant channel of expert e
        takes the value it has in the expert's uniform hi_bits[e]-bit quantization of the ORIGINAL W_gate / W_up
        (same groups, same quantizer).  w_gate, w_up: the original bf16 bit patterns [E+Es, f, d]."""
        assert len(hi_bits) == self.E
        for e in range(self.E):
            if self.hi[e] is not None:
                self.hi[e] = tuple(QuantMatrix(*quantize(w[e], self.G, int(hi_bits[e]))) for w in (w_gate, w_up))

    def set_channel_switch(self, sets: Sequence[np.ndarray]) -> None:
        """Install the significant-channel set of every routed expert (state depends only on it)."""
        assert len(sets) == self.E
        self.sig = [np.unique(np.asarray(s, dtype=np.int32)) for s in sets]

    def mask(self, e: int) -> Optional[np.ndarray]:
        if e >= self.E or self.hi[e] is None or len(self.sig[e]) == 0:
            return None
        mk = np.zeros((self.d,), np.uint8)
        mk[self.sig[e]] = 1
        return mk

    def effective_weights(self, e: int):
        """Dense float64 (W_gate_eff [f,d], W_up_eff [f,d], W_down [d,f]) of expert e."""
        g, u, dn = (dequantize(qm.q, qm.s, qm.m, self.G) for qm in self.base[e])
        mk = self.mask(e)
        if mk is not None:
            cols = np.nonzero(mk)[0]
            g8, u8 = (dequantize(qm.q, qm.s, qm.m, self.G) for qm in self.hi[e])
            g[:, cols] = g8[:, cols]
            u[:, cols] = u8[:, cols]
        mkd = self.mask_down(e)
        if mkd is not None:
            cols = np.nonzero(mkd)[0]
            qm = self.hi_down[e]
            dn[:, cols] = dequantize(qm.q, qm.s, qm.m, self.G)[:, cols]
        return g, u, dn

    def expert_ffn(self, x_u16: np.ndarray, e: int, rows: np.ndarray) -> np.ndarray:
        """y_e for the tokens ``rows`` of x (float64 [len(rows), d])."""
        rows = np.ascontiguousarray(rows, dtype=np.int32)
        out = np.empty((len(rows), self.d), np.float64)
        bg, bu, bd = self.base[e]
        mk = self.mask(e)
        u8, u16 = ctypes.c_uint8, ctypes.c_uint16
        args = []
        for qm in (bg, bu, bd):
            args += [_p(qm.q, u8), _p(qm.s, u16), _p(qm.m, u16)]
        if mk is not None:
            for qm in self.hi[e]:
                args += [_p(qm.q, u8), _p(qm.s, u16), _p(qm.m, u16)]
        else:
            args += [_p(None, u8), _p(None, u16), _p(None, u16)] * 2
        mkd = self.mask_down(e)
        if mkd is not None:
            qm = self.hi_down[e]
            dargs = [_p(qm.q, u8), _p(qm.s, u16), _p(qm.m, u16), _p(mkd, u8)]
        else:
            dargs = [_p(None, u8), _p(None, u16), _p(None, u16), _p(None, u8)]
        lib().orc_expert_ffn(_p(np.ascontiguousarray(x_u16), u16), _p(rows, ctypes.c_int32), len(rows),
                             self.d, self.f, self.G, *args, _p(mk, u8), *dargs, _p(out, ctypes.c_double))
        return out

    def forward(self, x_u16: np.ndarray, logits: np.ndarray, tokens: Optional[np.ndarray] = None):
        """Whole layer.  Returns dict(idx, w, offsets, perm, y).  ``y`` is float64 [T, d];
        if ``tokens`` is given only those rows of y are computed (the others are NaN)."""
        T = x_u16.shape[0]
        idx, w = route(logits, self.k, self.renormalize)
        offsets, perm = permute(idx, self.E)
        sel = np.arange(T, dtype=np.int32) if tokens is None else np.asarray(tokens, dtype=np.int32)
        want = np.zeros((T,), bool)
        want[sel] = True
        # per-pair expert outputs, expert-major
        pair_out = {}
        for e in range(self.E):
            seg = perm[offsets[e]:offsets[e + 1]]
            seg = seg[want[seg // self.k]] if len(seg) else seg
            if len(seg) == 0:
                continue
            ye = self.expert_ffn(x_u16, e, (seg // self.k).astype(np.int32))
            for i, pr in enumerate(seg):
                pair_out[int(pr)] = ye[i]
        shared = []
        for e in range(self.E, self.n_total):
            shared.append(self.expert_ffn(x_u16, e, sel))
        y = np.full((T, self.d), np.nan, np.float64)
        for i, t in enumerate(sel):
            acc = np.zeros((self.d,), np.float64)
            for j in range(self.k):          # fixed order: slots 0..k-1, then the shared experts
                acc = acc + w[t, j] * pair_out[int(t) * self.k + j]
            for sh in shared:
                acc = acc + sh[i]
            y[t] = acc
        return {"idx": idx, "w": w, "offsets": offsets, "perm": perm, "y": y}


# ---- runtime selection of the significant channels (Sections IV-B, V-A; a "next" row of the scope table) ----
# The paper leaves the statistic loose; the reading taken is the activation mass of an input channel over the tokens
# routed to the expert.  Plain float64 sums: |x| of a bf16 value is exact, and so are sums of a few thousand of them.

def channel_stats_update(stats: np.ndarray, x_u16: np.ndarray, idx: np.ndarray, pool: np.ndarray) -> np.ndarray:
    """stats float64 [E, P] + per expert e, cached channel pool[e][j]: sum over the tokens routed to e of
    |x[t][pool[e][j]]|.  x_u16: bf16 bit patterns [T, d]; idx: int32 [T, k] chosen experts; returns the new stats."""
    E, P = pool.shape
    xa = np.abs((x_u16.astype(np.uint32) << 16).view(np.float32)).astype(np.float64)
    out = np.array(stats, dtype=np.float64, copy=True)
    for e in range(E):
        for t in range(xa.shape[0]):
            if (idx[t] == e).any():
                out[e] += xa[t, pool[e]]
    return out


def select_significant(stats: np.ndarray, pool: np.ndarray, n_select: int, switchable: Sequence[bool]):
    """Per expert: the n_select cached channels with the largest statistic, ties -> lower channel index, in rank
    order; experts that are not switchable (8-bit base) get the empty set."""
    sets = []
    for e in range(pool.shape[0]):
        if not switchable[e]:
            sets.append(np.zeros((0,), np.int32))
            continue
        order = sorted(range(pool.shape[1]), key=lambda j: (-float(stats[e, j]), int(pool[e, j])))
        sets.append(np.array([pool[e, j] for j in order[: min(n_select, pool.shape[1])]], dtype=np.int32))
    return sets


from . import assign  # noqa: E402,F401  (offline bit-width assignment, Algorithm 1)
