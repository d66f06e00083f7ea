"""Thin ctypes binding of ``libdynamo.so`` (argument marshalling only).

Module-level functions carry the C-ABI names (``dynamo_create``, ``dynamo_pack_experts``,
``dynamo_set_channel_switch``, ``dynamo_moe_forward`` ...) and take raw pointers / sizes;
``DynamoLayer`` wraps one context together with the torch tensors that own its device
memory.  Every step of the path runs in the library's CUDA kernels; torch is used for
device memory and streams only.  A missing library raises: there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdynamo.so")
_lib = None

OK = 0
BF16, F32 = 0, 1
MAT_GATE, MAT_UP, MAT_DOWN = 0, 1, 2
OPERAND_FP16, OPERAND_BF16 = 0, 1
CODES_BASE, CODES_HI_POOL, CODES_HI_ACTIVE = 0, 1, 2
SWITCH_SELECT, SWITCH_REQUANT = 0, 1

STATUS_NAMES = ["OK", "ERR_NULL", "ERR_SHAPE", "ERR_BITS", "ERR_ALIGN", "ERR_ARENA_TOO_SMALL", "ERR_INDEX_RANGE",
                "ERR_INDEX_DUP", "ERR_NOT_CACHED", "ERR_STATE", "ERR_TOKENS", "ERR_CUDA", "ERR_TIMEOUT", "ERR_ARG", "ERR_RANGE"]

EXPORTED = ["dynamo_create", "dynamo_destroy", "dynamo_arena_bytes", "dynamo_pack_experts",
            "dynamo_set_channel_switch", "dynamo_set_channel_switch_many", "dynamo_set_switch_mode",
            "dynamo_moe_forward", "dynamo_moe_forward_router", "dynamo_moe_forward_host", "dynamo_export_codes", "dynamo_expert_stream_bytes",
            "dynamo_poll_status", "dynamo_set_profile_events", "dynamo_set_tc_min_rows", "dynamo_set_operand_dtype", "dynamo_set_stats_collection", "dynamo_set_channel_precision", "dynamo_assign_bits",
            "dynamo_down_cache_bytes", "dynamo_pack_down_cache", "dynamo_set_channel_switch_down",
            "dynamo_set_channel_precision_down",
            "dynamo_get_channel_stats", "dynamo_select_significant", "dynamo_sync_sets", "dynamo_route_permute_static",
            "dynamo_debug_expire_wait", "dynamo_debug_check_guards",
            "dynamo_kernel_launches", "dynamo_status_str"]


class LayerDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("d_model", "d_ff", "n_experts", "n_shared", "top_k", "group_size", "max_sig", "cache_size",
                 "max_tokens", "renormalize")]


class DebugOut(ctypes.Structure):
    _fields_ = [("topk_idx", ctypes.c_void_p), ("topk_w", ctypes.c_void_p), ("expert_offsets", ctypes.c_void_p),
                ("perm", ctypes.c_void_p)]


class DynamoError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{where}: {name} ({status_str(status)})")


def load():
    """Open the library; raises if it has not been built (no CPU fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with paper_2503_21135_b200.build.build_library()")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
        i32p = ctypes.POINTER(ctypes.c_int32)
        L.dynamo_create.argtypes = [ctypes.POINTER(LayerDesc), ctypes.POINTER(vp)]
        L.dynamo_destroy.argtypes = [vp]
        L.dynamo_arena_bytes.argtypes = [ctypes.POINTER(LayerDesc), i32p, ctypes.POINTER(sz), ctypes.POINTER(sz)]
        L.dynamo_pack_experts.argtypes = [vp, vp, vp, vp, i32p, i32p, vp, sz, vp, sz, vp]
        L.dynamo_set_channel_switch.argtypes = [vp, i32p, i32p, vp]
        L.dynamo_set_channel_switch_many.argtypes = [ctypes.POINTER(vp), i32, i32p, i32p, vp]
        L.dynamo_set_switch_mode.argtypes = [vp, i32]
        L.dynamo_moe_forward.argtypes = [vp, vp, vp, i32, vp, i32, ctypes.POINTER(DebugOut), vp]
        L.dynamo_moe_forward_host.argtypes = [vp, vp, vp, i32, vp, i32, vp]
        L.dynamo_moe_forward_router.argtypes = [vp, vp, vp, vp, i32, vp, i32, vp, ctypes.POINTER(DebugOut), vp]
        L.dynamo_export_codes.argtypes = [vp, i32, i32, vp, vp, vp, i32, vp]
        L.dynamo_expert_stream_bytes.argtypes = [vp, i32, ctypes.POINTER(sz)]
        L.dynamo_poll_status.argtypes = [vp, vp]
        L.dynamo_set_profile_events.argtypes = [vp, vp, vp, vp]
        L.dynamo_set_tc_min_rows.argtypes = [vp, i32]
        L.dynamo_set_operand_dtype.argtypes = [vp, i32]
        L.dynamo_set_stats_collection.argtypes = [vp, i32]
        L.dynamo_set_channel_precision.argtypes = [vp, i32p, vp]
        L.dynamo_set_channel_precision_down.argtypes = [vp, i32p, vp]
        L.dynamo_down_cache_bytes.argtypes = [vp, i32p, i32, i32, ctypes.POINTER(ctypes.c_size_t)]
        L.dynamo_pack_down_cache.argtypes = [vp, vp, i32p, i32, i32, vp, ctypes.c_size_t, vp]
        L.dynamo_set_channel_switch_down.argtypes = [vp, i32p, i32p, vp]
        f64p = ctypes.POINTER(ctypes.c_double)
        L.dynamo_assign_bits.argtypes = [f64p, i32, i32, i32, ctypes.c_double, ctypes.c_double, i32, f64p, f64p, i32p,
                                         ctypes.c_double, i32p, i32p, f64p, f64p, i32p]
        L.dynamo_get_channel_stats.argtypes = [vp, vp, vp]
        L.dynamo_select_significant.argtypes = [vp, i32, i32, i32p, i32p, vp]
        L.dynamo_sync_sets.argtypes = [vp, i32p, i32p]
        L.dynamo_route_permute_static.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, vp, vp]
        L.dynamo_debug_expire_wait.argtypes = [vp, ctypes.c_int64, vp]
        L.dynamo_debug_check_guards.argtypes = [vp, ctypes.POINTER(ctypes.c_int64), vp]
        L.dynamo_kernel_launches.argtypes = [vp]
        L.dynamo_kernel_launches.restype = ctypes.c_int64
        L.dynamo_status_str.argtypes = [i32]
        L.dynamo_status_str.restype = ctypes.c_char_p
        for name in EXPORTED[:-2]:
            getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def status_str(status: int) -> str:
    return load().dynamo_status_str(int(status)).decode()


def _i32p(a: Optional[np.ndarray]):
    if a is None:
        return ctypes.cast(None, ctypes.POINTER(ctypes.c_int32))
    assert a.dtype == np.int32 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


# ---- C-ABI names (raw pointers and sizes) --------------------------------------------------

def dynamo_create(desc: LayerDesc) -> "tuple[int, Optional[int]]":
    h = ctypes.c_void_p()
    st = load().dynamo_create(ctypes.byref(desc) if desc is not None else None, ctypes.byref(h))
    return st, h.value


def dynamo_destroy(ctx) -> int:
    return load().dynamo_destroy(ctx)


def dynamo_arena_bytes(desc: LayerDesc, bits: Optional[np.ndarray]):
    wb, sb = ctypes.c_size_t(), ctypes.c_size_t()
    st = load().dynamo_arena_bytes(ctypes.byref(desc), _i32p(bits), ctypes.byref(wb), ctypes.byref(sb))
    return st, wb.value, sb.value


def dynamo_pack_experts(ctx, w_gate, w_up, w_down, bits, cache_idx, arena, arena_bytes, ws, ws_bytes, stream) -> int:
    return load().dynamo_pack_experts(ctx, w_gate, w_up, w_down, _i32p(bits), _i32p(cache_idx), arena, arena_bytes,
                                      ws, ws_bytes, stream)


def dynamo_set_channel_switch(ctx, sig_idx, sig_cnt, stream) -> int:
    return load().dynamo_set_channel_switch(ctx, _i32p(sig_idx), _i32p(sig_cnt), stream)


def dynamo_set_channel_switch_many(ctxs: Sequence[int], sig_idx, sig_cnt, stream) -> int:
    arr = (ctypes.c_void_p * len(ctxs))(*ctxs)
    return load().dynamo_set_channel_switch_many(arr, len(ctxs), _i32p(sig_idx), _i32p(sig_cnt), stream)


def dynamo_set_switch_mode(ctx, mode: int) -> int:
    return load().dynamo_set_switch_mode(ctx, mode)


def dynamo_moe_forward(ctx, x, logits, T, y, y_dtype, dbg: Optional[DebugOut], stream) -> int:
    return load().dynamo_moe_forward(ctx, x, logits, T, y, y_dtype, ctypes.byref(dbg) if dbg is not None else None,
                                     stream)


def dynamo_moe_forward_router(ctx, x, w_router, bias, T, y, y_dtype, logits_out, dbg: Optional[DebugOut], stream) -> int:
    return load().dynamo_moe_forward_router(ctx, x, w_router, bias, T, y, y_dtype, logits_out,
                                            ctypes.byref(dbg) if dbg is not None else None, stream)


def dynamo_moe_forward_host(ctx, x_host, logits_host, T, y_host, y_dtype, stream) -> int:
    return load().dynamo_moe_forward_host(ctx, x_host, logits_host, T, y_host, y_dtype, stream)


def dynamo_export_codes(ctx, expert, matrix, q, scale, zero, which, stream) -> int:
    return load().dynamo_export_codes(ctx, expert, matrix, q, scale, zero, which, stream)


def dynamo_expert_stream_bytes(ctx, expert: int):
    b = ctypes.c_size_t()
    st = load().dynamo_expert_stream_bytes(ctx, expert, ctypes.byref(b))
    return st, b.value


def dynamo_poll_status(ctx, stream) -> int:
    return load().dynamo_poll_status(ctx, stream)


def dynamo_set_tc_min_rows(ctx, rows: int) -> int:
    return load().dynamo_set_tc_min_rows(ctx, rows)


def dynamo_set_operand_dtype(ctx, operand_dtype: int) -> int:
    return load().dynamo_set_operand_dtype(ctx, operand_dtype)


def dynamo_set_profile_events(ctx, e0, e1, e2) -> int:
    return load().dynamo_set_profile_events(ctx, e0, e1, e2)


def dynamo_route_permute_static(logits, T, n_experts, top_k, renormalize, topk_idx, topk_w, offsets, perm,
                                stream) -> int:
    """Routing + permutation without any device allocation (scratch lives inside the library)."""
    return load().dynamo_route_permute_static(logits, T, n_experts, top_k, renormalize, topk_idx, topk_w, offsets,
                                              perm, stream)


def dynamo_kernel_launches(ctx) -> int:
    return int(load().dynamo_kernel_launches(ctx))


# ---- convenience wrapper owning the torch buffers ------------------------------------------

def _check(st: int, where: str) -> None:
    if st != OK:
        raise DynamoError(st, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


class DynamoLayer:
    """One MoE layer context plus the torch tensors that own its arenas."""

    def __init__(self, d_model, d_ff, n_experts, top_k, group_size, max_sig, cache_size, max_tokens,
                 n_shared=0, renormalize=True, workspace: Optional[torch.Tensor] = None, device="cuda:0"):
        self.desc = LayerDesc(d_model, d_ff, n_experts, n_shared, top_k, group_size, max_sig, cache_size, max_tokens,
                              1 if renormalize else 0)
        st, self.ctx = dynamo_create(self.desc)
        _check(st, "dynamo_create")
        self.device = torch.device(device)
        self.arena: Optional[torch.Tensor] = None
        self.workspace = workspace

    @classmethod
    def from_config(cls, cfg, max_tokens=None, **kw):
        return cls(cfg.d_model, cfg.d_ff, cfg.n_experts, cfg.top_k, cfg.group_size, cfg.max_sig, cfg.cache_size,
                   max_tokens or max(cfg.tokens), n_shared=cfg.n_shared, **kw)

    def close(self):
        if self.ctx:
            dynamo_destroy(self.ctx)
            self.ctx = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    def arena_bytes(self, bits: np.ndarray):
        st, wb, sb = dynamo_arena_bytes(self.desc, np.ascontiguousarray(bits, dtype=np.int32))
        _check(st, "dynamo_arena_bytes")
        return wb, sb

    def pack_experts(self, w_gate: torch.Tensor, w_up: torch.Tensor, w_down: torch.Tensor, bits, cache_idx):
        bits = np.ascontiguousarray(bits, dtype=np.int32)
        cache_idx = np.ascontiguousarray(cache_idx, dtype=np.int32)
        wb, sb = self.arena_bytes(bits)
        self.arena = torch.empty(wb, dtype=torch.uint8, device=self.device)
        if self.workspace is None or self.workspace.numel() < sb:
            self.workspace = torch.empty(sb, dtype=torch.uint8, device=self.device)
        for w in (w_gate, w_up, w_down):
            assert w.is_cuda and w.dtype == torch.bfloat16 and w.is_contiguous()
        st = dynamo_pack_experts(self.ctx, w_gate.data_ptr(), w_up.data_ptr(), w_down.data_ptr(), bits, cache_idx,
                                 self.arena.data_ptr(), self.arena.numel(), self.workspace.data_ptr(),
                                 self.workspace.numel(), _stream())
        _check(st, "dynamo_pack_experts")

    def sig_arrays(self, sets: Sequence[np.ndarray]):
        E, S = self.desc.n_experts, self.desc.max_sig
        idx = np.full((E, max(S, 1)), -1, dtype=np.int32)
        cnt = np.zeros((E,), dtype=np.int32)
        for e, s in enumerate(sets):
            s = np.asarray(s, dtype=np.int32)
            cnt[e] = len(s)
            idx[e, : min(len(s), S)] = s[:S]
        return idx[:, :S] if S > 0 else idx[:, :0], cnt

    def set_channel_switch(self, sets: Sequence[np.ndarray]):
        idx, cnt = self.sig_arrays(sets)
        st = dynamo_set_channel_switch(self.ctx, np.ascontiguousarray(idx), cnt, _stream())
        _check(st, "dynamo_set_channel_switch")

    def pack_down_cache(self, w_down: torch.Tensor, bits, cache_idx_down, max_sig_down: int):
        """Channel cache on the d_ff side: cache_idx_down int [E, P2] (sorted hidden-unit indices per expert)."""
        bits = np.ascontiguousarray(bits, dtype=np.int32)
        ci = np.ascontiguousarray(cache_idx_down, dtype=np.int32)
        assert ci.ndim == 2 and ci.shape[0] == self.desc.n_experts
        assert w_down.is_cuda and w_down.dtype == torch.bfloat16 and w_down.is_contiguous()
        P2 = int(ci.shape[1])
        nbytes = ctypes.c_size_t(0)
        _check(load().dynamo_down_cache_bytes(ctypes.byref(self.desc), _i32p(bits), P2, int(max_sig_down),
                                              ctypes.byref(nbytes)), "dynamo_down_cache_bytes")
        arena = torch.empty(nbytes.value, dtype=torch.uint8, device=self.device)
        st = load().dynamo_pack_down_cache(self.ctx, w_down.data_ptr(), _i32p(ci), P2, int(max_sig_down),
                                           arena.data_ptr(), arena.numel(), _stream())
        _check(st, "dynamo_pack_down_cache")
        self.down_arena = arena                  # on an error the previous arena stays referenced (and in use)
        self.max_sig_down = int(max_sig_down)

    def set_channel_switch_down(self, sets: Sequence[np.ndarray]):
        E, S2 = self.desc.n_experts, self.max_sig_down
        idx = np.full((E, max(S2, 1)), -1, dtype=np.int32)
        cnt = np.zeros((E,), dtype=np.int32)
        for e, s_ in enumerate(sets):
            s_ = np.asarray(s_, dtype=np.int32)
            cnt[e] = len(s_)
            idx[e, : min(len(s_), S2)] = s_[:S2]
        idx = np.ascontiguousarray(idx[:, :S2] if S2 > 0 else idx[:, :1])
        st = load().dynamo_set_channel_switch_down(self.ctx, _i32p(idx), _i32p(cnt), _stream())
        _check(st, "dynamo_set_channel_switch_down")

    def set_switch_mode(self, mode: int):
        _check(dynamo_set_switch_mode(self.ctx, mode), "dynamo_set_switch_mode")

    def forward(self, x: torch.Tensor, logits: torch.Tensor, y_dtype=F32, debug=False, y: Optional[torch.Tensor] = None):
        T = x.shape[0]
        assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous()
        assert logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous()
        if y is None:
            y = torch.empty((T, self.desc.d_model), dtype=torch.float32 if y_dtype == F32 else torch.bfloat16,
                            device=x.device)
        dbg, outs = None, None
        if debug:
            k, E = self.desc.top_k, self.desc.n_experts
            outs = {"idx": torch.empty((T, k), dtype=torch.int32, device=x.device),
                    "w": torch.empty((T, k), dtype=torch.float32, device=x.device),
                    "offsets": torch.empty((E + 1,), dtype=torch.int32, device=x.device),
                    "perm": torch.empty((T * k,), dtype=torch.int32, device=x.device)}
            dbg = DebugOut(outs["idx"].data_ptr(), outs["w"].data_ptr(), outs["offsets"].data_ptr(),
                           outs["perm"].data_ptr())
        st = dynamo_moe_forward(self.ctx, x.data_ptr(), logits.data_ptr(), T, y.data_ptr(), y_dtype, dbg, _stream())
        _check(st, "dynamo_moe_forward")
        return (y, outs) if debug else y

    def forward_router(self, x: torch.Tensor, w_router: torch.Tensor, bias: Optional[torch.Tensor] = None, y_dtype=F32,
                       want_logits=False, debug=False):
        """Forward with the router GEMM + top-k fused in front; returns y (, logits) (, debug outputs)."""
        T = x.shape[0]
        E, k = self.desc.n_experts, self.desc.top_k
        assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous()
        assert w_router.is_cuda and w_router.dtype == torch.bfloat16 and w_router.is_contiguous()
        assert tuple(w_router.shape) == (E, self.desc.d_model)
        assert bias is None or (bias.is_cuda and bias.dtype == torch.float32 and bias.numel() == E)
        y = torch.empty((T, self.desc.d_model), dtype=torch.float32 if y_dtype == F32 else torch.bfloat16, device=x.device)
        lg = torch.empty((T, E), dtype=torch.float32, device=x.device) if want_logits else None
        dbg, outs = None, None
        if debug:
            outs = {"idx": torch.empty((T, k), dtype=torch.int32, device=x.device),
                    "w": torch.empty((T, k), dtype=torch.float32, device=x.device),
                    "offsets": torch.empty((E + 1,), dtype=torch.int32, device=x.device),
                    "perm": torch.empty((T * k,), dtype=torch.int32, device=x.device)}
            dbg = DebugOut(outs["idx"].data_ptr(), outs["w"].data_ptr(), outs["offsets"].data_ptr(),
                           outs["perm"].data_ptr())
        st = dynamo_moe_forward_router(self.ctx, x.data_ptr(), w_router.data_ptr(),
                                       bias.data_ptr() if bias is not None else None, T, y.data_ptr(), y_dtype,
                                       lg.data_ptr() if lg is not None else None, dbg, _stream())
        _check(st, "dynamo_moe_forward_router")
        res = (y,) + ((lg,) if want_logits else ()) + ((outs,) if debug else ())
        return res if len(res) > 1 else y

    def forward_host(self, x_host: torch.Tensor, logits_host: torch.Tensor, y_host: torch.Tensor, y_dtype=F32):
        T = x_host.shape[0]
        st = dynamo_moe_forward_host(self.ctx, x_host.data_ptr(), logits_host.data_ptr(), T, y_host.data_ptr(),
                                     y_dtype, _stream())
        _check(st, "dynamo_moe_forward_host")
        return y_host

    def export_codes(self, expert: int, matrix: int, which: int = CODES_BASE):
        d, f, G = self.desc.d_model, self.desc.d_ff, self.desc.group_size
        N, K = (d, f) if matrix == MAT_DOWN else (f, d)
        q = torch.empty((N, K), dtype=torch.uint8, device=self.device)
        s = torch.empty((N, K // G), dtype=torch.int16, device=self.device)
        m = torch.empty((N, K // G), dtype=torch.int16, device=self.device)
        st = dynamo_export_codes(self.ctx, expert, matrix, q.data_ptr(), s.data_ptr(), m.data_ptr(), which, _stream())
        _check(st, "dynamo_export_codes")
        return q, s, m

    def stream_bytes(self, expert: int) -> int:
        st, b = dynamo_expert_stream_bytes(self.ctx, expert)
        _check(st, "dynamo_expert_stream_bytes")
        return b

    def set_tc_min_rows(self, rows: int):
        _check(dynamo_set_tc_min_rows(self.ctx, rows), "dynamo_set_tc_min_rows")

    def set_operand_dtype(self, operand_dtype: int):
        """OPERAND_FP16 (default) or OPERAND_BF16: precision the hidden activations carry into the second projection."""
        _check(dynamo_set_operand_dtype(self.ctx, operand_dtype), "dynamo_set_operand_dtype")

    def set_channel_precision(self, hi_bits):
        """Precision the significant channels of each routed expert are served at: int [E], each in {2,3,4,6,8}."""
        hb = np.ascontiguousarray(np.asarray(hi_bits, dtype=np.int32))
        assert hb.shape == (self.desc.n_experts,)
        _check(load().dynamo_set_channel_precision(self.ctx, _i32p(hb), _stream()), "dynamo_set_channel_precision")

    def set_channel_precision_down(self, hi_bits):
        """Precision the significant hidden units (d_ff side) of each routed expert are served at: int [E]."""
        hb = np.ascontiguousarray(np.asarray(hi_bits, dtype=np.int32))
        assert hb.shape == (self.desc.n_experts,)
        _check(load().dynamo_set_channel_precision_down(self.ctx, _i32p(hb), _stream()),
               "dynamo_set_channel_precision_down")

    def set_stats_collection(self, on: bool):
        _check(load().dynamo_set_stats_collection(self.ctx, int(bool(on))), "dynamo_set_stats_collection")

    def channel_stats(self) -> torch.Tensor:
        """Accumulated activation mass fp32 [E, P] (column j = cached channel cache_idx[e][j])."""
        out = torch.empty((self.desc.n_experts, self.desc.cache_size), dtype=torch.float32, device=self.device)
        _check(load().dynamo_get_channel_stats(self.ctx, out.data_ptr(), _stream()), "dynamo_get_channel_stats")
        return out

    def select_significant(self, n_select: int, reset: bool = True, wait: bool = True):
        """Install, per expert, the n_select cached channels with the largest statistics.  wait=True returns the sets;
        wait=False only enqueues the selection (fetch the sets later with sync_sets)."""
        if not wait:
            _check(load().dynamo_select_significant(self.ctx, n_select, int(bool(reset)), None, None, _stream()),
                   "dynamo_select_significant")
            return None
        E, S = self.desc.n_experts, self.desc.max_sig
        idx = np.full((E, max(S, 1)), -1, dtype=np.int32)
        cnt = np.zeros((E,), dtype=np.int32)
        _check(load().dynamo_select_significant(self.ctx, n_select, int(bool(reset)), _i32p(idx), _i32p(cnt), _stream()),
               "dynamo_select_significant")
        return [idx[e, : cnt[e]].copy() for e in range(E)]

    def sync_sets(self):
        """The significant sets now installed (waits for a selection still on its way)."""
        E, S = self.desc.n_experts, self.desc.max_sig
        idx = np.full((E, max(S, 1)), -1, dtype=np.int32)
        cnt = np.zeros((E,), dtype=np.int32)
        _check(load().dynamo_sync_sets(self.ctx, _i32p(idx), _i32p(cnt)), "dynamo_sync_sets")
        return [idx[e, : cnt[e]].copy() for e in range(E)]

    def set_profile_events(self, events=None):
        """events: three torch.cuda.Event (already recorded once, so that their handles exist) or None."""
        h = [None, None, None] if events is None else [e.cuda_event for e in events]
        _check(dynamo_set_profile_events(self.ctx, *h), "dynamo_set_profile_events")

    def poll_status(self) -> int:
        return dynamo_poll_status(self.ctx, _stream())

    def debug_expire_wait(self, limit_ns: int):
        _check(load().dynamo_debug_expire_wait(self.ctx, int(limit_ns), _stream()), "dynamo_debug_expire_wait")

    def debug_check_guards(self) -> int:
        n = ctypes.c_int64(-1)
        _check(load().dynamo_debug_check_guards(self.ctx, ctypes.byref(n), _stream()), "dynamo_debug_check_guards")
        return int(n.value)

    def kernel_launches(self) -> int:
        return dynamo_kernel_launches(self.ctx)


def set_channel_switch_many(layers: List[DynamoLayer], sets_per_layer: Sequence[Sequence[np.ndarray]]):
    """One switch event for a stack of layers: one upload, one launch."""
    idxs, cnts = zip(*(l.sig_arrays(s) for l, s in zip(layers, sets_per_layer)))
    idx = np.ascontiguousarray(np.stack(idxs), dtype=np.int32)
    cnt = np.ascontiguousarray(np.stack(cnts), dtype=np.int32)
    st = dynamo_set_channel_switch_many([l.ctx for l in layers], idx, cnt, _stream())
    _check(st, "dynamo_set_channel_switch_many")


def assign_bits(x, levels, c: int = 4, m: float = 2.0, eps: float = 1e-9, max_iter: int = 1000, u0=None,
                token_share=None, overlap: float = 0.0):
    """Offline bit-width assignment (Algorithm 1 + cluster-to-precision map).  Host arrays in, host arrays out:
    returns dict(bits [n], cluster [n], V [c, dim], U [n, c], iters)."""
    x = np.ascontiguousarray(np.asarray(x, dtype=np.float64))
    if x.ndim == 1:
        x = x[:, None]
    n, dim = x.shape
    f64p = ctypes.POINTER(ctypes.c_double)
    as_f64 = lambda a: None if a is None else np.ascontiguousarray(np.asarray(a, dtype=np.float64))
    u0a, sha = as_f64(u0), as_f64(token_share)
    if u0a is not None:
        assert u0a.shape == (n, c)
    if sha is not None:
        assert sha.shape == (n,)
    lv = np.ascontiguousarray(np.asarray(levels, dtype=np.int32))
    assert lv.shape == (c,)
    bits, cluster = np.zeros(n, np.int32), np.zeros(n, np.int32)
    V, U, iters = np.zeros((c, dim)), np.zeros((n, c)), np.zeros(1, np.int32)
    ptr = lambda a: None if a is None else a.ctypes.data_as(f64p)
    st = load().dynamo_assign_bits(ptr(x), n, dim, c, m, eps, max_iter, ptr(u0a), ptr(sha), _i32p(lv), overlap,
                                   _i32p(bits), _i32p(cluster), ptr(V), ptr(U), _i32p(iters))
    _check(st, "dynamo_assign_bits")
    return dict(bits=bits, cluster=cluster, V=V, U=U, iters=int(iters[0]))
