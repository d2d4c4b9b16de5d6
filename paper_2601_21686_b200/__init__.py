"""Python binding of libstief.so: decode attention over a rank-compressed KV cache on B200.

Argument marshalling only.  Every function has the name and the meaning of the C entry point
declared in ``include/stief.h``; tensors are torch CUDA tensors used as device memory, and the work is
enqueued on torch's current stream.  There is no fallback: if the CUDA library has not been built the
first call raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libstief.so")

STIEF_OK, STIEF_ERR_INVALID_ARG, STIEF_ERR_UNSUPPORTED, STIEF_ERR_WORKSPACE = 0, 1, 2, 3
STIEF_ERR_CUDA, STIEF_ERR_BOUNDS, STIEF_ERR_TIMEOUT, STIEF_ERR_INFEASIBLE = 4, 5, 6, 7
PAGE = 64
D_HEAD = 128
STIEF_DECODE_OVERLAP_PREVIOUS = 1
STIEF_PREFILL_OVERLAP_PREVIOUS = 1


class StiefError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


class _CLayer(ctypes.Structure):
    _fields_ = [("Hq", ctypes.c_int32), ("Hkv", ctypes.c_int32), ("d", ctypes.c_int32),
                ("r_k", ctypes.c_int32), ("r_v", ctypes.c_int32), ("num_pages", ctypes.c_int32),
                ("U_k", ctypes.c_void_p), ("uk_head_stride", ctypes.c_int64),
                ("U_v", ctypes.c_void_p), ("uv_head_stride", ctypes.c_int64),
                ("k_pool", ctypes.c_void_p), ("v_pool", ctypes.c_void_p)]


class _CQLayer(ctypes.Structure):
    _fields_ = [("Hq", ctypes.c_int32), ("Hkv", ctypes.c_int32), ("d", ctypes.c_int32),
                ("r_k", ctypes.c_int32), ("r_v", ctypes.c_int32), ("num_pages", ctypes.c_int32),
                ("U_k", ctypes.c_void_p), ("uk_head_stride", ctypes.c_int64),
                ("U_v", ctypes.c_void_p), ("uv_head_stride", ctypes.c_int64),
                ("k_params", ctypes.c_void_p), ("k_codes", ctypes.c_void_p), ("v_codes", ctypes.c_void_p),
                ("v_params", ctypes.c_void_p)]


class _CBatch(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("max_pages_per_seq", ctypes.c_int32),
                ("block_table", ctypes.c_void_p), ("seq_lens", ctypes.c_void_p)]


_SURFACE_FN = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(ctypes.c_int32),
                               ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_double))

_lib_handle = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library (loads it on first use; raises if it was never built)."""
    global _lib_handle
    if _lib_handle is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2601_21686_b200.build` "
                               "(there is no non-CUDA path)")
        L = ctypes.CDLL(LIB_PATH)
        P, I32, I64, SZ, U32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t, ctypes.c_uint32
        LP, BP, QP = ctypes.POINTER(_CLayer), ctypes.POINTER(_CBatch), ctypes.POINTER(_CQLayer)
        sig = {
            "stief_prefill_compress": (ctypes.c_int, [LP, BP, P, P, I64, I64, I64, I64, I32, U32, P, P]),
            "stief_append": (ctypes.c_int, [LP, BP, P, P, P, P]),
            "stief_append_chunk": (ctypes.c_int, [LP, BP, P, P, I64, I64, I64, I64, I32, P, I32, P, P]),
            "stief_decode_num_parts": (I32, []),
            "stief_decode_workspace_bytes": (SZ, [I32, I32, I32, I32, I32]),
            "stief_decode_workspace_init": (ctypes.c_int, [P, SZ, P]),
            "stief_decode_attention": (ctypes.c_int, [LP, BP, P, I32, P, SZ, I32, P, P, U32, P, P]),
            "stief_split_combine": (ctypes.c_int, [LP, BP, I32, P, I32, P, P, P, P]),
            "stief_decode_attention_static": (ctypes.c_int, [LP, BP, P, I32, I32, P, P, P, P]),
            "stief_decode_step": (ctypes.c_int, [LP, BP, P, P, P, P, SZ, I32, P, P, U32, P, P]),
            "stief_host_staging_bytes": (SZ, [I32, I32, I32]),
            "stief_decode_step_host": (ctypes.c_int, [LP, BP, P, P, P, P, P, SZ, I32, P, U32, P, P]),
            "stief_advance_seq_lens": (ctypes.c_int, [P, I32, I32, P]),
            "stief_time_next_decode_kernel": (ctypes.c_int, [P, P]),
            "stief_q8_prefill_compress": (ctypes.c_int, [QP, BP, P, P, I64, I64, I32, U32, P, P]),
            "stief_q8_append": (ctypes.c_int, [QP, BP, P, P, P, P]),
            "stief_q8_decode_attention": (ctypes.c_int, [QP, BP, P, I32, P, SZ, I32, P, P, U32, P, P]),
            "stief_q8_decode_step": (ctypes.c_int, [QP, BP, P, P, P, P, SZ, I32, P, P, U32, P, P]),
            "stief_q4_prefill_compress": (ctypes.c_int, [QP, BP, P, P, I64, I64, I32, U32, P, P]),
            "stief_q4_append": (ctypes.c_int, [QP, BP, P, P, P, P]),
            "stief_q4_decode_attention": (ctypes.c_int, [QP, BP, P, I32, P, SZ, I32, P, P, U32, P, P]),
            "stief_q4_decode_step": (ctypes.c_int, [QP, BP, P, P, P, P, SZ, I32, P, P, U32, P, P]),
            "stief_mq_attention": (ctypes.c_int, [LP, BP, P, I64, I64, I32, P, P, SZ, I32, P, I64, I64, P, U32, P, P]),
            "stief_mq_num_splits": (I32, [I32, I32, I32, I32, I32]),
            "stief_mq_workspace_bytes": (SZ, [I32, I32, I32, I32, I32]),
            "stief_select_ranks": (ctypes.c_int, [I32, I32, P, I32, P, I32, ctypes.c_double, P, _SURFACE_FN, P, P, P, P, P]),
            "stief_selftest_wait_limit": (ctypes.c_int, [P, P, I32, P]),
            "stief_trace_next_decode_kernel": (ctypes.c_int, [P, SZ]),
            "stief_measure_read_stream": (ctypes.c_int, [P, SZ, P, P]),
            "stief_status_string": (ctypes.c_char_p, [ctypes.c_int]),
            "stief_version": (ctypes.c_int, []),
        }
        for name, (res, args) in sig.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib_handle = L
    return _lib_handle


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


@dataclass
class Layer:
    """One decoder layer's compressed cache and bases (device tensors).  U_k [Hkv or 1, 128, r_k],
    U_v [Hkv or 1, 128, r_v] bf16 (None = that side kept full rank); pools [num_pages, Hkv, 64, r] bf16."""
    Hq: int
    Hkv: int
    r_k: int
    r_v: int
    U_k: Optional[torch.Tensor]
    U_v: Optional[torch.Tensor]
    k_pool: torch.Tensor
    v_pool: torch.Tensor

    @property
    def num_pages(self) -> int:
        return self.k_pool.shape[0]

    def c(self) -> _CLayer:
        # the descriptor is rebuilt only when a tensor was replaced (marshalling is on the path of every step)
        key = (_ptr(self.U_k), _ptr(self.U_v), _ptr(self.k_pool), _ptr(self.v_pool), self.Hq, self.Hkv, self.r_k, self.r_v)
        cached = self.__dict__.get("_c")
        if cached is not None and cached[0] == key:
            return cached[1]
        uk_stride = 0 if self.U_k is None or self.U_k.shape[0] == 1 else self.U_k.stride(0)
        uv_stride = 0 if self.U_v is None or self.U_v.shape[0] == 1 else self.U_v.stride(0)
        st = _CLayer(self.Hq, self.Hkv, D_HEAD, self.r_k, self.r_v, self.num_pages, _ptr(self.U_k), uk_stride,
                     _ptr(self.U_v), uv_stride, _ptr(self.k_pool), _ptr(self.v_pool))
        self.__dict__["_c"] = (key, st)
        return st


@dataclass
class QLayer:
    """One decoder layer's quantised compressed cache (device tensors): U_k [Hkv or 1, 128, r_k], U_v [Hkv or 1, 128, r_v]
    bf16; k_params [Hkv, groups(r_k), 2] fp32 (scale, zero; static); v_params [num_pages, Hkv, 64, groups(r_v), 2] fp32
    (scale, zero per token and group), groups(r) = ceil(r / 64).  Code pools as uint8 tensors: 8-bit k_codes
    [num_pages, Hkv, 64, r_k], v_codes [num_pages, Hkv, r_v, 64]; 4-bit k_codes [num_pages, Hkv, 64, krow] (krow = r_k / 2,
    32 for r_k = 48), v_codes [num_pages, Hkv, r_v, 32] (channel-major pages, permuted token positions, nibble order: see
    stief.h).  The same object serves the stief_q8_* and the stief_q4_* calls; the pools must have the matching form."""
    Hq: int
    Hkv: int
    r_k: int
    r_v: int
    U_k: torch.Tensor
    U_v: torch.Tensor
    k_params: torch.Tensor
    k_codes: torch.Tensor
    v_codes: torch.Tensor
    v_params: torch.Tensor

    @property
    def num_pages(self) -> int:
        return self.k_codes.shape[0]

    def c(self) -> _CQLayer:
        uk_stride = 0 if self.U_k.shape[0] == 1 else self.U_k.stride(0)
        uv_stride = 0 if self.U_v.shape[0] == 1 else self.U_v.stride(0)
        return _CQLayer(self.Hq, self.Hkv, D_HEAD, self.r_k, self.r_v, self.num_pages, _ptr(self.U_k), uk_stride,
                        _ptr(self.U_v), uv_stride, _ptr(self.k_params), _ptr(self.k_codes), _ptr(self.v_codes),
                        _ptr(self.v_params))


@dataclass
class Batch:
    """Paging state: block_table [B, max_pages_per_seq] int32, seq_lens [B] int32 (device tensors)."""
    block_table: torch.Tensor
    seq_lens: torch.Tensor

    def c(self) -> _CBatch:
        key = (_ptr(self.block_table), _ptr(self.seq_lens), self.block_table.shape[0], self.block_table.shape[1])
        cached = self.__dict__.get("_c")
        if cached is not None and cached[0] == key:
            return cached[1]
        st = _CBatch(self.block_table.shape[0], self.block_table.shape[1], _ptr(self.block_table), _ptr(self.seq_lens))
        self.__dict__["_c"] = (key, st)
        return st


def _check(rc: int, where: str):
    if rc != STIEF_OK:
        raise StiefError(rc, where)


def status_string(code: int) -> str:
    return lib().stief_status_string(code).decode()


def stief_version() -> int:
    return lib().stief_version()


def stief_prefill_compress(layer: Layer, batch: Batch, K: torch.Tensor, V: torch.Tensor, T_max: Optional[int] = None,
                           status: Optional[torch.Tensor] = None, flags: int = 0):
    """K, V [B, T, Hkv, 128] bf16 (strides over b and t free, heads and d contiguous) -> paged compressed cache.
    A side without basis takes rows of r elements: [B, T, Hkv, r]."""
    assert K.stride(3) == 1 and K.stride(2) == K.shape[3] and V.stride(3) == 1 and V.stride(2) == V.shape[3]
    assert K.shape[3] == (D_HEAD if layer.U_k is not None else layer.r_k) and V.shape[3] == (D_HEAD if layer.U_v is not None else layer.r_v)
    cl, cb = layer.c(), batch.c()
    _check(lib().stief_prefill_compress(ctypes.byref(cl), ctypes.byref(cb), _ptr(K), _ptr(V), K.stride(0), K.stride(1),
                                        V.stride(0), V.stride(1), K.shape[1] if T_max is None else T_max, flags, _ptr(status),
                                        _stream()),
           "stief_prefill_compress")


def qkey_row_bytes(r_k: int, bits: int) -> int:
    """Bytes of one key row of the quantised cache (4-bit rank-48 rows are padded to 32 bytes)."""
    return r_k if bits == 8 else (32 if r_k == 48 else r_k // 2)


def qgroups(r: int) -> int:
    return (r + 63) // 64


def stief_q8_prefill_compress(layer: QLayer, batch: Batch, K: torch.Tensor, V: torch.Tensor, T_max: Optional[int] = None,
                              status: Optional[torch.Tensor] = None, flags: int = 0):
    """K, V [B, T, Hkv, 128] bf16 -> 8-bit quantised paged compressed cache."""
    assert K.stride(3) == 1 and K.stride(2) == D_HEAD and V.stride() == K.stride()
    cl, cb = layer.c(), batch.c()
    _check(lib().stief_q8_prefill_compress(ctypes.byref(cl), ctypes.byref(cb), _ptr(K), _ptr(V), K.stride(0), K.stride(1),
                                           K.shape[1] if T_max is None else T_max, flags, _ptr(status), _stream()),
           "stief_q8_prefill_compress")


def stief_q8_append(layer: QLayer, batch: Batch, k_new: torch.Tensor, v_new: torch.Tensor, status: Optional[torch.Tensor] = None):
    cl, cb = layer.c(), batch.c()
    _check(lib().stief_q8_append(ctypes.byref(cl), ctypes.byref(cb), _ptr(k_new), _ptr(v_new), _ptr(status), _stream()),
           "stief_q8_append")


def stief_q8_decode_attention(layer: QLayer, batch: Batch, q: torch.Tensor, workspace: torch.Tensor, out: torch.Tensor,
                              num_parts: int = 0, out_lse: Optional[torch.Tensor] = None, len_add: int = 0,
                              status: Optional[torch.Tensor] = None, flags: int = 0):
    cl, cb = layer.c(), batch.c()
    _check(lib().stief_q8_decode_attention(ctypes.byref(cl), ctypes.byref(cb), _ptr(q), len_add, _ptr(workspace),
                                           workspace.numel() * workspace.element_size(), num_parts, _ptr(out), _ptr(out_lse),
                                           flags, _ptr(status), _stream()), "stief_q8_decode_attention")


def stief_q8_decode_step(layer: QLayer, batch: Batch, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor,
                         workspace: torch.Tensor, out: torch.Tensor, num_parts: int = 0, out_lse: Optional[torch.Tensor] = None,
                         status: Optional[torch.Tensor] = None, flags: int = 0):
    cl, cb = layer.c(), batch.c()
    _check(lib().stief_q8_decode_step(ctypes.byref(cl), ctypes.byref(cb), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(workspace),
                                      workspace.numel() * workspace.element_size(), num_parts, _ptr(out), _ptr(out_lse),
                                      flags, _ptr(status), _stream()), "stief_q8_decode_step")


def stief_append(layer: Layer, batch: Batch, k_new: torch.Tensor, v_new: torch.Tensor, status: Optional[torch.Tensor] = None):
    cl, cb = layer.c(), batch.c()
    _check(lib().stief_append(ctypes.byref(cl), ctypes.byref(cb), _ptr(k_new), _ptr(v_new), _ptr(status), _stream()),
           "stief_append")


def stief_decode_num_parts() -> int:
    return lib().stief_decode_num_parts()


def stief_decode_workspace_bytes(B: int, Hq: int, Hkv: int, r_v: int, num_parts: int = 0) -> int:
    return lib().stief_decode_workspace_bytes(B, Hq, Hkv, r_v, num_parts)


def stief_decode_workspace_init(workspace: torch.Tensor):
    _check(lib().stief_decode_workspace_init(_ptr(workspace), workspace.numel() * workspace.element_size(), _stream()),
           "stief_decode_workspace_init")


def stief_decode_attention(layer: Layer, batch: Batch, q: torch.Tensor, workspace: torch.Tensor, num_parts: int = 0,
                           out: Optional[torch.Tensor] = None, out_lse: Optional[torch.Tensor] = None, len_add: int = 0,
                           status: Optional[torch.Tensor] = None, flags: int = 0):
    cl, cb = layer.c(), batch.c()
    _check(lib().stief_decode_attention(ctypes.byref(cl), ctypes.byref(cb), _ptr(q), len_add, _ptr(workspace),
                                        workspace.numel() * workspace.element_size(), num_parts, _ptr(out), _ptr(out_lse),
                                        flags, _ptr(status), _stream()), "stief_decode_attention")


STATIC_WORKSPACE_BYTES = 8 << 20


def stief_decode_attention_static(layer: Layer, batch: Batch, q: torch.Tensor, out: torch.Tensor, num_parts: int = 0,
                                  out_lse: Optional[torch.Tensor] = None, len_add: int = 0,
                                  status: Optional[torch.Tensor] = None):
    """stief_decode_attention without a workspace argument, for callers that have no means of allocating one
    (a plug-in inside an engine that owns all device memory; a path where cudaMalloc's device-wide
    synchronisation is not acceptable).  The scratch is a fixed STATIC_WORKSPACE_BYTES array inside the
    library, shared by every call on the device: calls must not overlap on the GPU, and shapes whose
    workspace would be larger raise StiefError(STIEF_ERR_WORKSPACE).  Make the first call on a device
    outside any stream capture."""
    cl, cb = layer.c(), batch.c()
    _check(lib().stief_decode_attention_static(ctypes.byref(cl), ctypes.byref(cb), _ptr(q), len_add, num_parts, _ptr(out),
                                               _ptr(out_lse), _ptr(status), _stream()), "stief_decode_attention_static")


def stief_split_combine(layer: Layer, batch: Batch, workspace: torch.Tensor, num_parts: int, out: torch.Tensor,
                        out_lse: Optional[torch.Tensor] = None, len_add: int = 0, status: Optional[torch.Tensor] = None):
    cl, cb = layer.c(), batch.c()
    _check(lib().stief_split_combine(ctypes.byref(cl), ctypes.byref(cb), len_add, _ptr(workspace), num_parts, _ptr(out),
                                     _ptr(out_lse), _ptr(status), _stream()), "stief_split_combine")


def stief_decode_step(layer: Layer, batch: Batch, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor,
                      workspace: torch.Tensor, out: torch.Tensor, num_parts: int = 0, out_lse: Optional[torch.Tensor] = None,
                      status: Optional[torch.Tensor] = None, flags: int = 0):
    cl, cb = layer.c(), batch.c()
    _check(lib().stief_decode_step(ctypes.byref(cl), ctypes.byref(cb), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(workspace),
                                   workspace.numel() * workspace.element_size(), num_parts, _ptr(out), _ptr(out_lse),
                                   flags, _ptr(status), _stream()), "stief_decode_step")


def stief_host_staging_bytes(B: int, Hq: int, Hkv: int) -> int:
    return lib().stief_host_staging_bytes(B, Hq, Hkv)


def stief_decode_step_host(layer: Layer, batch: Batch, q_host: torch.Tensor, k_new_host: torch.Tensor, v_new_host: torch.Tensor,
                           staging: torch.Tensor, workspace: torch.Tensor, out_host: torch.Tensor, num_parts: int = 0,
                           status: Optional[torch.Tensor] = None, flags: int = 0):
    """Host (pinned) q/k/v/out buffers; copies and kernels are enqueued, nothing is synchronised."""
    assert not q_host.is_cuda and not out_host.is_cuda
    cl, cb = layer.c(), batch.c()
    _check(lib().stief_decode_step_host(ctypes.byref(cl), ctypes.byref(cb), _ptr(q_host), _ptr(k_new_host), _ptr(v_new_host),
                                        _ptr(staging), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                        num_parts, _ptr(out_host), flags, _ptr(status), _stream()), "stief_decode_step_host")


def stief_advance_seq_lens(seq_lens: torch.Tensor, delta: int = 1):
    _check(lib().stief_advance_seq_lens(_ptr(seq_lens), seq_lens.numel(), delta, _stream()), "stief_advance_seq_lens")


def stief_time_next_decode_kernel(start_event: Optional[torch.cuda.Event], stop_event: Optional[torch.cuda.Event]):
    """Have the next decode call of this thread record the two (timing-enabled) events around its split-T kernel."""
    if start_event is None:
        _check(lib().stief_time_next_decode_kernel(None, None), "stief_time_next_decode_kernel")
        return
    for ev in (start_event, stop_event):
        if not ev.cuda_event:                 # torch creates the handle lazily, on first record
            ev.record()
    _check(lib().stief_time_next_decode_kernel(start_event.cuda_event, stop_event.cuda_event), "stief_time_next_decode_kernel")


def stief_select_ranks(L: int, cand_k: Sequence[int], cand_v: Sequence[int], rho: float, surfaces=None, surface=None,
                       d_h: int = D_HEAD):
    """Sequential budgeted rank selection (Algorithm 2) on the host.  ``surfaces``: array-like [L][n_k][n_v] of layer
    errors, or ``surface(l, chosen)`` -> table [n_k][n_v], called once per layer with the list of (r_k, r_v) already
    chosen.  Returns (ranks, spent): L pairs and their total cost."""
    import numpy as np
    ck = (ctypes.c_int32 * len(cand_k))(*cand_k)
    cv = (ctypes.c_int32 * len(cand_v))(*cand_v)
    rk, rv = (ctypes.c_int32 * max(L, 1))(), (ctypes.c_int32 * max(L, 1))()
    spent, failed = ctypes.c_double(0.0), ctypes.c_int32(-1)
    tab, cb, raised = None, _SURFACE_FN(), []
    if surfaces is not None:
        tab = np.ascontiguousarray(surfaces, dtype=np.float64)
        if tab.shape != (L, len(cand_k), len(cand_v)):
            raise ValueError("surfaces must be [L][len(cand_k)][len(cand_v)]")
    if surface is not None:
        def _cb(_ctx, l, prk, prv, delta):
            try:
                t = np.asarray(surface(l, [(prk[i], prv[i]) for i in range(l)]), dtype=np.float64)
                if t.shape != (len(cand_k), len(cand_v)):
                    raise ValueError("surface() must return [len(cand_k)][len(cand_v)]")
                for n, x in enumerate(t.ravel()):
                    delta[n] = x
                return 0
            except Exception as e:      # an exception must not unwind through the C frame
                raised.append(e)
                return 1
        cb = _SURFACE_FN(_cb)
    rc = lib().stief_select_ranks(L, d_h, ck, len(cand_k), cv, len(cand_v), float(rho),
                                  None if tab is None else tab.ctypes.data, cb, None, rk, rv,
                                  ctypes.byref(spent), ctypes.byref(failed))
    if raised:
        raise raised[0]
    _check(rc, f"stief_select_ranks (layer {failed.value})" if failed.value >= 0 else "stief_select_ranks")
    return [(rk[l], rv[l]) for l in range(L)], spent.value


def stief_mq_num_splits(B: int, n_q: int, Hq: int, Hkv: int, max_pages_per_seq: int) -> int:
    return lib().stief_mq_num_splits(B, n_q, Hq, Hkv, max_pages_per_seq)


def stief_mq_workspace_bytes(B: int, n_q: int, Hq: int, r_v: int, num_splits: int) -> int:
    return lib().stief_mq_workspace_bytes(B, n_q, Hq, r_v, num_splits)


def stief_mq_attention(layer: Layer, batch: Batch, q: torch.Tensor, out: torch.Tensor, q_lens: Optional[torch.Tensor] = None,
                       out_lse: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None, flags: int = 0,
                       workspace: Optional[torch.Tensor] = None, num_splits: int = 1):
    """Several causal query rows per head: q [B, n_q, Hq, d_q] bf16 -> out [B, n_q, Hq, d_out] bf16 (strides over b and
    t free).  The queries are the last q_lens[b] (default n_q) tokens of each cached sequence.  num_splits > 1 needs a
    workspace tensor of stief_mq_workspace_bytes(...) bytes."""
    assert q.dtype == torch.bfloat16 and out.dtype == torch.bfloat16 and q.dim() == 4 and out.dim() == 4
    assert q.stride(3) == 1 and q.stride(2) == q.shape[3] and out.stride(3) == 1 and out.stride(2) == out.shape[3]
    assert q.shape[3] == (D_HEAD if layer.U_k is not None else layer.r_k)
    assert out.shape[3] == (D_HEAD if layer.U_v is not None else layer.r_v) and out.shape[:3] == q.shape[:3]
    if out_lse is not None:
        assert out_lse.dtype == torch.float32 and out_lse.is_contiguous() and tuple(out_lse.shape) == tuple(q.shape[:3])
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().stief_mq_attention(ctypes.byref(layer.c()), ctypes.byref(batch.c()), _ptr(q), q.stride(0), q.stride(1),
                                    q.shape[1], _ptr(q_lens), _ptr(workspace), ws_bytes, num_splits, _ptr(out), out.stride(0),
                                    out.stride(1), _ptr(out_lse), flags, _ptr(status), _stream()), "stief_mq_attention")


def stief_append_chunk(layer: Layer, batch: Batch, K: torch.Tensor, V: torch.Tensor, chunk_lens: Optional[torch.Tensor] = None,
                       ends_at_len: bool = False, status: Optional[torch.Tensor] = None):
    """K, V [B, T_chunk, Hkv, 128 (or r on a side without basis)] bf16: project and store a run of new tokens per sequence,
    starting at seq_lens[b] (default) or ending at seq_lens[b] - 1 (``ends_at_len``)."""
    assert K.dtype == torch.bfloat16 and V.dtype == torch.bfloat16 and K.dim() == 4 and V.dim() == 4
    assert K.stride(3) == 1 and K.stride(2) == K.shape[3] and V.stride(3) == 1 and V.stride(2) == V.shape[3]
    assert K.shape[3] == (D_HEAD if layer.U_k is not None else layer.r_k) and V.shape[3] == (D_HEAD if layer.U_v is not None else layer.r_v)
    assert K.shape[:3] == V.shape[:3]
    _check(lib().stief_append_chunk(ctypes.byref(layer.c()), ctypes.byref(batch.c()), _ptr(K), _ptr(V), K.stride(0), K.stride(1),
                                    V.stride(0), V.stride(1), K.shape[1], _ptr(chunk_lens), 1 if ends_at_len else 0,
                                    _ptr(status), _stream()), "stief_append_chunk")


def stief_selftest_wait_limit(status: torch.Tensor, report: torch.Tensor, poll_limit: int = 256):
    """Run the kernels' bounded waits to their limit on purpose (see stief.h): status <- STIEF_ERR_TIMEOUT, report int32[8]."""
    assert status.dtype == torch.int32 and report.dtype == torch.int32 and report.numel() >= 8
    _check(lib().stief_selftest_wait_limit(_ptr(status), _ptr(report), poll_limit, _stream()), "stief_selftest_wait_limit")


TRACE_SLOTS = 16


def stief_trace_next_decode_kernel(trace: Optional[torch.Tensor]):
    """Have the next decode call of this thread fill `trace` (zeroed int64 [num_parts, TRACE_SLOTS] on the device) with
    per-CTA time stamps of the GPU's nanosecond timer (slot meanings in stief.h)."""
    if trace is None:
        _check(lib().stief_trace_next_decode_kernel(None, 0), "stief_trace_next_decode_kernel")
        return
    assert trace.dtype == torch.int64 and trace.is_contiguous()
    _check(lib().stief_trace_next_decode_kernel(_ptr(trace), trace.numel() * 8), "stief_trace_next_decode_kernel")


def _q(name: str, bits: int):
    if bits not in (8, 4):
        raise ValueError("code width must be 8 or 4")
    return getattr(lib(), f"stief_q{bits}_{name}")


def stief_q_prefill_compress(bits: int, layer: QLayer, batch: Batch, K: torch.Tensor, V: torch.Tensor, T_max: Optional[int] = None,
                             status: Optional[torch.Tensor] = None, flags: int = 0):
    """stief_q8_prefill_compress / stief_q4_prefill_compress by code width."""
    assert K.stride(3) == 1 and K.stride(2) == D_HEAD and V.stride() == K.stride()
    cl, cb = layer.c(), batch.c()
    _check(_q("prefill_compress", bits)(ctypes.byref(cl), ctypes.byref(cb), _ptr(K), _ptr(V), K.stride(0), K.stride(1),
                                        K.shape[1] if T_max is None else T_max, flags, _ptr(status), _stream()),
           f"stief_q{bits}_prefill_compress")


def stief_q_append(bits: int, layer: QLayer, batch: Batch, k_new: torch.Tensor, v_new: torch.Tensor, status: Optional[torch.Tensor] = None):
    cl, cb = layer.c(), batch.c()
    _check(_q("append", bits)(ctypes.byref(cl), ctypes.byref(cb), _ptr(k_new), _ptr(v_new), _ptr(status), _stream()), f"stief_q{bits}_append")


def stief_q_decode_attention(bits: int, layer: QLayer, batch: Batch, q: torch.Tensor, workspace: torch.Tensor, out: torch.Tensor,
                             num_parts: int = 0, out_lse: Optional[torch.Tensor] = None, len_add: int = 0,
                             status: Optional[torch.Tensor] = None, flags: int = 0):
    cl, cb = layer.c(), batch.c()
    _check(_q("decode_attention", bits)(ctypes.byref(cl), ctypes.byref(cb), _ptr(q), len_add, _ptr(workspace),
                                        workspace.numel() * workspace.element_size(), num_parts, _ptr(out), _ptr(out_lse),
                                        flags, _ptr(status), _stream()), f"stief_q{bits}_decode_attention")


def stief_q_decode_step(bits: int, layer: QLayer, batch: Batch, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor,
                        workspace: torch.Tensor, out: torch.Tensor, num_parts: int = 0, out_lse: Optional[torch.Tensor] = None,
                        status: Optional[torch.Tensor] = None, flags: int = 0):
    cl, cb = layer.c(), batch.c()
    _check(_q("decode_step", bits)(ctypes.byref(cl), ctypes.byref(cb), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(workspace),
                                   workspace.numel() * workspace.element_size(), num_parts, _ptr(out), _ptr(out_lse),
                                   flags, _ptr(status), _stream()), f"stief_q{bits}_decode_step")


def stief_measure_read_stream(buffer: torch.Tensor, status: Optional[torch.Tensor] = None):
    """One read-only pass over a device tensor (time it with events): the bandwidth a kernel that only reads can get."""
    _check(lib().stief_measure_read_stream(_ptr(buffer), buffer.numel() * buffer.element_size(), _ptr(status), _stream()),
           "stief_measure_read_stream")
