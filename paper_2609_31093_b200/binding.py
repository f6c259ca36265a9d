"""ctypes binding with the C ABI's names (include/pisa.h).  No arithmetic happens here."""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libpisa.so")
_lib = None

BF16, FP32 = 0, 1
SCORE_LSE, SCORE_MEAN, SCORE_MEAN_VAR = 0, 1, 2
OP_ROUTE, OP_BSA, OP_FORWARD, OP_FLAT, OP_FORWARD_HOST, OP_DECODE, OP_BSA_BWD, OP_FORWARD_PACKED, OP_BSA_BWD_PACKED = 0, 1, 2, 3, 4, 5, 6, 7, 8
IMPL_AUTO, IMPL_SIMT, IMPL_TENSOR = 0, 1, 2
DEBUG_BOUNDS = 1
_SCORE = {"lse": SCORE_LSE, "mean": SCORE_MEAN, "mean_var": SCORE_MEAN_VAR}


class PisaError(RuntimeError):
    pass


class _CParams(C.Structure):
    _fields_ = [
        ("B", C.c_int32), ("N", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32),
        ("d", C.c_int32), ("C", C.c_int32), ("g", C.c_int32), ("K", C.c_int32),
        ("causal", C.c_int32), ("dtype", C.c_int32), ("score_mode", C.c_int32), ("impl", C.c_int32),
        ("scale", C.c_float), ("debug", C.c_int32),
        ("q_stride", C.c_int64 * 3), ("k_stride", C.c_int64 * 3),
        ("v_stride", C.c_int64 * 3), ("o_stride", C.c_int64 * 3),
    ]


def lib():
    """Loads libpisa.so (once).  There is no fallback: a missing library is an error."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise PisaError(f"{_LIB_PATH} is missing: build it with `python -m paper_2609_31093_b200.build`")
    L = C.CDLL(_LIB_PATH)
    vp, i32p, f32p, szp = C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_float), C.POINTER(C.c_size_t)
    pp = C.POINTER(_CParams)
    L.pisa_version.restype = C.c_int
    L.pisa_status_string.restype = C.c_char_p
    L.pisa_status_string.argtypes = [C.c_int]
    L.pisa_last_cuda_error.restype = C.c_char_p
    L.pisa_pyramid_layout.argtypes = [pp, i32p, i32p, C.POINTER(C.c_int64), szp]
    L.pisa_workspace_bytes.argtypes = [pp, C.c_int, szp]
    L.pisa_build_pyramid.argtypes = [pp, vp, vp, vp]
    L.pisa_route.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]
    L.pisa_bsa_fwd.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]
    L.pisa_forward.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]
    L.pisa_forward_host.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]
    L.pisa_flat_select.argtypes = [pp, vp, vp, vp, vp, C.c_size_t, vp]
    L.pisa_decode_step.argtypes = [pp, C.c_int32, vp, vp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]
    L.pisa_pyramid_regrow.argtypes = [pp, pp, vp, vp, vp]
    L.pisa_bsa_bwd.argtypes = [pp] + [vp] * 11 + [C.c_size_t, vp]
    L.pisa_forward_packed.argtypes = [pp, i32p, C.c_int32] + [vp] * 8 + [C.c_size_t, vp]
    L.pisa_bsa_bwd_packed.argtypes = [pp, i32p, C.c_int32] + [vp] * 11 + [C.c_size_t, vp]
    L.pisa_packed_plan.argtypes = [pp, i32p, C.c_int32, i32p, i32p, i32p]
    L.pisa_read_status.argtypes = [vp, i32p]
    L.pisa_route_static.argtypes = [pp, vp, vp, vp, vp, vp, vp]
    L.pisa_route_static.restype = C.c_int
    L.pisa_route_static_capacity.restype = C.c_size_t
    L.pisa_set_stage_timing.argtypes = [C.c_int]
    L.pisa_set_forward_chunks.argtypes = [C.c_int]
    L.pisa_get_stage_ms.argtypes = [f32p, f32p, f32p]
    L.pisa_launch_count.restype = C.c_ulonglong
    L.pisa_get_kernel_ms.argtypes = [C.c_int, C.c_char_p, C.c_size_t, f32p]
    L.pisa_get_kernel_ms.restype = C.c_int
    L.pisa_debug_wait_timeout.argtypes = [vp, C.c_ulonglong, vp]
    L.pisa_debug_wait_timeout.restype = C.c_int
    for name in ("pisa_pyramid_layout", "pisa_workspace_bytes", "pisa_build_pyramid", "pisa_route",
                 "pisa_bsa_fwd", "pisa_forward", "pisa_forward_host", "pisa_flat_select", "pisa_read_status",
                 "pisa_decode_step", "pisa_pyramid_regrow", "pisa_bsa_bwd", "pisa_forward_packed", "pisa_bsa_bwd_packed",
                 "pisa_set_stage_timing", "pisa_get_stage_ms", "pisa_set_forward_chunks", "pisa_packed_plan"):
        getattr(L, name).restype = C.c_int
    _lib = L
    return L


def _check(st: int, what: str):
    if st != 0:
        L = lib()
        msg = L.pisa_status_string(st).decode()
        cuda = L.pisa_last_cuda_error().decode()
        raise PisaError(f"{what}: {msg} ({st})" + (f" [{cuda}]" if cuda and st == -4 else ""))


class Params:
    """Problem description in the paper's notation; mirrors pisa_params_t."""

    def __init__(self, B, N, Hq, Hkv, d, C, g, K, dtype="bf16", score_mode="lse", scale=0.0, impl=IMPL_AUTO, debug=0):
        self.c = _CParams()
        self.c.B, self.c.N, self.c.Hq, self.c.Hkv = B, N, Hq, Hkv
        self.c.d, self.c.C, self.c.g, self.c.K = d, C, g, K
        self.c.causal = 1
        self.c.dtype = BF16 if dtype == "bf16" else FP32
        self.c.score_mode = _SCORE[score_mode] if isinstance(score_mode, str) else int(score_mode)
        self.c.impl = impl
        self.c.scale = float(scale)
        self.c.debug = int(debug)
        self.dtype = dtype
        self.B, self.N, self.Hq, self.Hkv, self.d, self.C, self.g, self.K = B, N, Hq, Hkv, d, C, g, K

    def set_strides(self, q=None, k=None, v=None, o=None):
        """Element strides (batch, token, head) of q, k, v and out; None keeps a tensor dense [B, N, H, d].
        The last dimension is always contiguous."""
        for name, val in (("q_stride", q), ("k_stride", k), ("v_stride", v), ("o_stride", o)):
            arr = getattr(self.c, name)
            for i in range(3):
                arr[i] = 0 if val is None else int(val[i])
        return self

    @classmethod
    def from_workload(cls, w, B=None, **kw):
        return cls(w.B if B is None else B, w.N, w.Hq, w.Hkv, w.d, w.C, w.g, w.K, dtype=w.dtype, **kw)

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    def ref(self):
        return C.byref(self.c)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def pyramid_layout(p: Params) -> Tuple[int, list, list, int]:
    """(L, M[0..L], level_off[0..L] in elements, bytes)."""
    L = C.c_int32()
    M = (C.c_int32 * 34)()
    off = (C.c_int64 * 34)()
    nbytes = C.c_size_t()
    _check(lib().pisa_pyramid_layout(p.ref(), C.byref(L), M, off, C.byref(nbytes)), "pisa_pyramid_layout")
    return L.value, list(M[:L.value + 1]), list(off[:L.value + 1]), nbytes.value


def workspace_bytes(p: Params, op: int) -> int:
    n = C.c_size_t()
    _check(lib().pisa_workspace_bytes(p.ref(), op, C.byref(n)), "pisa_workspace_bytes")
    return n.value


def alloc_pyramid(p: Params, device="cuda") -> torch.Tensor:
    nbytes = pyramid_layout(p)[3]
    es = 2 if p.dtype == "bf16" else 4
    return torch.empty(nbytes // es, dtype=p.torch_dtype, device=device)


def alloc_workspace(p: Params, op: int, device="cuda") -> torch.Tensor:
    return torch.zeros(max(workspace_bytes(p, op), 256), dtype=torch.uint8, device=device)


def pisa_build_pyramid(p: Params, k: torch.Tensor, pyramid: torch.Tensor):
    _check(lib().pisa_build_pyramid(p.ref(), _ptr(k), _ptr(pyramid), _stream()), "pisa_build_pyramid")


def pisa_route(p: Params, q, k, pyramid, idx, margin, ws, sel_lse=None):
    """sel_lse: optional float [B, Hq, N, K] output (per-head denominators of the kept leaves)."""
    _check(lib().pisa_route(p.ref(), _ptr(q), _ptr(k), _ptr(pyramid), _ptr(idx), _ptr(sel_lse), _ptr(margin),
                            _ptr(ws), ws.numel(), _stream()), "pisa_route")


def pisa_route_static(p: Params, q, k, pyramid, idx, margin):
    """pisa_route without a workspace argument: scratch lives in a device array inside the library.
    For callers that may not allocate device memory; refuses problems above
    pisa_route_static_capacity() and must not overlap with another such call on the same GPU."""
    _check(lib().pisa_route_static(p.ref(), _ptr(q), _ptr(k), _ptr(pyramid), _ptr(idx), _ptr(margin), _stream()),
           "pisa_route_static")


def route_static_capacity() -> int:
    return int(lib().pisa_route_static_capacity())


def pisa_bsa_fwd(p: Params, q, k, v, idx, out, lse, ws, sel_lse=None):
    """sel_lse: optional float [B, Hq, N, K] input, as pisa_route wrote it for these idx."""
    _check(lib().pisa_bsa_fwd(p.ref(), _ptr(q), _ptr(k), _ptr(v), _ptr(idx), _ptr(sel_lse), _ptr(out), _ptr(lse),
                              _ptr(ws), ws.numel(), _stream()), "pisa_bsa_fwd")


def pisa_forward(p: Params, q, k, v, pyramid, idx, out, lse, ws):
    _check(lib().pisa_forward(p.ref(), _ptr(q), _ptr(k), _ptr(v), _ptr(pyramid), _ptr(idx), _ptr(out),
                              _ptr(lse), _ptr(ws), ws.numel(), _stream()), "pisa_forward")


def pisa_forward_packed(p: Params, cu_seqlens, q, k, v, pyramid, idx, out, lse, ws):
    """Packed variable-length batch; cu_seqlens is a host sequence of nseq + 1 offsets, p.N the longest length."""
    cu = (C.c_int32 * len(cu_seqlens))(*[int(x) for x in cu_seqlens])
    _check(lib().pisa_forward_packed(p.ref(), cu, len(cu_seqlens) - 1, _ptr(q), _ptr(k), _ptr(v), _ptr(pyramid),
                                     _ptr(idx), _ptr(out), _ptr(lse), _ptr(ws), ws.numel(), _stream()),
           "pisa_forward_packed")


def packed_plan(p: Params, cu_seqlens):
    """Host-only: (group, padded, n_groups) of pisa_forward_packed's grouping; group -1 = the sequence runs alone."""
    n = len(cu_seqlens) - 1
    cu = (C.c_int32 * len(cu_seqlens))(*[int(x) for x in cu_seqlens])
    group, padded, ng = (C.c_int32 * max(n, 1))(), (C.c_int32 * max(n, 1))(), C.c_int32(0)
    _check(lib().pisa_packed_plan(p.ref(), cu, n, group, padded, C.byref(ng)), "pisa_packed_plan")
    return list(group)[:n], list(padded)[:n], int(ng.value)


def pisa_forward_host(p: Params, q_host, k_host, v_host, out_host, lse_host, idx_host, ws):
    """Host tensors in, host tensors out; `ws` is a device arena sized for OP_FORWARD_HOST."""
    for t in (q_host, k_host, v_host, out_host, lse_host):
        assert not t.is_cuda and t.is_contiguous()
    _check(lib().pisa_forward_host(p.ref(), _ptr(q_host), _ptr(k_host), _ptr(v_host), _ptr(out_host),
                                   _ptr(lse_host), _ptr(idx_host), _ptr(ws), ws.numel(), _stream()),
           "pisa_forward_host")


def pisa_bsa_bwd(p: Params, q, k, v, idx, out, lse, dout, dq, dk, dv, ws):
    """Gradients of the block-sparse attention for fixed idx; dq, dk, dv are dense outputs."""
    _check(lib().pisa_bsa_bwd(p.ref(), _ptr(q), _ptr(k), _ptr(v), _ptr(idx), _ptr(out), _ptr(lse), _ptr(dout),
                              _ptr(dq), _ptr(dk), _ptr(dv), _ptr(ws), ws.numel(), _stream()), "pisa_bsa_bwd")


def pisa_bsa_bwd_packed(p: Params, cu_seqlens, q, k, v, idx, out, lse, dout, dq, dk, dv, ws):
    """pisa_bsa_bwd over a packed variable-length batch laid out as for pisa_forward_packed."""
    cu = (C.c_int32 * len(cu_seqlens))(*[int(x) for x in cu_seqlens])
    _check(lib().pisa_bsa_bwd_packed(p.ref(), cu, len(cu_seqlens) - 1, _ptr(q), _ptr(k), _ptr(v), _ptr(idx),
                                     _ptr(out), _ptr(lse), _ptr(dout), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(ws),
                                     ws.numel(), _stream()), "pisa_bsa_bwd_packed")


def pisa_decode_step(p: Params, pos: int, q, k_cache, v_cache, pyramid, idx, out, lse, ws):
    """One decoding step at position `pos`; p.N is the capacity of the caches."""
    _check(lib().pisa_decode_step(p.ref(), int(pos), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(pyramid),
                                  _ptr(idx), _ptr(out), _ptr(lse), _ptr(ws), ws.numel(), _stream()),
           "pisa_decode_step")


def pisa_pyramid_regrow(p_old: Params, p_new: Params, pyramid_old, pyramid_new):
    _check(lib().pisa_pyramid_regrow(p_old.ref(), p_new.ref(), _ptr(pyramid_old), _ptr(pyramid_new), _stream()),
           "pisa_pyramid_regrow")


def pisa_flat_select(p: Params, q, pyramid, idx, ws):
    _check(lib().pisa_flat_select(p.ref(), _ptr(q), _ptr(pyramid), _ptr(idx), _ptr(ws), ws.numel(), _stream()),
           "pisa_flat_select")


def debug_wait_timeout(ws, limit_ns: int):
    """Launches the bounded-wait self-test (one CTA waiting on a barrier nobody arrives at)."""
    _check(lib().pisa_debug_wait_timeout(_ptr(ws), int(limit_ns), _stream()), "pisa_debug_wait_timeout")


def read_status(ws) -> int:
    st = C.c_int32()
    _check(lib().pisa_read_status(_ptr(ws), C.byref(st)), "pisa_read_status")
    return st.value


def set_stage_timing(enable: bool):
    _check(lib().pisa_set_stage_timing(1 if enable else 0), "pisa_set_stage_timing")


def get_stage_ms() -> Tuple[float, float, float]:
    a, b, c = C.c_float(), C.c_float(), C.c_float()
    _check(lib().pisa_get_stage_ms(C.byref(a), C.byref(b), C.byref(c)), "pisa_get_stage_ms")
    return a.value, b.value, c.value


def launch_count() -> int:
    return int(lib().pisa_launch_count())


def set_forward_chunks(max_chunks: int):
    """0 = automatic chunking of pisa_forward over two streams, 1 = never split."""
    _check(lib().pisa_set_forward_chunks(int(max_chunks)), "pisa_set_forward_chunks")


def get_kernel_brackets() -> list:
    """[(bracket name, device ms)] of the last pisa_forward issued with stage timing on, one entry per
    launch bracket (a name occurs once per chunk); the closing brackets of the streams are left out."""
    out = []
    buf = C.create_string_buffer(64)
    ms = C.c_float()
    i = 0
    while lib().pisa_get_kernel_ms(i, buf, 64, C.byref(ms)) == 0:
        name = buf.value.decode()
        if name != "end":
            out.append((name, ms.value))
        i += 1
    return out


def get_kernel_ms() -> dict:
    """{bracket name: device ms summed over its launches} of the last pisa_forward with stage timing on."""
    out = {}
    for name, t in get_kernel_brackets():
        out[name] = out.get(name, 0.0) + t
    return out
