"""ctypes binding of libpquant.so: the C entry points under their own names.

Argument marshalling only -- torch tensors are turned into device pointers and
the current CUDA stream is passed along; every step of the layer runs in the
library's kernels.  A missing library is an error (there is no fallback).
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpquant.so")

PQ_OK = 0
PQ_ERR_NULL, PQ_ERR_SHAPE, PQ_ERR_ALIGN, PQ_ERR_WORKSPACE = -1, -2, -3, -4
PQ_ERR_UNSUPPORTED, PQ_ERR_CUDA, PQ_ERR_TIMEOUT, PQ_ERR_TOO_LARGE = -5, -6, -7, -8
PQ_SCALE_VECTOR = 1
PQ_DECODE_DUMP_ACC = 2
PQ_FUSED_RMSNORM = 8
PQ_UNIT_GATES = 4
PQ_PHASE_PACK, PQ_PHASE_FWD, PQ_PHASE_BWD, PQ_PHASE_DECODE = 0, 1, 2, 3

EXPORTS = ("pq_status_string", "pq_workspace_bytes", "pq_saved_bytes", "pq_saved_view_init",
           "pq_decode_view_init", "pq_bwd_view_init", "pq_decode_batch", "pq_decode_pack_bytes", "pq_pack_decode", "pq_decode_pack_hp8_bytes", "pq_pack_decode_hp8", "pq_pack_weights", "pq_pack_weights_static", "pq_pack_experts", "pq_linear_forward", "pq_linear_forward_hp8", "pq_linear_forward_rms", "pq_ffn_workspace_bytes", "pq_ffn_forward", "pq_ffn_view_init", "pq_linear_backward", "pq_debug_gemm", "pq_debug_gemm_tile",
           "pq_device_status", "pq_kernel_launches", "pq_profile_events", "pq_set_option")

KERNEL_IDS = dict(pack_sums=0, binarize_pack=1, router=2, route_scan=3, act_quant=4, hp_up=5, fwd=6, scatter_rows=7,
                  scaled_sign=8, scaled_b=9, hp_dh=10, bwd_dx=11, bwd_dw=12, hp_db=13, hp_da=14, router_wgrad=15,
                  sum_partials=16, sum_scalar=17, debug=18, decode_prep=19, decode_main=20, reduce_db=21, reduce_da=22, decode_pack=23, decode_stream=24)


class PqError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        super().__init__(f"{fn} failed: {status} ({pq_status_string(status)})")


class pq_desc(ctypes.Structure):
    _fields_ = [("size", ctypes.c_uint32), ("flags", ctypes.c_uint32),
                ("T", ctypes.c_int32), ("K", ctypes.c_int32), ("N", ctypes.c_int32),
                ("r", ctypes.c_int32), ("E", ctypes.c_int32), ("top_k", ctypes.c_int32)]


class pq_saved_view(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("q", "xt", "xs", "gamma", "gate", "probs", "expert", "perm", "pos", "offsets", "h",
                 "n_items", "items", "tile_item_begin", "expert_item_begin")] + [("max_items", ctypes.c_int32)]


class pq_decode_item(ctypes.Structure):
    _fields_ = [("desc", pq_desc)] + [(n, ctypes.c_void_p) for n in
                                      ("X", "w_bits", "w_scales", "A", "B", "Wr", "alpha", "beta", "Y", "ws")] + [
        ("ws_bytes", ctypes.c_size_t), ("norm_weight", ctypes.c_void_p), ("norm_eps", ctypes.c_float),
        ("w_bits_il", ctypes.c_void_p), ("B_il", ctypes.c_void_p), ("A8", ctypes.c_void_p), ("B8_il", ctypes.c_void_p),
        ("hp_scales", ctypes.c_void_p)]


class pq_decode_view(ctypes.Structure):
    _fields_ = [("tokens", ctypes.c_void_p), ("acc", ctypes.c_void_p), ("hp_h_int", ctypes.c_void_p), ("hp_z_int", ctypes.c_void_p)]


class pq_ffn_desc(ctypes.Structure):
    _fields_ = [("size", ctypes.c_uint32), ("flags", ctypes.c_uint32), ("T", ctypes.c_int32), ("D", ctypes.c_int32),
                ("F1", ctypes.c_int32), ("r", ctypes.c_int32)]


class pq_ffn_view(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("G1", "U1", "M1", "g_int", "u_int", "qm", "gamma_m", "q_m1", "gamma_m1")]


class pq_bwd_view(ctypes.Structure):
    _fields_ = [("dl", ctypes.c_void_p)]


_lib = None


def lib() -> ctypes.CDLL:
    """Open libpquant.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run __graft_entry__.build() (nvcc, sm_100a) first")
        L = ctypes.CDLL(LIB_PATH)
        vp, sz, ci = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
        dp = ctypes.POINTER(pq_desc)
        L.pq_status_string.restype = ctypes.c_char_p
        L.pq_status_string.argtypes = [ci]
        L.pq_workspace_bytes.restype = sz
        L.pq_workspace_bytes.argtypes = [dp, ci]
        L.pq_saved_bytes.restype = sz
        L.pq_saved_bytes.argtypes = [dp]
        L.pq_saved_view_init.restype = ci
        L.pq_saved_view_init.argtypes = [dp, vp, ctypes.POINTER(pq_saved_view)]
        L.pq_decode_view_init.restype = ci
        L.pq_decode_view_init.argtypes = [dp, vp, ctypes.POINTER(pq_decode_view)]
        L.pq_bwd_view_init.restype = ci
        L.pq_bwd_view_init.argtypes = [dp, vp, ctypes.POINTER(pq_bwd_view)]
        L.pq_decode_batch.restype = ci
        L.pq_decode_batch.argtypes = [ctypes.POINTER(pq_decode_item), ci, vp]
        L.pq_pack_weights.restype = ci
        L.pq_pack_weights.argtypes = [dp, vp, vp, vp, vp, vp, sz, vp]
        L.pq_pack_weights_static.restype = ci
        L.pq_pack_weights_static.argtypes = [dp, vp, vp, vp, vp, vp]
        L.pq_pack_experts.restype = ci
        L.pq_pack_experts.argtypes = [dp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.pq_decode_pack_bytes.restype = ci
        L.pq_decode_pack_bytes.argtypes = [dp, ctypes.POINTER(sz), ctypes.POINTER(sz)]
        L.pq_pack_decode.restype = ci
        L.pq_pack_decode.argtypes = [dp, vp, vp, vp, vp, vp]
        L.pq_decode_pack_hp8_bytes.restype = sz
        L.pq_decode_pack_hp8_bytes.argtypes = [dp]
        L.pq_pack_decode_hp8.restype = ci
        L.pq_pack_decode_hp8.argtypes = [dp, vp, vp, sz, vp]
        L.pq_linear_forward.restype = ci
        L.pq_linear_forward.argtypes = [dp] + [vp] * 10 + [vp, sz, vp, sz, vp]
        L.pq_linear_forward_rms.restype = ci
        L.pq_linear_forward_rms.argtypes = [dp, vp, vp, ctypes.c_float] + [vp] * 8 + [vp, sz, vp, sz, vp]
        L.pq_linear_forward_hp8.restype = ci
        L.pq_linear_forward_hp8.argtypes = [dp] + [vp] * 10 + [vp, sz, vp, sz, vp]
        fp = ctypes.POINTER(pq_ffn_desc)
        L.pq_ffn_workspace_bytes.restype = sz
        L.pq_ffn_workspace_bytes.argtypes = [fp]
        L.pq_ffn_forward.restype = ci
        L.pq_ffn_forward.argtypes = [fp] + [vp] * 15 + [sz, vp]
        L.pq_ffn_view_init.restype = ci
        L.pq_ffn_view_init.argtypes = [fp, vp, ctypes.POINTER(pq_ffn_view)]
        L.pq_linear_backward.restype = ci
        L.pq_linear_backward.argtypes = [dp] + [vp] * 9 + [vp, sz] + [vp] * 7 + [vp, sz, vp]
        L.pq_debug_gemm.restype = ci
        L.pq_debug_gemm.argtypes = [ci, ci, ci, ci, vp, vp, vp, vp]
        L.pq_debug_gemm_tile.restype = ci
        L.pq_debug_gemm_tile.argtypes = [ci, ci, ci, ci, vp, vp, vp, ci, vp]
        L.pq_device_status.restype = ci
        L.pq_device_status.argtypes = [vp, ctypes.POINTER(ci), ctypes.POINTER(ci)]
        L.pq_kernel_launches.restype = ctypes.c_longlong
        L.pq_kernel_launches.argtypes = []
        L.pq_set_option.restype = ci
        L.pq_set_option.argtypes = [ci, ci]
        L.pq_profile_events.restype = ci
        L.pq_profile_events.argtypes = [ci, vp, vp]
        _lib = L
    return _lib


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _nbytes(t):
    return 0 if t is None else t.numel() * t.element_size()


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(fn, status):
    if status != PQ_OK:
        raise PqError(fn, status)


def make_desc(T, K, N, r=0, E=0, top_k=1, scale_vector=False, dump_acc=False, fused_rmsnorm=False, unit_gates=False) -> pq_desc:
    flags = ((PQ_SCALE_VECTOR if scale_vector else 0) | (PQ_DECODE_DUMP_ACC if dump_acc else 0) | (PQ_FUSED_RMSNORM if fused_rmsnorm else 0)
             | (PQ_UNIT_GATES if unit_gates else 0))
    return pq_desc(ctypes.sizeof(pq_desc), flags, T, K, N, r, E, top_k)


def pq_status_string(status: int) -> str:
    return lib().pq_status_string(status).decode()


def pq_workspace_bytes(d: pq_desc, phase: int) -> int:
    return lib().pq_workspace_bytes(ctypes.byref(d), phase)


def pq_saved_bytes(d: pq_desc) -> int:
    return lib().pq_saved_bytes(ctypes.byref(d))


def pq_saved_view_init(d: pq_desc, saved: torch.Tensor) -> dict:
    """Typed torch views into the `saved` byte buffer, keyed like the C struct."""
    v = pq_saved_view()
    _check("pq_saved_view_init", lib().pq_saved_view_init(ctypes.byref(d), _ptr(saved), ctypes.byref(v)))
    base = saved.data_ptr()
    E = max(d.E, 1) if d.r > 0 else 1
    mt = (d.T + 127) // 128

    def view(ptr, dtype, *shape):
        if not ptr:
            return None
        n = 1
        for s in shape:
            n *= s
        nbytes = n * torch.empty(0, dtype=dtype).element_size()
        return saved[ptr - base: ptr - base + nbytes].view(dtype).view(*shape)

    return dict(
        q=view(v.q, torch.int8, d.T, d.K), xt=view(v.xt, torch.bfloat16, d.T, d.K),
        xs=view(v.xs, torch.bfloat16, d.T, d.K), gamma=view(v.gamma, torch.float32, d.T),
        gate=view(v.gate, torch.float32, d.T), probs=view(v.probs, torch.float32, d.T, E),
        expert=view(v.expert, torch.int32, d.T), perm=view(v.perm, torch.int32, d.T),
        pos=view(v.pos, torch.int32, d.T), offsets=view(v.offsets, torch.int32, E + 1),
        h=view(v.h, torch.bfloat16, 2, v.max_items * 128, d.r) if d.r > 0 else None,
        n_items=view(v.n_items, torch.int32, 1), items=view(v.items, torch.int32, v.max_items, 4),
        tile_item_begin=view(v.tile_item_begin, torch.int32, mt + 1),
        expert_item_begin=view(v.expert_item_begin, torch.int32, E + 1), max_items=v.max_items)


def pq_decode_view_init(d: pq_desc, ws: torch.Tensor) -> dict:
    """Views into the decode workspace: per-token expert / gate / gamma / code sum, and the int32 sums if dumped."""
    v = pq_decode_view()
    _check("pq_decode_view_init", lib().pq_decode_view_init(ctypes.byref(d), _ptr(ws), ctypes.byref(v)))
    base = ws.data_ptr()
    raw = ws[v.tokens - base: v.tokens - base + 16 * d.T]
    out = dict(expert=raw.view(torch.int32).view(d.T, 4)[:, 0], gate=raw.view(torch.float32).view(d.T, 4)[:, 1],
               gamma=raw.view(torch.float32).view(d.T, 4)[:, 2], code_sum=raw.view(torch.int32).view(d.T, 4)[:, 3], acc=None)
    if v.acc:
        out["acc"] = ws[v.acc - base: v.acc - base + 4 * d.T * d.N].view(torch.int32).view(d.T, d.N)
    if v.hp_h_int and d.r > 0:
        out["hp_h_int"] = ws[v.hp_h_int - base: v.hp_h_int - base + 4 * d.T * d.r].view(torch.int32).view(d.T, d.r)
    if v.hp_z_int:
        out["hp_z_int"] = ws[v.hp_z_int - base: v.hp_z_int - base + 4 * d.T * d.N].view(torch.int32).view(d.T, d.N)
    return out


def pq_bwd_view_init(d: pq_desc, ws: torch.Tensor) -> dict:
    """Views into the backward workspace: dl [T,E], the router-logit gradient in sorted token order (None when E <= 1)."""
    v = pq_bwd_view()
    _check("pq_bwd_view_init", lib().pq_bwd_view_init(ctypes.byref(d), _ptr(ws), ctypes.byref(v)))
    out = dict(dl=None)
    if v.dl:
        off = v.dl - ws.data_ptr()
        out["dl"] = ws[off: off + 4 * d.T * d.E].view(torch.float32).view(d.T, d.E)
    return out


def pq_pack_weights(d, W, w_bits, w_s8, w_scales, ws, stream=None):
    _check("pq_pack_weights", lib().pq_pack_weights(ctypes.byref(d), _ptr(W), _ptr(w_bits), _ptr(w_s8), _ptr(w_scales),
                                                     _ptr(ws), _nbytes(ws), _stream(stream)))


def pq_pack_weights_static(d, W, w_bits, w_s8, w_scales, stream=None):
    """pq_pack_weights without a workspace argument: for callers that cannot allocate device memory
    (the reduction scratch is a fixed 64 KiB array inside the library; N * K <= 67,108,864)."""
    _check("pq_pack_weights_static", lib().pq_pack_weights_static(ctypes.byref(d), _ptr(W), _ptr(w_bits), _ptr(w_s8),
                                                                   _ptr(w_scales), _stream(stream)))


def pq_pack_experts(d, A, B, A8, B8, hp_scales, ws, stream=None):
    """INT8 codes and per-matrix scales of the expert matrices (Sec. 3.2)."""
    _check("pq_pack_experts", lib().pq_pack_experts(ctypes.byref(d), _ptr(A), _ptr(B), _ptr(A8), _ptr(B8), _ptr(hp_scales), _ptr(ws),
                                                     _nbytes(ws), _stream(stream)))


def pq_linear_forward(d, X, w_bits, w_s8, w_scales, A, B, Wr, alpha, beta, Y, saved, ws, stream=None):
    _check("pq_linear_forward", lib().pq_linear_forward(
        ctypes.byref(d), _ptr(X), _ptr(w_bits), _ptr(w_s8), _ptr(w_scales), _ptr(A), _ptr(B), _ptr(Wr), _ptr(alpha),
        _ptr(beta), _ptr(Y), _ptr(saved), _nbytes(saved), _ptr(ws), _nbytes(ws), _stream(stream)))


def pq_linear_forward_rms(d, X, norm_weight, norm_eps, w_s8, w_scales, A, B, Wr, alpha, beta, Y, saved, ws, stream=None):
    """Training-size forward from un-normalised X with RMSNorm fused in front of the quantiser (d built with fused_rmsnorm=True)."""
    _check("pq_linear_forward_rms", lib().pq_linear_forward_rms(
        ctypes.byref(d), _ptr(X), _ptr(norm_weight), ctypes.c_float(norm_eps), _ptr(w_s8), _ptr(w_scales), _ptr(A), _ptr(B), _ptr(Wr),
        _ptr(alpha), _ptr(beta), _ptr(Y), _ptr(saved), _nbytes(saved), _ptr(ws), _nbytes(ws), _stream(stream)))


def pq_linear_forward_hp8(d, X, w_s8, w_scales, A8, B8, hp_scales, Wr, alpha, beta, Y, saved, ws, stream=None):
    """Forward with the INT8 high-precision branch (Sec. 3.2); A8, B8, hp_scales come from pq_pack_experts."""
    _check("pq_linear_forward_hp8", lib().pq_linear_forward_hp8(
        ctypes.byref(d), _ptr(X), _ptr(w_s8), _ptr(w_scales), _ptr(A8), _ptr(B8), _ptr(hp_scales), _ptr(Wr), _ptr(alpha),
        _ptr(beta), _ptr(Y), _ptr(saved), _nbytes(saved), _ptr(ws), _nbytes(ws), _stream(stream)))


def make_ffn_desc(T, D, F1, r) -> pq_ffn_desc:
    return pq_ffn_desc(ctypes.sizeof(pq_ffn_desc), 0, T, D, F1, r)


def pq_ffn_workspace_bytes(d: pq_ffn_desc) -> int:
    return lib().pq_ffn_workspace_bytes(ctypes.byref(d))


def pq_ffn_forward(d, X, g_s8, g_scales, u_s8, u_scales, d_s8, d_scales, G8, U8, D8, hp_scales, alpha, beta, Y, ws, stream=None):
    """Eq. 11: Y = alpha FFN_INT8[:r](x) + beta FFN_INT1[r:](x) (forward)."""
    _check("pq_ffn_forward", lib().pq_ffn_forward(
        ctypes.byref(d), _ptr(X), _ptr(g_s8), _ptr(g_scales), _ptr(u_s8), _ptr(u_scales), _ptr(d_s8), _ptr(d_scales), _ptr(G8), _ptr(U8),
        _ptr(D8), _ptr(hp_scales), _ptr(alpha), _ptr(beta), _ptr(Y), _ptr(ws), _nbytes(ws), _stream(stream)))


def pq_ffn_view_init(d: pq_ffn_desc, ws: torch.Tensor) -> dict:
    """Typed views of what pq_ffn_forward left in its workspace."""
    v = pq_ffn_view()
    _check("pq_ffn_view_init", lib().pq_ffn_view_init(ctypes.byref(d), _ptr(ws), ctypes.byref(v)))
    base = ws.data_ptr()
    rows = (d.T + 127) // 128 * 128

    def view(ptr, dtype, *shape):
        n = 1
        for s in shape:
            n *= s
        nbytes = n * torch.empty(0, dtype=dtype).element_size()
        return ws[ptr - base: ptr - base + nbytes].view(dtype).view(*shape)

    return dict(G1=view(v.G1, torch.bfloat16, d.T, d.F1), U1=view(v.U1, torch.bfloat16, d.T, d.F1), M1=view(v.M1, torch.bfloat16, d.T, d.F1),
                g_int=view(v.g_int, torch.int32, rows, d.r), u_int=view(v.u_int, torch.int32, rows, d.r),
                qm=view(v.qm, torch.int8, rows, d.r), gamma_m=view(v.gamma_m, torch.float32, rows),
                q_m1=view(v.q_m1, torch.int8, d.T, d.F1), gamma_m1=view(v.gamma_m1, torch.float32, d.T))


def make_decode_items(entries):
    """ctypes array of pq_decode_item from (desc, X, w_bits, w_scales, A, B, Wr, alpha, beta, Y, ws[, norm_weight, norm_eps
    [, w_bits_il, B_il[, A8, B8_il, hp_scales]]]) tuples of tensors (norm_weight, norm_eps: bf16 RMSNorm gain [K] and its epsilon, for un-normalised X;
    w_bits_il, B_il: the weights as laid out by pq_pack_decode).
    The array only holds pointers: keep the tensors alive while it is in use."""
    arr = (pq_decode_item * len(entries))()
    for i, entry in enumerate(entries):
        d, X, w_bits, w_scales, A, B, Wr, alpha, beta, Y, ws = entry[:11]
        norm_weight, norm_eps = (entry[11], entry[12]) if len(entry) > 11 else (None, 0.0)
        arr[i].norm_weight = None if norm_weight is None else norm_weight.data_ptr()
        arr[i].norm_eps = float(norm_eps)
        w_bits_il, B_il = (entry[13], entry[14]) if len(entry) > 13 else (None, None)
        arr[i].w_bits_il = None if w_bits_il is None else w_bits_il.data_ptr()
        arr[i].B_il = None if B_il is None else B_il.data_ptr()
        A8, B8_il, hp_scales = entry[15:18] if len(entry) > 15 else (None, None, None)   # INT8 high-precision branch
        arr[i].A8 = None if A8 is None else A8.data_ptr()
        arr[i].B8_il = None if B8_il is None else B8_il.data_ptr()
        arr[i].hp_scales = None if hp_scales is None else hp_scales.data_ptr()
        arr[i].desc = d
        for name, t in (("X", X), ("w_bits", w_bits), ("w_scales", w_scales), ("A", A), ("B", B), ("Wr", Wr), ("alpha", alpha),
                        ("beta", beta), ("Y", Y), ("ws", ws)):
            setattr(arr[i], name, None if t is None else t.data_ptr())
        arr[i].ws_bytes = _nbytes(ws)
    return arr


def pq_decode_pack_bytes(d) -> tuple[int, int]:
    a, b = ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check("pq_decode_pack_bytes", lib().pq_decode_pack_bytes(ctypes.byref(d), ctypes.byref(a), ctypes.byref(b)))
    return a.value, b.value


def pq_pack_decode(d, w_bits, B, w_bits_il, B_il, stream=None):
    """Lay the sign bits and the rows of B_e out for the streaming decode kernel (one-time, per linear)."""
    _check("pq_pack_decode", lib().pq_pack_decode(ctypes.byref(d), _ptr(w_bits), _ptr(B), _ptr(w_bits_il), _ptr(B_il), _stream(stream)))


def pq_decode_pack_hp8_bytes(d) -> int:
    return lib().pq_decode_pack_hp8_bytes(ctypes.byref(d))


def pq_pack_decode_hp8(d, B8, B8_il, stream=None):
    """The int8 codes of B (pq_pack_experts) in the streaming decode kernel's order."""
    _check("pq_pack_decode_hp8", lib().pq_pack_decode_hp8(ctypes.byref(d), _ptr(B8), _ptr(B8_il), _nbytes(B8_il), _stream(stream)))


def pq_decode_batch(items, stream=None):
    """Decode forward of independent linears in one launch pair; `items` comes from make_decode_items."""
    _check("pq_decode_batch", lib().pq_decode_batch(items, len(items), _stream(stream)))


def pq_linear_backward(d, dY, X, w_s8, w_scales, A, B, Wr, alpha, beta, saved, dX, dW, dA, dB, dWr, dalpha, dbeta, ws,
                       stream=None):
    _check("pq_linear_backward", lib().pq_linear_backward(
        ctypes.byref(d), _ptr(dY), _ptr(X), _ptr(w_s8), _ptr(w_scales), _ptr(A), _ptr(B), _ptr(Wr), _ptr(alpha), _ptr(beta),
        _ptr(saved), _nbytes(saved), _ptr(dX), _ptr(dW), _ptr(dA), _ptr(dB), _ptr(dWr), _ptr(dalpha), _ptr(dbeta),
        _ptr(ws), _nbytes(ws), _stream(stream)))


def pq_debug_gemm(mode, M, N, K, A, B, D, stream=None):
    _check("pq_debug_gemm", lib().pq_debug_gemm(mode, M, N, K, _ptr(A), _ptr(B), _ptr(D), _stream(stream)))


def pq_debug_gemm_tile(mode, M, N, K, A, B, D, tile_n, stream=None):
    _check("pq_debug_gemm_tile", lib().pq_debug_gemm_tile(mode, M, N, K, _ptr(A), _ptr(B), _ptr(D), tile_n, _stream(stream)))


def pq_device_status(stream=None) -> tuple[int, int]:
    code, where = ctypes.c_int(0), ctypes.c_int(0)
    _check("pq_device_status", lib().pq_device_status(_stream(stream), ctypes.byref(code), ctypes.byref(where)))
    return code.value, where.value


PQ_OPT_DECODE_PDL = 1
PQ_OPT_SIDE_STREAM = 2
PQ_OPT_SPIN_CYCLES = 3
PQ_OPT_DECODE_STREAM = 4
PQ_OPT_DECODE_PREFETCH = 5
PQ_OPT_DECODE_MMA_FROM = 6
PQ_OPT_DECODE_INTERLEAVE = 7


def pq_set_option(option: int, value: int):
    _check("pq_set_option", lib().pq_set_option(option, value))


def pq_kernel_launches() -> int:
    return lib().pq_kernel_launches()


def pq_profile_events(kernel_id: int, start: "torch.cuda.Event | None", stop: "torch.cuda.Event | None"):
    """Bracket every later launch of kernel `kernel_id` with the two events (None, None clears).
    The events must have been created with enable_timing=True and recorded once already
    (torch creates the underlying cudaEvent lazily)."""
    s = None if start is None else ctypes.c_void_p(start.cuda_event)
    e = None if stop is None else ctypes.c_void_p(stop.cuda_event)
    _check("pq_profile_events", lib().pq_profile_events(kernel_id, s, e))
