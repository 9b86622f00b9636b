"""Thin ctypes binding of libturboboa.so: argument marshalling only.

Every function has the name of the C entry point it calls (include/turboboa.h)
and takes torch CUDA tensors; torch provides device memory and the stream and
nothing else.  There is no CPU path: a missing library or a missing GPU raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

from . import _build

TB_OK = 0
TB_F32, TB_BF16 = 0, 1
TB_F_ADAPTIVE_GRID, TB_F_CD_REFINE, TB_F_DYNAMIC_GRID = 1, 2, 4

_STATUS_NAMES = {0: "TB_OK", 1: "TB_ERR_INVALID_ARG", 2: "TB_ERR_UNSUPPORTED", 3: "TB_ERR_WORKSPACE",
                 4: "TB_ERR_NOT_SPD", 5: "TB_ERR_CUDA", 6: "TB_ERR_TIMEOUT"}


class TurboBoAError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {_STATUS_NAMES.get(status, status)} ({status_string(status)})")


class LayerDesc(ctypes.Structure):
    """tb_layer_desc"""
    _fields_ = [("d_out", ctypes.c_int), ("d_in", ctypes.c_int), ("n_heads", ctypes.c_int),
                ("d_head", ctypes.c_int), ("n_hin", ctypes.c_int), ("bits", ctypes.c_int),
                ("quant_group", ctypes.c_int), ("out_block", ctypes.c_int), ("n_cand", ctypes.c_int),
                ("cd_iters", ctypes.c_int), ("flags", ctypes.c_uint)]

    @property
    def n_groups(self) -> int:
        return 1 if self.quant_group == 0 else self.d_in // self.quant_group


def layer_desc(d_out, d_in, n_heads, d_head, bits, quant_group=0, out_block=1, n_hin=1, n_cand=16,
               cd_iters=1, flags=0) -> LayerDesc:
    return LayerDesc(d_out, d_in, n_heads, d_head, n_hin, bits, quant_group, out_block, n_cand,
                     cd_iters, flags)


class Stats(ctypes.Structure):
    """tb_stats"""
    _fields_ = [("near_tie_codes", ctypes.c_ulonglong), ("clamped_codes", ctypes.c_ulonglong),
                ("column_steps", ctypes.c_ulonglong), ("reserved", ctypes.c_ulonglong * 5)]


_lib = None
_vp, _sz, _ll, _int, _f = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_longlong, ctypes.c_int, ctypes.c_float
_SIGNATURES = {
    "tb_status_string": (ctypes.c_char_p, [_int]),
    "tb_accumulate_hessian": (_int, [_vp, _vp, _int, _ll, _int, _vp]),
    "tb_device_error_flag": (_int, []),
    "tb_selftest_bounded_wait": (_int, [_ll, _vp, _vp]),
    "tb_accumulate_cross_workspace": (_sz, [_int, _ll, _int]),
    "tb_accumulate_cross": (_int, [_vp, _vp, _vp, _int, _ll, _int, _f, _vp, _sz, _vp]),
    "tb_finalize_hessian": (_int, [_vp, _vp, _vp, _int, _ll, _f, _vp]),
    "tb_build_hout_workspace": (_sz, [_int, _int, _int]),
    "tb_build_hout": (_int, [_vp, _vp, _vp, _int, _int, _int, _int, _f, _vp, _sz, _vp]),
    "tb_factor_workspace": (_sz, [_int, _int]),
    "tb_factor": (_int, [_vp, _int, _int, _vp, _vp, _vp, _vp, _sz, _vp]),
    "tb_factor_static_capacity": (_sz, []),
    "tb_factor_static": (_int, [_vp, _int, _int, _vp, _vp, _vp]),
    "tb_prepare_correction_workspace": (_sz, [_int, _int]),
    "tb_prepare_correction": (_int, [_vp, _vp, _int, _int, _vp, _vp, _vp, _sz, _vp]),
    "tb_quantize_layer_workspace": (_sz, [ctypes.POINTER(LayerDesc), _int, _int]),
    "tb_quantize_layer": (_int, [ctypes.POINTER(LayerDesc)] + [_vp] * 16 + [_vp, _sz, _vp]),
    "tb_quantize_block": (_int, [_vp, _int, _int, _vp]),
    "tb_attention_layer_info_count": (_int, [_vp, _int]),
    "tb_attention_layer_workspace": (_sz, [_vp, _vp]),
    "tb_attention_layer": (_int, [_vp, _vp, _vp, _sz, _vp]),
    "tb_launch_count": (ctypes.c_ulonglong, []),
    "tb_packed_bytes": (_sz, [_int, _int, _int]),
    "tb_pack_codes": (_int, [_vp, _int, _int, _int, _vp, _vp]),
    "tb_unpack_dequant": (_int, [_vp, _vp, _vp, _int, _int, _int, _int, _vp, _vp, _vp, _vp, _f, _vp, _vp]),
    "tb_profile_enable": (None, [_int]),
    "tb_profile_read": (_int, [ctypes.POINTER(ctypes.c_double), _int]),
    "tb_quantize_from_host_workspace": (_sz, [ctypes.POINTER(LayerDesc), _ll, _int]),
    "tb_quantize_from_host": (_int, [ctypes.POINTER(LayerDesc), _vp, _vp, _ll, _vp, _int, _f, _f,
                                     _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
}


def library_path() -> str:
    return _build.LIB


def load(build_if_missing: bool = True) -> ctypes.CDLL:
    """Load libturboboa.so (building it in-tree first if it is absent or stale)."""
    global _lib
    if _lib is None:
        if build_if_missing:
            _build.build()
        if not os.path.exists(_build.LIB):
            raise RuntimeError("libturboboa.so is missing; run `python -m paper_2602_04929_b200._build`")
        lib = ctypes.CDLL(_build.LIB)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def exported_symbols() -> list[str]:
    return sorted(_SIGNATURES)


def status_string(status: int) -> str:
    return load().tb_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != TB_OK:
        raise TurboBoAError(status, where)


def _ptr(t, dtype=None, allow_none=False):
    if t is None:
        if allow_none:
            return None
        raise ValueError("a required tensor is None")
    if not t.is_cuda:
        raise ValueError("tensors must live on a CUDA device (there is no CPU path)")
    if not t.is_contiguous():
        raise ValueError("tensors must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected {dtype}, got {t.dtype}")
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _workspace(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def _xtype(X):
    if X.dtype == torch.bfloat16:
        return TB_BF16
    if X.dtype == torch.float32:
        return TB_F32
    raise ValueError("activations must be bfloat16 or float32")


def tb_accumulate_hessian(H, X) -> None:
    n_tok, d = X.shape
    _check(load().tb_accumulate_hessian(_ptr(H, torch.float32), _ptr(X) if n_tok else None, _xtype(X), n_tok, d,
                                        _stream()),
           "tb_accumulate_hessian")


def tb_device_error_flag() -> int:
    return int(load().tb_device_error_flag())


def tb_selftest_bounded_wait(budget_cycles: int, gave_up=None) -> None:
    _check(load().tb_selftest_bounded_wait(int(budget_cycles), _ptr(gave_up, torch.int32, True), _stream()),
           "tb_selftest_bounded_wait")


def tb_accumulate_cross(R, X, Xfp, alpha: float) -> None:
    n_tok, d = X.shape
    if Xfp.dtype != X.dtype or Xfp.shape != X.shape:
        raise ValueError("X and Xfp must agree in shape and dtype")
    lib = load()
    nbytes = lib.tb_accumulate_cross_workspace(_xtype(X), n_tok, d)
    ws = _workspace(nbytes, X.device) if nbytes else None
    _check(lib.tb_accumulate_cross(_ptr(R, torch.float32), _ptr(X), _ptr(Xfp), _xtype(X), n_tok, d, float(alpha),
                                   _ptr(ws, None, True), nbytes if ws is not None else 0, _stream()),
           "tb_accumulate_cross")


def tb_finalize_hessian(H, R, n_total: int, damp: float, Hsum_out=None) -> None:
    d = H.shape[-1]
    _check(load().tb_finalize_hessian(_ptr(H, torch.float32), _ptr(R, torch.float32, True),
                                      _ptr(Hsum_out, torch.float32, True), d, int(n_total), float(damp),
                                      _stream()), "tb_finalize_hessian")


def tb_build_hout(G, Hsum, n_heads: int, d_head: int, damp: float):
    rows, d = G.shape
    g_heads = rows // d_head
    lib = load()
    H_out = torch.empty((n_heads, d_head, d_head), dtype=torch.float32, device=G.device)
    ws = _workspace(lib.tb_build_hout_workspace(g_heads, d_head, d), G.device)
    _check(lib.tb_build_hout(_ptr(H_out), _ptr(G, torch.float32), _ptr(Hsum, torch.float32, True), n_heads,
                             g_heads, d_head, d, float(damp), _ptr(ws), ws.numel(), _stream()),
           "tb_build_hout")
    return H_out


def tb_factor(H, want_inverse: bool = False):
    """Returns (U, info[, Hinv]) for H of shape [n_batch, d, d] or [d, d]."""
    squeeze = H.dim() == 2
    Hb = H.unsqueeze(0) if squeeze else H
    n_batch, d, _ = Hb.shape
    lib = load()
    U = torch.empty_like(Hb)
    Hinv = torch.empty_like(Hb) if want_inverse else None
    info = torch.empty(n_batch, dtype=torch.int32, device=H.device)
    ws = _workspace(lib.tb_factor_workspace(n_batch, d), H.device)
    _check(lib.tb_factor(_ptr(Hb, torch.float32), n_batch, d, _ptr(U), _ptr(Hinv, None, True), _ptr(info),
                         _ptr(ws), ws.numel(), _stream()), "tb_factor")
    if squeeze:
        U = U[0]
        Hinv = Hinv[0] if want_inverse else None
    return (U, info, Hinv) if want_inverse else (U, info)


def tb_factor_static(H, U=None, info=None):
    """tb_factor through the library's own fixed scratch array: no workspace is
    allocated here or in the library.  Pass preallocated U and info to make the
    call itself allocation-free; otherwise they are created with torch."""
    squeeze = H.dim() == 2
    Hb = H.unsqueeze(0) if squeeze else H
    n_batch, d, _ = Hb.shape
    if U is None:
        U = torch.empty_like(Hb)
    if info is None:
        info = torch.empty(n_batch, dtype=torch.int32, device=H.device)
    _check(load().tb_factor_static(_ptr(Hb, torch.float32), n_batch, d, _ptr(U, torch.float32), _ptr(info),
                                   _stream()), "tb_factor_static")
    return (U[0] if squeeze and U.dim() == 3 else U), info


def tb_prepare_correction(R, U_in):
    squeeze = R.dim() == 2
    Rb = R.unsqueeze(0) if squeeze else R
    Ub = U_in.unsqueeze(0) if squeeze else U_in
    n_batch, d, _ = Rb.shape
    lib = load()
    P = torch.empty_like(Rb)
    C = torch.empty_like(Rb)
    ws = _workspace(lib.tb_prepare_correction_workspace(n_batch, d), R.device)
    _check(lib.tb_prepare_correction(_ptr(Rb, torch.float32), _ptr(Ub, torch.float32), n_batch, d, _ptr(P),
                                     _ptr(C), _ptr(ws), ws.numel(), _stream()), "tb_prepare_correction")
    return (P[0], C[0]) if squeeze else (P, C)


@dataclass
class QuantizeResult:
    codes: torch.Tensor
    scales: torch.Tensor
    zeros: torch.Tensor
    cand: torch.Tensor
    w_hat: torch.Tensor
    loss: torch.Tensor | None
    stats: torch.Tensor
    w_comp: torch.Tensor | None = None   # float64 [d_out][d_in], the compensated weights (optional output)

    def stats_dict(self) -> dict:
        v = self.stats.cpu().tolist()
        return {"near_tie_codes": v[0], "clamped_codes": v[1], "column_steps": v[2]}


def tb_quantize_layer_workspace(desc: LayerDesc, with_r: bool, with_loss: bool) -> int:
    return int(load().tb_quantize_layer_workspace(ctypes.byref(desc), int(with_r), int(with_loss)))


def tb_quantize_layer(desc: LayerDesc, W, H_in, U_in, H_out=None, U_out=None, R=None, P=None, C=None,
                      want_loss: bool = True, ws=None, out: QuantizeResult | None = None,
                      want_w_comp: bool = False) -> QuantizeResult:
    lib = load()
    dev = W.device
    ng = desc.n_groups
    if out is None:
        out = QuantizeResult(
            codes=torch.empty((desc.d_out, desc.d_in), dtype=torch.uint8, device=dev),
            scales=torch.empty((desc.d_out, ng), dtype=torch.float32, device=dev),
            zeros=torch.empty((desc.d_out, ng), dtype=torch.int32, device=dev),
            cand=torch.empty((desc.d_out, ng), dtype=torch.uint8, device=dev),
            w_hat=torch.empty((desc.d_out, desc.d_in), dtype=torch.float32, device=dev),
            loss=torch.empty(desc.n_heads, dtype=torch.float64, device=dev) if want_loss else None,
            stats=torch.zeros(8, dtype=torch.int64, device=dev),
            w_comp=torch.empty((desc.d_out, desc.d_in), dtype=torch.float64, device=dev) if want_w_comp else None)
    if ws is None:
        ws = _workspace(tb_quantize_layer_workspace(desc, R is not None, out.loss is not None), dev)
    f32 = torch.float32
    _check(lib.tb_quantize_layer(
        ctypes.byref(desc), _ptr(W, f32), _ptr(H_in, f32), _ptr(U_in, f32), _ptr(H_out, f32, True),
        _ptr(U_out, f32, True), _ptr(R, f32, True), _ptr(P, f32, True), _ptr(C, f32, True),
        _ptr(out.codes), _ptr(out.scales), _ptr(out.zeros), _ptr(out.cand), _ptr(out.w_hat),
        _ptr(out.w_comp, torch.float64, True), _ptr(out.loss, None, True), _ptr(out.stats), _ptr(ws), ws.numel(), _stream()), "tb_quantize_layer")
    return out


def tb_quantize_from_host_workspace(desc: LayerDesc, n_tok: int, g_heads: int) -> int:
    return int(load().tb_quantize_from_host_workspace(ctypes.byref(desc), int(n_tok), int(g_heads)))


def tb_quantize_from_host(desc: LayerDesc, W_host, X_host, G_host, damp_in: float, damp_out: float,
                          out_host: dict, dev_ws) -> None:
    """All *_host arguments are CPU tensors (pinned for asynchronous copies);
    out_host holds preallocated CPU tensors codes, scales, zeros, w_hat, loss."""
    lib = load()

    def hp(t):
        if t is None:
            return None
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("host tensors must be contiguous CPU tensors")
        return ctypes.c_void_p(t.data_ptr())

    n_tok = X_host.shape[0]
    g_heads = 0 if G_host is None else G_host.shape[0] // desc.d_head
    _check(lib.tb_quantize_from_host(
        ctypes.byref(desc), hp(W_host), hp(X_host), n_tok, hp(G_host), g_heads, float(damp_in),
        float(damp_out), hp(out_host["codes"]), hp(out_host["scales"]), hp(out_host["zeros"]),
        hp(out_host.get("w_hat")), hp(out_host.get("loss")), _ptr(dev_ws), dev_ws.numel(), _stream()),
        "tb_quantize_from_host")


class ProjectionJob(ctypes.Structure):
    """tb_projection_job"""
    _fields_ = ([("desc", LayerDesc)] +
                [(n, ctypes.c_void_p) for n in ("W", "H_in", "U_in", "H_out", "U_out", "R", "P", "C", "codes", "scales",
                                                "zeros", "cand", "W_hat", "W_comp", "loss", "stats", "ws")] +
                [("ws_bytes", ctypes.c_size_t)])


class AttentionDesc(ctypes.Structure):
    """tb_attention_desc"""
    _fields_ = [("d_model", ctypes.c_int), ("n_q_heads", ctypes.c_int), ("n_kv_heads", ctypes.c_int),
                ("d_head", ctypes.c_int), ("bits", ctypes.c_int), ("quant_group", ctypes.c_int),
                ("out_block", ctypes.c_int), ("n_cand", ctypes.c_int), ("cd_iters", ctypes.c_int),
                ("flags", ctypes.c_uint), ("n_tok", ctypes.c_longlong), ("damp", ctypes.c_float),
                ("alpha", ctypes.c_float), ("on_host", ctypes.c_int), ("concurrent", ctypes.c_int)]


class AttentionIO(ctypes.Structure):
    """tb_attention_io"""
    _fields_ = [("X", ctypes.c_void_p), ("X_fp", ctypes.c_void_p), ("X_v", ctypes.c_void_p), ("X_o", ctypes.c_void_p),
                ("X_o_fp", ctypes.c_void_p), ("W", ctypes.c_void_p * 4), ("codes", ctypes.c_void_p * 4),
                ("scales", ctypes.c_void_p * 4), ("zeros", ctypes.c_void_p * 4), ("W_hat", ctypes.c_void_p * 4),
                ("loss", ctypes.c_void_p * 4), ("info", ctypes.c_void_p)]


def attention_desc(d_model, n_q_heads, n_kv_heads, d_head, bits, quant_group, out_block, n_tok, n_cand=16, cd_iters=1,
                   flags=0, damp=0.01, alpha=0.25, on_host=False, concurrent=True) -> AttentionDesc:
    return AttentionDesc(d_model, n_q_heads, n_kv_heads, d_head, bits, quant_group, out_block, n_cand, cd_iters, flags,
                         int(n_tok), float(damp), float(alpha), int(on_host), int(concurrent))


def projection_job(desc: LayerDesc, W, H_in, U_in, H_out, U_out, R, P, C, out: "QuantizeResult", ws) -> ProjectionJob:
    """tb_projection_job from torch CUDA tensors (argument marshalling only; the caller keeps them alive)."""
    f32 = torch.float32

    def v(t, dt=None):
        q = _ptr(t, dt, True)
        return None if q is None else q.value

    return ProjectionJob(desc, v(W, f32), v(H_in, f32), v(U_in, f32), v(H_out, f32), v(U_out, f32), v(R, f32), v(P, f32),
                         v(C, f32), v(out.codes), v(out.scales), v(out.zeros), v(out.cand), v(out.w_hat),
                         v(out.w_comp, torch.float64), v(out.loss), v(out.stats), v(ws), ws.numel())


def tb_quantize_block(jobs: list, concurrent: bool = True) -> None:
    arr = (ProjectionJob * len(jobs))(*jobs)
    _check(load().tb_quantize_block(ctypes.cast(arr, ctypes.c_void_p), len(jobs), int(bool(concurrent)), _stream()),
           "tb_quantize_block")


def empty_result(desc: LayerDesc, device, want_loss=True, want_w_comp=False) -> "QuantizeResult":
    ng = desc.n_groups
    return QuantizeResult(
        codes=torch.empty((desc.d_out, desc.d_in), dtype=torch.uint8, device=device),
        scales=torch.empty((desc.d_out, ng), dtype=torch.float32, device=device),
        zeros=torch.empty((desc.d_out, ng), dtype=torch.int32, device=device),
        cand=torch.empty((desc.d_out, ng), dtype=torch.uint8, device=device),
        w_hat=torch.empty((desc.d_out, desc.d_in), dtype=torch.float32, device=device),
        loss=torch.empty(desc.n_heads, dtype=torch.float64, device=device) if want_loss else None,
        stats=torch.zeros(8, dtype=torch.int64, device=device),
        w_comp=torch.empty((desc.d_out, desc.d_in), dtype=torch.float64, device=device) if want_w_comp else None)


def attention_io(desc: AttentionDesc, X, X_o, W, out, X_fp=None, X_v=None, X_o_fp=None, info=None) -> AttentionIO:
    """tb_attention_io from torch tensors: all on the device (desc.on_host = 0) or all on the host.
    W: the four weights q, k, v, o; out: four dicts with codes, scales, zeros and optionally w_hat, loss."""
    host = bool(desc.on_host)

    def v(t):
        if t is None:
            return None
        if t.is_cuda == host or not t.is_contiguous():
            raise ValueError("tensors must be contiguous and all on the %s" % ("host" if host else "device"))
        return t.data_ptr()

    io = AttentionIO()
    io.X, io.X_fp, io.X_v, io.X_o, io.X_o_fp, io.info = v(X), v(X_fp), v(X_v), v(X_o), v(X_o_fp), v(info)
    for i in range(4):
        io.W[i] = v(W[i])
        io.codes[i], io.scales[i], io.zeros[i] = v(out[i]["codes"]), v(out[i]["scales"]), v(out[i]["zeros"])
        io.W_hat[i], io.loss[i] = v(out[i].get("w_hat")), v(out[i].get("loss"))
    return io


def attention_layer_shapes(desc: AttentionDesc):
    """(d_out, d_in, n_heads) of the q, k, v, o projections."""
    dq, dkv = desc.n_q_heads * desc.d_head, desc.n_kv_heads * desc.d_head
    return [(dq, desc.d_model, desc.n_q_heads), (dkv, desc.d_model, desc.n_kv_heads),
            (dkv, desc.d_model, desc.n_kv_heads), (desc.d_model, dq, 1)]


def attention_outputs(desc: AttentionDesc, device=None, pin=False, w_hat=True, loss=True):
    """Result buffers of tb_attention_layer, on `device` or (device None) on the host."""
    outs = []
    for d_out, d_in, heads in attention_layer_shapes(desc):
        ng = 1 if desc.quant_group == 0 else d_in // desc.quant_group
        o = {"codes": torch.empty((d_out, d_in), dtype=torch.uint8, device=device),
             "scales": torch.empty((d_out, ng), dtype=torch.float32, device=device),
             "zeros": torch.empty((d_out, ng), dtype=torch.int32, device=device)}
        if w_hat:
            o["w_hat"] = torch.empty((d_out, d_in), dtype=torch.float32, device=device)
        if loss:
            o["loss"] = torch.empty(heads, dtype=torch.float64, device=device)
        outs.append({k: (t.pin_memory() if pin else t) for k, t in o.items()})
    return outs


def tb_attention_layer_info_count(desc: AttentionDesc, per_head_v: bool) -> int:
    return int(load().tb_attention_layer_info_count(ctypes.byref(desc), int(bool(per_head_v))))


def tb_attention_layer_workspace(desc: AttentionDesc, io: AttentionIO) -> int:
    return int(load().tb_attention_layer_workspace(ctypes.byref(desc), ctypes.byref(io)))


def tb_attention_layer(desc: AttentionDesc, io: AttentionIO, ws) -> None:
    _check(load().tb_attention_layer(ctypes.byref(desc), ctypes.byref(io), _ptr(ws), ws.numel(), _stream()),
           "tb_attention_layer")


PHASES = ("setup", "grid", "sweep", "compensation", "cd", "output", "loss",
          "hessian", "cross", "hout", "factor", "prep", "copy")


def tb_pack_codes(codes, bits: int):
    """codes [d_out, d_in] uint8 -> packed int32 [d_out, d_in * bits / 32] (bit stream per row)."""
    d_out, d_in = codes.shape
    nbytes = int(load().tb_packed_bytes(d_out, d_in, bits))
    if nbytes == 0:
        raise ValueError("unsupported shape or bit width for packing")
    packed = torch.empty((d_out, nbytes // (4 * d_out)), dtype=torch.int32, device=codes.device)
    _check(load().tb_pack_codes(_ptr(codes, torch.uint8), d_out, d_in, bits, _ptr(packed), _stream()), "tb_pack_codes")
    return packed


def tb_unpack_dequant(packed, scales, zeros, d_in: int, bits: int, quant_group: int, want_codes=True, want_w_hat=True,
                      codes_ref=None, w_hat_ref=None, tol: float = 2.0 ** -22):
    """Returns (codes, w_hat, mismatch): mismatch is None without a reference, else an int64 tensor
    [code mismatches, values beyond tol]."""
    d_out = packed.shape[0]
    dev = packed.device
    codes = torch.empty((d_out, d_in), dtype=torch.uint8, device=dev) if want_codes else None
    w_hat = torch.empty((d_out, d_in), dtype=torch.float32, device=dev) if want_w_hat else None
    mism = torch.zeros(2, dtype=torch.int64, device=dev) if (codes_ref is not None or w_hat_ref is not None) else None
    _check(load().tb_unpack_dequant(_ptr(packed, torch.int32), _ptr(scales, torch.float32), _ptr(zeros, torch.int32),
                                    d_out, d_in, bits, quant_group, _ptr(codes, None, True), _ptr(w_hat, None, True),
                                    _ptr(codes_ref, torch.uint8, True), _ptr(w_hat_ref, torch.float32, True), float(tol),
                                    _ptr(mism, None, True), _stream()), "tb_unpack_dequant")
    return codes, w_hat, mism


def tb_launch_count() -> int:
    return int(load().tb_launch_count())


def tb_profile_enable(on: bool) -> None:
    load().tb_profile_enable(int(bool(on)))


def tb_profile_read() -> dict:
    """Milliseconds per phase of the tb_quantize_layer calls since tb_profile_enable(True)."""
    buf = (ctypes.c_double * len(PHASES))()
    load().tb_profile_read(buf, len(PHASES))
    return dict(zip(PHASES, [float(v) for v in buf]))
