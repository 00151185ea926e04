"""ctypes binding of libtcmoe.so: the same entry points as include/tcmoe.h.

Argument marshalling only - every step of the path runs in the library's CUDA
kernels.  PyTorch supplies device memory and streams.  There is no fallback:
if the shared library is missing or cannot be loaded, importing a function from
here raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

from .synth import MoEConfig

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtcmoe.so")

MOE_OK = 0
MOE_ERR_INVALID_ARG = -1
MOE_ERR_UNSUPPORTED_SHAPE = -2
MOE_ERR_WORKSPACE_TOO_SMALL = -3
MOE_ERR_MISALIGNED = -4
MOE_ERR_CUDA = -5
MOE_ERR_SCRATCH_LIMIT = -6
MOE_NOALLOC_SCRATCH_BYTES = 2 << 20
MOE_DEV_TIMEOUT = 1
MOE_DEV_INDEX_OUT_OF_RANGE = 2
MOE_WARN_NONFINITE_LOGIT = 1
MOE_FLAG_WEIGHT_IN_COMBINE = 1
MOE_FLAG_COMBINE_IN_EPILOGUE = 2
MOE_FLAG_SPARSE_TOPK = 4
MOE_FLAG_FUSED_FFN = 8
MOE_FLAG_SM_PARTITION = 16
MOE_FLAG_GEMM2_PAIR = 32
MOE_FLAG_GEMM2_SINGLE = 64
MOE_FLAG_GEMM1_PAIR = 128
MOE_FLAG_TRACK_DISPATCH = 256
MOE_FLAG_GEMM1_GATHER = 512

EXPORTS = ("moe_workspace_bytes", "moe_workspace_layout", "moe_status_reset", "moe_status", "moe_strerror",
           "moe_route", "moe_dispatch", "moe_expert_ffn", "moe_combine", "moe_layer", "moe_layer_host",
           "moe_profile_enable", "moe_profile_read", "moe_dispatch_noalloc", "moe_quantize_rows",
           "moe_quantize_weights", "moe_expert_ffn_fp8", "moe_layer_fp8", "moe_layer_fp8_host", "moe_selftest_wait_timeout", "moe_traffic_stats", "moe_ep_pack", "moe_ep_finish",
           "moe_payload_efficiency", "moe_backward_workspace_bytes", "moe_layer_backward", "moe_clear_cache", "moe_gate_backward")


class MoEShape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("T", "d", "f", "E", "k", "G", "score_fn", "flags")]


class MoELayoutC(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("expert_counts", "expert_offsets", "group_counts", "group_offsets", "pair_row", "row_pair",
                 "al", "disp_token", "row_src")]


class MoEError(RuntimeError):
    def __init__(self, fn: str, code: int):
        self.code = code
        super().__init__(f"{fn} failed: {code} ({strerror(code)})")


_lib_handle = None


def lib() -> ctypes.CDLL:
    """Load the C-ABI library (built in-tree by paper_2605_05607_b200.build)."""
    global _lib_handle
    if _lib_handle is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2605_05607_b200.build` "
                               "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i64, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t
        shp, lay = ctypes.POINTER(MoEShape), ctypes.POINTER(MoELayoutC)
        L.moe_workspace_bytes.argtypes = [shp, ctypes.POINTER(sz)]
        L.moe_workspace_layout.argtypes = [shp, ctypes.POINTER(sz)]
        L.moe_status_reset.argtypes = [vp, vp]
        L.moe_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int32), vp]
        L.moe_strerror.argtypes = [ctypes.c_int]
        L.moe_strerror.restype = ctypes.c_char_p
        L.moe_route.argtypes = [shp, vp, vp, vp, i64, vp, vp, vp, vp, sz, vp]
        L.moe_dispatch.argtypes = [shp, vp, vp, lay, vp, vp, sz, vp]
        L.moe_expert_ffn.argtypes = [shp, vp, lay, vp, vp, vp, vp, vp, vp, sz, vp]
        L.moe_combine.argtypes = [shp, vp, lay, vp, vp, vp, vp, vp, sz, vp]
        L.moe_layer.argtypes = [shp, vp, vp, vp, i64, vp, vp, vp, vp, vp, vp, vp, lay, vp, sz, vp]
        L.moe_layer_host.argtypes = [shp, vp, vp, vp, vp, i64, vp, vp, vp, vp, vp, vp, sz, vp]
        L.moe_dispatch_noalloc.argtypes = [shp, vp, vp, lay, vp, vp, vp]
        L.moe_quantize_rows.argtypes = [vp, i64, i64, vp, vp, vp]
        L.moe_quantize_weights.argtypes = [vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, vp, vp, vp]
        L.moe_expert_ffn_fp8.argtypes = [shp, vp, vp, lay, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.moe_layer_fp8.argtypes = [shp, vp, vp, vp, i64, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, lay, vp, sz, vp]
        L.moe_layer_fp8_host.argtypes = [shp, vp, vp, vp, vp, i64, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.moe_selftest_wait_timeout.argtypes = [vp, ctypes.c_uint64, vp]
        L.moe_traffic_stats.argtypes = [shp, lay, ctypes.POINTER(ctypes.c_double), vp]
        L.moe_payload_efficiency.argtypes = [i64, ctypes.c_int32, ctypes.POINTER(ctypes.c_double)]
        L.moe_backward_workspace_bytes.argtypes = [shp, ctypes.POINTER(sz)]
        L.moe_layer_backward.argtypes = [shp, vp, vp, vp, vp, lay, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.moe_gate_backward.argtypes = [shp, vp, vp, i64, vp, vp, lay, vp, vp, vp, vp, sz, vp]
        L.moe_ep_pack.argtypes = [shp, vp, vp, lay, vp, vp, vp]
        L.moe_ep_finish.argtypes = [shp, vp, lay, vp, vp]
        L.moe_profile_enable.argtypes = [ctypes.c_int]
        L.moe_profile_read.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32)]
        for name in EXPORTS:
            if name != "moe_strerror":
                getattr(L, name).restype = ctypes.c_int
        _lib_handle = L
    return _lib_handle


def make_shape(cfg: MoEConfig, flags: int = 0) -> MoEShape:
    return MoEShape(cfg.T, cfg.d, cfg.f, cfg.E, cfg.k, cfg.G, cfg.score_fn, flags)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous(), "tensors passed to the C ABI must be contiguous"
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream() if torch.cuda.is_available() else None
    return None if stream is None else stream.cuda_stream


def _check(fn: str, rc: int) -> None:
    if rc != MOE_OK:
        raise MoEError(fn, rc)


def strerror(code: int) -> str:
    return lib().moe_strerror(code).decode()


@dataclass
class Layout:
    """Device int32 tensors of moe_layout_t."""
    expert_counts: torch.Tensor
    expert_offsets: torch.Tensor
    group_counts: torch.Tensor
    group_offsets: torch.Tensor
    pair_row: torch.Tensor
    row_pair: torch.Tensor
    al: torch.Tensor
    disp_token: torch.Tensor
    row_src: torch.Tensor

    def c(self) -> MoELayoutC:
        return MoELayoutC(*[getattr(self, n).data_ptr() for n, _ in MoELayoutC._fields_])


def alloc_layout(shape: MoEShape, device="cuda") -> Layout:
    T, E, k, G = shape.T, shape.E, shape.k, shape.G
    z = lambda n: torch.zeros(max(n, 4), dtype=torch.int32, device=device)
    return Layout(z(E), z(E + 1), z(G), z(G + 1), z(T * k), z(T * k), z(G * T), z(T * min(k, G)), z(T * k))


def moe_workspace_bytes(shape: MoEShape) -> int:
    out = ctypes.c_size_t(0)
    _check("moe_workspace_bytes", lib().moe_workspace_bytes(ctypes.byref(shape), ctypes.byref(out)))
    return out.value


def moe_workspace_layout(shape: MoEShape) -> dict:
    out = (ctypes.c_size_t * 4)()
    _check("moe_workspace_layout", lib().moe_workspace_layout(ctypes.byref(shape), out))
    return {"status": out[0], "h": out[1], "o": out[2], "mt_prefix": out[3]}


def alloc_workspace(shape: MoEShape, device="cuda") -> torch.Tensor:
    """Zero-filled workspace (the status block must start at zero)."""
    return torch.zeros(moe_workspace_bytes(shape), dtype=torch.uint8, device=device)


def moe_status_reset(ws: torch.Tensor, stream=None) -> None:
    _check("moe_status_reset", lib().moe_status_reset(_ptr(ws), _stream(stream)))


def moe_status(ws: torch.Tensor, stream=None) -> list:
    out = (ctypes.c_int32 * 8)()
    _check("moe_status", lib().moe_status(_ptr(ws), out, _stream(stream)))
    return list(out)


def moe_route(shape, x, w_gate, logit_bias, logits, topk_idx, topk_w, ws, stream=None) -> None:
    stride = 0 if logit_bias is None or logit_bias.dim() == 1 else shape.E
    _check("moe_route", lib().moe_route(ctypes.byref(shape), _ptr(x), _ptr(w_gate), _ptr(logit_bias), stride,
                                        _ptr(logits), _ptr(topk_idx), _ptr(topk_w), _ptr(ws), ws.numel(),
                                        _stream(stream)))


def moe_dispatch(shape, x, topk_idx, layout: Layout, xg, ws, stream=None) -> None:
    c = layout.c()
    _check("moe_dispatch", lib().moe_dispatch(ctypes.byref(shape), _ptr(x), _ptr(topk_idx), ctypes.byref(c),
                                              _ptr(xg), _ptr(ws), ws.numel(), _stream(stream)))


def moe_dispatch_noalloc(shape, x, topk_idx, layout: Layout, xg, status_out=None, stream=None) -> None:
    """moe_dispatch for callers that cannot pass a workspace (plugins inside a pre-planned memory
    arena, allocation-free serving loops): the scratch tables live in a fixed array inside the
    library.  Shapes beyond MOE_NOALLOC_SCRATCH_BYTES raise MoEError(MOE_ERR_SCRATCH_LIMIT).  Calls
    on one device share that array, so keep them ordered on one stream."""
    c = layout.c()
    _check("moe_dispatch_noalloc", lib().moe_dispatch_noalloc(ctypes.byref(shape), _ptr(x), _ptr(topk_idx),
                                                              ctypes.byref(c), _ptr(xg), _ptr(status_out),
                                                              _stream(stream)))


def moe_expert_ffn(shape, xg, layout: Layout, topk_w, w1, w3, w2, o, ws, stream=None) -> None:
    c = layout.c()
    _check("moe_expert_ffn", lib().moe_expert_ffn(ctypes.byref(shape), _ptr(xg), ctypes.byref(c), _ptr(topk_w),
                                                  _ptr(w1), _ptr(w3), _ptr(w2), _ptr(o), _ptr(ws), ws.numel(),
                                                  _stream(stream)))


def moe_quantize_rows(src, dst, scale, stream=None) -> None:
    """src bf16 [rows, cols] -> dst uint8 [rows, cols] (E4M3 codes), scale fp32 [rows]."""
    rows, cols = src.shape
    _check("moe_quantize_rows", lib().moe_quantize_rows(_ptr(src), ctypes.c_int64(rows), ctypes.c_int64(cols),
                                                        _ptr(dst), _ptr(scale), _stream(stream)))


def moe_quantize_weights(w, wq, scale, stream=None) -> None:
    """w bf16 [E, K, N] -> wq uint8 [E, N, K] (E4M3 codes, K contiguous), scale fp32 [E, N]."""
    E, K, N = w.shape
    _check("moe_quantize_weights", lib().moe_quantize_weights(_ptr(w), E, K, N, _ptr(wq), _ptr(scale),
                                                              _stream(stream)))


def moe_expert_ffn_fp8(shape, xq, sx, layout: Layout, topk_w, w1q, s1, w3q, s3, w2q, s2, o, ws, stream=None) -> None:
    c = layout.c()
    _check("moe_expert_ffn_fp8", lib().moe_expert_ffn_fp8(ctypes.byref(shape), _ptr(xq), _ptr(sx), ctypes.byref(c),
                                                          _ptr(topk_w), _ptr(w1q), _ptr(s1), _ptr(w3q), _ptr(s3),
                                                          _ptr(w2q), _ptr(s2), _ptr(o), _ptr(ws), ws.numel(),
                                                          _stream(stream)))


def moe_layer_fp8(shape, x, w_gate, logit_bias, w1q, s1, w3q, s3, w2q, s2, y, ws, logits=None, topk_idx=None,
                  topk_w=None, layout: Optional[Layout] = None, stream=None) -> None:
    stride = 0 if logit_bias is None or logit_bias.dim() == 1 else shape.E
    c = layout.c() if layout is not None else None
    _check("moe_layer_fp8", lib().moe_layer_fp8(ctypes.byref(shape), _ptr(x), _ptr(w_gate), _ptr(logit_bias), stride,
                                                _ptr(w1q), _ptr(s1), _ptr(w3q), _ptr(s3), _ptr(w2q), _ptr(s2),
                                                _ptr(y), _ptr(logits), _ptr(topk_idx), _ptr(topk_w),
                                                ctypes.byref(c) if c is not None else None, _ptr(ws), ws.numel(),
                                                _stream(stream)))


def moe_layer_fp8_host(shape, x_host, x_dev, w_gate, logit_bias, w1q, s1, w3q, s3, w2q, s2, y_dev, y_host, ws,
                       stream=None) -> None:
    stride = 0 if logit_bias is None or logit_bias.dim() == 1 else shape.E
    _check("moe_layer_fp8_host", lib().moe_layer_fp8_host(ctypes.byref(shape), _ptr(x_host), _ptr(x_dev), _ptr(w_gate),
                                                          _ptr(logit_bias), stride, _ptr(w1q), _ptr(s1), _ptr(w3q),
                                                          _ptr(s3), _ptr(w2q), _ptr(s2), _ptr(y_dev), _ptr(y_host),
                                                          _ptr(ws), ws.numel(), _stream(stream)))


def moe_ep_pack(shape, topk_idx, topk_w, layout: Layout, send_idx, send_w, stream=None) -> None:
    c = layout.c()
    _check("moe_ep_pack", lib().moe_ep_pack(ctypes.byref(shape), _ptr(topk_idx), _ptr(topk_w), ctypes.byref(c),
                                            _ptr(send_idx), _ptr(send_w), _stream(stream)))


def moe_ep_finish(shape, back, layout: Layout, y, stream=None) -> None:
    c = layout.c()
    _check("moe_ep_finish", lib().moe_ep_finish(ctypes.byref(shape), _ptr(back), ctypes.byref(c), _ptr(y),
                                                _stream(stream)))


def moe_traffic_stats(shape, layout: Layout, stream=None) -> dict:
    c = layout.c()
    out = (ctypes.c_double * 8)()
    _check("moe_traffic_stats", lib().moe_traffic_stats(ctypes.byref(shape), ctypes.byref(c), out, _stream(stream)))
    names = ("T", "P", "n_disp", "D", "dedup", "allgather_useless", "redundant_share", "ideal_speedup")
    return dict(zip(names, list(out)))


def moe_payload_efficiency(transfer_bytes: int, n_targets: int) -> dict:
    out = (ctypes.c_double * 4)()
    _check("moe_payload_efficiency", lib().moe_payload_efficiency(transfer_bytes, n_targets, out))
    return dict(zip(("data_flits", "ideal", "explicit", "dynamic"), list(out)))


def moe_backward_workspace_bytes(shape: MoEShape) -> int:
    out = ctypes.c_size_t(0)
    _check("moe_backward_workspace_bytes", lib().moe_backward_workspace_bytes(ctypes.byref(shape), ctypes.byref(out)))
    return out.value


def moe_layer_backward(shape, x, dy, topk_idx, topk_w, layout: Layout, w1, w3, w2, dx, dw1, dw3, dw2, ws,
                       stream=None) -> None:
    c = layout.c()
    _check("moe_layer_backward", lib().moe_layer_backward(ctypes.byref(shape), _ptr(x), _ptr(dy), _ptr(topk_idx),
                                                          _ptr(topk_w), ctypes.byref(c), _ptr(w1), _ptr(w3), _ptr(w2),
                                                          _ptr(dx), _ptr(dw1), _ptr(dw3), _ptr(dw2), _ptr(ws),
                                                          ws.numel(), _stream(stream)))


def moe_gate_backward(shape, logits, logit_bias, topk_idx, topk_w, layout: Layout, w_gate, dx, dw_gate, ws,
                      stream=None) -> None:
    """Gate gradient after moe_layer_backward on the same backward workspace: adds the gate path to dx, writes dw_gate."""
    stride = 0 if logit_bias is None or logit_bias.dim() == 1 else shape.E
    c = layout.c()
    _check("moe_gate_backward", lib().moe_gate_backward(ctypes.byref(shape), _ptr(logits), _ptr(logit_bias), stride,
                                                        _ptr(topk_idx), _ptr(topk_w), ctypes.byref(c), _ptr(w_gate),
                                                        _ptr(dx), _ptr(dw_gate), _ptr(ws), ws.numel(), _stream(stream)))


def moe_selftest_wait_timeout(ws, limit_ns: int, stream=None) -> None:
    _check("moe_selftest_wait_timeout", lib().moe_selftest_wait_timeout(_ptr(ws), limit_ns, _stream(stream)))


def moe_combine(shape, o, layout: Layout, topk_idx, topk_w, pg, y, ws, stream=None) -> None:
    c = layout.c()
    _check("moe_combine", lib().moe_combine(ctypes.byref(shape), _ptr(o), ctypes.byref(c), _ptr(topk_idx),
                                            _ptr(topk_w), _ptr(pg), _ptr(y), _ptr(ws), ws.numel(), _stream(stream)))


def moe_layer(shape, x, w_gate, logit_bias, w1, w3, w2, y, ws, logits=None, topk_idx=None, topk_w=None,
              layout: Optional[Layout] = None, stream=None) -> None:
    stride = 0 if logit_bias is None or logit_bias.dim() == 1 else shape.E
    c = layout.c() if layout is not None else None
    _check("moe_layer", lib().moe_layer(ctypes.byref(shape), _ptr(x), _ptr(w_gate), _ptr(logit_bias), stride,
                                        _ptr(w1), _ptr(w3), _ptr(w2), _ptr(y), _ptr(logits), _ptr(topk_idx),
                                        _ptr(topk_w), ctypes.byref(c) if c is not None else None, _ptr(ws),
                                        ws.numel(), _stream(stream)))


def moe_layer_host(shape, x_host, x_dev, w_gate, logit_bias, w1, w3, w2, y_dev, y_host, ws, stream=None) -> None:
    stride = 0 if logit_bias is None or logit_bias.dim() == 1 else shape.E
    _check("moe_layer_host", lib().moe_layer_host(ctypes.byref(shape), _ptr(x_host), _ptr(x_dev), _ptr(w_gate),
                                                  _ptr(logit_bias), stride, _ptr(w1), _ptr(w3), _ptr(w2),
                                                  _ptr(y_dev), _ptr(y_host), _ptr(ws), ws.numel(), _stream(stream)))


KERNEL_IDS = {"topk": 1, "masks": 2, "fill": 3, "dispatch": 4, "gemm1": 5, "gemm2": 6, "combine": 7, "gate": 8,
              "wgrad": 10, "bwd_gather": 11, "gate_bwd": 12}


def moe_profile_enable(kernel_id: int) -> None:
    _check("moe_profile_enable", lib().moe_profile_enable(kernel_id))


def moe_clear_cache() -> None:
    """Forget the cached TMA tensor maps (host memory only)."""
    _check("moe_clear_cache", lib().moe_clear_cache())


def moe_profile_read():
    """(total device milliseconds, launches) of the profiled kernel since the last read."""
    ms, n = ctypes.c_float(0), ctypes.c_int32(0)
    _check("moe_profile_read", lib().moe_profile_read(ctypes.byref(ms), ctypes.byref(n)))
    return ms.value, n.value
