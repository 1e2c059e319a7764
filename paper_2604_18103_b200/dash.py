"""Thin ctypes binding over the C-ABI CUDA library (include/dash.h).

Argument marshalling only: every step of the path runs in the library's
kernels.  Tensors are torch CUDA tensors (torch provides device memory and the
current stream); the only tensor operations here move data (concatenating the
Q | K | V and gate | up weight matrices, copies to the device) -- no arithmetic.  If the library cannot be
loaded the import of a symbol raises -- there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import (POINTER, Structure, c_char_p, c_double, c_float, c_int, c_int32, c_int64,
                    c_size_t, c_uint8, c_void_p)
from typing import Optional, Sequence

import torch

F32, BF16 = 0, 1
NORM_REL, NORM_ABS = 0, 1
SEL_THRESHOLD, SEL_KEEP_COUNT, SEL_THRESHOLD_HALT_HIGH, SEL_KEEP_COUNT_HALT_HIGH = 0, 1, 2, 3
SIGNAL_ATTN, SIGNAL_BLOCK = 0, 1
WS_COMPACT, WS_ATTENTION, WS_DECODE = 1, 2, 3
OK = 0

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdash.so")

EXPORTS = [
    "dash_status_string", "dash_check_status", "dash_keep_count", "dash_flops_per_layer", "dash_flops_speedup",
    "dash_delta_norm", "dash_select", "dash_compact", "dash_scatter", "dash_varlen_attention",
    "dash_layer_workspace", "dash_layer_step", "dash_workspace_bytes", "dash_compact_static",
    "dash_block_workspace", "dash_block_step", "dash_decode_attention", "dash_varlen_attention_indexed",
    "dash_keep_counts_device", "dash_fold_norm_weight", "dash_rope_table",
]
TEST_HOOKS = ["dash_testing_compact_stalled"]        # include/dash_testing.h
COMPACT_STATIC_MAX_ROWS = 1 << 20


class Threshold(Structure):
    _fields_ = [("tau", c_float), ("keep_first", c_int), ("keep_last", c_int),
                ("cu_seqlens", c_void_p), ("S", c_int), ("mask_out", c_void_p)]


class Rows(Structure):
    _fields_ = [("src", c_void_p), ("dst", c_void_p), ("row_bytes", c_int64),
                ("src_ld_bytes", c_int64), ("dst_ld_bytes", c_int64)]


class LayerCfg(Structure):
    _fields_ = [("d", c_int), ("Hq", c_int), ("Hkv", c_int), ("D", c_int), ("dt", c_int),
                ("Wqkv", c_void_p), ("Wo", c_void_p), ("rms_weight", c_void_p), ("rms_eps", c_float),
                ("rope_base", c_double), ("norm_mode", c_int), ("norm_eps", c_float), ("sel_mode", c_int),
                ("tau", c_float), ("keep_counts", c_void_p), ("keep_first", c_int), ("keep_last", c_int),
                ("scatter_which", c_int), ("k_cache", c_void_p), ("v_cache", c_void_p), ("rms_folded", c_int),
                ("rope_table", c_void_p), ("rope_table_len", c_int64), ("inv_rms_in", c_void_p), ("inv_rms_next", c_void_p)]


class LayerWsLayout(Structure):
    _fields_ = [("Hn", c_size_t), ("QKV", c_size_t), ("O", c_size_t), ("U", c_size_t), ("Ht", c_size_t),
                ("scratch", c_size_t), ("total", c_size_t)]


class BlockCfg(Structure):
    _fields_ = [("attn", LayerCfg), ("m", c_int), ("Wgu", c_void_p), ("Wd", c_void_p), ("rms2_weight", c_void_p), ("signal", c_int), ("rms2_folded", c_int)]


class BlockWsLayout(Structure):
    _fields_ = [("attn", LayerWsLayout), ("GU", c_size_t), ("ACT", c_size_t), ("F", c_size_t), ("total", c_size_t)]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libdash.so (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2604_18103_b200.build` "
                               "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        L.dash_status_string.restype = c_char_p
        L.dash_status_string.argtypes = [c_int]
        L.dash_check_status.argtypes = [c_void_p]
        L.dash_keep_count.restype = c_int64
        L.dash_keep_count.argtypes = [c_int64, c_double, c_int, c_int, c_int]
        L.dash_flops_per_layer.restype = c_double
        L.dash_flops_per_layer.argtypes = [c_double] * 3
        L.dash_flops_speedup.restype = c_double
        L.dash_flops_speedup.argtypes = [c_double, c_double, c_int, c_int, c_double, c_double]
        L.dash_delta_norm.argtypes = [c_void_p, c_void_p, c_int64, c_int, c_int64, c_int64, c_int, c_int, c_float,
                                      c_void_p, c_void_p, c_int64, c_void_p, POINTER(Threshold), c_void_p, c_void_p]
        L.dash_select.argtypes = [c_void_p, c_int64, c_void_p, c_int, c_int, c_float, c_void_p, c_int, c_int,
                                  c_void_p, c_void_p]
        L.dash_compact.argtypes = [c_void_p, c_int64, c_void_p, c_int, POINTER(Rows), c_int, c_void_p, c_void_p,
                                   c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
        L.dash_compact_static.argtypes = [c_void_p, c_int64, c_void_p, c_int, POINTER(Rows), c_int, c_void_p, c_void_p,
                                          c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
        L.dash_scatter.argtypes = [c_void_p, c_int64, c_int64, c_int64, c_void_p, c_void_p, c_int, c_void_p,
                                   c_void_p, c_int64, c_void_p]
        L.dash_varlen_attention.argtypes = [c_void_p] * 5 + [c_int64] * 4 + [c_void_p, c_int, c_int64, c_int64,
                                                                          c_int, c_int, c_int, c_float, c_int, c_int,
                                                                          c_void_p, c_size_t, c_void_p]
        L.dash_varlen_attention_indexed.argtypes = [c_void_p] * 5 + [c_int64] * 4 + [c_void_p, c_int64, c_int, c_void_p, c_int, c_int64, c_int64,
                                                                                  c_int, c_int, c_int, c_float, c_int, c_int,
                                                                                  c_void_p, c_size_t, c_void_p]
        L.dash_keep_counts_device.argtypes = [c_void_p, c_int, c_double, c_int, c_int, c_int, c_void_p, c_void_p]
        L.dash_fold_norm_weight.argtypes = [c_void_p, c_void_p, c_int, c_int64, c_int64, c_int, c_void_p, c_int64, c_void_p]
        L.dash_rope_table.argtypes = [c_double, c_int, c_int64, c_void_p, c_void_p]
        L.dash_layer_workspace.argtypes = [POINTER(LayerCfg), c_int64, c_int, POINTER(LayerWsLayout)]
        L.dash_layer_step.argtypes = [POINTER(LayerCfg), c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_int64, c_int64,
                                      c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                      c_void_p, c_size_t, c_void_p]
        L.dash_decode_attention.argtypes = [c_void_p] * 5 + [c_int64] * 4 + [c_void_p, c_int, c_int64, c_int, c_int, c_int, c_float, c_int,
                                                                          c_void_p, c_size_t, c_void_p]
        L.dash_block_workspace.argtypes = [POINTER(BlockCfg), c_int64, c_int, POINTER(BlockWsLayout)]
        L.dash_block_step.argtypes = [POINTER(BlockCfg), c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_int64, c_int64,
                                      c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                      c_void_p, c_size_t, c_void_p]
        L.dash_testing_compact_stalled.argtypes = [c_void_p, c_int64, c_void_p, c_int, c_void_p, c_void_p, c_void_p, ctypes.c_uint32,
                                                   c_void_p, c_size_t, c_void_p]
        L.dash_workspace_bytes.restype = c_size_t
        L.dash_workspace_bytes.argtypes = [c_int, c_int64, c_int, c_int, c_int, c_int, c_int]
        _lib = L
    return _lib


class DashError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib().dash_status_string(status).decode()} (status {status})")


def _check(status: int, where: str):
    if status != OK:
        raise DashError(status, where)


def _p(t: Optional[torch.Tensor]):
    return None if t is None else c_void_p(t.data_ptr())


def _stream():
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise TypeError(f"unsupported dtype {t.dtype}")


def _dev(t: torch.Tensor, *more):
    for x in (t, *more):
        if x is not None and not x.is_cuda:
            raise ValueError("device tensor expected")


# ---- host helpers -------------------------------------------------------------
def dash_keep_count(n: int, rho: float, keep_first: int = 0, keep_last: int = 0, mode: int = 0) -> int:
    return int(lib().dash_keep_count(n, rho, keep_first, keep_last, mode))


def dash_flops_per_layer(n, d, m) -> float:
    return float(lib().dash_flops_per_layer(n, d, m))


def dash_flops_speedup(n, n_hat, L, l_s, d, m) -> float:
    return float(lib().dash_flops_speedup(n, n_hat, L, l_s, d, m))


def dash_check_status() -> int:
    return int(lib().dash_check_status(_stream()))


def dash_workspace_bytes(op: int, n: int, S: int = 1, Hq: int = 0, Hkv: int = 0, D: int = 0, dt: int = BF16) -> int:
    return int(lib().dash_workspace_bytes(op, n, S, Hq, Hkv, D, dt))


def workspace(nbytes: int, device) -> torch.Tensor:
    """256-byte aligned scratch buffer (torch's caching allocator aligns to 512)."""
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


# ---- step 1 ---------------------------------------------------------------------
def dash_delta_norm(U: torch.Tensor, H: Optional[torch.Tensor], mode: int = NORM_REL, eps: float = 1e-12,
                    r_out: Optional[torch.Tensor] = None, Hres_out: Optional[torch.Tensor] = None,
                    res_index: Optional[torch.Tensor] = None, tau: Optional[float] = None,
                    cu_seqlens: Optional[torch.Tensor] = None, keep_first: int = 0, keep_last: int = 0,
                    mask_out: Optional[torch.Tensor] = None, n_dev: Optional[torch.Tensor] = None) -> torch.Tensor:
    _dev(U, H, r_out, Hres_out)
    n, d = U.shape
    if r_out is None:
        r_out = torch.empty(n, dtype=torch.float32, device=U.device)
    fused = None
    if mask_out is not None:
        fused = Threshold(float(tau), keep_first, keep_last, cu_seqlens.data_ptr(), cu_seqlens.numel() - 1, mask_out.data_ptr())
    st = lib().dash_delta_norm(_p(U), _p(H), n, d, U.stride(0), H.stride(0) if H is not None else d, dtype_code(U), mode, eps,
                               _p(r_out), _p(Hres_out), Hres_out.stride(0) if Hres_out is not None else d, _p(res_index),
                               ctypes.byref(fused) if fused is not None else None, _p(n_dev), _stream())
    _check(st, "dash_delta_norm")
    return r_out


# ---- step 2 ---------------------------------------------------------------------
def dash_select(r: torch.Tensor, cu_seqlens: torch.Tensor, mode: int, tau: float = 0.0,
                keep_counts: Optional[torch.Tensor] = None, keep_first: int = 0, keep_last: int = 0,
                mask_out: Optional[torch.Tensor] = None) -> torch.Tensor:
    _dev(r, cu_seqlens, keep_counts)
    n = r.numel()
    if mask_out is None:
        mask_out = torch.empty(n, dtype=torch.uint8, device=r.device)
    st = lib().dash_select(_p(r), n, _p(cu_seqlens), cu_seqlens.numel() - 1, mode, tau, _p(keep_counts), keep_first, keep_last,
                           _p(mask_out), _stream())
    _check(st, "dash_select")
    return mask_out


def dash_keep_counts_device(cu_seqlens: torch.Tensor, rho: float, keep_first: int = 0, keep_last: int = 0, mode: int = 0,
                            out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Kept length of every sequence (int32 [S], on the device) from the lengths in cu_seqlens: no host round trip."""
    _dev(cu_seqlens)
    S = cu_seqlens.numel() - 1
    if out is None:
        out = torch.empty(S, dtype=torch.int32, device=cu_seqlens.device)
    st = lib().dash_keep_counts_device(_p(cu_seqlens), S, float(rho), keep_first, keep_last, mode, _p(out), _stream())
    _check(st, "dash_keep_counts_device")
    return out


# ---- step 3 ---------------------------------------------------------------------
def dash_compact(mask: torch.Tensor, cu_in: torch.Tensor, rows: Sequence[torch.Tensor] = (),
                 rows_out: Optional[Sequence[torch.Tensor]] = None, pos_in: Optional[torch.Tensor] = None,
                 tok_in: Optional[torch.Tensor] = None, want_idx: bool = True, ws: Optional[torch.Tensor] = None,
                 outputs: Optional[dict] = None, static_scratch: bool = False):
    """Returns dict(idx, cu_out, n_out (device int32 [1]), rows (list), pos_out, tok_out); outputs are sized n.

    `outputs` may hand in preallocated idx / pos_out / tok_out / cu_out / n_out tensors.  With
    static_scratch=True the call goes to dash_compact_static, the entry point for callers that
    must not allocate: it takes no workspace and uses the library's fixed scratch array."""
    _dev(mask, cu_in)
    n = mask.numel()
    S = cu_in.numel() - 1
    dev = mask.device
    if rows_out is None:
        rows_out = [torch.empty_like(x) for x in rows]
    arr = (Rows * max(len(rows), 1))()
    for i, (x, y) in enumerate(zip(rows, rows_out)):
        rb = x.shape[1] * x.element_size() if x.dim() > 1 else x.element_size()
        rb = int(x[0].numel() * x.element_size()) if x.shape[0] > 0 else rb
        arr[i] = Rows(x.data_ptr(), y.data_ptr(), rb, x.stride(0) * x.element_size(), y.stride(0) * y.element_size())
    o = outputs or {}
    idx = o.get("idx", torch.empty(n, dtype=torch.int32, device=dev) if want_idx else None)
    pos_out = o.get("pos_out", torch.empty(n, dtype=torch.int32, device=dev) if pos_in is not None else None)
    tok_out = o.get("tok_out", torch.empty(n, dtype=torch.int32, device=dev) if tok_in is not None else None)
    cu_out = o.get("cu_out", torch.empty(S + 1, dtype=torch.int32, device=dev))
    n_out = o.get("n_out", torch.empty(1, dtype=torch.int32, device=dev))
    if static_scratch:
        st = lib().dash_compact_static(_p(mask), n, _p(cu_in), S, arr, len(rows), _p(pos_in), _p(pos_out), _p(tok_in),
                                       _p(tok_out), _p(idx), _p(cu_out), _p(n_out), _stream())
        _check(st, "dash_compact_static")
        return {"idx": idx, "cu_out": cu_out, "n_out": n_out, "rows": list(rows_out), "pos_out": pos_out, "tok_out": tok_out}
    if ws is None:
        ws = workspace(dash_workspace_bytes(WS_COMPACT, n, S), dev)
    st = lib().dash_compact(_p(mask), n, _p(cu_in), S, arr, len(rows), _p(pos_in), _p(pos_out), _p(tok_in), _p(tok_out),
                            _p(idx), _p(cu_out), _p(n_out), _p(ws), ws.numel(), _stream())
    _check(st, "dash_compact")
    return {"idx": idx, "cu_out": cu_out, "n_out": n_out, "rows": list(rows_out), "pos_out": pos_out, "tok_out": tok_out}


def dash_testing_compact_stalled(mask: torch.Tensor, cu_in: torch.Tensor, spin_limit: int = 1000):
    """Test hook (include/dash_testing.h): the look-back compaction with tile 0 never taken, so that a bounded device-side
    wait runs out.  Returns dict(idx, cu_out, n_out); the device status word then holds DASH_ERR_TIMEOUT."""
    _dev(mask, cu_in)
    n, S, dev = mask.numel(), cu_in.numel() - 1, mask.device
    idx = torch.zeros(n, dtype=torch.int32, device=dev)
    cu_out = torch.zeros(S + 1, dtype=torch.int32, device=dev)
    n_out = torch.zeros(1, dtype=torch.int32, device=dev)
    ws = workspace(dash_workspace_bytes(WS_COMPACT, n, S), dev)
    st = lib().dash_testing_compact_stalled(_p(mask), n, _p(cu_in), S, _p(idx), _p(cu_out), _p(n_out), int(spin_limit), _p(ws), ws.numel(), _stream())
    _check(st, "dash_testing_compact_stalled")
    return {"idx": idx, "cu_out": cu_out, "n_out": n_out}


def dash_scatter(src: torch.Tensor, dst_full: torch.Tensor, tok_index: Optional[torch.Tensor] = None,
                 sel: Optional[torch.Tensor] = None, which: int = 2, n_dev: Optional[torch.Tensor] = None) -> torch.Tensor:
    _dev(src, dst_full, tok_index, sel)
    n = src.shape[0]
    rb = int(src[0].numel() * src.element_size()) if n > 0 else 4
    st = lib().dash_scatter(_p(src), n, rb, src.stride(0) * src.element_size(), _p(tok_index), _p(sel), which, _p(n_dev),
                            _p(dst_full), dst_full.stride(0) * dst_full.element_size(), _stream())
    _check(st, "dash_scatter")
    return dst_full


# ---- step 4 ---------------------------------------------------------------------
def dash_varlen_attention(Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, cu_seqlens: torch.Tensor, max_seqlen: int,
                          scale: Optional[float] = None, O: Optional[torch.Tensor] = None, want_lse: bool = False,
                          ws: Optional[torch.Tensor] = None):
    """Q [n,Hq,D], K,V [n,Hkv,D] (last two dims contiguous).  Returns O (and lse [Hq,n] if asked)."""
    _dev(Q, K, V, cu_seqlens)
    n, Hq, D = Q.shape
    Hkv = K.shape[1]
    if scale is None:
        scale = 1.0 / (D ** 0.5)
    if O is None:
        O = torch.empty(n, Hq, D, dtype=Q.dtype, device=Q.device)
    lse = torch.empty(Hq, n, dtype=torch.float32, device=Q.device) if want_lse else None
    dt = dtype_code(Q)
    if ws is None:
        ws = workspace(dash_workspace_bytes(WS_ATTENTION, n, cu_seqlens.numel() - 1, Hq, Hkv, D, dt), Q.device)
    st = lib().dash_varlen_attention(_p(Q), _p(K), _p(V), _p(O), _p(lse), Q.stride(0), K.stride(0), V.stride(0), O.stride(0),
                                     _p(cu_seqlens), cu_seqlens.numel() - 1, n, int(max_seqlen), Hq, Hkv, D, float(scale), 1, dt,
                                     _p(ws), ws.numel(), _stream())
    _check(st, "dash_varlen_attention")
    return (O, lse) if want_lse else O


def dash_varlen_attention_indexed(Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, idx: torch.Tensor, cu_seqlens: torch.Tensor,
                                  max_seqlen: int, n: Optional[int] = None, kv_packed: bool = False, scale: Optional[float] = None,
                                  O: Optional[torch.Tensor] = None, want_lse: bool = False, ws: Optional[torch.Tensor] = None):
    """Q [n_full,Hq,D] full-length (bf16); packed row i of the active set is its row idx[i].  K, V: packed [n,Hkv,D]
    (kv_packed=True, the fast arrangement) or full-length [n_full,Hkv,D] fetched by idx as well.
    n: rows of the packed set allocated (default: idx.numel()).  Returns the packed O [n,Hq,D] (and lse [Hq,n] if asked)."""
    _dev(Q, K, V, idx, cu_seqlens)
    n_full, Hq, D = Q.shape
    Hkv = K.shape[1]
    if n is None:
        n = idx.numel()
    if idx.dtype != torch.int32 or idx.numel() < n:
        raise ValueError("idx must be int32 with at least n entries")
    if scale is None:
        scale = 1.0 / (D ** 0.5)
    if O is None:
        O = torch.empty(n, Hq, D, dtype=Q.dtype, device=Q.device)
    lse = torch.empty(Hq, n, dtype=torch.float32, device=Q.device) if want_lse else None
    dt = dtype_code(Q)
    if ws is None:
        ws = workspace(dash_workspace_bytes(WS_ATTENTION, n, cu_seqlens.numel() - 1, Hq, Hkv, D, dt), Q.device)
    st = lib().dash_varlen_attention_indexed(_p(Q), _p(K), _p(V), _p(O), _p(lse), Q.stride(0), K.stride(0), V.stride(0), O.stride(0),
                                             _p(idx), n_full, int(bool(kv_packed)), _p(cu_seqlens), cu_seqlens.numel() - 1, n, int(max_seqlen), Hq, Hkv, D,
                                             float(scale), 1, dt, _p(ws), ws.numel(), _stream())
    _check(st, "dash_varlen_attention_indexed")
    return (O, lse) if want_lse else O


def dash_decode_attention(q: torch.Tensor, Kc: torch.Tensor, Vc: torch.Tensor, cu_seqlens: torch.Tensor, scale: Optional[float] = None,
                          out: Optional[torch.Tensor] = None, want_lse: bool = False, ws: Optional[torch.Tensor] = None):
    """q [S,Hq,D] (one new token per sequence), Kc, Vc [n,Hkv,D] packed caches.  Returns out [S,Hq,D] (and lse [S,Hq])."""
    _dev(q, Kc, Vc, cu_seqlens)
    S, Hq, D = q.shape
    n, Hkv = Kc.shape[0], Kc.shape[1]
    if scale is None:
        scale = 1.0 / (D ** 0.5)
    if out is None:
        out = torch.empty(S, Hq, D, dtype=q.dtype, device=q.device)
    lse = torch.empty(S, Hq, dtype=torch.float32, device=q.device) if want_lse else None
    if ws is None:
        ws = workspace(dash_workspace_bytes(WS_DECODE, n, S, Hq, Hkv, D, dtype_code(q)), q.device)
    st = lib().dash_decode_attention(_p(q), _p(Kc), _p(Vc), _p(out), _p(lse), q.stride(0), Kc.stride(0) if n else Hkv * D,
                                     Vc.stride(0) if n else Hkv * D, out.stride(0), _p(cu_seqlens), S, n, Hq, Hkv, D, float(scale),
                                     dtype_code(q), _p(ws), ws.numel(), _stream())
    _check(st, "dash_decode_attention")
    return (out, lse) if want_lse else out


# ---- the block step ---------------------------------------------------------------
def dash_fold_norm_weight(W: torch.Tensor, rms_weight: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """W_out[i, :] = rms_weight[i] * W[i, :] on the device (the norm's weight folded into the projection behind it)."""
    _dev(W, rms_weight, out)
    if out is None:
        out = torch.empty_like(W)
    st = lib().dash_fold_norm_weight(_p(W), _p(rms_weight), W.shape[0], W.shape[1], W.stride(0), dtype_code(W), _p(out), out.stride(0), _stream())
    _check(st, "dash_fold_norm_weight")
    return out


def dash_rope_table(rope_base: float, D: int, n_pos: int, device) -> torch.Tensor:
    """(cos, sin) of pos * rope_base^(-2i/D) for pos < n_pos, i < D/2: fp32 [n_pos, D/2, 2], made once per prefill."""
    table = torch.empty(n_pos, D // 2, 2, dtype=torch.float32, device=device)
    _check(lib().dash_rope_table(float(rope_base), D, n_pos, _p(table), _stream()), "dash_rope_table")
    return table


def _set_handover(cfg, holder, rope_table, inv_rms_in, inv_rms_next):
    holder._handover = (rope_table, inv_rms_in, inv_rms_next)           # keeps the tensors alive
    cfg.rope_table = rope_table.data_ptr() if rope_table is not None else None
    cfg.rope_table_len = rope_table.shape[0] if rope_table is not None else 0
    cfg.inv_rms_in = inv_rms_in.data_ptr() if inv_rms_in is not None else None
    cfg.inv_rms_next = inv_rms_next.data_ptr() if inv_rms_next is not None else None


def _projections_fit(shape) -> bool:
    """True if every projection of the block runs with its fused epilogue (256-column tiles, depth in steps of 64)."""
    nq, hd = (shape.Hq + 2 * shape.Hkv) * shape.D, shape.Hq * shape.D
    ok = shape.d % 256 == 0 and nq % 256 == 0 and ((shape.Hq + shape.Hkv) * shape.D) % 256 == 0 and hd % 64 == 0
    return ok and (shape.m == 0 or shape.m % 128 == 0)


class Layer:
    """Device-resident weights and configuration of one block for dash_layer_step."""

    def __init__(self, shape, weights, device, norm_mode=NORM_REL, norm_eps=1e-12, sel_mode=SEL_THRESHOLD, tau=0.0,
                 keep_counts: Optional[torch.Tensor] = None, keep_first=0, keep_last=0, scatter_which=2, fold_norms=True):
        self.shape = shape
        self.Wqkv = torch.cat([weights["Wq"], weights["Wk"], weights["Wv"]], dim=1).contiguous().to(device)
        self.Wo = weights["Wo"].contiguous().to(device)
        self.rms_w = weights["rms_w"].contiguous().to(device)
        # where the projections run with their fused epilogues (bf16, whole 256-column tiles) the norm's weight is folded into the
        # projection once, here, by the library: the step then needs no normalisation pass (the row factor 1 / rms is applied to the
        # projection's accumulators).  fold_norms=False keeps the norm as a pass of its own.
        self.rms_folded = bool(fold_norms) and self.Wqkv.dtype == torch.bfloat16 and _projections_fit(shape)
        if self.rms_folded:
            dash_fold_norm_weight(self.Wqkv, self.rms_w, out=self.Wqkv)
        self.keep_counts = keep_counts
        self.cfg = LayerCfg(shape.d, shape.Hq, shape.Hkv, shape.D, dtype_code(self.Wo), self.Wqkv.data_ptr(), self.Wo.data_ptr(),
                            self.rms_w.data_ptr(), shape.rms_eps, shape.rope_base, norm_mode, norm_eps, sel_mode, tau,
                            keep_counts.data_ptr() if keep_counts is not None else None, keep_first, keep_last, scatter_which, None, None, int(self.rms_folded),
                            None, 0, None, None)

    def set_tau(self, tau: float):
        self.cfg.tau = float(tau)

    def set_handover(self, rope_table=None, inv_rms_in=None, inv_rms_next=None):
        """What a prefill hands from block to block (needs the folded norm): the rotary table of dash_rope_table, the row factors
        1 / rms of the entering rows (fp32 [n], a previous step's inv_rms_next) and a buffer for those of the rows that stay."""
        _set_handover(self.cfg, self, rope_table, inv_rms_in, inv_rms_next)

    def set_kv_cache(self, k_cache: Optional[torch.Tensor], v_cache: Optional[torch.Tensor]):
        """[n, Hkv, D] buffers that receive this block's keys (rotary applied) and values, or None."""
        self.k_cache, self.v_cache = k_cache, v_cache
        self.cfg.k_cache = k_cache.data_ptr() if k_cache is not None else None
        self.cfg.v_cache = v_cache.data_ptr() if v_cache is not None else None


def dash_layer_workspace(layer: Layer, n: int, S: int) -> LayerWsLayout:
    out = LayerWsLayout()
    _check(lib().dash_layer_workspace(ctypes.byref(layer.cfg), n, S, ctypes.byref(out)), "dash_layer_workspace")
    return out


def dash_layer_step(layer: Layer, H_in, tok_index_in, pos_in, cu_in, max_seqlen: int, x_full, H_next, tok_index_next, pos_next,
                    cu_next, n_next, r_out, mask_out, ws):
    n = H_in.shape[0]
    st = lib().dash_layer_step(ctypes.byref(layer.cfg), _p(H_in), _p(tok_index_in), _p(pos_in), _p(cu_in), cu_in.numel() - 1, n,
                               int(max_seqlen), _p(x_full), _p(H_next), _p(tok_index_next), _p(pos_next), _p(cu_next), _p(n_next),
                               _p(r_out), _p(mask_out), _p(ws), ws.numel(), _stream())
    _check(st, "dash_layer_step")


# ---- the whole block, feed-forward included -------------------------------------------
class Block:
    """Device-resident weights and configuration of one whole block (attention + gated FFN) for dash_block_step."""

    def __init__(self, shape, weights, device, signal=SIGNAL_ATTN, **layer_kwargs):
        self.layer = Layer(shape, weights, device, **layer_kwargs)
        self.shape = shape
        self.Wgu = torch.cat([weights["Wg"], weights["Wu"]], dim=1).contiguous().to(device)
        self.Wd = weights["Wd"].contiguous().to(device)
        self.rms2_w = weights["rms2_w"].contiguous().to(device)
        self.rms2_folded = self.layer.rms_folded and signal == SIGNAL_ATTN
        if self.rms2_folded:
            dash_fold_norm_weight(self.Wgu, self.rms2_w, out=self.Wgu)
        self.cfg = BlockCfg(self.layer.cfg, shape.m, self.Wgu.data_ptr(), self.Wd.data_ptr(), self.rms2_w.data_ptr(), signal, int(self.rms2_folded))

    def set_tau(self, tau: float):
        self.cfg.attn.tau = float(tau)

    def set_handover(self, rope_table=None, inv_rms_in=None, inv_rms_next=None):
        """As Layer.set_handover (the row factors handed on are those of H', the block's output)."""
        _set_handover(self.cfg.attn, self, rope_table, inv_rms_in, inv_rms_next)

    def set_kv_cache(self, k_cache: Optional[torch.Tensor], v_cache: Optional[torch.Tensor]):
        """[n, Hkv, D] buffers that receive this block's keys (rotary applied) and values, or None."""
        self.k_cache, self.v_cache = k_cache, v_cache
        self.cfg.attn.k_cache = k_cache.data_ptr() if k_cache is not None else None
        self.cfg.attn.v_cache = v_cache.data_ptr() if v_cache is not None else None

    def set_keep_counts(self, keep_counts: Optional[torch.Tensor], sel_mode: int):
        self.keep_counts = keep_counts
        self.cfg.attn.sel_mode = sel_mode
        self.cfg.attn.keep_counts = keep_counts.data_ptr() if keep_counts is not None else None


def dash_block_workspace(block: Block, n: int, S: int) -> BlockWsLayout:
    out = BlockWsLayout()
    _check(lib().dash_block_workspace(ctypes.byref(block.cfg), n, S, ctypes.byref(out)), "dash_block_workspace")
    return out


def dash_block_step(block: Block, H_in, tok_index_in, pos_in, cu_in, max_seqlen: int, x_full, H_next, tok_index_next, pos_next,
                    cu_next, n_next, r_out, mask_out, ws):
    n = H_in.shape[0]
    st = lib().dash_block_step(ctypes.byref(block.cfg), _p(H_in), _p(tok_index_in), _p(pos_in), _p(cu_in), cu_in.numel() - 1, n,
                               int(max_seqlen), _p(x_full), _p(H_next), _p(tok_index_next), _p(pos_next), _p(cu_next), _p(n_next),
                               _p(r_out), _p(mask_out), _p(ws), ws.numel(), _stream())
    _check(st, "dash_block_step")
