"""CPU oracle for the per-layer halted-prefill path (DASH).

TEST INFRASTRUCTURE -- not part of the product.  Only the tests, the smoke
check and the benchmark's ``cpu_baseline`` / reference arm may import this
package; the CUDA library and its Python binding never do, and this package
imports nothing from them.

Everything is plain fp64 numpy, one statement per step of the method, in the
paper's order and notation; the only compiled piece is the brute-force
attention loop in ``attention_ref.c`` (same directory).  Inputs may be torch CPU
tensors (bf16 / fp32 / ints) or numpy arrays; they are widened exactly to fp64.

Parity pins (tests/test_oracle_pins.py): every function below is pinned by
closed forms, brute force on tiny inputs, printed values of the paper's
Appendix-A table, or a library routine.  The paper's *accuracy* claims
(benchmark scores) need its datasets and weights: parity unpinned, out of scope.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess
from typing import Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None


# --------------------------------------------------------------------------
# plumbing: widening inputs, building/loading the C attention loop
# --------------------------------------------------------------------------
def f64(x) -> np.ndarray:
    """Exact widening of a tensor/array to a contiguous fp64 numpy array."""
    if hasattr(x, "detach"):  # torch tensor
        x = x.detach().cpu().double().numpy()
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def i32(x) -> np.ndarray:
    if hasattr(x, "detach"):
        x = x.detach().cpu().numpy()
    return np.ascontiguousarray(np.asarray(x, dtype=np.int32))


def build(force: bool = False) -> str:
    """Compile attention_ref.c with gcc (OpenMP) into this directory."""
    src = os.path.join(_HERE, "attention_ref.c")
    out = os.path.join(_HERE, "libdash_oracle.so")
    if force or not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(src):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", out, src, "-lm"])
    return out


def _lib():
    global _LIB
    if _LIB is None:
        lib = ctypes.CDLL(build())
        lib.dash_oracle_attention.restype = ctypes.c_int
        lib.dash_oracle_attention.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int] * 4 + [
            ctypes.c_double, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
        lib.dash_oracle_num_threads.restype = ctypes.c_int
        _LIB = lib
    return _LIB


def num_threads() -> int:
    return int(_lib().dash_oracle_num_threads())


# --------------------------------------------------------------------------
# Appendix A: kept length and the FLOPs proxy
# --------------------------------------------------------------------------
def keep_count(n: int, rho: float, keep_first: int = 0, keep_last: int = 0, mode: int = 0) -> int:
    """Number of tokens that stay active out of n.

    mode 0 -- Eq. 3: K = floor((1 - rho) * n).
    mode 1 -- Appendix A ("Effective kept length" and the caption of the table
    of theoretical speedups): a prefix of keep_first and a suffix of keep_last
    tokens always stay; of the n - n_fix others, drop_target =
    floor(round(c * (n - n_fix))) are dropped, c = rho.
    """
    if mode == 0:
        return int(math.floor((1.0 - rho) * n))
    n_fix = min(n, keep_first + keep_last)
    drop_target = int(math.floor(round(rho * (n - n_fix))))
    return n - drop_target


def flops_per_layer(n: float, d: int, m: int) -> float:
    """Appendix A, FLOPs proxy: A(n) = 4 n d^2 + 2 n^2 d + 2 n d m."""
    return 4.0 * n * d * d + 2.0 * n * n * d + 2.0 * n * d * m


def flops_single_shot(n: int, n_hat: int, L: int, l_s: int, d: int, m: int):
    """Appendix A: C_full = L A(n); C_ours = l_s A(n) + (L - l_s) A(n_hat);
    returns (r_FLOPs, s_FLOPs) = (1 - C_ours / C_full, C_full / C_ours)."""
    c_full = L * flops_per_layer(n, d, m)
    c_ours = l_s * flops_per_layer(n, d, m) + (L - l_s) * flops_per_layer(n_hat, d, m)
    return 1.0 - c_ours / c_full, c_full / c_ours


# --------------------------------------------------------------------------
# step 1: token-wise delta-attention score
# --------------------------------------------------------------------------
REL, ABS = 0, 1


def delta_norm(U, H, mode: int = REL, eps: float = 1e-12) -> np.ndarray:
    """Eq. 2: Delta_t = ||U_t||_2 (ABS).  REL divides by the norm of the
    residual stream entering the block, ||H_t||_2 (the "relative" Delta_attn of
    Fig. 1), guarded as max(||H_t||, eps).  Result rounded to fp32."""
    U = f64(U)
    num = np.sqrt(np.sum(U * U, axis=1))
    if mode == ABS:
        return num.astype(np.float32)
    H = f64(H)
    den = np.sqrt(np.sum(H * H, axis=1))
    return (num / np.maximum(den, eps)).astype(np.float32)


def residual(H, U) -> np.ndarray:
    """Preliminaries: H~ = H + U."""
    return f64(H) + f64(U)


# --------------------------------------------------------------------------
# step 2: halting rule
# --------------------------------------------------------------------------
THRESHOLD, KEEP_COUNT = 0, 1


def select(r, cu, mode: int, tau: float = 0.0, keep_counts: Optional[Sequence[int]] = None,
           keep_first: int = 0, keep_last: int = 0, halt_high: bool = False) -> np.ndarray:
    """Keep mask (1 = stays active) from the scores r, per sequence.

    Protected tokens (first keep_first / last keep_last of each sequence in its
    current order; Appendix A) always stay.
    THRESHOLD: a token halts iff r_t < tau (low-Delta tokens are the halted
      ones; NaN compares false and therefore stays).
    KEEP_COUNT: Eq. 3, S* = TopK(S, K, Delta): K_s tokens of sequence s stay in
      total -- the protected ones plus the K_s - n_protected largest scores of
      the others, ties broken toward the lower index, NaN ranked as +inf.
    halt_high (the paper's direction ablation, "High Delta_attn"): the rule runs on the negated
    scores -- a token halts iff r_t > tau, or the K_s smallest scores stay.
    """
    r = np.asarray(r, dtype=np.float32)
    cu = i32(cu)
    n = r.shape[0]
    mask = np.zeros(n, dtype=np.uint8)
    for s in range(cu.shape[0] - 1):
        a, b = int(cu[s]), int(cu[s + 1])
        ns = b - a
        protected = np.zeros(ns, dtype=bool)
        protected[:min(keep_first, ns)] = True
        if keep_last > 0:
            protected[max(0, ns - keep_last):] = True
        rs = r[a:b]
        if halt_high:
            rs = -rs
        if mode == THRESHOLD:
            halted = (rs < np.float32(-tau if halt_high else tau)) & ~protected
            mask[a:b] = (~halted).astype(np.uint8)
        else:
            K = int(keep_counts[s])
            elig = np.flatnonzero(~protected)
            k_elig = min(max(K - int(protected.sum()), 0), elig.size)
            key = rs[elig].astype(np.float64)
            key[np.isnan(key)] = np.inf
            order = sorted(range(elig.size), key=lambda t: (-key[t], t))  # r descending, index ascending
            keep = np.zeros(ns, dtype=bool)
            keep[protected] = True
            keep[elig[order[:k_elig]]] = True
            mask[a:b] = keep.astype(np.uint8)
    return mask


# --------------------------------------------------------------------------
# step 3: order-preserving compaction and scatter of frozen states
# --------------------------------------------------------------------------
def compact(mask, cu_in, rows: Sequence = (), pos_in=None, tok_in=None) -> Dict[str, object]:
    """Gather the active tokens (Alg. 1, "gathering tokens indexed by S_l").

    A serial exclusive prefix sum over the mask gives every active token its
    dense output slot; order is preserved.  Returns idx (source row of each
    output row), the new packed sequence boundaries cu_out, n_out, the gathered
    copies of every tensor in `rows` (bit-exact rows) and of pos / tok index.
    """
    mask = np.asarray(mask.cpu() if hasattr(mask, "cpu") else mask, dtype=np.uint8)
    cu_in = i32(cu_in)
    n = mask.shape[0]
    slot = np.zeros(n + 1, dtype=np.int64)      # exclusive prefix sum
    running = 0
    for t in range(n):
        slot[t] = running
        running += 1 if mask[t] else 0
    slot[n] = running
    n_out = running
    idx = np.zeros(n_out, dtype=np.int32)
    for t in range(n):
        if mask[t]:
            idx[slot[t]] = t
    cu_out = np.array([slot[int(c)] for c in cu_in], dtype=np.int32)
    out = {"idx": idx, "cu_out": cu_out, "n_out": int(n_out), "rows": []}
    for x in rows:
        if hasattr(x, "detach"):
            out["rows"].append(x[idx.astype(np.int64)])       # torch fancy index: exact row copy
        else:
            out["rows"].append(np.asarray(x)[idx])
    if pos_in is not None:
        out["pos_out"] = i32(pos_in)[idx]
    if tok_in is not None:
        out["tok_out"] = i32(tok_in)[idx]
    return out


def scatter(src, tok_index, sel, which: int, dst_full):
    """dst_full[tok_index[i]] = src[i] for rows with sel[i] == which (which = 2:
    every row).  Sec. 3.4: the hidden state of a halted token stays fixed at its
    last updated value -- this is how that value reaches the full-length output.
    Works on torch tensors or numpy arrays; dst_full is modified and returned."""
    tok_index = i32(tok_index)
    n = tok_index.shape[0]
    if sel is not None:
        sel = np.asarray(sel.cpu() if hasattr(sel, "cpu") else sel, dtype=np.uint8)
    for i in range(n):
        if which == 2 or int(sel[i]) == which:
            dst_full[int(tok_index[i])] = src[i]
    return dst_full


# --------------------------------------------------------------------------
# step 4: causal GQA attention over the packed active set
# --------------------------------------------------------------------------
def attention(Q, K, V, cu, scale: Optional[float] = None, rows=None):
    """Brute-force causal softmax attention inside each packed sequence; kv head
    of query head h is h // (Hq // Hkv).  Halted tokens are simply absent from
    the packed buffers, hence contribute no key or value (Sec. 3.4; the KV cache
    of deeper layers is shortened, Appendix C "DASH settings").

    Q [n,Hq,D], K,V [n,Hkv,D].  rows: packed row indices to evaluate (default
    all).  Returns (O [len(rows),Hq,D] fp64, lse [len(rows),Hq] fp64)."""
    Q, K, V = f64(Q), f64(K), f64(V)
    cu = i32(cu)
    n, Hq, D = Q.shape
    Hkv = K.shape[1]
    if scale is None:
        scale = 1.0 / math.sqrt(D)
    if rows is None:
        rows = np.arange(int(cu[-1]), dtype=np.int64)
    else:
        rows = np.ascontiguousarray(np.asarray(rows.cpu() if hasattr(rows, "cpu") else rows, dtype=np.int64))
    O = np.zeros((rows.shape[0], Hq, D), dtype=np.float64)
    lse = np.zeros((rows.shape[0], Hq), dtype=np.float64)
    if rows.shape[0] == 0:
        return O, lse
    rc = _lib().dash_oracle_attention(Q.ctypes.data, K.ctypes.data, V.ctypes.data, cu.ctypes.data,
                                      cu.shape[0] - 1, Hq, Hkv, D, float(scale),
                                      rows.ctypes.data, rows.shape[0], O.ctypes.data, lse.ctypes.data)
    if rc != 0:
        raise ValueError("row index outside every sequence")
    return O, lse


# --------------------------------------------------------------------------
# glue of the block: LN, projections, rotary embedding
# --------------------------------------------------------------------------
def rmsnorm(H, w, eps: float = 1e-6) -> np.ndarray:
    """LN of Eq. 1, read as RMSNorm (the backbones are Qwen2.5 / Qwen2-VL):
    y = x / sqrt(mean(x^2) + eps) * w."""
    H = f64(H)
    ms = np.mean(H * H, axis=1, keepdims=True)
    return H / np.sqrt(ms + eps) * f64(w)[None, :]


def rope(X, pos, base: float) -> np.ndarray:
    """Rotary embedding, rotate-half convention: the pair (x_i, x_{i+D/2}) of
    every head is rotated by the angle pos * base^(-2i/D)."""
    X = f64(X)
    pos = f64(pos)
    D = X.shape[-1]
    half = D // 2
    inv_freq = base ** (-2.0 * np.arange(half, dtype=np.float64) / D)
    ang = pos[:, None] * inv_freq[None, :]                 # [n, D/2]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    x1, x2 = X[..., :half], X[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def layer_step(H, weights: Dict[str, object], cu, pos, shape, norm_mode: int = REL,
               sel_mode: int = THRESHOLD, tau: float = 0.0, keep_counts=None,
               keep_first: int = 0, keep_last: int = 0, eps: float = 1e-12,
               attn_rows=None) -> Dict[str, object]:
    """One halted block without its FFN, on the packed active tokens H [n,d]
    (Alg. 1, the body of the loop): U = Attn(LN(H)); H~ = H + U; score; select;
    compact.  No intermediate rounding.  `shape` needs Hq, Hkv, D, rope_base,
    rms_eps.  With attn_rows given, attention (and everything after it) is only
    evaluated for those packed rows: returns U, Ht, r restricted to them and no
    selection."""
    Hf = f64(H)
    n = Hf.shape[0]
    Hn = rmsnorm(Hf, weights["rms_w"], shape.rms_eps)
    Q = (Hn @ f64(weights["Wq"])).reshape(n, shape.Hq, shape.D)
    K = (Hn @ f64(weights["Wk"])).reshape(n, shape.Hkv, shape.D)
    V = (Hn @ f64(weights["Wv"])).reshape(n, shape.Hkv, shape.D)
    Q = rope(Q, pos, shape.rope_base)
    K = rope(K, pos, shape.rope_base)
    O, lse = attention(Q, K, V, cu, 1.0 / math.sqrt(shape.D), rows=attn_rows)
    U = O.reshape(O.shape[0], shape.Hq * shape.D) @ f64(weights["Wo"])
    Hsel = Hf if attn_rows is None else Hf[np.asarray(attn_rows, dtype=np.int64)]
    Ht = Hsel + U
    r = delta_norm(U, Hsel, norm_mode, eps)
    out = {"Q": Q, "K": K, "V": V, "O": O, "lse": lse, "U": U, "Ht": Ht, "r": r}
    if attn_rows is not None:
        return out
    mask = select(r, cu, sel_mode, tau, keep_counts, keep_first, keep_last)
    out["mask"] = mask
    out.update(compact(mask, cu, rows=[Ht], pos_in=pos))
    return out


def ffn_swiglu(X, Wg, Wu, Wd) -> np.ndarray:
    """FFN of Alg. 1, read as the gated feed-forward of the Qwen2.5 backbones:
    FFN(x) = (silu(x Wg) * (x Wu)) Wd with silu(z) = z / (1 + exp(-z))."""
    X = f64(X)
    g = X @ f64(Wg)
    u = X @ f64(Wu)
    return ((g / (1.0 + np.exp(-g))) * u) @ f64(Wd)


def block_step(H, weights: Dict[str, object], cu, pos, shape, norm_mode: int = REL,
               sel_mode: int = THRESHOLD, tau: float = 0.0, keep_counts=None,
               keep_first: int = 0, keep_last: int = 0, eps: float = 1e-12,
               attn_rows=None, signal: str = "attn", halt_high: bool = False) -> Dict[str, object]:
    """One whole block of Alg. 1 on the packed active tokens: U = Attn(LN(H)); H~ = H + U;
    H' = H~ + FFN(LN(H~)); the score is taken from U, the selection from the score; the tokens that
    stay carry H' into the next block, and H' is also the last updated value of the tokens that halt
    here (Sec. 3.4).  `weights` holds the attention weights of layer_step plus Wg, Wu, Wd, rms2_w.
    With attn_rows given only those rows are evaluated (no selection).
    signal = "block" (the paper's ablation of the delta signal): the score is the change over the whole
    block, ||H' - H|| (relative: / ||H||), instead of the attention branch's ||U||."""
    out = layer_step(H, weights, cu, pos, shape, norm_mode, sel_mode, tau, keep_counts, keep_first, keep_last, eps, attn_rows)
    Hn2 = rmsnorm(out["Ht"], weights["rms2_w"], shape.rms_eps)
    out["F"] = ffn_swiglu(Hn2, weights["Wg"], weights["Wu"], weights["Wd"])
    out["H1"] = out["Ht"] + out["F"]
    Hsel = f64(H) if attn_rows is None else f64(H)[np.asarray(attn_rows, dtype=np.int64)]
    if signal == "block":
        out["r"] = delta_norm(out["H1"] - Hsel, Hsel, norm_mode, eps)
    if attn_rows is not None:
        return out
    if signal == "block" or halt_high:
        out["mask"] = select(out["r"], cu, sel_mode, tau, keep_counts, keep_first, keep_last, halt_high)
    out.update(compact(out["mask"], cu, rows=[out["H1"]], pos_in=pos))
    return out


def decode_attention(q, Kc, Vc, cu, scale: Optional[float] = None):
    """Attention of one new token per sequence over that sequence's cached keys and values (the decoding
    stage, Preliminaries; halted prompt tokens have left the cache of the deeper layers, Appendix C "DASH
    settings", so the packed cache simply holds fewer rows there).  No mask: the new token sees every cached
    row of its sequence.  q [S,Hq,D]; Kc, Vc [n,Hkv,D] packed, cu int32 [S+1].  Returns (O [S,Hq,D], lse [S,Hq]);
    an empty cache gives O = 0 and lse = -inf."""
    q, Kc, Vc = f64(q), f64(Kc), f64(Vc)
    cu = i32(cu)
    S, Hq, D = q.shape
    G = Hq // Kc.shape[1]
    if scale is None:
        scale = 1.0 / math.sqrt(D)
    O = np.zeros((S, Hq, D))
    lse = np.full((S, Hq), -np.inf)
    for s in range(S):
        a, b = int(cu[s]), int(cu[s + 1])
        if b <= a:
            continue
        for h in range(Hq):
            sc = (Kc[a:b, h // G] @ q[s, h]) * scale
            mx = sc.max()
            p = np.exp(sc - mx)
            l = p.sum()
            O[s, h] = (p / l) @ Vc[a:b, h // G]
            lse[s, h] = mx + math.log(l)
    return O, lse


def kth_largest(r, k: int) -> float:
    """The k-th largest score (k >= 1): with tau set to it and the rule
    "halt iff r < tau", exactly k tokens stay when there are no ties."""
    r = np.sort(np.asarray(r, dtype=np.float32))[::-1]
    return float(r[k - 1])
