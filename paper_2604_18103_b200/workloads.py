"""Seeded synthetic inputs for the halted-prefill path.

This module only *draws data*: shapes, seeds, value distributions and the
sequence structure of the five benchmark workloads.  It contains none of the
method's arithmetic (no delta-norm, no selection, no compaction, no attention)
and imports neither the CUDA binding nor the CPU oracle, so both sides can be
fed the very same host tensors.

All tensors are created on the host with ``torch.Generator`` (seeded) and are
returned as CPU tensors in the workload's storage dtype (bf16 or fp32).  The
real long-context / vision-language prompts the paper evaluates on are not
available offline; these draws stand in for them with the same layer shape
(Qwen2.5-7B: d=3584, 28 query heads, 4 KV heads, head_dim 128; Appendix A),
the same prompt lengths (8k .. 131k; Table "theory_speedup_vs_len") and a
heavy-tailed per-token update magnitude (Fig. 1).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional

import torch


@dataclass(frozen=True)
class LayerShape:
    d: int          # hidden size
    Hq: int         # query heads
    Hkv: int        # key/value heads
    D: int          # head_dim
    rope_base: float
    dtype: torch.dtype
    rms_eps: float = 1e-6
    m: int = 0      # feed-forward width (0: the block is used without its FFN)

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv


QWEN = LayerShape(d=3584, Hq=28, Hkv=4, D=128, rope_base=1.0e6, dtype=torch.bfloat16, m=18944)
TINY = LayerShape(d=256, Hq=4, Hkv=4, D=64, rope_base=1.0e4, dtype=torch.float32, m=512)
# Qwen-like GQA shape small enough for full CPU checks of every row
MINI = LayerShape(d=512, Hq=8, Hkv=2, D=128, rope_base=1.0e6, dtype=torch.bfloat16, m=1024)

# active fraction after each layer of the cascaded workload (config 3)
CASCADE_FRACTIONS = (1.0, 0.9, 0.8, 0.7, 0.6, 0.5, 0.4, 0.35)


def _gen(seed: int, stream: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed((int(seed) * 1000003 + int(stream) * 7919 + 12345) & 0x7FFFFFFFFFFFFFFF)
    return g


def _randn(shape, seed, stream, std=1.0, dtype=torch.float32) -> torch.Tensor:
    x = torch.randn(*shape, generator=_gen(seed, stream), dtype=torch.float32)
    if std != 1.0:
        x.mul_(std)
    return x.to(dtype)


def hidden_states(T: int, d: int, seed: int, dtype, unit_rms: bool = True, stream: int = 0) -> torch.Tensor:
    """x ~ N(0,1) [T,d]; optionally rescaled as a whole tensor to RMS exactly 1."""
    x = torch.randn(T, d, generator=_gen(seed, stream), dtype=torch.float32)
    if unit_rms and x.numel() > 0:
        x.div_(x.double().pow(2).mean().sqrt().float())
    return x.to(dtype)


def layer_weights(shape: LayerShape, seed: int, layer: int = 0) -> Dict[str, torch.Tensor]:
    """Wq/Wk/Wv/Wo ~ N(0, 0.02^2), RMSNorm weight = 1.  Row-major [in, out]."""
    s = 100 + 10 * layer
    return {
        "Wq": _randn((shape.d, shape.Hq * shape.D), seed, s + 1, 0.02, shape.dtype),
        "Wk": _randn((shape.d, shape.Hkv * shape.D), seed, s + 2, 0.02, shape.dtype),
        "Wv": _randn((shape.d, shape.Hkv * shape.D), seed, s + 3, 0.02, shape.dtype),
        "Wo": _randn((shape.Hq * shape.D, shape.d), seed, s + 4, 0.02, shape.dtype),
        "rms_w": torch.ones(shape.d, dtype=shape.dtype),
    }


def ffn_weights(shape: LayerShape, seed: int, layer: int = 0) -> Dict[str, torch.Tensor]:
    """Gated feed-forward weights of width shape.m: Wg, Wu [d, m], Wd [m, d] ~ N(0, 0.02^2), second RMSNorm weight = 1."""
    s = 100 + 10 * layer
    return {
        "Wg": _randn((shape.d, shape.m), seed, s + 5, 0.02, shape.dtype),
        "Wu": _randn((shape.d, shape.m), seed, s + 6, 0.02, shape.dtype),
        "Wd": _randn((shape.m, shape.d), seed, s + 7, 0.02, shape.dtype),
        "rms2_w": torch.ones(shape.d, dtype=shape.dtype),
    }


def qkv(T: int, shape: LayerShape, seed: int, stream: int = 20):
    """Q,K,V ~ N(0,1) with the rotary embedding regarded as already applied."""
    q = _randn((T, shape.Hq, shape.D), seed, stream + 0, 1.0, shape.dtype)
    k = _randn((T, shape.Hkv, shape.D), seed, stream + 1, 1.0, shape.dtype)
    v = _randn((T, shape.Hkv, shape.D), seed, stream + 2, 1.0, shape.dtype)
    return q, k, v


def cu_from_lengths(lengths: List[int]) -> torch.Tensor:
    cu = [0]
    for L in lengths:
        cu.append(cu[-1] + int(L))
    return torch.tensor(cu, dtype=torch.int32)


def positions(cu: torch.Tensor) -> torch.Tensor:
    """Within-sequence position of every packed token."""
    out = []
    for s in range(cu.numel() - 1):
        out.append(torch.arange(int(cu[s + 1]) - int(cu[s]), dtype=torch.int32))
    return torch.cat(out) if out else torch.zeros(0, dtype=torch.int32)


@dataclass
class Workload:
    name: str
    shape: LayerShape
    cu: torch.Tensor                     # int32 [S+1]
    tensors: Dict[str, torch.Tensor] = field(default_factory=dict)
    weights: List[Dict[str, torch.Tensor]] = field(default_factory=list)
    rho: Optional[float] = None          # halting fraction chosen by percentile
    fractions: Optional[tuple] = None    # cascaded keep fractions of the original T
    tau: Optional[float] = None          # fixed threshold (config 5)

    @property
    def T(self) -> int:
        return int(self.cu[-1])

    @property
    def S(self) -> int:
        return self.cu.numel() - 1


def config1(T: int = 1024, seed: int = 0) -> Workload:
    """Single fp32 layer, d=256, 4 heads of 64; half of the tokens halt."""
    w = Workload("cfg1_tiny_fp32", TINY, cu_from_lengths([T]), rho=0.5)
    w.tensors["H"] = hidden_states(T, TINY.d, seed, TINY.dtype, unit_rms=False)
    w.weights = [layer_weights(TINY, seed)]
    return w


def config2(T: int = 8192, seed: int = 1, shape: LayerShape = QWEN) -> Workload:
    """Single Qwen2.5-7B-shaped bf16 layer; 40th-percentile threshold (60 % stay)."""
    w = Workload("cfg2_qwen_layer", shape, cu_from_lengths([T]), rho=0.4)
    w.tensors["H"] = hidden_states(T, shape.d, seed, shape.dtype)
    w.weights = [layer_weights(shape, seed)]
    return w


def config3(T: int = 32768, seed: int = 2, n_layers: int = 8, shape: LayerShape = QWEN) -> Workload:
    """Cascade of Qwen-shaped layers; per-layer keep fractions of the original T."""
    w = Workload("cfg3_cascade", shape, cu_from_lengths([T]), fractions=CASCADE_FRACTIONS[:n_layers])
    w.tensors["H"] = hidden_states(T, shape.d, seed, shape.dtype)
    w.weights = [layer_weights(shape, seed, layer=l) for l in range(n_layers)]
    return w


def _lognormal(T: int, mu, seed: int, stream: int) -> torch.Tensor:
    z = torch.randn(T, generator=_gen(seed, stream), dtype=torch.float64)
    return torch.exp(z + mu)


def config4(T: int = 131072, seed: int = 3, shape: LayerShape = QWEN) -> Workload:
    """Sparse long prompt: the update of token t is drawn as r*_t * g_t with
    r* ~ LogNormal(-3, 1), so its relative size is heavy-tailed; 80 % halt."""
    w = Workload("cfg4_sparse_131k", shape, cu_from_lengths([T]), rho=0.8)
    w.tensors["H"] = hidden_states(T, shape.d, seed, shape.dtype)
    rstar = _lognormal(T, -3.0, seed, 10).float()
    g = torch.randn(T, shape.d, generator=_gen(seed, 11), dtype=torch.float32)
    w.tensors["U"] = (g * rstar[:, None]).to(shape.dtype)
    q, k, v = qkv(T, shape, seed)
    w.tensors.update(Q=q, K=k, V=v)
    w.tensors["pos"] = positions(w.cu)
    return w


CFG5_LENGTHS = (4096, 12288, 16384, 16896)
CFG5_TAU = math.exp(-1.7184)   # 0.1793


def config5(lengths=CFG5_LENGTHS, seed: int = 4, shape: LayerShape = QWEN, patch: int = 256, rank: int = 8) -> Workload:
    """Packed multimodal-shaped batch.  Each sequence = image block (first 75 %,
    runs of `patch` tokens that share a rank-`rank` basis) followed by text.
    Seeded update sizes give about 90 % halting in image blocks and about 10 %
    in text under the single fixed threshold CFG5_TAU."""
    cu = cu_from_lengths(list(lengths))
    w = Workload("cfg5_multimodal_varlen", shape, cu, tau=CFG5_TAU)
    T = int(cu[-1])
    H = torch.empty(T, shape.d, dtype=torch.float32)
    scale = torch.ones(T, dtype=torch.float32)
    is_image = torch.zeros(T, dtype=torch.bool)
    stream = 40
    for s, L in enumerate(lengths):
        a0 = int(cu[s])
        n_img = (int(L) * 3) // 4
        is_image[a0:a0 + n_img] = True
        p0 = 0
        while p0 < n_img:
            m = min(patch, n_img - p0)
            A = torch.randn(m, rank, generator=_gen(seed, stream), dtype=torch.float32)
            B = torch.randn(rank, shape.d, generator=_gen(seed, stream + 1), dtype=torch.float32)
            H[a0 + p0:a0 + p0 + m] = (A @ B) / math.sqrt(rank)
            # size of the latent code of each token: keeps the drawn update
            # proportional to the token's own magnitude
            scale[a0 + p0:a0 + p0 + m] = A.pow(2).mean(dim=1).sqrt()
            stream += 2
            p0 += m
        n_txt = int(L) - n_img
        H[a0 + n_img:a0 + int(L)] = torch.randn(n_txt, shape.d, generator=_gen(seed, stream), dtype=torch.float32)
        stream += 1
    mu = torch.where(is_image, torch.tensor(-3.0, dtype=torch.float64), torch.tensor(-0.4369, dtype=torch.float64))
    rstar = _lognormal(T, mu, seed, 12).float() * scale
    g = torch.randn(T, shape.d, generator=_gen(seed, 13), dtype=torch.float32)
    w.tensors["H"] = H.to(shape.dtype)
    w.tensors["U"] = (g * rstar[:, None]).to(shape.dtype)
    q, k, v = qkv(T, shape, seed)
    w.tensors.update(Q=q, K=k, V=v)
    w.tensors["pos"] = positions(cu)
    w.tensors["is_image"] = is_image
    return w


def random_mask(n: int, keep_prob: float, seed: int, stream: int = 30) -> torch.Tensor:
    """Seeded 0/1 keep mask (uint8) for compaction tests."""
    u = torch.rand(n, generator=_gen(seed, stream))
    return (u < keep_prob).to(torch.uint8)


def sample_rows(cu: torch.Tensor, n_samples: int, seed: int, tile: int = 128) -> torch.Tensor:
    """Seeded sample of packed row indices for checks that cannot visit every row.  In this order, as far as the budget
    n_samples goes: the first and last row of every sequence; one row drawn inside every `tile`-row tile of every sequence
    (tiles counted from the start of the sequence), so that no tile goes unvisited; the rows on both sides of every tile
    boundary; uniform draws over all rows."""
    g = _gen(seed, 31)
    picks: List[int] = []
    seen = set()

    def add(rows) -> None:
        for r in rows:
            r = int(r)
            if r not in seen and len(picks) < n_samples:
                seen.add(r)
                picks.append(r)

    S = cu.numel() - 1
    bounds = [(int(cu[s]), int(cu[s + 1])) for s in range(S) if int(cu[s + 1]) > int(cu[s])]
    for a, b in bounds:
        add((a, b - 1))
    starts = [(t, min(t + tile, b)) for a, b in bounds for t in range(a, b, tile)]
    if starts:
        u = torch.rand(len(starts), generator=g)
        order = torch.randperm(len(starts), generator=g).tolist()         # if the budget is short, the tiles left out are random ones
        add(starts[i][0] + int(float(u[i]) * (starts[i][1] - starts[i][0])) for i in order)
    edges = [r for a, b in bounds for t in range(a + tile, b, tile) for r in (t - 1, t)]
    if edges:
        order = torch.randperm(len(edges) // 2, generator=g).tolist()
        add(r for i in order for r in edges[2 * i:2 * i + 2])
    T = int(cu[-1])
    if T > 0 and len(picks) < min(n_samples, T):
        extra = torch.randperm(T, generator=g) if T <= 4 * n_samples else torch.randint(0, T, (4 * n_samples,), generator=g)
        add(extra.tolist())
    return torch.tensor(sorted(picks), dtype=torch.int64)
