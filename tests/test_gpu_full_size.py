"""GPU parity at the full benchmark sizes (configs 2-5), in the launch configuration
the benchmark times.

Config 2: the whole oracle (every row, about half a minute of host time) against the block
step -- scores, halt mask (threshold from the oracle's own scores), compaction, H~ and O of
every token.  Configs 3-5: everything O(n d) is compared with the oracle in full; the
quadratic attention on a seeded sample of SAMPLE query rows that the oracle evaluates one by
one (what the oracle's cost allows: 2048 rows over 26214 keys are about 4e11 fp64 operations),
drawn so that every 128-row query tile of every sequence holds at least one of them, with the
first / last row of every sequence and both sides of the tile boundaries; the rest through
properties that hold at any size.  Measured error ratios are collected in
parity_errors.json in the session's record folder (see conftest.py)."""
import math

import numpy as np
import pytest
import torch

from conftest import record_error
from oracle import dash_oracle as oc
from paper_2604_18103_b200 import dash
from paper_2604_18103_b200 import workloads as wl
from test_gpu_kernels import assert_close_rms, r_close
from test_gpu_layer import BAND, StepBuffers, check_mask

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SAMPLE = 2048          # attention rows per layer the oracle evaluates at the sizes where it cannot visit them all


def oracle_delta_norm_chunked(U, H, chunk=8192):
    return np.concatenate([oc.delta_norm(U[i:i + chunk], H[i:i + chunk]) for i in range(0, U.shape[0], chunk)])


def test_config2_block_step_full_size_every_row():
    w = wl.config2()                                   # T = 8192, Qwen shape, bf16
    sh, T = w.shape, w.T
    H, W = w.tensors["H"], w.weights[0]
    pos = wl.positions(w.cu)
    ref = oc.layer_step(H, W, w.cu, pos, sh, tau=0.0)  # the whole oracle, every row
    K = oc.keep_count(T, w.rho)
    assert K == 4915
    tau = oc.kth_largest(ref["r"], K)                  # the oracle's own threshold: exactly K of its scores stay
    m_ref = oc.select(ref["r"], w.cu, oc.THRESHOLD, tau=tau)
    c_ref = oc.compact(m_ref, w.cu, rows=[ref["Ht"]], pos_in=pos)
    assert int(m_ref.sum()) == K

    layer = dash.Layer(sh, W, DEV, tau=tau)
    bufs = StepBuffers(layer, T, 1, T, sh.dtype)
    x_full = torch.zeros(T, sh.d, dtype=sh.dtype, device=DEV)
    tok = torch.arange(T, dtype=torch.int32, device=DEV)
    dash.dash_layer_step(layer, H.to(DEV), tok, pos.to(DEV), w.cu.to(DEV), T, x_full, bufs.H_next, bufs.tok_next, bufs.pos_next, bufs.cu_next,
                         bufs.n_next, bufs.r, bufs.mask, bufs.ws)
    torch.cuda.synchronize()
    assert dash.dash_check_status() == dash.OK
    r_gpu, mask = bufs.r.cpu().numpy(), bufs.mask.cpu().numpy()
    rel = np.abs(r_gpu - ref["r"]) / ref["r"]
    record_error("cfg2 r (relative)", float(rel.max()), float(rel.max()))
    assert rel.max() < 2e-2
    # halt mask: bit-exact against the oracle's decision outside the band around its threshold, the kernel's own score inside
    flips, in_band = check_mask(mask, r_gpu, ref["r"], tau, w.cu)
    k = int(bufs.n_next.item())
    idx = np.flatnonzero(mask)
    assert k == idx.size and abs(k - K) <= flips
    assert np.array_equal(bufs.tok_next[:k].cpu().numpy(), idx) and np.array_equal(bufs.pos_next[:k].cpu().numpy(), idx)
    assert bufs.cu_next.cpu().tolist() == [0, k]
    if flips == 0:
        assert np.array_equal(idx, c_ref["idx"]) and np.array_equal(bufs.cu_next.cpu().numpy(), c_ref["cu_out"])
    # attention output of every token (an intermediate of the step: it inherits the rounding of the stored V -- an early token
    # may copy one value row almost unchanged -- i.e. up to half a bf16 ulp of the largest |v| on top of the bar)
    O = bufs.view(bufs.lay.O, T, sh.Hq * sh.D, sh.dtype).float().cpu().numpy().reshape(T, sh.Hq, sh.D)
    half_ulp_v = 2.0 ** (math.floor(math.log2(float(np.abs(ref["V"]).max()))) - 8)
    record_error("cfg2 O", *error_ratios(O, ref["O"]))
    assert_close_rms(O, ref["O"], "attention O (every row)", atol=half_ulp_v)
    # H~ of every token (tok is the identity: the step writes it to x_full)
    Ht = x_full.float().cpu().numpy()
    record_error("cfg2 H~", *error_ratios(Ht, ref["Ht"]))
    assert_close_rms(Ht, ref["Ht"], "H~ (every row)")
    assert torch.equal(bufs.H_next[:k].cpu(), x_full.cpu()[idx])        # the gather is bit-exact


def error_ratios(got, ref):
    """(max |err| / RMS of the whole reference tensor, max over rows of max |err| / RMS of that row)."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    g2, r2 = got.reshape(-1, got.shape[-1]), ref.reshape(-1, ref.shape[-1])
    err = np.max(np.abs(g2 - r2), axis=1)
    row_rms = np.sqrt(np.mean(r2 * r2, axis=1))
    return float(err.max() / math.sqrt(float(np.mean(r2 * r2)))), float(np.max(err / np.maximum(row_rms, 1e-30)))


def test_config3_cascade_full_size():
    T, L = 32768, 8
    w = wl.config3(T=T, n_layers=L)
    sh = w.shape
    Ks = [oc.keep_count(T, 1.0 - f) for f in w.fractions]
    assert Ks == [32768, 29491, 26214, 22937, 19660, 16384, 13107, 11468]
    layers = [dash.Layer(sh, w.weights[l], DEV, tau=0.0) for l in range(L)]
    A, B = StepBuffers(layers[0], T, 1, T, sh.dtype), StepBuffers(layers[0], T, 1, T, sh.dtype)
    x_full = torch.zeros(T, sh.d, dtype=sh.dtype, device=DEV)
    H, tok, pos, cu = w.tensors["H"].to(DEV), torch.arange(T, dtype=torch.int32, device=DEV), wl.positions(w.cu).to(DEV), w.cu.to(DEV)
    # layer 1 (keep-all) against the oracle on SAMPLE rows, at least one in each of its 256 query tiles
    rows = wl.sample_rows(w.cu, SAMPLE, seed=3).numpy()
    assert len(rows) == SAMPLE and len(set((rows // 128).tolist())) == T // 128
    ref = oc.layer_step(w.tensors["H"], w.weights[0], w.cu, wl.positions(w.cu), sh, attn_rows=rows)
    n_l = T
    halted_at = np.full(T, -1)
    snapshots = {}
    for l in range(L):
        out = A if l % 2 == 0 else B
        a = (H[:n_l], tok[:n_l], pos[:n_l], cu, n_l, x_full, out.H_next, out.tok_next, out.pos_next, out.cu_next, out.n_next,
             out.r, out.mask, out.ws)
        layers[l].set_tau(0.0)
        dash.dash_layer_step(layers[l], *a)                     # scores of this layer
        if l == 0:
            torch.cuda.synchronize()
            Ht0, O0 = x_full[rows].float().cpu().numpy(), out.view(out.lay.O, T, sh.Hq * sh.D, sh.dtype)[rows].float().cpu().numpy()
            record_error("cfg3 layer-1 H~ (sampled rows)", *error_ratios(Ht0, ref["Ht"]))
            record_error("cfg3 layer-1 O (sampled rows)", *error_ratios(O0.reshape(len(rows), sh.Hq, sh.D), ref["O"]))
            assert_close_rms(Ht0, ref["Ht"], "layer-1 H~ (sampled rows)")
            half_ulp_v = 2.0 ** (math.floor(math.log2(float(np.abs(ref["V"]).max()))) - 8)
            assert_close_rms(O0.reshape(len(rows), sh.Hq, sh.D), ref["O"], "layer-1 O (sampled rows)", atol=half_ulp_v)
            assert np.max(np.abs(out.r.cpu().numpy()[rows] - ref["r"]) / ref["r"]) < 2e-2
        tau = float(torch.topk(out.r[:n_l], Ks[l]).values[-1].item())
        layers[l].set_tau(tau)
        dash.dash_layer_step(layers[l], *a)
        torch.cuda.synchronize()
        k = int(out.n_next.item())
        assert k == Ks[l], (l, k, Ks[l])                        # n' sequence = floor(f_l T)
        if l == 0:
            assert torch.equal(out.H_next[:k], x_full[:k])      # keep-all: identity path
        tok_in = tok[:n_l].cpu().numpy()
        mask = out.mask[:n_l].cpu().numpy()
        tok_out = out.tok_next[:k].cpu().numpy()
        assert np.array_equal(mask, oc.select(out.r[:n_l].cpu().numpy(), [0, n_l], oc.THRESHOLD, tau=tau))   # the rule, on every row
        assert np.all(np.diff(tok_out) > 0) and np.array_equal(tok_out, tok_in[mask == 1])     # stable compaction
        assert np.array_equal(out.pos_next[:k].cpu().numpy(), tok_out)
        assert torch.equal(out.H_next[:k], x_full[torch.as_tensor(tok_out, device=DEV).long()])   # rows that go on = their rows of x_full
        halted_at[tok_in[mask == 0]] = l
        snapshots[l] = (tok_in[mask == 0], x_full[torch.as_tensor(tok_in[mask == 0], device=DEV).long()].clone())
        H, tok, pos, cu, n_l = out.H_next, out.tok_next, out.pos_next, out.cu_next, k
    assert dash.dash_check_status() == dash.OK
    # frozen states: rows of x_full of tokens halted at layer l are never written again (bit-exact)
    for l, (toks, snap) in snapshots.items():
        assert torch.equal(x_full[torch.as_tensor(toks, device=DEV).long()], snap), f"layer {l}"
    assert (halted_at >= 0).sum() == T - Ks[-1]


def test_config3_deeper_layer_shape_against_the_oracle():
    """A block step of the size and kind the cascade's fifth layer sees (19660 of 32768 tokens still active: their rows of the
    full-length buffer and their rotary positions have gaps), on drawn inputs that both sides get -- the oracle cannot follow
    the free-running cascade at this size (every layer would cost it 8e12 operations), so each deeper shape is checked on its own."""
    T, n = 32768, 19660
    w = wl.config3(T=T, n_layers=5)
    sh, W = w.shape, w.weights[4]
    g = torch.Generator().manual_seed(35)
    tok_h = torch.sort(torch.randperm(T, generator=g)[:n]).values.to(torch.int32)     # the tokens that are still active
    H = wl.hidden_states(n, sh.d, seed=35, dtype=sh.dtype)
    cu = wl.cu_from_lengths([n])
    rows = wl.sample_rows(cu, SAMPLE // 2, seed=36).numpy()
    assert len(set((rows // 128).tolist())) == (n + 127) // 128
    ref = oc.layer_step(H, W, cu, tok_h, sh, attn_rows=rows)                          # positions = the tokens' original positions
    layer = dash.Layer(sh, W, DEV, tau=0.0)
    bufs = StepBuffers(layer, n, 1, T, sh.dtype)
    x_full = torch.zeros(T, sh.d, dtype=sh.dtype, device=DEV)
    dash.dash_layer_step(layer, H.to(DEV), tok_h.to(DEV), tok_h.to(DEV), cu.to(DEV), n, x_full, bufs.H_next, bufs.tok_next, bufs.pos_next,
                         bufs.cu_next, bufs.n_next, bufs.r, bufs.mask, bufs.ws)
    torch.cuda.synchronize()
    assert dash.dash_check_status() == dash.OK
    Ht = x_full[tok_h.long().to(DEV)][rows].float().cpu().numpy()
    record_error("cfg3 layer-5 shape H~ (sampled rows)", *error_ratios(Ht, ref["Ht"]))
    assert_close_rms(Ht, ref["Ht"], "H~ at the tokens' rows of x_full (sampled rows)")
    assert np.max(np.abs(bufs.r.cpu().numpy()[rows] - ref["r"]) / ref["r"]) < 2e-2
    untouched = np.ones(T, dtype=bool)
    untouched[tok_h.numpy()] = False
    assert not x_full[torch.as_tensor(np.flatnonzero(untouched), device=DEV)].any()   # rows of halted tokens are not written
    assert int(bufs.n_next.item()) == n and torch.equal(bufs.tok_next[:n].cpu(), tok_h)


def _sparse_path(w, tau_from_oracle_K=None):
    """a1 -> a2 -> a3 (gather H~, Q, K, V) -> a4 on the GPU and in the oracle; returns both sides."""
    sh, T, S = w.shape, w.T, w.S
    Hh, Uh, Qh, Kh, Vh = (w.tensors[k] for k in ("H", "U", "Q", "K", "V"))
    r_ref = oracle_delta_norm_chunked(Uh, Hh)
    tau = w.tau if tau_from_oracle_K is None else oc.kth_largest(r_ref, tau_from_oracle_K)
    m_ref = oc.select(r_ref, w.cu, oc.THRESHOLD, tau=tau)
    cu_d = w.cu.to(DEV)
    U, H, Q, K, V = (x.to(DEV) for x in (Uh, Hh, Qh, Kh, Vh))
    mask = torch.empty(T, dtype=torch.uint8, device=DEV)
    Ht = torch.empty_like(H)
    r = dash.dash_delta_norm(U, H, Hres_out=Ht, tau=tau, cu_seqlens=cu_d, mask_out=mask)
    pos = w.tensors["pos"].to(DEV)
    tok = torch.arange(T, dtype=torch.int32, device=DEV)
    c = dash.dash_compact(mask, cu_d, rows=[Ht, Q.view(T, -1), K.view(T, -1), V.view(T, -1)], pos_in=pos, tok_in=tok)
    k = int(c["n_out"].item())
    Qc, Kc, Vc = c["rows"][1].view(T, sh.Hq, sh.D), c["rows"][2].view(T, sh.Hkv, sh.D), c["rows"][3].view(T, sh.Hkv, sh.D)
    cu_out_host = c["cu_out"].cpu()
    max_len = int((cu_out_host[1:] - cu_out_host[:-1]).max())
    O = dash.dash_varlen_attention(Qc, Kc, Vc, c["cu_out"], max(max_len, 1))
    # the arrangement `bench.py --indexed-attention` times: Q left full-length, its active rows fetched by index (tok_out),
    # K and V packed -- the same numbers bit for bit, so the oracle comparison of O below covers it too
    O_idx = dash.dash_varlen_attention_indexed(Q, Kc, Vc, c["tok_out"], c["cu_out"], max(max_len, 1), n=T, kv_packed=True)
    torch.cuda.synchronize()
    assert dash.dash_check_status() == dash.OK
    assert torch.equal(O[:k], O_idx[:k])
    return dict(r=r.cpu().numpy(), r_ref=r_ref, tau=tau, mask=mask.cpu().numpy(), m_ref=m_ref, c=c, k=k, O=O, Ht=Ht, Q=Q, K=K, V=V)


def _check_sparse(w, g, n_sample):
    sh, T = w.shape, w.T
    r_close(g["r"], g["r_ref"])
    flips, in_band = check_mask(g["mask"], g["r"], g["r_ref"], g["tau"], w.cu)
    mask, k, c = g["mask"], g["k"], g["c"]
    idx = np.flatnonzero(mask)
    assert k == idx.size
    assert np.array_equal(c["idx"][:k].cpu().numpy(), idx) and np.array_equal(c["tok_out"][:k].cpu().numpy(), idx)
    assert np.array_equal(c["pos_out"][:k].cpu().numpy(), w.tensors["pos"].numpy()[idx])
    cu_ref = np.concatenate([[0], np.cumsum([mask[int(w.cu[s]):int(w.cu[s + 1])].sum() for s in range(w.S)])])
    assert np.array_equal(c["cu_out"].cpu().numpy(), cu_ref)
    idx_d = torch.as_tensor(idx, device=DEV)
    for got, src in zip(c["rows"], (g["Ht"], g["Q"].view(T, -1), g["K"].view(T, -1), g["V"].view(T, -1))):
        assert torch.equal(got[:k], src[idx_d])                                  # bit-exact gathers
    # oracle side: its own mask, its own compaction, brute-force attention on sampled rows
    oc_c = oc.compact(g["m_ref"], w.cu, rows=[w.tensors["Q"], w.tensors["K"], w.tensors["V"]], tok_in=np.arange(T, dtype=np.int32))
    cu_o = torch.as_tensor(oc_c["cu_out"])
    rows = wl.sample_rows(cu_o, n_sample, seed=5).numpy()
    n_tiles = sum((int(cu_o[s + 1]) - int(cu_o[s]) + 127) // 128 for s in range(w.S))
    seq_of = np.searchsorted(oc_c["cu_out"], rows, side="right") - 1
    assert len({(int(s_), int((r_ - oc_c["cu_out"][s_]) // 128)) for s_, r_ in zip(seq_of, rows)}) == n_tiles     # no query tile unvisited
    O_ref, _ = oc.attention(oc_c["rows"][0], oc_c["rows"][1], oc_c["rows"][2], oc_c["cu_out"], rows=rows)
    toks = oc_c["tok_out"][rows]                                                 # token ids of the sampled rows
    where = np.searchsorted(idx, toks)                                           # their rows on the GPU side
    present = (where < k) & (idx[np.minimum(where, k - 1)] == toks)
    assert present.sum() >= len(rows) - flips
    O_gpu = g["O"][torch.as_tensor(where[present], device=DEV)].float().cpu().numpy()
    record_error(f"{w.name} O over the compacted set (sampled rows)", *error_ratios(O_gpu, O_ref[present]))
    assert_close_rms(O_gpu, O_ref[present], "attention over the compacted set (sampled rows)")
    Ht_ref = oc.residual(w.tensors["H"], w.tensors["U"])
    record_error(f"{w.name} H~", *error_ratios(g["Ht"].float().cpu().numpy(), Ht_ref))
    assert_close_rms(g["Ht"].float().cpu().numpy(), Ht_ref, "H~ (every row)")
    return flips


def test_config4_sparse_131k_full_size():
    w = wl.config4()
    K = oc.keep_count(w.T, w.rho)
    assert K == 26214
    g = _sparse_path(w, tau_from_oracle_K=K)
    flips = _check_sparse(w, g, SAMPLE)
    assert abs(g["k"] - K) <= flips
    assert abs(math.log(float(np.median(g["r"]))) + 3.0) < 0.1          # recipe: relative delta ~ LogNormal(-3, 1)


def test_config5_multimodal_varlen_full_size():
    w = wl.config5()
    g = _sparse_path(w)
    _check_sparse(w, g, SAMPLE)
    img = w.tensors["is_image"].numpy()
    halted = g["mask"] == 0
    assert 0.85 < halted[img].mean() < 0.95 and 0.05 < halted[~img].mean() < 0.15
    assert 13500 < g["k"] < 16500
