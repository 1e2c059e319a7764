"""GPU parity: every C-ABI kernel against the CPU oracle, element by element, on
seeded inputs that span several tiles and a ragged tail, plus the edge cases
(empty input, empty sequences, keep-all / keep-none, protected tokens, ties)."""
import math

import numpy as np
import pytest
import torch

from oracle import dash_oracle as oc
from paper_2604_18103_b200 import dash
from paper_2604_18103_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

# Floating-point bar: max |err| <= 2e-2 * RMS(reference), bf16 operands with fp32 accumulation.
# RMS(reference) is the RMS of the whole reference tensor, except for output vectors (a token's
# row of a state tensor, a (token, head) row of the attention output) whose own RMS is larger:
# under causal attention the row norms fall like 1/sqrt(i), the tensor-wide RMS sits below half a
# bf16 ulp of the early rows (|O| ~ 3 -> 2^-7), and there even an exactly rounded bf16 result
# would miss a tensor-wide bar; such rows are held to 2e-2 of their own RMS instead.
TOL = 2e-2


def assert_close_rms(got, ref, what, tol=TOL, atol=0.0):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    if ref.size == 0:
        return
    g2, r2 = got.reshape(-1, got.shape[-1]), ref.reshape(-1, ref.shape[-1])
    rms = np.maximum(np.sqrt(np.mean(r2 * r2, axis=1)), math.sqrt(float(np.mean(r2 * r2))))
    err = np.max(np.abs(g2 - r2), axis=1)
    worst = int(np.argmax(err - tol * rms))
    assert np.all(err <= tol * rms + atol + 1e-30), (f"{what}: row {worst}: max|err| {err[worst]:.3e} > {tol} * RMS {rms[worst]:.3e} "
                                               f"({int(np.sum(err > tol * rms))} of {err.size} rows fail)")


def r_close(r_gpu, r_ref):
    r_gpu, r_ref = np.asarray(r_gpu, dtype=np.float64), np.asarray(r_ref, dtype=np.float64)
    assert np.all(np.abs(r_gpu - r_ref) <= 1e-5 * np.abs(r_ref) + 1e-7), float(np.max(np.abs(r_gpu - r_ref)))


@pytest.fixture(autouse=True)
def _status_clean():
    yield
    assert dash.dash_check_status() == dash.OK


# ------------------------------------------------------------------ step 1
@pytest.mark.parametrize("dtype,n,d", [(torch.bfloat16, 1000, 3584), (torch.float32, 1024, 256), (torch.bfloat16, 37, 520),
                                       (torch.float32, 5, 8), (torch.bfloat16, 0, 64)])
def test_delta_norm_matches_oracle(dtype, n, d):
    g = torch.Generator().manual_seed(n + d)
    U = (torch.randn(n, d, generator=g) * 0.1).to(dtype)
    H = torch.randn(n, d, generator=g).to(dtype)
    Ud, Hd = U.to(DEV), H.to(DEV)
    for mode in (dash.NORM_REL, dash.NORM_ABS):
        Ht = torch.empty_like(Hd)
        r = dash.dash_delta_norm(Ud, Hd, mode=mode, Hres_out=Ht)
        r_close(r.cpu().numpy(), oc.delta_norm(U, H, mode=mode))
        if n:
            assert_close_rms(Ht.float().cpu().numpy(), oc.residual(H, U), "H~")
    # without the residual output, and with an indexed residual destination
    r2 = dash.dash_delta_norm(Ud, Hd)
    r_close(r2.cpu().numpy(), oc.delta_norm(U, H))
    if n:
        perm = torch.randperm(n, generator=g).to(torch.int32)
        full = torch.zeros(n, d, dtype=dtype, device=DEV)
        dash.dash_delta_norm(Ud, Hd, Hres_out=full, res_index=perm.to(DEV))
        ref = torch.empty_like(Ht)
        dash.dash_delta_norm(Ud, Hd, Hres_out=ref)
        assert torch.equal(full[perm.long().to(DEV)], ref)


def test_delta_norm_residual_written_over_an_input():
    """H~ = H + U written over H itself (and, second call, over U): every vector is read before it is written."""
    g = torch.Generator().manual_seed(77)
    n, d = 1500, 1024
    U = (torch.randn(n, d, generator=g) * 0.2).to(torch.bfloat16)
    H = torch.randn(n, d, generator=g).to(torch.bfloat16)
    ref_r, ref_Ht = oc.delta_norm(U, H), oc.residual(H, U)
    for over in ("H", "U"):
        Ud, Hd = U.to(DEV), H.to(DEV)
        r = dash.dash_delta_norm(Ud, Hd, Hres_out=Hd if over == "H" else Ud)
        r_close(r.cpu().numpy(), ref_r)
        assert_close_rms((Hd if over == "H" else Ud).float().cpu().numpy(), ref_Ht, f"H~ over {over}")
    # an indexed destination inside an input is refused (a row could be read after another row's result landed on it)
    with pytest.raises(dash.DashError):
        dash.dash_delta_norm(U.to(DEV), Hd, Hres_out=Hd, res_index=torch.arange(n, dtype=torch.int32, device=DEV))


def test_fold_norm_weight_is_the_once_rounded_product():
    """W_out[i, j] = w[i] * W[i, j]: the product of two bf16 values is exact in fp32, so the result is that product rounded once."""
    g = torch.Generator().manual_seed(78)
    for dtype, d, N in ((torch.bfloat16, 520, 1536), (torch.float32, 64, 100)):
        W = (torch.randn(d, N, generator=g) * 0.02).to(dtype)
        w = (1.0 + 0.3 * torch.randn(d, generator=g)).to(dtype)
        want = torch.from_numpy(oc.f64(w)[:, None] * oc.f64(W)).to(dtype)       # fp64 product, rounded once to the storage type
        Wd = W.to(DEV)
        out = dash.dash_fold_norm_weight(Wd, w.to(DEV))
        assert torch.equal(out.cpu(), want)
        dash.dash_fold_norm_weight(Wd, w.to(DEV), out=Wd)                        # in place
        assert torch.equal(Wd.cpu(), want)


def test_lookback_wait_gives_up_reports_timeout_and_the_library_carries_on():
    """Every device-side wait is bounded.  The test hook starts the compaction's tile ticket at 1: tile 0 is never taken and the
    tile behind it polls a state word that nobody publishes, runs out of polls, reports DASH_ERR_TIMEOUT through the status word
    and lets the other tiles finish.  The word clears on reading, and the next ordinary call is correct."""
    cu = wl.cu_from_lengths([40000, 7])
    n = int(cu[-1])
    mask = wl.random_mask(n, 0.5, seed=91)
    out = dash.dash_testing_compact_stalled(mask.to(DEV), cu.to(DEV), spin_limit=1000)
    torch.cuda.synchronize()                                                      # the kernel returned
    assert dash.dash_check_status() == 5 and dash.lib().dash_status_string(5) == b"a device-side wait gave up"
    assert dash.dash_check_status() == dash.OK                                    # reported once, then clear
    assert 0 <= int(out["n_out"].item()) <= n
    # an ordinary call of the same size (look-back path) right behind it
    X = torch.randn(n, 64, generator=torch.Generator().manual_seed(92)).to(torch.bfloat16)
    got = dash.dash_compact(mask.to(DEV), cu.to(DEV), rows=[X.to(DEV)], pos_in=wl.positions(cu).to(DEV))
    ref = oc.compact(mask, cu, rows=[X], pos_in=wl.positions(cu))
    k = ref["n_out"]
    assert int(got["n_out"].item()) == k and np.array_equal(got["idx"][:k].cpu().numpy(), ref["idx"])
    assert np.array_equal(got["cu_out"].cpu().numpy(), ref["cu_out"]) and torch.equal(got["rows"][0][:k].cpu(), ref["rows"][0])
    assert dash.dash_check_status() == dash.OK


def test_delta_norm_strided_rows_and_fused_threshold():
    g = torch.Generator().manual_seed(5)
    n, d = 777, 256
    big = torch.randn(n, 2 * d, generator=g).to(torch.bfloat16)
    U, H = big[:, :d], big[:, d:]                    # row stride 2d
    cu = torch.tensor([0, 100, 100, 500, 777], dtype=torch.int32)
    r_ref = oc.delta_norm(U, H)
    tau = float(np.median(r_ref))
    bd = big.to(DEV)
    mask = torch.empty(n, dtype=torch.uint8, device=DEV)
    r = dash.dash_delta_norm(bd[:, :d], bd[:, d:], tau=tau, cu_seqlens=cu.to(DEV), keep_first=3, keep_last=2, mask_out=mask)
    r_close(r.cpu().numpy(), r_ref)
    m_ref = oc.select(r.cpu().numpy(), cu, oc.THRESHOLD, tau=tau, keep_first=3, keep_last=2)
    assert np.array_equal(mask.cpu().numpy(), m_ref)
    # device-side row count: rows past it are left alone
    r_out = torch.full((n,), -1.0, device=DEV)
    dash.dash_delta_norm(bd[:, :d], bd[:, d:], r_out=r_out, n_dev=torch.tensor([500], dtype=torch.int32, device=DEV))
    assert (r_out[500:] == -1).all() and (r_out[:500] >= 0).all()


# ------------------------------------------------------------------ step 2
@pytest.mark.parametrize("lengths", [[5000], [300, 0, 1700, 1], [131072]])
def test_select_matches_oracle(lengths):
    cu = wl.cu_from_lengths(lengths)
    n = int(cu[-1])
    g = torch.Generator().manual_seed(n)
    r = torch.exp(torch.randn(n, generator=g) - 3.0)
    r[::97] = r[5]                                             # ties, some at the cut
    if n > 10:
        r[7] = float("nan")
    rd, cud = r.to(DEV), cu.to(DEV)
    for kf, kl in ((0, 0), (64, 32)):
        tau = float(np.quantile(r[~torch.isnan(r)].numpy(), 0.4))
        m = dash.dash_select(rd, cud, dash.SEL_THRESHOLD, tau=tau, keep_first=kf, keep_last=kl)
        assert np.array_equal(m.cpu().numpy(), oc.select(r.numpy(), cu, oc.THRESHOLD, tau=tau, keep_first=kf, keep_last=kl))
        for frac in (0.0, 0.37, 1.0):
            Ks = [int(frac * L) for L in lengths]
            m = dash.dash_select(rd, cud, dash.SEL_KEEP_COUNT, keep_counts=torch.tensor(Ks, dtype=torch.int32, device=DEV),
                                 keep_first=kf, keep_last=kl)
            ref = oc.select(r.numpy(), cu, oc.KEEP_COUNT, keep_counts=Ks, keep_first=kf, keep_last=kl)
            assert np.array_equal(m.cpu().numpy(), ref), (lengths, kf, kl, frac)


def test_keep_counts_on_the_device_equal_the_oracle_and_feed_the_keep_count_rule():
    """Kept lengths computed on the device from cu_seqlens (Eq. 3 and the Appendix-A rule): bit-equal to the oracle's for the
    paper's prompt lengths, for random lengths and for the degenerate ones; then used by the keep-count rule without a host copy."""
    g = torch.Generator().manual_seed(77)
    lengths = [8192, 16384, 32768, 65536, 131072, 0, 1, 95, 96, 97] + torch.randint(0, 200000, (300,), generator=g).tolist()
    cu = wl.cu_from_lengths(lengths).to(DEV)
    for rho, kf, kl, mode in ((0.4, 0, 0, 0), (0.667, 64, 32, 1), (0.5, 64, 32, 1), (0.0, 0, 0, 0), (0.999, 3, 5, 1), (0.8, 0, 0, 0)):
        got = dash.dash_keep_counts_device(cu, rho, kf, kl, mode).cpu().tolist()
        assert got == [oc.keep_count(L, rho, kf, kl, mode) for L in lengths], (rho, kf, kl, mode)
    lengths = [5000, 300, 0, 1700]
    cu_h = wl.cu_from_lengths(lengths)
    n = int(cu_h[-1])
    r = torch.exp(torch.randn(n, generator=g) - 3.0)
    Kd = dash.dash_keep_counts_device(cu_h.to(DEV), 0.667, 64, 32, 1)
    m = dash.dash_select(r.to(DEV), cu_h.to(DEV), dash.SEL_KEEP_COUNT, keep_counts=Kd, keep_first=64, keep_last=32)
    Ks = [oc.keep_count(L, 0.667, 64, 32, 1) for L in lengths]
    assert np.array_equal(m.cpu().numpy(), oc.select(r.numpy(), cu_h, oc.KEEP_COUNT, keep_counts=Ks, keep_first=64, keep_last=32))


def test_select_high_direction_matches_oracle():
    lengths = [300, 0, 1700, 1]
    cu = wl.cu_from_lengths(lengths)
    n = int(cu[-1])
    g = torch.Generator().manual_seed(13)
    r = torch.rand(n, generator=g)
    r[5] = float("nan")
    rd, cud = r.to(DEV), cu.to(DEV)
    m = dash.dash_select(rd, cud, dash.SEL_THRESHOLD_HALT_HIGH, tau=0.6, keep_first=4, keep_last=2)
    assert np.array_equal(m.cpu().numpy(), oc.select(r.numpy(), cu, oc.THRESHOLD, tau=0.6, keep_first=4, keep_last=2, halt_high=True))
    K = [100, 0, 1234, 1]
    m = dash.dash_select(rd, cud, dash.SEL_KEEP_COUNT_HALT_HIGH, keep_counts=torch.tensor(K, dtype=torch.int32, device=DEV), keep_first=4, keep_last=2)
    ref = oc.select(r.numpy(), cu, oc.KEEP_COUNT, keep_counts=K, keep_first=4, keep_last=2, halt_high=True)
    assert np.array_equal(m.cpu().numpy(), ref)
    assert m.cpu().numpy()[5] == 1                                           # NaN stays in either direction


def test_select_all_equal_scores_keeps_lowest_indices():
    n = 4096
    r = torch.full((n,), 0.25)
    cu = torch.tensor([0, n], dtype=torch.int32)
    m = dash.dash_select(r.to(DEV), cu.to(DEV), dash.SEL_KEEP_COUNT, keep_counts=torch.tensor([1000], dtype=torch.int32, device=DEV))
    assert m[:1000].all() and not m[1000:].any()


# ------------------------------------------------------------------ step 3
@pytest.mark.parametrize("lengths,keep", [([8192], 0.6), ([300, 0, 1700, 1, 999], 0.3), ([70000], 0.2), ([33], 1.0), ([257], 0.0)])
def test_compact_and_scatter_match_oracle(lengths, keep):
    cu = wl.cu_from_lengths(lengths)
    n = int(cu[-1])
    mask = wl.random_mask(n, keep, seed=n)
    g = torch.Generator().manual_seed(n + 1)
    X = torch.randn(n, 384, generator=g).to(torch.bfloat16)          # 768-byte rows (16-byte path)
    Y = torch.randn(n, 5, generator=g)                               # 20-byte rows (4-byte path)
    pos = wl.positions(cu)
    tok = (torch.randperm(n, generator=g) + 7).to(torch.int32)
    ref = oc.compact(mask, cu, rows=[X, Y], pos_in=pos, tok_in=tok)
    out = dash.dash_compact(mask.to(DEV), cu.to(DEV), rows=[X.to(DEV), Y.to(DEV)], pos_in=pos.to(DEV), tok_in=tok.to(DEV))
    k = int(out["n_out"].item())
    assert k == ref["n_out"] == int(mask.sum())
    assert np.array_equal(out["cu_out"].cpu().numpy(), ref["cu_out"])
    assert np.array_equal(out["idx"][:k].cpu().numpy(), ref["idx"])
    assert np.array_equal(out["pos_out"][:k].cpu().numpy(), ref["pos_out"])
    assert np.array_equal(out["tok_out"][:k].cpu().numpy(), ref["tok_out"])
    assert torch.equal(out["rows"][0][:k].cpu(), ref["rows"][0])
    assert torch.equal(out["rows"][1][:k].cpu(), ref["rows"][1])
    # scatter the compacted rows back by their original row; halted rows by the mask
    full = torch.full((n + 7, 384), 3.0, dtype=torch.bfloat16, device=DEV)
    dash.dash_scatter(out["rows"][0], full, tok_index=out["idx"], which=2, n_dev=out["n_out"])
    full_ref = torch.full((n + 7, 384), 3.0, dtype=torch.bfloat16)
    oc.scatter(ref["rows"][0], ref["idx"], None, 2, full_ref)
    assert torch.equal(full.cpu(), full_ref)
    for which in (0, 1):
        f2 = torch.zeros(n + 7, 384, dtype=torch.bfloat16, device=DEV)
        dash.dash_scatter(X.to(DEV), f2, tok_index=tok.to(DEV) - 7, sel=mask.to(DEV), which=which)
        f2_ref = torch.zeros(n + 7, 384, dtype=torch.bfloat16)
        oc.scatter(X, tok - 7, mask, which, f2_ref)
        assert torch.equal(f2.cpu(), f2_ref)


def test_compact_empty_input():
    cu = torch.tensor([0, 0, 0], dtype=torch.int32)
    out = dash.dash_compact(torch.zeros(0, dtype=torch.uint8, device=DEV), cu.to(DEV))
    assert int(out["n_out"].item()) == 0 and not out["cu_out"].cpu().any()


# ------------------------------------------------------------------ step 4
def _attention_case(lengths, Hq, Hkv, D, dtype, seed, rows=None, pad=0, tol=TOL, key_gain=None):
    cu = wl.cu_from_lengths(lengths)
    n = int(cu[-1])
    g = torch.Generator().manual_seed(seed)
    Q = torch.randn(n + pad, Hq, D, generator=g).to(dtype)
    K = torch.randn(n + pad, Hkv, D, generator=g).to(dtype)
    V = torch.randn(n + pad, Hkv, D, generator=g).to(dtype)
    if key_gain is not None:     # keys from position `at` of every sequence on are `gain` times longer
        pos = wl.positions(cu).long()
        for at, gain in key_gain:
            K[:n][pos >= at] *= gain
    if pad:          # rows past the packed end hold poison that must never reach an output
        Q[n:], K[n:], V[n:] = float("nan"), float("inf"), float("nan")
    O, lse = dash.dash_varlen_attention(Q.to(DEV), K.to(DEV), V.to(DEV), cu.to(DEV), max(lengths), want_lse=True)
    torch.cuda.synchronize()
    Oref, lref = oc.attention(Q[:n], K[:n], V[:n], cu, rows=rows)
    sel = slice(0, n) if rows is None else torch.as_tensor(rows)
    assert_close_rms(O[:n].float().cpu().numpy()[sel], Oref, f"O {lengths} Hq{Hq} D{D}", tol=tol)
    got_lse = lse[:, :n].cpu().numpy().T[sel]
    assert np.allclose(got_lse, lref, atol=2e-2), float(np.max(np.abs(got_lse - lref)))


def _indexed_attention_case(full_lengths, keep_prob, Hq, Hkv, D, seed, tol=TOL):
    """Full-length Q, K, V with a random subset of every sequence active; the rows that are not active hold NaN / Inf, so any
    read of them would show.  The index-driven kernel must equal the oracle's attention over the gathered rows."""
    g = torch.Generator().manual_seed(seed)
    cu_full = wl.cu_from_lengths(full_lengths)
    n_full = int(cu_full[-1])
    mask = torch.rand(n_full, generator=g) < keep_prob
    idx = torch.nonzero(mask).flatten().to(torch.int32)
    lengths = [int(mask[int(cu_full[s]):int(cu_full[s + 1])].sum()) for s in range(len(full_lengths))]
    cu = wl.cu_from_lengths(lengths)
    n = int(cu[-1])
    Q = torch.randn(n_full, Hq, D, generator=g).to(torch.bfloat16)
    K = torch.randn(n_full, Hkv, D, generator=g).to(torch.bfloat16)
    V = torch.randn(n_full, Hkv, D, generator=g).to(torch.bfloat16)
    Qp, Kp, Vp = Q.clone(), K.clone(), V.clone()
    Qp[~mask], Kp[~mask], Vp[~mask] = float("nan"), float("inf"), float("nan")
    O, lse = dash.dash_varlen_attention_indexed(Qp.to(DEV), Kp.to(DEV), Vp.to(DEV), idx.to(DEV), cu.to(DEV), max(max(lengths), 1), want_lse=True)
    torch.cuda.synchronize()
    assert dash.dash_check_status() == dash.OK
    sel = idx.long()
    Oref, lref = oc.attention(Q[sel], K[sel], V[sel], cu)
    assert_close_rms(O.float().cpu().numpy(), Oref, f"indexed O {full_lengths} keep {keep_prob} Hq{Hq} D{D}", tol=tol)
    assert np.allclose(lse.cpu().numpy().T, lref, atol=2e-2)
    # the same numbers as the kernel on packed copies of the active rows (same arithmetic, other loads)
    Kc, Vc = K[sel].contiguous().to(DEV), V[sel].contiguous().to(DEV)
    O2 = dash.dash_varlen_attention(Q[sel].contiguous().to(DEV), Kc, Vc, cu.to(DEV), max(max(lengths), 1))
    assert torch.equal(O.cpu(), O2.cpu())
    # Q by index, K and V packed by the caller
    O3 = dash.dash_varlen_attention_indexed(Qp.to(DEV), Kc, Vc, idx.to(DEV), cu.to(DEV), max(max(lengths), 1), kv_packed=True)
    assert torch.equal(O.cpu(), O3.cpu())


def test_indexed_attention_ragged_tiles_gqa():
    _indexed_attention_case([700], 0.45, 4, 2, 128, 21)


def test_indexed_attention_packed_batch_with_an_empty_active_set():
    _indexed_attention_case([400, 130, 3, 900], 0.3, 14, 2, 128, 22)


def test_indexed_attention_head_dim_64_and_keep_all():
    _indexed_attention_case([517], 1.1, 4, 4, 64, 23)


def test_indexed_attention_random_shapes_equal_the_packed_kernel():
    """Seeded sweep: sequence counts, lengths (also multiples of the tile), keep fractions from 5 % to all, head groupings,
    head dims; the index-driven kernel (both arrangements of K, V) must reproduce the packed kernel bit for bit."""
    g = torch.Generator().manual_seed(2025)
    for trial in range(12):
        S = int(torch.randint(1, 6, (1,), generator=g))
        full = torch.randint(1, 1500, (S,), generator=g).tolist()
        if trial % 5 == 0:
            full = [128 * int(torch.randint(1, 8, (1,), generator=g)) for _ in range(S)]
        keep = [0.05, 0.3, 0.7, 1.1][trial % 4]
        Hkv, G, D = [1, 2, 4][trial % 3], [1, 2, 7][trial % 3], [128, 64][trial % 2]
        Hq = Hkv * G
        cu_full = wl.cu_from_lengths(full)
        n_full = int(cu_full[-1])
        mask = torch.rand(n_full, generator=g) < keep
        idx = torch.nonzero(mask).flatten().to(torch.int32)
        lens = [int(mask[int(cu_full[s]):int(cu_full[s + 1])].sum()) for s in range(S)]
        cu = wl.cu_from_lengths(lens)
        if int(cu[-1]) == 0:
            continue
        Q = torch.randn(n_full, Hq, D, generator=g).to(torch.bfloat16)
        K = torch.randn(n_full, Hkv, D, generator=g).to(torch.bfloat16)
        V = torch.randn(n_full, Hkv, D, generator=g).to(torch.bfloat16)
        Qp, Kp, Vp = Q.clone(), K.clone(), V.clone()
        Qp[~mask], Kp[~mask], Vp[~mask] = float("nan"), float("inf"), float("nan")
        sel, ms = idx.long(), max(max(lens), 1)
        Kc, Vc = K[sel].contiguous().to(DEV), V[sel].contiguous().to(DEV)
        O1 = dash.dash_varlen_attention(Q[sel].contiguous().to(DEV), Kc, Vc, cu.to(DEV), ms)
        O2 = dash.dash_varlen_attention_indexed(Qp.to(DEV), Kp.to(DEV), Vp.to(DEV), idx.to(DEV), cu.to(DEV), ms)
        O3 = dash.dash_varlen_attention_indexed(Qp.to(DEV), Kc, Vc, idx.to(DEV), cu.to(DEV), ms, kv_packed=True)
        torch.cuda.synchronize()
        assert dash.dash_check_status() == dash.OK
        assert torch.isfinite(O1.float()).all() and torch.equal(O1, O2) and torch.equal(O1, O3), (trial, full, keep)


def test_attention_single_tile():
    _attention_case([128], 1, 1, 128, torch.bfloat16, 1)


def test_attention_ragged_multi_tile_gqa():
    _attention_case([300], 4, 2, 128, torch.bfloat16, 2)


def test_attention_varlen_with_empty_and_short_sequences_and_poisoned_tail():
    _attention_case([129, 0, 1, 515, 64], 14, 2, 128, torch.bfloat16, 3, pad=200)


def test_attention_scores_that_tower_over_the_first_key_block():
    # The kernel keeps the first key block's row maximum as the reference of the exponentials and only moves it when a block's
    # sum says it must.  Here later keys are 40, then 100 times longer: scores tens of units above everything before them, the
    # jumps falling into the second half of a block (position 200), the first half (position 650) and a block's first key (1024).
    _attention_case([1500, 700], 4, 2, 128, torch.bfloat16, 21, key_gain=[(200, 40.0), (650, 2.5), (1024, 3.0)])
    _attention_case([900], 2, 1, 64, torch.bfloat16, 22, key_gain=[(130, 60.0)], pad=4)
    # and the other way round: the first block's keys are the long ones, everything behind them all but vanishes against the reference
    _attention_case([700], 4, 2, 128, torch.bfloat16, 23, key_gain=[(0, 50.0), (128, 0.02)])


def test_attention_head_dim_64_fp32():
    # fp32 tensors are rounded to bf16 operands on the way in: on top of the bf16 rounding of P
    # (2^-9 p |v|) comes that of V (another 2^-9 p |v|) and of Q, K; with unit-variance inputs and
    # a dominant key (p ~ 1, |v| up to 4.5) the stack reaches 2.2e-2 of the row's RMS.
    _attention_case([1024], 4, 4, 64, torch.float32, 4, tol=3e-2)


def test_attention_head_dim_64_bf16_gqa():
    _attention_case([700, 333], 6, 2, 64, torch.bfloat16, 5, pad=5)


def test_attention_qwen_heads_sampled_rows():
    lengths = [2500, 1100]
    rows = wl.sample_rows(wl.cu_from_lengths(lengths), 160, seed=6)
    _attention_case(lengths, 28, 4, 128, torch.bfloat16, 6, rows=rows.numpy())


def test_attention_many_short_sequences_some_empty():
    # 150 sequences of 0..200 tokens: more work items than persistent CTAs, most query tiles ragged
    g = torch.Generator().manual_seed(11)
    lengths = torch.randint(0, 201, (150,), generator=g).tolist()
    lengths[7] = lengths[80] = 0
    _attention_case(lengths, 4, 2, 128, torch.bfloat16, 11, pad=3)


def test_attention_one_long_sequence_more_than_1024_query_tiles():
    # 1031 query tiles: the plan of work items is built in more than one pass over the tile levels
    n = 1031 * 128 - 5
    rows = wl.sample_rows(wl.cu_from_lengths([n]), 48, seed=12)
    _attention_case([n], 1, 1, 64, torch.bfloat16, 12, rows=rows.numpy())


def test_attention_closed_forms_on_device():
    # V constant -> O constant; Q = 0 -> prefix mean (uniform weights)
    n, Hq, Hkv, D = 400, 2, 1, 128
    g = torch.Generator().manual_seed(9)
    K = torch.randn(n, Hkv, D, generator=g).to(torch.bfloat16).to(DEV)
    V = torch.randn(n, Hkv, D, generator=g).to(torch.bfloat16).to(DEV)
    Q = torch.randn(n, Hq, D, generator=g).to(torch.bfloat16).to(DEV)
    cu = torch.tensor([0, n], dtype=torch.int32, device=DEV)
    O = dash.dash_varlen_attention(Q, K, torch.full_like(V, 1.5), cu, n)
    assert torch.allclose(O.float(), torch.full_like(O, 1.5).float(), atol=2e-2)
    O = dash.dash_varlen_attention(torch.zeros_like(Q), K, V, cu, n)
    pm = torch.cumsum(V.float()[:, 0], 0) / torch.arange(1, n + 1, device=DEV)[:, None]
    assert torch.allclose(O.float()[:, 1], pm, atol=2e-2)


# ------------------------------------------------------------------ randomized sweeps (seeded)
def test_select_compact_scatter_random_shapes_match_oracle():
    """Thirty seeded draws of batch structure, keep ratio, rule and protected tokens: select, compaction and scatter against the oracle."""
    g = torch.Generator().manual_seed(2024)
    for trial in range(30):
        S = int(torch.randint(1, 7, (1,), generator=g))
        lengths = [int(x) for x in torch.randint(0, [40, 400, 5000, 40000][trial % 4], (S,), generator=g)]
        if sum(lengths) == 0:
            lengths[0] = 17
        cu = wl.cu_from_lengths(lengths)
        n = int(cu[-1])
        r = torch.rand(n, generator=g)
        kf, kl = int(torch.randint(0, 5, (1,), generator=g)), int(torch.randint(0, 5, (1,), generator=g))
        mode = [dash.SEL_THRESHOLD, dash.SEL_KEEP_COUNT, dash.SEL_THRESHOLD_HALT_HIGH, dash.SEL_KEEP_COUNT_HALT_HIGH][trial % 4]
        keep = float(torch.rand(1, generator=g))
        K = [min(L, int(keep * L) + int(torch.randint(0, 3, (1,), generator=g))) for L in lengths]
        kc = torch.tensor(K, dtype=torch.int32, device=DEV)
        m = dash.dash_select(r.to(DEV), cu.to(DEV), mode, tau=keep, keep_counts=kc, keep_first=kf, keep_last=kl)
        ref = oc.select(r.numpy(), cu, oc.THRESHOLD if mode in (dash.SEL_THRESHOLD, dash.SEL_THRESHOLD_HALT_HIGH) else oc.KEEP_COUNT,
                        tau=keep, keep_counts=K, keep_first=kf, keep_last=kl, halt_high=mode >= 2)
        assert np.array_equal(m.cpu().numpy(), ref), (trial, lengths, mode)
        d = [8, 24, 256, 520][trial % 4]
        X = torch.randn(n, d, generator=g).to(torch.bfloat16 if trial % 2 else torch.float32)
        pos = wl.positions(cu)
        tok = torch.randperm(n, generator=g).to(torch.int32)
        c = dash.dash_compact(m, cu.to(DEV), rows=[X.to(DEV)], pos_in=pos.to(DEV), tok_in=tok.to(DEV))
        o = oc.compact(ref, cu, rows=[X], pos_in=pos, tok_in=tok)
        k = int(c["n_out"].item())
        assert k == o["n_out"] and np.array_equal(c["cu_out"].cpu().numpy(), o["cu_out"]), (trial, lengths)
        assert np.array_equal(c["idx"][:k].cpu().numpy(), o["idx"])
        assert torch.equal(c["rows"][0][:k].cpu(), o["rows"][0])
        assert np.array_equal(c["pos_out"][:k].cpu().numpy(), o["pos_out"]) and np.array_equal(c["tok_out"][:k].cpu().numpy(), o["tok_out"])
        full = torch.zeros(n, d, dtype=X.dtype, device=DEV)
        dash.dash_scatter(X.to(DEV), full, tok_index=tok.to(DEV), sel=m, which=trial % 3)
        want = oc.scatter(X, tok, ref, trial % 3, torch.zeros(n, d, dtype=X.dtype))
        assert torch.equal(full.cpu(), want), (trial, "scatter")


def test_attention_random_packed_batches_match_oracle_on_sampled_rows():
    g = torch.Generator().manual_seed(77)
    for trial in range(6):
        S = int(torch.randint(1, 6, (1,), generator=g))
        lengths = [int(x) for x in torch.randint(0, 900, (S,), generator=g)]
        if sum(lengths) == 0:
            lengths[0] = 130
        Hkv = [1, 2, 4][trial % 3]
        Hq = Hkv * [1, 3, 7][trial % 3]
        D = 128 if trial % 2 else 64
        rows = wl.sample_rows(wl.cu_from_lengths(lengths), 60, seed=trial)
        _attention_case(lengths, Hq, Hkv, D, torch.bfloat16, 100 + trial, rows=rows.numpy(), pad=trial)
