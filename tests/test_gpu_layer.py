"""GPU parity of dash_layer_step (the whole block step) against the CPU oracle,
free-running from the same seeded inputs, plus the cascaded schedule."""
import math

import numpy as np
import pytest
import torch

from oracle import dash_oracle as oc
from paper_2604_18103_b200 import dash
from paper_2604_18103_b200 import workloads as wl
from conftest import record_error
from test_gpu_kernels import assert_close_rms

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
BAND = 1e-3        # tokens whose score lies this close to the threshold may fall either way


class StepBuffers:
    def __init__(self, layer, n, S, T, dtype):
        d = layer.shape.d
        self.lay = dash.dash_layer_workspace(layer, n, S)
        self.ws = dash.workspace(self.lay.total, DEV)
        self.H_next = torch.zeros(n, d, dtype=dtype, device=DEV)
        self.tok_next = torch.zeros(n, dtype=torch.int32, device=DEV)
        self.pos_next = torch.zeros(n, dtype=torch.int32, device=DEV)
        self.cu_next = torch.zeros(S + 1, dtype=torch.int32, device=DEV)
        self.n_next = torch.zeros(1, dtype=torch.int32, device=DEV)
        self.r = torch.zeros(n, dtype=torch.float32, device=DEV)
        self.mask = torch.zeros(n, dtype=torch.uint8, device=DEV)

    def view(self, off, rows, cols, dtype):
        es = torch.tensor([], dtype=dtype).element_size()
        return self.ws[off:off + rows * cols * es].view(dtype).view(rows, cols)


def run_step(layer, H, tok, pos, cu, max_seqlen, x_full, bufs):
    dash.dash_layer_step(layer, H, tok, pos, cu, max_seqlen, x_full, bufs.H_next, bufs.tok_next, bufs.pos_next,
                         bufs.cu_next, bufs.n_next, bufs.r, bufs.mask, bufs.ws)
    torch.cuda.synchronize()
    assert dash.dash_check_status() == dash.OK


def _ratios(got, ref):
    """(max |err| / RMS of the whole reference tensor, worst row's max |err| / RMS of that row)."""
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    g2, r2 = got.reshape(-1, got.shape[-1]), ref.reshape(-1, ref.shape[-1])
    err = np.max(np.abs(g2 - r2), axis=1)
    return float(err.max() / math.sqrt(float(np.mean(r2 * r2)))), float(np.max(err / np.maximum(np.sqrt(np.mean(r2 * r2, axis=1)), 1e-30)))


def check_mask(mask_gpu, r_gpu, r_ref, tau, cu, kf=0, kl=0):
    """Bit-exact outside the band around tau; inside it the GPU decision must follow its own score."""
    ref = oc.select(r_ref, cu, oc.THRESHOLD, tau=tau, keep_first=kf, keep_last=kl)
    own = oc.select(r_gpu, cu, oc.THRESHOLD, tau=tau, keep_first=kf, keep_last=kl)
    band = np.abs(np.asarray(r_ref, dtype=np.float64) - tau) <= BAND
    assert np.array_equal(mask_gpu[~band], ref[~band]), "mask differs outside the threshold band"
    assert np.array_equal(mask_gpu, own), "mask does not follow the kernel's own scores"
    return int((mask_gpu != ref).sum()), int(band.sum())


@pytest.mark.parametrize("fold", [False, True], ids=["norm_as_a_pass", "norm_folded"])
@pytest.mark.parametrize("cfg", ["cfg1", "mini_bf16", "mini_varlen"])
def test_layer_step_matches_oracle(cfg, fold):
    if cfg == "cfg1":
        w = wl.config1()
    elif cfg == "mini_bf16":
        w = wl.config2(T=1000, seed=21, shape=wl.MINI)
    else:
        w = wl.config2(T=900, seed=22, shape=wl.MINI)
        w.cu = wl.cu_from_lengths([300, 0, 471, 129])
    sh = w.shape
    H, W = w.tensors["H"], dict(w.weights[0])
    if cfg != "cfg1":
        # a norm weight that is not all ones: folded into Wqkv by dash_fold_norm_weight, or applied by the norm's own pass
        W["rms_w"] = (1.0 + 0.2 * torch.randn(sh.d, generator=torch.Generator().manual_seed(9))).to(sh.dtype)
    T, S = w.T, w.S
    pos = wl.positions(w.cu)
    ref0 = oc.layer_step(H, W, w.cu, pos, sh, tau=0.0)
    K = oc.keep_count(T, w.rho)
    tau = oc.kth_largest(ref0["r"], K)
    ref = oc.layer_step(H, W, w.cu, pos, sh, tau=tau)

    layer = dash.Layer(sh, W, DEV, tau=tau, fold_norms=fold)
    bufs = StepBuffers(layer, T, S, T, sh.dtype)
    x_full = torch.full((T, sh.d), 9.0, dtype=sh.dtype, device=DEV)
    tok = torch.arange(T, dtype=torch.int32, device=DEV)
    run_step(layer, H.to(DEV), tok, pos.to(DEV), w.cu.to(DEV), max(int(w.cu[i + 1] - w.cu[i]) for i in range(S)), x_full, bufs)

    nq = (sh.Hq + 2 * sh.Hkv) * sh.D
    QKV = bufs.view(bufs.lay.QKV, T, nq, sh.dtype).float().cpu().numpy()
    tag = f"layer step {cfg} {'folded' if fold else 'norm pass'}"
    record_error(f"{tag} Q", *_ratios(QKV[:, :sh.Hq * sh.D], ref["Q"].reshape(T, -1)))
    record_error(f"{tag} K", *_ratios(QKV[:, sh.Hq * sh.D:(sh.Hq + sh.Hkv) * sh.D], ref["K"].reshape(T, -1)))
    record_error(f"{tag} V", *_ratios(QKV[:, (sh.Hq + sh.Hkv) * sh.D:], ref["V"].reshape(T, -1)))
    record_error(f"{tag} O", *_ratios(bufs.view(bufs.lay.O, T, sh.Hq * sh.D, sh.dtype).float().cpu().numpy().reshape(T, sh.Hq, sh.D), ref["O"]))
    record_error(f"{tag} H~", *_ratios(x_full.float().cpu().numpy(), ref["Ht"]))
    # intermediates of the step, held to the bar of its outputs: Q and K come out of the projection's accumulators rotated and are
    # rounded to the storage type once (measured: at most 0.018 x RMS, V included)
    assert_close_rms(QKV[:, :sh.Hq * sh.D], ref["Q"].reshape(T, -1), "Q (rotary applied)")
    assert_close_rms(QKV[:, sh.Hq * sh.D:(sh.Hq + sh.Hkv) * sh.D], ref["K"].reshape(T, -1), "K (rotary applied)")
    assert_close_rms(QKV[:, (sh.Hq + sh.Hkv) * sh.D:], ref["V"].reshape(T, -1), "V")
    assert_close_rms(bufs.view(bufs.lay.O, T, sh.Hq * sh.D, sh.dtype).float().cpu().numpy(), ref["O"].reshape(T, -1), "attention O",
                     atol=(2.0 ** (math.floor(math.log2(float(np.abs(ref["V"]).max()))) - 8)) if sh.dtype == torch.bfloat16 else 0.0)
    if sh.dtype == torch.float32:
        # with bf16 tensors and whole 256-column tiles the output projection adds the residual on its accumulators and U is never
        # stored (r and H~ below are what it leaves)
        assert_close_rms(bufs.view(bufs.lay.U, T, sh.d, sh.dtype).float().cpu().numpy(), ref["U"], "U")
    # H~ of every entry token reaches x_full (threshold rule: score, residual, scatter and compaction run as one pass,
    # which writes H~ there and nowhere else); tok is the identity here
    assert_close_rms(x_full.float().cpu().numpy(), ref["Ht"], "H~ (x_full)")
    r_gpu = bufs.r.cpu().numpy()
    assert np.max(np.abs(r_gpu - ref["r"]) / ref["r"]) < 2e-2
    mask = bufs.mask.cpu().numpy()
    flips, in_band = check_mask(mask, r_gpu, ref["r"], tau, w.cu)
    # the compaction that follows is exact given the mask the kernel produced
    idx = np.flatnonzero(mask)
    k = int(bufs.n_next.item())
    assert k == idx.size and abs(k - K) <= flips
    assert torch.equal(bufs.H_next[:k].cpu(), x_full.cpu()[idx])         # gathered rows are bit-exact copies
    assert np.array_equal(bufs.tok_next[:k].cpu().numpy(), idx)
    assert np.array_equal(bufs.pos_next[:k].cpu().numpy(), pos.numpy()[idx])
    cu_ref = np.concatenate([[0], np.cumsum([mask[int(w.cu[s]):int(w.cu[s + 1])].sum() for s in range(S)])])
    assert np.array_equal(bufs.cu_next.cpu().numpy(), cu_ref)
    if flips == 0:                                                       # then everything equals the oracle's own compaction
        assert np.array_equal(idx, ref["idx"]) and np.array_equal(cu_ref, ref["cu_out"])
        assert_close_rms(bufs.H_next[:k].float().cpu().numpy(), ref["rows"][0], "H_next")


def test_layer_step_keep_count_mode_and_protected_tokens():
    w = wl.config2(T=640, seed=23, shape=wl.MINI)
    sh, H, W = w.shape, w.tensors["H"], w.weights[0]
    T = w.T
    pos = wl.positions(w.cu)
    K = oc.keep_count(T, 0.667, 64, 32, mode=1)
    kc = torch.tensor([K], dtype=torch.int32, device=DEV)
    layer = dash.Layer(sh, W, DEV, sel_mode=dash.SEL_KEEP_COUNT, keep_counts=kc, keep_first=64, keep_last=32, scatter_which=0)
    bufs = StepBuffers(layer, T, 1, T, sh.dtype)
    x_full = torch.full((T, sh.d), 9.0, dtype=sh.dtype, device=DEV)
    run_step(layer, H.to(DEV), torch.arange(T, dtype=torch.int32, device=DEV), pos.to(DEV), w.cu.to(DEV), T, x_full, bufs)
    mask = bufs.mask.cpu().numpy()
    r_gpu = bufs.r.cpu().numpy()
    assert int(bufs.n_next.item()) == K == int(mask.sum()) and mask[:64].all() and mask[-32:].all()
    assert np.array_equal(mask, oc.select(r_gpu, w.cu, oc.KEEP_COUNT, keep_counts=[K], keep_first=64, keep_last=32))
    ref = oc.layer_step(H, W, w.cu, pos, sh, sel_mode=oc.KEEP_COUNT, keep_counts=[K], keep_first=64, keep_last=32)
    assert (mask != ref["mask"]).sum() <= 8            # only near-ties at the cut may differ
    # scatter_which = 0: only halted rows reach x_full, active rows stay untouched
    xf = x_full.cpu()
    Ht = bufs.view(bufs.lay.Ht, T, sh.d, sh.dtype).cpu()
    assert torch.equal(xf[mask == 0], Ht[mask == 0]) and (xf[mask == 1] == 9.0).all()


@pytest.mark.parametrize("handover", [False, True], ids=["recomputed", "handed_on"])
def test_cascade_small_matches_oracle(handover):
    """Eight layers, per-layer keep fractions of the original T (multi-shot schedule), reduced T.  handed_on: the rotary angles come
    from one table made for the whole prefill and every block takes the norm's row factors from the block in front of it
    (no pass over its input at all) instead of forming both itself."""
    T = 768
    w = wl.config3(T=T, seed=24, n_layers=8, shape=wl.MINI)
    sh = w.shape
    Ks = [oc.keep_count(T, 1.0 - f) for f in w.fractions]
    # oracle, free-running in fp64
    H_o, cu_o, pos_o, tok_o = oc.f64(w.tensors["H"]), w.cu.numpy(), wl.positions(w.cu).numpy(), np.arange(T, dtype=np.int32)
    x_o = np.zeros((T, sh.d))
    taus, r_o, tok_hist = [], [], []
    for l in range(8):
        res0 = oc.layer_step(H_o, w.weights[l], cu_o, pos_o, sh, tau=0.0)
        tau = oc.kth_largest(res0["r"], Ks[l])
        mask = oc.select(res0["r"], cu_o, oc.THRESHOLD, tau=tau)
        oc.scatter(res0["Ht"], tok_o, None, 2, x_o)
        c = oc.compact(mask, cu_o, rows=[res0["Ht"]], pos_in=pos_o, tok_in=tok_o)
        taus.append(tau); r_o.append((tok_o.copy(), res0["r"])); tok_hist.append(c["tok_out"])
        H_o, cu_o, pos_o, tok_o = c["rows"][0], c["cu_out"], c["pos_out"], c["tok_out"]
        assert c["n_out"] == Ks[l]
    # GPU, same thresholds, no host sync between layers
    layers = [dash.Layer(sh, w.weights[l], DEV, tau=taus[l]) for l in range(8)]
    A = StepBuffers(layers[0], T, 1, T, sh.dtype)
    B = StepBuffers(layers[0], T, 1, T, sh.dtype)
    x_full = torch.zeros(T, sh.d, dtype=sh.dtype, device=DEV)
    H, tok, pos, cu = w.tensors["H"].to(DEV), torch.arange(T, dtype=torch.int32, device=DEV), wl.positions(w.cu).to(DEV), w.cu.to(DEV)
    n_l, flipped = T, set()
    if handover:
        table = dash.dash_rope_table(sh.rope_base, sh.D, T, DEV)
        inv = [torch.zeros(T, dtype=torch.float32, device=DEV) for _ in range(2)]
        assert all(L.rms_folded for L in layers)
    for l in range(8):
        out = A if l % 2 == 0 else B
        if handover:      # block 0 forms its own row factors; every later block gets them from the one in front
            layers[l].set_handover(table, inv[(l - 1) % 2] if l > 0 else None, inv[l % 2])
        dash.dash_layer_step(layers[l], H[:n_l], tok[:n_l], pos[:n_l], cu, n_l, x_full, out.H_next, out.tok_next, out.pos_next,
                             out.cu_next, out.n_next, out.r, out.mask, out.ws)
        torch.cuda.synchronize()
        k = int(out.n_next.item())
        tok_gpu = tok[:n_l].cpu().numpy()
        r_gpu = out.r[:n_l].cpu().numpy()
        # scores token by token, for the tokens present on both sides
        tok_ref, r_ref = r_o[l]
        common, ia, ib = np.intersect1d(tok_gpu, tok_ref, return_indices=True)
        assert common.size >= n_l - len(flipped)
        assert np.max(np.abs(r_gpu[ia] - r_ref[ib]) / r_ref[ib]) < 3e-2
        kept_gpu = set(out.tok_next[:k].cpu().numpy().tolist())
        kept_ref = set(tok_hist[l].tolist())
        diff = kept_gpu ^ kept_ref
        near = {int(t) for t, r in zip(tok_ref, r_ref) if abs(float(r) - taus[l]) <= BAND}
        assert diff <= (near | flipped), "active sets differ outside the threshold band"
        flipped |= diff
        H, tok, pos, cu, n_l = out.H_next, out.tok_next, out.pos_next, out.cu_next, k
    assert dash.dash_check_status() == dash.OK
    assert len(flipped) <= T // 50          # a handful of in-band tokens over eight layers
    # final full-length states of every token that took the same path on both sides.  Eight
    # bf16 roundings of H~ (half an ulp = 2^-7 at |x| in [2,4)) accumulate, so the bar for
    # the whole cascade is sqrt(8) x the single-step one, with a tight RMS bound beside it.
    same = np.ones(T, dtype=bool)
    same[list(flipped)] = False
    got = x_full.float().cpu().numpy()[same]
    assert_close_rms(got, x_o[same], "x_full after the cascade", tol=2e-2 * math.sqrt(8))
    assert math.sqrt(float(np.mean((got - x_o[same]) ** 2))) < 1e-2


def test_rope_table_holds_the_angles_of_every_position():
    for base, D, n_pos in ((1.0e6, 128, 5000), (1.0e4, 64, 300)):
        t = dash.dash_rope_table(base, D, n_pos, DEV).cpu().numpy().astype(np.float64)
        ang = np.arange(n_pos, dtype=np.float64)[:, None] * base ** (-2.0 * np.arange(D // 2, dtype=np.float64) / D)[None, :]
        assert np.max(np.abs(t[..., 0] - np.cos(ang))) < 1e-6 and np.max(np.abs(t[..., 1] - np.sin(ang))) < 1e-6
    # the same rotation as the oracle's: a vector rotated with the table's entries
    x = torch.randn(7, 1, 128, generator=torch.Generator().manual_seed(5), dtype=torch.float64).numpy()
    pos = np.array([0, 1, 2, 100, 999, 4321, 4999])
    t = dash.dash_rope_table(1.0e6, 128, 5000, DEV).cpu().numpy().astype(np.float64)[pos]
    x1, x2 = x[:, 0, :64], x[:, 0, 64:]
    mine = np.concatenate([x1 * t[..., 0] - x2 * t[..., 1], x2 * t[..., 0] + x1 * t[..., 1]], axis=-1)
    assert np.max(np.abs(mine - oc.rope(x, pos, 1.0e6)[:, 0])) < 1e-5


def test_layer_step_rows_beyond_the_packed_end_and_protected_tokens():
    """Buffers allocated for more rows than the batch holds (the true count lives in cu_seqlens[S] on the device),
    poisoned rows past the end, permuted rows in the full-length buffer, protected prefix/suffix under the threshold rule."""
    w = wl.config2(T=700, seed=25, shape=wl.MINI)
    w.cu = wl.cu_from_lengths([257, 0, 443])
    sh, T, S = w.shape, w.T, w.S
    H, W = w.tensors["H"], w.weights[0]
    pos = wl.positions(w.cu)
    kf, kl, pad = 5, 3, 77
    ref0 = oc.layer_step(H, W, w.cu, pos, sh, tau=0.0)
    tau = oc.kth_largest(ref0["r"], T // 2)
    ref = oc.layer_step(H, W, w.cu, pos, sh, tau=tau, keep_first=kf, keep_last=kl)
    g = torch.Generator().manual_seed(3)
    perm = torch.randperm(T + pad, generator=g)[:T].to(torch.int32)          # rows of the tokens in the full-length buffer
    Hp = torch.cat([H, torch.full((pad, sh.d), float("nan"), dtype=sh.dtype)])
    tokp = torch.cat([perm, torch.full((pad,), 0, dtype=torch.int32)])
    posp = torch.cat([pos, torch.zeros(pad, dtype=torch.int32)])
    layer = dash.Layer(sh, W, DEV, tau=tau, keep_first=kf, keep_last=kl)
    bufs = StepBuffers(layer, T + pad, S, T + pad, sh.dtype)
    x_full = torch.full((T + pad, sh.d), 9.0, dtype=sh.dtype, device=DEV)
    run_step(layer, Hp.to(DEV), tokp.to(DEV), posp.to(DEV), w.cu.to(DEV), 443, x_full, bufs)
    mask = bufs.mask[:T].cpu().numpy()
    r_gpu = bufs.r[:T].cpu().numpy()
    assert np.max(np.abs(r_gpu - ref["r"]) / ref["r"]) < 2e-2
    flips, _ = check_mask(mask, r_gpu, ref["r"], tau, w.cu, kf, kl)
    for s in range(S):
        a, b = int(w.cu[s]), int(w.cu[s + 1])
        assert mask[a:min(a + kf, b)].all() and mask[max(b - kl, a):b].all()
    k = int(bufs.n_next.item())
    idx = np.flatnonzero(mask)
    assert k == idx.size
    xf = x_full.cpu()
    assert_close_rms(xf[perm.long()].float().numpy(), ref["Ht"], "H~ at the tokens' rows of x_full")
    untouched = np.setdiff1d(np.arange(T + pad), perm.numpy())
    assert (xf[untouched] == 9.0).all()                                      # nothing written for rows past the packed end
    assert torch.equal(bufs.H_next[:k].cpu(), xf[perm.long()][idx])
    assert np.array_equal(bufs.tok_next[:k].cpu().numpy(), perm.numpy()[idx])
    assert np.array_equal(bufs.pos_next[:k].cpu().numpy(), pos.numpy()[idx])
    cu_ref = np.concatenate([[0], np.cumsum([mask[int(w.cu[s]):int(w.cu[s + 1])].sum() for s in range(S)])])
    assert np.array_equal(bufs.cu_next.cpu().numpy(), cu_ref)
    if flips == 0:
        assert np.array_equal(mask, ref["mask"])
