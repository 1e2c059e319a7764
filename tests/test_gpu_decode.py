"""GPU parity of the decoding-stage attention over the packed (shortened) KV cache against the CPU oracle, and of the
KV-cache rows a block step emits."""
import numpy as np
import pytest
import torch

from oracle import dash_oracle as oc
from paper_2604_18103_b200 import dash
from paper_2604_18103_b200 import workloads as wl
from test_gpu_kernels import assert_close_rms

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(autouse=True)
def _status_clean():
    yield
    assert dash.dash_check_status() == dash.OK


def _decode_case(lengths, Hq, Hkv, D, seed, pad=0):
    cu = wl.cu_from_lengths(lengths)
    n, S = int(cu[-1]), len(lengths)
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(S, Hq, D, generator=g).to(torch.bfloat16)
    K = torch.randn(n + pad, Hkv, D, generator=g).to(torch.bfloat16)
    V = torch.randn(n + pad, Hkv, D, generator=g).to(torch.bfloat16)
    if pad:                      # rows past the packed end hold poison that must never reach an output
        K[n:], V[n:] = float("inf"), float("nan")
    out, lse = dash.dash_decode_attention(q.to(DEV), K.to(DEV), V.to(DEV), cu.to(DEV), want_lse=True)
    torch.cuda.synchronize()
    Oref, lref = oc.decode_attention(q, K[:n], V[:n], cu)
    assert_close_rms(out.float().cpu().numpy(), Oref, f"decode O {lengths[:6]} Hq{Hq} D{D}")
    got = lse.cpu().numpy()
    live = np.isfinite(lref)
    assert np.allclose(got[live], lref[live], atol=2e-2) and np.all(np.isinf(got[~live]) & (got[~live] < 0))


def test_decode_single_sequence_ragged_blocks():
    _decode_case([300], 4, 2, 128, 1)


def test_decode_batch_with_empty_short_and_long_caches_and_poisoned_tail():
    _decode_case([129, 0, 1, 5000, 64, 128], 14, 2, 128, 2, pad=130)


def test_decode_qwen_heads_long_cache_split_over_many_ctas():
    _decode_case([100000], 28, 4, 128, 3)


def test_decode_one_kv_head_more_key_splits_than_one_merge_round_takes():
    # a single KV head: all CTAs split the same head group's keys (261 splits), more than the 256 the merge fetches in its first round
    _decode_case([100000], 8, 1, 128, 8)


def test_decode_few_long_sequences_one_item_per_cta():
    # unequal long caches whose keys are cut into one item per CTA (the last chunk of every sequence and head is shorter)
    _decode_case([40000, 30001, 20000, 9000], 28, 4, 128, 7, pad=3)


def test_decode_large_batch_takes_the_planned_path():
    # more sequences than the CTAs plan for themselves: items come from the plan kernel, by ticket
    g = torch.Generator().manual_seed(6)
    lengths = torch.randint(0, 700, (45,), generator=g).tolist()
    lengths[3] = 0
    lengths[10] = 9000
    _decode_case(lengths, 14, 2, 128, 6, pad=7)


def test_decode_random_batches_match_oracle():
    """Seeded sweep over batch sizes on both sides of the self-planning limit, length mixes (many short, one long, equal,
    block-aligned), head groupings and head dims."""
    g = torch.Generator().manual_seed(2024)
    for trial in range(16):
        S = int(torch.randint(1, 41, (1,), generator=g))
        kind = trial % 4
        if kind == 0:
            lens = torch.randint(0, 3000, (S,), generator=g).tolist()
        elif kind == 1:
            lens = [int(torch.randint(1, 60000, (1,), generator=g))] + torch.randint(0, 300, (S - 1,), generator=g).tolist()
        elif kind == 2:
            lens = [int(torch.randint(100, 9000, (1,), generator=g))] * S
        else:
            lens = (torch.randint(0, 40, (S,), generator=g) * 128).tolist()
        Hkv, G, D = [1, 2, 4][trial % 3], [1, 4, 7, 8][trial % 4], [64, 128][trial % 2]
        _decode_case(lens, Hkv * G, Hkv, D, 100 + trial)


def test_decode_head_dim_64_no_grouping_and_wide_grouping():
    _decode_case([777, 2000], 4, 4, 64, 4)
    _decode_case([1500], 8, 1, 64, 5, pad=3)


def test_block_step_emits_the_kv_cache_rows_a_decode_step_reads():
    w = wl.config2(T=600, seed=41, shape=wl.MINI)
    w.cu = wl.cu_from_lengths([250, 350])
    sh, T, S = w.shape, w.T, w.S
    H = w.tensors["H"]
    W = dict(w.weights[0]); W.update(wl.ffn_weights(sh, 41))
    pos = wl.positions(w.cu)
    ref = oc.block_step(H, W, w.cu, pos, sh, tau=0.0)
    block = dash.Block(sh, W, DEV, tau=0.0)
    Kc = torch.zeros(T, sh.Hkv, sh.D, dtype=sh.dtype, device=DEV)
    Vc = torch.zeros_like(Kc)
    block.set_kv_cache(Kc, Vc)
    lay = dash.dash_block_workspace(block, T, S)
    ws = dash.workspace(lay.total, DEV)
    outs = dict(H=torch.zeros(T, sh.d, dtype=sh.dtype, device=DEV), tok=torch.zeros(T, dtype=torch.int32, device=DEV),
                pos=torch.zeros(T, dtype=torch.int32, device=DEV), cu=torch.zeros(S + 1, dtype=torch.int32, device=DEV))
    x_full = torch.zeros(T, sh.d, dtype=sh.dtype, device=DEV)
    n_next, r, mask = torch.zeros(1, dtype=torch.int32, device=DEV), torch.zeros(T, device=DEV), torch.zeros(T, dtype=torch.uint8, device=DEV)
    cu_d = w.cu.to(DEV)
    dash.dash_block_step(block, H.to(DEV), torch.arange(T, dtype=torch.int32, device=DEV), pos.to(DEV), cu_d, 350, x_full, outs["H"],
                         outs["tok"], outs["pos"], outs["cu"], n_next, r, mask, ws)
    torch.cuda.synchronize()
    # the cache holds the rotary-applied keys and the values of every entering token
    assert_close_rms(Kc.float().cpu().numpy().reshape(T, -1), ref["K"].reshape(T, -1), "K cache")
    assert_close_rms(Vc.float().cpu().numpy().reshape(T, -1), ref["V"].reshape(T, -1), "V cache")
    nq = (sh.Hq + 2 * sh.Hkv) * sh.D
    QKV = ws[lay.attn.QKV:lay.attn.QKV + T * nq * 2].view(sh.dtype).view(T, nq)
    assert torch.equal(Kc.view(T, -1), QKV[:, sh.Hq * sh.D:(sh.Hq + sh.Hkv) * sh.D])
    # the last prompt token of each sequence, decoded over the emitted cache, reproduces its prefill attention output
    last = (w.cu[1:] - 1).long().to(DEV)
    q = QKV[last][:, :sh.Hq * sh.D].reshape(S, sh.Hq, sh.D).contiguous()
    out = dash.dash_decode_attention(q, Kc, Vc, cu_d)
    O = ws[lay.attn.O:lay.attn.O + T * sh.Hq * sh.D * 2].view(sh.dtype).view(T, sh.Hq, sh.D)[last]
    assert_close_rms(out.float().cpu().numpy(), O.float().cpu().numpy(), "decode over the emitted cache vs prefill row")
    assert_close_rms(out.float().cpu().numpy(), ref["O"][last.cpu().numpy()], "decode over the emitted cache vs oracle", atol=2.0 ** -8)
