"""dash_compact_static: the compaction entry point for callers that are not allowed to
allocate device memory (it takes no workspace; its scratch is a fixed array inside the
library).  Collected last on purpose: a run that stops at the first failure has then
already gone through every other test.

Checked through the C ABI against dash_compact, bit for bit, and against the CPU oracle, on
two calls in a row that both take the look-back path (more than 32768 rows), the second with
another mask and fewer tiles, so that tile states or a ticket left over from the first call
in the shared scratch would corrupt its indices and boundaries; at the exact size limit; and
that a call leaves the free device memory where it was."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import dash_oracle as oc
from paper_2604_18103_b200 import dash
from paper_2604_18103_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(lengths, keep, seed, width=256):
    cu = wl.cu_from_lengths(lengths)
    n = int(cu[-1])
    mask = wl.random_mask(n, keep, seed=seed)
    g = torch.Generator().manual_seed(seed)
    X = torch.randn(n, width, generator=g).to(torch.bfloat16)
    pos = wl.positions(cu)
    tok = (torch.randperm(n, generator=g) + 3).to(torch.int32)
    return cu, mask, X, pos, tok


def _same(a, b):
    k = int(a["n_out"].item())
    assert k == int(b["n_out"].item())
    assert torch.equal(a["cu_out"], b["cu_out"])
    for key in ("idx", "pos_out", "tok_out"):
        assert torch.equal(a[key][:k], b[key][:k]), key
    assert torch.equal(a["rows"][0][:k], b["rows"][0][:k])
    return k


def _matches_oracle(out, mask, cu, X, pos, tok):
    ref = oc.compact(mask, cu, rows=[X], pos_in=pos, tok_in=tok)
    k = ref["n_out"]
    assert int(out["n_out"].item()) == k == int(mask.sum())
    assert np.array_equal(out["idx"][:k].cpu().numpy(), ref["idx"])
    assert np.array_equal(out["cu_out"].cpu().numpy(), ref["cu_out"])
    assert np.array_equal(out["pos_out"][:k].cpu().numpy(), ref["pos_out"])
    assert np.array_equal(out["tok_out"][:k].cpu().numpy(), ref["tok_out"])
    assert torch.equal(out["rows"][0][:k].cpu(), ref["rows"][0])


def test_static_scratch_compaction_matches_workspace_variant_and_oracle_twice_in_a_row():
    total = 0
    # both inputs exceed 32768 rows, so both calls run the look-back scan over the shared scratch; the second has fewer tiles
    for lengths, keep, seed in (([70000, 0, 1234], 0.35, 41), ([33000, 17, 5000], 0.8, 42)):
        cu, mask, X, pos, tok = _case(lengths, keep, seed)
        d = [t.to(DEV) for t in (cu, mask, X, pos, tok)]
        ref = dash.dash_compact(d[1], d[0], rows=[d[2]], pos_in=d[3], tok_in=d[4])
        out = dash.dash_compact(d[1], d[0], rows=[d[2]], pos_in=d[3], tok_in=d[4], static_scratch=True)
        torch.cuda.synchronize()
        total += _same(out, ref)
        _matches_oracle(out, mask, cu, X, pos, tok)
    assert total > 0
    assert dash.dash_check_status() == dash.OK


def test_static_scratch_at_its_size_limit_and_beyond():
    n = dash.COMPACT_STATIC_MAX_ROWS
    cu, mask, X, pos, tok = _case([n - 5, 5], 0.1, 43, width=8)
    d = [t.to(DEV) for t in (cu, mask, X, pos, tok)]
    out = dash.dash_compact(d[1], d[0], rows=[d[2]], pos_in=d[3], tok_in=d[4], static_scratch=True)
    torch.cuda.synchronize()
    _matches_oracle(out, mask, cu, X, pos, tok)
    assert dash.dash_check_status() == dash.OK
    lib = dash.lib()
    fake, nul = ctypes.c_void_p(4096), ctypes.c_void_p(0)      # rejected before any pointer is used
    st = lib.dash_compact_static(fake, n + 1, fake, 1, None, 0, nul, nul, nul, nul, nul, fake, nul, nul)
    assert st == 6 and b"fixed scratch" in lib.dash_status_string(st)


def test_static_scratch_call_allocates_no_device_memory():
    cu, mask, X, pos, tok = _case([50000], 0.5, 44, width=64)
    n = int(cu[-1])
    d = [t.to(DEV) for t in (cu, mask, X, pos, tok)]
    outs = dict(idx=torch.empty(n, dtype=torch.int32, device=DEV), pos_out=torch.empty(n, dtype=torch.int32, device=DEV),
                tok_out=torch.empty(n, dtype=torch.int32, device=DEV), cu_out=torch.empty(2, dtype=torch.int32, device=DEV),
                n_out=torch.empty(1, dtype=torch.int32, device=DEV))
    rows_out = [torch.empty_like(d[2])]
    dash.dash_compact(d[1], d[0], rows=[d[2]], rows_out=rows_out, pos_in=d[3], tok_in=d[4], outputs=outs, static_scratch=True)   # first call on the device
    torch.cuda.synchronize()
    arr = (dash.Rows * 1)(dash.Rows(d[2].data_ptr(), rows_out[0].data_ptr(), 128, 128, 128))
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    free_before = torch.cuda.mem_get_info()[0]
    for _ in range(3):
        st = dash.lib().dash_compact_static(p(d[1]), n, p(d[0]), 1, arr, 1, p(d[3]), p(outs["pos_out"]), p(d[4]), p(outs["tok_out"]),
                                            p(outs["idx"]), p(outs["cu_out"]), p(outs["n_out"]), stream)
        assert st == dash.OK
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    assert int(outs["n_out"].item()) == int(mask.sum())
    assert dash.dash_check_status() == dash.OK
