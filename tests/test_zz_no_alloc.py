"""dash_compact_static: the compaction entry point for callers that are not allowed to
allocate device memory (it takes no workspace; its scratch is a fixed array inside the
library).  Collected last on purpose: a run that stops at the first failure has then
already gone through every other test.

Checked through the C ABI against dash_compact, bit for bit, on two calls in a row (the
second with another mask and size, so leftovers of the first call in the shared scratch
would show), plus the size limit."""
import ctypes

import pytest
import torch

from paper_2604_18103_b200 import dash
from paper_2604_18103_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(lengths, keep, seed):
    cu = wl.cu_from_lengths(lengths)
    n = int(cu[-1])
    mask = wl.random_mask(n, keep, seed=seed)
    g = torch.Generator().manual_seed(seed)
    X = torch.randn(n, 256, generator=g).to(torch.bfloat16)
    pos = wl.positions(cu)
    tok = (torch.randperm(n, generator=g) + 3).to(torch.int32)
    return cu.to(DEV), mask.to(DEV), X.to(DEV), pos.to(DEV), tok.to(DEV)


def _same(a, b):
    k = int(a["n_out"].item())
    assert k == int(b["n_out"].item())
    assert torch.equal(a["cu_out"], b["cu_out"])
    for key in ("idx", "pos_out", "tok_out"):
        assert torch.equal(a[key][:k], b[key][:k]), key
    assert torch.equal(a["rows"][0][:k], b["rows"][0][:k])
    return k


def test_static_scratch_compaction_matches_workspace_variant_twice_in_a_row():
    total = 0
    for lengths, keep, seed in (([70000, 0, 1234], 0.35, 41), ([5000, 17], 0.8, 42)):
        cu, mask, X, pos, tok = _case(lengths, keep, seed)
        ref = dash.dash_compact(mask, cu, rows=[X], pos_in=pos, tok_in=tok)
        out = dash.dash_compact(mask, cu, rows=[X], pos_in=pos, tok_in=tok, static_scratch=True)
        torch.cuda.synchronize()
        total += _same(out, ref)
        assert int(out["n_out"].item()) == int(mask.sum().item())
    assert total > 0
    assert dash.dash_check_status() == dash.OK


def test_static_scratch_rejects_inputs_beyond_its_limit():
    lib = dash.lib()
    fake, nul = ctypes.c_void_p(4096), ctypes.c_void_p(0)      # rejected before any pointer is used
    st = lib.dash_compact_static(fake, dash.COMPACT_STATIC_MAX_ROWS + 1, fake, 1, None, 0, nul, nul, nul, nul, nul, fake, nul, nul)
    assert st == 6 and b"fixed scratch" in lib.dash_status_string(st)
