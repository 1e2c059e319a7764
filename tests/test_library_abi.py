"""CPU-side checks of the boundary: the library builds/loads, exports every symbol
the header declares, rejects bad arguments before touching a device, and its pure
host helpers reproduce the paper's printed numbers."""
import ctypes
import os
import re

import pytest

from paper_2604_18103_b200 import build as dash_build
from paper_2604_18103_b200 import dash

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLD = os.path.join(ROOT, "tests", "golden", "theory_speedup_vs_len.txt")


@pytest.fixture(scope="module")
def lib():
    dash_build.build()
    return dash.lib()


def _declared(header):
    hdr = open(os.path.join(ROOT, "include", header)).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    return set(re.findall(r"\b(dash_[a-z_0-9]+)\s*\(", hdr))


def test_every_declared_symbol_is_exported(lib):
    assert sorted(os.listdir(os.path.join(ROOT, "include"))) == ["dash.h", "dash_testing.h"]
    assert _declared("dash.h") == set(dash.EXPORTS)
    assert _declared("dash_testing.h") == set(dash.TEST_HOOKS)
    for name in dash.EXPORTS + dash.TEST_HOOKS:
        assert hasattr(lib, name), name


def test_keep_count_and_flops_helpers_match_paper_table(lib):
    for line in open(GOLD):
        if line.startswith("#") or not line.strip():
            continue
        n, n_hat, r_pct, s = line.split()
        n, n_hat = int(n), int(n_hat)
        assert dash.dash_keep_count(n, 0.667, 64, 32, 1) == n_hat
        sp = dash.dash_flops_speedup(n, n_hat, 28, 11, 3584, 18944)
        assert round(sp, 2) == pytest.approx(float(s), abs=0.0051)
        assert round(100 * (1 - 1 / sp), 2) == pytest.approx(float(r_pct), abs=0.0051)
    assert dash.dash_keep_count(8192, 0.4) == 4915
    assert dash.dash_keep_count(131072, 0.8) == 26214
    assert dash.dash_keep_count(10, 1.0) == -1 and dash.dash_keep_count(-1, 0.5) == -1
    assert dash.dash_flops_per_layer(2, 3, 5) == 4 * 2 * 9 + 2 * 4 * 3 + 2 * 2 * 3 * 5


def test_invalid_arguments_are_rejected_before_any_launch(lib):
    nul = ctypes.c_void_p(0)
    fake = ctypes.c_void_p(4096)            # never dereferenced: validation fails first
    # d not a multiple of 8
    assert lib.dash_delta_norm(fake, fake, 4, 12, 12, 12, dash.BF16, 0, 0.0, fake, nul, 0, nul, None, nul, nul) == 1
    # null U
    assert lib.dash_delta_norm(nul, fake, 4, 16, 16, 16, dash.BF16, 0, 0.0, fake, nul, 0, nul, None, nul, nul) == 1
    # misaligned pointer
    assert lib.dash_delta_norm(ctypes.c_void_p(4100), fake, 4, 16, 16, 16, dash.BF16, 0, 0.0, fake, nul, 0, nul, None, nul, nul) == 1
    # select without sequence boundaries / keep-count without counts
    assert lib.dash_select(fake, 8, nul, 1, 0, 0.0, nul, 0, 0, fake, nul) == 1
    assert lib.dash_select(fake, 8, fake, 1, 1, 0.0, nul, 0, 0, fake, nul) == 1
    # compaction: missing / too-small workspace
    assert lib.dash_compact(fake, 8, fake, 1, None, 0, nul, nul, nul, nul, nul, fake, nul, nul, 0, nul) == 3
    assert lib.dash_compact(fake, 1 << 20, fake, 1, None, 0, nul, nul, nul, nul, nul, fake, nul, fake, 512, nul) == 3
    # scatter: bad `which`
    assert lib.dash_scatter(fake, 8, 64, 64, nul, nul, 3, nul, fake, 64, nul) == 1
    # attention: head_dim 96 unsupported, non-causal unsupported, Hq % Hkv
    args = lambda Hq, Hkv, D, causal: (fake, fake, fake, fake, nul, Hq * D, Hkv * D, Hkv * D, Hq * D, fake, 1, 256, 256,
                                       Hq, Hkv, D, 0.1, causal, dash.BF16, nul, 0, nul)
    assert lib.dash_varlen_attention(*args(4, 2, 96, 1)) == 2
    assert lib.dash_varlen_attention(*args(4, 2, 128, 0)) == 2
    assert lib.dash_varlen_attention(*args(4, 3, 128, 1)) == 1
    assert lib.dash_status_string(3).decode().startswith("workspace")
    assert dash.dash_workspace_bytes(dash.WS_COMPACT, 131072) >= 131072 // 32 * 8
