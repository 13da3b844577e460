"""The C-ABI library loads and exports every entry point the header declares (no GPU needed)."""
import ctypes
import os
import re

from paper_2512_09427_b200 import odma

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "odma.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(odma_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    names = _declared()
    assert len(names) >= 25
    lib = ctypes.CDLL(odma.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in odma.h but not exported"
        assert n in odma.EXPORTS, f"{n} has no Python binding"


def test_defaults_are_the_papers_constants():
    cfg = odma.config_default()
    # Section III-B: gamma = 0.2, tau = 0.8; Section III-C: B = 4, window 10,000, refresh 1,000
    assert (cfg.gamma_permille, cfg.tau_permille) == (200, 800)
    assert (cfg.n_levels, cfg.window, cfg.refresh) == (4, 10000, 1000)
    assert [cfg.p_num[i] for i in range(4)] == [1, 2, 3, 4] and cfg.p_den == 4


def test_struct_sizes_match_the_header():
    assert ctypes.sizeof(odma.Slab) == 24
    assert ctypes.sizeof(odma.Stats) == 16 * 8
    assert ctypes.sizeof(odma.Config) == (6 + 8 + 1 + 15) * 4
    assert ctypes.sizeof(odma.Tables) == 8 + 16 * 4 + 8 + 8


def test_strerror_and_argument_checks():
    assert odma.strerror(odma.OK) == "ok"
    assert "timed out" in odma.strerror(odma.ERR_TIMEOUT)
    try:
        odma.Pool(0, 1 << 20, 1, 1, 60, odma.DTYPE_BF16)      # row of 120 bytes: not 16-byte multiple
        raise AssertionError("expected ODMA_ERR_INVALID")
    except odma.OdmaError as e:
        assert e.code == odma.ERR_INVALID
    p = odma.Pool(0, 1 << 20, 1, 1, 64, odma.DTYPE_BF16)
    # a bookkeeping-only pool refuses device work instead of touching memory it does not have
    t = odma.Tables()
    assert odma._lib.odma_append_kv(p._h, 0, ctypes.byref(t), None, None, None) == odma.ERR_INVALID
    assert odma._lib.odma_decode_attention(p._h, 0, None, 1, ctypes.byref(t), None, None, None) == odma.ERR_INVALID
    assert p.check_status() == odma.ERR_INVALID
