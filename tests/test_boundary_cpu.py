"""Host-only checks of the C-ABI library: it loads, exports every symbol that include/sla.h declares,
and its host-side helpers behave; no kernel is launched."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2601_18401_b200 import build
    build.build_library()
    import paper_2601_18401_b200 as sla
    return sla.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "sla.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sla_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    import paper_2601_18401_b200.binding as b
    names = declared_symbols()
    assert len(names) >= 9
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(b.EXPORTS) == names


def test_status_strings(lib):
    assert lib.sla_status_string(0) == b"SLA_OK"
    assert lib.sla_status_string(-3) == b"SLA_ERR_WORKSPACE"
    assert lib.sla_status_string(-99) == b"SLA_ERR_UNKNOWN"
    assert lib.sla_last_error(None) == b"NULL handle"


def test_workspace_sizing_is_host_only_and_validates(lib):
    import paper_2601_18401_b200 as sla
    lay = sla.sla_layout_t(1, 32, 4, 128, sla.SLA_BF16, 0, 0, 128, 0, 4 * 1048832 * 128, 1048832 * 128, 128)
    par = sla.make_params(16, 1024)
    n = sla.sla_workspace_bytes(lay, par, 1, 1 << 20)
    assert 0 < n < (1 << 30)
    bad = sla.sla_layout_t(1, 32, 5, 128, sla.SLA_BF16, 0, 0, 128, 0, 0, 0, 128)
    assert sla.sla_workspace_bytes(bad, par, 1, 1 << 20) == 0
    bad = sla.sla_layout_t(1, 32, 4, 96, sla.SLA_BF16, 0, 0, 128, 0, 0, 0, 128)
    assert sla.sla_workspace_bytes(bad, par, 1, 1 << 20) == 0
    assert sla.sla_workspace_bytes(lay, sla.make_params(65, 1024), 1, 1 << 20) == 0
    assert sla.sla_host_staging_bytes(lay, par, 4096) > 0


@pytest.mark.parametrize("p", [1.0 / 3.0, 2.0 / 3.0, 0.54, 0.25])
def test_pattern_tables_follow_the_rounding_rule(lib, p):
    """The library's host-built tables for general exponents against the oracle's functions of the same
    rule (anchors at i + 1 - ceil((s+1)^(1/p)); l(i) = ceil(i^p)), entry by entry, and against exact
    integer powers where p is the reciprocal of an integer."""
    import paper_2601_18401_b200 as sla
    from oracle import sla_oracle as O
    reach = 200000
    off = sla.sla_pattern_offsets(p, reach)
    assert off == [O.stride_offset(s, p) for s in range(len(off))]
    assert O.stride_offset(len(off), p) > reach >= off[-1]
    steps = sla.sla_pattern_len_steps(p, reach)
    assert O.base_len(reach, 0, p) == len(steps)
    for v, first in list(enumerate(steps, start=1))[:: max(1, len(steps) // 300)]:
        assert O.base_len(first, 0, p) >= v and (first == 1 or O.base_len(first - 1, 0, p) < v)
    if abs(p - 1.0 / 3.0) < 1e-12:
        assert off[:5] == [1, 8, 27, 64, 125] and off[57] == 58 ** 3
    if p == 0.25:
        assert off[:4] == [1, 16, 81, 256]
    assert lib.sla_pattern_offsets(0.9, 100, None, 0) == -1
    assert lib.sla_pattern_offsets(0.75, 10 ** 9, None, 0) == -1      # more than 65536 strides


def test_calls_reject_null_handle(lib):
    assert lib.sla_destroy(None) == -1
    assert lib.sla_poll_status(None, None) == -1
    assert lib.sla_span_search(None, None, None, 1, 0, 1, None, None, None, None, None) == -1
    assert lib.sla_create(None, 0, 0) == -1


def test_product_path_does_not_touch_the_oracle():
    """Nothing under the package imports, links or executes the test oracle."""
    pkg = os.path.join(ROOT, "paper_2601_18401_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"sla_oracle|from\s+oracle|import\s+oracle|oracle/", text), f
