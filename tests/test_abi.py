"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, validates arguments before touching the device, and builds schedules."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import paper_2601_09212_b200 as csd
from paper_2601_09212_b200 import _build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    _build.build_library()
    return csd.library()


def test_exports_match_header(lib):
    header = open(os.path.join(ROOT, "include", "csd.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(csd_[a-z_]+)\s*\(", header))
    assert declared == set(csd.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_params_struct_matches_header():
    header = open(os.path.join(ROOT, "include", "csd.h")).read()
    body = header[header.index("typedef struct csd_params {"):header.index("} csd_params;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    names = re.findall(r"[\s\*]([A-Za-z_]+)\s*[,;]", body)
    assert names == [f[0] for f in csd.csd_params._fields_]


def test_version_and_error_strings(lib):
    assert csd.csd_version() == 400
    for code in range(0, -8, -1):
        assert len(csd.error_string(code)) > 1
    assert "unknown" in csd.error_string(-99)


def test_workspace_size(lib):
    assert csd.csd_workspace_size(64, 8, 16384, csd.CSD_F32) > 0
    assert csd.csd_workspace_size(64, 8, 16384, csd.CSD_BF16) > 0
    assert csd.csd_workspace_size(64, 8, 16384, csd.CSD_F32) % 256 == 0
    for bad in [(0, 8, 16384, 0), (1, 0, 16384, 0), (1, 33, 16384, 0), (1, 8, 1, 0), (1, 8, 2 ** 20 + 1, 0),
                (1, 8, 16384, 2)]:
        assert csd.csd_workspace_size(*bad) == 0
    # grows with the problem
    assert csd.csd_workspace_size(256, 16, 65536, 0) > csd.csd_workspace_size(64, 8, 16384, 0)


def test_host_validation_needs_no_device(lib):
    p = csd.csd_params()
    assert lib.csd_verify_ex(C.byref(p)) == -1          # NULL pointers
    assert lib.csd_verify_ex(None) == -1
    assert lib.csd_verify_host(None, None, 0) == -1
    assert lib.csd_host_staging_size(C.byref(p)) == 0
    assert lib.csd_verify(None, None, None, None, None, 0, 4, 16, None, None, None) == -2


def test_schedule_against_oracle(lib, oracle):
    """The library's schedule helper and the oracle's are separate code; both must satisfy
    the paper's constraints and agree to fp32 rounding."""
    for kind, delta, x, L in [(0, 1.3, 0.0, 7), (1, 1.1, 0.7, 4), (1, 1.1, 0.7, 8), (1, 2.0, 0.7, 16),
                              (1, 4.0, 1.5, 32), (2, 1.1, 8.0, 5), (2, 1.0, 8.0, 12)]:
        mine = csd.csd_make_schedule(kind, delta, x, L)
        ref = oracle.make_schedule(kind, delta, x, L)
        assert mine.dtype == np.float32 and mine.shape == (L,)
        assert np.allclose(mine, ref, rtol=3e-7, atol=0)
        assert np.isclose(mine.astype(np.float64).sum(), delta * L, rtol=1e-6)
    for bad in [(1, 1.1, 0.7, 0), (1, -1.0, 0.7, 4), (5, 1.0, 0.7, 4), (2, 1.0, 1.0, 4), (1, 1.0, -0.1, 4)]:
        with pytest.raises(csd.CsdError):
            csd.csd_make_schedule(*bad)


def test_no_cpu_fallback_in_binding():
    src = open(os.path.join(ROOT, "paper_2601_09212_b200", "__init__.py")).read()
    assert "import oracle" not in src and "from oracle" not in src
