"""CPU-side checks: the C-ABI library loads and exports every symbol the header declares,
argument validation that needs no device, and the host restatement of the Gaussian generator
against the published known-answer vectors."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2608_28941_b200 import rrf
from philox_ref import philox4x32_10, omega_reference

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "rrf.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(rrf_[a-z_]+)\s*\(", header))
    assert names == set(rrf.EXPORTS), names ^ set(rrf.EXPORTS)
    for name in names:
        assert hasattr(lib, name), name


def test_struct_layouts_match_header():
    assert ctypes.sizeof(rrf.rrf_params_t) == 64
    assert ctypes.sizeof(rrf.rrf_result_t) == 72


def test_workspace_query_validates_without_a_device(lib):
    good = rrf.make_params(rrf.RRF_F64, 1024, 768, 16, 1e-8, 256)
    assert rrf.rrf_workspace_bytes(good) > 1024 * 768 * 8
    inplace = rrf.make_params(rrf.RRF_F64, 1024, 768, 16, 1e-8, 256, flags=rrf.RRF_FLAG_INPLACE)
    assert rrf.rrf_workspace_bytes(inplace) < rrf.rrf_workspace_bytes(good)
    for bad in (dict(b=24), dict(max_rank=250), dict(max_rank=1024), dict(m=0), dict(tol=-1.0), dict(dtype=7),
                dict(dtype=rrf.RRF_F32, b=16)):
        kw = dict(dtype=rrf.RRF_F64, m=1024, n=768, b=16, tol=1e-8, max_rank=256)
        kw.update(bad)
        with pytest.raises(rrf.RrfError) as e:
            rrf.rrf_workspace_bytes(rrf.make_params(**kw))
        assert e.value.status == rrf.RRF_ERR_INVALID_ARG
    assert rrf.rrf_status_string(rrf.RRF_ERR_TIMEOUT) == "bounded device-side wait gave up"


def test_philox_known_answers():
    # published known-answer vectors of Philox-4x32-10 (Salmon et al., SC'11 reference suite)
    out = philox4x32_10([0, 0, 0, 0], [0, 0])
    assert [int(x) for x in out] == [0x6627e8d5, 0xe169c58d, 0xbc57ac4c, 0x9b00dbd8]
    out = philox4x32_10([0xffffffff] * 4, [0xffffffff] * 2)
    assert [int(x) for x in out] == [0x408f276d, 0x41c83b0e, 0xa20bc7c6, 0x6d5451fd]
    out = philox4x32_10([0x243f6a88, 0x85a308d3, 0x13198a2e, 0x03707344], [0xa4093822, 0x299f31d0])
    assert [int(x) for x in out] == [0xd16cfe09, 0x94fdcceb, 0x5001e420, 0x24126ea1]




def test_omega_reference_moments():
    x = omega_reference(11, 2000, 64)
    assert abs(x.mean()) < 1e-2 and abs(x.std() - 1) < 1e-2
    assert np.array_equal(omega_reference(11, 2000, 8, first=8), x[8:16])
