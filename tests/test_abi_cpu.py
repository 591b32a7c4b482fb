"""CPU-only checks of the C ABI: the library loads, exports every symbol the
header declares, and its host-side validation rejects bad arguments before
anything could be launched (no compute call needs a GPU here)."""
import ctypes as C
import os
import re

import pytest

from paper_2601_05149_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def test_exports_match_header(lib):
    header = open(os.path.join(ROOT, "include", "mulo.h")).read()
    declared = set(re.findall(r"\b(mulo_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_params_struct_layout():
    # the Python mirror must match the C struct: 18 x 4 bytes + u64 seed, 8-byte aligned
    assert C.sizeof(binding.MuloParams) == 80
    assert binding.MuloParams.seed.offset == 64
    assert binding.MuloParams.round.offset == 72


def test_status_strings(lib):
    assert binding.status_string(binding.OK) == "ok"
    assert len({binding.status_string(s) for s in range(6)}) == 6


def test_timeout_bit_maps_to_an_error_status(lib):
    """Host mapping of the device status word, on hand-set words (no kernel is made to time out)."""
    report_bits = binding.DEV_ZERO_DRAFT_PROB | binding.DEV_BAD_TOKEN | binding.DEV_DENSE_FALLBACK
    for word in (0, binding.DEV_DENSE_FALLBACK, report_bits):
        assert binding.status_of_device_flags(word) == binding.OK
    for word in (binding.DEV_TIMEOUT, binding.DEV_TIMEOUT | report_bits, 0xFFFFFFFF):
        assert binding.status_of_device_flags(word) == binding.ERR_TIMEOUT
    assert "timed out" in binding.status_string(binding.ERR_TIMEOUT)


def _ws(p):
    n = C.c_size_t()
    return binding.lib().mulo_workspace_bytes(C.byref(p), C.byref(n)), n.value


def test_validation_matrix(lib):
    good = dict(B=2, H=8, W=8, V=256, r=2, dtype=binding.BF16)
    st, n = _ws(binding.make_params(**good))
    assert st == binding.OK and n >= 256 + 2 * 64 * 9
    bad = [
        dict(good, V=250), dict(good, V=0), dict(good, H=7), dict(good, W=9), dict(good, r=0),
        dict(good, H=0), dict(good, B=-1), dict(good, dtype=7), dict(good, temperature=0.0),
        dict(good, temperature=-1.0), dict(good, temperature=float("nan")),
        dict(good, radius=-1), dict(good, accept_mode=5), dict(good, resample_mode=9),
        dict(good, cfg_scale=float("inf")), dict(good, pool_k=8, pool_delta=-0.5),
    ]
    for kw in bad:
        assert _ws(binding.make_params(**kw))[0] == binding.ERR_INVALID_ARG, kw
    unsupported = [dict(good, V=65544), dict(good, radius=32), dict(good, pool_k=4096, V=8192),
                   dict(good, pool_k=300), dict(good, H=4096, W=64)]
    for kw in unsupported:
        assert _ws(binding.make_params(**kw))[0] == binding.ERR_UNSUPPORTED, kw
    assert binding.lib().mulo_workspace_bytes(None, None) == binding.ERR_INVALID_ARG
    # B = 0 is a valid empty batch
    assert _ws(binding.make_params(**dict(good, B=0)))[0] == binding.OK


def test_null_context_is_rejected(lib):
    p = binding.make_params(1, 8, 8, 256, 2, binding.BF16)
    assert lib.mulo_round(None, C.byref(p), *([None] * 15)) == binding.ERR_INVALID_ARG
    assert lib.mulo_verify(None, C.byref(p), *([None] * 13)) == binding.ERR_INVALID_ARG
    assert lib.mulo_set_workspace(None, None, C.c_size_t(0)) == binding.ERR_INVALID_ARG


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libmulo.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.lib()
