"""Host-side checks that need no GPU: the library loads, exports every symbol the
header declares, and validates configurations before touching the device."""
import ctypes as C
import os
import re

import pytest

from paper_2503_05330_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "sdms.h")).read()
    declared = set(re.findall(r"\b(sdms_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_workspace_bytes_and_config_validation(lib):
    cfg = binding.make_config(1, 16, 1024, 128256, 4, 8)
    n = binding.sdms_workspace_bytes(cfg)
    # path store (tokens + probabilities) plus k_max tables of 2*N*L 32-byte buckets
    assert n >= 2 * 16 * 1024 * 4 + 4 * 2 * 16 * 1024 * 32
    assert n % 256 == 0
    assert binding.sdms_workspace_bytes(binding.make_config(1, 16, 1024, 128256, 4, 8, index_max_n=2)) < n - 2 * 2 * 16 * 1024 * 32 + 4096
    bigger = binding.make_config(1, 16, 1024, 128256, 4, 8, B=8, Ke=4)
    assert binding.sdms_workspace_bytes(bigger) > n
    bad = [dict(G=0), dict(N=0), dict(N=2000), dict(L=1), dict(V=0), dict(k_max=0), dict(k_max=17), dict(D=0),
           dict(D=33), dict(max_append=0), dict(max_append=10), dict(B=33), dict(B=4, Ke=0), dict(search_mode=3), dict(search_mode=2, pool_mode=1),
           dict(alpha=1.5), dict(alpha=-0.1), dict(match_capacity=-1), dict(epsilon=2), dict(epsilon=-1), dict(pool_mode=3), dict(pool_mode=-1),
           dict(max_matches_per_path=-1), dict(max_beams=9), dict(max_beams=-1), dict(max_beams=2, pool_mode=1), dict(index_max_n=4), dict(index_max_n=-1)]
    base = dict(G=1, N=4, L=64, V=100, k_max=3, D=4)
    for change in bad:
        kw = dict(base, **change)
        with pytest.raises(binding.SdmsError) as e:
            binding.sdms_workspace_bytes(binding.make_config(**kw))
        assert e.value.code == binding.ERR_INVALID_ARG, change
    cfg = binding.make_config(**base)
    cfg.struct_size = 8
    with pytest.raises(binding.SdmsError):
        binding.sdms_workspace_bytes(cfg)
    # fuzzy matching on small and on large prompts
    assert binding.sdms_workspace_bytes(binding.make_config(1, 256, 8192, 1000, 2, 4, epsilon=1)) > 0
    assert binding.sdms_workspace_bytes(binding.make_config(1, 16, 1024, 1000, 2, 4, epsilon=1)) > 0
    # positions must fit in int32
    with pytest.raises(binding.SdmsError):
        binding.sdms_workspace_bytes(binding.make_config(4096, 1024, 8192, 100, 2, 4))


def test_create_rejects_bad_arguments_without_touching_the_device(lib):
    cfg = binding.make_config(1, 4, 64, 100, 3, 4)
    h = C.c_void_p()
    assert lib.sdms_create(C.byref(cfg), None, 1 << 30, C.byref(h)) == binding.ERR_INVALID_ARG
    assert lib.sdms_create(C.byref(cfg), C.c_void_p(4096 + 8), 1 << 30, C.byref(h)) == binding.ERR_INVALID_ARG
    assert lib.sdms_create(C.byref(cfg), C.c_void_p(4096), 16, C.byref(h)) == binding.ERR_WORKSPACE_TOO_SMALL
    assert lib.sdms_create(C.byref(cfg), C.c_void_p(4096), 1 << 30, None) == binding.ERR_INVALID_ARG
    assert h.value is None
    assert lib.sdms_destroy(None) == binding.ERR_INVALID_ARG
    assert lib.sdms_append(None, None, None, None, 1, None) == binding.ERR_INVALID_ARG
    assert lib.sdms_strerror(binding.ERR_WORKSPACE_TOO_SMALL) == b"workspace too small"
    assert lib.sdms_kernel_name(2) == b"scan"
