"""The C-ABI library loads and exports every symbol the header declares (no compute)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib_path():
    from paper_2402_03694_b200 import build
    return build.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "serveflow.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sf_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_named_calls():
    names = _declared()
    for must in ("sf_extract_features", "sf_fast_infer", "sf_route", "sf_slow_infer", "sf_serve_batch",
                 "sf_table_create", "sf_table_ingest", "sf_table_lookup"):
        assert must in names


def test_every_declared_symbol_is_exported(lib_path):
    lib = ctypes.CDLL(lib_path)
    for name in _declared():
        assert hasattr(lib, name), name


def test_binding_lists_the_same_calls(lib_path):
    from paper_2402_03694_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()
    for name in binding.EXPORTS:
        if name in ("sf_strerror", "sf_last_cuda_error"):
            continue
        assert hasattr(binding, name), name
    assert binding.sf_strerror(0) == "ok" and "argument" in binding.sf_strerror(-1)
    assert "sm_100a" in binding.sf_version()


def test_host_only_calls_and_loud_failure_without_gpu(lib_path):
    import numpy as np
    import torch
    from paper_2402_03694_b200 import binding as sf
    import oracle
    u = np.random.default_rng(0).random(1000).astype(np.float32)
    got = sf.sf_universal_thresholds(u, [1, 25, 50, 76, 99, 100])
    assert np.array_equal(got, oracle.universal_thresholds(u, [1, 25, 50, 76, 99, 100]))
    assert sf.sf_universal_thresholds(np.array([.3, .1, .4, .2], np.float32), [50])[0] == np.float32(0.2)
    if not torch.cuda.is_available():
        with pytest.raises(sf.SfError):
            sf.sf_ctx_create(0)           # no device: the library refuses, it never falls back to the CPU
