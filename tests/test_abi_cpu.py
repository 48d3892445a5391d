"""Host-only checks of the C ABI: the library loads, exports every symbol include/cada.h
declares, and rejects invalid configurations without touching a GPU."""
import ctypes as C
import os
import re

import pytest

from paper_2012_15469_b200 import binding as B
from paper_2012_15469_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_mod.build()
    return B.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "cada.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cada_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert {"cada_create", "cada_step", "cada_stats", "cada_destroy"} <= set(names)
    assert set(names) == set(B.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def _cfg(**kw):
    cfg = B.cada_config()
    cfg.struct_size = C.sizeof(B.cada_config)
    cfg.abi_version = B.CADA_ABI_VERSION
    cfg.model, cfg.rule = B.CADA_MODEL_LOGISTIC, B.CADA_RULE_CADA2
    cfg.M, cfg.batch, cfg.n_features, cfg.n_classes, cfg.has_bias = 4, 8, 10, 1, 1
    cfg.p = 11
    cfg.alpha, cfg.beta1, cfg.beta2, cfg.eps, cfg.c = 0.01, 0.9, 0.99, 1e-8, 0.6
    cfg.d_max, cfg.D, cfg.ldx = 10, 100, 12
    for k, v in kw.items():
        setattr(cfg, k, v)
    return cfg


def test_workspace_bytes_valid_and_invalid(lib):
    assert B.cada_workspace_bytes(_cfg()) > 0
    assert B.cada_workspace_bytes(_cfg(rule=B.CADA_RULE_CADA1)) > 0
    bigger = B.cada_workspace_bytes(_cfg(history_capacity=100))
    assert bigger > B.cada_workspace_bytes(_cfg())
    assert B.cada_workspace_bytes(_cfg(host_step_rows=8)) > B.cada_workspace_bytes(_cfg())
    for bad in (dict(p=12), dict(M=0), dict(batch=0), dict(d_max=0), dict(D=0), dict(rule=7), dict(model=9),
                dict(alpha=0.0), dict(beta1=1.0), dict(c=-1.0), dict(c=float("nan")), dict(ldx=5),
                dict(struct_size=8), dict(abi_version=99), dict(n_classes=3), dict(host_step_rows=3),
                dict(x_dtype=B.CADA_X_BF16), dict(eps=-1.0)):
        assert B.cada_workspace_bytes(_cfg(**bad)) == 0, bad
    assert lib.cada_workspace_bytes(None) == 0
    # the worker index is a grid y-coordinate: more than 65535 workers are declined at planning time, not at the first launch
    assert B.cada_workspace_bytes(_cfg(M=65535)) > 0
    assert B.cada_workspace_bytes(_cfg(M=65536)) == 0
    h = C.c_void_p()
    big = _cfg(M=65536)
    assert lib.cada_create(C.byref(big), C.byref(h)) == B.CADA_ERR_UNSUPPORTED and b"65535" in lib.cada_last_error(None)
    assert lib.cada_set_wait_limit(None, 1) == B.CADA_ERR_INVALID_ARG
    # a handle may hold a subset of the problem's workers: the subset must lie inside M_total
    assert B.cada_workspace_bytes(_cfg(M_total=8, m_first=1, m_stride=2)) > 0
    for bad in (dict(M_total=3), dict(M_total=8, m_first=2, m_stride=2), dict(M_total=8, m_first=0, m_stride=0),
                dict(m_first=1), dict(M_total=8, m_first=-1, m_stride=1)):
        assert B.cada_workspace_bytes(_cfg(**bad)) == 0, bad
    assert lib.cada_step_local(None, None) == B.CADA_ERR_INVALID_ARG and lib.cada_step_apply(None, None) == B.CADA_ERR_INVALID_ARG


def test_softmax_and_infinite_c_are_accepted(lib):
    cfg = _cfg(model=B.CADA_MODEL_SOFTMAX, n_classes=10, n_features=784, p=7850, ldx=784, c=float("inf"))
    assert B.cada_workspace_bytes(cfg) > 0


def test_create_rejects_bad_arguments_without_a_gpu(lib):
    h = C.c_void_p()
    cfg = _cfg()
    rc = lib.cada_create(C.byref(cfg), C.byref(h))          # X, y, ... are NULL
    assert rc == B.CADA_ERR_INVALID_ARG and not h
    assert b"non-NULL" in lib.cada_last_error(None)
    assert lib.cada_create(C.byref(cfg), None) == B.CADA_ERR_INVALID_ARG
    bad = _cfg(p=99)
    assert lib.cada_create(C.byref(bad), C.byref(h)) == B.CADA_ERR_INVALID_ARG
    assert b"model shape implies 11" in lib.cada_last_error(None)
    # NULL handles
    assert lib.cada_step(None, 1) == B.CADA_ERR_INVALID_ARG
    assert lib.cada_stats(None, None) == B.CADA_ERR_INVALID_ARG
    assert lib.cada_destroy(None) == B.CADA_OK


def test_binding_struct_matches_header_size(lib):
    # a mismatch between the ctypes mirror and the C struct is caught by struct_size validation
    assert B.cada_workspace_bytes(_cfg()) > 0
    assert C.sizeof(B.cada_stats_t) == 96
