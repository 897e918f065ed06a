"""Host-side checks of the C ABI: the library loads, exports what include/lukv.h declares,
sizes its workspace and rejects bad arguments before anything is launched (no GPU needed)."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2602_08585_b200 import build as lukv_build
from paper_2602_08585_b200 import lukv

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    lukv_build.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "lukv.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(lukv_[a-z_]+)\s*\(", header))
    assert declared == set(lukv.EXPORTS)
    L = ctypes.CDLL(lukv.LIB_PATH)
    for name in declared:
        assert getattr(L, name) is not None


def test_strerror():
    assert lukv.strerror(0) == "ok"
    for code in range(-7, 0):
        assert lukv.strerror(code) not in ("ok", "unknown status")
    assert lukv.strerror(-99) == "unknown status"


def _p(**kw):
    base = dict(S=1, L=2, H=2, G=2, d=64, T=256, w=8, kp=3, dtype="bf16", P=17)
    base.update(kw)
    return lukv.make_params(**base)


def test_largest_head_count_is_accepted():
    assert lukv.lukv_workspace_bytes(_p(L=18944, H=1)) > 0


def test_workspace_bytes_grows_with_the_problem():
    a = lukv.lukv_workspace_bytes(_p())
    b = lukv.lukv_workspace_bytes(_p(T=512))
    c = lukv.lukv_workspace_bytes(_p(S=3))
    assert 0 < a < b and a < c and a % 256 == 0


@pytest.mark.parametrize("kw,code", [
    (dict(d=96), lukv.ERR_UNSUPPORTED), (dict(dtype=7), lukv.ERR_UNSUPPORTED), (dict(kp=4), lukv.ERR_UNSUPPORTED),
    (dict(P=18), lukv.ERR_UNSUPPORTED), (dict(G=64), lukv.ERR_UNSUPPORTED), (dict(P=8193, T=8192), lukv.ERR_UNSUPPORTED),
    (dict(L=18945, H=1), lukv.ERR_UNSUPPORTED),   # heads per sequence beyond the greedy kernel's shared memory
    (dict(w=256), lukv.ERR_INVALID_ARG), (dict(w=0), lukv.ERR_INVALID_ARG), (dict(S=0), lukv.ERR_INVALID_ARG),
    (dict(P=1), lukv.ERR_INVALID_ARG), (dict(kp=0), lukv.ERR_INVALID_ARG), (dict(scale=-1.0), lukv.ERR_INVALID_ARG),
])
def test_bad_parameters_are_rejected(kw, code):
    with pytest.raises(lukv.LukvError) as e:
        lukv.lukv_workspace_bytes(_p(**kw))
    assert e.value.code == code


class _Fake:
    """A stand-in with a non-null, aligned 'device pointer'; valid calls are never made with it."""
    def __init__(self, addr=0x10000, nbytes=1 << 40):
        self._a, self._n = addr, nbytes

    def data_ptr(self):
        return self._a

    def numel(self):
        return self._n

    def element_size(self):
        return 1


def test_argument_errors_come_back_before_any_launch():
    p = _p()
    f = _Fake()
    small = _Fake(nbytes=16)
    assert lukv.lukv_score(p, None, f, f, f, check=False) == lukv.ERR_INVALID_ARG
    assert lukv.lukv_score(p, _Fake(addr=0x10004), f, f, f, check=False) == lukv.ERR_INVALID_ARG   # misaligned
    assert lukv.lukv_score(p, f, f, f, small, check=False) == lukv.ERR_WORKSPACE_TOO_SMALL
    assert lukv.lukv_score(p, f, f, f, _Fake(addr=0x10010), check=False) == lukv.ERR_INVALID_ARG    # ws not 256-aligned
    n_max = p.N * p.n
    assert lukv.lukv_allocate(p, f, [n_max + 1], f, f, f, check=False) == lukv.ERR_BUDGET
    assert lukv.lukv_allocate(p, f, [-1], f, f, f, check=False) == lukv.ERR_BUDGET
    assert lukv.lukv_allocate(p, f, [10], f, f, small, check=False) == lukv.ERR_WORKSPACE_TOO_SMALL
    assert lukv.lukv_select_gather(p, f, f, f, f, f, f, f, None, 10, f, check=False) == lukv.ERR_INVALID_ARG
    rows = 100 + p.N * p.window
    assert lukv.lukv_compress(p, f, f, f, f, [100], f, f, f, f, f, rows - 1, None, f,
                              check=False) == lukv.ERR_OUTPUT_TOO_SMALL
    assert lukv.lukv_compress(p, f, f, f, f, [n_max + 5], f, f, f, f, f, 1 << 30, None, f,
                              check=False) == lukv.ERR_BUDGET
    bad = lukv.make_params(1, 2, 2, 2, 64, 256, 8, 3, "bf16", 17)
    bad.flags = 2                                     # an unknown flag bit
    assert lukv.lukv_score(bad, f, f, f, f, check=False) == lukv.ERR_INVALID_ARG
    bad.flags = lukv.FLAG_KEYDIFF                     # the KeyDiff metric is not pooled: pool_kernel must be 1
    assert lukv.lukv_score(bad, f, f, f, f, check=False) == lukv.ERR_INVALID_ARG


def test_binding_fails_loudly_without_the_library(monkeypatch):
    monkeypatch.setattr(lukv, "_lib", None)
    monkeypatch.setattr(lukv, "LIB_PATH", "/nonexistent/liblukv.so")
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        lukv.lib()


def test_profile_argument_errors_come_back_before_any_launch():
    calib = _p(T=256, P=257)
    f = _Fake()
    grid = [0.0, 0.5, 1.0]
    assert lukv.lukv_profile_workspace_bytes(calib, 3, 5) > 0
    assert lukv.lukv_profile_workspace_bytes(calib, 6, 5) > lukv.lukv_profile_workspace_bytes(calib, 3, 5)
    assert lukv.lukv_profile_build(calib, f, 2, grid, f, _Fake(nbytes=16), check=False) == lukv.ERR_WORKSPACE_TOO_SMALL
    assert lukv.lukv_profile_build(calib, f, 2, [0.5, 1.5], f, f, check=False) == lukv.ERR_BUDGET
    assert lukv.lukv_profile_build(calib, f, 0, grid, f, f, check=False) == lukv.ERR_INVALID_ARG
    assert lukv.lukv_profile_build(calib, None, 2, grid, f, f, check=False) == lukv.ERR_INVALID_ARG
    assert lukv.lukv_profile_build(_p(S=2, T=256, P=257), f, 2, grid, f, f, check=False) == lukv.ERR_INVALID_ARG
    p = _p(S=2)
    assert lukv.lukv_profile_budgets(p, f, [0.5, 0.5], [0.5, 0.5], f, f, check=False) == lukv.ERR_INVALID_ARG
    assert lukv.lukv_profile_budgets(p, f, grid, [0.5, 1.25], f, f, check=False) == lukv.ERR_BUDGET
    assert lukv.lukv_profile_budgets(p, f, [0.2, 0.8], [0.1, 0.5], f, f, check=False) == lukv.ERR_BUDGET
    assert lukv.lukv_profile_budgets(p, None, grid, [0.5, 0.5], f, f, check=False) == lukv.ERR_INVALID_ARG


def test_importance_argument_errors_come_back_before_any_launch():
    p = _p()
    f = _Fake()
    assert lukv.lukv_importance_workspace_bytes(p, 8) > 0
    assert lukv.lukv_importance_workspace_bytes(p, 64) > lukv.lukv_importance_workspace_bytes(p, 8)
    with pytest.raises(lukv.LukvError):
        lukv.lukv_importance_workspace_bytes(p, 0)
    args = (f, f, f, None, f, True, f)
    assert lukv.lukv_oracle_importance(p, 0, 16, *args, f, check=False) == lukv.ERR_INVALID_ARG
    assert lukv.lukv_oracle_importance(p, 8, 0, *args, f, check=False) == lukv.ERR_INVALID_ARG
    assert lukv.lukv_oracle_importance(p, 8, 16, None, f, f, None, f, True, f, f, check=False) == lukv.ERR_INVALID_ARG
    assert lukv.lukv_oracle_importance(p, 8, 16, *args, _Fake(nbytes=16), check=False) == lukv.ERR_WORKSPACE_TOO_SMALL
    assert lukv.lukv_oracle_importance(p, 8, 16, *args, _Fake(addr=0x10010), check=False) == lukv.ERR_INVALID_ARG


def test_deployment_settings_are_validated():
    f = _Fake()
    p = _p(min_keep=0.5)                      # n = 248, floor 124 tokens per head, N = 4
    assert lukv.lukv_allocate(p, f, [4 * 124 - 1], f, f, f, check=False) == lukv.ERR_BUDGET
    assert lukv.lukv_allocate(_p(min_keep=1.5), f, [10], f, f, f, check=False) == lukv.ERR_INVALID_ARG
    assert lukv.lukv_allocate(_p(min_keep=-0.1), f, [10], f, f, f, check=False) == lukv.ERR_INVALID_ARG
    assert lukv.lukv_score(_p(n_sink=-1), f, f, f, f, check=False) == lukv.ERR_INVALID_ARG
    assert lukv.lukv_score(_p(n_sink=249), f, f, f, f, check=False) == lukv.ERR_INVALID_ARG
    assert lukv.lukv_workspace_bytes(_p(n_sink=4, min_keep=0.01)) == lukv.lukv_workspace_bytes(_p())
