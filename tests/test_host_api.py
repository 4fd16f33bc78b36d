"""Host-side checks that need no GPU: the library loads, exports what include/mona.h declares, and the
planning and validation logic behaves."""
import ctypes as C
import os
import re

import pytest

import paper_2605_26842_b200 as pkg
from paper_2605_26842_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
DEFAULT_CHUNK_BUDGET = 768 << 20     # the library's built-in default; tests that change the knob put it back


@pytest.fixture(scope="module")
def L():
    build_mod.build()
    return pkg.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "mona.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mona_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = declared_functions()
    assert {"mona_create", "mona_step", "mona_destroy", "mona_query_sizes"} <= set(names)
    for n in names:
        assert hasattr(L, n), f"{n} declared in mona.h but not exported"


def test_default_hparams_follow_the_paper(L):
    hp = pkg.default_hparams()
    assert (hp.ns_a, hp.ns_b, hp.ns_c, hp.ns_steps) == (3.4445, -4.7750, 2.0315, 5)
    assert hp.scale_mode == 0 and hp.scale_value == 0.2
    assert abs(hp.accel_alpha - (-1.0 / (2 * (1 - hp.accel_beta)))) < 1e-12


def test_query_sizes_state_is_three_fp32_per_parameter(L):
    d = [pkg.MatrixDesc(768, 2048, 64, 0, 0, 0), pkg.MatrixDesc(2048, 768, 64, 0, 0, 0), pkg.MatrixDesc(32, 1024, 1, 0, 0, 0)]
    sb, wb = pkg.query_sizes(d)
    n = 2 * 64 * 768 * 2048 + 32 * 1024
    assert 12 * n <= sb <= 12 * n + 9 * 256          # three buckets, three 256-byte-aligned blocks each
    lite = [pkg.MatrixDesc(x.rows, x.cols, x.batch, 0, 0, 1) for x in d]
    sb_lite, _ = pkg.query_sizes(lite)
    assert 8 * n <= sb_lite <= 8 * n + 9 * 256      # bfloat16 storage of A and G_prev: 4 + 2 + 2 bytes per parameter
    single = [pkg.MatrixDesc(x.rows, x.cols, x.batch, 0, 0, pkg.MONA_STATE_COMBINED) for x in d]
    assert 8 * n <= pkg.query_sizes(single)[0] <= 8 * n + 6 * 256   # M and the single buffer Z
    assert wb > 0
    # same shapes share one bucket: once the chunk is bounded by the budget (not by the matrix count),
    # two descriptors of one shape need the workspace of one
    pkg.set_chunk_budget(64 << 20)
    try:
        sb2, wb2 = pkg.query_sizes([d[0], d[0]])
        assert wb2 == pkg.query_sizes([d[0]])[1] and sb2 == 2 * pkg.query_sizes([d[0]])[0]
    finally:
        pkg.set_chunk_budget(DEFAULT_CHUNK_BUDGET)


def test_chunk_budget_changes_workspace(L):
    d = [pkg.MatrixDesc(512, 1024, 32, 0, 0, 0)]
    try:
        pkg.set_chunk_budget(8 << 20)
        small = pkg.query_sizes(d)[1]
        pkg.set_chunk_budget(48 << 20)
        big = pkg.query_sizes(d)[1]
        assert small < big
        with pytest.raises(pkg.MonaError):
            pkg.set_chunk_budget(1000)
    finally:
        pkg.set_chunk_budget(DEFAULT_CHUNK_BUDGET)


@pytest.mark.parametrize("desc,status", [
    (pkg.MatrixDesc(0, 8, 1, 0, 0, 0), 1), (pkg.MatrixDesc(8, 8, 0, 0, 0, 0), 1), (pkg.MatrixDesc(8, 8, 1, 10, 0, 0), 1),
    (pkg.MatrixDesc(8, 8, 1, 0, 7, 0), 1), (pkg.MatrixDesc(8, 8, 1, 0, 0, 3), 1), (pkg.MatrixDesc(1 << 21, 8, 1, 0, 0, 0), 2)])
def test_bad_descriptors_are_rejected(L, desc, status):
    with pytest.raises(pkg.MonaError) as e:
        pkg.query_sizes([desc])
    assert e.value.status == status


def test_create_without_buffers_fails_cleanly(L):
    h = C.c_void_p()
    d = (pkg.MatrixDesc * 1)(pkg.MatrixDesc(64, 64, 1, 0, 0, 0))
    st = L.mona_create(C.byref(h), d, 1, None, 0, None, 0, 0)
    assert st == 1 and b"null" in L.mona_last_error(h)
    L.mona_destroy(h)
    assert L.mona_query_sizes(None, 0, None, None) == 1
    assert L.mona_step(None, None, None, None, None) == 1


def test_binding_fails_loudly_without_the_library(monkeypatch, L):
    from paper_2605_26842_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", "/nonexistent/libmona.so")
    with pytest.raises(ImportError):
        binding.lib()
