"""Host-side checks of the C-ABI library that need no GPU: it builds, loads, exports every symbol
the header declares, and rejects bad arguments before touching a device."""
import ctypes as C
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2506_17974_b200 import binding as B
from paper_2506_17974_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    entry.build()
    return B.load_library()


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "lqsgd.h")).read()
    body = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(lqsgd_[a-z0-9_]+)\s*\(", body))
    assert declared == set(B.EXPORTED), declared ^ set(B.EXPORTED)
    for name in declared:
        assert hasattr(lib, name), name
    assert lib.lqsgd_version() == 1


def test_config_struct_matches_header_layout():
    assert C.sizeof(B.Config) == 48 and C.sizeof(B.Shape) == 8 and C.sizeof(B.LayerLayout) == 64
    assert C.sizeof(B.LayerStats) == 64 and B.LayerStats.codes_p.offset == 24 and B.LayerStats.payload_bytes.offset == 56


def test_workspace_bytes_covers_the_persistent_state(lib):
    for w in (wl.config1(), wl.config2(), wl.config3(), wl.config4(4096, 4096), wl.config5(16, 8)):
        cfg = B.make_config(w.rank, w.bits, w.bits, w.alpha, w.workers)
        nbytes = B.workspace_bytes(w.layers, cfg)
        e_bytes = 4 * w.workers * wl.matrix_elements(w.layers)           # the error buffers alone
        assert nbytes >= e_bytes
        assert nbytes <= 1.35 * e_bytes + (64 << 20), (w.name, nbytes, e_bytes)
        staged = B.make_config(w.rank, w.bits, w.bits, w.alpha, w.workers, flags=B.FLAG_HOST_STAGING)
        assert B.workspace_bytes(w.layers, staged) >= nbytes + 4 * (w.workers + 1) * sum(n * m for n, m in w.layers)


@pytest.mark.parametrize("kw,code", [
    (dict(rank=0), B.ERR_INVALID_ARG), (dict(rank=65), B.ERR_INVALID_ARG),
    (dict(bits_p=1), B.ERR_INVALID_ARG), (dict(bits_q=9), B.ERR_INVALID_ARG),
    (dict(alpha=0.0), B.ERR_INVALID_ARG), (dict(alpha=float("nan")), B.ERR_INVALID_ARG),
    (dict(workers=0), B.ERR_INVALID_ARG), (dict(workers=257), B.ERR_INVALID_ARG),
    (dict(flags=256), B.ERR_INVALID_ARG), (dict(flags=128), B.ERR_INVALID_ARG), (dict(power_iters=9), B.ERR_INVALID_ARG), (dict(power_iters=-1), B.ERR_INVALID_ARG),
    (dict(power_iters=2, world_workers=2), B.ERR_INVALID_ARG),
])
def test_bad_config_is_rejected_on_the_host(lib, kw, code):
    base = dict(rank=2, bits_p=4, bits_q=4, alpha=127.0, workers=1, seed=0, flags=0)
    base.update(kw)
    cfg = B.make_config(**base)
    with pytest.raises(B.LqsgdError) as e:
        B.workspace_bytes([(8, 8)], cfg)
    assert e.value.code == code


def test_column_scales_flag_changes_only_the_scale_bytes(lib):
    layers = [(96, 200), (20, 1), (3, 5)]
    plain = B.workspace_bytes(layers, B.make_config(4, 4, 4, 127.0, 2))
    cols = B.workspace_bytes(layers, B.make_config(4, 4, 4, 127.0, 2, flags=B.FLAG_COLUMN_SCALES))
    assert plain <= cols <= plain + (1 << 16)


def test_bad_shapes_struct_size_and_null_pointers(lib):
    cfg = B.make_config(2, 4, 4, 127.0, 1)
    for bad in ([(0, 5)], [(4, -1)], [(1 << 16, 1 << 15)]):
        with pytest.raises(B.LqsgdError) as e:
            B.workspace_bytes(bad, cfg)
        assert e.value.code == B.ERR_BAD_SHAPE
    cfg2 = B.make_config(2, 4, 4, 127.0, 1)
    cfg2.struct_size = 12
    with pytest.raises(B.LqsgdError) as e:
        B.workspace_bytes([(8, 8)], cfg2)
    assert e.value.code == B.ERR_INVALID_ARG
    shapes = (B.Shape * 1)(B.Shape(8, 8))
    ctx = C.c_void_p()
    # null workspace / misaligned workspace / null outputs: refused before any CUDA call
    assert lib.lqsgd_create(shapes, 1, C.byref(cfg), None, 1 << 20, C.byref(ctx)) == B.ERR_INVALID_ARG
    assert lib.lqsgd_create(shapes, 1, C.byref(cfg), C.c_void_p(0x1001), 1 << 30, C.byref(ctx)) == B.ERR_MISALIGNED
    assert lib.lqsgd_create(shapes, 1, C.byref(cfg), C.c_void_p(0x1000), 16, C.byref(ctx)) == B.ERR_WORKSPACE_TOO_SMALL
    assert lib.lqsgd_workspace_bytes(shapes, 1, C.byref(cfg), None) == B.ERR_INVALID_ARG
    assert lib.lqsgd_step(None, None, None, None) == B.ERR_INVALID_ARG
    assert lib.lqsgd_strerror(B.ERR_MISALIGNED).decode() == "misaligned pointer"
    lib.lqsgd_destroy(None)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(FileNotFoundError):
        B.load_library()
