"""Host-side checks of the C-ABI library that need no GPU: it loads, it exports every
symbol the header declares, its size queries and argument checks work."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2407_10032_b200 import build
    build.build(debug_bounds=os.environ.get("LQ_LIBRARY_VARIANT") == "debug")
    import paper_2407_10032_b200 as lq
    return lq


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "lq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"lq_hessian_accumulate", "lq_prepare_hinv", "lq_fit_grid", "lq_quantize_layer"} <= set(names)
    cdll = C.CDLL(lib.library_path())
    for n in names:
        assert hasattr(cdll, n), f"{n} declared in lq.h but not exported"


def test_version_and_launch_counter(lib):
    assert "sm_100a" in lib.lq_version()
    assert lib.lq_launch_count() >= 0


def test_workspace_queries(lib):
    import torch
    assert lib.lq_hessian_workspace(torch.bfloat16, 4096, 1 << 18) == 0
    assert lib.lq_hessian_workspace(torch.float32, 512, 8192) >= 3 * 512 * 8192 * 2
    assert lib.lq_hessian_workspace(torch.bfloat16, 512, 8192, token_major=True) >= 512 * 8192 * 2
    assert lib.lq_prepare_hinv_workspace(200) >= 256 * 256 * 8          # padded to the 128-wide panel
    cfg = lib.Config.make(grid="nonuniform", bits=4)
    assert lib.lq_fit_grid_workspace(cfg, 16, 4096) >= 4096 * 8
    need = lib.lq_quantize_layer_workspace(cfg, 512, 512)
    assert need >= 512 * 512 * 4 + 3 * 512 * 512 * 2 + 3 * 512 * 128 * 2


def test_bad_configs_are_rejected_on_the_host(lib):
    bad = lib.Config.make(grid="nonuniform", bits=5)
    with pytest.raises(lib.LQError) as e:
        lib.lq_fit_grid_workspace(bad, 8, 128)
    assert e.value.code == 1
    bad = lib.Config.make(grid="nonuniform", bits=4, block=64)
    with pytest.raises(lib.LQError) as e:
        lib.lq_quantize_layer_workspace(bad, 8, 128)
    assert e.value.code == 2
    bad = lib.Config.make(grid="affine", bits=4, T=10, t=6)       # t > T/2
    with pytest.raises(lib.LQError):
        lib.lq_fit_grid_workspace(bad, 8, 128)
    with pytest.raises(lib.LQError):
        lib.lq_prepare_hinv_workspace(0)


def test_no_device_means_failure_not_fallback(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(lib.LQError) as e:
        lib.lq_create(0)
    assert e.value.code == 6


def test_default_shrink_counts(lib):
    assert lib.Config.make(grid="affine", bits=4).t_count == 409
    assert lib.Config.make(grid="affine", bits=3).t_count == 614
    assert lib.Config.make(grid="affine", bits=2).t_count == 819
