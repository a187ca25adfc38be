"""Parity of lq_quantize_exact (Algorithm 2, LeanQuant-Exact) with the float64 oracle, through the C ABI.

Isolated: the oracle runs on the inverse U^T U of the factor the GPU produced (widened to float64) and on
the GPU's grid, so that only the greedy loop itself is compared: its order, codes and loss must agree to
rounding.  Chained: everything from X on, against the oracle's own float64 pass, within the tolerances of the
other parity tests (0.1 % of codes, 1e-3 on the loss)."""
import os

import numpy as np
import pytest
import torch

import synth
from oracle import leanquant_oracle as O

pytestmark = pytest.mark.gpu

CODE_TOL = 1e-3
LOSS_TOL = 1e-3


@pytest.fixture(scope="module")
def lq():
    import paper_2407_10032_b200 as m
    from paper_2407_10032_b200 import build
    build.build(debug_bounds=os.environ.get("LQ_LIBRARY_VARIANT") == "debug")
    return m


@pytest.fixture(scope="module")
def h(lq):
    handle = lq.lq_create(0)
    yield handle
    lq.lq_destroy(handle)


def f64(t):
    return t.detach().double().cpu().numpy()


def gpu_front(lq, h, L, cfg):
    """Stages 1-3 on the GPU; returns the pass object with U, dinv and the grid filled in."""
    P = lq.LayerPass(h, L.r, L.c, cfg, w_dtype=torch.float32, x_dtype=L.X.dtype, n_chunk=L.n, device="cuda")
    W = L.W.cuda()
    P.H.zero_()
    P.accumulate(L.X.cuda())
    lq.lq_hessian_finalize(h, P.H)
    lq.lq_prepare_hinv(h, P.H, P.U, P.dinv, P.ws, 0.01, W)
    lq.lq_fit_grid(h, cfg, W, P.dinv, P.ws, P.grid, P.scale, P.zero)
    return P, W


def run_exact_gpu(lq, h, cfg, W, P):
    r, c = W.shape
    ws = torch.empty(max(lq.lq_quantize_exact_workspace(cfg, r, c), 256), dtype=torch.uint8, device="cuda")
    codes = torch.full((r, c), 255, dtype=torch.uint8, device="cuda")
    what = torch.empty((r, c), dtype=torch.float32, device="cuda")
    loss = torch.zeros(1, dtype=torch.float64, device="cuda")
    lq.lq_quantize_exact(h, cfg, W, P.U, codes, ws, P.grid, P.scale, P.zero, what, loss)
    lq.lq_sync_status(h)
    return codes.cpu().numpy().astype(np.int64), f64(what), loss.item()


@pytest.mark.parametrize("recipe,r,c,n,kw", [
    ("c2", 24, 160, 1024, dict(grid="nonuniform", bits=4, p=4.0, n_iter=10)),       # five batches of 32 steps
    ("c1", 9, 72, 512, dict(grid="nonuniform", bits=2, p=2.0, n_iter=10)),          # ragged: less than one 128-wide strip
    ("c2", 40, 300, 2048, dict(grid="nonuniform", bits=3, p=4.0, n_iter=10)),
    ("c3", 16, 256, 1024, dict(grid="affine", bits=4, p=4.0, group=32, T=40, t=8)),
    ("c3", 6, 132, 1024, dict(grid="affine", bits=3, p=4.0, group=0, T=40, t=8)),   # ragged width, one group per row
    ("c2", 700, 64, 512, dict(grid="nonuniform", bits=3, p=4.0, n_iter=5)),         # more rows than resident CTAs: each CTA takes several
])
def test_exact_loop_isolated(lq, h, recipe, r, c, n, kw):
    L = synth.make_layer(recipe, r, c, n, seed=r + c)
    cfg = lq.Config.make(**kw)
    P, W = gpu_front(lq, h, L, cfg)
    codes, what, loss = run_exact_gpu(lq, h, cfg, W, P)
    U = f64(P.U)
    Hinv = U.T @ U
    if kw["grid"] == "nonuniform":
        ref = O.quantize_exact(f64(W), Hinv, grid=f64(P.grid), bits=kw["bits"])
    else:
        ref = O.quantize_exact(f64(W), Hinv, scale=f64(P.scale), zero=f64(P.zero), bits=kw["bits"], group=kw["group"])
    codes_o, what_o, loss_o = ref
    assert codes.max() < (1 << kw["bits"])                          # every weight was visited
    rows_same = (codes == codes_o).all(axis=1)
    assert rows_same.mean() >= 0.95                                 # a row differs only through an exact tie
    np.testing.assert_allclose(what[rows_same], what_o[rows_same], rtol=1e-6, atol=1e-9)
    if rows_same.all():
        np.testing.assert_allclose(loss, loss_o, rtol=1e-9)
    # the sum of the loss errors is the quadratic loss of the result, whatever happened on the way
    H_d = np.linalg.inv(Hinv)
    D = f64(W) - what
    np.testing.assert_allclose(loss, 0.5 * np.einsum("ri,ij,rj->", D, H_d, D), rtol=1e-6)


def test_exact_chained(lq, h):
    L = synth.make_layer("c2", 48, 256, 4096, seed=77)
    kw = dict(grid="nonuniform", bits=3, p=4.0, n_iter=20)
    cfg = lq.Config.make(**kw)
    P, W = gpu_front(lq, h, L, cfg)
    codes, what, loss = run_exact_gpu(lq, h, cfg, W, P)
    ref = O.run_exact(f64(L.W), f64(L.X), bits=3, p=4.0, n_iter=20)
    assert (codes != ref["codes"]).mean() <= max(CODE_TOL, 2.0 / codes.size)
    assert abs(loss / ref["loss"] - 1) <= LOSS_TOL
    proxy = O.proxy_loss(f64(L.W), what, ref["H"])
    assert abs(proxy / ref["proxy"] - 1) <= LOSS_TOL


def test_exact_rejects_bad_arguments(lq, h):
    cfg = lq.Config.make(grid="nonuniform", bits=4)
    with pytest.raises(lq.LQError) as e:
        lq.lq_quantize_exact_workspace(cfg, 4, 8192 + 128)
    assert e.value.code == 2
    W = torch.zeros(4, 64, device="cuda")
    U = torch.eye(64, device="cuda")
    grid = torch.zeros(4, 16, device="cuda")
    codes = torch.empty(4, 64, dtype=torch.uint8, device="cuda")
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(lq.LQError) as e:
        lq.lq_quantize_exact(h, cfg, W, U, codes, small, grid)
    assert e.value.code == 3
