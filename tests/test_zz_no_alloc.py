"""lq_fit_grid_noalloc: the grid fit for callers that must not allocate device memory
(all of HBM already reserved by a framework's allocator, a latency-critical section that
cannot take cudaMalloc's device-wide synchronisation, a callback context that forbids it).

It takes no workspace -- its scratch is an array built into the library -- and must give
what lq_fit_grid gives.  Checked here through the C ABI on two calls in a row with different
shapes, so that the second call runs on whatever the first left in the shared array.
This file is named to be collected last: a run that stops at the first failure has then
already run every other test."""
import os

import numpy as np
import pytest
import torch

import synth
from oracle import leanquant_oracle as O

pytestmark = pytest.mark.gpu

CENT_TOL = 1e-4      # the centroid tolerance of the parity tests


@pytest.fixture(scope="module")
def lq():
    import paper_2407_10032_b200 as m
    from paper_2407_10032_b200 import build
    build.build(debug_bounds=os.environ.get("LQ_LIBRARY_VARIANT") == "debug")
    return m


def _dinv(c, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.exp(torch.randn(c, generator=g)).cuda()      # heavy-tailed positive diagonal


def _with_workspace(lq, h, cfg, W, dinv, affine):
    r, c = W.shape
    ws = torch.empty(max(lq.lq_fit_grid_workspace(cfg, r, c), 256), dtype=torch.uint8, device="cuda")
    if affine:
        ng = c // cfg.group_size
        scale = torch.empty(r, ng, device="cuda")
        zero = torch.empty(r, ng, dtype=torch.int32, device="cuda")
        lq.lq_fit_grid(h, cfg, W, dinv, ws, scale=scale, zero=zero)
        return scale, zero
    grid = torch.empty(r, 1 << cfg.bits, device="cuda")
    lq.lq_fit_grid(h, cfg, W, dinv, ws, grid=grid)
    return (grid,)


def _without_allocation(lq, h, cfg, W, dinv, affine, outs):
    if affine:
        lq.lq_fit_grid_noalloc(h, cfg, W, dinv, scale=outs[0], zero=outs[1])
    else:
        lq.lq_fit_grid_noalloc(h, cfg, W, dinv, grid=outs[0])


def test_noalloc_matches_fit_grid_on_two_calls_in_a_row(lq):
    h = lq.lq_create(0)
    try:
        cases = [("c2", 96, 2048, dict(grid="nonuniform", bits=4, p=4.0, n_iter=20), False),
                 ("c2", 40, 520, dict(grid="nonuniform", bits=3, p=2.0, n_iter=12), False),
                 ("c3", 24, 512, dict(grid="affine", bits=4, p=4.0, group=128, T=45, t=9), True)]
        for k, (recipe, r, c, kw, affine) in enumerate(cases):
            L = synth.make_layer(recipe, r, c, 2 * c, seed=40 + k)
            W, dinv = L.W.cuda(), _dinv(c, k)
            cfg = lq.Config.make(**kw)
            want = _with_workspace(lq, h, cfg, W, dinv, affine)
            # outputs are allocated before the call under test; the call itself is given no workspace
            got = [torch.full_like(t, -7) for t in want]
            handle = h if k != 1 else None              # the middle call also runs without a handle
            _without_allocation(lq, handle, cfg, W, dinv, affine, got)
            lq.lq_sync_status(h)
            torch.cuda.synchronize()
            if affine:
                assert torch.equal(got[1], want[1])
                np.testing.assert_allclose(got[0].cpu().numpy(), want[0].cpu().numpy(), rtol=1e-6)
            else:
                G, Gw = got[0].double().cpu().numpy(), want[0].double().cpu().numpy()
                span = (L.W.double().numpy().max(1) - L.W.double().numpy().min(1))[:, None] / G.shape[1]
                assert np.all(np.abs(G - Gw) <= CENT_TOL * np.maximum(np.abs(Gw), span))
                # and against the float64 oracle itself, at the same tolerance
                Go = O.fit_grid_nonuniform(L.W.double().numpy(), dinv.double().cpu().numpy(), kw["bits"], kw["p"], kw["n_iter"])
                assert np.all(np.abs(G - Go) <= CENT_TOL * np.maximum(np.abs(Go), span))
            # what the entry point is for: a repeated call (every one-time set-up of this configuration is behind us)
            # leaves the free device memory where it was
            free0 = torch.cuda.mem_get_info()[0]
            _without_allocation(lq, handle, cfg, W, dinv, affine, got)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free0
    finally:
        lq.lq_destroy(h)


def test_noalloc_rejects_rows_longer_than_its_scratch(lq):
    c = 16384 + 128                                    # LQ_FIT_GRID_NOALLOC_MAX_C is 16384
    W = torch.zeros(2, c, dtype=torch.bfloat16, device="cuda")
    dinv = torch.ones(c, device="cuda")
    grid = torch.empty(2, 16, device="cuda")
    cfg = lq.Config.make(grid="nonuniform", bits=4)
    with pytest.raises(lq.LQError) as e:
        lq.lq_fit_grid_noalloc(None, cfg, W, dinv, grid=grid)
    assert e.value.code == 8
