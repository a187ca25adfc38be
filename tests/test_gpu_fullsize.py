"""Parity at the full sizes of the benchmark configurations, in the launch configuration the
benchmark times.  The float64 oracle cannot redo these layers in full within minutes, so:

  stage 1  sampled 64 x 64 tiles of H against the oracle's Hessian of the same rows of X;
  stage 2  the oracle's dampen / invert / factor in full where c <= 4096; for wider layers the
           properties that fix U: upper triangular, positive diagonal, U H_d U^T z = z on probe
           vectors, and dinv_j = (H_d^-1)_jj on sampled columns (float64 on the device);
  stage 3  sampled rows against the oracle fed the library's dinv (rows are independent problems);
  stage 4  sampled rows against the oracle's column loop fed the library's U and grid, over a
           prefix of the columns (column j only depends on columns before it), first differing
           code of a row must be a near-tie of the float64 trajectory; plus two checks over the
           whole layer: W_hat is the grid value of its code everywhere, and the damped proxy loss
           tr((W - W_hat) H_d (W - W_hat)^T) equals twice the summed loss error the library
           returns (an identity of the column loop, Eq. 3 with the Cholesky rows);
  Eq. 7 at T = 2048 on the 8B-shaped down_proj and Algorithm 2 on a 768 x 768 layer: sampled groups / rows."""
import os

import numpy as np
import pytest
import torch

import synth
from oracle import leanquant_oracle as O

pytestmark = pytest.mark.gpu

CODE_TOL = 1e-3
LOSS_TOL = 1e-3
CENT_TOL = 1e-4


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


def check_hessian_tiles(X, H, rng, n_tiles=6, alpha=2.0):
    c = X.shape[0]
    scale = torch.sqrt(torch.diagonal(H)).double().cpu().numpy()
    for t in range(n_tiles):
        i0 = int(rng.integers(0, c - 64))
        j0 = i0 if t == 0 else int(rng.integers(0, c - 64))
        rows = np.r_[i0:i0 + 64, j0:j0 + 64]
        Href = O.hessian(f64(X[torch.from_numpy(rows).cuda()]), alpha)[:64, 64:]
        got = f64(H[i0:i0 + 64, j0:j0 + 64])
        denom = np.outer(scale[i0:i0 + 64], scale[j0:j0 + 64])
        assert np.max(np.abs(got - Href) / denom) < 5e-6, (i0, j0)
    # symmetric
    i0, j0 = int(rng.integers(0, c - 256)), int(rng.integers(0, c - 256))
    assert torch.equal(H[i0:i0 + 256, j0:j0 + 256], H[j0:j0 + 256, i0:i0 + 256].T)


def check_factor_properties(H, U, dinv, damp_frac, rng, n_probe=4, n_cols=6):
    """What fixes U without a float64 factorisation: H_d^-1 = U^T U."""
    c = H.shape[0]
    assert bool((torch.diagonal(U) > 0).all())
    i0 = int(rng.integers(1, c - 64))
    assert float(U[i0:i0 + 64, :i0].abs().max()) == 0.0                   # upper triangular
    Hd = H.double()
    Hd.diagonal().add_(damp_frac * float(torch.diagonal(H).double().mean()))
    Ud = U.double()
    g = torch.Generator(device="cuda").manual_seed(int(rng.integers(1 << 30)))
    z = torch.randn(c, n_probe, generator=g, device="cuda", dtype=torch.float64)
    back = Ud @ (Hd @ (Ud.T @ z))
    assert float((back - z).norm() / z.norm()) < 2e-3
    cols = torch.from_numpy(rng.integers(0, c, size=n_cols)).cuda()
    E = torch.zeros(c, n_cols, device="cuda", dtype=torch.float64)
    E[cols, torch.arange(n_cols, device="cuda")] = 1.0
    Xc = Ud.T @ (Ud @ E)                                                 # columns of H_d^-1
    assert float((Hd @ Xc - E).abs().max()) < 2e-3
    got = dinv[cols].double()
    want = Xc[cols, torch.arange(n_cols, device="cuda")]
    assert float(((got - want).abs() / want).max()) < 1e-5
    del Ud
    return Hd


def tie_ok(codes, codes_o, Wpre, points, tie_tol=2e-4):
    diff = codes != codes_o
    for i in np.nonzero(diff.any(axis=1))[0]:
        j = int(np.argmax(diff[i]))
        pts = points(i, j)
        w = Wpre[i, j]
        k = int(np.argmin(np.abs(pts - w)))
        gaps = np.diff(pts)
        spacing = np.min(gaps[gaps > 0]) if (gaps > 0).any() else 1.0
        assert abs(int(codes[i, j]) - int(codes_o[i, j])) == 1, (i, j)
        assert abs(pts[k] - w) <= tie_tol * max(spacing, abs(w) * 1e-3), (i, j, w, pts[k], spacing)
    return int(diff.any(axis=1).sum())


def run_and_check_layer(lq, h, W, X, kw, seed, n_rows=24, prefix=4096, chunk=None, P=None, reuse_hessian=False,
                        full_stage2=False):
    """One layer through the four calls; returns the LayerPass for further use."""
    rng = np.random.default_rng(seed)
    r, c = W.shape
    n = X.shape[1]
    cfg = lq.Config.make(**kw)
    chunk = chunk or n
    if P is None:
        P = lq.LayerPass(h, r, c, cfg, w_dtype=W.dtype, x_dtype=X.dtype, n_chunk=chunk, device="cuda")
    if not reuse_hessian:
        P.H.zero_()
        for j in range(0, n, chunk):
            P.accumulate(X[:, j:j + chunk])
    P.finish(W, 0.01)
    lq.lq_sync_status(h)

    if not reuse_hessian:
        check_hessian_tiles(X, P.H, rng)
    if full_stage2:
        Uo, dinvo, _, _ = O.prepare_hinv(f64(P.H), 0.01)
        print(f"stage 2 c={c}: max |dU| / max |U| = {np.abs(f64(P.U) - Uo).max() / np.abs(Uo).max():.2e}")
        assert np.abs(f64(P.U) - Uo).max() <= 3e-7 * np.abs(Uo).max()
        np.testing.assert_allclose(f64(P.dinv), dinvo, rtol=3e-7)
        del Uo
    Hd = check_factor_properties(P.H, P.U, P.dinv, 0.01, rng)

    rows = np.sort(rng.choice(r, size=min(n_rows, r), replace=False))
    rows_t = torch.from_numpy(rows).cuda()
    Ws = f64(W[rows_t])
    dinv64 = f64(P.dinv)
    m = min(prefix, c)
    U64 = f64(P.U[:m, :m])
    K = 1 << cfg.bits
    affine = kw["grid"] == "affine"
    if affine:
        g = kw.get("group", 0) or c
        So, Zo = O.fit_grid_affine(Ws, dinv64, cfg.bits, kw["p"], kw.get("group", 0), kw["T"], kw["t"])
        S, Z = f64(P.scale[rows_t]), P.zero[rows_t].cpu().numpy()
        same = (Z == Zo) & (np.abs(S / So - 1) < 1e-6)
        assert same.mean() >= 0.995
        ng = m // g if g <= m else 1
        codes_o, What_o, _, Wpre = O.quantize_layer(Ws[:, :m], U64, scale=S[:, :max(ng, 1)], zero=Z[:, :max(ng, 1)].astype(np.float64),
                                                    bits=cfg.bits, group=(g if g <= m else 0), block=128, return_pre=True)

        def points(i, j):
            return (np.arange(K - 1) + 0.5 - Z[i, j // g]) * S[i, j // g]
    else:
        Go = O.fit_grid_nonuniform(Ws, dinv64, cfg.bits, kw["p"], kw["n_iter"])
        G = f64(P.grid[rows_t])
        span = (Ws.max(1) - Ws.min(1))[:, None] / K
        assert np.all(np.abs(G - Go) <= CENT_TOL * np.maximum(np.abs(Go), span))
        codes_o, What_o, _, Wpre = O.quantize_layer(Ws[:, :m], U64, grid=G, bits=cfg.bits, block=128, return_pre=True)

        def points(i, j):
            return 0.5 * (G[i, :-1] + G[i, 1:])
    codes = P.codes[rows_t][:, :m].cpu().numpy().astype(np.int64)
    n_diverged = tie_ok(codes, codes_o, Wpre, points)      # every divergence must start at a near-tie ...
    assert n_diverged <= max(1, len(rows) // 12), n_diverged   # ... and only a few of the sampled rows may diverge at all
    frac = float((codes != codes_o).mean())                # ... and the sampled codes stay inside the 0.1 % budget
    print(f"{r} x {c} {kw['grid']} {cfg.bits}-bit: {100 * frac:.4f} % of {codes.size} sampled codes differ ({n_diverged} rows)")
    assert frac <= CODE_TOL, frac

    # whole layer: codes in range, W_hat is the grid value of its code, loss identity
    assert int(P.codes.max()) < K
    Wh = P.W_hat.float()
    if affine:
        gsz = kw.get("group", 0) or c
        Sx = P.scale.repeat_interleave(gsz, dim=1)
        Zx = P.zero.repeat_interleave(gsz, dim=1).float()
        want = (P.codes.float() - Zx) * Sx
    else:
        want = torch.gather(P.grid, 1, P.codes.long())
    if P.W_hat.dtype == torch.bfloat16:
        want = want.bfloat16().float()
    assert torch.equal(Wh, want)
    del want
    if P.W_hat.dtype == torch.float32:
        proxy_d = 0.0
        for i0 in range(0, r, 2048):                      # tr(D H_d D^T) in float64 on the device, in row slabs
            D = (W[i0:i0 + 2048].double() - P.W_hat[i0:i0 + 2048].double())
            proxy_d += float(((D @ Hd) * D).sum())
        assert abs(proxy_d / (2.0 * P.loss.item()) - 1.0) <= LOSS_TOL
    del Hd
    return P


def nu(bits, p=4.0):
    return dict(grid="nonuniform", bits=bits, p=p, n_iter=20)


def test_config2_q_proj_full_size(lq, h):
    """Llama-3-8B-shaped q_proj, W 4096 x 4096 bf16, X 4096 x 262144 bf16: 4-bit p=4 with a full
    float64 stage 2, then 3-bit p=2 and 4-bit p=1 reusing the Hessian."""
    L = synth.make_layer("c2", 4096, 4096, 262144, seed=2, device="cuda")
    P = None
    for k, (bits, p) in enumerate([(4, 4.0), (3, 2.0), (4, 1.0)]):
        cfg = lq.Config.make(**nu(bits, p))
        Pk = lq.LayerPass(h, 4096, 4096, cfg, w_dtype=torch.float32, x_dtype=L.X.dtype, n_chunk=262144, device="cuda")
        if P is not None:
            Pk.H = P.H
        P = run_and_check_layer(lq, h, L.W, L.X, nu(bits, p), seed=20 + k, P=Pk, reuse_hessian=k > 0, full_stage2=k == 0)


def test_config3_down_proj_affine_full_size(lq, h):
    """Llama-3-8B-shaped down_proj, W 4096 x 14336 bf16, X 14336 x 131072 (product of Gaussians),
    affine 4-bit, groups of 128, 100 candidates per group (T = 45, t = 9); tokens in two chunks."""
    L = synth.make_layer("c3", 4096, 14336, 131072, seed=3, device="cuda")
    kw = dict(grid="affine", bits=4, p=4.0, group=128, T=45, t=9)
    cfg = lq.Config.make(**kw)
    P = lq.LayerPass(h, 4096, 14336, cfg, w_dtype=torch.float32, x_dtype=L.X.dtype, n_chunk=65536, device="cuda")
    run_and_check_layer(lq, h, L.W, L.X, kw, seed=30, P=P, chunk=65536, n_rows=16)


def test_config4_decoder_block_full_size(lq, h):
    """The linear layers of one Llama-3-8B-shaped decoder block in order, 3-bit non-uniform p = 4,
    131072 tokens; q/k/v share one Hessian and so do gate/up."""
    n = 131072
    shapes = [("attn_in", 4096, [("q", 4096), ("k", 1024), ("v", 1024)]), ("o_in", 4096, [("o", 4096)]),
              ("mlp_in", 4096, [("gate", 14336), ("up", 14336)]), ("down_in", 14336, [("down", 4096)])]
    seed = 40
    for hname, c, layers in shapes:
        recipe = "c3" if hname == "down_in" else "c2"
        X = synth.make_layer(recipe, 8, c, n, seed=seed, device="cuda").X
        Hshared = None
        for lname, r in layers:
            seed += 1
            W = synth.make_layer(recipe, r, c, 8, seed=seed, device="cuda").W
            cfg = lq.Config.make(**nu(3))
            P = lq.LayerPass(h, r, c, cfg, w_dtype=torch.float32, x_dtype=X.dtype, n_chunk=n, device="cuda")
            if Hshared is not None:
                P.H = Hshared
            run_and_check_layer(lq, h, W, X, nu(3), seed=seed, P=P, reuse_hessian=Hshared is not None, n_rows=12,
                                prefix=2048)
            Hshared = P.H
            del P
        del X, Hshared
        torch.cuda.empty_cache()


@pytest.mark.parametrize("name,r,c,kw", [
    ("up_proj-nu2", 53248, 16384, dict(grid="nonuniform", bits=2, p=4.0, n_iter=20)),
    ("up_proj-aff4", 53248, 16384, dict(grid="affine", bits=4, p=4.0, group=128, T=45, t=9)),
    ("down_proj-nu2", 16384, 53248, dict(grid="nonuniform", bits=2, p=4.0, n_iter=20)),
    ("down_proj-aff4", 16384, 53248, dict(grid="affine", bits=4, p=4.0, group=128, T=45, t=9)),
])
def test_config5_405b_mlp_full_size(lq, h, name, r, c, kw):
    """Llama-3.1-405B-shaped MLP layers (H up to 53248^2 fp32), heavy-tailed X at 65536 tokens
    streamed in chunks of 8192."""
    torch.cuda.empty_cache()
    n = 65536
    L = synth.make_layer("c3", r, c, n, seed=50 + len(name), device="cuda")
    cfg = lq.Config.make(**kw)
    P = lq.LayerPass(h, r, c, cfg, w_dtype=torch.float32, x_dtype=L.X.dtype, n_chunk=8192, device="cuda")
    run_and_check_layer(lq, h, L.W, L.X, kw, seed=50, P=P, chunk=8192, n_rows=8, prefix=2048)
    del P, L
    torch.cuda.empty_cache()


def test_affine_search_at_the_papers_granularity_full_size(lq, h):
    """Eq. 7 with T = 2048, t = 409 (168100 candidates per group) on the 8B-shaped down_proj, 458752 groups of 128, as
    the benchmark times it; sampled groups against the oracle's all-candidate search."""
    r, c, g, T, t, bits = 4096, 14336, 128, 2048, 409, 4
    L = synth.make_layer("c3", r, c, 256, seed=61, device="cuda")
    gen = torch.Generator().manual_seed(62)
    dinv = torch.exp(0.5 * torch.randn(c, generator=gen)).cuda()
    cfg = lq.Config.make(grid="affine", bits=bits, p=4.0, group=g, T=T, t=t)
    scale = torch.empty(r, c // g, device="cuda")
    zero = torch.empty(r, c // g, dtype=torch.int32, device="cuda")
    ws = torch.empty(max(lq.lq_fit_grid_workspace(cfg, r, c), 256), dtype=torch.uint8, device="cuda")
    lq.lq_fit_grid(h, cfg, L.W, dinv, ws, scale=scale, zero=zero)
    lq.lq_sync_status(h)
    rng = np.random.default_rng(63)
    rows = np.sort(rng.choice(r, 6, replace=False))
    s = O.sample_weights(f64(dinv), 4.0)
    K = 1 << bits
    n_same = 0
    for gi in rng.choice(c // g, 2, replace=False):
        w = f64(L.W[torch.from_numpy(rows).cuda(), gi * g:(gi + 1) * g])
        sg = s[gi * g:(gi + 1) * g]
        So, Zo = O.affine_search_group(w, sg, K, T, t)
        Sg, Zg = f64(scale[torch.from_numpy(rows).cuda(), gi]), zero[torch.from_numpy(rows).cuda(), gi].cpu().numpy()
        for k in range(len(rows)):
            if Zg[k] == Zo[k] and abs(Sg[k] / So[k] - 1) < 1e-6:
                n_same += 1
                continue
            # another member of the winning class, or a tie to rounding: same loss by the oracle's arithmetic
            loss_ref = (sg * (O.quant_aff(w[k], So[k], Zo[k], K) - w[k]) ** 2).sum()
            loss_gpu = (sg * (O.quant_aff(w[k], Sg[k], float(Zg[k]), K) - w[k]) ** 2).sum()
            assert loss_gpu <= loss_ref * (1 + 1e-5)        # S went through fp32 on the way out
    assert n_same >= 10
    assert torch.isfinite(scale).all() and (scale > 0).all()


def test_exact_full_size_bert_base_layer(lq, h):
    """Algorithm 2 on a 768 x 768 layer (as the benchmark times it): sampled rows against the oracle fed the library's
    factor and grid, and the quadratic-loss identity over the whole layer."""
    r, c, bits = 768, 768, 4
    L = synth.make_layer("c2", r, c, 8192, seed=71, device="cuda")
    cfg = lq.Config.make(grid="nonuniform", bits=bits, p=4.0, n_iter=20)
    P = lq.LayerPass(h, r, c, cfg, w_dtype=torch.float32, x_dtype=L.X.dtype, n_chunk=L.n, device="cuda")
    P.H.zero_()
    P.accumulate(L.X)
    lq.lq_hessian_finalize(h, P.H)
    lq.lq_prepare_hinv(h, P.H, P.U, P.dinv, P.ws, 0.01, L.W)
    lq.lq_fit_grid(h, cfg, L.W, P.dinv, P.ws, P.grid, P.scale, P.zero)
    ws = torch.empty(lq.lq_quantize_exact_workspace(cfg, r, c), dtype=torch.uint8, device="cuda")
    codes = torch.empty((r, c), dtype=torch.uint8, device="cuda")
    what = torch.empty((r, c), dtype=torch.float32, device="cuda")
    loss = torch.zeros(1, dtype=torch.float64, device="cuda")
    lq.lq_quantize_exact(h, cfg, L.W, P.U, codes, ws, P.grid, None, None, what, loss)
    lq.lq_sync_status(h)
    U = f64(P.U)
    Hinv = U.T @ U
    rows = np.array([0, 301, 767])
    co, wo, lo = O.quantize_exact(f64(L.W)[rows], Hinv, grid=f64(P.grid)[rows], bits=bits)
    cg = codes.cpu().numpy().astype(np.int64)[rows]
    assert (cg == co).all(axis=1).sum() >= 2                      # a row may differ through an exact tie only
    same = (cg == co).all(axis=1)
    np.testing.assert_allclose(f64(what)[rows][same], wo[same], rtol=1e-6, atol=1e-9)
    D = f64(L.W) - f64(what)
    H_d = np.linalg.inv(Hinv)
    np.testing.assert_allclose(loss.item(), 0.5 * np.einsum("ri,ij,rj->", D, H_d, D), rtol=1e-6)
