"""Pins for the float64 oracle: each test checks it against something that is not
the oracle itself -- a brute-force statement of the paper's equations, a closed
form, a value the paper prints, or a textbook library routine.  CPU only."""
import itertools
import os

import numpy as np
import pytest
import torch

import synth
from oracle import leanquant_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.default_rng(seed)


def spd(c, seed, cond=1e3):
    """Random symmetric positive definite matrix with a prescribed spectrum."""
    g = rng(seed)
    Q, _ = np.linalg.qr(g.standard_normal((c, c)))
    lam = np.logspace(0, np.log10(cond), c)
    return (Q * lam) @ Q.T


# Linear layers of one Llama-3-8B-shaped decoder block, (r, c): what the paper's bit widths average over.
LLAMA3_8B_BLOCK = [(4096, 4096), (1024, 4096), (1024, 4096), (4096, 4096), (14336, 4096), (14336, 4096), (4096, 14336)]


def test_record_format_costs_the_bits_the_paper_prints():
    """Codes plus a 2^b-entry fp16 table per row (non-uniform) or an fp16 scale and a 16-bit zero point per group
    (affine), averaged over the linear layers of a Llama-3-8B-shaped block, give the bit widths of the paper's tables
    to the two decimals it prints (4.0505 -> 4.05, 3.0252 -> 3.02, 2.0126 -> 2.01, 4.0063 -> 4.00: the printed figures
    are the averages cut after two decimals).  A table per 128 columns, fp32 tables, or (S, Z) stored wider would not."""
    total = sum(r * c for r, c in LLAMA3_8B_BLOCK)
    for line in open(os.path.join(GOLDEN, "table_bits.txt")):
        if line.startswith("#") or not line.strip():
            continue
        grid_type, bits, group, printed = line.split()
        avg = sum(r * c * O.record_bits_per_weight(int(bits), c, grid_type, int(group)) for r, c in LLAMA3_8B_BLOCK) / total
        assert int(avg * 100 + 1e-9) == round(float(printed) * 100), (line, avg)


def test_pack_layer_by_hand_and_round_trip():
    g = rng(21)
    # non-uniform, 2 bits, 3 x 5: header fields, section offsets, table bytes and the weights it stands for
    codes = g.integers(0, 4, size=(3, 5))
    grid = np.sort(g.standard_normal((3, 4)), axis=1)
    rec = O.pack_layer(codes, 2, grid=grid)
    assert rec[:4].tobytes() == b"LQP1" and rec.dtype == np.uint8
    assert list(rec[4:16].view("<u4")) == [2, 0, 0]
    r, c, oc, ot, oz, tot = (int(v) for v in rec[16:64].view("<i8"))
    assert (r, c, oc) == (3, 5, 64) and ot == 64 + 16 and tot == ot + 32 and oz == tot and tot == rec.size
    assert np.array_equal(rec[oc:oc + 6].reshape(3, 2), O.pack_codes(codes, 2))
    t16 = rec[ot:ot + 24].view(np.float16).reshape(3, 4)
    assert np.array_equal(t16, grid.astype(np.float16))
    np.testing.assert_array_equal(O.unpack_layer(rec), np.take_along_axis(grid.astype(np.float16).astype(np.float64), codes, 1))
    # affine, 4 bits, groups of 8 in a 2 x 16 layer
    codes = g.integers(0, 16, size=(2, 16))
    S = np.abs(g.standard_normal((2, 2))) * 0.01 + 0.001
    Z = g.integers(-3, 12, size=(2, 2)).astype(np.float64)
    rec = O.pack_layer(codes, 4, scale=S, zero=Z, group=8)
    assert list(rec[4:16].view("<u4")) == [4, 1, 8]
    want = (codes - np.repeat(Z, 8, axis=1)).astype(np.float32) * np.repeat(S.astype(np.float16).astype(np.float32), 8, axis=1)
    np.testing.assert_array_equal(O.unpack_layer(rec), want.astype(np.float64))
    assert rec.size == 64 + 16 + 16 + 16


# ------------------------------------------------------------------ P1 ---- #
def obq_fixed_order(W, Hinv, quant_row, order=None):
    """Eq. 3 and Eq. 9 taken literally, column by column in fixed order (left to right, or the given `order`):
    quantise w_j, w <- w - (w_j - q)/Hinv_jj * Hinv[:, j], then remove row/column j
    from the inverse by Hinv <- Hinv - Hinv[:, j] Hinv[j, :]/Hinv_jj."""
    W = W.copy()
    Hinv = Hinv.copy()
    r, c = W.shape
    Q = np.zeros_like(W)
    eps = 0.0
    for j in (range(c) if order is None else order):
        d = Hinv[j, j]
        for k in range(r):
            q = quant_row(k, j, W[k, j])
            Q[k, j] = q
            delta = (q - W[k, j]) / d * Hinv[:, j]
            eps += 0.5 * (q - W[k, j]) ** 2 / d
            W[k, :] += delta
            W[k, j] = q
        Hinv = Hinv - np.outer(Hinv[:, j], Hinv[j, :]) / d
    return Q, eps


@pytest.mark.parametrize("c,block", [(8, 3), (24, 8), (48, 128), (64, 16)])
def test_p1_column_loop_equals_explicit_obq(c, block):
    g = rng(c)
    r = 5
    W = g.standard_normal((r, c)) * 0.05
    H = spd(c, 7 + c, 1e2)
    U, dinv, H_d, _ = O.prepare_hinv(H, 0.01)
    grid = np.sort(g.standard_normal((r, 4)) * 0.05, axis=1)

    def quant_row(k, j, w):
        return grid[k, np.argmin(np.abs(grid[k] - w))]

    Q_ref, eps_ref = obq_fixed_order(W, np.linalg.inv(H_d), quant_row)
    codes, What, loss = O.quantize_layer(W, U, grid=grid, bits=2, block=block)
    assert np.array_equal(np.take_along_axis(grid, codes, 1), What)
    np.testing.assert_allclose(What, Q_ref, rtol=0, atol=1e-10)
    np.testing.assert_allclose(loss, eps_ref, rtol=1e-9)


def test_activation_order_is_obq_in_that_order():
    """Activation ordering = the same loop with the columns taken in the order of decreasing diag(H).  The oracle permutes
    the layer, runs the pass and puts the outputs back; the pin takes Eq. 3 / Eq. 9 on the layer as it is and simply visits
    the columns in that order.  (A wrong inverse permutation, or H permuted on one side only, fails it.)"""
    g = rng(31)
    r, c = 4, 40
    X = g.standard_normal((c, 300)) * np.exp(g.standard_normal((c, 1)))
    X[7] = X[3]                                        # two channels with the same diagonal entry: ties keep index order
    W = g.standard_normal((r, c)) * 0.05
    H = O.hessian(X)
    perm = O.act_order(H)
    d = np.diag(H)[perm]
    assert (np.diff(d) <= 0).all() and sorted(perm) == list(range(c))
    assert list(perm).index(3) + 1 == list(perm).index(7)
    out = O.run_pass(W, X, bits=3, p=2.0, block=16, n_iter=5, act_ordering=True)
    grid = out["grid"]

    def quant_row(k, j, w):
        return grid[k, O.assign_nu(np.array([w]), grid[k])[0]]

    _, _, H_d, _ = O.prepare_hinv(H, 0.01)
    Q_ref, eps_ref = obq_fixed_order(W, np.linalg.inv(H_d), quant_row, order=perm)
    np.testing.assert_allclose(out["W_hat"], Q_ref, rtol=0, atol=1e-10)
    np.testing.assert_allclose(out["loss"], eps_ref, rtol=1e-9)
    assert np.array_equal(np.take_along_axis(grid, out["codes"], 1), out["W_hat"])
    plain = O.run_pass(W, X, bits=3, p=2.0, block=16, n_iter=5)
    assert not np.array_equal(plain["codes"], out["codes"])          # the order matters


def test_p1b_block_size_does_not_matter():
    g = rng(3)
    r, c = 6, 40
    W = g.standard_normal((r, c))
    U, *_ = O.prepare_hinv(spd(c, 11, 1e3), 0.01)
    grid = O.grid_init_uniform(W.min(1), W.max(1), 8)
    ref = O.quantize_layer(W, U, grid=grid, bits=3, block=c)
    for B in (1, 7, 16, 128):
        out = O.quantize_layer(W, U, grid=grid, bits=3, block=B)
        assert np.array_equal(out[0], ref[0])
        np.testing.assert_allclose(out[2], ref[2], rtol=1e-12)


# ------------------------------------------------------------------ P2 ---- #
def test_p2_damped_proxy_equals_twice_loss():
    g = rng(5)
    r, c = 7, 32
    W = g.standard_normal((r, c)) * 0.1
    X = g.standard_normal((c, 100)) * np.exp(g.standard_normal(c))[:, None]
    out = O.run_pass(W, X, bits=3, block=8, n_iter=5)
    np.testing.assert_allclose(out["proxy_d"], 2.0 * out["loss"], rtol=1e-9)


# ------------------------------------------------------------------ P3 ---- #
def test_p3_identity_hessian_is_round_to_nearest():
    g = rng(9)
    r, c = 9, 50
    W = g.standard_normal((r, c))
    U, dinv, _, _ = O.prepare_hinv(np.eye(c), 0.01)
    assert np.allclose(U, np.diag(np.diag(U)))
    G = O.fit_grid_nonuniform(W, dinv, 3, 4.0, 10)
    codes, What, _ = O.quantize_layer(W, U, grid=G, bits=3, block=16)
    nearest = np.abs(W[:, :, None] - G[:, None, :]).argmin(-1)
    assert np.array_equal(codes, nearest)
    assert np.array_equal(What, np.take_along_axis(G, nearest, 1))


# ------------------------------------------------------------------ P4 ---- #
def kmeans_dp_optimum(w, s, K):
    """Optimal weighted 1-D K-means cost by dynamic programming over sorted points:
    clusters of a 1-D optimum are contiguous in sorted order."""
    order = np.argsort(w)
    w, s = w[order], s[order]
    n = len(w)

    def cost(a, b):  # points a..b-1 in one cluster
        ss = s[a:b].sum()
        mu = (s[a:b] * w[a:b]).sum() / ss
        return (s[a:b] * (w[a:b] - mu) ** 2).sum()

    D = np.full((K + 1, n + 1), np.inf)
    D[0, 0] = 0.0
    for k in range(1, K + 1):
        for b in range(1, n + 1):
            for a in range(k - 1, b):
                if D[k - 1, a] < np.inf:
                    D[k, b] = min(D[k, b], D[k - 1, a] + cost(a, b))
    return D[1:, n].min()


def objective(w, s, grid):
    return float((s * (np.abs(w[:, None] - grid[None, :]).min(1)) ** 2).sum())


def test_p4_lloyd_vs_dp_optimum():
    g = rng(21)
    for trial in range(6):
        c, K = 20, 4
        w = g.standard_normal(c)
        dinv = np.exp(g.standard_normal(c))
        s = O.sample_weights(dinv, 2.0)
        G, trace = O.fit_grid_nonuniform(w[None], dinv, 2, 2.0, 30, return_trace=True)
        opt = kmeans_dp_optimum(w, s, K)
        assert objective(w, s, G[0]) >= opt * (1 - 1e-12)
        assert all(b <= a * (1 + 1e-12) for a, b in zip(trace, trace[1:]))
        np.testing.assert_allclose(trace[-1], objective(w, s, G[0]), rtol=1e-12)
    # four well-separated clumps: Lloyd from the evenly spaced start reaches the optimum
    centres = np.array([-3.0, -1.0, 1.0, 3.0])
    w = (centres[:, None] + 0.05 * g.standard_normal((4, 6))).ravel()
    dinv = np.exp(0.3 * g.standard_normal(w.size))
    s = O.sample_weights(dinv, 4.0)
    G = O.fit_grid_nonuniform(w[None], dinv, 2, 4.0, 20)
    np.testing.assert_allclose(objective(w, s, G[0]), kmeans_dp_optimum(w, s, 4), rtol=1e-10)


# ------------------------------------------------------------------ P5 ---- #
def plain_lloyd(w, K, n_iter):
    """Unweighted Lloyd from evenly spaced centres, written with explicit loops."""
    lo, hi = min(w), max(w)
    g = [lo + (hi - lo) * t / (K - 1) for t in range(K)]
    for _ in range(n_iter):
        members = [[] for _ in range(K)]
        for x in w:
            best = 0
            for k in range(1, K):
                if abs(x - g[k]) < abs(x - g[best]):
                    best = k
            members[best].append(x)
        g = [sum(m) / len(m) if m else g[k] for k, m in enumerate(members)]
    return g


def test_p5_p_zero_is_plain_lloyd():
    g = rng(33)
    W = g.standard_normal((4, 200))
    dinv = np.exp(2 * g.standard_normal(200))
    G = O.fit_grid_nonuniform(W, dinv, 3, 0.0, 12)
    for i in range(4):
        np.testing.assert_allclose(G[i], plain_lloyd(list(W[i]), 8, 12), rtol=1e-12, atol=1e-14)
    assert np.allclose(O.sample_weights(dinv, 0.0), 1.0)


# ------------------------------------------------------------------ P6 ---- #
def test_p6_appendix_a_worked_example():
    rows = {}
    for line in open(os.path.join(GOLDEN, "appendix_a_grid.txt")):
        if line.startswith("#") or not line.strip():
            continue
        key, *vals = line.split()
        rows[key] = [float(v) for v in vals]
    mn, mx, bits = rows["range"]
    G = O.grid_init_uniform([mn], [mx], 1 << int(bits))[0]
    np.testing.assert_allclose(G, rows["grid"], atol=0.005)      # printed to 2 decimals
    w, nearest = rows["nearest"]
    code = O.assign_nu(np.array([[w]]), G[None])[0, 0]
    assert abs(G[code] - nearest) < 0.005
    assert abs(G[code] - 1 / 3) < 1e-15


def test_p6b_appendix_b_shrink_defaults():
    spec = {}
    for line in open(os.path.join(GOLDEN, "appendix_b_shrink.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, v = line.split()
        spec[k] = float(v)
    T = int(spec.pop("T"))
    g = rng(2)
    w = g.standard_normal((1, 16))
    dinv = np.ones(16)
    for bits, frac in spec.items():
        bits = int(bits)
        # the default t equals floor(frac*T): compare on a coarse T where the search is cheap
        Tc = 40
        a = O.fit_grid_affine(w, dinv, bits, 0.0, 0, T=Tc, t=None)
        b = O.fit_grid_affine(w, dinv, bits, 0.0, 0, T=Tc, t=int(np.floor(frac * Tc)))
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


# ------------------------------------------------------------------ P7 ---- #
def affine_bruteforce(w, s, bits, T, t):
    """Eq. 7 with explicit scalar loops (Python round() is round-half-to-even)."""
    K = (1 << bits) - 1
    mn, mx = min(w), max(w)
    R = mx - mn
    best = (float("inf"), None, None)
    for t_min in range(t + 1):
        for t_max in range(t + 1):
            lo = mn + t_min * R / T
            hi = mx - t_max * R / T
            S = (hi - lo) / K
            if S <= 0:
                continue
            Z = -round(lo / S)
            loss = 0.0
            for wi, si in zip(w, s):
                q = min(max(round(wi / S) + Z, 0), K)
                loss += si * ((q - Z) * S - wi) ** 2
            if loss < best[0]:
                best = (loss, S, Z)
    return best


def test_p7_affine_search():
    g = rng(41)
    r, c, group = 5, 32, 16
    W = g.standard_normal((r, c)) * 0.03
    W[0, 3] = 0.4          # an outlier the search should clip away from
    dinv = np.exp(g.standard_normal(c))
    s = O.sample_weights(dinv, 2.0)
    for bits in (2, 4):
        S, Z = O.fit_grid_affine(W, dinv, bits, 2.0, group, T=24, t=6)
        S0, Z0 = O.fit_grid_affine(W, dinv, bits, 2.0, group, T=24, t=0)
        Sm, Zm = O.minmax_affine_params(W, bits, group)
        np.testing.assert_allclose(S0, Sm, rtol=1e-15)
        assert np.array_equal(Z0, Zm)
        K = 1 << bits
        for i in range(r):
            for gi in range(c // group):
                w = W[i, gi * group:(gi + 1) * group]
                sg = s[gi * group:(gi + 1) * group]
                loss_b, S_b, Z_b = affine_bruteforce(list(w), list(sg), bits, 24, 6)
                np.testing.assert_allclose(S[i, gi], S_b, rtol=1e-14)
                assert Z[i, gi] == Z_b
                mine = float((sg * (O.quant_aff(w, S[i, gi], Z[i, gi], K) - w) ** 2).sum())
                mm = float((sg * (O.quant_aff(w, Sm[i, gi], Zm[i, gi], K) - w) ** 2).sum())
                np.testing.assert_allclose(mine, loss_b, rtol=1e-12)
                assert mine <= mm * (1 + 1e-12)
                # min-max formulas of Section 2.1
                assert np.isclose(Sm[i, gi], (w.max() - w.min()) / (K - 1))
                assert Zm[i, gi] == -round(w.min() / Sm[i, gi])
    # constant group: reproduced exactly
    Wc = np.full((1, 8), 0.25)
    S, Z = O.fit_grid_affine(Wc, np.ones(8), 4, 1.0, 0, T=8, t=2)
    np.testing.assert_allclose(O.quant_aff(Wc, S, Z, 16), Wc, atol=1e-15)


def test_quant_aff_round_half_even_and_clip():
    w = np.array([0.5, 1.5, 2.5, -0.5, 100.0, -100.0])
    assert list(O.affine_codes(w, 1.0, 3.0, 16)) == [3, 5, 5, 3, 15, 0]
    np.testing.assert_allclose(O.quant_aff(w, 1.0, 3.0, 16), [0, 2, 2, 0, 12, -3])


# ------------------------------------------------------------------ P8 ---- #
def test_p8_loss_ordering_on_ill_conditioned_layer():
    L = synth.make_layer("c1", 96, 128, 1024, seed=4)
    W = L.W.double().numpy()
    X = L.X.double().numpy()
    bits = 3
    lean = O.run_pass(W, X, bits=bits, p=4.0, block=32, n_iter=20)
    H, U = lean["H"], lean["U"]
    Sm, Zm = O.minmax_affine_params(W, bits)
    _, What_mm_loop, loss_mm_loop = O.quantize_layer(W, U, scale=Sm, zero=Zm, bits=bits, block=32)
    What_rtn = O.quant_aff(W, Sm, Zm, 1 << bits)
    p_lean = lean["proxy"]
    p_loop = O.proxy_loss(W, What_mm_loop, H)
    p_rtn = O.proxy_loss(W, What_rtn, H)
    assert p_lean < p_loop < p_rtn
    assert lean["loss"] < loss_mm_loop
    # affine loss-error-aware grid also beats min-max inside the same loop
    aff = O.run_pass(W, X, grid_type="affine", bits=bits, p=4.0, block=32, T=40, t=12)
    assert aff["proxy"] < p_loop


# ------------------------------------------------------------------ P9 ---- #
def test_p9_invariances():
    L = synth.make_layer("c1", 24, 48, 256, seed=8)
    W = L.W.double().numpy()
    X = L.X.double().numpy()
    a = O.run_pass(W, X, bits=3, block=16, n_iter=8)
    b = O.run_pass(W, 4.0 * X, bits=3, block=16, n_iter=8)          # exact power-of-two scaling
    assert np.array_equal(a["codes"], b["codes"])
    np.testing.assert_allclose(a["grid"], b["grid"], rtol=1e-9)
    np.testing.assert_allclose(b["proxy"], 16.0 * a["proxy"], rtol=1e-8)
    perm = rng(1).permutation(24)
    cperm = O.run_pass(W[perm], X, bits=3, block=16, n_iter=8)
    assert np.array_equal(cperm["codes"], a["codes"][perm])
    sub = O.run_pass(W[5:11], X, bits=3, block=16, n_iter=8)
    assert np.array_equal(sub["codes"], a["codes"][5:11])
    np.testing.assert_allclose(sub["grid"], a["grid"][5:11], rtol=0, atol=0)
    # tokens arriving in chunks give the same Hessian
    Hc = O.hessian([X[:, :100], X[:, 100:]])
    np.testing.assert_allclose(Hc, a["H"], rtol=1e-12, atol=1e-12 * np.abs(a["H"]).max())


# ------------------------------------------------------------------ P10 --- #
def test_p10_library_and_residuals():
    g = rng(17)
    c, n = 40, 300
    X = g.standard_normal((c, n)) * np.exp(g.standard_normal(c))[:, None]
    H = O.hessian(X)
    ref = np.zeros((c, c))
    for tkn in range(n):
        ref += 2.0 * np.outer(X[:, tkn], X[:, tkn])
    np.testing.assert_allclose(H, ref, rtol=1e-12, atol=1e-12 * np.abs(ref).max())
    U, dinv, H_d, _ = O.prepare_hinv(H, 0.01)
    np.testing.assert_allclose(H_d - H, 0.01 * np.trace(H) / c * np.eye(c), atol=1e-9 * np.trace(H))
    assert np.allclose(U, np.triu(U)) and (np.diag(U) > 0).all()
    np.testing.assert_allclose(U.T @ U @ H_d, np.eye(c), atol=1e-8)
    np.testing.assert_allclose(dinv, np.diag(np.linalg.inv(H_d)), rtol=1e-10)
    np.testing.assert_allclose(dinv, (U * U).sum(axis=0), rtol=1e-10)
    # second route to the same factor: H_d = R R^T with R upper, then U = R^-1
    J = np.eye(c)[::-1]
    R = J @ np.linalg.cholesky(J @ H_d @ J) @ J
    np.testing.assert_allclose(np.linalg.inv(R), U, rtol=1e-8, atol=1e-12)
    # Eq. 9: U[j, j:] is the j-th row of the downdated inverse over sqrt of its diagonal,
    # and the remaining inverse diagonals only decrease along the downdate
    Hinv = np.linalg.inv(H_d)
    for j in range(c):
        np.testing.assert_allclose(U[j, j:], Hinv[j, j:] / np.sqrt(Hinv[j, j]), rtol=1e-7, atol=1e-13)
        new = Hinv - np.outer(Hinv[:, j], Hinv[j, :]) / Hinv[j, j]
        assert (np.diag(new)[j + 1:] <= np.diag(Hinv)[j + 1:] * (1 + 1e-12)).all()
        Hinv = new


def test_dead_channel_convention():
    g = rng(6)
    c = 12
    X = g.standard_normal((c, 60))
    X[4] = 0.0
    W = g.standard_normal((3, c))
    U, dinv, H_d, Wf = O.prepare_hinv(O.hessian(X), 0.01, W)
    assert (Wf[:, 4] == 0).all() and np.array_equal(np.delete(Wf, 4, 1), np.delete(W, 4, 1))
    assert np.isfinite(U).all() and np.isfinite(dinv).all()


def test_dead_channel_is_the_layer_without_it():
    """What the convention (H_ii = 1, weight column zeroed) must achieve: a channel that never fires is decoupled from
    the others, so the live columns are quantised exactly as in the layer with that channel deleted.  The two
    layers' damping terms coincide when the live diagonal averages 1 (the dead entry counts as 1), which a rescaling
    of X arranges; then the factor and the inverse diagonal restricted to the live channels must be those of the
    smaller layer, the dead row and column of U must hold nothing but the diagonal entry 1 / sqrt(1 + damp), and the
    column loop must give the same codes and values on the live columns.  A mistake in the convention (dead entry
    left at 0, set to the mean, column not zeroed, coupling left in) fails one of these."""
    g = rng(16)
    c, dead, r = 40, 13, 6
    X = g.standard_normal((c, 200)) * np.exp(g.standard_normal((c, 1)))
    X[dead] = 0.0
    live = np.delete(np.arange(c), dead)
    X *= 1.0 / np.sqrt(np.mean(np.diag(O.hessian(X))[live]))           # mean of the live diagonal -> 1
    W = g.standard_normal((r, c)) * 0.05
    H = O.hessian(X)
    U, dinv, H_d, Wf = O.prepare_hinv(H, 0.01, W)
    Us, dinvs, H_ds, _ = O.prepare_hinv(H[np.ix_(live, live)], 0.01)
    damp = H_d[0, 0] - H[0, 0]
    np.testing.assert_allclose(damp, H_ds[0, 0] - H[live[0], live[0]], rtol=1e-12)
    np.testing.assert_allclose(U[np.ix_(live, live)], Us, rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(dinv[live], dinvs, rtol=1e-9)
    np.testing.assert_allclose(U[dead, dead], 1.0 / np.sqrt(1.0 + damp), rtol=1e-12)
    assert np.abs(np.delete(U[dead], dead)).max() < 1e-12 and np.abs(np.delete(U[:, dead], dead)).max() < 1e-12
    grid = O.grid_init_uniform(W.min(1), W.max(1), 8)
    codes, What, loss = O.quantize_layer(Wf, U, grid=grid, bits=3, block=16)
    codes_s, What_s, loss_s = O.quantize_layer(W[:, live], Us, grid=grid, bits=3, block=16)
    assert np.array_equal(codes[:, live], codes_s)
    np.testing.assert_allclose(What[:, live], What_s, rtol=0, atol=1e-12)
    # the dead column itself: the value 0 rounded to the grid, its loss error on top of the smaller layer's
    q0 = np.take_along_axis(grid, O.assign_nu(np.zeros((r, 1)), grid), 1)[:, 0]
    np.testing.assert_allclose(What[:, dead], q0)
    np.testing.assert_allclose(loss, loss_s + 0.5 * np.sum(q0 ** 2) * (1.0 + damp), rtol=1e-9)


def test_weighted_quantile_init_is_deterministic_and_sorted():
    g = rng(12)
    W = g.standard_normal((3, 64))
    dinv = np.exp(g.standard_normal(64))
    s = O.sample_weights(dinv, 1.0)
    G = O.grid_init_weighted_quantile(W, s, 8)
    assert (np.diff(G, axis=1) >= 0).all()
    # brute force for one row
    order = sorted(range(64), key=lambda j: W[0, j])
    acc_total = 0.0
    for j in order:
        acc_total += s[j]
    for k in range(8):
        acc = 0.0
        for j in order:
            acc += s[j]
            if acc >= (k + 0.5) / 8 * acc_total:
                assert G[0, k] == W[0, j]
                break
    G2 = O.fit_grid_nonuniform(W, dinv, 3, 1.0, 5, init="weighted_quantile")
    assert (np.diff(G2, axis=1) >= 0).all()


def test_sample_weights_definition():
    dinv = np.array([0.5, 2.0, 8.0])
    s = O.sample_weights(dinv, 2.0)
    raw = dinv ** -2.0
    np.testing.assert_allclose(s / s[0], raw / raw[0], rtol=1e-13)
    np.testing.assert_allclose(np.prod(s), 1.0, rtol=1e-12)


# ------------------------------------------------------------- packed codes ---- #
def test_pack_codes_by_hand_and_round_trip():
    """2-bit codes 1, 2, 3, 0, 3 -> bits 01 10 11 00 | 11 -> bytes 0b00111001, 0b00000011 (worked by hand);
    3-bit codes straddle bytes; packing then unpacking gives the codes back for every width."""
    assert O.pack_codes(np.array([[1, 2, 3, 0, 3]]), 2).tolist() == [[0b00111001, 0b00000011]]
    # 3-bit codes 5, 7, 1: bits (low first) 1,0,1, 1,1,1, 1,0,0 -> byte 0 = 0b01111101, byte 1 = 0
    assert O.pack_codes(np.array([[5, 7, 1]]), 3).tolist() == [[0b01111101, 0b00000000]]
    g = rng(11)
    for bits in (2, 3, 4):
        codes = g.integers(0, 1 << bits, size=(7, 37))
        packed = O.pack_codes(codes, bits)
        assert packed.shape == (7, (37 * bits + 7) // 8)
        assert np.array_equal(O.unpack_codes(packed, bits, 37), codes)


# ---------------------------------------------------- Algorithm 2 (LeanQuant-Exact) ---- #
def exact_by_submatrix_inverses(w, H, quant):
    """Algorithm 2 for one row without the Eq. 9 downdate: the inverse of the remaining problem is
    recomputed at every step as the inverse of the principal submatrix of H over the weights not yet
    quantised (what removing a row and a column from the inverse stands for), and Eq. 3 is applied
    with it."""
    w = w.copy()
    c = w.size
    todo = list(range(c))
    what = np.zeros(c)
    order = []
    eps = 0.0
    while todo:
        Hi = np.linalg.inv(H[np.ix_(todo, todo)])
        q = np.array([quant(w[j]) for j in todo])
        score = (q - w[todo]) ** 2 / (2.0 * np.diag(Hi))
        k = int(np.argmin(score))
        i = todo[k]
        eps += score[k]
        delta = -(w[i] - q[k]) / Hi[k, k] * Hi[:, k]
        for m, j in enumerate(todo):
            w[j] += delta[m]
        w[i] = q[k]
        what[i] = q[k]
        order.append(i)
        todo.pop(k)
    return what, eps, order


@pytest.mark.parametrize("c,seed", [(5, 0), (9, 1), (14, 2)])
def test_e1_exact_equals_submatrix_inverse_recomputation(c, seed):
    g = rng(100 + seed)
    r = 4
    W = g.standard_normal((r, c)) * 0.05
    H = spd(c, 50 + seed, 1e2)
    grid = np.sort(g.standard_normal((r, 4)) * 0.05, axis=1)
    codes, What, loss, orders = O.quantize_exact(W, np.linalg.inv(H), grid=grid, bits=2, return_order=True)
    total = 0.0
    for k in range(r):
        what, eps, order = exact_by_submatrix_inverses(W[k], H, lambda x: grid[k, np.argmin(np.abs(grid[k] - x))])
        assert order == list(orders[k])
        np.testing.assert_allclose(What[k], what, rtol=0, atol=1e-12)
        total += eps
    np.testing.assert_allclose(loss, total, rtol=1e-9)
    assert np.array_equal(np.take_along_axis(grid, codes, 1), What)


def test_e2_exact_sum_of_loss_errors_is_the_quadratic_loss():
    """Every step's loss error is the exact increase of 1/2 dw H dw^T under the constraint it adds, so the
    sum over the row is the quadratic loss of the final row, whatever the order."""
    g = rng(7)
    r, c = 6, 20
    W = g.standard_normal((r, c)) * 0.05
    H = spd(c, 3, 1e3)
    grid = np.sort(g.standard_normal((r, 8)) * 0.06, axis=1)
    for order in ("greedy", "natural"):
        codes, What, loss = O.quantize_exact(W, np.linalg.inv(H), grid=grid, bits=3, order=order)
        D = W - What
        np.testing.assert_allclose(loss, 0.5 * np.einsum("ri,ij,rj->", D, H, D), rtol=1e-9)


def test_e3_exact_with_identity_hessian_is_round_to_nearest():
    g = rng(8)
    r, c = 5, 33
    W = g.standard_normal((r, c))
    S = np.full((r, 1), 0.25)
    Z = np.full((r, 1), 8.0)
    codes, What, loss = O.quantize_exact(W, np.eye(c), scale=S, zero=Z, bits=4)
    ref = (np.clip(np.rint(W / 0.25) + 8, 0, 15) - 8) * 0.25
    assert np.array_equal(What, ref)
    np.testing.assert_allclose(loss, 0.5 * ((W - ref) ** 2).sum(), rtol=1e-12)


def test_e4_exact_in_natural_order_is_algorithm_1():
    """With the greedy choice replaced by i = 0, 1, 2, ... Algorithm 2 is OBQ in fixed order, which the
    column loop of Algorithm 1 computes through the Cholesky factor."""
    g = rng(9)
    r, c = 7, 40
    W = g.standard_normal((r, c)) * 0.05
    H = spd(c, 11, 1e2)
    U, dinv, H_d, _ = O.prepare_hinv(H, 0.01)
    grid = O.fit_grid_nonuniform(W, dinv, 3, 4.0, 10)
    c1, w1, l1 = O.quantize_layer(W, U, grid=grid, bits=3, block=16)
    c2, w2, l2 = O.quantize_exact(W, np.linalg.inv(H_d), grid=grid, bits=3, order="natural")
    assert np.array_equal(c1, c2)
    np.testing.assert_allclose(w1, w2, rtol=0, atol=1e-12)
    np.testing.assert_allclose(l1, l2, rtol=1e-9)


# ------------------------------------------ lazy per-group refit of the affine grid ---- #
def test_l1_lazy_refit_without_feedback_is_the_upfront_fit():
    """With H = I nothing is fed back, the columns never change, and fitting a group when the loop reaches it
    is fitting it beforehand."""
    g = rng(21)
    r, c = 6, 64
    W = g.standard_normal((r, c)) * 0.05
    dinv = np.exp(g.standard_normal(c))
    s = O.sample_weights(dinv, 4.0)
    S, Z = O.fit_grid_affine(W, dinv, 3, 4.0, 16, 30, 6)
    c0, w0, l0 = O.quantize_layer(W, np.eye(c), scale=S, zero=Z, bits=3, group=16, block=32)
    c1, w1, l1, S1, Z1 = O.quantize_layer(W, np.eye(c), bits=3, group=16, block=32, lazy=dict(s=s, T=30, t=6))
    assert np.array_equal(S, S1) and np.array_equal(Z, Z1)
    assert np.array_equal(c0, c1) and np.array_equal(w0, w1)


def test_l2_lazy_refit_sees_the_fed_back_columns():
    """First group: nothing has been fed back yet, so its (S, Z) are the up-front ones.  A later group: its (S, Z)
    are the Eq. 7 fit of the columns as the up-front loop with the lazy grids leaves them at that moment, which a
    second run with those grids given up front reproduces (same grids in, same trajectory)."""
    g = rng(22)
    r, c, grp = 5, 48, 16
    W = g.standard_normal((r, c)) * 0.05
    H = spd(c, 23, 1e2)
    U, dinv, H_d, _ = O.prepare_hinv(H, 0.01)
    s = O.sample_weights(dinv, 4.0)
    S0, Z0 = O.fit_grid_affine(W, dinv, 4, 4.0, grp, 20, 4)
    codes, What, loss, S, Z = O.quantize_layer(W, U, bits=4, group=grp, block=16, lazy=dict(s=s, T=20, t=4))
    assert np.array_equal(S[:, 0], S0[:, 0]) and np.array_equal(Z[:, 0], Z0[:, 0])
    assert not np.array_equal(S[:, 1:], S0[:, 1:])                      # feedback moved the later groups
    c2, w2, l2 = O.quantize_layer(W, U, scale=S, zero=Z, bits=4, group=grp, block=16)
    assert np.array_equal(codes, c2) and np.array_equal(What, w2)
    for k in range(1, c // grp):                                        # and each later pair is the fit of what stood there
        Sk, Zk = O.affine_search_group(_columns_at_group_start(W, U, S, Z, grp, k), s[k * grp:(k + 1) * grp], 16, 20, 4)
        np.testing.assert_allclose(Sk, S[:, k], rtol=1e-9)               # the unblocked loop sums in another order
        assert np.array_equal(Zk, Z[:, k])


def _columns_at_group_start(W, U, S, Z, grp, k):
    """Columns of group k after the columns of groups < k were quantised with the given grids (unblocked loop)."""
    Wc = W.copy()
    c = W.shape[1]
    for j in range(k * grp):
        q = O.quant_aff(Wc[:, j], S[:, j // grp], Z[:, j // grp], 16)
        e = (Wc[:, j] - q) / U[j, j]
        Wc[:, j:] -= np.outer(e, U[j, j:])
    return Wc[:, k * grp:(k + 1) * grp]


def test_p7b_candidates_with_one_grid_have_one_loss():
    """Eq. 7 on a fine partition: S depends on t_min + t_max only and Z = -rint(lo / S) is an integer, so many
    candidates give the same grid.  Their float64 losses agree to rounding noise, there are far fewer distinct
    grids than candidates, and the search's answer is a member of the class with the least loss."""
    g = rng(31)
    w = g.standard_normal(64) * 0.05
    s = np.exp(g.standard_normal(64))
    K, T, t = 16, 512, 102
    mn, mx = w.min(), w.max()
    classes = {}
    for t_min in range(t + 1):
        for t_max in range(t + 1):
            S, Z = O.affine_candidate(mn, mx, t_min, t_max, T, K)
            loss = (s * (O.quant_aff(w, S, Z, K) - w) ** 2).sum()
            classes.setdefault((t_min + t_max, Z), []).append(loss)
    assert len(classes) < (t + 1) ** 2 / 10
    for losses in classes.values():
        assert max(losses) <= min(losses) * (1 + 1e-10)
    So, Zo = O.affine_search_group(w[None, :], s, K, T, t)
    best_class = min(classes, key=lambda k: min(classes[k]))
    assert Zo[0] == best_class[1]
    R = mx - mn
    assert abs(So[0] / (R * (T - best_class[0]) / (T * (K - 1))) - 1) < 1e-12
