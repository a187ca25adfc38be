#!/usr/bin/env python
"""Precision budget of the pass: how exact must each stage's arithmetic be?  CPU only.

The float64 oracle is re-run with one stage's arithmetic degraded in a controlled way and
the damage is measured where the tolerances are stated: max |dU| / max |U| of the factor,
fraction of codes that differ from the all-float64 pass, relative drift of the proxy loss
tr((W - W_hat) H (W - W_hat)^T).

Stage 2 (Algorithm 1 line 4) is emulated as the blocked sweep a GPU would run (128-wide
block columns, last to first: factor the diagonal block, form the panel, update the rest);
only the *update products* P Q (inner dimension 128) are degraded, everything else stays
float64.  Models of an update product:

  f64            exact (the sweep itself against the oracle's inverse-then-Cholesky route)
  f32all         the whole sweep in float32 (factor, panel and updates)
  f32ops         operands rounded to float32, product and accumulation exact
  bf16xS         operands split into S bf16 terms (each the bf16 rounding of what is left),
                 all term products with s + t <= S + 1 accumulated in float32 over the 128-deep
                 product (what a bf16 tensor-core product with a float32 accumulator gives),
                 the products added to the matrix in float64
  tf32xS         the same with 11-bit terms (TF32 operands)
  fix<k>         operands rounded to k bits below the largest entry of their row (left operand) or
                 column (right operand) -- fixed-point slices whose integer products a tensor core
                 accumulates exactly -- product and accumulation exact
  slice<S>       the tensor-core form of fix<8S>: operands as S slices of 8-bit integer digits below the row /
                 column exponent, the digit products of each level s + t <= S + 1 summed exactly, the levels
                 added in float32 (one rounding of the 128-deep product to 24 bits), then float64
  slice<S>t      the same with the leading level (s = t = 1) kept exact as a result of its own, the other
                 levels combined in float32, and the two added in float64
  <model>@ob     the sweep with the updates in two levels (outer blocks of 8 block columns = 1024 columns, see
                 sweep_two_level): only the deferred products, of inner dimension up to 1024, go through the model
  f32all+rK      float32 sweep followed by K steps of the first-order correction
                 U <- (I - triu(E) + diag(E)/2) U,  E = U H_d U^T - I evaluated in float64

Stage 4 (Algorithm 1 line 20) models: the lazy update E U[i:i+B, i+B:] with operands as S bf16
terms and a float32 accumulator per 128 columns of inner dimension, against float32 operands
with exact products.

Usage:  python tests/precision_budget.py [--quick]
Prints two markdown tables (the ones the design notes quote).  Calls only oracle/ and synth/.
"""
from __future__ import annotations

import argparse
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import synth  # noqa: E402
from oracle import leanquant_oracle as O  # noqa: E402

NB = 128


def to_bf16(x):
    """Round float64/float32 to bf16 (round to nearest even), returned as float64."""
    x32 = np.asarray(x, dtype=np.float32)
    u = x32.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


def to_tf32(x):
    x32 = np.asarray(x, dtype=np.float32)
    u = x32.view(np.uint32).astype(np.uint64)
    u = (u + 0xFFF + ((u >> 13) & 1)) & 0xFFFFE000
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


def split_terms(x, S, rnd):
    terms, rest = [], np.asarray(x, dtype=np.float64)
    for _ in range(S):
        t = rnd(rest)
        terms.append(t)
        rest = rest - t
    return terms


def prod_split(P, Q, S, rnd):
    """sum over s + t <= S + 1 of P_s Q_t, each product accumulated in float32."""
    Ps, Qs = split_terms(P, S, rnd), split_terms(Q, S, rnd)
    out = np.zeros((P.shape[0], Q.shape[1]))
    for s in range(S):
        for t in range(S - s):
            out += (Ps[s].astype(np.float32) @ Qs[t].astype(np.float32)).astype(np.float64)
    return out


def fix_round(x, k, axis):
    """k bits below the largest magnitude along `axis` (per row: axis=1, per column: axis=0)."""
    m = np.abs(x).max(axis=axis, keepdims=True)
    e = np.ceil(np.log2(np.where(m > 0, m, 1.0)))
    q = np.exp2(e - k)
    return np.rint(x / q) * q


def slices(x, S, axis):
    """x = 2^e * sum_s d_s 2^(-8 s) + remainder, s = 1..S, with integer digits |d_s| <= 128 and e the exponent
    of the largest magnitude along `axis`: the fixed-point slices a bf16 (or int8) tensor core multiplies exactly."""
    m = np.abs(x).max(axis=axis, keepdims=True)
    e = np.ceil(np.log2(np.where(m > 0, m, 1.0))) + 1.0          # |x| 2^-e <= 1/2
    rest = x * np.exp2(-e)
    out = []
    for s in range(1, S + 1):
        d = np.rint(rest * 2.0 ** (8 * s))
        out.append(d)
        rest = rest - d * 2.0 ** (-8 * s)
    return out, e


def prod_slices(P, Q, S, top_apart=False):
    """The product as the tensor-core path forms it: digit products of every level l = s + t <= S + 1 summed exactly
    (integers below 2^24), the levels added smallest first in float32, the result scaled by the row and column exponents.
    `top_apart`: the leading level (s = t = 1, exact) is kept as a result of its own and only the others are
    combined in float32; the two are added in float64."""
    dP, eP = slices(P, S, 1)
    dQ, eQ = slices(Q, S, 0)
    acc = np.zeros((P.shape[0], Q.shape[1]), dtype=np.float32)
    if top_apart:
        top = (dP[0] @ dQ[0]) * 2.0 ** -16
    for l in range(S + 1, 2 if top_apart else 1, -1):
        lvl = np.zeros((P.shape[0], Q.shape[1]))
        for s in range(1, S + 1):
            t = l - s
            if 1 <= t <= S:
                lvl += dP[s - 1] @ dQ[t - 1]
        # (the library sums a level in chunks of 128 of the inner dimension, each exact in float32, and adds the chunks
        # in float32; one rounding of the level's sum stands for that here)
        acc = acc + (lvl * 2.0 ** (-8 * l)).astype(np.float32)
    out = acc.astype(np.float64) + top if top_apart else acc.astype(np.float64)
    return out * np.exp2(eP) * np.exp2(eQ)


def make_product(model):
    if model == "f64":
        return lambda P, Q: P @ Q
    if model == "f32ops":
        return lambda P, Q: P.astype(np.float32).astype(np.float64) @ Q.astype(np.float32).astype(np.float64)
    if model.startswith("bf16x"):
        S = int(model[5:])
        return lambda P, Q: prod_split(P, Q, S, to_bf16)
    if model.startswith("tf32x"):
        S = int(model[5:])
        return lambda P, Q: prod_split(P, Q, S, to_tf32)
    if model.startswith("fix"):
        k = int(model[3:])
        return lambda P, Q: fix_round(P, k, 1) @ fix_round(Q, k, 0)
    if model.startswith("slice"):
        S = int(model[5])
        return lambda P, Q: prod_slices(P, Q, S, model.endswith("t"))        # exact while the inner dimension is at most 1024
    raise ValueError(model)


def sweep(H_d, product, dtype=np.float64):
    """U with H_d^-1 = U^T U by the blocked sweep: H_d = R R^T with R upper (last block column first),
    inverted in place by block Gauss-Jordan steps in the same order.  `product(P, Q)` computes the
    update products; `dtype` is the arithmetic of everything else."""
    c = H_d.shape[0]
    A = np.triu(H_d).astype(dtype)
    nblk = -(-c // NB)
    for k in range(nblk - 1, -1, -1):
        k0, k1 = k * NB, min((k + 1) * NB, c)
        D = A[k0:k1, k0:k1]
        D = np.triu(D) + np.triu(D, 1).T
        # D = R R^T with R upper  <=>  flip(D) = L L^T with L lower
        L = np.linalg.cholesky(D[::-1, ::-1].astype(dtype))
        R = L[::-1, ::-1]
        V = np.linalg.inv(R.astype(np.float64)).astype(dtype) if dtype == np.float64 else \
            np.linalg.solve(R, np.eye(R.shape[0], dtype=dtype)).astype(dtype)
        V = np.triu(V)
        P = (A[:k0, k0:k1] @ V.T).astype(dtype)                    # R[i][k], rows above the block
        right = (V @ A[k0:k1, k1:]).astype(dtype)                  # final rows of U right of the block
        A[k0:k1, k1:] = right
        A[k0:k1, k0:k1] = V
        if k0 > 0:
            Q = np.concatenate([P.T, np.zeros((k1 - k0, k1 - k0), dtype=dtype), right], axis=1)
            upd = product(P.astype(np.float64), Q.astype(np.float64)).astype(dtype)
            upd[:, k0:k1] = 0.0
            A[:k0, :] -= upd
            A[:k0, k0:k1] = -(P @ V).astype(dtype)
            A[:k0, :k0] = np.triu(A[:k0, :k0])
    return np.triu(A).astype(np.float64)


def sweep_two_level(H_d, product, obb=8):
    """The same sweep with the updates in two levels, as the library runs it: inside an outer block of `obb` block
    columns every step updates the outer block's rows and columns at once (exactly); all other tiles get the updates of
    the outer block's steps in one product of inner dimension 128 * obb when the outer block is complete, and only that
    product goes through `product`.  The operands of that product are whole rows of the outer block's panels, so
    a fixed-point model scales by the largest entry over 128 * obb columns, not 128."""
    c = H_d.shape[0]
    A = np.triu(H_d).astype(np.float64)
    nblk = -(-c // NB)
    for m in range(-(-nblk // obb) - 1, -1, -1):
        o_lo, o_hi = m * obb, min((m + 1) * obb, nblk) - 1
        r_lo, r_hi = o_lo * NB, min((o_hi + 1) * NB, c)
        Ps, Qs = [], []
        for k in range(o_hi, o_lo - 1, -1):
            k0, k1 = k * NB, min((k + 1) * NB, c)
            D = A[k0:k1, k0:k1]
            D = np.triu(D) + np.triu(D, 1).T
            R = np.linalg.cholesky(D[::-1, ::-1])[::-1, ::-1]
            V = np.triu(np.linalg.inv(R))
            P = A[:k0, k0:k1] @ V.T
            right = V @ A[k0:k1, k1:]
            A[k0:k1, k1:] = right
            A[k0:k1, k0:k1] = V
            if k0 > 0:
                Q = np.concatenate([P.T, np.zeros((k1 - k0, k1 - k0)), right], axis=1)
                upd = P @ Q
                A[r_lo:k0, :k0] -= upd[r_lo:k0, :k0]
                A[r_lo:k0, k1:] -= upd[r_lo:k0, k1:]
                A[:r_lo, r_lo:k0] -= upd[:r_lo, r_lo:k0]
                A[:r_lo, k1:r_hi] -= upd[:r_lo, k1:r_hi]
                A[:k0, k0:k1] = -(P @ V)
                A[:k0, :k0] = np.triu(A[:k0, :k0])
                Ps.append(P[:r_lo])
                Qs.append(np.concatenate([Q[:, :r_lo], Q[:, r_hi:]], axis=1))
        if o_lo > 0:
            upd = product(np.concatenate(Ps, axis=1), np.concatenate(Qs, axis=0))
            A[:r_lo, :r_lo] -= upd[:, :r_lo]
            A[:r_lo, r_hi:] -= upd[:, r_lo:]
            A[:r_lo, :r_lo] = np.triu(A[:r_lo, :r_lo])
    return np.triu(A)


def refine(U, H_d, steps):
    for _ in range(steps):
        E = U @ H_d @ U.T - np.eye(U.shape[0])
        C = -(np.triu(E, 1) + 0.5 * np.diag(np.diag(E)))
        U = np.triu(U + C @ U)
    return U


def stage2_models(quick):
    m = ["f64", "f32all", "f32all+r1", "f32ops", "bf16x3", "bf16x5", "tf32x3", "fix24", "fix32", "fix40", "fix48",
         "slice4", "slice3t", "slice4t", "slice5t", "slice4t@ob", "slice5t@ob"]
    return m[:2] + ["f32ops", "fix32", "slice4t", "slice4t@ob", "slice5t@ob"] if quick else m


def column_loop(W, U32, grid, bits, far_product):
    """Algorithm 1 lines 10-21 in float64 on the factor rounded to float32 (what the library stores), with the lazy
    update E U[i:i+B, i+B:] computed by `far_product` (None: exact).  Codes and W_hat."""
    Wc = np.array(W, dtype=np.float64, copy=True)
    r, c = Wc.shape
    codes = np.zeros((r, c), dtype=np.int64)
    What = np.zeros((r, c))
    for i in range(0, c, NB):
        e_end = min(i + NB, c)
        E = np.zeros((r, e_end - i))
        for j in range(i, e_end):
            w = Wc[:, j]
            a = O.assign_nu(w[:, None], grid)[:, 0]
            q = np.take_along_axis(grid, a[:, None], 1)[:, 0]
            codes[:, j], What[:, j] = a, q
            e = (w - q) / U32[j, j]
            E[:, j - i] = e
            Wc[:, j:e_end] -= np.outer(e, U32[j, j:e_end])
        if e_end < c:
            Ublk = U32[i:e_end, e_end:]
            Wc[:, e_end:] -= (E @ Ublk) if far_product is None else far_product(E, Ublk)
    return codes, What


def far_models():
    def split(S):
        return lambda E, Ub: prod_split(E.astype(np.float32).astype(np.float64), Ub, S, to_bf16)
    return {"f32 operands, exact product": lambda E, Ub: E.astype(np.float32).astype(np.float64) @ Ub,
            "bf16 x 1 (1 product)": split(1), "bf16 x 2 (3 products)": split(2), "bf16 x 3 (6 products)": split(3)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--quick", action="store_true")
    args = ap.parse_args()
    cases = [("c1", 64, 512, 8192), ("c2", 64, 1024, 16384), ("c2", 96, 2048, 32768), ("c3", 64, 2048, 16384)]
    if not args.quick:
        cases += [("c2", 96, 3000, 32768), ("c2", 96, 4096, 65536)]
    bits, p = 4, 4.0
    print("### Stage 2: the update products of the blocked sweep\n")
    print("| recipe, c | cond(H_d) | model | max abs dU / max abs U | codes differing | proxy drift |")
    print("|---|---:|---|---:|---:|---:|")
    for recipe, r, c, n in cases:
        L = synth.make_layer(recipe, r, c, n, seed=5)
        W = L.W.double().numpy()
        H = O.hessian(L.X.double().numpy())
        H = H.astype(np.float32).astype(np.float64)             # the library's H is float32
        U, dinv, H_d, _ = O.prepare_hinv(H, 0.01)
        ev = np.linalg.eigvalsh(H_d)
        cond = ev[-1] / ev[0]
        G = O.fit_grid_nonuniform(W, dinv, bits, p, 20)
        U32 = U.astype(np.float32).astype(np.float64)
        codes0, What0, _ = O.quantize_layer(W, U32, grid=G, bits=bits)
        proxy0 = O.proxy_loss(W, What0, H)
        for model in stage2_models(args.quick):
            t0 = time.time()
            if model.startswith("f32all"):
                Um = sweep(H_d, lambda P, Q: (P.astype(np.float32) @ Q.astype(np.float32)).astype(np.float64), np.float32)
                if "+r" in model:
                    Um = refine(Um, H_d, int(model[-1]))
            elif model.endswith("@ob"):
                Um = sweep_two_level(H_d, make_product(model[:-3]))
            else:
                Um = sweep(H_d, make_product(model))
            dU = np.abs(Um - U).max() / np.abs(U).max()
            Um32 = Um.astype(np.float32).astype(np.float64)
            codes, What, _ = O.quantize_layer(W, Um32, grid=G, bits=bits)
            mism = float((codes != codes0).mean())
            drift = abs(O.proxy_loss(W, What, H) / proxy0 - 1)
            print(f"| {recipe}, {c} | {cond:.1e} | {model} | {dU:.1e} | {100 * mism:.3f} % | {drift:.1e} |", flush=True)
            sys.stderr.write(f"  [{recipe} {c} {model}: {time.time() - t0:.1f} s]\n")
    print("\n### Stage 4: operands of the lazy update E U[i:i+B, i+B:]\n")
    print("| recipe, r x c, bits | model | codes differing | rows that diverge | proxy drift |")
    print("|---|---|---:|---:|---:|")
    cases4 = [("c1", 256, 512, 8192, 4), ("c2", 128, 1024, 16384, 4)] if args.quick else \
        [("c1", 512, 512, 8192, 4), ("c2", 512, 2048, 32768, 4), ("c2", 512, 2048, 32768, 2), ("c3", 512, 2048, 16384, 4),
         ("c2", 256, 4096, 65536, 3)]
    for recipe, r, c, n, b in cases4:
        L = synth.make_layer(recipe, r, c, n, seed=9)
        W = L.W.double().numpy()
        H = O.hessian(L.X.double().numpy()).astype(np.float32).astype(np.float64)
        U, dinv, _, _ = O.prepare_hinv(H, 0.01)
        G = O.fit_grid_nonuniform(W, dinv, b, p, 20)
        U32 = U.astype(np.float32).astype(np.float64)
        codes0, What0, _ = O.quantize_layer(W, U32, grid=G, bits=b)
        proxy0 = O.proxy_loss(W, What0, H)
        for name, fn in far_models().items():
            codes, What = column_loop(W, U32, G, b, fn)
            diff = codes != codes0
            drift = abs(O.proxy_loss(W, What, H) / proxy0 - 1)
            print(f"| {recipe}, {r} x {c}, {b} | {name} | {100 * diff.mean():.4f} % | {int(diff.any(axis=1).sum())} of {r} | {drift:.1e} |",
                  flush=True)


if __name__ == "__main__":
    main()
