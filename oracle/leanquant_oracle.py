"""Float64 CPU oracle for the LeanQuant per-linear-layer pass (Algorithm 1).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
pass computes; the CUDA library is checked against it.  It shares no code with
the CUDA path and must never be imported by it: only tests, the smoke check and
the benchmark's CPU-baseline leg call it.

Everything is numpy float64.  Inputs in a narrower type (bf16 / fp32) are widened
exactly by the caller.  Notation follows the paper: W is r x c, X is c x n,
H = 2 X X^T, K = 2^b grid points, B the block width of the column loop.

Where the paper leaves a detail open this file takes one reading and says so at
the spot; the design notes list all of them.

Pinned by tests/test_oracle_pins.py against: brute-force fixed-order OBQ with the
explicit inverse-Hessian downdate (column loop), the trace identity of the damped
proxy loss, H = I giving round-to-nearest, dynamic-programming optimal weighted
1-D k-means, an independently written plain Lloyd for p = 0, the worked 2-bit grid
example of Appendix A, a triple-loop affine search, textbook library inverses and
Cholesky factors, and scale / permutation / row-subset invariances; Algorithm 2
(quantize_exact) against principal-submatrix inverses recomputed at every step, the
identity sum of loss errors = 1/2 dw H dw^T, H = I, and Algorithm 1 in natural order.  The numbers
it produces on the benchmark configurations themselves are not printed anywhere in
the paper: for those, parity is "unpinned" beyond these properties.
"""
from __future__ import annotations

import numpy as np
import scipy.linalg as sla

F64 = np.float64


# --------------------------------------------------------------------------- #
# Stage 1 -- Algorithm 1 line 3, Section 2.2: H = 2 X X^T
# --------------------------------------------------------------------------- #
def hessian(X_chunks, alpha: float = 2.0, H: np.ndarray | None = None) -> np.ndarray:
    """H (+)= alpha * sum_chunks X_chunk X_chunk^T.  ``X_chunks`` is one c x n array
    or an iterable of c x n_i arrays (tokens may arrive in pieces; the sum is the same)."""
    if isinstance(X_chunks, np.ndarray):
        X_chunks = [X_chunks]
    for Xc in X_chunks:
        Xc = np.asarray(Xc, dtype=F64)
        G = alpha * (Xc @ Xc.T)
        H = G if H is None else H + G
    return H


# --------------------------------------------------------------------------- #
# Stage 2 -- Algorithm 1 line 4 and the "Cholesky and Dampening" paragraph
# --------------------------------------------------------------------------- #
def prepare_hinv(H: np.ndarray, damp_frac: float = 0.01, W: np.ndarray | None = None):
    """Dampen, invert, factor.

    Returns (U, dinv, H_d, W_fixed):
      H_d  = H + damp_frac * mean(diag H) * I           (1 % of the average diagonal)
      dinv = diag(H_d^-1)
      U    = the upper-triangular Cholesky factor of H_d^-1, H_d^-1 = U^T U, U_jj > 0.

    Reading: the factor is the *upper* one.  Only then do the rows "H^-1[j, j:]" used
    by lines 17-20 of Algorithm 1 reproduce Eq. 3 with the Eq. 9 downdate.
    Reading (the paper is silent; GPTQ's convention, on which the method builds): an
    input channel that never fires (H_ii = 0) gets H_ii = 1 and its weight column is
    zeroed before anything else.
    """
    H = np.array(H, dtype=F64, copy=True)
    c = H.shape[0]
    dead = np.diag(H) == 0.0
    if dead.any():
        H[dead, dead] = 1.0
    if W is not None:
        W = np.array(W, dtype=F64, copy=True)
        W[:, dead] = 0.0
    damp = damp_frac * np.mean(np.diag(H))
    H_d = H + damp * np.eye(c)
    Hinv = sla.inv(H_d)
    dinv = np.diag(Hinv).copy()
    U = sla.cholesky(Hinv, lower=False)
    return U, dinv, H_d, W


# --------------------------------------------------------------------------- #
# Stage 3 -- loss-error-aware grids
# --------------------------------------------------------------------------- #
def sample_weights(dinv: np.ndarray, p: float) -> np.ndarray:
    """s_j = (H^-1_jj)^(-p), Eq. 5 / Eq. 7, divided by its geometric mean.

    Reading: the common factor changes neither the arg-min of Eq. 5 / Eq. 7 nor any
    Lloyd centroid; it is taken out so that p = 4 cannot overflow a narrow float."""
    ld = np.log(np.asarray(dinv, dtype=F64))
    return np.exp(-p * (ld - ld.mean()))


def grid_init_uniform(w_min, w_max, K: int) -> np.ndarray:
    """Eq. 6: K evenly spaced points from min(w) to max(w), per row."""
    t = np.arange(K, dtype=F64)
    w_min = np.asarray(w_min, dtype=F64)[..., None]
    w_max = np.asarray(w_max, dtype=F64)[..., None]
    return w_min + (w_max - w_min) * t / (K - 1)


def grid_init_weighted_quantile(W: np.ndarray, s: np.ndarray, K: int) -> np.ndarray:
    """Alternative deterministic init: per row, sort ascending, accumulate sample
    weight, and take the value at the first position whose cumulative weight reaches
    (k + 1/2)/K of the total, k = 0..K-1."""
    W = np.asarray(W, dtype=F64)
    r, c = W.shape
    G = np.empty((r, K), dtype=F64)
    for i in range(r):
        order = np.argsort(W[i], kind="stable")
        cw = np.cumsum(s[order])
        for k in range(K):
            pos = int(np.searchsorted(cw, (k + 0.5) / K * cw[-1], side="left"))
            G[i, k] = W[i, order[min(pos, c - 1)]]
    return G


def assign_nu(w: np.ndarray, grid: np.ndarray) -> np.ndarray:
    """quant_nu's arg-min as an index.  ``grid`` is ascending along its last axis;
    the nearest point is found by counting the midpoints m_k = (g_k + g_{k+1})/2 that
    lie strictly below w, so a weight exactly on a midpoint takes the lower point.
    w: (..., c), grid: (..., K) -> codes (..., c) in 0..K-1."""
    mid = 0.5 * (grid[..., :-1] + grid[..., 1:])
    return (w[..., :, None] > mid[..., None, :]).sum(axis=-1)


def fit_grid_nonuniform(W, dinv, bits: int, p: float = 4.0, n_iter: int = 20,
                        init: str = "uniform", return_trace: bool = False):
    """Eq. 5 by Lloyd's algorithm, one independent problem per row.

    K = 2^bits centroids, sample weights ``sample_weights(dinv, p)`` shared by all rows,
    start from Eq. 6 (or the weighted-quantile alternative), then exactly ``n_iter``
    rounds of: assign every weight to its nearest centroid (``assign_nu``), move each
    centroid to the weighted mean of its members.  Readings: a fixed iteration count
    with no early stop; a centroid whose members carry zero total weight stays where
    it was.  Centroids remain ascending.
    """
    W = np.asarray(W, dtype=F64)
    r, c = W.shape
    K = 1 << bits
    s = sample_weights(dinv, p)
    if init == "uniform":
        G = grid_init_uniform(W.min(axis=1), W.max(axis=1), K)
    elif init == "weighted_quantile":
        G = grid_init_weighted_quantile(W, s, K)
    else:
        raise ValueError(init)
    trace = []
    for _ in range(n_iter):
        a = assign_nu(W, G)
        if return_trace:
            trace.append(float((s * (np.take_along_axis(G, a, 1) - W) ** 2).sum()))
        for k in range(K):
            member = a == k
            den = (member * s).sum(axis=1)
            num = (member * (s * W)).sum(axis=1)
            ok = den > 0.0
            G[ok, k] = num[ok] / den[ok]
    if return_trace:
        a = assign_nu(W, G)
        trace.append(float((s * (np.take_along_axis(G, a, 1) - W) ** 2).sum()))
        return G, trace
    return G


def affine_codes(w, S, Z, K: int):
    """w_int = clip(round(w / S) + Z, 0, K - 1) with round-half-to-even."""
    return np.clip(np.rint(w / S) + Z, 0, K - 1)


def quant_aff(w, S, Z, K: int):
    """quant_aff(w, S, Z) = (w_int - Z) * S."""
    return (affine_codes(w, S, Z, K) - Z) * S


def affine_candidate(mn: float, mx: float, t_min: int, t_max: int, T: int, K: int):
    """One element of the search space of Eq. 7: shrink the range by t_min*R/T from
    below and t_max*R/T from above; S = (hi - lo)/(K-1), Z = -round(lo/S).
    Reading for a constant group (R = 0): widen the range to include 0; if it is
    still empty use S = 1, Z = 0 (the constant is then reproduced exactly when it is
    an integer in range, and this only matters for all-equal groups)."""
    R = mx - mn
    if R == 0.0:
        lo, hi = min(mn, 0.0), max(mx, 0.0)
        if hi == lo:
            return 1.0, 0.0
        S = (hi - lo) / (K - 1)
        return S, -np.rint(lo / S)
    lo = mn + t_min * R / T
    hi = mx - t_max * R / T
    S = (hi - lo) / (K - 1)
    if not S > 0.0:
        return None
    return S, -np.rint(lo / S)


def affine_search_group(w, sg, K: int, T: int, t: int):
    """Eq. 7 for one group of columns, all rows at once: w is r x g, sg the g sample weights.
    Returns (S, Z), each of length r."""
    w = np.asarray(w, dtype=F64)
    r = w.shape[0]
    mn = w.min(axis=1)
    mx = w.max(axis=1)
    R = mx - mn
    bS = np.ones(r)
    bZ = np.zeros(r)
    flat = R == 0.0
    for i in np.nonzero(flat)[0]:
        bS[i], bZ[i] = affine_candidate(mn[i], mx[i], 0, 0, T, K)
    live = ~flat
    if live.any():
        wl, mnl, mxl, Rl = w[live], mn[live], mx[live], R[live]
        bl = np.full(wl.shape[0], np.inf)
        Sl = np.ones(wl.shape[0])
        Zl = np.zeros(wl.shape[0])
        for t_min in range(t + 1):
            lo = mnl + t_min * Rl / T
            for t_max in range(t + 1):
                hi = mxl - t_max * Rl / T
                S = (hi - lo) / (K - 1)
                valid = S > 0.0
                Ssafe = np.where(valid, S, 1.0)
                Z = -np.rint(lo / Ssafe)
                q = quant_aff(wl, Ssafe[:, None], Z[:, None], K)
                loss = (sg * (q - wl) ** 2).sum(axis=1)
                better = valid & (loss < bl)
                bl[better] = loss[better]
                Sl[better] = S[better]
                Zl[better] = Z[better]
        bS[live], bZ[live] = Sl, Zl
    return bS, bZ


def fit_grid_affine(W, dinv, bits: int, p: float = 4.0, group: int = 0,
                    T: int = 2048, t: int | None = None):
    """Eq. 7: enumerate (t_min, t_max) in {0..t}^2 per (row, group) and keep the pair
    (S, Z) with the least weighted squared error; ties keep the first candidate in
    t_min-major, t_max-minor order.  ``group`` = 0 means one group per row.
    Appendix B: t = 0.2T / 0.3T / 0.4T for 4 / 3 / 2 bits (floored to an integer).
    Returns scale (r x n_groups) and zero (r x n_groups, integer-valued float64)."""
    W = np.asarray(W, dtype=F64)
    r, c = W.shape
    K = 1 << bits
    if t is None:
        t = int(np.floor({4: 0.2, 3: 0.3, 2: 0.4}[bits] * T))
    g = c if group in (0, None) else group
    if c % g:
        raise ValueError("c must be a multiple of the group size")
    ng = c // g
    s = sample_weights(dinv, p)
    scale = np.empty((r, ng), dtype=F64)
    zero = np.empty((r, ng), dtype=F64)
    for gi in range(ng):
        scale[:, gi], zero[:, gi] = affine_search_group(W[:, gi * g:(gi + 1) * g], s[gi * g:(gi + 1) * g], K, T, t)
    return scale, zero


# --------------------------------------------------------------------------- #
# Stage 4 -- Algorithm 1 lines 10-21: block-wise column loop with error feedback
# --------------------------------------------------------------------------- #
def quantize_layer(W, U, *, grid=None, scale=None, zero=None, bits: int = 4,
                   group: int = 0, block: int = 128, return_pre: bool = False, lazy=None):
    """The iterative loss-error-based loop on a learned grid.

    For each block of ``block`` columns, for each column j in it: quantise W[:, j] for
    all rows (nearest point of the row's grid, or quant_aff with the parameters of
    group j // group), E[:, j-i] = (W[:, j] - What[:, j]) / U[j, j], and
    W[:, j:i+B] -= E[:, j-i] * U[j, j:i+B] inside the block; after the block
    W[:, i+B:] -= E @ U[i:i+B, i+B:].

    Returns codes (r x c, int64), W_hat (r x c) and loss = 1/2 * sum(E^2), the summed
    loss error of Eq. 3 with the damped inverse.  With ``return_pre`` a fourth array holds
    every weight as it stood at the moment it was quantised (for tie analysis in tests).

    ``lazy`` = dict(s=sample weights (c), T=, t=) selects the variant in which the (S, Z) of an affine group are
    fitted by Eq. 7 when the loop reaches the group's first column, on the group's columns as they stand then
    (all earlier errors fed back), instead of beforehand; ``scale`` / ``zero`` are then filled in and returned
    at the end of the tuple."""
    Wc = np.array(W, dtype=F64, copy=True)
    U = np.asarray(U, dtype=F64)
    r, c = Wc.shape
    K = 1 << bits
    codes = np.zeros((r, c), dtype=np.int64)
    What = np.zeros((r, c), dtype=F64)
    Wpre = np.zeros((r, c), dtype=F64) if return_pre else None
    loss = 0.0
    g = c if group in (0, None) else group
    if lazy is not None:
        scale = np.zeros((r, c // g), dtype=F64)
        zero = np.zeros((r, c // g), dtype=F64)
    for i in range(0, c, block):
        e_end = min(i + block, c)
        E = np.zeros((r, e_end - i), dtype=F64)
        for j in range(i, e_end):
            if lazy is not None and j % g == 0:
                if g > block and g % block:
                    raise ValueError("lazy refit: a group longer than a block must be made of whole blocks")
                if j + g > e_end and j != i:
                    raise ValueError("lazy refit: a group must start on a block boundary or lie inside one block")
                # columns beyond this block have not received this block's earlier errors yet: only allowed when the
                # group starts the block (then there are none)
                scale[:, j // g], zero[:, j // g] = affine_search_group(Wc[:, j:j + g], lazy["s"][j:j + g], K, lazy["T"], lazy["t"])
            w = Wc[:, j]
            if return_pre:
                Wpre[:, j] = w
            if grid is not None:
                a = assign_nu(w[:, None], grid)[:, 0]
                q = np.take_along_axis(grid, a[:, None], 1)[:, 0]
            else:
                S = scale[:, j // g]
                Z = zero[:, j // g]
                a = affine_codes(w, S, Z, K)
                q = (a - Z) * S
            codes[:, j] = a
            What[:, j] = q
            e = (w - q) / U[j, j]
            E[:, j - i] = e
            Wc[:, j:e_end] -= np.outer(e, U[j, j:e_end])
        loss += 0.5 * float((E * E).sum())
        if e_end < c:
            Wc[:, e_end:] -= E @ U[i:e_end, e_end:]
    extra = (scale, zero) if lazy is not None else ()
    if return_pre:
        return (codes, What, loss, Wpre) + extra
    return (codes, What, loss) + extra


# --------------------------------------------------------------------------- #
# Algorithm 2 (Appendix, "LeanQuant-Exact"): greedy order, full inverse-Hessian downdate per row
# --------------------------------------------------------------------------- #
def quantize_exact(W, Hinv, *, grid=None, scale=None, zero=None, bits: int = 4, group: int = 0,
                   order: str = "greedy", return_order: bool = False):
    """Algorithm 2, rows independent.  For a row w with its own copy of the inverse Hessian:
    repeat c times { among the weights not yet quantised pick i with the least
    (quant(w_i) - w_i)^2 / (2 Hinv_ii) (the loss error of Eq. 3; ties: lowest index);
    w_hat_i = quant(w_i);  w <- w - Hinv[:, i] / Hinv_ii * (w_i - w_hat_i)  (Eq. 3's update);
    Hinv <- Hinv - Hinv[:, i] Hinv[i, :] / Hinv_ii  (Eq. 9, removes i) }.

    The grid (non-uniform ``grid`` r x K, or ``scale`` / ``zero`` r x n_groups) is fitted beforehand on
    the original row, as lines 3-7 of the algorithm say.  ``Hinv`` is the c x c inverse the caller
    chose (Algorithm 2 writes (2 X X^T)^-1; the dampening of Algorithm 1 is the caller's decision).
    ``order="natural"`` replaces the greedy choice by i = 0, 1, 2, ... (OBQ in fixed order, which is
    what Algorithm 1 computes through the Cholesky factor); used by the pins.

    Returns codes (r x c int64), W_hat (r x c), loss = sum of the chosen loss errors, and with
    ``return_order`` the r x c array of indices in the order they were quantised."""
    W = np.asarray(W, dtype=F64)
    Hinv0 = np.asarray(Hinv, dtype=F64)
    r, c = W.shape
    K = 1 << bits
    g = c if group in (0, None) else group
    codes = np.zeros((r, c), dtype=np.int64)
    What = np.zeros((r, c), dtype=F64)
    orders = np.zeros((r, c), dtype=np.int64)
    loss = 0.0
    cols = np.arange(c)
    for row in range(r):
        w = W[row].copy()
        Hi = Hinv0.copy()
        todo = np.ones(c, dtype=bool)
        for step in range(c):
            if grid is not None:
                a = assign_nu(w[None, :], grid[row:row + 1])[0]
                q = grid[row][a]
            else:
                S = scale[row, cols // g]
                Z = zero[row, cols // g]
                a = affine_codes(w, S, Z, K)
                q = (a - Z) * S
            if order == "greedy":
                score = np.full(c, np.inf)
                score[todo] = (q[todo] - w[todo]) ** 2 / (2.0 * np.diag(Hi)[todo])
                i = int(np.argmin(score))                       # first minimum
            else:
                i = step
            dii = Hi[i, i]
            err = w[i] - q[i]
            loss += err * err / (2.0 * dii)
            codes[row, i] = a[i]
            What[row, i] = q[i]
            orders[row, step] = i
            col = Hi[:, i].copy()
            w -= col / dii * err
            w[i] = q[i]
            Hi -= np.outer(col, col) / dii
            Hi[i, :] = 0.0
            Hi[:, i] = 0.0
            todo[i] = False
    if return_order:
        return codes, What, loss, orders
    return codes, What, loss


def run_exact(W, X, *, grid_type="nonuniform", bits=4, p=4.0, damp=0.01, n_iter=20, init="uniform",
              group=0, T=2048, t=None, alpha=2.0):
    """Algorithm 2 end to end with the dampening of Algorithm 1 (damp = 0 gives (2 X X^T)^-1 to the letter)."""
    H = hessian(X, alpha)
    U, dinv, H_d, Wf = prepare_hinv(H, damp, W)
    Hinv = U.T @ U
    out = dict(H=H, U=U, dinv=dinv, H_d=H_d, Hinv=Hinv)
    if grid_type == "nonuniform":
        G = fit_grid_nonuniform(Wf, dinv, bits, p, n_iter, init)
        codes, What, loss = quantize_exact(Wf, Hinv, grid=G, bits=bits)
        out.update(grid=G)
    else:
        S, Z = fit_grid_affine(Wf, dinv, bits, p, group, T, t)
        codes, What, loss = quantize_exact(Wf, Hinv, scale=S, zero=Z, bits=bits, group=group)
        out.update(scale=S, zero=Z)
    out.update(codes=codes, W_hat=What, loss=loss, proxy=proxy_loss(Wf, What, H), proxy_d=proxy_loss(Wf, What, H_d))
    return out


def pack_codes(codes, bits: int) -> np.ndarray:
    """Storage format behind the paper's bit columns: every row's b-bit codes as one little-endian
    bit stream (code j in bits [j b, (j+1) b) of the row), padded with zero bits to whole bytes."""
    codes = np.asarray(codes, dtype=np.uint8)
    r, c = codes.shape
    bit_planes = (codes[:, :, None] >> np.arange(bits, dtype=np.uint8)) & 1       # least significant bit first
    stream = bit_planes.reshape(r, c * bits)
    return np.packbits(stream, axis=1, bitorder="little")


def unpack_codes(packed, bits: int, c: int) -> np.ndarray:
    """Inverse of pack_codes."""
    stream = np.unpackbits(np.asarray(packed, dtype=np.uint8), axis=1, bitorder="little")[:, :c * bits]
    planes = stream.reshape(stream.shape[0], c, bits).astype(np.int64)
    return (planes << np.arange(bits)).sum(axis=2)


RECORD_MAGIC = 0x3150514C      # "LQP1"


def _align16(n: int) -> int:
    return (n + 15) // 16 * 16


def record_bits_per_weight(bits: int, c: int, grid_type: str = "nonuniform", group: int = 0) -> float:
    """Storage cost per weight behind the bit columns of the paper's result tables: b-bit codes plus, per output
    row, a 2^b-entry fp16 table (non-uniform), or per group an fp16 scale and a 16-bit zero point (affine)."""
    if grid_type == "nonuniform":
        return bits + 16.0 * (1 << bits) / c
    g = c if group in (0, None) else group
    return bits + 32.0 / g


def pack_layer(codes, bits: int, *, grid=None, scale=None, zero=None, group: int = 0) -> np.ndarray:
    """One quantised layer as a byte record: 64-byte header (magic "LQP1", bits, grid type 0 / 1, group size as given,
    r, c, byte offsets of the codes, of the tables or scales, of the zero points, total bytes; int32 x 4 then int64 x 6,
    little endian), the packed codes (pack_codes), then the fp16 tables (r x 2^b) or the fp16 scales and int16 zero points
    (r x n_groups each); every section starts on a 16-byte boundary, padding bytes are zero."""
    codes = np.asarray(codes)
    r, c = codes.shape
    packed = pack_codes(codes, bits)
    row_bytes = packed.shape[1]
    affine = grid is None
    off_codes = 64
    off_table = off_codes + _align16(r * row_bytes)
    if affine:
        ng = np.asarray(scale).shape[1]
        off_zero = off_table + _align16(r * ng * 2)
        total = off_zero + _align16(r * ng * 2)
    else:
        off_zero = off_table + _align16(r * (1 << bits) * 2)
        total = off_zero
    rec = np.zeros(total, dtype=np.uint8)
    rec[:16] = np.array([RECORD_MAGIC, bits, 1 if affine else 0, group or 0], dtype="<u4").view(np.uint8)
    rec[16:64] = np.array([r, c, off_codes, off_table, off_zero, total], dtype="<i8").view(np.uint8)
    rec[off_codes:off_codes + r * row_bytes] = packed.reshape(-1)
    if affine:
        s16 = np.asarray(scale, dtype=np.float32).astype(np.float16)
        z16 = np.clip(np.asarray(zero), -32768, 32767).astype("<i2")
        rec[off_table:off_table + s16.size * 2] = s16.reshape(-1).view(np.uint8)
        rec[off_zero:off_zero + z16.size * 2] = z16.reshape(-1).view(np.uint8)
    else:
        t16 = np.asarray(grid, dtype=np.float32).astype(np.float16)
        rec[off_table:off_table + t16.size * 2] = t16.reshape(-1).view(np.uint8)
    return rec


def unpack_layer(rec: np.ndarray) -> np.ndarray:
    """The weights a record stands for, in float64: table[row][code], or (code - Z) * S with the stored fp16 / int16
    values (the product rounded to float32, as the format's consumers compute it)."""
    rec = np.asarray(rec, dtype=np.uint8)
    magic, bits, affine, group = (int(v) for v in rec[:16].view("<u4"))
    r, c, off_codes, off_table, off_zero, total = (int(v) for v in rec[16:64].view("<i8"))
    if magic != RECORD_MAGIC or total != rec.size:
        raise ValueError("not a layer record")
    row_bytes = (c * bits + 7) // 8
    codes = unpack_codes(rec[off_codes:off_codes + r * row_bytes].reshape(r, row_bytes), bits, c)
    if affine:
        g = c if group == 0 else group
        ng = c // g
        S = rec[off_table:off_table + r * ng * 2].view(np.float16).reshape(r, ng).astype(np.float32)
        Z = rec[off_zero:off_zero + r * ng * 2].view("<i2").reshape(r, ng).astype(np.float32)
        gi = np.arange(c) // g
        return ((codes.astype(np.float32) - Z[:, gi]) * S[:, gi]).astype(F64)
    table = rec[off_table:off_table + r * (1 << bits) * 2].view(np.float16).reshape(r, 1 << bits)
    return np.take_along_axis(table, codes, 1).astype(F64)


def run_stack(groups, **kw):
    """A stack of layers quantised in order, as a model-level driver calls the pass: `groups` is a list of
    (X, [W, ...]) -- every W of a group reads the same activations X, so the group shares stages 1-2 (one Hessian,
    one factor) and each W gets its own grid and column loop.  Returns one run_pass-style dict per layer, in order."""
    out = []
    for X, Ws in groups:
        for W in Ws:
            out.append(run_pass(W, X, **kw))
    return out


def proxy_loss(W, What, H) -> float:
    """tr((W - What) H (W - What)^T); with the undamped H = 2XX^T this is
    2 * ||W X - What X||_F^2, the layer objective of Eq. 1 up to the factor 2."""
    D = np.asarray(W, dtype=F64) - np.asarray(What, dtype=F64)
    return float(np.einsum("ij,ij->", D @ np.asarray(H, dtype=F64), D))


# --------------------------------------------------------------------------- #
# Baseline grids used for the loss comparison of ablation Q1
# --------------------------------------------------------------------------- #
def minmax_affine_params(W, bits: int, group: int = 0):
    """Plain min-max asymmetric affine grid of Section 2.1: S = (max - min)/(K-1),
    Z = -round(min / S), per (row, group)."""
    W = np.asarray(W, dtype=F64)
    r, c = W.shape
    K = 1 << bits
    g = c if group in (0, None) else group
    ng = c // g
    scale = np.empty((r, ng))
    zero = np.empty((r, ng))
    for gi in range(ng):
        w = W[:, gi * g:(gi + 1) * g]
        for i in range(r):
            scale[i, gi], zero[i, gi] = affine_candidate(w[i].min(), w[i].max(), 0, 0, 1, K)
    return scale, zero


def act_order(H) -> np.ndarray:
    """Activation ordering (appendix "Experiment Details", the option switched on for the GPTQ baseline): the columns in
    the order of decreasing diag(H); equal entries keep their index order."""
    return np.argsort(-np.diag(np.asarray(H, dtype=F64)), kind="stable")


def run_pass(W, X, *, grid_type="nonuniform", bits=4, p=4.0, block=128, damp=0.01,
             n_iter=20, init="uniform", group=0, T=2048, t=None, alpha=2.0, weight_src="inv_diag", lazy_refit=False,
             act_ordering=False):
    """Algorithm 1 end to end; returns a dict with every intermediate.
    ``weight_src``: "inv_diag" weights the grid objective by diag(H_d^-1)^-p as Eq. 5 / Eq. 7 say;
    "chol_diag" by diag(U)^-p, Algorithm 1 lines 6 and 8 read to the letter (the symbol H^-1 holds
    the Cholesky factor from line 4 on)."""
    H = hessian(X, alpha)
    if act_ordering:
        # the pass on the layer with its columns in the order of decreasing diag(H); codes and W_hat are put back
        # into the layer's own column order, everything else (U, dinv, scale / zero of groups) stays in pass order
        perm = act_order(H)
        Xp = np.asarray(X, dtype=F64)[perm]
        res = run_pass(np.asarray(W, dtype=F64)[:, perm], Xp, grid_type=grid_type, bits=bits, p=p, block=block, damp=damp,
                       n_iter=n_iter, init=init, group=group, T=T, t=t, alpha=alpha, weight_src=weight_src,
                       lazy_refit=lazy_refit)
        inv = np.empty_like(perm)
        inv[perm] = np.arange(perm.size)
        res["perm"] = perm
        res["codes"] = res["codes"][:, inv]
        res["W_hat"] = res["W_hat"][:, inv]
        res["H_perm"], res["H"] = res["H"], H
        return res
    U, dinv, H_d, Wf = prepare_hinv(H, damp, W)
    out = dict(H=H, U=U, dinv=dinv, H_d=H_d)
    if weight_src == "chol_diag":
        dinv = np.diag(U).copy()
    elif weight_src != "inv_diag":
        raise ValueError("weight_src")
    if grid_type == "nonuniform":
        G = fit_grid_nonuniform(Wf, dinv, bits, p, n_iter, init)
        codes, What, loss = quantize_layer(Wf, U, grid=G, bits=bits, block=block)
        out.update(grid=G)
    elif lazy_refit:
        if t is None:
            t = int(np.floor({4: 0.2, 3: 0.3, 2: 0.4}[bits] * T))
        codes, What, loss, S, Z = quantize_layer(Wf, U, bits=bits, group=group, block=block,
                                                 lazy=dict(s=sample_weights(dinv, p), T=T, t=t))
        out.update(scale=S, zero=Z)
    else:
        S, Z = fit_grid_affine(Wf, dinv, bits, p, group, T, t)
        codes, What, loss = quantize_layer(Wf, U, scale=S, zero=Z, bits=bits, group=group, block=block)
        out.update(scale=S, zero=Z)
    out.update(codes=codes, W_hat=What, loss=loss, proxy=proxy_loss(Wf, What, H),
               proxy_d=proxy_loss(Wf, What, H_d))
    return out
