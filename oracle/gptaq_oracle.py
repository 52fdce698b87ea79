"""Float64 CPU oracle for the GPTAQ per-layer solve.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain restatement of the paper's Algorithm 1 that the
CUDA path is checked against.  It shares no code with the CUDA path, is never
imported by the product package, and is only used by the tests, by the smoke
check and by the benchmark's CPU-baseline leg.

Notation follows the paper (Section 3.1): W is m x n (rows = output
channels), X is n x k (features x tokens), H = X X^T.  Activations arrive
token-major (``[tokens, n]``), i.e. as X^T.  The paper's lower factor L of
H^-1 = L L^T is kept as its transpose U = L^T (upper), so "row j of L^T" in
Algorithm 1 is ``U[j, :]``.

Library routines used as single steps: numpy matmul, LAPACK Cholesky and
triangular solves (through scipy).  Nothing is blocked, fused or reordered
beyond what the paper states, except that the column loop is evaluated in its
unblocked form (Eq. "divided update" applied to all later columns at once),
of which the lazy-batch form (Step 4) is a pure re-association; the blocked
form is also provided and tested to agree.

Readings of points the paper leaves open (each also listed in the design
notes): alpha scales P (alpha = 1 is Theorem 4.2, alpha = 0 is GPTQ); H and
dXX^T are divided by the token count before factoring (result-invariant
because the damping is relative); dead inputs (H_qq = 0) get H_qq = 1 and a
zeroed weight column; the second term uses the column's value just before it
is quantized; quant() is a min/max grid that always contains zero with
round-half-to-even; group grids are taken from the current (already updated)
weights at the first column of each group, per-channel grids from the
original row.

Pins (tests/test_oracle_*.py): brute-force sums for the statistics, Lemma 4.1
by direct inversion of trailing sub-blocks, Theorem 4.2 against the row-by-row
form and against the direct definition, every column step against a generic
equality-constrained least-squares solve, the GPTQ limit against an
elimination-form GPTQ, the RTN limit, block-size invariance, the quadratic-form
objective against the direct one, and the memory table of the appendix.
Parity of end results on the full-size configurations is unpinned beyond these
(the paper prints no worked numeric example).
"""
from __future__ import annotations

import dataclasses

import numpy as np
import scipy.linalg as sla

F64 = np.float64


# --------------------------------------------------------------------------
# Step 1 (Algorithm 1, the statistics step): H = X X^T, dXX^T = (X~ - X) X^T
# --------------------------------------------------------------------------
@dataclasses.dataclass
class Stats:
    n: int
    H: np.ndarray          # sum_t x_t x_t^T
    D: np.ndarray          # sum_t (x~_t - x_t) x_t^T   (row index: the delta)
    G: np.ndarray | None   # sum_t (x~_t - x_t)(x~_t - x_t)^T, evaluation only
    tokens: int = 0


def new_stats(n: int, with_gram_of_delta: bool = False) -> Stats:
    return Stats(n, np.zeros((n, n), F64), np.zeros((n, n), F64),
                 np.zeros((n, n), F64) if with_gram_of_delta else None, 0)


def accumulate(st: Stats, X_tm: np.ndarray, Xfp_tm: np.ndarray) -> None:
    """Add one token batch.  ``X_tm``, ``Xfp_tm``: ``[tokens, n]`` (X^T, X~^T)."""
    X = np.asarray(X_tm, dtype=F64)
    dX = np.asarray(Xfp_tm, dtype=F64) - X
    st.H += X.T @ X
    st.D += dX.T @ X
    if st.G is not None:
        st.G += dX.T @ dX
    st.tokens += X.shape[0]


# --------------------------------------------------------------------------
# Step 2 (Algorithm 1, the inverse-Cholesky step): L = Inverse_Cholesky(H + lambda_1 I)
# --------------------------------------------------------------------------
def damped_hessian(H_sum: np.ndarray, tokens: int, damp: float):
    """H/k with dead diagonal entries set to 1, plus damp * mean(diag) * I.
    Returns (H_d, dead) where ``dead`` marks inputs that never fired."""
    H = np.array(H_sum, dtype=F64) / float(max(tokens, 1))
    dead = np.diag(H) == 0.0
    idx = np.nonzero(dead)[0]
    H[idx, idx] = 1.0
    lam = damp * float(np.mean(np.diag(H)))
    H[np.diag_indices_from(H)] += lam
    return H, dead


def factor(H_sum: np.ndarray, tokens: int, damp: float):
    """Upper factor U of the damped inverse Hessian, H_d^-1 = U^T U = L L^T.

    The paper's route: Cholesky of H_d, inverse through two triangular
    solves, Cholesky of the inverse (lower L), U = L^T.
    Raises ``np.linalg.LinAlgError`` if H_d is not positive definite.
    """
    Hd, dead = damped_hessian(H_sum, tokens, damp)
    C = sla.cholesky(Hd, lower=True)
    Hinv = sla.cho_solve((C, True), np.eye(Hd.shape[0]))
    Hinv = 0.5 * (Hinv + Hinv.T)
    L = sla.cholesky(Hinv, lower=True)
    return np.ascontiguousarray(L.T), dead


# --------------------------------------------------------------------------
# Step 3 (Algorithm 1, the step that forms P; Theorem 4.2): P = ((dXX^T L) .* M_U) L^T
# --------------------------------------------------------------------------
def build_P(D_sum: np.ndarray, tokens: int, U: np.ndarray, alpha: float) -> np.ndarray:
    D = np.asarray(D_sum, dtype=F64) / float(max(tokens, 1))
    O = np.triu(D @ U.T, k=1)          # (dXX^T L) masked to strictly upper
    return alpha * (O @ U)


def build_P_rowwise(D_sum: np.ndarray, tokens: int, U: np.ndarray, alpha: float) -> np.ndarray:
    """The un-parallel form (Eq. "unparallel"): row q uses L[q+1:, q+1:]."""
    D = np.asarray(D_sum, dtype=F64) / float(max(tokens, 1))
    n = D.shape[0]
    L = U.T
    P = np.zeros((n, n), F64)
    for q in range(n - 1):
        Lq = L[q + 1:, q + 1:]
        P[q, q + 1:] = D[q, q + 1:] @ Lq @ Lq.T
    return alpha * P


def build_P_rows(D_rows: np.ndarray, rows, tokens: int, U: np.ndarray, alpha: float,
                 chunk: int = 2048) -> np.ndarray:
    """Rows ``rows`` of P by Theorem 4.2, ``P[q, :] = alpha * ((D[q, :] U^T) .* [a > q]) U``, from the
    matching rows ``D_rows`` of the raw sum dXX^T.  For layers whose n x n matrices are too large
    to hold several float64 copies of: ``U`` may be float32 and is widened a block of rows at a
    time."""
    D_rows = np.asarray(D_rows, dtype=F64) / float(max(tokens, 1))
    rows = np.asarray(rows)
    n = U.shape[0]
    O = np.zeros((len(rows), n), F64)
    for a0 in range(0, n, chunk):
        O[:, a0:a0 + chunk] = D_rows @ np.asarray(U[a0:a0 + chunk], dtype=F64).T
    O *= (np.arange(n)[None, :] > rows[:, None])
    P = np.zeros((len(rows), n), F64)
    for k0 in range(0, n, chunk):
        P += O[:, k0:k0 + chunk] @ np.asarray(U[k0:k0 + chunk], dtype=F64)
    return alpha * P


# --------------------------------------------------------------------------
# quant(.)  (Section 3.1; setup of Section 5): min/max grid, round half even
# --------------------------------------------------------------------------
def grid(w: np.ndarray, bits: int, sym: bool):
    """Per-row grid from ``w`` (``[rows, cols]``): returns (scale, zero)."""
    w = np.asarray(w, dtype=F64)
    if sym:
        a = np.max(np.abs(w), axis=1)
        a = np.where(a == 0.0, 1.0, a)
        scale = a / float(2 ** (bits - 1) - 1)
        zero = np.full_like(scale, float(2 ** (bits - 1)))
        return scale, zero
    maxq = float(2 ** bits - 1)
    lo = np.minimum(w.min(axis=1), 0.0)
    hi = np.maximum(w.max(axis=1), 0.0)
    flat = hi == lo
    scale = np.where(flat, 1.0, (hi - lo) / maxq)
    zero = np.where(flat, 0.0, np.rint(-lo / scale))
    return scale, zero


def qcode(w: np.ndarray, scale: np.ndarray, zero: np.ndarray, bits: int) -> np.ndarray:
    """Integer code in [0, 2^bits - 1] (symmetric grids store code = s + 2^(bits-1))."""
    maxq = float(2 ** bits - 1)
    return np.clip(np.rint(np.asarray(w, F64) / scale) + zero, 0.0, maxq)


def dequant(code: np.ndarray, scale: np.ndarray, zero: np.ndarray) -> np.ndarray:
    return scale * (code - zero)


def clip_candidates(w: np.ndarray, bits: int, sym: bool, steps: int, min_ratio: float):
    """All candidate grids of the clipping-range search (setup of Section 5; the paper says only that
    the range is chosen for the least squared error): candidate k shrinks the min/max range by
    p_k = 1 - k (1 - min_ratio) / steps.  Returns (scales, zeros, errors), each ``[steps, rows]``;
    errors are the sums of squared rounding errors of ``w`` on the candidate grid."""
    w = np.asarray(w, dtype=F64)
    scales, zeros, errs = [], [], []
    for k in range(steps):
        p = 1.0 - k * (1.0 - min_ratio) / steps
        if sym:
            a = p * np.max(np.abs(w), axis=1)
            a = np.where(a == 0.0, 1.0, a)
            s = a / float(2 ** (bits - 1) - 1)
            z = np.full_like(s, float(2 ** (bits - 1)))
        else:
            lo = p * np.minimum(w.min(axis=1), 0.0)
            hi = p * np.maximum(w.max(axis=1), 0.0)
            flat = hi == lo
            s = np.where(flat, 1.0, (hi - lo) / float(2 ** bits - 1))
            z = np.where(flat, 0.0, np.rint(-lo / s))
        q = dequant(qcode(w, s[:, None], z[:, None], bits), s[:, None], z[:, None])
        scales.append(s); zeros.append(z); errs.append(np.sum((q - w) ** 2, axis=1))
    return np.array(scales), np.array(zeros), np.array(errs)


def grid_search(w: np.ndarray, bits: int, sym: bool, steps: int, min_ratio: float):
    """Per-row grid with the least squared rounding error among the candidates; the widest on ties."""
    scales, zeros, errs = clip_candidates(w, bits, sym, steps, min_ratio)
    k = np.argmin(errs, axis=0)                      # first minimum = smallest k = widest range
    r = np.arange(scales.shape[1])
    return scales[k, r], zeros[k, r]


def _grid_fn(bits, sym, clip):
    if clip is None or clip[0] <= 0:
        return lambda blk: grid(blk, bits, sym)
    return lambda blk: grid_search(blk, bits, sym, clip[0], clip[1])


# --------------------------------------------------------------------------
# Steps 3-4 (Algorithm 1, the blocked loop): quantize and propagate
# --------------------------------------------------------------------------
@dataclasses.dataclass
class QuantResult:
    codes: np.ndarray      # [m, n] uint8
    scales: np.ndarray     # [m, n_groups] float64
    zeros: np.ndarray      # [m, n_groups] float64
    Wq: np.ndarray         # [m, n] dequantized weights
    pre: np.ndarray | None = None   # [m, n] pre-rounding w/scale (diagnostics)


def _ngroups(n: int, group: int) -> int:
    return 1 if group <= 0 else (n + group - 1) // group


def static_group_grids(W: np.ndarray, dead: np.ndarray | None, bits: int, group: int, sym: bool, clip=None):
    """Static groups (the companion of act_order in the setup of Section 5: per-group grids that survive a
    column permutation): one grid per output channel and per group of ``group`` consecutive columns of the
    ORIGINAL column order, taken from the original weights before the loop starts.  Returns
    (scales, zeros), each ``[m, ceil(n / group)]``."""
    W = np.array(W, dtype=F64)
    if dead is not None and dead.any():
        W[:, dead] = 0.0
    m, n = W.shape
    ng = _ngroups(n, group)
    make = _grid_fn(bits, sym, clip)
    scales = np.zeros((m, ng), F64)
    zeros = np.zeros((m, ng), F64)
    for g in range(ng):
        scales[:, g], zeros[:, g] = make(W[:, g * group:(g + 1) * group])
    return scales, zeros


def quantize(W: np.ndarray, U: np.ndarray, P: np.ndarray | None, dead: np.ndarray | None,
             bits: int, group: int, sym: bool, update: bool = True,
             keep_pre: bool = False, error_term: bool = True, clip=None, static=None) -> QuantResult:
    """Unblocked column loop (Eq. "divided update"), all rows at once.

    For column j: quantize the current column, e = (w - q) / U[j, j], then
    W[:, j+1:] += -e U[j, j+1:] + w P[j, j+1:], w being the value of column j
    just before it was quantized.  ``P = None`` drops the second term (GPTQ);
    ``error_term = False`` drops the first (the ablation's GPTAQ');
    ``update = False`` drops both (round to nearest).
    ``static = (scales, zeros, group_of_column)``: static groups -- the grids are given (see
    static_group_grids) and column j uses grid number ``group_of_column[j]``; nothing is re-taken from
    updated weights.
    """
    W = np.array(W, dtype=F64)
    m, n = W.shape
    if dead is not None and dead.any():
        W[:, dead] = 0.0
    ng = _ngroups(n, group)
    codes = np.zeros((m, n), np.uint8)
    scales = np.zeros((m, ng), F64)
    zeros = np.zeros((m, ng), F64)
    Wq = np.zeros((m, n), F64)
    pre = np.zeros((m, n), F64) if keep_pre else None
    make = _grid_fn(bits, sym, clip)      # ``clip = (steps, min_ratio)``: clipping-range search of every grid
    if static is not None:
        scales, zeros = np.array(static[0], F64), np.array(static[1], F64)
        gidx = np.asarray(static[2])
    elif group <= 0:
        s, z = make(W)
        scales[:, 0], zeros[:, 0] = s, z
    for j in range(n):
        if static is not None:
            s, z = scales[:, gidx[j]], zeros[:, gidx[j]]
        elif group > 0 and j % group == 0:
            s, z = make(W[:, j:j + group])
            scales[:, j // group], zeros[:, j // group] = s, z
        w = W[:, j].copy()
        c = qcode(w, s, z, bits)
        q = dequant(c, s, z)
        codes[:, j] = c.astype(np.uint8)
        Wq[:, j] = q
        if keep_pre:
            pre[:, j] = w / s
        if update and j + 1 < n:
            if error_term:
                e = (w - q) / U[j, j]
                W[:, j + 1:] -= np.outer(e, U[j, j + 1:])
            if P is not None:
                W[:, j + 1:] += np.outer(w, P[j, j + 1:])
    return QuantResult(codes, scales, zeros, Wq, pre)


def quantize_blocked(W: np.ndarray, U: np.ndarray, P: np.ndarray | None, dead,
                     bits: int, group: int, sym: bool, blocksize: int,
                     second_term_uses_quantized: bool = False) -> QuantResult:
    """Algorithm 1 as printed: in-block rank-1 updates, then the lazy-batch
    update of all later columns (Step 4).  ``second_term_uses_quantized``
    switches to the literal reading in which the block that multiplies
    P[Q, Q:] holds the already-quantized columns (sensitivity study only)."""
    W = np.array(W, dtype=F64)
    m, n = W.shape
    if dead is not None and dead.any():
        W[:, dead] = 0.0
    ng = _ngroups(n, group)
    codes = np.zeros((m, n), np.uint8)
    scales = np.zeros((m, ng), F64)
    zeros = np.zeros((m, ng), F64)
    Wq = np.zeros((m, n), F64)
    if group <= 0:
        s, z = grid(W, bits, sym)
        scales[:, 0], zeros[:, 0] = s, z
    for i in range(0, n, blocksize):
        i2 = min(i + blocksize, n)
        E = np.zeros((m, i2 - i), F64)
        Wpre = np.zeros((m, i2 - i), F64)
        for j in range(i, i2):
            if group > 0 and j % group == 0:
                s, z = grid(W[:, j:j + group], bits, sym)
                scales[:, j // group], zeros[:, j // group] = s, z
            w = W[:, j].copy()
            c = qcode(w, s, z, bits)
            q = dequant(c, s, z)
            codes[:, j] = c.astype(np.uint8)
            Wq[:, j] = q
            E[:, j - i] = (w - q) / U[j, j]
            Wpre[:, j - i] = q if second_term_uses_quantized else w
            W[:, j + 1:i2] -= np.outer(E[:, j - i], U[j, j + 1:i2])
            if P is not None:
                W[:, j + 1:i2] += np.outer(w, P[j, j + 1:i2])
        if i2 < n:
            W[:, i2:] -= E @ U[i:i2, i2:]
            if P is not None:
                W[:, i2:] += Wpre @ P[i:i2, i2:]
    return QuantResult(codes, scales, zeros, Wq)


# --------------------------------------------------------------------------
# Objective (Eq. "asym obj"): J = || W^ X - W X~ ||_F^2, summed over rows
# --------------------------------------------------------------------------
def objective(W: np.ndarray, Wq: np.ndarray, st: Stats) -> float:
    """J through the quadratic form  tr(dW H dW^T) - 2 tr(dW D^T W^T) + tr(W G W^T),
    dW = W^ - W, using the undamped float64 sums."""
    W = np.asarray(W, F64)
    dW = np.asarray(Wq, F64) - W
    t1 = float(np.sum((dW @ st.H) * dW))
    t2 = float(np.sum((dW @ st.D.T) * W))
    t3 = float(np.sum((W @ st.G) * W)) if st.G is not None else 0.0
    return t1 - 2.0 * t2 + t3


def objective_terms_chunked(W, Wq, H_upper: np.ndarray, D: np.ndarray, chunk: int = 2048) -> float:
    """The W^-dependent part of J, ``tr(dW H dW^T) - 2 tr(dW D^T W^T)``, for (a few rows of) W, from
    sums that may be float32 and of which H only needs a valid upper triangle: H and D are widened
    a block of rows at a time, H is completed by symmetry."""
    W = np.asarray(W, F64)
    dW = np.asarray(Wq, F64) - W
    n = W.shape[1]
    t1 = 0.0
    t2 = 0.0
    for a0 in range(0, n, chunk):
        a1 = min(a0 + chunk, n)
        Hc = np.triu(np.asarray(H_upper[a0:a1], dtype=F64), k=a0)      # rows a0..a1 of triu(H)
        left = dW[:, a0:a1] @ Hc                                      # sum_{a in chunk} dW[a] H[a, b], b >= a
        diag = np.einsum("ra,a,ra->", dW[:, a0:a1], np.diagonal(Hc, offset=a0).copy(), dW[:, a0:a1])
        t1 += 2.0 * float(np.sum(left * dW)) - float(diag)
        t2 += float(np.sum((dW @ np.asarray(D[a0:a1], dtype=F64).T) * W[:, a0:a1]))
    return t1 - 2.0 * t2


def objective_direct(W, Wq, X_tm, Xfp_tm) -> float:
    W = np.asarray(W, F64)
    r = np.asarray(X_tm, F64) @ np.asarray(Wq, F64).T - np.asarray(Xfp_tm, F64) @ W.T
    return float(np.sum(r * r))


# --------------------------------------------------------------------------
# Code comparison in "follow" mode (tie-aware): replay each row with the
# candidate's codes and grids as history, judge every code against the
# float64 pre-rounding value.
# --------------------------------------------------------------------------
@dataclasses.dataclass
class FollowReport:
    total: int
    mismatches: int        # candidate code != rint of the float64 value
    allowed: int           # ... of which within ``band`` of a rounding boundary
    disallowed: int
    worst_dist: float      # largest distance to a boundary among mismatches
    grid_rel_err: float    # max relative error of candidate scales
    zero_mismatch: int     # zero points that differ and are not near a tie


def follow(W: np.ndarray, U: np.ndarray, P: np.ndarray | None, dead,
           bits: int, group: int, sym: bool,
           cand_codes: np.ndarray, cand_scales: np.ndarray, cand_zeros: np.ndarray,
           band: float = 1e-4, error_term: bool = True, clip=None, static=None) -> FollowReport:
    """``static = (W_original, group_of_column[, dead_original])``: static groups -- the candidate's grids are
    judged once, against the grids of the original weights in their original column order with dead inputs
    counting as zero weights (``W`` is then the working copy in processing order), and column j uses the
    candidate's grid number ``group_of_column[j]``."""
    W = np.array(W, dtype=F64)
    m, n = W.shape
    if dead is not None and dead.any():
        W[:, dead] = 0.0
    maxq = float(2 ** bits - 1)
    cand_scales = np.asarray(cand_scales, F64).reshape(m, -1)
    cand_zeros = np.asarray(cand_zeros, F64).reshape(m, -1)
    mism = allowed = disallowed = zero_mis = 0
    worst = 0.0
    grid_err = 0.0

    def check_grid(block, g):
        nonlocal grid_err, zero_mis
        s_c, z_c = cand_scales[:, g], cand_zeros[:, g]
        if clip is not None and clip[0] > 0:
            # clipping-range search: the candidate's grid must be one of the candidate grids, and its
            # squared error (in float64) must equal the best one up to rounding: near-ties may fall
            # either way in float32.  A candidate whose zero point sits on a rounding tie before it is
            # rounded (-lo / scale within 10 * band of x.5: exact for weights with short mantissas and
            # symmetric extremes) exists in two versions, zero point rounded down or up; the searcher may
            # have met either one, so the bar is the best candidate in its worse version.
            S, Z, E = clip_candidates(block, bits, sym, clip[0], clip[1])
            Zalt, Ealt = Z, E
            if not sym:
                pk = 1.0 - np.arange(clip[0]) * (1.0 - clip[1]) / clip[0]
                t = -pk[:, None] * np.minimum(block.min(axis=1), 0.0)[None, :] / S
                tie = np.abs(t - np.floor(t) - 0.5) <= 10 * band
                Zalt = np.where(tie, 2.0 * np.floor(t) + 1.0 - Z, Z)
                Ealt = E.copy()
                for kk, rr in zip(*np.nonzero(tie)):
                    q = dequant(qcode(block[rr], S[kk, rr], Zalt[kk, rr], bits), S[kk, rr], Zalt[kk, rr])
                    Ealt[kk, rr] = np.sum((q - block[rr]) ** 2)
            rel = np.abs(S - s_c[None, :]) / S
            k = np.argmin(rel, axis=0)
            r = np.arange(S.shape[1])
            grid_err = max(grid_err, float(np.max(rel[k, r])))
            bar = np.maximum(E, Ealt).min(axis=0)
            mine = np.where(z_c == Z[k, r], E[k, r], np.where(z_c == Zalt[k, r], Ealt[k, r], np.inf))
            worse = mine > bar * (1.0 + 1e-5) + 1e-30
            zero_mis += int(np.sum(worse))
            return s_c, z_c
        s_o, z_o = grid(block, bits, sym)
        grid_err = max(grid_err, float(np.max(np.abs(s_c - s_o) / s_o)))
        if not sym:
            lo = np.minimum(block.min(axis=1), 0.0)
            t = -lo / s_c
            bad = (z_c != z_o) & (np.abs(t - np.floor(t) - 0.5) > 10 * band)
            zero_mis += int(bad.sum())
        return s_c, z_c

    if static is not None:
        W0 = np.array(static[0], dtype=F64)
        gidx = np.asarray(static[1])
        if len(static) > 2 and static[2] is not None and np.any(static[2]):
            W0[:, np.asarray(static[2], bool)] = 0.0
        for g in range(cand_scales.shape[1]):
            check_grid(W0[:, g * group:(g + 1) * group], g)
    elif group <= 0:
        s, z = check_grid(W, 0)
    for j in range(n):
        if static is not None:
            s, z = cand_scales[:, gidx[j]], cand_zeros[:, gidx[j]]
        elif group > 0 and j % group == 0:
            s, z = check_grid(W[:, j:j + group], j // group)
        w = W[:, j].copy()
        t = w / s
        want = np.clip(np.rint(t) + z, 0.0, maxq)
        got = cand_codes[:, j].astype(F64)
        bad = got != want
        if bad.any():
            frac = np.abs(t[bad] - np.floor(t[bad]) - 0.5)   # distance to x.5
            # the tie's other choice: of floor(t) and floor(t) + 1, the one that rint did not take
            other = np.clip(2.0 * np.floor(t[bad]) + 1.0 - np.rint(t[bad]) + z[bad], 0.0, maxq)
            near = (frac <= band) & (got[bad] == other)
            mism += int(bad.sum())
            allowed += int(near.sum())
            disallowed += int((~near).sum())
            worst = max(worst, float(frac.max()))
        q = dequant(got, s, z)
        if j + 1 < n:
            if error_term:
                e = (w - q) / U[j, j]
                W[:, j + 1:] -= np.outer(e, U[j, j + 1:])
            if P is not None:
                W[:, j + 1:] += np.outer(w, P[j, j + 1:])
    return FollowReport(m * n, mism, allowed, disallowed, worst, grid_err, zero_mis)


# --------------------------------------------------------------------------
# Whole layer, and the working-set table of the appendix (matrix dimensions)
# --------------------------------------------------------------------------
def solve_layer(W, batches, damp, alpha, bits, group, sym, with_gram_of_delta=True):
    """Algorithm 1 end to end.  ``batches`` yields (X_tm, Xfp_tm) pairs."""
    W = np.asarray(W, F64)
    st = new_stats(W.shape[1], with_gram_of_delta)
    for X, Xfp in batches:
        accumulate(st, X, Xfp)
    U, dead = factor(st.H, st.tokens, damp)
    P = build_P(st.D, st.tokens, U, alpha)
    res = quantize(W, U, P, dead, bits, group, sym)
    return st, U, P, dead, res


# --------------------------------------------------------------------------
# act_order (Section 5, setup): columns sorted by the Hessian diagonal
# --------------------------------------------------------------------------
def act_order_perm(H_sum: np.ndarray, tokens: int) -> np.ndarray:
    """Sorted position -> column: decreasing diag(H / k), dead inputs counting as 1 (they are set
    to 1 before sorting), ties keeping the lower index first."""
    d = np.diag(np.asarray(H_sum, F64)) / float(max(tokens, 1))
    d = np.where(d == 0.0, 1.0, d)
    return np.argsort(-d, kind="stable")


def solve_act_order(W, H_sum, D_sum, tokens, damp, alpha, bits, group, sym, perm=None, static_groups=False):
    """Algorithm 1 on the layer with its inputs relabelled by ``perm`` (default: act_order_perm):
    H and dXX^T are permuted on both sides, W on its columns; codes and dequantized weights are
    returned in the original column order.  Group grids belong to groups of consecutive columns of
    the sorted order, or, with ``static_groups``, to groups of consecutive columns of the ORIGINAL order
    (taken from the original weights; the column at sorted position j uses group ``perm[j] // group``).
    Returns (U, P, dead, result, perm), U / P / dead in sorted order."""
    W = np.asarray(W, F64)
    if perm is None:
        perm = act_order_perm(H_sum, tokens)
    perm = np.asarray(perm)
    Hp = np.asarray(H_sum, F64)[np.ix_(perm, perm)]
    Dp = np.asarray(D_sum, F64)[np.ix_(perm, perm)]
    U, dead = factor(Hp, tokens, damp)
    P = build_P(Dp, tokens, U, alpha)
    static = None
    if static_groups and group > 0:
        dead0 = np.zeros(W.shape[1], bool)
        dead0[perm] = dead
        sc, zr = static_group_grids(W, dead0, bits, group, sym)
        static = (sc, zr, perm // group)
    res = quantize(W[:, perm], U, P, dead, bits, group, sym, static=static)
    codes = np.empty_like(res.codes)
    Wq = np.empty_like(res.Wq)
    codes[:, perm] = res.codes
    Wq[:, perm] = res.Wq
    return U, P, dead, QuantResult(codes, res.scales, res.zeros, Wq), perm


def working_set_elements(m: int, n: int, blocksize: int, asymmetric: bool) -> dict:
    """Matrix dimensions held during the loop (appendix memory table):
    W, H (then L), Q, E for GPTQ; GPTAQ adds dXX^T (then P).  The table lists
    E at m x n."""
    d = {"W": m * n, "H": n * n, "Q": m * n, "E": m * n}
    if asymmetric:
        d["dXXT"] = n * n
    return d
