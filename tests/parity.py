"""Helpers of the GPU parity tests: staged, teacher-forced comparison of the CUDA quantizer with the
CPU oracle, and the tolerances (from the task's acceptance rule):

  - integer partials: bit-exact;
  - codes: bit-exact except elements within 1e-6 (relative) of a decision boundary of the oracle
    (a BST midpoint, or a zero residue in the greedy step); such elements are counted and must stay
    below 1e-4 of all elements;
  - coefficients: 1e-4 relative, coefficient by coefficient: |d alpha_i| <= 1e-4 |alpha_i| for every coefficient
    that is not negligible in its row (|alpha_i| >= 1e-3 max_j |alpha_j|); a negligible one is held to
    1e-4 max_j |alpha_j| instead (relative to itself it carries no information: it is the difference of sums that
    cancel, as in a constant row, whose second coefficient is zero);
  - outputs: 1e-3 * (sum_i |alpha_i|) * (sum_j |beta_j|) * n.

The quantizer is discontinuous: one legitimately flipped element changes the next least-squares refit
by O(1/n), far above the coefficient tolerance.  So rows are compared stage by stage (T = 0, 1, .., T):
a row whose codes differ at an earlier stage is "diverged" from then on; diverged rows must be rare and
must reach the same objective value within 1e-3, the rest must meet the strict tolerances.
"""
import numpy as np

import oracle

CODE_REL = 1e-6
COEFF_REL = 1e-4
COEFF_NEGLIGIBLE = 1e-3
OUT_REL = 1e-3
MAX_FLIP_FRACTION = 1e-4
MAX_DIVERGED_ROWS = 5e-3


def unpack_rows(codes, n):
    """(rows, k, wpr) uint32 -> (rows, k, n) int8 of +-1 via numpy bit unpacking (no oracle code)."""
    codes = np.ascontiguousarray(codes).view(np.uint32)
    rows, k, wpr = codes.shape
    bits = np.unpackbits(codes.view(np.uint8).reshape(rows, k, wpr * 4), axis=2, bitorder="little")
    return np.where(bits[:, :, :n] > 0, 1, -1).astype(np.int8)


def pad_bits_zero(codes, n):
    codes = np.ascontiguousarray(codes).view(np.uint32)
    rows, k, wpr = codes.shape
    bits = np.unpackbits(codes.view(np.uint8).reshape(rows, k, wpr * 4), axis=2, bitorder="little")
    return not bits[:, :, n:].any()


def _boundary_distance(w, stage_T, k):
    """Per element: smallest relative distance to a decision boundary of the oracle's LAST stage."""
    w = np.asarray(w, dtype=np.float64)
    if stage_T == 0:
        alpha, _ = oracle.greedy(w, k)
        scale = np.abs(alpha).sum() + 1e-300
        r = w.copy()
        dist = np.full(w.shape, np.inf)
        for i in range(k):
            dist = np.minimum(dist, np.abs(r) / scale)
            r = r - alpha[i] * np.where(r >= 0, 1.0, -1.0)
        return dist
    alpha, b = oracle.quantize(w, k, stage_T - 1)
    alpha, _ = oracle.ls_refit(w, b, alpha_prev=alpha)
    v, _ = oracle.levels(alpha)
    thr = (v[:-1] + v[1:]) / 2
    scale = np.maximum(np.abs(thr), np.abs(alpha).sum() + 1e-300)
    return (np.abs(w[:, None] - thr[None, :]) / scale[None, :]).min(axis=1)


def coefficient_bound(o_coeffs):
    """Per-coefficient bound on |gpu - oracle| for one row (see the module docstring)."""
    o = np.abs(np.asarray(o_coeffs, dtype=np.float64))
    return COEFF_REL * np.where(o >= COEFF_NEGLIGIBLE * o.max(), o, o.max()) + 1e-30


def compare_quantizer(x, k, T, gpu_quantize):
    """x: (rows, n) float32.  gpu_quantize(x, k, T) -> (codes uint32 (rows,k,wpr), coeffs float32 (rows,k)).
    Returns a dict of counters; raises AssertionError on a violation."""
    x = np.asarray(x, dtype=np.float32)
    rows, n = x.shape
    x64 = x.astype(np.float64)
    diverged = np.zeros(rows, dtype=bool)
    flips_total = 0
    stats = {}
    for stage in range(T + 1):
        g_codes, g_coeffs = gpu_quantize(x, k, stage)
        assert pad_bits_zero(g_codes, n), "pad bits must be zero"
        gb = unpack_rows(g_codes, n)
        o_codes, o_coeffs = oracle.quantize_rows(x64, k, stage)
        ob = unpack_rows(o_codes, n)
        newly = np.zeros(rows, dtype=bool)
        for r in range(rows):
            if diverged[r]:
                # same quality: objective within 1e-3 of the oracle's
                og = oracle.objective(x64[r], g_coeffs[r].astype(np.float64), gb[r])
                oo = oracle.objective(x64[r], o_coeffs[r], ob[r])
                assert abs(og - oo) <= 1e-3 * max(oo, 1e-30) + 1e-12 * (x64[r] ** 2).sum(), \
                    "diverged row %d: objective %g vs %g" % (r, og, oo)
                continue
            scale = np.abs(o_coeffs[r]).max()
            err = np.abs(g_coeffs[r].astype(np.float64) - o_coeffs[r])
            assert np.all(err <= coefficient_bound(o_coeffs[r])), \
                "row %d stage %d: coefficients %s vs %s" % (r, stage, g_coeffs[r], o_coeffs[r])
            bad = np.any(gb[r] != ob[r], axis=0)
            if bad.any():
                # duplicate levels make several codes correct: compare reconstructions there
                rec_g = oracle.reconstruct(o_coeffs[r], gb[r])
                rec_o = oracle.reconstruct(o_coeffs[r], ob[r])
                bad &= np.abs(rec_g - rec_o) > 1e-12 * (scale + 1e-300)
            if bad.any():
                dist = _boundary_distance(x64[r], stage, k)
                assert np.all(dist[bad] <= CODE_REL), \
                    "row %d stage %d: %d flipped elements away from any boundary (min dist %g)" % (
                        r, stage, int((dist[bad] > CODE_REL).sum()), dist[bad].max())
                flips_total += int(bad.sum())
                newly[r] = True
        diverged |= newly
        stats["stage%d_diverged_rows" % stage] = int(diverged.sum())
    stats["flipped_elements"] = flips_total
    stats["rows"] = rows
    assert flips_total <= max(2, MAX_FLIP_FRACTION * rows * n * (T + 1)), stats
    assert diverged.sum() <= max(2, MAX_DIVERGED_ROWS * rows), stats
    return stats


def output_tolerance(Walpha, xbeta, n):
    """(batch, m) array: 1e-3 * sum|alpha_r| * sum|beta_b| * n."""
    a = np.abs(np.asarray(Walpha, dtype=np.float64)).sum(axis=1)
    b = np.abs(np.asarray(xbeta, dtype=np.float64)).sum(axis=1)
    return OUT_REL * b[:, None] * a[None, :] * n
