"""GPU-vs-oracle comparison rules.

Codes: bit-exact for every value pair whose oracle nearest-point margin exceeds 1e-4 (relative gap
between the best and second-best squared distance); pairs under the margin may differ.  Scales:
bit-exact unless the oracle's unrounded scale sits within 2e-6 (relative) of an fp16 rounding
boundary; such rows are reported and left out of the code check (their normalisation differs).
Reconstructions: |gpu - oracle| <= 2e-3 * max(|oracle|, row RMS), or the two are adjacent 16-bit
numbers (a one-ulp rounding flip of the stored format).
"""
import numpy as np
import torch

from paper_2501_19392_b200 import synth
from util import bits_to_f64, unpack_codes

MARGIN = 1e-4
REL_TOL = 2e-3


def gpu_bits(t: torch.Tensor) -> np.ndarray:
    return synth.to_bits(t)


def scale_rows_ok(gpu_scales: np.ndarray, ora_scales: np.ndarray, ora_exact: np.ndarray, tol: float = 2e-6):
    """Returns (rows whose scales all match, number of tolerated mismatches).  Fails on a mismatch
    that is not explained by an fp16 rounding boundary: the oracle's unrounded scale must lie within
    `tol` (relative) of the midpoint between the two fp16 values."""
    gs = gpu_scales.view(np.uint16) if gpu_scales.dtype != np.uint16 else gpu_scales
    neq = gs != ora_scales
    if neq.any():
        lo = np.minimum(gs, ora_scales)[neq].astype(np.uint16)
        hi = np.maximum(gs, ora_scales)[neq].astype(np.uint16)
        assert np.all(hi - lo == 1), "scale differs by more than one fp16 step"
        mid = 0.5 * (lo.view(np.float16).astype(np.float64) + hi.view(np.float16).astype(np.float64))
        rel = np.abs(ora_exact[neq] - mid) / mid
        assert np.all(rel < tol), "scale mismatch away from a rounding boundary: %g" % rel.max()
    return ~neq.any(axis=1), int(neq.sum())


# Share of value pairs whose oracle margin is NOT above 1e-4.  Measured with the oracle on 4000
# Gaussian rows per setting (d_kv 1024 / block 1024 and d_kv 512 / block 64, n = 16, 64, 256):
# 1.08e-4 ... 1.27e-4, i.e. 99.987-99.989 % of pairs are clear -- the rotated, normalised values are
# close to N(0, 1) whatever the input, so the rate is a property of the grid and the margin.  The
# tests allow this rate plus sampling noise; a "clear" pair must match bit for bit.
UNCLEAR_RATE = 1.4e-4


def max_unclear(n_pairs: int) -> float:
    """Largest number of pairs under the margin a sample of n_pairs may hold (mean + 4 sigma + 2)."""
    mean = UNCLEAR_RATE * n_pairs
    return mean + 4.0 * np.sqrt(mean) + 2.0


def min_same_rows(n_rows: int, d_kv: int) -> float:
    """Fewest rows (of n_rows) whose codes must ALL equal the oracle's: a row can differ only where
    one of its d_kv/2 pairs is under the margin, which happens to a share (d_kv/2) * UNCLEAR_RATE of
    the rows at most (7 % at d_kv = 1024); 3 sigma and one row of slack for small samples."""
    p = min(1.0, d_kv / 2 * UNCLEAR_RATE)
    return n_rows - (n_rows * p + 3.0 * np.sqrt(n_rows * p * (1.0 - p)) + 1.0)


def check_same_rows(same: np.ndarray, d_kv: int, n_excluded: int = 0):
    """`same`: rows whose scales and codes all equal the oracle's (the rows the reconstruction check
    runs on).  Fails if more rows dropped out than near-ties explain; n_excluded rows were left out
    for an fp16 scale-rounding boundary."""
    need = min_same_rows(same.size, d_kv) - n_excluded
    assert same.sum() >= need, "only %d of %d rows agree in every code (need %.1f)" % (same.sum(), same.size, need)


def check_codes(gpu_codes: np.ndarray, ora: dict, bits: int, rows_ok=None):
    gi, oi = unpack_codes(gpu_codes, bits), unpack_codes(ora["codes"], bits)
    margins = ora["margins"]
    clear = margins > MARGIN
    if rows_ok is not None:
        clear = clear & rows_ok[:, None]
        margins = margins[rows_ok]
    n_pairs = margins.size
    n_unclear = int((margins <= MARGIN).sum())
    assert n_unclear <= max_unclear(n_pairs), \
        "%d of %d pairs are under the margin (allowed %.1f)" % (n_unclear, n_pairs, max_unclear(n_pairs))
    bad = (gi != oi) & clear
    assert not bad.any(), "%d code mismatches above the margin (of %d)" % (bad.sum(), clear.sum())
    frac = 1.0 - n_unclear / max(1, n_pairs)
    return dict(clear_fraction=float(frac), near_tie_mismatches=int(((gi != oi) & ~clear).sum()))


def check_recon(gpu_hat_bits: np.ndarray, ora_exact: np.ndarray, ora_hat_bits: np.ndarray, dtype: int,
                rows_ok=None):
    """rows_ok: rows whose scales (and hence code meaning) agree; the others are skipped, since a
    scale one fp16 step away legitimately moves the whole group by up to 1e-3 of the residual."""
    if rows_ok is not None:
        gpu_hat_bits, ora_exact, ora_hat_bits = gpu_hat_bits[rows_ok], ora_exact[rows_ok], ora_hat_bits[rows_ok]
    g = bits_to_f64(gpu_hat_bits, dtype)
    rms = np.sqrt((ora_exact ** 2).mean(axis=1, keepdims=True))
    tol = REL_TOL * np.maximum(np.abs(ora_exact), rms)
    ok = np.abs(g - ora_exact) <= tol
    adjacent = np.abs(gpu_hat_bits.astype(np.int64) - ora_hat_bits.astype(np.int64)) <= 1
    assert np.all(ok | adjacent), "reconstruction off by more than 2e-3 / one ulp at %d elements" % (~(ok | adjacent)).sum()
    return dict(ulp_flips=int((gpu_hat_bits != ora_hat_bits).sum()), max_rel=float((np.abs(g - ora_exact) / np.maximum(np.abs(ora_exact), rms)).max()))
