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


def scale_rows_ok(gpu_scales: np.ndarray, ora_scales: np.ndarray, ora_exact: np.ndarray):
    """Returns (rows whose scales all match, number of tolerated mismatches).  Fails on a mismatch
    that is not explained by an fp16 rounding boundary."""
    gs = gpu_scales.view(np.uint16) if gpu_scales.dtype != np.uint16 else gpu_scales
    neq = gs != ora_scales
    if neq.any():
        lo = np.minimum(gs, ora_scales)[neq].astype(np.uint16)
        hi = np.maximum(gs, ora_scales)[neq].astype(np.uint16)
        assert np.all(hi - lo == 1), "scale differs by more than one fp16 step"
        mid = 0.5 * (lo.view(np.float16).astype(np.float64) + hi.view(np.float16).astype(np.float64))
        rel = np.abs(ora_exact[neq] - mid) / mid
        assert np.all(rel < 2e-6), "scale mismatch away from a rounding boundary: %g" % rel.max()
    return ~neq.any(axis=1), int(neq.sum())


MIN_CLEAR = {4: 0.9995, 6: 0.999, 8: 0.998}   # expected share of pairs clear of the margin, by code width


def check_codes(gpu_codes: np.ndarray, ora: dict, bits: int, rows_ok=None):
    gi, oi = unpack_codes(gpu_codes, bits), unpack_codes(ora["codes"], bits)
    clear = ora["margins"] > MARGIN
    if rows_ok is not None:
        clear = clear & rows_ok[:, None]
        frac = (ora["margins"][rows_ok] > MARGIN).mean() if rows_ok.any() else 1.0
    else:
        frac = clear.mean()
    if clear.size >= 20000:   # a statistical statement: only meaningful on enough pairs
        assert frac >= MIN_CLEAR[bits], "only %.5f of pairs are clear of the margin" % frac
    bad = (gi != oi) & clear
    assert not bad.any(), "%d code mismatches above the margin (of %d)" % (bad.sum(), clear.sum())
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
