"""CPU oracle of the predictor calibration (Algorithm 1; Section 3.2; the regularizer of Appendix A).

TEST INFRASTRUCTURE ONLY, like the rest of this package: plain numpy in double precision, one
statement per step of the paper's procedure, no blocking.  The CUDA library never imports it.

What it computes.  For one layer the key predictor is the linear map that minimises
||f(K_old) - K||^2 over the calibration tokens, the value predictor the one that minimises
||f([V_old ; K_rec]) - V||^2 (Algorithm 1: keys from the previous layer's keys, values from the
previous layer's values and the current keys), both fitted in closed form with the regularizer rate 1e-3
(Appendix A).  Layers are fitted one after another on RECONSTRUCTED inputs: K_rec = f_key(K_old) +
Q^-1(Q(K - f_key(K_old))) is produced by the codec oracle itself (Section 3.2: "Each subsequent set
of predictors is trained using reconstructed cache entries as inputs").

Readings (the paper is silent or at odds with itself here):
  * regularizer rate r: ridge term r * trace(X^T X) / n_in on the diagonal of the normal equations
    (relative to the mean feature energy, so that the fit does not depend on the scale of the cache);
  * the first layer: Algorithm 1 as printed carries the first layer's exact K, V forward, the text of
    Section 3.2 has the first layer compressed without a predictor and later layers trained on reconstructions;
    the text is followed (first_layer_exact=False) because that is what a decoder has (the first
    layer of Algorithm 2), and the printed listing can be had with first_layer_exact=True;
  * intercept: off by default (the benchmark configurations use no bias); with fit_bias the inputs and
    targets are centred, the map fitted on the centred data and b = mean(Y) - mean(X) W^T;
  * the fitted matrix is stored in the cache's 16-bit type, [d_kv][n_in] like a linear layer's weight,
    and it is that rounded matrix which produces the reconstructions the next fit sees.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import numpy as np

from . import BF16, F16, Oracle


# ---------------------------------------------------------------------------------------------
# 16-bit <-> double, whole arrays
# ---------------------------------------------------------------------------------------------
def bits_to_double(a: np.ndarray, dtype: int) -> np.ndarray:
    """Raw 16-bit patterns -> float64 (exact)."""
    a = np.ascontiguousarray(a, dtype=np.uint16)
    if dtype == F16:
        return a.view(np.float16).astype(np.float64)
    return (a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def double_to_bits(x: np.ndarray, dtype: int) -> np.ndarray:
    """float64 -> nearest 16-bit value, ties to even, as raw bit patterns (finite inputs)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    if dtype == F16:
        return x.astype(np.float16).view(np.uint16)      # numpy rounds double -> half once, to nearest even
    # bf16 keeps 7 of the double's 52 mantissa bits: round the other 45 to nearest, ties to even, on the
    # double's own bit pattern (a carry moves into the exponent as it should); the result is exactly
    # representable in float32, whose upper 16 bits are the bf16 pattern.  (Magnitudes in float32's
    # normal range or zero; the adapters and caches here are.)
    u = x.view(np.uint64)
    lsb = (u >> np.uint64(45)) & np.uint64(1)
    r = (u + np.uint64((1 << 44) - 1) + lsb) & ~np.uint64((1 << 45) - 1)
    y = r.view(np.float64).astype(np.float32)
    return (y.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


# ---------------------------------------------------------------------------------------------
# one predictor: closed-form ridge regression
# ---------------------------------------------------------------------------------------------
def ridge_fit(X: np.ndarray, Y: np.ndarray, rate: float = 1e-3,
              fit_bias: bool = False) -> Tuple[np.ndarray, Optional[np.ndarray]]:
    """argmin_W ||X W^T (+ b) - Y||^2 + rate * trace(X^T X)/n_in * ||W||^2 in double precision.

    X [T, n_in], Y [T, d_out] float64.  Returns W [d_out, n_in] (a linear layer's weight) and the
    intercept b [d_out] or None.  (Algorithm 1, its two least-squares fits; Appendix A for the rate.)
    """
    X = np.asarray(X, dtype=np.float64)
    Y = np.asarray(Y, dtype=np.float64)
    T, n_in = X.shape
    if fit_bias:
        mx, my = X.mean(axis=0), Y.mean(axis=0)
        X = X - mx
        Y = Y - my
    G = X.T @ X                                  # normal equations
    C = X.T @ Y
    ridge = rate * np.trace(G) / n_in
    Wt = np.linalg.solve(G + ridge * np.eye(n_in), C)       # [n_in, d_out]
    W = np.ascontiguousarray(Wt.T)
    b = (my - mx @ Wt) if fit_bias else None
    return W, b


def fit_predictor(inputs: Sequence[np.ndarray], target: np.ndarray, dtype: int, rate: float = 1e-3,
                  fit_bias: bool = False):
    """The fit on 16-bit tensors (raw bits): inputs are concatenated along the features.

    Returns dict(W=uint16 [d_out, n_in] rounded to the cache type, W_exact=float64, bias=float32 or None).
    """
    X = np.concatenate([bits_to_double(a, dtype) for a in inputs], axis=1)
    Y = bits_to_double(target, dtype)
    W, b = ridge_fit(X, Y, rate, fit_bias)
    return dict(W=double_to_bits(W, dtype), W_exact=W, bias=None if b is None else b.astype(np.float32))


# ---------------------------------------------------------------------------------------------
# Algorithm 1
# ---------------------------------------------------------------------------------------------
def calibrate(oracle: Oracle, K: List[np.ndarray], V: List[np.ndarray], rate: float = 1e-3,
              fit_bias: bool = False, first_layer_exact: bool = False):
    """Sequential calibration of all layers' predictors (Algorithm 1).

    K[l], V[l]: uint16 [T, d_kv] raw bits of the calibration tokens' keys / values of layer l.
    Returns a list with one dict per layer l >= 1: Wk, Wv (uint16), bk, bv (float32 or None), and
    Khat, Vhat (uint16) = the reconstructions that layer hands to the next.
    """
    dt = oracle.dtype
    if first_layer_exact:
        K_old, V_old = K[0], V[0]
    else:
        k0 = oracle.encode_phase(K[0], [], None, None, "k")          # Q alone (the first layer of Algorithm 2)
        v0 = oracle.encode_phase(V[0], [], None, None, "v")
        K_old, V_old = k0["hat"], v0["hat"]
    out = []
    for l in range(1, len(K)):
        fk = fit_predictor([K_old], K[l], dt, rate, fit_bias)                     # f_key
        k = oracle.encode_phase(K[l], [K_old], fk["W"], fk["bias"], "k")           # K_rec = f_key(K_old) + Q^-1(Q(K - f_key(K_old)))
        fv = fit_predictor([V_old, k["hat"]], V[l], dt, rate, fit_bias)            # f_value on [V_old ; K_rec]
        v = oracle.encode_phase(V[l], [V_old, k["hat"]], fv["W"], fv["bias"], "v")
        out.append(dict(Wk=fk["W"], Wv=fv["W"], bk=fk["bias"], bv=fv["bias"], Wk_exact=fk["W_exact"],
                        Wv_exact=fv["W_exact"], Khat=k["hat"], Vhat=v["hat"]))
        K_old, V_old = k["hat"], v["hat"]
    return out


def relative_error(X_bits: np.ndarray, Xhat_bits: np.ndarray, dtype: int) -> float:
    """||X - Xhat||^2 / ||X - mean_channel(X)||^2: one minus the explained variance with per-channel means
    (the measure of the paper's Figure 2, Appendix A)."""
    X = bits_to_double(X_bits, dtype)
    Xh = bits_to_double(Xhat_bits, dtype)
    return float(((X - Xh) ** 2).sum() / ((X - X.mean(axis=0)) ** 2).sum())
