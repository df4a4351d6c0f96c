"""Calibration driver (Algorithm 1): the predictors of all layers, fitted one layer after another on
reconstructed inputs (Section 3.2).

Host loop only: every fit is one call of aquakv_fit_predictor, every reconstruction one call of
aquakv_encode_phase; nothing is computed here.  The first layer is compressed as is (the first
layer of Algorithm 2) and its reconstruction is what the second layer's predictors are fitted on, unless
`first_layer_exact` asks for the exact first-layer tensors that Algorithm 1 as printed carries forward.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional

import torch

from . import api


@dataclasses.dataclass
class Predictors:
    """Per layer (index 0 is None: the first layer has no predictor), in the layout the codec's entry
    points take: Wk [d, d], Wv [d, 2d] (columns 0..d-1 act on V_old, d..2d-1 on K_rec), optional fp32 biases."""
    Wk: List[Optional[torch.Tensor]]
    Wv: List[Optional[torch.Tensor]]
    bk: List[Optional[torch.Tensor]]
    bv: List[Optional[torch.Tensor]]


def calibrate(codec: api.Codec, K: List[torch.Tensor], V: List[torch.Tensor], rate: float = 1e-3,
              fit_bias: bool = False, first_layer_exact: bool = False, keep_reconstructions: bool = False):
    """Returns Predictors (and, with keep_reconstructions, the per-layer (K_rec, V_rec) the fits saw next)."""
    if first_layer_exact:
        K_old, V_old = K[0], V[0]
    else:
        _, _, K_old = codec.encode_phase(api.ROLE_KEY, K[0])
        _, _, V_old = codec.encode_phase(api.ROLE_VALUE, V[0])
    out = Predictors([None], [None], [None], [None])
    recs = [(K_old, V_old)]
    for l in range(1, len(K)):
        Wk, bk, _ = codec.fit_predictor(K[l], K_old, None, rate, fit_bias)
        _, _, K_rec = codec.encode_phase(api.ROLE_KEY, K[l], K_old, None, Wk, bk)
        Wv, bv, _ = codec.fit_predictor(V[l], V_old, K_rec, rate, fit_bias)
        _, _, V_rec = codec.encode_phase(api.ROLE_VALUE, V[l], V_old, K_rec, Wv, bv)
        out.Wk.append(Wk)
        out.Wv.append(Wv)
        out.bk.append(bk)
        out.bv.append(bv)
        K_old, V_old = K_rec, V_rec
        if keep_reconstructions:
            recs.append((K_rec, V_rec))
    return (out, recs) if keep_reconstructions else out
