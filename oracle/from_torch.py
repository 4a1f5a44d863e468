"""Glue that turns seeded torch tensors into the oracle's float64 numpy model.

TEST INFRASTRUCTURE ONLY (see clasp_oracle).  No arithmetic of the method
lives here: only dtype conversion (bf16/fp32 values -> float64, exactly).
"""
from __future__ import annotations

from typing import Callable, Dict, Optional

import numpy as np
import torch

from . import clasp_oracle as orc


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def model_from_tensors(cfg, layers, head: Optional[Dict[str, torch.Tensor]] = None,
                       resident: bool = True) -> orc.Model:
    """`layers` is a list of dicts of torch tensors, or a callable l -> dict.

    resident=True converts every layer once and keeps the float64 copies (small
    models); resident=False converts on each request so that only one layer's
    float64 weights are alive at a time (8B / 70B shapes).
    """
    get: Callable[[int], Dict[str, torch.Tensor]] = layers if callable(layers) else (lambda l: layers[l])
    if resident:
        conv = [{k: to_f64(v) for k, v in get(l).items()} for l in range(cfg.L)]
        layer_fn = lambda l: conv[l]
    else:
        layer_fn = lambda l: {k: to_f64(v) for k, v in get(l).items()}
    head64 = {k: to_f64(v) for k, v in head.items()} if head is not None else None
    return orc.Model(cfg, layer_fn, head64)


def model_from_datagen(cfg, resident: bool = True, device="cpu", seed=None) -> orc.Model:
    import datagen
    head = datagen.head_weights(cfg, device, seed)
    return model_from_tensors(cfg, lambda l: datagen.layer_weights(cfg, l, device, seed), head, resident)
