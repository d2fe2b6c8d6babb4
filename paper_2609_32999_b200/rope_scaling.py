"""Rotary frequencies for model variants, to be passed as `inv_freq` to a plan.

The library's kernels take the D/2 per-pair frequencies as data (tessera_model_cfg.inv_freq); this
module only computes such tables on the host.  It holds no rotation arithmetic."""
from __future__ import annotations

import math

import numpy as np


def default_inv_freq(head_dim: int, theta: float) -> np.ndarray:
    """Pair m turns by theta^(-2m/D) per position."""
    return theta ** (-2.0 * np.arange(head_dim // 2, dtype=np.float64) / head_dim)


def llama31_inv_freq(head_dim: int, theta: float = 500000.0, factor: float = 8.0, low_freq_factor: float = 1.0,
                     high_freq_factor: float = 4.0, original_max_position: int = 8192) -> np.ndarray:
    """Long-context frequency scaling of the Llama-3.1 family (the Llama-3.1-8B-Instruct the paper serves
    uses it): pairs whose wavelength is shorter than original_max_position / high_freq_factor keep their
    frequency, pairs whose wavelength exceeds original_max_position / low_freq_factor turn `factor` times
    slower, and the band in between is blended linearly in (original_max_position / wavelength)."""
    inv = default_inv_freq(head_dim, theta)
    low_wavelen = original_max_position / low_freq_factor
    high_wavelen = original_max_position / high_freq_factor
    out = np.empty_like(inv)
    for m, f in enumerate(inv):
        wavelen = 2.0 * math.pi / f
        if wavelen < high_wavelen:
            out[m] = f
        elif wavelen > low_wavelen:
            out[m] = f / factor
        else:
            smooth = (original_max_position / wavelen - low_freq_factor) / (high_freq_factor - low_freq_factor)
            out[m] = (1.0 - smooth) * f / factor + smooth * f
    return out
