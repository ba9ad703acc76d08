"""fp64 oracle of the recency-window attention diagnostics (numpy, written out plainly).

TEST INFRASTRUCTURE ONLY: imported by the test-suite; the CUDA library never loads this
module and this module never loads the CUDA library.

What is computed (Sec. 3.2 "Curse of Fixed Recent Window" and Sec. 7.1 of the Moment-KV
paper, which look at how the attention of the current step is spread over the most recently
decoded tokens): for one decode step with step id t, given for every cached decode token its
position id and the attention it received averaged over heads (Eq. 4),

  * the window is the set of cached decode tokens among the last W decoded ones, i.e. with
    t - W < position id <= t (the token decoded at this step included);
  * ``mass`` is the attention those tokens received together (a share of 1: the rest went to
    older decode tokens and to the prompt);
  * ``curve[j]`` is the share of ``mass`` held by the j+1 most attended tokens of the window
    (the paper's cumulative-attention curve; tokens attended uniformly would give
    (j+1)/count, the baseline the paper draws).

The paper gives the analysis as a figure, not as formulas; the definitions above are this
repository's reading of it.
"""
from __future__ import annotations

import numpy as np


def recency_window(abar, pos, t, window):
    """abar[i], pos[i]: Eq. 4 value and position id of cached decode token i (any order);
    t: step id of the current step; window: W >= 1.
    Returns (mass, count, curve) with curve of length count (fp64)."""
    abar = np.asarray(abar, dtype=np.float64)
    pos = np.asarray(pos, dtype=np.int64)
    assert abar.shape == pos.shape and abar.ndim == 1 and window >= 1
    inside = [i for i in range(len(pos)) if t - window < pos[i] <= t]
    vals = sorted((float(abar[i]) for i in inside), reverse=True)
    mass = 0.0
    for v in vals:
        mass += v
    curve = np.zeros(len(vals), dtype=np.float64)
    run = 0.0
    for j, v in enumerate(vals):
        run += v
        curve[j] = run / mass if mass > 0.0 else 0.0
    return mass, len(vals), curve


def uniform_baseline(count):
    """The curve of a window whose tokens are attended equally."""
    return (np.arange(count, dtype=np.float64) + 1.0) / max(count, 1)
