"""Host-side schedule of the method: which scale steps run densely, which run under the
fidelity-refinement approximation and which are skipped, and the rank r of every block group.

Sec. 4.1: the Infinity schedule keeps scales {1, ..., 32} dense and applies the approximation at
{40, 48, 64} with thresholds alpha = {0.96, 0, 0}; alpha = 0 skips the step.  App. A.1 tabulates,
for alpha = 0.96, the mean rank ratio of every block chunk at each late scale; a ratio is a
fraction of n = min(M, d) (Sec. 3.2, Eq. "low_rank_percent").
"""
from __future__ import annotations

import math
from typing import List, Sequence

DENSE, LOWRANK_RTR, SKIP = 0, 1, 2

INFINITY_SCALES = (1, 2, 4, 6, 8, 12, 16, 20, 24, 32, 40, 48, 64)
INFINITY_LATE_SCALES = (40, 48, 64)
INFINITY_ALPHA = (0.96, 0.0, 0.0)

# rows: block chunk 0..7, columns: scale 40, 48, 64 (alpha = 0.96)
RANK_RATIO_ALPHA_096 = (
    (0.016, 0.013, 0.008),
    (0.136, 0.117, 0.054),
    (0.210, 0.189, 0.083),
    (0.250, 0.222, 0.066),
    (0.256, 0.234, 0.056),
    (0.198, 0.183, 0.029),
    (0.157, 0.134, 0.038),
    (0.191, 0.163, 0.055),
)


def rank_from_keep_ratio(M: int, rho: float) -> int:
    return max(1, min(M, int(math.floor(rho * M + 0.5))))


def rank_from_table_ratio(M: int, width: int, ratio: float) -> int:
    n = min(M, width)
    return max(1, min(M, int(math.floor(ratio * n + 0.5))))


def infinity_group_ranks(scale_side: int, width: int = 2048, n_groups: int = 8) -> List[int]:
    """Rank per block group at a late Infinity scale (40, 48 or 64); groups other than 8 take the
    ratio of the chunk at the nearest relative depth."""
    col = INFINITY_LATE_SCALES.index(scale_side)
    M = scale_side * scale_side
    out = []
    for g in range(n_groups):
        chunk = min(7, int((g + 0.5) * 8 / n_groups))
        out.append(rank_from_table_ratio(M, width, RANK_RATIO_ALPHA_096[chunk][col]))
    return out


def infinity_stage_modes(paper_schedule: bool = True) -> List[int]:
    """Mode per scale step of the 13-step Infinity schedule.  paper_schedule: alpha = {0.96, 0, 0},
    i.e. scale 40 approximated and 48, 64 skipped; otherwise all three late scales approximated."""
    modes = []
    for s in INFINITY_SCALES:
        if s not in INFINITY_LATE_SCALES:
            modes.append(DENSE)
        elif not paper_schedule or INFINITY_ALPHA[INFINITY_LATE_SCALES.index(s)] > 0:
            modes.append(LOWRANK_RTR)
        else:
            modes.append(SKIP)
    return modes


def cache_rows(scales: Sequence[int]) -> List[int]:
    """KV-cache length after each scale of a square schedule."""
    acc, out = 0, []
    for s in scales:
        acc += s * s
        out.append(acc)
    return out
