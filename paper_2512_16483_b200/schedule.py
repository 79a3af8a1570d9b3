"""The method's schedule, as the C ABI exports it (include/fvar.h, "The method's schedule"): which scale
steps run densely, which run under the fidelity-refinement approximation and which are skipped
(Sec. 4.1), and the rank r of every block group (App. A.1; Sec. 3.2, Eq. "low_rank_percent").

Argument marshalling only: the table, the thresholds and the rounding live in the library
(csrc/schedule.cu).  These calls need no GPU.
"""
from __future__ import annotations

import ctypes as ct
from typing import List, Sequence, Tuple

from . import binding

DENSE, LOWRANK_RTR, SKIP = binding.DENSE, binding.LOWRANK_RTR, binding.SKIP
INFINITY_LATE_SCALES = (40, 48, 64)


def _check(status: int, what: str) -> None:
    if status != binding.OK:
        raise binding.FvarError(status, what)


def rank_from_keep_ratio(M: int, rho: float) -> int:
    return int(binding.load_library().fvar_rank_from_keep_ratio(int(M), float(rho)))


def rank_from_table_ratio(M: int, width: int, ratio: float) -> int:
    return int(binding.load_library().fvar_rank_from_table_ratio(int(M), int(width), float(ratio)))


def rank_ratio_table() -> Tuple[Tuple[float, ...], ...]:
    """App. A.1 (alpha = 0.96): rows = block chunk 0..7, columns = scale 40, 48, 64."""
    lib = binding.load_library()
    rows = []
    for chunk in range(8):
        row = []
        for side in INFINITY_LATE_SCALES:
            v = ct.c_double()
            _check(lib.fvar_infinity_rank_ratio(chunk, side, ct.byref(v)), "infinity_rank_ratio")
            row.append(v.value)
        rows.append(tuple(row))
    return tuple(rows)


def infinity_group_ranks(scale_side: int, width: int = 2048, n_groups: int = 8) -> List[int]:
    out = (ct.c_int * n_groups)()
    _check(binding.load_library().fvar_infinity_group_ranks(int(scale_side), int(width), int(n_groups), out),
           "infinity_group_ranks(%d)" % scale_side)
    return list(out)


def infinity_schedule(paper_schedule: bool = True) -> Tuple[List[int], List[int]]:
    """(side length, mode) per scale step of the 13-step Infinity schedule."""
    sides, modes, n = (ct.c_int * 16)(), (ct.c_int * 16)(), ct.c_int()
    _check(binding.load_library().fvar_infinity_schedule(int(bool(paper_schedule)), 16, sides, modes, ct.byref(n)),
           "infinity_schedule")
    return list(sides[:n.value]), list(modes[:n.value])


def infinity_stage_modes(paper_schedule: bool = True) -> List[int]:
    return infinity_schedule(paper_schedule)[1]


def cache_rows(scales: Sequence[int]) -> List[int]:
    """KV-cache length after each scale of a square schedule (prefix sums of side^2)."""
    acc, out = 0, []
    for s in scales:
        acc += s * s
        out.append(acc)
    return out
