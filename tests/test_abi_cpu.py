"""CPU-side checks of the boundary: the library builds, loads and exports every symbol the public
header declares; the schedule the library exports agrees with the printed table.  No compute calls."""
import os
import re

import numpy as np

import synth_inputs as si
from paper_2512_16483_b200 import build as fbuild
from paper_2512_16483_b200 import schedule

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "fvar.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fvar_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    fbuild.build()
    from paper_2512_16483_b200 import binding
    lib = binding.load_library()
    names = _declared()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTED) == names


def test_workspace_bytes_and_bad_shapes_without_gpu():
    import ctypes as ct
    from paper_2512_16483_b200 import binding
    lib = binding.load_library()
    hw = (ct.c_int * 4)(2, 2, 3, 3)
    cfg = binding._Cfg(2, 1, 128, 2, 64, 256, 2, ct.cast(hw, ct.POINTER(ct.c_int)), 2, 0, 0, 0, 1e-6)
    n = lib.fvar_workspace_bytes(ct.byref(cfg))
    assert n > 0 and n % 1024 == 0
    cfg.head_dim = 32                                    # unsupported head size
    assert lib.fvar_workspace_bytes(ct.byref(cfg)) == 0
    cfg.head_dim, cfg.blocks_per_group = 64, 3           # 2 blocks do not split into groups of 3
    assert lib.fvar_workspace_bytes(ct.byref(cfg)) == 0
    ctx = ct.c_void_p(None)
    w = binding._Weights()
    st = lib.fvar_init(ct.byref(w), ct.byref(cfg), None, 0, None, ct.byref(ctx))
    assert st == binding.EINVAL and not ctx.value
    assert b"shape" in lib.fvar_last_error(None)
    assert lib.fvar_kv_append(None, 0) == binding.EINVAL


def test_schedule_matches_printed_table():
    rows = []
    with open(os.path.join(ROOT, "tests", "golden", "rank_ratio_alpha096.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                rows.append(tuple(float(v) for v in line.split()))
    assert tuple(rows) == schedule.rank_ratio_table()
    assert schedule.infinity_group_ranks(40) == [26, 218, 336, 400, 410, 317, 251, 306]
    assert schedule.infinity_group_ranks(64) == [16, 111, 170, 135, 115, 59, 78, 113]
    assert schedule.infinity_stage_modes(True) == [0] * 10 + [1, 2, 2]
    assert schedule.infinity_stage_modes(False) == [0] * 10 + [1, 1, 1]
    assert schedule.cache_rows(si.INFINITY_SCALES)[-1] == 10521 and schedule.cache_rows(si.VAR_SCALES)[-1] == 680
    assert schedule.rank_from_keep_ratio(169, 0.5) == 85 and schedule.rank_from_keep_ratio(100, 0.001) == 1
    assert schedule.infinity_schedule(True)[0] == list(si.INFINITY_SCALES)
    assert schedule.rank_from_table_ratio(1600, 2048, 0.016) == 26 and schedule.rank_from_table_ratio(4096, 2048, 0.083) == 170
    assert schedule.infinity_group_ranks(48, 2048, 4) == [schedule.infinity_group_ranks(48)[c] for c in (1, 3, 5, 7)]


def test_bf16_rounding_of_the_input_generator():
    x = np.array([1.0, 1.00390625, 1.005859375, -2.5, 3.0e38, 1e-40], dtype=np.float32)
    r = si.round_to_bf16(x)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == np.float32(1.0078125)     # ties to even, then up
    assert np.all((r.view(np.uint32) & 0xFFFF) == 0)
    assert np.array_equal(si.bf16_bits_to_f32(si.bf16_bits(r)), r)
