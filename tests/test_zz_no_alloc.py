"""The allocation-free row selection (fvar_select_rows_static) against the two-call form.

Some users of the library run where they may not allocate device memory: everything on the GPU was
handed out at start-up by a server or another framework, or an allocation would stall a latency-
critical loop.  For them the scores between the score kernel and the selection kernel live in a
fixed array inside the library.  This test calls that entry point through the C ABI twice in a row
(the array is shared and keeps the previous call's contents, so the second call must not be
disturbed by the first) and requires the same index lists, bit for bit, as fvar_row_scores +
fvar_select_topr; it also checks that a request larger than the built-in array is refused with a
message instead of being run.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import synth_inputs as si

pytestmark = pytest.mark.gpu


def test_static_selection_matches_two_call_form_twice():
    from paper_2512_16483_b200 import binding as fv
    fv.load_library()
    cases = [(3, 1600, 256, 400, 11), (2, 256, 1024, 128, 12)]       # second call: smaller, different data
    for B, M, C, r, seed in cases:
        x = torch.from_numpy(si.make_tokens(seed, B, M, C, "spread")).cuda()
        ref_idx, ref_inv = fv.fvar_select_topr(fv.fvar_row_scores(x), r)
        idx = torch.full((B, r), -5, dtype=torch.int32, device="cuda")
        inv = torch.full((B, M), -5, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        held, free = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
        fv.fvar_select_rows_static(x, r, idx, inv)
        torch.cuda.synchronize()
        # nothing was allocated: not through torch, and (from the second call on, once the kernels' code is loaded)
        # not behind its back either
        assert torch.cuda.memory_allocated() == held
        if seed == 12:
            assert torch.cuda.mem_get_info()[0] >= free
        assert torch.equal(idx, ref_idx) and torch.equal(inv, ref_inv)
        assert bool((idx[:, 1:] > idx[:, :-1]).all())


def test_static_selection_rejects_oversized_requests():
    import ctypes as ct
    from paper_2512_16483_b200 import binding as fv
    lib = fv.load_library()
    B, M, C = 3, 32768, 4                                             # 98304 rows > 65536
    x = torch.zeros((B, M, C), dtype=torch.float32, device="cuda")
    idx = torch.zeros((B, 8), dtype=torch.int32, device="cuda")
    inv = torch.zeros((B, M), dtype=torch.int32, device="cuda")
    st = lib.fvar_select_rows_static(x.data_ptr(), B, M, C, 8, idx.data_ptr(), inv.data_ptr(), None)
    assert st == fv.EUNSUPPORTED
    assert b"exceeds" in lib.fvar_last_error(None)
    assert lib.fvar_select_rows_static(None, 1, 1, 4, 1, idx.data_ptr(), inv.data_ptr(), None) == fv.EINVAL
