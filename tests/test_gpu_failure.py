"""Failure detection without a fault: a device-side wait that runs out is reported through the status word
and leaves the context usable.  Every wait in the library's kernels is bounded by a clock budget; here a
one-CTA kernel waits on a barrier that nothing signals, with a budget of about a millisecond."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from helpers import assert_out_close, bf16_to_numpy, to_bf16_cuda
from test_gpu_step import Pair, _step_both

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fv():
    from paper_2512_16483_b200 import binding
    binding.load_library()
    return binding


def test_wait_runs_out_on_a_context_and_the_context_survives(fv):
    shp = si.shape_tiny(n_blocks=2, blocks_per_group=1, width=128, n_heads=2, head_dim=64, ffn_dim=256, scales=(1, 2, 3, 5))
    p = Pair(fv, shp, seed=71, B=2, std=0.05)
    p.check_ok()
    p.gpu.selftest_wait_timeout(2_000_000)                       # about 1 ms at boost clock
    assert p.gpu.poll_status() == fv.ETIMEOUT
    assert b"wait ran out" in (p.gpu.lib.fvar_last_error(p.gpu.ctx) or b"")
    assert p.gpu.poll_status() == fv.OK                          # the word was cleared by the first poll
    for k in range(3):                                           # and the context still computes correctly
        toks = si.make_tokens(71, 2, shp.tokens_per_scale()[k], 128)
        got, ref = _step_both(p, toks, k, mode=fv.DENSE)
        assert_out_close(got, ref, what="dense step %d after a timeout" % k)
        p.gpu.kv_append(k)
        p.oracle.kv_append(k)


def test_wait_runs_out_at_kernel_level_then_a_gemm_passes(fv):
    lib = fv.load_library()
    assert fv.kernel_poll_status() == fv.OK
    with pytest.raises(Exception):
        fv._check_kernel(lib.fvar_selftest_wait_timeout(None, 0, None))        # a budget must be positive
    fv._check_kernel(lib.fvar_selftest_wait_timeout(None, 2_000_000, torch.cuda.current_stream().cuda_stream))
    assert fv.kernel_poll_status() == fv.ETIMEOUT
    assert fv.kernel_poll_status() == fv.OK
    rng = np.random.default_rng(5)
    A, W = si.normal_bf16(rng, (130, 256)), si.normal_bf16(rng, (200, 256), 0.05)
    for form, bn in ((fv.GEMM_AUTO, 0), (fv.GEMM_SKINNY, 0), (fv.GEMM_PAIR, 128)):
        got = fv.fvar_gemm_bf16_form(to_bf16_cuda(A), to_bf16_cuda(W), None, form, bn).cpu().numpy()
        assert fv.kernel_poll_status() == fv.OK
        ref = A.astype(np.float64) @ W.astype(np.float64).T
        np.testing.assert_allclose(got, ref, atol=1e-5 * (np.abs(A).astype(np.float64) @ np.abs(W).astype(np.float64).T).max() + 1e-6, rtol=0)
