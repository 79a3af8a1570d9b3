"""Parity at the full sizes of the workloads, in the launch configuration the benchmark times
(CUDA graphs on, free-running selection), on what the oracle can compute in seconds:
  * the VAR-d16 stack (16 blocks, batch 16, late scales 10 / 13 / 16, null-only, keep ratio 0.5);
  * a VAR-d30-shaped block (C = 1920, 30 heads);
  * an Infinity-2B-shaped block group (4 blocks, C = 2048, 16 x 128 heads, cross-attention to 256
    context tokens) at the last scale (4096 tokens over a 6425-row cache) at the paper's rank 170;
  * one Infinity-2B-shaped block run densely at the last scale, on a seeded sample of query rows
    (keys and values come from all rows).
The Infinity-shaped cases use a bar of 3e-2 x RMS instead of 2e-2: with N(0, 0.02) weights at C = 2048,
F = 8192 the branches are as large as the residual stream, and rounding the two FFN operands to bf16 --
which any bf16 tensor-core path must do -- already costs 1.6e-2 x RMS (tests/test_tolerance_floor.py).
Index lists are compared exactly where the two sides agree on every group of an element, and by
overlap otherwise (a last-bit difference of a score can flip a near tie)."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import fvar_oracle as orc
from helpers import assert_close, assert_out_close, bf16_to_numpy, to_bf16_cuda
from test_gpu_step import Pair

pytestmark = pytest.mark.gpu

INF_BAR = 3e-2      # see the module docstring


@pytest.fixture(scope="module")
def fv():
    from paper_2512_16483_b200 import binding
    binding.load_library()
    return binding


def test_var_d16_stack_bench_workload(fv):
    shp = si.shape_var_d16()
    B, k0 = 16, 7
    p = Pair(fv, shp, seed=2512, B=B)
    p.prefill(k0)
    Ms = shp.tokens_per_scale()
    E = B // 2
    toks = {k: si.make_tokens(2512, B, Ms[k], 1024, "spread") for k in (7, 8, 9)}
    ranks = {k: orc.rank_from_keep_ratio(Ms[k], 0.5) for k in (7, 8, 9)}
    for k in (7, 8, 9):
        p.set_projections(k, [ranks[k]] * 16)
    # pass 1 -- the benchmark's configuration: graph replay, selection by the kernels
    free, free_idx = {}, {}
    for k in (7, 8, 9):
        free[k] = p.gpu.scale_step(to_bf16_cuda(toks[k]), k, mode=fv.LOWRANK_RTR, cfg_mode=fv.CFG_NULL_ONLY,
                                   keep_ratio=0.5).clone()
        free_idx[k] = [p.gpu.get_indices(g, E, Ms[k]).cpu().numpy() for g in range(16)]
        p.gpu.kv_append(k)
    p.check_ok()
    assert p.gpu.cache_len(15) == 155 + 50 + 85 + 128
    # pass 2 -- the same kernels teacher-forced with the oracle's index lists, from the same start state
    p.gpu.restore_loaded()
    agree_all_scales = np.ones(E, bool)
    for k in (7, 8, 9):
        M, r = Ms[k], ranks[k]
        ref = p.oracle.scale_step(toks[k], k, orc.Policy("lowrank_rtr", "null_only", 0.5))
        out = p.gpu.scale_step(to_bf16_cuda(toks[k]), k, mode=fv.LOWRANK_RTR, cfg_mode=fv.CFG_NULL_ONLY, keep_ratio=0.5,
                               forced_indices=p.forced_tensor([r] * 16, E))
        p.check_ok()
        assert_out_close(bf16_to_numpy(out), ref, what="d16 stack, scale %d, teacher-forced" % k)
        g32 = p.gpu.get_group_output(15, M).cpu().numpy()[1::2]
        assert_close(g32, np.stack([p.oracle.group_cache[15][b] for b in range(1, B, 2)]), what="fp32 last group output")
        inter = total = 0
        for g in range(16):
            for e in range(E):
                a, b = free_idx[k][g][e], p.oracle.last_indices[e][g]
                assert np.all(np.diff(a) > 0) and a[0] >= 0 and a[-1] < M and len(a) == r
                inter += len(np.intersect1d(a, b))
                total += r
                agree_all_scales[e] &= np.array_equal(a, b)
        assert inter / total >= 0.97, (k, inter / total)
        for e in np.nonzero(agree_all_scales)[0]:      # same lists so far: same kernels, same inputs, same bits
            assert torch.equal(free[k][e], out[e])
        p.gpu.kv_append(k)
        p.oracle.kv_append(k)
    assert p.gpu.cache_len(15) == 155 + 50 + 85 + 128 == p.oracle.cache_len(15, 1)


def test_var_d30_block(fv):
    shp = si.shape_var_d30(n_blocks=1)
    B, k = 4, 8
    p = Pair(fv, shp, seed=30, B=B)
    p.prefill(k)
    M = shp.tokens_per_scale()[k]
    for rho in (0.75, 0.5):
        r = orc.rank_from_keep_ratio(M, rho)
        p.set_projections(k, [r])
        toks = si.make_tokens(30, B, M, 1920, "spread")
        ref = p.oracle.scale_step(toks, k, orc.Policy("lowrank_rtr", "pair", rho))
        out = p.gpu.scale_step(to_bf16_cuda(toks), k, mode=fv.LOWRANK_RTR, keep_ratio=rho)
        p.check_ok()
        idx = p.gpu.get_indices(0, B, M).cpu().numpy()
        for e in range(B):
            assert np.array_equal(idx[e], p.oracle.last_indices[e][0])
        assert_out_close(bf16_to_numpy(out), ref, what="d30 block rho=%.2f" % rho)
        assert_close(p.gpu.get_group_output(0, M).cpu().numpy(), np.stack(p.oracle.group_cache[0]), what="d30 fp32")
        p.gpu.restore_loaded()
        p.oracle.load_group_cache(k - 1, si.make_group_cache(30, 1, B, shp.tokens_per_scale()[k - 1], 1920))


def test_infinity_group_last_scale_rank_170(fv):
    shp = si.shape_infinity_2b(n_blocks=4, blocks_per_group=4)
    B, k, r = 2, 12, 170
    p = Pair(fv, shp, seed=64, B=B)
    assert p.prefill(k) == 6425
    p.set_projections(k, [r])
    toks = si.make_tokens(64, B, 4096, 2048, "spread")
    ref = p.oracle.scale_step(toks, k, orc.Policy("lowrank_rtr", "null_only", rank_per_group=[r]))
    out = p.gpu.scale_step(to_bf16_cuda(toks), k, mode=fv.LOWRANK_RTR, cfg_mode=fv.CFG_NULL_ONLY, rank_per_group=[r])
    p.check_ok()
    idx = p.gpu.get_indices(0, 1, 4096).cpu().numpy()
    assert np.array_equal(idx[0], p.oracle.last_indices[0][0])
    assert_out_close(bf16_to_numpy(out), ref, what="Infinity-shaped group, r=170", max_rel=INF_BAR)
    assert_close(p.gpu.get_group_output(0, 4096).cpu().numpy()[1], p.oracle.group_cache[0][1], what="Infinity fp32", max_rel=INF_BAR)
    p.gpu.kv_append(k)
    assert [p.gpu.cache_len(b) for b in range(4)] == [6425 + r] * 4


def test_infinity_block_dense_last_scale_sampled_rows(fv):
    shp = si.shape_infinity_2b(n_blocks=1, blocks_per_group=1)
    B, k = 2, 12
    p = Pair(fv, shp, seed=65, B=B)
    p.prefill(k)
    toks = si.make_tokens(65, B, 4096, 2048)
    out = p.gpu.scale_step(to_bf16_cuda(toks), k, mode=fv.DENSE)
    p.check_ok()
    g32 = p.gpu.get_group_output(0, 4096).cpu().numpy()
    rows = np.sort(np.random.default_rng(65).choice(4096, 192, replace=False))
    o = p.oracle
    for b in range(B):
        ref, _, _ = orc.block_forward(toks[b].astype(np.float64), o.ada[0][b], o.w[0], o.K[0][b], o.V[0][b], shp.n_heads,
                                      shp.ln_eps, o.cross_kv[0][b], query_rows=rows)
        assert_close(g32[b][rows], ref, what="Infinity dense block, sampled rows, element %d" % b, max_rel=INF_BAR)
        assert_out_close(bf16_to_numpy(out[b])[rows], ref, what="Infinity dense block bf16, element %d" % b, max_rel=INF_BAR)
