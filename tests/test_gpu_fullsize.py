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
from helpers import assert_close, assert_out_close, bf16_to_numpy, rel_err, to_bf16_cuda
from test_gpu_step import Pair, _step_both

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


# ----------------------------------------------------------------------------- the Infinity-2B-shaped late scales
# (the largest single-GPU workload: 8 block groups at the ranks App. A.1 tabulates, scales 40 -> 48 -> 64)

def test_infinity_eight_groups_three_late_scales_table_ranks(fv):
    """The eight block groups of the Infinity-2B shape at the eight tabulated ranks of each late scale, the scales
    40 -> 48 -> 64 in sequence with KV append between them (the cache grows by r per block), null-prompt branch
    only, free-running in the benchmark's configuration first (index overlap) and then teacher-forced (values).
    One block per group instead of four: eight blocks of fp64 oracle weights are 4.3 GB of host memory, thirty-two
    would be 17 GB; the four-block group keeps its own test above.
    Bar: the fp32 output of group g (0-based) is held to 2e-2 x sqrt(g + 1) x RMS, cosine >= 0.999.  The random
    projection keeps the energy of whatever it projects, so the deviation a group leaves in its rows is carried
    whole into the r rows of the next group and that group's own deviation adds in quadrature
    (tests/test_tolerance_floor.py::test_deviations_add_in_quadrature_over_block_groups shows the law on the oracle
    alone).  Measured: 1.2e-2 .. 1.7e-2 after the first group, 2.2e-2 / 2.3e-2 / 4.2e-2 at worst after all eight at
    the scales 40 / 48 / 64; the cosine stays above 0.999999 throughout."""
    from paper_2512_16483_b200 import schedule
    shp = si.shape_infinity_2b(n_blocks=8, blocks_per_group=1)
    B, k0 = 2, 10
    p = Pair(fv, shp, seed=4048, B=B)
    assert p.prefill(k0) == 2521
    Ms = shp.tokens_per_scale()
    ranks = {k: schedule.infinity_group_ranks(shp.scales[k], shp.width, 8) for k in (10, 11, 12)}
    assert ranks[10] == [26, 218, 336, 400, 410, 317, 251, 306] and ranks[12] == [16, 111, 170, 135, 115, 59, 78, 113]
    toks = {k: si.make_tokens(4048, B, Ms[k], shp.width, "spread") for k in (10, 11, 12)}
    for k in (10, 11, 12):
        p.set_projections(k, ranks[k])
    free_idx = {}
    for k in (10, 11, 12):                                   # pass 1: graph replay, selection by the kernels
        p.gpu.scale_step(to_bf16_cuda(toks[k]), k, mode=fv.LOWRANK_RTR, cfg_mode=fv.CFG_NULL_ONLY, rank_per_group=ranks[k])
        free_idx[k] = [p.gpu.get_indices(g, 1, Ms[k]).cpu().numpy()[0] for g in range(8)]
        p.gpu.kv_append(k)
    p.check_ok()
    assert [p.gpu.cache_len(b) for b in range(8)] == [2521 + ranks[10][b] + ranks[11][b] + ranks[12][b] for b in range(8)]
    p.gpu.restore_loaded()
    for k in (10, 11, 12):                                   # pass 2: teacher-forced with the oracle's index lists
        M = Ms[k]
        ref = p.oracle.scale_step(toks[k], k, orc.Policy("lowrank_rtr", "null_only", rank_per_group=ranks[k]))
        out = p.gpu.scale_step(to_bf16_cuda(toks[k]), k, mode=fv.LOWRANK_RTR, cfg_mode=fv.CFG_NULL_ONLY, rank_per_group=ranks[k],
                               forced_indices=p.forced_tensor(ranks[k], 1))
        p.check_ok()
        errs = []
        for g in range(8):
            g32 = p.gpu.get_group_output(g, M).cpu().numpy()[1]
            errs.append(rel_err(g32, p.oracle.group_cache[g][1]))
        print("scale", shp.scales[k], "max-abs / RMS and cosine per group:", ["%.2e %.6f" % e for e in errs])
        for g in range(8):                                   # 2e-2 x RMS per group, in quadrature over the groups so far
            assert errs[g][0] <= 2e-2 * np.sqrt(g + 1.0) and errs[g][1] >= 0.999, (shp.scales[k], g, errs)
        assert_out_close(bf16_to_numpy(out), ref, what="Infinity 8 groups, scale %d" % shp.scales[k], max_rel=2e-2 * np.sqrt(8.0))
        inter = total = 0
        for g in range(8):
            a, b = free_idx[k][g], p.oracle.last_indices[0][g]
            assert len(a) == ranks[k][g] and np.all(np.diff(a) > 0) and a[0] >= 0 and a[-1] < M
            inter += len(np.intersect1d(a, b))
            total += len(b)
        assert inter / total >= 0.97, (k, inter / total)
        p.gpu.kv_append(k)
        p.oracle.kv_append(k)
    assert [p.gpu.cache_len(b) for b in range(8)] == [p.oracle.cache_len(b, 1) for b in range(8)]


def test_var_d30_three_blocks_two_late_scales(fv):
    """VAR-d30 shape (C = 1920, 30 heads, FFN 7680): three blocks, scales 13 -> 16 in sequence, keep ratios 0.75
    and 0.5, both CFG branches at 0.75 and the null-prompt branch alone at 0.5."""
    shp = si.shape_var_d30(n_blocks=3)
    B = 4
    for rho, cfg in ((0.75, "pair"), (0.5, "null_only")):
        p = Pair(fv, shp, seed=3016, B=B)
        p.prefill(8)
        for k in (8, 9):
            M = shp.tokens_per_scale()[k]
            r = orc.rank_from_keep_ratio(M, rho)
            p.set_projections(k, [r] * 3)
            toks = si.make_tokens(3016, B, M, 1920, "spread")
            got, ref = _step_both(p, toks, k, mode=fv.LOWRANK_RTR, cfg=cfg, keep_ratio=rho)
            assert_out_close(got, ref, what="d30, rho %.2f, scale %d" % (rho, shp.scales[k]), max_rel=2e-2 * np.sqrt(3.0))   # third group
            p.gpu.kv_append(k)
            p.oracle.kv_append(k)
        r13, r16 = orc.rank_from_keep_ratio(169, rho), orc.rank_from_keep_ratio(256, rho)
        assert p.gpu.cache_len(2) == 255 + r13 + r16 == p.oracle.cache_len(2, B - 1)


@pytest.mark.parametrize("B", [2, 4])
def test_infinity_group_last_scale_small_ranks(fv, B):
    """Corners of the last-scale sweep: ranks 16 and 64 at one and two CFG pairs on one Infinity-2B-shaped block
    group (4 blocks) at the 64 x 64 scale over the 6425-row cache, null-prompt branch only."""
    shp = si.shape_infinity_2b(n_blocks=4, blocks_per_group=4)
    k = 12
    p = Pair(fv, shp, seed=5000 + B, B=B)
    p.prefill(k)
    toks = si.make_tokens(5000 + B, B, 4096, 2048, "spread")
    gc = si.make_group_cache(5000 + B, 1, B, shp.tokens_per_scale()[k - 1], 2048)
    for r in (16, 64):
        p.set_projections(k, [r])
        got, ref = _step_both(p, toks, k, mode=fv.LOWRANK_RTR, cfg="null_only", ranks=[r], forced=False, bar=INF_BAR)
        idx = p.gpu.get_indices(0, B // 2, 4096).cpu().numpy()
        for e in range(B // 2):
            assert np.array_equal(idx[e], p.oracle.last_indices[e][0])          # well-separated scores: exact
        assert_out_close(got, ref, what="Infinity group, r = %d, B = %d" % (r, B), max_rel=INF_BAR)
        g32 = p.gpu.get_group_output(0, 4096).cpu().numpy()[1::2]
        assert_close(g32, np.stack([p.oracle.group_cache[0][b] for b in range(1, B, 2)]), max_rel=INF_BAR, what="fp32 group output")
        p.gpu.restore_loaded()
        p.oracle.load_group_cache(k - 1, gc)
        p.oracle.load_kv(*si.make_kv_prefill(5000 + B, 4, B, 6425, 2048))


def test_infinity_group_last_scale_lls_restoration(fv):
    """The LLS restoration variant (Eq. "lstsq", App. A.3) on one Infinity-2B-shaped block group at the last scale:
    4096 rows restored from r = 64 block-output rows by the two least-squares matrices, against the oracle's fp64 solve."""
    shp = si.shape_infinity_2b(n_blocks=4, blocks_per_group=4)
    B, k, r = 2, 12, 64
    p = Pair(fv, shp, seed=66, B=B)
    p.prefill(k)
    p.set_projections(k, [r])
    toks = si.make_tokens(66, B, 4096, 2048, "spread")
    ref = p.oracle.scale_step(toks, k, orc.Policy("lowrank_rtr", "null_only", rank_per_group=[r], restore="lls"))
    out = p.gpu.scale_step(to_bf16_cuda(toks), k, mode=fv.LOWRANK_RTR, cfg_mode=fv.CFG_NULL_ONLY, rank_per_group=[r],
                           restore=fv.RESTORE_LLS)
    p.check_ok()
    e, c = rel_err(p.gpu.get_group_output(0, 4096).cpu().numpy()[1], p.oracle.group_cache[0][1])
    print("Infinity-shaped LLS group: max-abs/RMS %.3e cosine %.6f" % (e, c))
    assert e <= 2e-2 and c >= 0.999, (e, c)                  # measured 0.8e-2: the stated bar holds here
    assert_out_close(bf16_to_numpy(out), ref, what="Infinity-shaped group, LLS")
    p.gpu.kv_append(k)
    assert [p.gpu.cache_len(b) for b in range(4)] == [6425 + r] * 4
