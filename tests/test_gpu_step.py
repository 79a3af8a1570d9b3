"""Parity of the whole scale step (through the C ABI) against the CPU oracle on the same seeded
inputs.  Acceptance bar for block outputs in bf16: max-abs error <= 2e-2 x output RMS and cosine
similarity >= 0.999; index lists bit-exact when the index set is teacher-forced or the scores are
well separated."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import fvar_oracle as orc
from helpers import assert_close, assert_out_close, bf16_to_numpy, rel_err, to_bf16_cuda, weights_to_cuda

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fv():
    from paper_2512_16483_b200 import binding
    binding.load_library()
    return binding


class Pair:
    """The GPU context and the oracle on identical weights and conditioning."""

    def __init__(self, fv, shp: si.ModelShape, seed: int, B: int, std: float = 0.02):
        self.fv, self.shp, self.seed, self.B = fv, shp, seed, B
        w = si.make_weights(seed, shp, std)
        self.oracle = orc.Oracle(w, shp.n_heads, shp.blocks_per_group, shp.hw(), shp.ln_eps)
        self.gpu = fv.Fvar(weights_to_cuda(w), blocks_per_group=shp.blocks_per_group, n_heads=shp.n_heads,
                           head_dim=shp.head_dim, ffn_dim=shp.ffn_dim, scale_hw=shp.hw(), max_batch=B,
                           ctx_len=shp.ctx_len, ctx_width=shp.ctx_width, ln_eps=shp.ln_eps)
        cond = si.make_cond(seed, B, shp.width)
        ctx = si.make_context(seed, B, shp.ctx_len, shp.ctx_width) if shp.has_cross_attn else None
        self.oracle.set_cond(cond, ctx)
        self.gpu.set_cond(to_bf16_cuda(cond), to_bf16_cuda(ctx) if ctx is not None else None)

    def prefill(self, upto_scale: int):
        """Stand-in earlier scales 0..upto_scale-1: random K/V rows and random group outputs of the
        last of them."""
        shp = self.shp
        L = sum(shp.tokens_per_scale()[:upto_scale])
        K, V = si.make_kv_prefill(self.seed, shp.n_blocks, self.B, L, shp.width)
        self.oracle.load_kv(K, V)
        self.gpu.load_kv(to_bf16_cuda(K), to_bf16_cuda(V))
        M_prev = shp.tokens_per_scale()[upto_scale - 1]
        gc = si.make_group_cache(self.seed, shp.n_groups, self.B, M_prev, shp.width)
        self.oracle.load_group_cache(upto_scale - 1, gc)
        self.gpu.load_group_cache(upto_scale - 1, torch.from_numpy(gc).cuda())
        return L

    def set_projections(self, k: int, ranks):
        M = self.shp.tokens_per_scale()[k]
        for g, r in enumerate(ranks):
            if r < M:
                Q = si.make_projection(self.seed, k, g, M, r)
                self.oracle.set_projection(k, g, Q)
                self.gpu.set_projection(k, g, to_bf16_cuda(np.ascontiguousarray(Q.T)))

    def forced_tensor(self, ranks, E):
        """Oracle's index lists as the [G][E][r_max] device array the policy takes."""
        G, r_max = len(ranks), max(ranks)
        arr = np.zeros((G, E, r_max), np.int32)
        for g in range(G):
            for e in range(E):
                idx = self.oracle.last_indices[e][g]
                if len(idx) <= r_max:                        # dense groups (r == M) carry no list
                    arr[g, e, :len(idx)] = idx
        return torch.from_numpy(arr).cuda()

    def check_ok(self):
        assert self.gpu.poll_status() == self.fv.OK


def _step_both(p: Pair, toks, k, *, mode, cfg="pair", ranks=None, keep_ratio=1.0, forced=True, bar=2e-2):
    """One step on both sides.  Besides returning the bf16 result and the oracle's, holds the fp32 output of every
    block group (what the next group and the next scale read) to the block-output bar: max-abs error <= bar x RMS,
    cosine >= 0.999, on the batch elements the step computed.  Under RP + RTR the bar of group g (0-based) is
    bar x sqrt(g + 1): the projection carries the whole deviation of a group's rows into the rows of the next
    one, so the groups' deviations add in quadrature (tests/test_tolerance_floor.py shows the law on the oracle)."""
    fv = p.fv
    pol = orc.Policy({fv.DENSE: "dense", fv.LOWRANK_RTR: "lowrank_rtr"}[mode], cfg, keep_ratio, ranks)
    ref = p.oracle.scale_step(toks, k, pol)
    E = ref.shape[0]
    fi = None
    if mode == fv.LOWRANK_RTR and forced:
        M = toks.shape[1]
        rk = ranks if ranks is not None else [orc.rank_from_keep_ratio(M, keep_ratio)] * p.shp.n_groups
        if any(r < M for r in rk):
            fi = p.forced_tensor([r if r < M else 1 for r in rk], E)
    out = p.gpu.scale_step(to_bf16_cuda(toks), k, mode=mode, cfg_mode=fv.CFG_NULL_ONLY if cfg == "null_only" else fv.CFG_PAIR,
                           keep_ratio=keep_ratio, rank_per_group=ranks, forced_indices=fi)
    p.check_ok()
    els = list(range(1, p.B, 2)) if cfg == "null_only" else list(range(p.B))
    if forced or mode == fv.DENSE:
        for g in range(p.shp.n_groups):
            g32 = p.gpu.get_group_output(g, toks.shape[1]).cpu().numpy()
            assert_close(g32[els], np.stack([p.oracle.group_cache[g][b] for b in els]),
                         max_rel=bar * (np.sqrt(g + 1.0) if mode == fv.LOWRANK_RTR else 1.0),
                         what="fp32 output of group %d, scale %d" % (g, k))
    return bf16_to_numpy(out), ref


# ----------------------------------------------------------------------------- one d16 block, last 256px scale

@pytest.mark.parametrize("r", [256, 128, 32])
@pytest.mark.parametrize("kind", ["normal", "spread"])
def test_single_block_last_scale(fv, r, kind):
    """One VAR-d16-shaped block, B = 2 (one CFG pair), 256 query tokens over a 424-row cache."""
    shp = si.shape_var_d16(n_blocks=1)
    p = Pair(fv, shp, seed=100, B=2)
    k = 9
    assert p.prefill(k) == 424
    toks = si.make_tokens(100, 2, 256, 1024, kind)
    mode = fv.DENSE if r == 256 else fv.LOWRANK_RTR
    if r < 256:
        p.set_projections(k, [r])
    free = (kind == "spread")                              # well-separated scores: selection must agree exactly
    got, ref = _step_both(p, toks, k, mode=mode, ranks=[r] if r < 256 else None, forced=not free)
    assert_out_close(got, ref, what="block output r=%d %s" % (r, kind))
    if r < 256:
        idx = p.gpu.get_indices(0, 2, 256).cpu().numpy()
        for e in range(2):
            assert np.array_equal(idx[e], p.oracle.last_indices[e][0])
    g32 = p.gpu.get_group_output(0, 256).cpu().numpy()
    assert_close(g32, np.stack(p.oracle.group_cache[0]), what="fp32 group output")
    p.gpu.kv_append(k)
    p.oracle.kv_append(k)
    assert p.gpu.cache_len(0) == p.oracle.cache_len(0, 0) == 424 + r


def test_full_rank_is_bitwise_the_dense_path(fv):
    shp = si.shape_var_d16(n_blocks=2)
    toks = to_bf16_cuda(si.make_tokens(101, 2, 169, 1024))
    outs = []
    for mode, kw in ((fv.DENSE, {}), (fv.LOWRANK_RTR, {"keep_ratio": 1.0})):
        p = Pair(fv, shp, seed=101, B=2)
        p.prefill(8)
        outs.append(p.gpu.scale_step(toks, 8, mode=mode, **kw).clone())
        p.check_ok()
    assert torch.equal(outs[0], outs[1])


# ----------------------------------------------------------------------------- multi-scale, multi-group

@pytest.mark.parametrize("cross,D", [(False, 64), (True, 64), (True, 128)])
def test_generation_dense_then_late(fv, cross, D):
    """Dense early scales, then two late scales under RP + RTR with different ranks per group,
    the second one null-prompt only; KV append between scales; indices teacher-forced."""
    shp = si.shape_tiny(n_blocks=4, blocks_per_group=2, width=2 * D, n_heads=2, head_dim=D, ffn_dim=320,
                        scales=(1, 2, 4, 7, 12), cross=cross, ctx_len=20,
                        scale_hw=((1, 1), (2, 2), (4, 3), (7, 7), (12, 11)))
    B = 4
    p = Pair(fv, shp, seed=102, B=B, std=0.05)
    Ms = shp.tokens_per_scale()
    toks = [si.make_tokens(102, B, m, shp.width) for m in Ms]
    for k in range(3):
        got, ref = _step_both(p, toks[k], k, mode=fv.DENSE)
        assert_out_close(got, ref, what="dense scale %d" % k)
        p.gpu.kv_append(k)
        p.oracle.kv_append(k)
    ranks3 = [20, 33]
    p.set_projections(3, ranks3)
    got, ref = _step_both(p, toks[3], 3, mode=fv.LOWRANK_RTR, ranks=ranks3)
    assert_out_close(got, ref, what="late scale 3")
    p.gpu.kv_append(3)
    p.oracle.kv_append(3)
    assert [p.gpu.cache_len(b) for b in range(4)] == [p.oracle.cache_len(b, 0) for b in range(4)]
    ranks4 = [132, 40]                                      # first group dense (r == M), second low-rank
    p.set_projections(4, ranks4)
    got, ref = _step_both(p, toks[4], 4, mode=fv.LOWRANK_RTR, cfg="null_only", ranks=ranks4)
    assert got.shape == (2, 132, shp.width)
    assert_out_close(got, ref, what="late scale 4 (null-only)")
    p.gpu.kv_append(4)
    p.oracle.kv_append(4)
    assert [p.gpu.cache_len(b) for b in range(4)] == [p.oracle.cache_len(b, 1) for b in range(4)]


def test_d16_stack_three_late_scales(fv):
    """VAR-d16-shaped stack (4 of its 16 blocks to keep the oracle quick), late scales 10, 13, 16 at
    keep ratio 0.5, batch 4, teacher-forced; plus free-running index overlap."""
    shp = si.shape_var_d16(n_blocks=4)
    B = 4
    p = Pair(fv, shp, seed=103, B=B)
    p.prefill(7)
    overlaps = []
    for k in (7, 8, 9):
        M = shp.tokens_per_scale()[k]
        r = orc.rank_from_keep_ratio(M, 0.5)
        p.set_projections(k, [r] * 4)
        toks = si.make_tokens(103, B, M, 1024, "spread")
        got, ref = _step_both(p, toks, k, mode=fv.LOWRANK_RTR, keep_ratio=0.5)
        assert_out_close(got, ref, what="d16 stack scale %d" % k)
        p.gpu.kv_append(k)
        p.oracle.kv_append(k)
    assert p.gpu.cache_len(3) == 155 + 50 + 85 + 128


def test_free_running_selection_overlap(fv):
    """Without teacher forcing the index sets may differ only where scores are nearly tied."""
    shp = si.shape_var_d16(n_blocks=3)
    B = 2
    p = Pair(fv, shp, seed=104, B=B)
    p.prefill(9)
    p.set_projections(9, [128] * 3)
    toks = si.make_tokens(104, B, 256, 1024, "spread")
    got, ref = _step_both(p, toks, 9, mode=fv.LOWRANK_RTR, keep_ratio=0.5, forced=False)
    for g in range(3):
        idx = p.gpu.get_indices(g, B, 256).cpu().numpy()
        for e in range(B):
            inter = len(set(idx[e].tolist()) & set(p.oracle.last_indices[e][g].tolist()))
            assert inter >= 126, (g, e, inter)
            assert np.all(np.diff(idx[e]) > 0)


# ----------------------------------------------------------------------------- host-buffer entry point, state rules

def test_host_entry_point_matches_device_entry_point(fv):
    shp = si.shape_var_d16(n_blocks=1)
    toks = si.make_tokens(105, 2, 256, 1024)
    outs = []
    for host in (False, True):
        p = Pair(fv, shp, seed=105, B=2)
        p.prefill(9)
        p.set_projections(9, [128])
        if host:
            th = to_bf16_cuda(toks).cpu().pin_memory()
            oh = torch.empty((2, 256, 1024), dtype=torch.bfloat16).pin_memory()
            p.gpu.scale_step_host(th, 9, oh, mode=fv.LOWRANK_RTR, keep_ratio=0.5)
            outs.append(oh.clone())
        else:
            outs.append(p.gpu.scale_step(to_bf16_cuda(toks), 9, mode=fv.LOWRANK_RTR, keep_ratio=0.5).cpu())
        p.check_ok()
    assert torch.equal(outs[0], outs[1])


def test_state_and_argument_errors(fv):
    shp = si.shape_tiny(n_blocks=2, width=128, n_heads=2, head_dim=64, ffn_dim=256, scales=(2, 3, 4))
    p = Pair(fv, shp, seed=106, B=2)
    g = p.gpu
    t0 = to_bf16_cuda(si.make_tokens(106, 2, 4, 128))
    t1 = to_bf16_cuda(si.make_tokens(106, 2, 9, 128))

    def status_of(fn):
        try:
            fn()
        except fv.FvarError as e:
            return e.status
        return fv.OK

    assert status_of(lambda: g.kv_append(0)) == fv.ESTATE                      # nothing staged
    assert status_of(lambda: g.scale_step(t1, 1, mode=fv.LOWRANK_RTR, keep_ratio=0.5)) == fv.ESTATE   # no projection
    g.set_projection(1, 0, to_bf16_cuda(np.ascontiguousarray(si.make_projection(1, 1, 0, 9, 5).T)))
    g.set_projection(1, 1, to_bf16_cuda(np.ascontiguousarray(si.make_projection(1, 1, 1, 9, 5).T)))
    assert status_of(lambda: g.scale_step(t1, 1, mode=fv.LOWRANK_RTR, keep_ratio=0.5)) == fv.ESTATE   # no group cache
    assert status_of(lambda: g.scale_step(t0, 0, mode=fv.LOWRANK_RTR, rank_per_group=[5, 2])) == fv.EINVAL   # r > M
    assert status_of(lambda: g.scale_step(t0, 7, mode=fv.DENSE)) == fv.EINVAL
    assert g.scale_step(t0, 0, mode=fv.SKIP) is None                           # skip: nothing staged
    assert status_of(lambda: g.kv_append(0)) == fv.ESTATE
    g.scale_step(t0, 0, mode=fv.DENSE)
    g.kv_append(0)
    assert status_of(lambda: g.kv_append(0)) == fv.ESTATE                      # appended twice
    assert g.cache_len(0) == 4
    g.scale_step(t1, 1, mode=fv.LOWRANK_RTR, cfg_mode=fv.CFG_NULL_ONLY, keep_ratio=0.5)
    assert status_of(lambda: g.scale_step(t0, 0, mode=fv.DENSE)) == fv.ESTATE  # scale index decreased
    assert status_of(lambda: g.scale_step(t1, 1, mode=fv.DENSE)) == fv.ESTATE  # pair step after null-only
    assert g.poll_status() == fv.OK
    # a forced index list that is not ascending is reported through the status word, not by a fault
    bad = torch.tensor([[[3, 1, 2, 8, 8], [0, 1, 2, 3, 4]]] * 2, dtype=torch.int32, device="cuda")
    g.reset()
    p2 = Pair(fv, shp, seed=106, B=2)
    p2.gpu.scale_step(t0, 0, mode=fv.DENSE)
    p2.gpu.kv_append(0)
    for grp in range(2):
        p2.gpu.set_projection(1, grp, to_bf16_cuda(np.ascontiguousarray(si.make_projection(1, 1, grp, 9, 5).T)))
    p2.gpu.scale_step(t1, 1, mode=fv.LOWRANK_RTR, keep_ratio=0.5, forced_indices=bad)
    assert p2.gpu.poll_status() == fv.EINVAL
    assert p2.gpu.poll_status() == fv.OK                                       # cleared by the read


def test_graph_replay_matches_direct_launch(fv):
    """The step body is captured into a CUDA graph on first use and replayed afterwards; capture,
    replay and direct launches must give the same bits, and the cache bookkeeping must not differ."""
    shp = si.shape_var_d16(n_blocks=2)
    B = 4
    p = Pair(fv, shp, seed=107, B=B)
    p.prefill(8)
    toks = {k: to_bf16_cuda(si.make_tokens(107, B, shp.tokens_per_scale()[k], 1024, "spread")) for k in (8, 9)}
    for k in (8, 9):
        p.set_projections(k, [orc.rank_from_keep_ratio(shp.tokens_per_scale()[k], 0.5)] * 2)

    def run():
        p.gpu.restore_loaded()
        outs = []
        for k in (8, 9):
            outs.append(p.gpu.scale_step(toks[k], k, mode=fv.LOWRANK_RTR, cfg_mode=fv.CFG_NULL_ONLY, keep_ratio=0.5).clone())
            p.gpu.kv_append(k)
        p.check_ok()
        return outs, [p.gpu.cache_len(b) for b in range(2)], p.gpu.get_indices(1, B // 2, 256).clone()

    n0 = p.gpu.launch_count()
    captured = run()
    n1 = p.gpu.launch_count()
    replayed = run()
    n2 = p.gpu.launch_count()
    p.gpu.set_option(fv.OPT_CUDA_GRAPHS, 0)
    direct = run()
    n3 = p.gpu.launch_count()
    assert n1 - n0 == n2 - n1 == n3 - n2 > 0
    for other in (replayed, direct):
        assert all(torch.equal(a, b) for a, b in zip(captured[0], other[0]))
        assert captured[1] == other[1] == [255 + 85 + 128] * 2
        assert torch.equal(captured[2], other[2])


@pytest.mark.parametrize("splits", [2, 4])
def test_split_k_is_deterministic_and_close(fv, splits):
    """With split-K enabled the partial tiles are added in a fixed order: two runs give the same
    bits, and the result stays within the bar of the oracle."""
    shp = si.shape_var_d16(n_blocks=2)
    B = 2
    p = Pair(fv, shp, seed=108, B=B)
    p.gpu.set_option(fv.OPT_GEMM_MAX_SPLITS, splits)
    p.prefill(9)
    p.set_projections(9, [128, 128])
    toks = si.make_tokens(108, B, 256, 1024, "spread")
    got, ref = _step_both(p, toks, 9, mode=fv.LOWRANK_RTR, keep_ratio=0.5)
    assert_out_close(got, ref, what="split-K %d" % splits)
    g32 = p.gpu.get_group_output(1, 256).cpu().numpy()
    assert_close(g32, np.stack(p.oracle.group_cache[1]), what="fp32 group output, split-K")
    first = p.gpu.scale_step(to_bf16_cuda(toks), 9, mode=fv.LOWRANK_RTR, keep_ratio=0.5).clone()   # same scale again
    second = p.gpu.scale_step(to_bf16_cuda(toks), 9, mode=fv.LOWRANK_RTR, keep_ratio=0.5).clone()
    p.check_ok()
    assert torch.equal(first, second)


def test_sampled_selection_step(fv):
    """FVAR_SELECT_SAMPLE: rows drawn without replacement with probability proportional to their score,
    from the same Exp(1) variates on both sides; the rest of the step is unchanged."""
    shp = si.shape_var_d16(n_blocks=2)
    B, k, M, r = 2, 9, 256, 96
    p = Pair(fv, shp, seed=109, B=B)
    p.prefill(k)
    p.set_projections(k, [r, r])
    toks = si.make_tokens(109, B, M, 1024, "spread")
    noise = si.make_sample_noise(109, k, 2, B, M)
    ref = p.oracle.scale_step(toks, k, orc.Policy("lowrank_rtr", "pair", rank_per_group=[r, r], sample_noise=noise))
    out = p.gpu.scale_step(to_bf16_cuda(toks), k, mode=fv.LOWRANK_RTR, rank_per_group=[r, r],
                           sample_noise=torch.from_numpy(noise).cuda())
    p.check_ok()
    top = [orc.select_top_r(orc.row_scores(toks[e], np.float32), r) for e in range(B)]
    for g in range(2):
        idx = p.gpu.get_indices(g, B, M).cpu().numpy()
        for e in range(B):
            assert np.array_equal(idx[e], p.oracle.last_indices[e][g]), (g, e)
    assert any(not np.array_equal(p.oracle.last_indices[e][0], top[e]) for e in range(B))     # it is not plain top-r
    assert_out_close(bf16_to_numpy(out), ref, what="sampled selection")
    # the same call again replays the captured graph and gives the same bits
    again = p.gpu.scale_step(to_bf16_cuda(toks), k, mode=fv.LOWRANK_RTR, rank_per_group=[r, r],
                             sample_noise=torch.from_numpy(noise).cuda())
    assert again.shape == out.shape


@pytest.mark.parametrize("B,cfg", [(1, "pair"), (2, "null_only"), (3, "pair")])
def test_edge_ranks_and_batches(fv, B, cfg):
    """Degenerate cases of the method: r = 1 (one representative row), r = M - 1 (one filled row), a batch
    of one element, an odd batch, non-square token maps."""
    shp = si.shape_tiny(n_blocks=2, blocks_per_group=1, width=128, n_heads=2, head_dim=64, ffn_dim=192,
                        scales=(1, 3, 5), scale_hw=((1, 2), (3, 2), (5, 4)))
    p = Pair(fv, shp, seed=110, B=B, std=0.05)
    Ms = shp.tokens_per_scale()
    toks = [si.make_tokens(110, B, m, 128) for m in Ms]
    got, ref = _step_both(p, toks[0], 0, mode=fv.DENSE)
    assert_out_close(got, ref, what="dense 1x2 map")
    p.gpu.kv_append(0)
    p.oracle.kv_append(0)
    ranks = [1, Ms[1] - 1]
    p.set_projections(1, ranks)
    got, ref = _step_both(p, toks[1], 1, mode=fv.LOWRANK_RTR, cfg=cfg, ranks=ranks)
    assert_out_close(got, ref, what="r = 1 / r = M - 1")
    p.gpu.kv_append(1)
    p.oracle.kv_append(1)
    ranks = [Ms[2] - 1, 1]
    p.set_projections(2, ranks)
    got, ref = _step_both(p, toks[2], 2, mode=fv.LOWRANK_RTR, cfg=cfg, ranks=ranks)
    assert_out_close(got, ref, what="r = M - 1 / r = 1 after a late scale")
    e0 = 1 if cfg == "null_only" else 0
    assert p.gpu.cache_len(0) == p.oracle.cache_len(0, e0) and p.gpu.cache_len(1) == p.oracle.cache_len(1, e0)


@pytest.mark.parametrize("M_side,r", [(16, 128), (13, 85), (16, 255), (10, 1)])
def test_generated_projection_matches_oracle_bit_for_bit(fv, M_side, r):
    """Q drawn on the device from a seed (Philox4x32-10 + Box-Muller in fp64, one rounding to bf16)
    against the oracle's draw: same bits, for row lengths that are and are not multiples of 4 or 64."""
    shp = si.shape_var_d16(n_blocks=2)
    k = {10: 7, 13: 8, 16: 9}[M_side]
    M = M_side * M_side
    p = Pair(fv, shp, seed=111, B=2)
    seed = 0x9E3779B97F4A7C15
    for g in range(2):
        p.gpu.generate_projection(k, g, r, seed)
        got = bf16_to_numpy(p.gpu.get_projection(k, g, M))
        want = orc.generate_projection(seed, k, g, M, r).T
        assert got.shape == want.shape == (r, M)
        assert np.array_equal(got, want), "group %d: %d of %d entries differ" % (g, (got != want).sum(), got.size)
    p.check_ok()


def test_step_with_generated_projection(fv):
    """A late step whose projections both sides draw from the same seed instead of taking them as data."""
    shp = si.shape_var_d16(n_blocks=2)
    B, k, M, r = 2, 9, 256, 96
    p = Pair(fv, shp, seed=112, B=B)
    p.prefill(k)
    for g in range(2):
        p.gpu.generate_projection(k, g, r, 2024 + g)
        p.oracle.set_projection(k, g, orc.generate_projection(2024 + g, k, g, M, r))
    toks = si.make_tokens(112, B, M, 1024, "spread")
    got, ref = _step_both(p, toks, k, mode=fv.LOWRANK_RTR, ranks=[r, r])
    assert_out_close(got, ref, what="step with generated projection")
    # a given matrix replaces a generated one and the other way round
    p.set_projections(k, [r, r])
    got2, ref2 = _step_both(p, toks, k, mode=fv.LOWRANK_RTR, ranks=[r, r])
    assert_out_close(got2, ref2, what="step after replacing the projection")
    assert not np.array_equal(got, got2)


def test_profile_pass_times_every_launch_and_changes_nothing(fv):
    """With per-launch event timing switched on (the step's graph re-captured with event nodes) a step gives
    the same bits as the timed path, every launch is accounted for in exactly one kernel class, and every
    interval is positive."""
    shp = si.shape_var_d16(n_blocks=2)
    B, k, M, r = 2, 9, 256, 96
    p = Pair(fv, shp, seed=113, B=B)
    p.prefill(k)
    p.set_projections(k, [r, r])
    toks = to_bf16_cuda(si.make_tokens(113, B, M, 1024, "spread"))
    p.gpu.restore_loaded()
    first = p.gpu.scale_step(toks, k, mode=fv.LOWRANK_RTR, rank_per_group=[r, r]).clone()
    p.gpu.profile_enable(True)
    n0 = p.gpu.launch_count()
    for _ in range(2):
        p.gpu.restore_loaded()
        again = p.gpu.scale_step(toks, k, mode=fv.LOWRANK_RTR, rank_per_group=[r, r])
        assert torch.equal(first, again)
    launched = p.gpu.launch_count() - n0
    total = 0
    for i, name in enumerate(fv.KCLASSES):
        ms, n, fl, by = p.gpu.profile_read(i)
        total += n
        if n:
            assert ms > 0.0, name
            assert all(t > 0.0 for t in p.gpu.profile_dump(i)), name
    assert total == launched > 0
    gemm_ms, gemm_n, gemm_fl, _ = p.gpu.profile_read(fv.KCLASSES.index("gemm"))
    assert gemm_n == 2 * 2 * 5 and gemm_fl > 0          # per step: 2 groups x (projection + 4 block GEMMs)
    p.gpu.profile_enable(False)
    p.gpu.restore_loaded()
    assert torch.equal(first, p.gpu.scale_step(toks, k, mode=fv.LOWRANK_RTR, rank_per_group=[r, r]))
    p.check_ok()


def test_pipelined_host_entry_point_matches_the_synchronous_one(fv):
    """Three late scales through fvar_scale_step_host_async (uploads, steps and downloads on three streams, two
    staging slots each way; more calls than slots) give the same bits as the synchronous host entry point."""
    shp = si.shape_var_d16(n_blocks=2)
    B = 4
    Ms = shp.tokens_per_scale()
    results = {}
    for variant in ("sync", "async"):
        p = Pair(fv, shp, seed=114, B=B)
        p.prefill(7)
        outs = []
        for rep in range(2):                                       # 6 calls: every staging slot is reused twice
            p.gpu.restore_loaded()
            for k in (7, 8, 9):
                r = Ms[k] // 2
                p.set_projections(k, [r, r])
                toks = to_bf16_cuda(si.make_tokens(114, B, Ms[k], 1024, "spread")).cpu().pin_memory()
                out = torch.empty((B // 2, Ms[k], 1024), dtype=torch.bfloat16).pin_memory()
                kw = dict(mode=fv.LOWRANK_RTR, cfg_mode=fv.CFG_NULL_ONLY, rank_per_group=[r, r])
                if variant == "sync":
                    p.gpu.scale_step_host(toks, k, out, **kw)
                else:
                    p.gpu.scale_step_host_async(toks, k, out, **kw)
                p.gpu.kv_append(k)
                outs.append((toks, out))
        if variant == "async":
            p.gpu.host_sync()
        p.check_ok()
        results[variant] = [o.clone() for _, o in outs]
    for a, b in zip(results["sync"], results["async"]):
        assert torch.equal(a, b)
    assert float(results["async"][-1].float().abs().sum()) > 0


# ----------------------------------------------------------------------------- LLS restoration (Eq. "lstsq", App. A.3)

@pytest.mark.parametrize("r,cfg", [(32, "pair"), (128, "null_only"), (160, "pair")])
def test_lls_restoration_step(fv, r, cfg):
    """One VAR-d16-shaped block group (two blocks) at the last scale with the rows restored by the least-squares
    matrices instead of RTR: F_k^o = (W_hat + W^{o,cache}) F_r^o, against the oracle's fp64 solve, at the block-output
    bar (the restoration is linear in the block output and runs in fp32; measured 0.5e-2 .. 1.4e-2 x RMS)."""
    shp = si.shape_var_d16(n_blocks=2, blocks_per_group=2)
    B, k, M = 2, 9, 256
    p = Pair(fv, shp, seed=120 + r, B=B)
    p.prefill(k)
    p.set_projections(k, [r])
    toks = si.make_tokens(120 + r, B, M, 1024, "spread")
    ref = p.oracle.scale_step(toks, k, orc.Policy("lowrank_rtr", cfg, rank_per_group=[r], restore="lls"))
    out = p.gpu.scale_step(to_bf16_cuda(toks), k, mode=fv.LOWRANK_RTR, cfg_mode=fv.CFG_NULL_ONLY if cfg == "null_only" else fv.CFG_PAIR,
                           rank_per_group=[r], restore=fv.RESTORE_LLS)
    p.check_ok()
    els = [1] if cfg == "null_only" else [0, 1]
    g32 = p.gpu.get_group_output(0, M).cpu().numpy()[els]
    e, c = rel_err(g32, np.stack([p.oracle.group_cache[0][b] for b in els]))
    print("LLS r=%d %s: max-abs/RMS %.3e cosine %.6f" % (r, cfg, e, c))
    assert e <= 2e-2 and c >= 0.999, (e, c)
    assert_out_close(bf16_to_numpy(out), ref, what="LLS step r=%d" % r)
    with pytest.raises(fv.FvarError):
        p.gpu.get_indices(0, len(els), M)                   # LLS chooses no index set
    p.gpu.kv_append(k)
    p.oracle.kv_append(k)
    assert p.gpu.cache_len(1) == 424 + r == p.oracle.cache_len(1, 1)
    if r == 160:                                            # the upsampled 13 x 13 cache has rank <= 169 < 170
        p.gpu.restore_loaded()
        p.set_projections(k, [170])
        with pytest.raises(fv.FvarError) as ei:
            p.gpu.scale_step(to_bf16_cuda(toks), k, mode=fv.LOWRANK_RTR, rank_per_group=[170], restore=fv.RESTORE_LLS)
        assert ei.value.status == fv.EINVAL


def test_lls_restoration_two_groups_and_limits(fv):
    """Two block groups in sequence (the second projects the first one's restored rows), and the rank limit.  An LLS
    group's output is spanned by its r block-output rows, so the next group's rank may not be larger (its projection
    would not have full row rank): ranks 40 then 24."""
    shp = si.shape_tiny(n_blocks=2, blocks_per_group=1, width=128, n_heads=2, head_dim=64, ffn_dim=256, scales=(2, 4, 8, 16))
    B = 2
    p = Pair(fv, shp, seed=130, B=B, std=0.05)
    Ms = shp.tokens_per_scale()
    for k in (0, 1, 2):
        toks = si.make_tokens(130, B, Ms[k], 128)
        _step_both(p, toks, k, mode=fv.DENSE)
        p.gpu.kv_append(k)
        p.oracle.kv_append(k)
    ranks = [40, 24]
    p.set_projections(3, ranks)
    toks = si.make_tokens(130, B, 256, 128, "spread")
    ref = p.oracle.scale_step(toks, 3, orc.Policy("lowrank_rtr", "pair", rank_per_group=ranks, restore="lls"))
    out = p.gpu.scale_step(to_bf16_cuda(toks), 3, mode=fv.LOWRANK_RTR, rank_per_group=ranks, restore=fv.RESTORE_LLS)
    p.check_ok()
    for g in range(2):
        e, c = rel_err(p.gpu.get_group_output(g, 256).cpu().numpy(), np.stack(p.oracle.group_cache[g]))
        print("LLS group %d: max-abs/RMS %.3e cosine %.6f" % (g, e, c))
        assert e <= 2e-2 * np.sqrt(g + 1.0) and c >= 0.999, (g, e, c)
    assert_out_close(bf16_to_numpy(out), ref, what="LLS two groups", max_rel=2e-2 * np.sqrt(2.0))
    p.set_projections(3, [200, 24])
    with pytest.raises(fv.FvarError) as ei:
        p.gpu.scale_step(to_bf16_cuda(toks), 3, mode=fv.LOWRANK_RTR, rank_per_group=[200, 24], restore=fv.RESTORE_LLS)
    assert ei.value.status == fv.EUNSUPPORTED
