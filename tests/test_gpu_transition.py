"""Parity of the transition between two scale steps (nearest codeword on the tensor cores, Up-accumulate,
area Down; Algorithm 1, Eq. "var_upf", Eq. "var_downf") against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import fvar_oracle as orc
from helpers import bf16_to_numpy, to_bf16_cuda, weights_to_cuda

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fv():
    from paper_2512_16483_b200 import binding
    binding.load_library()
    return binding


def _ctx(fv, shp, B, seed=300):
    w = si.make_weights(seed, shp)
    return fv.Fvar(weights_to_cuda(w), blocks_per_group=shp.blocks_per_group, n_heads=shp.n_heads, head_dim=shp.head_dim,
                   ffn_dim=shp.ffn_dim, scale_hw=shp.hw(), max_batch=B, ctx_len=shp.ctx_len, ctx_width=shp.ctx_width,
                   ln_eps=shp.ln_eps)


def _check_codes(got, fo, Z, what):
    """Codes must equal the oracle's wherever the oracle's own fp64 margin between the two candidates exceeds
    what fp32 accumulation order can move (the decision is taken on fp32 scores on both sides); a differing
    code must still be a maximiser within that margin."""
    want = orc.nearest_codeword(fo, Z)
    diff = np.nonzero(got != want)[0]
    Z64 = Z.astype(np.float64)
    hn = 0.5 * (Z64 * Z64).sum(axis=1)
    for i in diff:
        s = Z64 @ fo[i].astype(np.float64) - hn
        tol = 4e-6 * (np.abs(Z64[[got[i], want[i]]]) @ np.abs(fo[i].astype(np.float64))).max() + 1e-6
        assert s[got[i]] >= s.max() - tol, "%s: row %d picked code %d (score %.6f), best %d (%.6f)" % (
            what, i, got[i], s[got[i]], want[i], s.max())
    return len(diff)


@pytest.mark.parametrize("V,M_side,B,noise", [(4096, 16, 2, 0.05), (4096, 13, 3, 1.0), (1000, 16, 1, 1.0), (37, 10, 2, 0.05),
                                             (8192, 16, 8, 0.5)])
def test_nearest_codeword_on_the_tensor_cores(fv, V, M_side, B, noise):
    shp = si.shape_var_d16(n_blocks=1)
    k = {10: 7, 13: 8, 16: 9}[M_side]
    M, C = M_side * M_side, shp.width
    g = _ctx(fv, shp, B)
    Z = si.make_codebook(301, V, C)
    g.set_codebook(to_bf16_cuda(Z))
    # the transition wants the scales in order: run the earlier ones on throw-away data
    for kk in range(k):
        Mk = shp.tokens_per_scale()[kk]
        g.scale_transition(to_bf16_cuda(si.make_step_outputs(302, kk, B, Mk, Z, 0.05)), kk, shp.tokens_per_scale()[kk + 1])
    fo = si.make_step_outputs(302, k, B, M, Z, noise)
    codes, _ = g.scale_transition(to_bf16_cuda(fo), k, shp.tokens_per_scale()[k + 1] if k + 1 < len(shp.hw()) else None)
    assert g.poll_status() == fv.OK
    got = codes.cpu().numpy()
    flips = sum(_check_codes(got[b], fo[b], Z, "b=%d" % b) for b in range(B))
    if noise <= 0.1:
        assert flips == 0                       # well-separated rows: bit-exact codes
    assert flips <= max(1, B * M // 200)


@pytest.mark.parametrize("shape", ["tiny", "d16"])
def test_transition_chain_matches_oracle(fv, shape):
    """Every scale of a schedule in order: codes, the accumulated map F_k and the next step's tokens."""
    if shape == "tiny":
        shp, V, B = si.shape_tiny(n_blocks=1), 64, 3
    else:
        shp, V, B = si.shape_var_d16(n_blocks=1), 4096, 2
    g = _ctx(fv, shp, B)
    C, Ms, hw = shp.width, shp.tokens_per_scale(), shp.hw()
    Z = si.make_codebook(303, V, C)
    g.set_codebook(to_bf16_cuda(Z))
    F_ref = [np.zeros((Ms[-1], C)) for _ in range(B)]
    for k in range(len(shp.hw())):
        fo = si.make_step_outputs(304, k, B, Ms[k], Z, 0.05)
        last = k == len(shp.hw()) - 1
        codes, nxt = g.scale_transition(to_bf16_cuda(fo), k, None if last else Ms[k + 1])
        assert g.poll_status() == fv.OK
        got_F = g.get_feature(B, Ms[-1], C).cpu().numpy().astype(np.float64)
        for b in range(B):
            c_ref, F_ref[b], n_ref = orc.scale_transition(F_ref[b], fo[b], Z, hw[k], hw[-1], None if last else hw[k + 1])
            assert np.array_equal(codes[b].cpu().numpy(), c_ref), (k, b)
            # fp32 interpolation weights and accumulation over at most n_scales terms of magnitude ~|Z|
            np.testing.assert_allclose(got_F[b], F_ref[b], rtol=0, atol=2e-5 * (k + 1) * np.abs(Z).max())
            if not last:
                got_n = bf16_to_numpy(nxt[b])
                np.testing.assert_allclose(got_n, n_ref, rtol=2 ** -8, atol=1e-5 * np.abs(Z).max())
        assert (nxt is None) == last


def test_transition_state_and_argument_errors(fv):
    shp = si.shape_tiny(n_blocks=1)
    g = _ctx(fv, shp, 2)
    C, Ms = shp.width, shp.tokens_per_scale()
    Z = si.make_codebook(305, 32, C)
    fo0 = to_bf16_cuda(si.make_step_outputs(306, 0, 2, Ms[0], Z, 0.05))
    with pytest.raises(fv.FvarError):
        g.scale_transition(fo0, 0, Ms[1])                        # no codebook yet
    g.set_codebook(to_bf16_cuda(Z))
    fo1 = to_bf16_cuda(si.make_step_outputs(306, 1, 2, Ms[1], Z, 0.05))
    with pytest.raises(fv.FvarError):
        g.scale_transition(fo1, 1, Ms[2])                        # scale 1 before scale 0
    codes_a, none = g.scale_transition(fo0, 0, None)             # allowed: the caller stops here (remaining steps skipped)
    assert none is None
    codes_b, _ = g.scale_transition(fo0, 0, Ms[1])               # scale 0 starts a new accumulation
    assert torch.equal(codes_a, codes_b)
    g.scale_transition(fo1, 1, Ms[2])
    with pytest.raises(fv.FvarError):
        g.scale_transition(fo1[:1].contiguous(), 2, Ms[3] if len(shp.hw()) > 3 else None)   # batch changed midway
    assert g.poll_status() == fv.OK


@pytest.mark.parametrize("guidance", [0.0, 1.0, 3.0])
def test_cfg_combine(fv, guidance):
    rng = np.random.default_rng(31)
    x = si.normal_bf16(rng, (6, 100, 128))
    got = bf16_to_numpy(fv.fvar_cfg_combine(to_bf16_cuda(x), guidance))
    ref = np.stack([orc.cfg_combine(x[2 * p], x[2 * p + 1], guidance) for p in range(3)])
    # fp32 arithmetic on bf16 inputs, one rounding to bf16
    np.testing.assert_allclose(got, ref, rtol=2 ** -8, atol=1e-6)
    if guidance == 0.0:
        assert np.array_equal(got, x[1::2])                      # CFG = 0: the null-prompt branch, bit for bit


def test_transition_at_the_infinity_shape(fv):
    """The last two scales of the Infinity-2B-shaped schedule (48 x 48 and 64 x 64 tokens, C = 2048) with the 8192
    codewords the closed-loop benchmark uses: every code, the whole accumulated map and the next tokens."""
    shp = si.ModelShape(n_blocks=1, blocks_per_group=1, width=2048, n_heads=16, head_dim=128, ffn_dim=2048,
                        scales=(48, 64))
    B, V = 1, 8192
    g = _ctx(fv, shp, B, seed=307)
    C, Ms, hw = shp.width, shp.tokens_per_scale(), shp.hw()
    Z = si.make_codebook(308, V, C)
    g.set_codebook(to_bf16_cuda(Z))
    F_ref = np.zeros((Ms[-1], C))
    for k in range(2):
        fo = si.make_step_outputs(309, k, B, Ms[k], Z, 0.05)
        codes, nxt = g.scale_transition(to_bf16_cuda(fo), k, None if k == 1 else Ms[1])
        assert g.poll_status() == fv.OK
        c_ref, F_ref, n_ref = orc.scale_transition(F_ref, fo[0], Z, hw[k], hw[-1], None if k == 1 else hw[1])
        assert np.array_equal(codes[0].cpu().numpy(), c_ref)
        got_F = g.get_feature(B, Ms[-1], C)[0].cpu().numpy().astype(np.float64)
        np.testing.assert_allclose(got_F, F_ref, rtol=0, atol=2e-5 * (k + 1) * np.abs(Z).max())
        if k == 0:
            np.testing.assert_allclose(bf16_to_numpy(nxt[0]), n_ref, rtol=2 ** -8, atol=1e-5 * np.abs(Z).max())


def test_closed_generation_loop_matches_oracle(fv):
    """Algorithm 1 as a closed loop on a tiny stack, the library and the oracle each feeding themselves: a start token,
    then for every scale step -> (CFG combination of the two branches) -> R_k = Q(F_k^o), F_k = F_{k-1} + Up(R_k),
    next tokens = Down(F_k) -> next step.  Scales 0 and 1 run densely with both branches (guidance 3), scales 2 and 3
    under RP + RTR on the null-prompt branch alone (teacher-forced index sets), scale 4 is skipped (Sec. 4.1: alpha = 0),
    so the map accumulated after scale 3 is the result.  Both sides see the same interface types: the step returns
    bf16, the combination returns bf16, the next tokens are bf16.  Codes must agree at every scale; F_k then agrees to
    fp32 accumulation accuracy and the next tokens to one bf16 rounding."""
    from test_gpu_step import Pair
    shp = si.shape_tiny(n_blocks=4, blocks_per_group=2, width=128, n_heads=2, head_dim=64, ffn_dim=256, scales=(1, 2, 3, 5, 8))
    B, V, guidance = 2, 48, 3.0
    p = Pair(fv, shp, seed=77, B=B, std=0.05)
    C, Ms, hw = shp.width, shp.tokens_per_scale(), shp.hw()
    Z = si.make_codebook(77, V, C)
    p.gpu.set_codebook(to_bf16_cuda(Z))
    ranks = {2: [4, 5], 3: [10, 12]}
    for k, rk in ranks.items():
        p.set_projections(k, rk)
    bf = lambda a: si.round_to_bf16(np.asarray(a, np.float32)).astype(np.float64)
    start = si.make_tokens(77, 1, 1, C)
    tok_o = np.concatenate([start, start], axis=0)                      # both branches of the pair start alike
    tok_g = to_bf16_cuda(tok_o)
    F_o = np.zeros((Ms[-1], C))
    for k in range(4):
        late, more = k in ranks, k < 3
        if late:
            pol = orc.Policy("lowrank_rtr", "null_only", rank_per_group=ranks[k])
            out_o = p.oracle.scale_step(tok_o, k, pol)
            out_g = p.gpu.scale_step(tok_g, k, mode=fv.LOWRANK_RTR, cfg_mode=fv.CFG_NULL_ONLY, rank_per_group=ranks[k],
                                     forced_indices=p.forced_tensor(ranks[k], 1))
            fo_o, fo_g = bf(out_o[0]), out_g                             # CFG = 0: the null-prompt branch is the output
        else:
            out_o = p.oracle.scale_step(tok_o, k, orc.Policy("dense", "pair"))
            out_g = p.gpu.scale_step(tok_g, k, mode=fv.DENSE)
            fo_o = bf(orc.cfg_combine(bf(out_o[0]), bf(out_o[1]), guidance))
            fo_g = fv.fvar_cfg_combine(out_g, guidance)
        p.check_ok()
        p.gpu.kv_append(k)
        p.oracle.kv_append(k)
        codes_g, nxt_g = p.gpu.scale_transition(fo_g, k, Ms[k + 1] if more else None, pairs=True)
        codes_o, F_o, nxt_o = orc.scale_transition(F_o, fo_o, Z, hw[k], hw[-1], hw[k + 1] if more else None)
        assert np.array_equal(codes_g.cpu().numpy()[0], codes_o), (k, codes_g.cpu().numpy()[0], codes_o)
        got_F = p.gpu.get_feature(1, Ms[-1], C).cpu().numpy()[0].astype(np.float64)
        np.testing.assert_allclose(got_F, F_o, rtol=0, atol=2e-5 * (k + 1) * np.abs(Z).max())
        if more:
            assert nxt_g.shape == (2, Ms[k + 1], C) and torch.equal(nxt_g[0], nxt_g[1])       # written for both branches
            np.testing.assert_allclose(bf16_to_numpy(nxt_g[0]), nxt_o, rtol=2 ** -8, atol=1e-5 * np.abs(Z).max())
            tok_o = np.stack([bf(nxt_o), bf(nxt_o)])
            tok_g = nxt_g
        else:
            assert nxt_g is None
    # the skipped scale: nothing is enqueued, nothing staged, the accumulated map stands as the result
    assert p.gpu.scale_step(tok_g, 4, mode=fv.SKIP) is None
    assert p.gpu.poll_status() == fv.OK
