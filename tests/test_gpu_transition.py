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
