"""Parity of the individual CUDA kernels (through the C ABI) against the CPU oracle, element by
element, on seeded inputs that span several tiles and a ragged tail."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import fvar_oracle as orc
from helpers import assert_close, assert_out_close, bf16_to_numpy, to_bf16_cuda

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fv():
    from paper_2512_16483_b200 import binding
    binding.load_library()
    return binding


def _poll(fv):
    assert fv.kernel_poll_status() == fv.OK


# ----------------------------------------------------------------------------- score

@pytest.mark.parametrize("B,M,C", [(2, 256, 1024), (3, 169, 1920), (1, 4096, 2048), (2, 1, 64), (1, 7, 4)])
def test_row_scores(fv, B, M, C):
    x = si.make_tokens(31, B, M, C, "spread" if M > 64 else "normal")
    got = fv.fvar_row_scores(torch.from_numpy(x).cuda()).cpu().numpy()
    ref = orc.row_scores(x, np.float64)
    np.testing.assert_allclose(got, ref, rtol=2e-6)       # fp32 sum of C squares, pairwise-ish order


# ----------------------------------------------------------------------------- selection (bit-exact)

def _check_select(fv, scores: np.ndarray, r: int):
    B, M = scores.shape
    idx, inv = fv.fvar_select_topr(torch.from_numpy(scores).cuda(), r)
    idx, inv = idx.cpu().numpy(), inv.cpu().numpy()
    for b in range(B):
        ref = orc.select_top_r(scores[b], r)
        assert np.array_equal(idx[b], ref), (b, M, r)
        exp_inv = np.full(M, -1, np.int32)
        exp_inv[ref] = np.arange(r, dtype=np.int32)
        assert np.array_equal(inv[b], exp_inv)


@pytest.mark.parametrize("M", [1, 2, 33, 100, 169, 256, 1024, 1600, 4096, 5000])
def test_select_random_scores(fv, M):
    rng = np.random.default_rng(M)
    s = (rng.standard_normal((3, M)) ** 2).astype(np.float32) * 1000
    for r in sorted({1, max(1, M // 4), max(1, M // 2), M - 1 if M > 1 else 1, M}):
        _check_select(fv, s, r)


def test_select_ties_nan_inf_zero(fv):
    rng = np.random.default_rng(5)
    M = 1500
    s = rng.integers(0, 5, size=(4, M)).astype(np.float32)          # heavy ties: index order decides
    s[0, 17] = np.nan
    s[0, 900] = np.inf
    s[1, :] = 3.0                                                    # all equal
    s[2, ::7] = -0.0
    s[3, 5] = np.nan
    s[3, 6] = np.nan
    for r in (1, 2, 100, 750, 1499, 1500):
        _check_select(fv, s, r)
    # scores of real rows, chi-square concentrated (closely spaced keys)
    x = si.make_tokens(6, 2, 256, 1024)
    sc = orc.row_scores(x, np.float32).astype(np.float32)
    for r in (32, 128):
        _check_select(fv, sc, r)


# ----------------------------------------------------------------------------- LN + modulate

@pytest.mark.parametrize("B,n,C", [(2, 128, 1024), (3, 85, 1920), (1, 16, 2048), (2, 5, 64)])
def test_ln_modulate(fv, B, n, C):
    rng = np.random.default_rng(7)
    x = (rng.standard_normal((B, n, C)) * 1.7 + 0.3).astype(np.float32)
    shift = rng.standard_normal((B, C)).astype(np.float32) * 0.5
    scale = rng.standard_normal((B, C)).astype(np.float32) * 0.5
    got = bf16_to_numpy(fv.fvar_ln_modulate(torch.from_numpy(x).cuda(), torch.from_numpy(shift).cuda(),
                                           torch.from_numpy(scale).cuda(), 1e-6))
    ref = np.stack([orc.modulate(x[b].astype(np.float64), shift[b], scale[b], 1e-6) for b in range(B)])
    # bf16 output: half an ulp is 2^-9 relative
    np.testing.assert_allclose(got, ref, rtol=2 ** -8, atol=2e-3)


# ----------------------------------------------------------------------------- GEMM

@pytest.mark.parametrize("R,N,K", [(128, 64, 64), (300, 200, 136), (1000, 1024, 1024), (130, 3072, 1024),
                                   (2048, 4096, 1024), (64, 1024, 4096), (1, 8, 8), (257, 96, 4000)])
@pytest.mark.parametrize("bias", [False, True])
def test_gemm_bf16(fv, R, N, K, bias):
    rng = np.random.default_rng(R + N + K)
    A = si.normal_bf16(rng, (R, K))
    W = si.normal_bf16(rng, (N, K), 0.05)
    b = si.normal_bf16(rng, (N,)) if bias else None
    got = fv.fvar_gemm_bf16(to_bf16_cuda(A), to_bf16_cuda(W), to_bf16_cuda(b) if bias else None).cpu().numpy()
    _poll(fv)
    ref = A.astype(np.float64) @ W.astype(np.float64).T + (b.astype(np.float64) if bias else 0.0)
    # exact bf16 products, fp32 accumulation over K terms
    tol = 1e-5 * (np.abs(A).astype(np.float64) @ np.abs(W).astype(np.float64).T).max() + 1e-6
    np.testing.assert_allclose(got, ref, atol=tol, rtol=0)


# Every launch form and tile width against the same fp64 product: single CTAs (64 / 128 / 256 columns)
# and CTA pairs (256-row tiles of 128 / 256 columns), on shapes with ragged row, column and K edges, an
# odd number of 128-row tiles (the second CTA of the last pair has no rows) and more tiles than CTAs.
@pytest.mark.parametrize("R,N,K", [(256, 256, 64), (129, 128, 72), (300, 200, 136), (641, 1000, 520),
                                   (1024, 3072, 1024), (3000, 4096, 256), (4500, 512, 2048)])
@pytest.mark.parametrize("form,block_n", [("single", 64), ("single", 128), ("single", 256), ("pair", 128), ("pair", 256)])
def test_gemm_bf16_every_form(fv, R, N, K, form, block_n):
    rng = np.random.default_rng(7 * R + N + K)
    A = si.normal_bf16(rng, (R, K))
    W = si.normal_bf16(rng, (N, K), 0.05)
    b = si.normal_bf16(rng, (N,))
    f = fv.GEMM_PAIR if form == "pair" else fv.GEMM_SINGLE
    got = fv.fvar_gemm_bf16_form(to_bf16_cuda(A), to_bf16_cuda(W), to_bf16_cuda(b), f, block_n).cpu().numpy()
    _poll(fv)
    ref = A.astype(np.float64) @ W.astype(np.float64).T + b.astype(np.float64)
    tol = 1e-5 * (np.abs(A).astype(np.float64) @ np.abs(W).astype(np.float64).T).max() + 1e-6
    np.testing.assert_allclose(got, ref, atol=tol, rtol=0)


# The weight-streaming form (few rows; the weights are the M side of the MMA and the K range of a 128-feature tile is
# spread over a cluster of S CTAs that reduce through distributed shared memory): one and two column chunks (R <= 256,
# R > 256), every cluster size, ragged rows, a ragged last feature tile, a ragged last K block, more K ranges than
# some sizes divide evenly, and the shapes of the Infinity-2B-shaped late steps.
@pytest.mark.parametrize("R,N,K", [(1, 128, 64), (16, 256, 512), (17, 200, 136), (170, 2048, 2048), (256, 384, 1024),
                                   (257, 128, 520), (410, 1024, 2048), (512, 256, 256), (50, 6144, 2048), (111, 2048, 8192),
                                   (336, 8192, 2048)])
@pytest.mark.parametrize("splits", [0, 1, 2, 3, 4, 5, 6, 7, 8])
def test_gemm_bf16_weight_streaming_form(fv, R, N, K, splits):
    rng = np.random.default_rng(11 * R + N + K)
    A = si.normal_bf16(rng, (R, K))
    W = si.normal_bf16(rng, (N, K), 0.05)
    b = si.normal_bf16(rng, (N,))
    num_kb = -(-K // 64)
    if splits and -(-num_kb // -(-num_kb // splits)) != splits:
        with pytest.raises(fv.FvarError):          # a K range would be empty: refused, not launched
            fv.fvar_gemm_bf16_form(to_bf16_cuda(A), to_bf16_cuda(W), to_bf16_cuda(b), fv.GEMM_SKINNY, splits)
        return
    got = fv.fvar_gemm_bf16_form(to_bf16_cuda(A), to_bf16_cuda(W), to_bf16_cuda(b), fv.GEMM_SKINNY, splits).cpu().numpy()
    _poll(fv)
    ref = A.astype(np.float64) @ W.astype(np.float64).T + b.astype(np.float64)
    tol = 1e-5 * (np.abs(A).astype(np.float64) @ np.abs(W).astype(np.float64).T).max() + 1e-6
    np.testing.assert_allclose(got, ref, atol=tol, rtol=0)


# The same K split over a cluster with 128 x 128 output tiles (rows on the M side): ragged rows, features and K, one to
# four row tiles, every cluster size.
@pytest.mark.parametrize("R,N,K", [(1, 128, 64), (130, 200, 136), (336, 2048, 2048), (257, 384, 520), (512, 256, 1024),
                                   (410, 2048, 8192), (700, 128, 256)])
@pytest.mark.parametrize("splits", [0, 1, 2, 3, 4, 6, 8])
def test_gemm_bf16_cluster_split_tiles(fv, R, N, K, splits):
    rng = np.random.default_rng(13 * R + N + K)
    A = si.normal_bf16(rng, (R, K))
    W = si.normal_bf16(rng, (N, K), 0.05)
    b = si.normal_bf16(rng, (N,))
    num_kb = -(-K // 64)
    if splits and -(-num_kb // -(-num_kb // splits)) != splits:
        with pytest.raises(fv.FvarError):
            fv.fvar_gemm_bf16_form(to_bf16_cuda(A), to_bf16_cuda(W), to_bf16_cuda(b), fv.GEMM_KSPLIT, splits)
        return
    got = fv.fvar_gemm_bf16_form(to_bf16_cuda(A), to_bf16_cuda(W), to_bf16_cuda(b), fv.GEMM_KSPLIT, splits).cpu().numpy()
    _poll(fv)
    ref = A.astype(np.float64) @ W.astype(np.float64).T + b.astype(np.float64)
    tol = 1e-5 * (np.abs(A).astype(np.float64) @ np.abs(W).astype(np.float64).T).max() + 1e-6
    np.testing.assert_allclose(got, ref, atol=tol, rtol=0)


@pytest.mark.parametrize("R,N,K", [(128, 64, 64), (300, 200, 136), (1000, 1024, 512), (130, 1920, 344), (64, 2048, 8192)])
@pytest.mark.parametrize("block_n", [0, 64, 128, 256])
def test_gemm_bf16_second_operand_transposed(fv, R, N, K, block_n):
    """out = A Wt with Wt stored [K][N]: the tensor core reads it as an MN-major operand (no transpose in memory)."""
    rng = np.random.default_rng(R + N + K)
    A = si.normal_bf16(rng, (R, K))
    Wt = si.normal_bf16(rng, (K, N), 0.05)
    b = si.normal_bf16(rng, (N,))
    got = fv.fvar_gemm_bf16_wt(to_bf16_cuda(A), to_bf16_cuda(Wt), to_bf16_cuda(b), block_n).cpu().numpy()
    _poll(fv)
    ref = A.astype(np.float64) @ Wt.astype(np.float64) + b.astype(np.float64)
    tol = 1e-5 * (np.abs(A).astype(np.float64) @ np.abs(Wt).astype(np.float64)).max() + 1e-6
    np.testing.assert_allclose(got, ref, atol=tol, rtol=0)


def test_gemm_form_rejects_what_the_problem_does_not_allow(fv):
    A = to_bf16_cuda(np.zeros((128, 64), np.float32))
    W = to_bf16_cuda(np.zeros((128, 64), np.float32))
    with pytest.raises(fv.FvarError):
        fv.fvar_gemm_bf16_form(A, W, None, fv.GEMM_PAIR, 128)       # a single row tile has no partner
    A2 = to_bf16_cuda(np.zeros((256, 64), np.float32))
    with pytest.raises(fv.FvarError):
        fv.fvar_gemm_bf16_form(A2, W, None, fv.GEMM_PAIR, 64)       # pairs come 128 or 256 columns wide
    with pytest.raises(fv.FvarError):
        fv.fvar_gemm_bf16_form(A2, W, None, fv.GEMM_SINGLE, 96)


# ----------------------------------------------------------------------------- attention

def _cache_layout(K, V, H, D, L_cap):
    """K, V [B][L][H*D] -> K cache [B][H][L_cap][D], V^T cache [B][H][D][L_cap] (zero padded)."""
    B, L, _ = K.shape
    Kc = np.zeros((B, H, L_cap, D), np.float32)
    Vt = np.zeros((B, H, D, L_cap), np.float32)
    Kc[:, :, :L] = K.reshape(B, L, H, D).transpose(0, 2, 1, 3)
    Vt[:, :, :, :L] = V.reshape(B, L, H, D).transpose(0, 2, 3, 1)
    return Kc, Vt


# The last five shapes have few (element, head, query tile) CTAs over a long cache, so the key range is split over a
# cluster (2, 4 and 8 ranges; one and two query tiles; a ragged last range; a single query row).
@pytest.mark.parametrize("B,H,D,r,L,L_cap", [(2, 16, 64, 256, 680, 768), (1, 4, 128, 170, 1000, 1024),
                                             (2, 2, 64, 32, 456, 768), (1, 2, 128, 300, 129, 136),
                                             (1, 1, 64, 1, 1, 8), (2, 3, 64, 130, 128, 128),
                                             (1, 2, 64, 128, 2000, 2048), (1, 16, 128, 16, 6441, 6528),
                                             (1, 16, 128, 170, 6595, 6656), (2, 4, 64, 300, 3000, 3072),
                                             (1, 3, 128, 1, 1100, 1104), (1, 5, 64, 77, 2500, 2560)])
def test_attention(fv, B, H, D, r, L, L_cap):
    rng = np.random.default_rng(B * 1000 + r + L)
    C = H * D
    q = si.normal_bf16(rng, (B, r, C))
    K = si.normal_bf16(rng, (B, L, C))
    V = si.normal_bf16(rng, (B, L, C))
    Kc, Vt = _cache_layout(K, V, H, D, L_cap)
    got = bf16_to_numpy(fv.fvar_attention(to_bf16_cuda(q), to_bf16_cuda(Kc), to_bf16_cuda(Vt), L))
    _poll(fv)
    ref = np.stack([orc.attention(q[b].astype(np.float64), K[b].astype(np.float64), V[b].astype(np.float64), H)
                    for b in range(B)])
    assert_out_close(got, ref, what="attention")      # bf16 result: the bar plus the rounding of the output
    assert_close(got, ref, max_rel=1.0, min_cos=0.9995, what="attention cosine")


def test_attention_scaled_down_scores_uniform(fv):
    """Zero queries: uniform softmax, output = mean of the values (masking of keys >= L must hold
    even when stale rows beyond L are large)."""
    B, H, D, r, L, L_cap = 1, 2, 64, 64, 200, 256
    rng = np.random.default_rng(3)
    C = H * D
    V = si.normal_bf16(rng, (B, L, C))
    K = si.normal_bf16(rng, (B, L, C))
    Kc, Vt = _cache_layout(K, V, H, D, L_cap)
    Kc[:, :, L:] = 50.0                                   # stale rows past L: must be masked
    Vt[:, :, :, L:] = 1000.0
    q = np.zeros((B, r, C), np.float32)
    got = bf16_to_numpy(fv.fvar_attention(to_bf16_cuda(q), to_bf16_cuda(Kc), to_bf16_cuda(Vt), L))
    _poll(fv)
    ref = np.broadcast_to(V.astype(np.float64).mean(axis=1, keepdims=True), (B, r, C))
    np.testing.assert_allclose(got, ref, atol=2e-3, rtol=2 ** -7)


# ----------------------------------------------------------------------------- restoration fill

@pytest.mark.parametrize("hw_in,hw_out,C", [((13, 13), (16, 16), 1024), ((10, 10), (13, 13), 64), ((4, 6), (5, 9), 128),
                                            ((16, 16), (16, 16), 256), ((1, 1), (2, 2), 64)])
def test_rtr_fill(fv, hw_in, hw_out, C):
    rng = np.random.default_rng(9)
    B = 2
    M0, M1 = hw_in[0] * hw_in[1], hw_out[0] * hw_out[1]
    prev = rng.standard_normal((B, M0, C)).astype(np.float32)
    r = max(1, M1 // 3)
    inv = np.full((B, M1), -1, np.int32)
    for b in range(B):
        sel = np.sort(rng.choice(M1, r, replace=False))
        inv[b, sel] = np.arange(r)
    sentinel = np.float32(-777.0)
    out = torch.full((B, M1, C), float(sentinel), dtype=torch.float32, device="cuda")
    fv.fvar_rtr_fill(torch.from_numpy(prev).cuda(), hw_in, hw_out, torch.from_numpy(inv).cuda(), out)
    got = out.cpu().numpy()
    for b in range(B):
        up = orc.upsample_bilinear(prev[b].astype(np.float64), hw_in, hw_out)
        keep = inv[b] >= 0
        assert np.all(got[b][keep] == sentinel)           # representative rows are not touched
        np.testing.assert_allclose(got[b][~keep], up[~keep], atol=2e-5, rtol=1e-5)
    out2 = torch.empty((B, M1, C), dtype=torch.float32, device="cuda")
    fv.fvar_rtr_fill(torch.from_numpy(prev).cuda(), hw_in, hw_out, None, out2)      # inv == NULL fills all rows
    np.testing.assert_allclose(out2.cpu().numpy()[0], orc.upsample_bilinear(prev[0].astype(np.float64), hw_in, hw_out),
                               atol=2e-5, rtol=1e-5)


# ----------------------------------------------------------------------------- sampled selection keys

@pytest.mark.parametrize("B,M,C", [(2, 256, 1024), (1, 4096, 2048), (3, 100, 64)])
def test_row_keys_and_sampled_selection(fv, B, M, C):
    """Keys s_i / E_i of the sampled selection: the division is exact in fp32 on both sides, so the keys
    differ only by the summation order of the score; selection on identical keys is bit-exact."""
    x = si.make_tokens(41, B, M, C, "spread")
    noise = si.make_sample_noise(41, 0, 1, B, M)[0]
    got = fv.fvar_row_keys(torch.from_numpy(x).cuda(), torch.from_numpy(noise).cuda()).cpu().numpy()
    ref64 = orc.row_scores(x, np.float64) / noise.astype(np.float64)
    np.testing.assert_allclose(got, ref64, rtol=3e-6)
    keys = np.stack([orc.sampling_keys(orc.row_scores(x[b], np.float32), noise[b]) for b in range(B)])
    for r in (1, max(1, M // 4), M // 2):
        _check_select(fv, keys, r)
    # a key is one correctly rounded fp32 division of the kernel's own score
    s_gpu = fv.fvar_row_scores(torch.from_numpy(x).cuda()).cpu().numpy()
    assert np.array_equal(got, (s_gpu / noise).astype(np.float32))


# ----------------------------------------------------------------------------- run-to-run determinism of the cluster reductions

def test_cluster_reductions_are_bit_stable(fv):
    """The K split of the cluster GEMMs and the key split of attention add their partial results in rank order, so
    repeated launches on the same operands give the same bits."""
    rng = np.random.default_rng(77)
    A = to_bf16_cuda(si.normal_bf16(rng, (170, 8192)))
    W = to_bf16_cuda(si.normal_bf16(rng, (2048, 8192), 0.05))
    for form in (fv.GEMM_SKINNY, fv.GEMM_KSPLIT):
        first = fv.fvar_gemm_bf16_form(A, W, None, form, 0).clone()
        for _ in range(3):
            assert torch.equal(first, fv.fvar_gemm_bf16_form(A, W, None, form, 0))
    B, H, D, r, L, L_cap = 1, 16, 128, 170, 6595, 6656
    q = to_bf16_cuda(si.normal_bf16(rng, (B, r, H * D)))
    Kc = to_bf16_cuda(si.normal_bf16(rng, (B, H, L_cap, D)))
    Vt = to_bf16_cuda(si.normal_bf16(rng, (B, H, D, L_cap)))
    first = fv.fvar_attention(q, Kc, Vt, L).clone()
    for _ in range(3):
        assert torch.equal(first, fv.fvar_attention(q, Kc, Vt, L))
    _poll(fv)
