"""Pins for the CPU oracle: closed forms, invariants, brute force on tiny inputs, library
routines for the special cases that reduce to one, and the values the paper prints.
None of these needs a GPU; none calls the CUDA path."""
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import synth_inputs as si
from oracle import fvar_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_rows(name):
    rows = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


# ----------------------------------------------------------------------------- elementary pieces

def test_gelu_tanh_closed_form_and_identities():
    x = np.linspace(-6, 6, 241)
    g = orc.gelu_tanh(x)
    assert orc.gelu_tanh(np.array([0.0]))[0] == 0.0
    np.testing.assert_allclose(g - orc.gelu_tanh(-x), x, atol=1e-12)       # g(x) - g(-x) = x
    ref = F.gelu(torch.from_numpy(x), approximate="tanh").numpy()           # library routine
    np.testing.assert_allclose(g, ref, atol=1e-12)
    # not the erf GELU: they differ by ~5e-4 around |x| ~ 2
    erf = F.gelu(torch.from_numpy(x)).numpy()
    assert np.max(np.abs(g - erf)) > 1e-4


def test_silu_and_ada_chunk_order():
    rng = np.random.default_rng(0)
    C = 16
    c = rng.standard_normal(C)
    W = rng.standard_normal((6 * C, C))
    b = rng.standard_normal(6 * C)
    np.testing.assert_allclose(orc.silu(c), F.silu(torch.from_numpy(c)).numpy(), atol=1e-12)
    ada = orc.ada_vectors(c, W, b)
    ref = F.linear(F.silu(torch.from_numpy(c)), torch.from_numpy(W), torch.from_numpy(b)).numpy()
    for j in range(6):                       # chunk j is rows [jC, (j+1)C) of the 6C output
        np.testing.assert_allclose(ada[j], ref[j * C:(j + 1) * C], atol=1e-10)


def test_layer_norm_moments_and_library():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((7, 64)) * 3.0 + 1.5
    y = orc.layer_norm(x, 1e-6)
    np.testing.assert_allclose(y.mean(-1), 0.0, atol=1e-12)
    np.testing.assert_allclose(y.var(-1), 1.0, atol=1e-5)
    ref = F.layer_norm(torch.from_numpy(x), (64,), eps=1e-6).numpy()
    np.testing.assert_allclose(y, ref, atol=1e-10)


def _attention_loops(q, K, V, H):
    """Brute force with explicit Python loops and a two-pass softmax."""
    n, C = len(q), len(q[0])
    L = len(K)
    D = C // H
    out = [[0.0] * C for _ in range(n)]
    for i in range(n):
        for h in range(H):
            s = []
            for l in range(L):
                acc = 0.0
                for d in range(D):
                    acc += q[i][h * D + d] * K[l][h * D + d]
                s.append(acc / math.sqrt(D))
            m = max(s)
            e = [math.exp(v - m) for v in s]
            z = sum(e)
            for d in range(D):
                acc = 0.0
                for l in range(L):
                    acc += e[l] / z * V[l][h * D + d]
                out[i][h * D + d] = acc
    return np.array(out)


@pytest.mark.parametrize("n,L,H,D", [(3, 5, 2, 4), (8, 16, 1, 8), (1, 1, 2, 2)])
def test_attention_brute_force_and_sdpa(n, L, H, D):
    rng = np.random.default_rng(2)
    C = H * D
    q, K, V = rng.standard_normal((n, C)), rng.standard_normal((L, C)), rng.standard_normal((L, C))
    a = orc.attention(q, K, V, H)
    np.testing.assert_allclose(a, _attention_loops(q.tolist(), K.tolist(), V.tolist(), H), atol=1e-12)
    tq = torch.from_numpy(q).view(n, H, D).transpose(0, 1)
    tk = torch.from_numpy(K).view(L, H, D).transpose(0, 1)
    tv = torch.from_numpy(V).view(L, H, D).transpose(0, 1)
    ref = F.scaled_dot_product_attention(tq, tk, tv).transpose(0, 1).reshape(n, C).numpy()
    np.testing.assert_allclose(a, ref, atol=1e-10)


def test_attention_special_cases():
    rng = np.random.default_rng(3)
    q, K = rng.standard_normal((4, 8)), rng.standard_normal((6, 8))
    Vconst = np.tile(rng.standard_normal((1, 8)), (6, 1))
    np.testing.assert_allclose(orc.attention(q, K, Vconst, 2), np.tile(Vconst[:1], (4, 1)), atol=1e-12)
    v1 = rng.standard_normal((1, 8))                     # single key: output is its value
    np.testing.assert_allclose(orc.attention(q, K[:1], v1, 2), np.tile(v1, (4, 1)), atol=1e-12)
    p = orc.softmax_rows(rng.standard_normal((5, 9)) * 30)
    np.testing.assert_allclose(p.sum(-1), 1.0, atol=1e-12)


# ----------------------------------------------------------------------------- the block

def _weights(seed, shp, std=0.05):
    return si.make_weights(seed, shp, std)


def _torch_block(x, ada6, w, Kc, Vc, H, eps, cross_kv=None):
    """The same block written against torch's library routines (an independent route)."""
    t = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    x = t(x)
    C = x.shape[-1]
    D = C // H
    sh1, sc1, g1, sh2, sc2, g2 = [t(v) for v in ada6]

    def heads(a):
        return a.view(a.shape[0], H, D).transpose(0, 1)

    y = F.layer_norm(x, (C,), eps=eps) * (1 + sc1) + sh1
    qkv = F.linear(y, t(w["w_qkv"]), t(w["b_qkv"]))
    q, k, v = qkv.split(C, dim=-1)
    K = torch.cat([t(Kc), k], 0)
    V = torch.cat([t(Vc), v], 0)
    a = F.scaled_dot_product_attention(heads(q), heads(K), heads(V)).transpose(0, 1).reshape(-1, C)
    x = x + g1 * F.linear(a, t(w["w_o"]), t(w["b_o"]))
    if cross_kv is not None:
        yc = F.layer_norm(x, (C,), weight=t(w["ln_c_gamma"]), eps=eps)
        qc = F.linear(yc, t(w["w_cq"]))
        ac = F.scaled_dot_product_attention(heads(qc), heads(t(cross_kv[0])), heads(t(cross_kv[1])))
        x = x + F.linear(ac.transpose(0, 1).reshape(-1, C), t(w["w_co"]))
    y = F.layer_norm(x, (C,), eps=eps) * (1 + sc2) + sh2
    x = x + g2 * F.linear(F.gelu(F.linear(y, t(w["w_fc1"]), t(w["b_fc1"])), approximate="tanh"),
                          t(w["w_fc2"]), t(w["b_fc2"]))
    return x.numpy(), k.numpy(), v.numpy()


@pytest.mark.parametrize("cross", [False, True])
def test_block_matches_library_route(cross):
    shp = si.shape_tiny(n_blocks=1, width=32, n_heads=4, head_dim=8, ffn_dim=48, cross=cross, ctx_len=5)
    w = {k: v.astype(np.float64) for k, v in _weights(10, shp, 0.3)[0].items()}
    rng = np.random.default_rng(4)
    x = rng.standard_normal((6, 32))
    ada6 = rng.standard_normal((6, 32)) * 0.5
    Kc, Vc = rng.standard_normal((9, 32)), rng.standard_normal((9, 32))
    ckv = (rng.standard_normal((5, 32)), rng.standard_normal((5, 32))) if cross else None
    got = orc.block_forward(x, ada6, w, Kc, Vc, 4, 1e-6, ckv)
    ref = _torch_block(x, ada6, w, Kc, Vc, 4, 1e-6, ckv)
    for a, b in zip(got, ref):
        np.testing.assert_allclose(a, b, atol=1e-9)
    # query_rows: a subset of output rows, keys from all rows
    rows = np.array([0, 3, 5])
    sub, _, _ = orc.block_forward(x, ada6, w, Kc, Vc, 4, 1e-6, ckv, query_rows=rows)
    np.testing.assert_allclose(sub, got[0][rows], atol=1e-12)


def test_block_gate_zero_is_identity_and_plain_prelen():
    shp = si.shape_tiny(n_blocks=1, width=32, n_heads=2, head_dim=16, ffn_dim=64)
    w = {k: v.astype(np.float64) for k, v in _weights(11, shp, 0.3)[0].items()}
    rng = np.random.default_rng(5)
    x = rng.standard_normal((5, 32))
    K0 = np.zeros((0, 32))
    ada = rng.standard_normal((6, 32))
    ada[2] = 0.0
    ada[5] = 0.0                                             # both gates zero
    out, _, _ = orc.block_forward(x, ada, w, K0, K0, 2, 1e-6)
    np.testing.assert_array_equal(out, x)
    ada = np.zeros((6, 32))
    ada[2] = 1.0
    ada[5] = 1.0                                             # plain pre-LN block
    out, _, _ = orc.block_forward(x, ada, w, K0, K0, 2, 1e-6)
    y = orc.layer_norm(x, 1e-6)
    qkv = y @ w["w_qkv"].T + w["b_qkv"]
    a = orc.attention(qkv[:, :32], qkv[:, 32:64], qkv[:, 64:], 2)
    x1 = x + a @ w["w_o"].T + w["b_o"]
    x2 = x1 + orc.gelu_tanh(orc.layer_norm(x1, 1e-6) @ w["w_fc1"].T + w["b_fc1"]) @ w["w_fc2"].T + w["b_fc2"]
    np.testing.assert_allclose(out, x2, atol=1e-12)


def test_kv_cache_concatenation_order():
    """Attention over [cache; own rows] equals attention over the concatenated array, and a
    permutation of the keys (with their values) leaves the output unchanged."""
    rng = np.random.default_rng(6)
    q = rng.standard_normal((4, 16))
    K, V = rng.standard_normal((10, 16)), rng.standard_normal((10, 16))
    a = orc.attention(q, K, V, 2)
    perm = rng.permutation(10)
    np.testing.assert_allclose(orc.attention(q, K[perm], V[perm], 2), a, atol=1e-12)
    # mismatched permutation of K against V changes the result (guards a K/V mix-up)
    assert np.max(np.abs(orc.attention(q, K[perm], V, 2) - a)) > 1e-3


# ----------------------------------------------------------------------------- score / selection

def test_row_probabilities_sum_to_one_and_definition():
    rng = np.random.default_rng(7)
    X = rng.standard_normal((9, 5))
    p = orc.row_probabilities(X)
    assert abs(p.sum() - 1.0) < 1e-12
    fro2 = sum(float(v) ** 2 for v in X.ravel())
    for i in range(9):
        assert abs(p[i] - sum(float(v) ** 2 for v in X[i]) / fro2) < 1e-12
    np.testing.assert_allclose(orc.row_scores(X, np.float64), np.linalg.norm(X, axis=1) ** 2, atol=1e-12)


def _brute_top_r(s, r):
    M = len(s)
    key = [(math.inf if math.isnan(v) else float(v)) for v in s]
    taken = []
    for _ in range(r):                                      # repeated argmax, lowest index on ties
        best = None
        for i in range(M):
            if i in taken:
                continue
            if best is None or key[i] > key[best]:
                best = i
        taken.append(best)
    return sorted(taken)


def test_select_matches_brute_force_with_ties_and_nan():
    rng = np.random.default_rng(8)
    for trial in range(20):
        M = int(rng.integers(1, 40))
        s = rng.integers(0, 6, size=M).astype(np.float32)    # many ties
        if trial % 3 == 0 and M > 2:
            s[rng.integers(0, M)] = np.nan
            s[rng.integers(0, M)] = np.inf
        if trial % 4 == 0:
            s[0] = -0.0
        for r in {1, M, max(1, M // 2)}:
            idx = orc.select_top_r(s, r)
            assert idx.dtype == np.int32 and len(idx) == r
            assert list(idx) == _brute_top_r(s.tolist(), r)
            assert all(idx[i] < idx[i + 1] for i in range(r - 1))
    # library route on tie-free scores
    s = rng.permutation(100).astype(np.float32)
    top = torch.topk(torch.from_numpy(s), 17).indices.numpy()
    assert list(orc.select_top_r(s, 17)) == sorted(top.tolist())


# ----------------------------------------------------------------------------- random projection

def test_random_projection_loops_linearity_and_jl():
    rng = np.random.default_rng(9)
    M, r, C = 7, 3, 4
    Q, X, Y = rng.standard_normal((M, r)), rng.standard_normal((M, C)), rng.standard_normal((M, C))
    P = orc.random_projection(Q, X)
    assert P.shape == (r, C)
    for j in range(r):
        for c in range(C):
            assert abs(P[j, c] - sum(Q[m, j] * X[m, c] for m in range(M))) < 1e-12
    np.testing.assert_allclose(orc.random_projection(Q, 2 * X - 3 * Y), 2 * P - 3 * orc.random_projection(Q, Y),
                               atol=1e-12)
    # Q_ij ~ N(0, 1/r): E[Q Q^T] = I and E||Q^T x||^2 = ||x||^2
    M, r = 64, 32
    x = rng.standard_normal((M, 1))
    acc, norms, n = np.zeros((M, M)), [], 300
    for s in range(n):
        Qs = si.make_projection(s, 0, 0, M, r).astype(np.float64)
        acc += Qs @ Qs.T
        norms.append(float(np.sum(orc.random_projection(Qs, x) ** 2)))
    acc /= n
    assert abs(np.mean(np.diag(acc)) - 1.0) < 0.02
    off = acc - np.diag(np.diag(acc))
    assert np.abs(off).max() < 6.0 / math.sqrt(n * r) * 2     # ~ N(0, 1/(n r)) entries
    assert abs(np.mean(norms) / float(np.sum(x ** 2)) - 1.0) < 0.05


# ----------------------------------------------------------------------------- Up(.) and restoration

@pytest.mark.parametrize("hw_in,hw_out", [((3, 3), (5, 5)), ((4, 6), (5, 7)), ((13, 13), (16, 16)), ((2, 2), (2, 2)),
                                          ((1, 1), (3, 2))])
def test_upsample_matches_library_and_exact_cases(hw_in, hw_out):
    rng = np.random.default_rng(10)
    C = 3
    Fm = rng.standard_normal((hw_in[0] * hw_in[1], C))
    up = orc.upsample_bilinear(Fm, hw_in, hw_out)
    t = torch.from_numpy(Fm).view(1, hw_in[0], hw_in[1], C).permute(0, 3, 1, 2)
    ref = F.interpolate(t, size=hw_out, mode="bilinear", align_corners=False)
    ref = ref.permute(0, 2, 3, 1).reshape(-1, C).numpy()
    np.testing.assert_allclose(up, ref, atol=1e-12)
    if hw_in == hw_out:
        np.testing.assert_array_equal(up, Fm)
    const = np.full((hw_in[0] * hw_in[1], 1), 2.5)
    np.testing.assert_allclose(orc.upsample_bilinear(const, hw_in, hw_out), 2.5, atol=1e-12)


def test_upsample_linear_ramp_interior_exact():
    h0, w0, h1, w1 = 4, 4, 8, 8
    ys, xs = np.meshgrid(np.arange(h0), np.arange(w0), indexing="ij")
    ramp = (2.0 * ys + 3.0 * xs).reshape(-1, 1).astype(np.float64)
    up = orc.upsample_bilinear(ramp, (h0, w0), (h1, w1)).reshape(h1, w1)
    for y in range(1, h1 - 1):
        for x in range(1, w1 - 1):
            sy, sx = (y + 0.5) * h0 / h1 - 0.5, (x + 0.5) * w0 / w1 - 0.5
            assert abs(up[y, x] - (2.0 * sy + 3.0 * sx)) < 1e-12


def test_rtr_restore_row_identities():
    rng = np.random.default_rng(11)
    M, r, C = 12, 5, 4
    cache_up = rng.standard_normal((M, C))
    Fr = rng.standard_normal((r, C))
    idx = np.array(sorted(rng.choice(M, r, replace=False)), dtype=np.int32)
    out = orc.rtr_restore(Fr, idx, cache_up)
    inset = set(idx.tolist())
    for j, i in enumerate(idx):
        np.testing.assert_array_equal(out[i], Fr[j])         # row j of F_r^o lands at the j-th smallest index
    for i in range(M):
        if i not in inset:
            np.testing.assert_array_equal(out[i], cache_up[i])
    # if the cache already equals the dense output, exact rows at any index set give the dense output
    dense = rng.standard_normal((M, C))
    np.testing.assert_array_equal(orc.rtr_restore(dense[idx], idx, dense), dense)


# ----------------------------------------------------------------------------- schedule / printed values

def test_rank_table_matches_paper_and_mean_is_17_6_percent():
    rows = [[float(v) for v in r] for r in _read_rows("rank_ratio_alpha096.txt")]
    assert len(rows) == 8 and all(len(r) == 3 for r in rows)
    assert tuple(tuple(r) for r in rows) == orc.INFINITY_RANK_RATIO
    col40 = [r[0] for r in rows]
    assert abs(sum(col40) / 8 - 0.17675) < 1e-12             # "17.6 % rank" at alpha = 0.96
    pct = {float(a): float(p) for a, p in _read_rows("alpha_to_rank_percent.txt")}
    assert abs(pct[0.96] - 100 * sum(col40) / 8) < 0.1


def test_rank_rules_and_counts():
    assert orc.rank_from_keep_ratio(256, 0.5) == 128
    assert orc.rank_from_keep_ratio(169, 0.5) == 85 and orc.rank_from_keep_ratio(100, 0.5) == 50
    assert orc.rank_from_keep_ratio(169, 0.75) == 127 and orc.rank_from_keep_ratio(256, 0.75) == 192
    assert orc.rank_from_keep_ratio(256, 1.0) == 256
    # ratios are of n = min(M, d): scale 40 (M=1600 < d=2048) and scale 64 (M=4096 > d=2048)
    got40 = [orc.rank_from_table_ratio(1600, 2048, row[0]) for row in orc.INFINITY_RANK_RATIO]
    got64 = [orc.rank_from_table_ratio(4096, 2048, row[2]) for row in orc.INFINITY_RANK_RATIO]
    assert got40 == [26, 218, 336, 400, 410, 317, 251, 306]
    assert got64 == [16, 111, 170, 135, 115, 59, 78, 113]


def test_scale_schedules_prefix_sums():
    rows = {r[0]: [int(v) for v in r[1:]] for r in _read_rows("scale_schedules.txt")}
    assert tuple(rows["infinity"]) == si.INFINITY_SCALES and tuple(rows["var256"]) == si.VAR_SCALES
    for name in ("infinity", "var256"):
        acc, sums = 0, []
        for s in rows[name]:
            acc += s * s
            sums.append(acc)
        assert sums == rows[name + "_cache_rows"]
    assert rows["infinity_cache_rows"][-1] == 10521 and rows["var256_cache_rows"][-1] == 680


def test_energy_rank_on_known_spectrum():
    rng = np.random.default_rng(12)
    U, _ = np.linalg.qr(rng.standard_normal((20, 20)))
    V, _ = np.linalg.qr(rng.standard_normal((12, 12)))
    sv = np.array([4.0, 2.0, 1.0, 1.0] + [0.0] * 8)           # energies 16, 4, 1, 1 of 22
    X = U[:, :12] * sv @ V.T
    assert orc.energy_rank(X, 0.70) == 1                      # 16/22 = 0.727
    assert orc.energy_rank(X, 0.90) == 2                      # 20/22 = 0.909
    assert orc.energy_rank(X, 0.95) == 3                      # 21/22 = 0.9545
    assert orc.energy_rank(X, 0.96) == 4


# ----------------------------------------------------------------------------- the whole step

def _mk_oracle(shp, seed=20, B=2):
    w = si.make_weights(seed, shp, 0.05)
    o = orc.Oracle(w, shp.n_heads, shp.blocks_per_group, shp.hw())
    ctx = si.make_context(seed, B, shp.ctx_len, shp.ctx_width) if shp.has_cross_attn else None
    o.set_cond(si.make_cond(seed, B, shp.width), ctx)
    return o


@pytest.mark.parametrize("cross", [False, True])
def test_full_rank_equals_dense_exactly(cross):
    """r = M (keep ratio 1.0) is defined as Q = I, I = all rows: bitwise the dense step."""
    shp = si.shape_tiny(n_blocks=4, blocks_per_group=2, width=32, n_heads=2, head_dim=16, ffn_dim=64,
                        scales=(1, 2, 3), cross=cross, ctx_len=4)
    toks = [si.make_tokens(21, 2, m, 32) for m in shp.tokens_per_scale()]
    a, b = _mk_oracle(shp), _mk_oracle(shp)
    for k in range(3):
        oa = a.scale_step(toks[k], k, orc.Policy("dense"))
        ob = b.scale_step(toks[k], k, orc.Policy("lowrank_rtr", keep_ratio=1.0))
        np.testing.assert_array_equal(oa, ob)
        a.kv_append(k)
        b.kv_append(k)
        assert a.cache_len(0, 0) == sum(shp.tokens_per_scale()[:k + 1])


def test_step_late_mode_structure():
    """Late step: |I| = r per group, ascending; rows outside I equal Up(previous group output);
    rows in I equal the blocks applied to Q^T X; the cache grows by r rows; null-only computes
    only the odd (unconditional) batch elements."""
    shp = si.shape_tiny(n_blocks=2, blocks_per_group=1, width=32, n_heads=2, head_dim=16, ffn_dim=64,
                        scales=(2, 3, 4))
    B, C = 4, 32
    o = _mk_oracle(shp, B=B)
    toks = [si.make_tokens(22, B, m, C) for m in shp.tokens_per_scale()]
    for k in range(2):
        o.scale_step(toks[k], k, orc.Policy("dense"))
        o.kv_append(k)
    prev = [[o.group_cache[g][b].copy() for b in range(B)] for g in range(2)]
    L0 = o.cache_len(1, 1)
    M, ranks = 16, [6, 9]
    for g in range(2):
        o.set_projection(2, g, si.make_projection(22, 2, g, M, ranks[g]))
    out = o.scale_step(toks[2], 2, orc.Policy("lowrank_rtr", "null_only", rank_per_group=ranks))
    assert out.shape == (2, M, C)
    for e, b in enumerate((1, 3)):
        X = toks[2][b].astype(np.float64)
        for g in range(2):
            idx = o.last_indices[e][g]
            assert len(idx) == ranks[g] and np.all(np.diff(idx) > 0) and idx[0] >= 0 and idx[-1] < M
            assert list(idx) == list(orc.select_top_r(orc.row_scores(X, np.float32), ranks[g]))
            up = orc.upsample_bilinear(prev[g][b], (3, 3), (4, 4))
            xr, k_new, _ = orc.block_forward(orc.random_projection(o.proj[(2, g)], X), o.ada[g][b], o.w[g],
                                             o.K[g][b], o.V[g][b], 2, 1e-6)
            res = o.group_cache[g][b]
            mask = np.ones(M, bool)
            mask[idx] = False
            np.testing.assert_array_equal(res[mask], up[mask])
            np.testing.assert_allclose(res[idx], xr, atol=1e-12)
            assert k_new.shape[0] == ranks[g]
            X = res
        np.testing.assert_array_equal(out[e], X)
    o.kv_append(2)
    assert o.cache_len(0, 1) == L0 + 6 and o.cache_len(1, 3) == L0 + 9
    assert o.cache_len(0, 0) == L0                            # conditional element not computed
    assert o.scale_step(toks[2], 2, orc.Policy("skip")) is None


def test_forced_indices_are_used():
    shp = si.shape_tiny(n_blocks=1, width=32, n_heads=2, head_dim=16, ffn_dim=64, scales=(2, 3))
    o = _mk_oracle(shp)
    toks = [si.make_tokens(23, 2, m, 32) for m in shp.tokens_per_scale()]
    o.scale_step(toks[0], 0, orc.Policy("dense"))
    o.kv_append(0)
    o.set_projection(1, 0, si.make_projection(23, 1, 0, 9, 4))
    forced = [[np.array([0, 2, 5, 8])], [np.array([1, 3, 4, 7])]]
    o.scale_step(toks[1], 1, orc.Policy("lowrank_rtr", rank_per_group=[4], forced_indices=forced))
    assert list(o.last_indices[0][0]) == [0, 2, 5, 8] and list(o.last_indices[1][0]) == [1, 3, 4, 7]


def test_sampling_keys_exponential_race():
    """The first pick of the sampled selection is row i with probability s_i / sum s (property of the
    exponential race), r picks are distinct, and equal noise reduces the rule to plain top-r."""
    s = np.array([5.0, 1.0, 3.0, 0.5, 0.5], dtype=np.float32)
    n = 20000
    noise = si.make_sample_noise(3, 0, 1, n, 5)[0]
    first = np.array([orc.select_top_r(orc.sampling_keys(s, noise[t]), 1)[0] for t in range(n)])
    freq = np.bincount(first, minlength=5) / n
    expect = s / s.sum()
    assert np.all(np.abs(freq - expect) < 4 * np.sqrt(expect * (1 - expect) / n) + 1e-3)
    picks = orc.select_top_r(orc.sampling_keys(s, noise[0]), 3)
    assert len(set(picks.tolist())) == 3 and list(picks) == sorted(picks)
    ones = np.ones(5, dtype=np.float32)
    assert list(orc.select_top_r(orc.sampling_keys(s, ones), 2)) == list(orc.select_top_r(s, 2))
    k = orc.sampling_keys(np.array([3.0], np.float32), np.array([7.0], np.float32))
    assert k.dtype == np.float32 and k[0] == np.float32(3.0) / np.float32(7.0)


# ----------------------------------------------------------------------------- seeded projection

def test_philox_known_answers():
    """The counter-based generator behind the seeded projection against its published vectors."""
    n = 0
    with open(os.path.join(GOLD, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if not line.strip() or line.startswith("#"):
                continue
            v = [int(t, 16) for t in line.split()]
            out = orc.philox4x32_10(np.array(v[0:4], dtype=np.uint32), (v[4], v[5]))
            assert [int(o) for o in out] == v[6:10]
            n += 1
    assert n == 2
    # a bijection of the counter: distinct counters, distinct outputs; vectorised == one by one
    ctr = np.zeros((64, 4), dtype=np.uint32)
    ctr[:, 0] = np.arange(64)
    outs = orc.philox4x32_10(ctr, (7, 9))
    assert len({tuple(int(x) for x in o) for o in outs}) == 64
    assert np.array_equal(outs[5], orc.philox4x32_10(ctr[5], (7, 9)))


def test_round_f64_to_bf16_is_one_correct_rounding():
    """Against exact rational arithmetic on the two neighbouring bf16 values, including values that a
    detour through fp32 would round the wrong way (fp32 result exactly on a bf16 tie)."""
    from fractions import Fraction
    rng = np.random.default_rng(3)
    xs = list(rng.standard_normal(200) * 10.0 ** rng.integers(-3, 3, 200))
    base = float(np.float32(1.0) + np.float32(2.0 ** -8))           # a bf16 tie: 1 + half an ulp (ulp = 2^-7)
    xs += [base, base * (1 + 2.0 ** -40), base * (1 - 2.0 ** -40), -base * (1 + 2.0 ** -40), 3 * base, 0.0, 2.0 ** -7]
    got = orc.round_f64_to_bf16(np.array(xs))
    for x, g in zip(xs, got):
        if x == 0.0:
            assert g == 0.0
            continue
        # neighbours: truncate |x| to 8 significant bits, and the next one up
        m, e = math.frexp(abs(x))                         # |x| = m 2^e, m in [0.5, 1)
        lo = Fraction(int(m * 256), 256) * Fraction(2) ** e
        hi = lo + Fraction(1, 256) * Fraction(2) ** e
        fx = Fraction(abs(x))
        if fx - lo < hi - fx:
            want = lo
        elif fx - lo > hi - fx:
            want = hi
        else:                                             # tie: even significand
            want = lo if int(m * 256) % 2 == 0 else hi
        assert Fraction(float(abs(g))) == want, (x, g)
        assert (g < 0) == (x < 0)


def test_generated_projection_layout_and_distribution():
    from scipy import stats
    seed, k, g, M, r = 0x1234567812345678, 9, 3, 256, 96
    Q = orc.generate_projection(seed, k, g, M, r)
    assert Q.shape == (M, r) and Q.dtype == np.float32
    assert np.array_equal(si.round_to_bf16(Q), Q)                      # bf16-representable
    # layout: element n = j * M + i of the flattened Q^T comes from call n // 4, word pair (n % 4) // 2
    for (i, j) in [(0, 0), (5, 0), (255, 95), (17, 40)]:
        n = j * M + i
        x = orc.philox4x32_10(np.array([n // 4, g, k, 0], dtype=np.uint32), (seed & 0xFFFFFFFF, seed >> 32))
        a = 2 * ((n % 4) // 2)
        u0, u1 = (int(x[a]) + 0.5) / 2 ** 32, (int(x[a + 1]) + 0.5) / 2 ** 32
        rad, ang = math.sqrt(-2.0 * math.log(u0)), 2.0 * math.pi * u1
        z = rad * (math.cos(ang) if n % 2 == 0 else math.sin(ang)) / math.sqrt(r)
        assert abs(float(Q[i, j]) - z) <= 2.0 ** -8 * abs(z) + 1e-12
    # distribution: N(0, 1/r) by Kolmogorov-Smirnov (bf16 rounding moves the CDF by < 2^-8 relative)
    z = Q.astype(np.float64).ravel() * math.sqrt(r)
    assert stats.kstest(z, "norm").pvalue > 1e-3
    assert abs(z.mean()) < 5.0 / math.sqrt(z.size) and abs(z.var() - 1.0) < 0.03
    # E[Q Q^T] = I_M: diagonal near 1, off-diagonal near 0 with the spread 1/sqrt(r)
    QQ = Q.astype(np.float64) @ Q.astype(np.float64).T
    assert abs(np.diag(QQ).mean() - 1.0) < 0.03
    off = QQ[~np.eye(M, dtype=bool)]
    assert abs(off.mean()) < 0.01 and abs(off.std() - 1.0 / math.sqrt(r)) < 0.02
    # other (seed, scale, group) give other draws; the same arguments give the same matrix
    assert np.array_equal(Q, orc.generate_projection(seed, k, g, M, r))
    assert not np.array_equal(Q, orc.generate_projection(seed, k, g + 1, M, r))
    assert not np.array_equal(Q, orc.generate_projection(seed + 1, k, g, M, r))


# ----------------------------------------------------------------------------- between two scale steps

def test_nearest_codeword_is_the_euclidean_argmin():
    rng = np.random.default_rng(21)
    Z = rng.standard_normal((37, 16))
    X = rng.standard_normal((50, 16))
    got = orc.nearest_codeword(X, Z, dtype=np.float64)
    want = np.array([min(range(37), key=lambda v: (float(((x - Z[v]) ** 2).sum()), v)) for x in X])
    assert np.array_equal(got, want)
    assert np.array_equal(got, torch.cdist(torch.from_numpy(X), torch.from_numpy(Z)).argmin(dim=1).numpy())
    # a codeword maps to itself; duplicates resolve to the lowest code
    Z2 = np.concatenate([Z, Z[:5]])
    assert np.array_equal(orc.nearest_codeword(Z2, Z2, dtype=np.float64)[-5:], np.arange(5))
    assert np.array_equal(orc.nearest_codeword(Z, Z, dtype=np.float64), np.arange(37))


@pytest.mark.parametrize("hw_in,hw_out", [((16, 16), (13, 13)), ((64, 64), (48, 48)), ((6, 10), (4, 3)), ((8, 8), (8, 8)),
                                          ((16, 16), (1, 1)), ((5, 7), (2, 7))])
def test_downsample_area_matches_library_and_exact_cases(hw_in, hw_out):
    rng = np.random.default_rng(22)
    C = 5
    Fm = rng.standard_normal((hw_in[0] * hw_in[1], C))
    got = orc.downsample_area(Fm, hw_in, hw_out)
    t = torch.from_numpy(Fm.reshape(hw_in[0], hw_in[1], C)).permute(2, 0, 1)[None]
    ref = F.interpolate(t, size=hw_out, mode="area")[0].permute(1, 2, 0).reshape(-1, C).numpy()
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)
    const = orc.downsample_area(np.full_like(Fm, 3.25), hw_in, hw_out)
    np.testing.assert_allclose(const, 3.25, atol=1e-13)
    if hw_in == hw_out:
        assert np.array_equal(got, Fm)
    if hw_out == (1, 1):
        np.testing.assert_allclose(got[0], Fm.mean(axis=0), atol=1e-12)


def test_scale_transition_telescopes_to_the_sum_of_upsampled_residuals():
    """Eq. "var_upf": after k transitions F_k = sum_i Up(R_i, (h_K, w_K)); the next input is Down of it
    (Eq. "var_downf"); at the last scale Up is the identity and there is no next input."""
    rng = np.random.default_rng(23)
    C, V = 8, 20
    sides = [1, 2, 3, 5, 8]
    Z = rng.standard_normal((V, C))
    hwK = (sides[-1], sides[-1])
    Fk = np.zeros((hwK[0] * hwK[1], C))
    total = np.zeros_like(Fk)
    for k, sd in enumerate(sides):
        Fo = rng.standard_normal((sd * sd, C))
        nxt_hw = (sides[k + 1], sides[k + 1]) if k + 1 < len(sides) else None
        codes, Fk, nxt = orc.scale_transition(Fk, Fo, Z, (sd, sd), hwK, nxt_hw)
        assert codes.dtype == np.int32 and codes.shape == (sd * sd,)
        total += orc.upsample_bilinear(Z[codes], (sd, sd), hwK)
        np.testing.assert_allclose(Fk, total, atol=1e-12)
        if nxt_hw is None:
            assert nxt is None
            np.testing.assert_allclose(Fk - prev, Z[codes], atol=1e-12)         # Up at equal size is the identity
        else:
            np.testing.assert_allclose(nxt, orc.downsample_area(total, hwK, nxt_hw), atol=1e-12)
        prev = Fk.copy()
    # an output that is exactly a codeword everywhere adds that codeword everywhere (constant maps stay constant)
    codes, F1, nxt = orc.scale_transition(np.zeros((64, C)), np.tile(Z[7], (9, 1)), Z, (3, 3), (8, 8), (5, 5))
    assert (codes == 7).all()
    np.testing.assert_allclose(F1, np.tile(Z[7], (64, 1)), atol=1e-12)
    np.testing.assert_allclose(nxt, np.tile(Z[7], (25, 1)), atol=1e-12)


def test_cfg_combine_end_points_and_linearity():
    rng = np.random.default_rng(24)
    a, b = rng.standard_normal((7, 5)), rng.standard_normal((7, 5))
    assert np.array_equal(orc.cfg_combine(a, b, 0.0), b)                 # CFG = 0: the null-prompt branch alone
    np.testing.assert_allclose(orc.cfg_combine(a, b, 1.0), a, atol=1e-15)
    np.testing.assert_allclose(orc.cfg_combine(a, b, 3.0), 3.0 * a - 2.0 * b, atol=1e-14)
    np.testing.assert_allclose(orc.cfg_combine(a, a, 7.5), a, atol=1e-14)  # equal branches: guidance changes nothing


# ----------------------------------------------------------------------------- LLS restoration (Eq. "lstsq", App. A.3)

def test_lls_restoration_matrix_is_the_least_squares_solution():
    """Against numpy's SVD-based lstsq on the transposed problem F_r^T W^T ~ F^T, and the normal-equation residual
    property: the residual is orthogonal to the rows of F_r."""
    rng = np.random.default_rng(41)
    M, r, d = 37, 9, 24
    F = rng.standard_normal((M, d))
    F_r = rng.standard_normal((r, d))
    W = orc.lls_restoration_matrix(F_r, F)
    ref = np.linalg.lstsq(F_r.T, F.T, rcond=None)[0].T
    np.testing.assert_allclose(W, ref, rtol=1e-9, atol=1e-10)
    np.testing.assert_allclose((W @ F_r - F) @ F_r.T, 0.0, atol=1e-9)
    # brute force on one row: no other w gives a smaller residual
    w0, f0 = W[3], F[3]
    base = np.linalg.norm(w0 @ F_r - f0)
    for _ in range(50):
        assert np.linalg.norm((w0 + 1e-3 * rng.standard_normal(r)) @ F_r - f0) >= base - 1e-12


def test_lls_restores_exactly_what_lies_in_the_row_space():
    """rank(F) <= r: F_hat = Q^T F spans the row space of F, so W_hat F_hat = F exactly.  r = M with Q = I: W_hat = I."""
    rng = np.random.default_rng(42)
    M, r, d = 40, 6, 30
    F = rng.standard_normal((M, 5)) @ rng.standard_normal((5, d))          # rank 5 <= r ... plus one direction so F_hat has rank r
    F = F + np.outer(rng.standard_normal(M), rng.standard_normal(d))
    Q = rng.standard_normal((M, r)) / np.sqrt(r)
    F_hat = orc.random_projection(Q, F)
    W = orc.lls_restoration_matrix(F_hat, F)
    np.testing.assert_allclose(W @ F_hat, F, rtol=1e-8, atol=1e-8)
    F2 = rng.standard_normal((8, 20))
    np.testing.assert_allclose(orc.lls_restoration_matrix(orc.random_projection(np.eye(8), F2), F2), np.eye(8), atol=1e-10)


def test_lls_restore_is_the_sum_of_the_two_restorations():
    """F_k^o = (W_hat + W^{o,cache}) F_r^o.  If the blocks were the identity (F_r^o = F_hat) and the cache equalled the
    input, each term would restore the best rank-r fit of the input, so the result is twice that fit."""
    rng = np.random.default_rng(43)
    M, r, d = 30, 7, 16
    F = rng.standard_normal((M, d))
    Q = rng.standard_normal((M, r)) / np.sqrt(r)
    F_hat = orc.random_projection(Q, F)
    fit = orc.lls_restoration_matrix(F_hat, F) @ F_hat
    np.testing.assert_allclose(orc.lls_restore(F_hat, F_hat, F, Q, F), 2.0 * fit, rtol=1e-9, atol=1e-10)
    # linear in the block output
    Fo1, Fo2 = rng.standard_normal((r, d)), rng.standard_normal((r, d))
    cache = rng.standard_normal((M, d))
    a = orc.lls_restore(Fo1, F_hat, F, Q, cache) + 2.0 * orc.lls_restore(Fo2, F_hat, F, Q, cache)
    np.testing.assert_allclose(orc.lls_restore(Fo1 + 2.0 * Fo2, F_hat, F, Q, cache), a, rtol=1e-9, atol=1e-9)


def test_lls_step_structure():
    """A late step under LLS restoration: every row of the group output comes from W F_r^o (no row is a copy of the
    upsampled cache), the cache grows by r rows per block as under RTR, and no index set is produced."""
    shp = si.shape_tiny(n_blocks=2, blocks_per_group=1, width=64, n_heads=1, head_dim=64, ffn_dim=128, scales=(2, 3, 4))
    w = si.make_weights(44, shp, 0.05)
    o = orc.Oracle(w, shp.n_heads, shp.blocks_per_group, shp.hw(), shp.ln_eps)
    o.set_cond(si.make_cond(44, 2, 64))
    for k in (0, 1):
        o.scale_step(si.make_tokens(44, 2, shp.tokens_per_scale()[k], 64), k, orc.Policy("dense"))
        o.kv_append(k)
    r = 5
    for g in range(2):
        o.set_projection(2, g, si.make_projection(44, 2, g, 16, r))
    up = [orc.upsample_bilinear(o.group_cache[g][1], (3, 3), (4, 4)) for g in range(2)]
    out = o.scale_step(si.make_tokens(44, 2, 16, 64), 2, orc.Policy("lowrank_rtr", "null_only", rank_per_group=[r, r], restore="lls"))
    assert out.shape == (1, 16, 64) and all(len(o.last_indices[0][g]) == 0 for g in range(2))
    for g in range(2):
        assert np.abs(o.group_cache[g][1] - up[g]).min(axis=1).max() > 0      # no row copied from the cache
        assert np.linalg.matrix_rank(o.group_cache[g][1], tol=1e-8) <= r       # M rows spanned by the r block-output rows
    o.kv_append(2)
    assert o.cache_len(0, 1) == 4 + 9 + r and o.cache_len(0, 0) == 4 + 9


# ----------------------------------------------------------------------------- wiring of the stateful oracle

def test_sample_noise_is_indexed_by_group_then_computed_element_then_row():
    """Oracle.scale_step under sampled selection: group g of computed element e (here the null-prompt elements b = 1, 3)
    uses sample_noise[g][e].  Rebuilt outside the class from the group inputs it leaves behind."""
    shp = si.shape_tiny(n_blocks=3, blocks_per_group=1, width=64, n_heads=1, head_dim=64, ffn_dim=128, scales=(2, 3, 4))
    o = orc.Oracle(si.make_weights(51, shp, 0.05), shp.n_heads, 1, shp.hw(), shp.ln_eps)
    B, r = 4, 5
    o.set_cond(si.make_cond(51, B, 64))
    for k in (0, 1):
        o.scale_step(si.make_tokens(51, B, shp.tokens_per_scale()[k], 64), k, orc.Policy("dense"))
        o.kv_append(k)
    for g in range(3):
        o.set_projection(2, g, si.make_projection(51, 2, g, 16, r))
    toks = si.make_tokens(51, B, 16, 64, "spread")
    noise = si.make_sample_noise(51, 2, 3, 2, 16)                       # [G = 3][E = 2][M = 16]
    o.scale_step(toks, 2, orc.Policy("lowrank_rtr", "null_only", rank_per_group=[r] * 3, sample_noise=noise))
    for e, b in enumerate((1, 3)):
        X = toks[b].astype(np.float64)
        for g in range(3):
            want = orc.select_top_r(orc.sampling_keys(orc.row_scores(X, np.float32), noise[g][e]), r)
            assert np.array_equal(o.last_indices[e][g], want), (e, g)
            X = o.group_cache[g][b]                                     # the next group's input
    # the lists really depend on the noise slice: another slice gives another list somewhere
    assert any(not np.array_equal(o.last_indices[0][g], o.last_indices[1][g]) for g in range(3))


def test_context_weight_rows_are_keys_then_values():
    """set_cond splits w_ckv [2C][ctx_width] into keys (first C rows) and values (last C rows).  With the value rows
    zeroed the cross-attention adds exactly nothing; with the key rows zeroed its scores are all equal, so it adds
    the mean value row through W_co."""
    shp = si.shape_tiny(n_blocks=1, width=64, n_heads=1, head_dim=64, ffn_dim=128, scales=(2,), cross=True, ctx_len=6)
    w = si.make_weights(52, shp, 0.05)
    cond, ctx = si.make_cond(52, 1, 64), si.make_context(52, 1, 6, 64)
    toks = si.make_tokens(52, 1, 4, 64)

    def run(wts):
        o = orc.Oracle(wts, 1, 1, shp.hw(), shp.ln_eps)
        o.set_cond(cond, ctx)
        return o.scale_step(toks, 0, orc.Policy("dense"))[0]

    no_values = [dict(w[0], w_ckv=np.concatenate([w[0]["w_ckv"][:64], np.zeros_like(w[0]["w_ckv"][64:])]))]
    no_cross = [dict(w[0], w_co=np.zeros_like(w[0]["w_co"]))]
    np.testing.assert_allclose(run(no_values), run(no_cross), rtol=0, atol=1e-12)
    no_keys = [dict(w[0], w_ckv=np.concatenate([np.zeros_like(w[0]["w_ckv"][:64]), w[0]["w_ckv"][64:]]))]
    # uniform scores: the cross-attention output of every row is mean_t(ctx_t W_v^T) W_co^T, independent of the query
    add = (ctx[0].astype(np.float64) @ w[0]["w_ckv"][64:].astype(np.float64).T).mean(axis=0) @ w[0]["w_co"].astype(np.float64).T
    o = orc.Oracle(no_keys, 1, 1, shp.hw(), shp.ln_eps)
    o.set_cond(cond, ctx)
    x = toks[0].astype(np.float64)
    o.ada[0][0].reshape(6, -1)[5] = 0.0                                  # gate2 = 0
    got, _, _ = orc.block_forward(x, o.ada[0][0], o.w[0], np.zeros((0, 64)), np.zeros((0, 64)), 1, shp.ln_eps, o.cross_kv[0][0])
    ref, _, _ = orc.block_forward(x, o.ada[0][0], dict(o.w[0], w_co=np.zeros((64, 64))), np.zeros((0, 64)), np.zeros((0, 64)), 1,
                                  shp.ln_eps, o.cross_kv[0][0])
    np.testing.assert_allclose(got - ref, np.broadcast_to(add, got.shape), rtol=1e-9, atol=1e-12)
