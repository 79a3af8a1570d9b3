"""CPU oracle for the late-scale step of VAR next-scale prediction under FasterVAR.

TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, obviously-correct numpy
restatement of what the GPU library computes.  It is imported by the tests, by
the smoke check and by the benchmark's CPU-baseline leg, and by nothing else;
it shares no code with the CUDA path and never calls it.

Arithmetic is fp64 (numpy) on bf16-representable inputs, except the row score
that decides the index set, which is taken in fp32 -- the precision the GPU
kernel decides it in -- so that both sides take the integer decision alike.

What the paper fixes and this file follows:
  * row score  p_i = ||F^(i)||^2 / ||F||_F^2            (Sec. 3.3, RTR paragraph)
  * index set I: the r most important rows, |I| = r       (Sec. 3.3; Algorithm 1)
  * random projection  F_r = Q^T F,  Q in R^{M x r}, Q_ij ~ N(0, 1/r)
                                                          (Sec. 3.3 RP; Algorithm 1)
    Q is either given as data or drawn from a seed (Philox4x32-10 + Box-Muller, below)
  * between two steps: R_k = Q(F_k^o), F_k = F_{k-1} + Up(R_k, (h_K, w_K)), next input Down(F_k, (h_{k+1}, w_{k+1}))
                                                          (Algorithm 1; Eq. "var_upf", Eq. "var_downf")
  * cached output upsampled, F^{o,cache}_{k-1} = Up(F^o_{k-1})   (Eq. "upcache")
  * restoration F^o_k := {F^o_r rows at I} U {cache rows elsewhere} (Eq. "redefine")
  * CFG = 0 in the fidelity-refinement stage = null-prompt branch only
                                                          (Sec. 3.2; Algorithm 1)
  * rank schedule: ratio of min(M, d) per block chunk and late scale
                                                          (Eq. "low_rank_percent"; App. A.1 table)
The paper gives no internals for its VAR block; the block below (AdaLN
shift/scale/gate, multi-head attention over a multi-scale KV cache, tanh-GELU
FFN, optional cross-attention) is the synthetic definition both sides use.

Parity pins live in tests/test_oracle_*.py.  The composite RP -> blocks -> RTR
numerics have no worked example in the paper: parity unpinned for the composite
beyond the invariants tested there (r = M equals the dense block, restoration
row identities, linearity and norm preservation of the projection).
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence

import numpy as np

# --------------------------------------------------------------------------- elementary pieces


def gelu_tanh(x: np.ndarray) -> np.ndarray:
    """tanh-approximated GELU: x/2 * (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3)))."""
    return 0.5 * x * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (x + 0.044715 * x ** 3)))


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def layer_norm(x: np.ndarray, eps: float) -> np.ndarray:
    """LayerNorm over the last axis, no affine, biased variance."""
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps)


def ada_vectors(cond: np.ndarray, w_ada: np.ndarray, b_ada: np.ndarray) -> np.ndarray:
    """AdaLN vectors of one block for one batch element: W_ada SiLU(c) + b_ada, as
    6 rows [shift1, scale1, gate1, shift2, scale2, gate2] of width C."""
    C = cond.shape[-1]
    return (w_ada @ silu(cond) + b_ada).reshape(6, C)


def modulate(x: np.ndarray, shift: np.ndarray, scale: np.ndarray, eps: float) -> np.ndarray:
    return layer_norm(x, eps) * (1.0 + scale) + shift


def softmax_rows(s: np.ndarray) -> np.ndarray:
    s = s - s.max(axis=-1, keepdims=True)
    e = np.exp(s)
    return e / e.sum(axis=-1, keepdims=True)


def attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, n_heads: int) -> np.ndarray:
    """Multi-head attention of queries q [n][C] over keys K [L][C] and values V [L][C];
    heads are contiguous slices of width C / n_heads; no mask; scores scaled by 1/sqrt(D)."""
    n, C = q.shape
    D = C // n_heads
    out = np.empty_like(q)
    for h in range(n_heads):
        sl = slice(h * D, (h + 1) * D)
        p = softmax_rows(q[:, sl] @ K[:, sl].T / math.sqrt(D))
        out[:, sl] = p @ V[:, sl]
    return out


# --------------------------------------------------------------------------- the method's own steps


def row_scores(X: np.ndarray, dtype=np.float32) -> np.ndarray:
    """s_i = sum_c X[i,c]^2 (numerator of the row probability; Sec. 3.3 RTR)."""
    Xd = np.asarray(X, dtype=dtype)
    return np.sum(Xd * Xd, axis=-1, dtype=dtype)


def row_probabilities(X: np.ndarray) -> np.ndarray:
    """p_i = ||X^(i)||^2 / ||X||_F^2 (Sec. 3.3 RTR)."""
    s = row_scores(X, np.float64)
    return s / s.sum()


def select_top_r(scores: np.ndarray, r: int) -> np.ndarray:
    """Indices of the r highest-scoring rows, returned ascending.
    Order: score descending, then index ascending; NaN ranks as +inf; -0 equals +0."""
    s = np.asarray(scores, dtype=np.float32).copy()
    s[np.isnan(s)] = np.inf
    s = s + np.float32(0.0)                      # -0 -> +0
    M = s.shape[0]
    order = sorted(range(M), key=lambda i: (-float(s[i]), i))
    return np.array(sorted(order[:r]), dtype=np.int32)


def sampling_keys(scores: np.ndarray, noise: np.ndarray) -> np.ndarray:
    """Keys for drawing rows without replacement with probability proportional to the row score
    (Sec. 3.3 RTR, read as sampling: row i is drawn with probability proportional to ||F^(i)||^2): with
    E_i ~ Exp(1) independent, the r largest s_i / E_i are a sample without replacement in which the
    first pick is row i with probability s_i / sum_j s_j (exponential race).  The noise E is an
    input; the keys are one fp32 division each, the precision the kernel decides in."""
    return (np.asarray(scores, dtype=np.float32) / np.asarray(noise, dtype=np.float32)).astype(np.float32)


def random_projection(Q: np.ndarray, X: np.ndarray) -> np.ndarray:
    """F_r = Q^T X: [r][C] from Q [M][r] and X [M][C] (Algorithm 1, RP step)."""
    return Q.T @ X


# --------------------------------------------------------------------------- seeded projection
# The method draws Q itself (Sec. 3.3 RP: Q_ij ~ N(0, 1/r); the robustness figure redraws it per
# generation), so both sides need the same draws from a seed.  The generator is Philox4x32-10
# (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC'11), a counter-based
# generator: output = ten rounds of a fixed bijection of a 128-bit counter under a 64-bit key.

PHILOX_M0, PHILOX_M1 = 0xD2511F53, 0xCD9E8D57      # round multipliers
PHILOX_W0, PHILOX_W1 = 0x9E3779B9, 0xBB67AE85      # key increments (Weyl sequence)


def philox4x32_10(counter: np.ndarray, key) -> np.ndarray:
    """counter uint32 [..., 4], key (k0, k1) -> uint32 [..., 4].  One round maps (c0, c1, c2, c3) to
    (hi(M1 c2) ^ c1 ^ k0, lo(M1 c2), hi(M0 c0) ^ c3 ^ k1, lo(M0 c0)); the key is bumped by (W0, W1)
    between rounds."""
    c = np.asarray(counter, dtype=np.uint64) & np.uint64(0xFFFFFFFF)
    c0, c1, c2, c3 = c[..., 0], c[..., 1], c[..., 2], c[..., 3]
    k0, k1 = int(key[0]) & 0xFFFFFFFF, int(key[1]) & 0xFFFFFFFF
    mask, sh = np.uint64(0xFFFFFFFF), np.uint64(32)
    for _ in range(10):
        p0 = np.uint64(PHILOX_M0) * c0
        p1 = np.uint64(PHILOX_M1) * c2
        c0, c1, c2, c3 = ((p1 >> sh) ^ c1 ^ np.uint64(k0), p1 & mask, (p0 >> sh) ^ c3 ^ np.uint64(k1), p0 & mask)
        k0, k1 = (k0 + PHILOX_W0) & 0xFFFFFFFF, (k1 + PHILOX_W1) & 0xFFFFFFFF
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def round_f64_to_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest bf16 value (ties to even) of each fp64 element, in ONE rounding, returned as fp32.
    Going through fp32 first would round twice: when the fp32 result lands exactly on a bf16 tie the
    direction has to come from the fp64 value."""
    x = np.asarray(x, dtype=np.float64)
    f = x.astype(np.float32)
    u = f.view(np.uint32).astype(np.int64)
    tie = (u & 0xFFFF) == 0x8000
    back = f.astype(np.float64)
    # magnitude of the fp32 value above / below the true one: step the bits off the tie accordingly
    u = np.where(tie & (np.abs(back) > np.abs(x)), u - 1, u)
    u = np.where(tie & (np.abs(back) < np.abs(x)), u + 1, u)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32)


def generate_projection(seed: int, scale_idx: int, group: int, M: int, r: int) -> np.ndarray:
    """Q [M][r] with Q_ij ~ N(0, 1/r) (Sec. 3.3 RP), bf16-rounded, from a 64-bit seed.

    Layout of the draws: Q^T is flattened row-major (element n = j * M + i holds Q_ij); call t of the
    generator, counter (t, group, scale_idx, 0) under key (seed low, seed high), yields elements
    4t .. 4t + 3.  From its words x0..x3: u = (x + 0.5) 2^-32 in (0, 1); Box-Muller on (u0, u1) and
    (u2, u3): z = sqrt(-2 ln u_a) * (cos 2 pi u_b, sin 2 pi u_b); Q = z / sqrt(r), all in fp64, then
    one rounding to bf16."""
    n = M * r
    calls = (n + 3) // 4
    ctr = np.zeros((calls, 4), dtype=np.uint32)
    ctr[:, 0] = np.arange(calls, dtype=np.uint32)
    ctr[:, 1] = group
    ctr[:, 2] = scale_idx
    x = philox4x32_10(ctr, (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)).astype(np.float64)
    u = (x + 0.5) * 2.0 ** -32
    z = np.empty((calls, 4), dtype=np.float64)
    for a in (0, 2):
        rad = np.sqrt(-2.0 * np.log(u[:, a]))
        ang = 2.0 * np.pi * u[:, a + 1]
        z[:, a] = rad * np.cos(ang)
        z[:, a + 1] = rad * np.sin(ang)
    qt = (z.reshape(-1)[:n] / math.sqrt(r)).reshape(r, M)
    return np.ascontiguousarray(round_f64_to_bf16(qt).T)


def upsample_bilinear(F: np.ndarray, hw_in, hw_out) -> np.ndarray:
    """Up(.) on a row-major (h, w) token grid, per channel: bilinear, half-pixel
    centres, source coordinate clamped at 0, neighbours clamped at the edge.
    F is [h_in*w_in][C]; returns [h_out*w_out][C].  Equal sizes give the identity."""
    h0, w0 = hw_in
    h1, w1 = hw_out
    C = F.shape[-1]
    G = F.reshape(h0, w0, C)
    out = np.empty((h1, w1, C), dtype=F.dtype)
    for y in range(h1):
        sy = max((y + 0.5) * h0 / h1 - 0.5, 0.0)
        y0 = min(int(math.floor(sy)), h0 - 1)
        y1 = min(y0 + 1, h0 - 1)
        fy = sy - y0
        for x in range(w1):
            sx = max((x + 0.5) * w0 / w1 - 0.5, 0.0)
            x0 = min(int(math.floor(sx)), w0 - 1)
            x1 = min(x0 + 1, w0 - 1)
            fx = sx - x0
            top = (1.0 - fx) * G[y0, x0] + fx * G[y0, x1]
            bot = (1.0 - fx) * G[y1, x0] + fx * G[y1, x1]
            out[y, x] = (1.0 - fy) * top + fy * bot
    return out.reshape(h1 * w1, C)


# --------------------------------------------------------------------------- between two scale steps
# Algorithm 1 ("Vanilla VAR" lines, the same in both stages), Eq. "var_upf" and Eq. "var_downf":
#   R_k = Q(F_k^o);  F_k = F_{k-1} + Up(R_k, (h_K, w_K));  next input = Down(F_k, (h_{k+1}, w_{k+1})).
# The paper leaves Q, Up and Down abstract (Algorithm 1 lists a codebook Z of V codewords of width d among the inputs of Q); here
# Q is the nearest codeword in Euclidean distance (ties: lowest code), Up is upsample_bilinear above and
# Down averages the source cells each target cell covers ("area" resampling).

def nearest_codeword(F_o: np.ndarray, Z: np.ndarray, dtype=np.float32) -> np.ndarray:
    """argmin_v ||F_o[i] - Z[v]||^2 for every row i, as argmax_v (F_o[i] . Z[v] - ||Z[v]||^2 / 2); the
    score that decides is taken in `dtype` (fp32: the precision the kernel decides in).  int32 [rows]."""
    F64, Z64 = np.asarray(F_o, dtype=np.float64), np.asarray(Z, dtype=np.float64)
    score = (F64 @ Z64.T).astype(dtype) - (0.5 * (Z64 * Z64).sum(axis=1)).astype(dtype)[None, :]
    return np.argmax(score, axis=1).astype(np.int32)          # first maximum = lowest code on ties


def downsample_area(F: np.ndarray, hw_in, hw_out) -> np.ndarray:
    """Down(.) on a row-major (h, w) grid, per channel: target cell (y, x) is the mean of the source cells
    [floor(y h_in / h_out), ceil((y + 1) h_in / h_out)) x [floor(x w_in / w_out), ceil((x + 1) w_in / w_out)).
    F is [h_in*w_in][C]; returns [h_out*w_out][C].  Equal sizes give the identity."""
    (h0, w0), (h1, w1) = hw_in, hw_out
    G = np.asarray(F, dtype=np.float64).reshape(h0, w0, -1)
    out = np.empty((h1, w1, G.shape[2]), dtype=np.float64)
    for y in range(h1):
        ya, yb = (y * h0) // h1, -((-(y + 1) * h0) // h1)
        for x in range(w1):
            xa, xb = (x * w0) // w1, -((-(x + 1) * w0) // w1)
            out[y, x] = G[ya:yb, xa:xb].mean(axis=(0, 1))
    return out.reshape(h1 * w1, -1)


def scale_transition(F_prev: np.ndarray, F_o: np.ndarray, Z: np.ndarray, hw_k, hw_K, hw_next):
    """One transition for one batch element.  F_prev [h_K*w_K][C] (F_{k-1}; zeros before the first
    scale), F_o [h_k*w_k][C] (the step's output), Z [V][C].  Returns (codes int32 [h_k*w_k], F_k
    [h_K*w_K][C], next tokens [h_next*w_next][C] or None when hw_next is None)."""
    codes = nearest_codeword(F_o, Z)
    R = np.asarray(Z, dtype=np.float64)[codes]
    F_k = np.asarray(F_prev, dtype=np.float64) + upsample_bilinear(R, hw_k, hw_K)
    nxt = downsample_area(F_k, hw_K, hw_next) if hw_next is not None else None
    return codes, F_k, nxt


def cfg_combine(F_prompt: np.ndarray, F_null: np.ndarray, s: float) -> np.ndarray:
    """Classifier-free guidance on the two branches of a CFG pair: F_null + s (F_prompt - F_null).  s = 0 is
    the null-prompt branch alone, which is what a CFG of 0 in the fidelity-refinement stage amounts to
    (Sec. 3.3: CFG = 0 amounts to running the null text prompt alone)."""
    a, b = np.asarray(F_prompt, dtype=np.float64), np.asarray(F_null, dtype=np.float64)
    return b + s * (a - b)


def rtr_restore(F_r_out: np.ndarray, idx: np.ndarray, cache_up: np.ndarray) -> np.ndarray:
    """Eq. "redefine": row idx[j] takes row j of the block output, every other row
    takes the upsampled cached row."""
    out = cache_up.copy()
    out[idx] = F_r_out
    return out


def lls_restoration_matrix(F_r: np.ndarray, F_full: np.ndarray) -> np.ndarray:
    """Eq. "lstsq" (Sec. 3.3 RP): the restoration matrix W in R^{M x r} that minimises || F_r^T W^T - F_full^T ||_F,
    i.e. the least-squares map from the r-row feature F_r [r][d] back to the M-row feature F_full [M][d].  With
    F_r of full row rank the normal equations give W = F_full F_r^T (F_r F_r^T)^-1; solved in fp64 through the
    Cholesky factor of the r x r Gram matrix."""
    F_r, F_full = np.asarray(F_r, dtype=np.float64), np.asarray(F_full, dtype=np.float64)
    assert F_r.shape[0] <= min(F_full.shape), "the r-row feature cannot have full row rank"
    G = F_r @ F_r.T
    L = np.linalg.cholesky(G)
    P = F_full @ F_r.T                                   # [M][r]
    Y = np.linalg.solve(L, P.T)                          # L Y = P^T
    return np.linalg.solve(L.T, Y).T                     # L^T W^T = Y


def lls_restore(F_r_out: np.ndarray, F_hat: np.ndarray, F_tilde: np.ndarray, Q: np.ndarray, cache_up: np.ndarray) -> np.ndarray:
    """The LLS restoration the paper tries before RTR (Sec. 3.3 RP, Eq. "lstsq"; App. A.3; Tab. "lowrank" row 5):
    F_k^o = W_r^o F_r^o with W_r^o ~ W_hat_r + W_r^{o,cache}.  W_hat_r restores the step's input from its projection
    (F_tilde from F_hat = Q^T F_tilde).  W_r^{o,cache} comes from a second least-squares problem posed on the cached
    counterpart feature; the paper does not name the r-row feature of that second problem -- read here as the
    projection of the cached feature by the same Q, Q^T Up(F_{k-1}^o), restored to Up(F_{k-1}^o).  The sum of the
    two matrices is taken as the paper writes it.  Both problems need their r-row feature of full row rank, so
    r <= min(M_{k-1}, d): bilinear upsampling does not raise the rank of the cached M_{k-1} rows."""
    W_hat = lls_restoration_matrix(F_hat, F_tilde)
    W_cache = lls_restoration_matrix(random_projection(Q, cache_up), cache_up)
    return (W_hat + W_cache) @ np.asarray(F_r_out, dtype=np.float64)


def rank_from_keep_ratio(M: int, rho: float) -> int:
    return max(1, min(M, int(math.floor(rho * M + 0.5))))


def rank_from_table_ratio(M: int, C: int, ratio: float) -> int:
    """r for a tabulated rank ratio: the ratio is of n = min(M, d) singular values
    (Sec. 3.2, low-rank paragraph)."""
    n = min(M, C)
    return max(1, min(M, int(math.floor(ratio * n + 0.5))))


def energy_rank(X: np.ndarray, alpha: float) -> int:
    """r = min{ r : eta_r >= alpha }, eta_r = sum_{i<=r} sigma_i^2 / sum_i sigma_i^2
    (Eq. "low_rank_percent")."""
    sv = np.linalg.svd(np.asarray(X, dtype=np.float64), compute_uv=False)
    eta = np.cumsum(sv ** 2) / np.sum(sv ** 2)
    return int(np.searchsorted(eta, alpha - 1e-15) + 1)


# Rank ratios per block chunk (rows) and late scale 40 / 48 / 64 (columns) of the
# Infinity backbone at alpha = 0.96 (App. A.1, rank table; means only).
INFINITY_RANK_RATIO = (
    (0.016, 0.013, 0.008),
    (0.136, 0.117, 0.054),
    (0.210, 0.189, 0.083),
    (0.250, 0.222, 0.066),
    (0.256, 0.234, 0.056),
    (0.198, 0.183, 0.029),
    (0.157, 0.134, 0.038),
    (0.191, 0.163, 0.055),
)

# --------------------------------------------------------------------------- the block


def block_forward(x: np.ndarray, ada6: np.ndarray, w: Dict[str, np.ndarray], K_cache: np.ndarray,
                  V_cache: np.ndarray, n_heads: int, eps: float, cross_kv=None,
                  query_rows: Optional[np.ndarray] = None):
    """One AdaLN transformer block on rows x [n][C].

    Keys/values are the committed cache rows followed by this call's own rows (no
    mask inside the scale).  Returns (x_out, k_new, v_new).  With query_rows the
    output is computed for that subset of rows only (keys still come from all rows).
    """
    sh1, sc1, g1, sh2, sc2, g2 = ada6
    C = x.shape[-1]
    y = modulate(x, sh1, sc1, eps)
    qkv = y @ w["w_qkv"].T + w["b_qkv"]
    q, k, v = qkv[:, :C], qkv[:, C:2 * C], qkv[:, 2 * C:]
    K_all = np.concatenate([K_cache, k], axis=0)
    V_all = np.concatenate([V_cache, v], axis=0)
    if query_rows is not None:
        x = x[query_rows]
        q = q[query_rows]
    a = attention(q, K_all, V_all, n_heads)
    x = x + g1 * (a @ w["w_o"].T + w["b_o"])
    if cross_kv is not None:
        Kc, Vc = cross_kv
        yc = layer_norm(x, eps) * w["ln_c_gamma"]
        qc = yc @ w["w_cq"].T
        x = x + attention(qc, Kc, Vc, n_heads) @ w["w_co"].T
    y = modulate(x, sh2, sc2, eps)
    hdn = gelu_tanh(y @ w["w_fc1"].T + w["b_fc1"])
    x = x + g2 * (hdn @ w["w_fc2"].T + w["b_fc2"])
    return x, k, v


# --------------------------------------------------------------------------- the step, with state


class Policy:
    """Per-call policy of a scale step (mirrors the C ABI's keep policy)."""

    def __init__(self, mode: str = "dense", cfg_mode: str = "pair", keep_ratio: float = 1.0,
                 rank_per_group: Optional[Sequence[int]] = None, forced_indices=None, sample_noise=None,
                 restore: str = "rtr"):
        assert mode in ("dense", "lowrank_rtr", "skip")
        assert restore in ("rtr", "lls")
        self.restore = restore                    # how the M rows come back from the r rows: RTR (the method) or LLS (variant 5)
        assert cfg_mode in ("pair", "null_only")
        self.mode, self.cfg_mode = mode, cfg_mode
        self.keep_ratio, self.rank_per_group = keep_ratio, rank_per_group
        self.forced_indices = forced_indices      # [B_eff][G] -> int array, or None
        self.sample_noise = sample_noise          # [G][B_eff][M] Exp(1) variates: sampled selection; None: top-r


class Oracle:
    """State across scale steps: weights, hoisted conditioning, the multi-scale KV
    cache per block and batch element, and the block-group outputs of the last
    stepped scale."""

    def __init__(self, weights: List[Dict[str, np.ndarray]], n_heads: int, blocks_per_group: int,
                 scale_hw: Sequence, ln_eps: float = 1e-6, dtype=np.float64):
        self.dt = dtype
        self.w = [{k: np.asarray(v, dtype=dtype) for k, v in blk.items()} for blk in weights]
        self.n_blocks = len(weights)
        self.bpg = blocks_per_group
        self.G = self.n_blocks // blocks_per_group
        self.H = n_heads
        self.hw = [tuple(x) for x in scale_hw]
        self.eps = ln_eps
        self.C = self.w[0]["w_o"].shape[0]
        self.cross = "w_cq" in self.w[0]
        self.reset()

    def reset(self):
        self.B = 0
        self.ada = None
        self.cross_kv = None
        self.K = self.V = None
        self.staged = None
        self.group_cache = None          # [G][B] -> [M][C] of scale self.cache_scale
        self.cache_scale = -1
        self.proj: Dict = {}
        self.last_indices = None

    def set_cond(self, cond: np.ndarray, context: Optional[np.ndarray] = None):
        cond = np.asarray(cond, dtype=self.dt)
        self.B = cond.shape[0]
        self.ada = [[ada_vectors(cond[b], w["w_ada"], w["b_ada"]) for b in range(self.B)] for w in self.w]
        C = self.C
        if self.cross:
            ctx = np.asarray(context, dtype=self.dt)
            self.cross_kv = []
            for w in self.w:
                per_b = []
                for b in range(self.B):
                    kv = ctx[b] @ w["w_ckv"].T
                    per_b.append((kv[:, :C], kv[:, C:]))
                self.cross_kv.append(per_b)
        empty = np.zeros((0, C), dtype=self.dt)
        self.K = [[empty for _ in range(self.B)] for _ in range(self.n_blocks)]
        self.V = [[empty for _ in range(self.B)] for _ in range(self.n_blocks)]
        self.staged = None

    def set_projection(self, scale_idx: int, group: int, Q: np.ndarray):
        self.proj[(scale_idx, group)] = np.asarray(Q, dtype=self.dt)

    def load_kv(self, K: np.ndarray, V: np.ndarray):
        """Stand-in earlier scales: K, V [n_blocks][B][L][C] become the committed cache."""
        for blk in range(self.n_blocks):
            for b in range(self.B):
                self.K[blk][b] = np.asarray(K[blk][b], dtype=self.dt)
                self.V[blk][b] = np.asarray(V[blk][b], dtype=self.dt)

    def load_group_cache(self, scale_idx: int, cache: np.ndarray):
        """Stand-in block-group outputs of scale scale_idx: [G][B][M][C]."""
        self.group_cache = [[np.asarray(cache[g][b], dtype=self.dt) for b in range(self.B)]
                            for g in range(self.G)]
        self.cache_scale = scale_idx

    def ranks(self, M: int, pol: Policy) -> List[int]:
        if pol.mode == "dense":
            return [M] * self.G
        if pol.rank_per_group is not None:
            return [int(r) for r in pol.rank_per_group]
        return [rank_from_keep_ratio(M, pol.keep_ratio)] * self.G

    def scale_step(self, tokens: np.ndarray, scale_idx: int, pol: Policy) -> Optional[np.ndarray]:
        """One scale step.  tokens [B][M][C]; returns [B_eff][M][C] (None for skip)."""
        if pol.mode == "skip":
            return None
        tokens = np.asarray(tokens, dtype=self.dt)
        B, M, C = tokens.shape
        assert B == self.B and M == self.hw[scale_idx][0] * self.hw[scale_idx][1]
        elems = list(range(B)) if pol.cfg_mode == "pair" else list(range(1, B, 2))
        ranks = self.ranks(M, pol)
        new_cache = [[None] * B for _ in range(self.G)]
        staged = [[None] * B for _ in range(self.n_blocks)]
        indices = [[None] * self.G for _ in elems]
        outs = []
        for e, b in enumerate(elems):
            X = tokens[b]
            for g in range(self.G):
                r = ranks[g]
                blocks = range(g * self.bpg, (g + 1) * self.bpg)
                if r >= M:                                 # dense: Q = I, I = all rows
                    x = X
                    idx = np.arange(M, dtype=np.int32)
                else:
                    if pol.restore == "lls":
                        idx = np.zeros(0, dtype=np.int32)  # no index set: every row comes from W F_r^o
                    elif pol.forced_indices is not None:
                        idx = np.asarray(pol.forced_indices[e][g], dtype=np.int32)
                    elif pol.sample_noise is not None:
                        idx = select_top_r(sampling_keys(row_scores(X, np.float32), pol.sample_noise[g][e]), r)
                    else:
                        idx = select_top_r(row_scores(X, np.float32), r)
                    x = random_projection(self.proj[(scale_idx, g)], X)
                    x_hat = x
                for blk in blocks:
                    ckv = self.cross_kv[blk][b] if self.cross else None
                    x, k, v = block_forward(x, self.ada[blk][b], self.w[blk], self.K[blk][b],
                                            self.V[blk][b], self.H, self.eps, ckv)
                    staged[blk][b] = (k, v)
                if r >= M:
                    out = x
                else:
                    assert self.group_cache is not None and self.cache_scale >= 0
                    up = upsample_bilinear(self.group_cache[g][b], self.hw[self.cache_scale],
                                           self.hw[scale_idx])
                    out = (lls_restore(x, x_hat, X, self.proj[(scale_idx, g)], up) if pol.restore == "lls"
                           else rtr_restore(x, idx, up))
                indices[e][g] = idx
                new_cache[g][b] = out
                X = out
            outs.append(X)
        # elements not computed keep no cache entry for this scale
        self.group_cache = new_cache
        self.cache_scale = scale_idx
        self.staged = (scale_idx, staged)
        self.last_indices = indices
        return np.stack(outs, axis=0)

    def kv_append(self, scale_idx: int):
        """Commit the rows the last step staged (per block: the r rows its group computed)."""
        assert self.staged is not None and self.staged[0] == scale_idx
        for blk in range(self.n_blocks):
            for b in range(self.B):
                if self.staged[1][blk][b] is not None:
                    k, v = self.staged[1][blk][b]
                    self.K[blk][b] = np.concatenate([self.K[blk][b], k], axis=0)
                    self.V[blk][b] = np.concatenate([self.V[blk][b], v], axis=0)
        self.staged = None

    def cache_len(self, blk: int, b: int) -> int:
        return self.K[blk][b].shape[0]
