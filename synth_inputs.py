"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke check.

This module only draws random numbers and shapes them; it holds none of the
method's arithmetic.  Everything is generated with numpy's PCG64 from one
64-bit seed, in fp32, and rounded to the nearest bf16 value (ties to even) so
that the CPU oracle and the GPU library receive bit-identical operands.

Stand-in recipe (trained VAR / Infinity weights and the prompt benchmarks are
not available offline): weights and biases N(0, 0.02^2), tokens, conditioning
vectors and context tokens N(0, 1), earlier-scale K/V rows N(0, 1), projection
matrix Q with entries N(0, 1/r).  A second, "spread" token distribution has a
decaying singular spectrum and log-normal row scales so that row norms are
well separated.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

VAR_SCALES: Tuple[int, ...] = (1, 2, 3, 4, 5, 6, 8, 10, 13, 16)
INFINITY_SCALES: Tuple[int, ...] = (1, 2, 4, 6, 8, 12, 16, 20, 24, 32, 40, 48, 64)


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round an fp32 array to the nearest bf16-representable fp32 values."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    r = (u + bias) & np.uint32(0xFFFF0000)
    nan = np.isnan(a)
    if nan.any():
        r = np.where(nan, np.uint32(0x7FC00000), r)
    return r.view(np.float32)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of an array that already holds bf16-representable values."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(rng: np.random.Generator, shape, std: float = 1.0) -> np.ndarray:
    x = rng.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return round_to_bf16(x)


@dataclasses.dataclass
class ModelShape:
    """Static shape of a block stack (the fields the C ABI's fvar_cfg carries)."""
    n_blocks: int
    blocks_per_group: int
    width: int
    n_heads: int
    head_dim: int
    ffn_dim: int
    scales: Tuple[int, ...]            # side length per scale (square maps) ...
    scale_hw: Optional[Tuple[Tuple[int, int], ...]] = None   # ... or explicit (h, w)
    has_cross_attn: bool = False
    ctx_len: int = 0
    ctx_width: int = 0
    ln_eps: float = 1e-6

    def hw(self) -> List[Tuple[int, int]]:
        if self.scale_hw is not None:
            return [tuple(x) for x in self.scale_hw]
        return [(s, s) for s in self.scales]

    def tokens_per_scale(self) -> List[int]:
        return [h * w for h, w in self.hw()]

    @property
    def n_groups(self) -> int:
        return self.n_blocks // self.blocks_per_group


def shape_var_d16(n_blocks: int = 16, blocks_per_group: int = 1) -> ModelShape:
    return ModelShape(n_blocks, blocks_per_group, 1024, 16, 64, 4096, VAR_SCALES)


def shape_var_d30(n_blocks: int = 30, blocks_per_group: int = 1) -> ModelShape:
    return ModelShape(n_blocks, blocks_per_group, 1920, 30, 64, 7680, VAR_SCALES)


def shape_infinity_2b(n_blocks: int = 32, blocks_per_group: int = 4) -> ModelShape:
    return ModelShape(n_blocks, blocks_per_group, 2048, 16, 128, 8192, INFINITY_SCALES,
                      has_cross_attn=True, ctx_len=256, ctx_width=2048)


def shape_tiny(n_blocks: int = 2, blocks_per_group: int = 1, width: int = 128, n_heads: int = 2,
               head_dim: int = 64, ffn_dim: int = 256, scales: Sequence[int] = (1, 2, 3, 5),
               cross: bool = False, ctx_len: int = 8, scale_hw=None) -> ModelShape:
    return ModelShape(n_blocks, blocks_per_group, width, n_heads, head_dim, ffn_dim, tuple(scales),
                      scale_hw=scale_hw, has_cross_attn=cross, ctx_len=ctx_len if cross else 0,
                      ctx_width=width if cross else 0)


WEIGHT_NAMES = ("w_qkv", "b_qkv", "w_o", "b_o", "w_fc1", "b_fc1", "w_fc2", "b_fc2", "w_ada", "b_ada")
CROSS_NAMES = ("w_cq", "w_ckv", "w_co", "ln_c_gamma")


def make_block_weights(rng: np.random.Generator, shp: ModelShape, std: float = 0.02) -> Dict[str, np.ndarray]:
    """One block's parameters; every matrix is stored [out_features][in_features]."""
    C, F = shp.width, shp.ffn_dim
    w = {
        "w_qkv": normal_bf16(rng, (3 * C, C), std), "b_qkv": normal_bf16(rng, (3 * C,), std),
        "w_o": normal_bf16(rng, (C, C), std), "b_o": normal_bf16(rng, (C,), std),
        "w_fc1": normal_bf16(rng, (F, C), std), "b_fc1": normal_bf16(rng, (F,), std),
        "w_fc2": normal_bf16(rng, (C, F), std), "b_fc2": normal_bf16(rng, (C,), std),
        "w_ada": normal_bf16(rng, (6 * C, C), std), "b_ada": normal_bf16(rng, (6 * C,), std),
    }
    if shp.has_cross_attn:
        w["w_cq"] = normal_bf16(rng, (C, C), std)
        w["w_ckv"] = normal_bf16(rng, (2 * C, shp.ctx_width), std)
        w["w_co"] = normal_bf16(rng, (C, C), std)
        w["ln_c_gamma"] = round_to_bf16(1.0 + 0.1 * rng.standard_normal(C, dtype=np.float32))
    return w


def make_weights(seed: int, shp: ModelShape, std: float = 0.02) -> List[Dict[str, np.ndarray]]:
    rng = np.random.default_rng([seed, 1])
    return [make_block_weights(rng, shp, std) for _ in range(shp.n_blocks)]


def make_tokens(seed: int, B: int, M: int, C: int, kind: str = "normal") -> np.ndarray:
    """Token rows [B][M][C].  kind = "normal": N(0,1); "spread": low-rank-plus-noise rows with
    log-normal row scales (row norms well separated, energy concentrated in few directions)."""
    rng = np.random.default_rng([seed, 2, M])
    if kind == "normal":
        return normal_bf16(rng, (B, M, C))
    if kind == "spread":
        n = min(M, C)
        inner = max(1, int(round(0.176 * n)))
        out = np.empty((B, M, C), dtype=np.float32)
        for b in range(B):
            A = rng.standard_normal((M, inner), dtype=np.float32)
            decay = (1.0 / np.sqrt(1.0 + np.arange(inner, dtype=np.float32)))
            Bm = rng.standard_normal((inner, C), dtype=np.float32)
            row_scale = np.exp(0.5 * rng.standard_normal((M, 1), dtype=np.float32))
            x = (A * decay) @ Bm / np.float32(np.sqrt(np.sum(decay ** 2)))
            out[b] = row_scale * x + np.float32(0.05) * rng.standard_normal((M, C), dtype=np.float32)
        return round_to_bf16(out)
    raise ValueError(kind)


def make_cond(seed: int, B: int, C: int) -> np.ndarray:
    return normal_bf16(np.random.default_rng([seed, 3]), (B, C))


def make_context(seed: int, B: int, ctx_len: int, ctx_width: int) -> np.ndarray:
    return normal_bf16(np.random.default_rng([seed, 4]), (B, ctx_len, ctx_width))


def make_projection(seed: int, scale_idx: int, group: int, M: int, r: int) -> np.ndarray:
    """Q in R^{M x r}, entries N(0, 1/r), bf16-rounded.  One matrix per (scale, group), shared by the batch."""
    rng = np.random.default_rng([seed, 5, scale_idx, group])
    return normal_bf16(rng, (M, r), 1.0 / np.sqrt(r))


def make_kv_prefill(seed: int, n_blocks: int, B: int, L: int, C: int) -> Tuple[np.ndarray, np.ndarray]:
    """Stand-in K and V rows of the earlier scales: [n_blocks][B][L][C] each, N(0,1)."""
    rng = np.random.default_rng([seed, 6])
    return normal_bf16(rng, (n_blocks, B, L, C)), normal_bf16(rng, (n_blocks, B, L, C))


def make_group_cache(seed: int, G: int, B: int, M_prev: int, C: int) -> np.ndarray:
    """Stand-in for the previous scale's block-group outputs: [G][B][M_prev][C], N(0,1) in fp32."""
    rng = np.random.default_rng([seed, 7])
    return rng.standard_normal((G, B, M_prev, C), dtype=np.float32)


def make_sample_noise(seed: int, scale_idx: int, G: int, B_eff: int, M: int) -> np.ndarray:
    """Exp(1) variates [G][B_eff][M] (fp32) for the sampled row selection; one draw per (scale, group, element, row)."""
    rng = np.random.default_rng([seed, 8, scale_idx])
    return rng.standard_exponential(size=(G, B_eff, M)).astype(np.float32) + np.float32(1e-30)


def make_codebook(seed: int, V: int, C: int) -> np.ndarray:
    """Quantizer codebook Z [V][C], entries N(0, 1), bf16-rounded (stands in for a trained codebook)."""
    return normal_bf16(np.random.default_rng([seed, 9]), (V, C))


def make_step_outputs(seed: int, scale_idx: int, B: int, M: int, Z: np.ndarray, noise: float) -> np.ndarray:
    """Stand-in block outputs F_k^o [B][M][C] for the transition between steps: a randomly chosen codeword per
    token plus N(0, noise^2), bf16-rounded.  Small noise keeps every token's nearest codeword well separated;
    noise >= 1 gives generic rows with near ties."""
    rng = np.random.default_rng([seed, 10, scale_idx])
    pick = rng.integers(0, Z.shape[0], size=(B, M))
    return round_to_bf16(Z[pick] + noise * rng.standard_normal((B, M, Z.shape[1]), dtype=np.float32))
