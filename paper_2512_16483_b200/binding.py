"""ctypes binding of libfvar (include/fvar.h).  Argument marshalling only: every step of the
path runs inside the library's CUDA kernels.  torch supplies device memory and the stream.

The library is loaded from this package's directory; loading fails loudly when it has not been
built (python -m paper_2512_16483_b200.build) -- there is no fallback path.
"""
from __future__ import annotations

import ctypes as ct
import os
from typing import Dict, List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfvar.so")

OK, EINVAL, ENOMEM, ESTATE, ECUDA, ETIMEOUT, EUNSUPPORTED = range(7)
DENSE, LOWRANK_RTR, SKIP = 0, 1, 2
CFG_PAIR, CFG_NULL_ONLY = 0, 1
SELECT_TOPR, SELECT_SAMPLE = 0, 1
RESTORE_RTR, RESTORE_LLS = 0, 1
OPT_CUDA_GRAPHS, OPT_GEMM_MAX_SPLITS, OPT_SKINNY_MAX_ROWS, OPT_WAIT_KCYCLES = 0, 1, 2, 3
GEMM_AUTO, GEMM_SINGLE, GEMM_PAIR, GEMM_SKINNY, GEMM_KSPLIT = 0, 1, 2, 3, 4
KCLASSES = ("gemm", "attention", "ln_modulate", "row_scores", "select_topr", "rtr_fill", "convert")
STATUS_NAMES = ("FVAR_OK", "FVAR_EINVAL", "FVAR_ENOMEM", "FVAR_ESTATE", "FVAR_ECUDA", "FVAR_ETIMEOUT",
                "FVAR_EUNSUPPORTED")


class FvarError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__("%s: %s" % (STATUS_NAMES[status] if 0 <= status < 7 else status, msg))
        self.status = status


class _Cfg(ct.Structure):
    _fields_ = [("n_blocks", ct.c_int), ("blocks_per_group", ct.c_int), ("width", ct.c_int), ("n_heads", ct.c_int),
                ("head_dim", ct.c_int), ("ffn_dim", ct.c_int), ("n_scales", ct.c_int),
                ("scale_hw", ct.POINTER(ct.c_int)), ("max_batch", ct.c_int), ("has_cross_attn", ct.c_int),
                ("ctx_len", ct.c_int), ("ctx_width", ct.c_int), ("ln_eps", ct.c_float)]


_WEIGHT_FIELDS = ("w_qkv", "b_qkv", "w_o", "b_o", "w_fc1", "b_fc1", "w_fc2", "b_fc2", "w_ada", "b_ada",
                  "w_cq", "w_ckv", "w_co", "ln_c_gamma")


class _Weights(ct.Structure):
    _fields_ = [(n, ct.POINTER(ct.c_void_p)) for n in _WEIGHT_FIELDS]


class _Policy(ct.Structure):
    _fields_ = [("mode", ct.c_int), ("cfg_mode", ct.c_int), ("rank_per_group", ct.POINTER(ct.c_int)),
                ("keep_ratio", ct.c_float), ("forced_indices", ct.c_void_p), ("select", ct.c_int),
                ("sample_noise", ct.c_void_p), ("restore", ct.c_int)]


_lib = None


def load_library() -> ct.CDLL:
    """Loads libfvar.so and declares every prototype of include/fvar.h."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError("libfvar.so is not built: run `python -m paper_2512_16483_b200.build` "
                                "(needs nvcc; there is no CPU fallback)")
    lib = ct.CDLL(LIB_PATH)
    vp, i, f, ll = ct.c_void_p, ct.c_int, ct.c_float, ct.c_longlong
    P = ct.POINTER
    sigs = {
        "fvar_workspace_bytes": (ct.c_size_t, [P(_Cfg)]),
        "fvar_init": (i, [P(_Weights), P(_Cfg), vp, ct.c_size_t, vp, P(vp)]),
        "fvar_set_cond": (i, [vp, i, vp, vp]),
        "fvar_set_projection": (i, [vp, i, i, vp, i]),
        "fvar_generate_projection": (i, [vp, i, i, i, ct.c_ulonglong]),
        "fvar_set_codebook": (i, [vp, vp, i]),
        "fvar_scale_transition": (i, [vp, vp, i, i, vp, vp]),
        "fvar_scale_transition_pairs": (i, [vp, vp, i, i, vp, vp]),
        "fvar_get_feature": (i, [vp, vp]),
        "fvar_cfg_combine": (i, [vp, i, ll, f, vp, vp]),
        "fvar_get_projection": (i, [vp, i, i, vp, P(i)]),
        "fvar_scale_step": (i, [vp, vp, i, P(_Policy), vp]),
        "fvar_scale_step_host": (i, [vp, vp, i, P(_Policy), vp]),
        "fvar_scale_step_host_async": (i, [vp, vp, i, P(_Policy), vp]),
        "fvar_host_sync": (i, [vp]),
        "fvar_kv_append": (i, [vp, i]),
        "fvar_get_indices": (i, [vp, i, vp, P(i)]),
        "fvar_get_group_output": (i, [vp, i, vp]),
        "fvar_load_kv": (i, [vp, vp, vp, i]),
        "fvar_load_group_cache": (i, [vp, i, vp]),
        "fvar_cache_len": (i, [vp, i]),
        "fvar_launch_count": (ll, [vp]),
        "fvar_poll_status": (i, [vp]),
        "fvar_reset": (i, [vp]),
        "fvar_restore_loaded": (i, [vp]),
        "fvar_set_option": (i, [vp, i, i]),
        "fvar_profile_enable": (i, [vp, i]),
        "fvar_profile_read": (i, [vp, i, P(ct.c_double), P(ll), P(ct.c_double), P(ct.c_double)]),
        "fvar_profile_dump": (i, [vp, i, P(ct.c_float), i, P(i)]),
        "fvar_destroy": (None, [vp]),
        "fvar_last_error": (ct.c_char_p, [vp]),
        "fvar_row_scores": (i, [vp, i, i, i, vp, vp]),
        "fvar_row_keys": (i, [vp, vp, i, i, i, vp, vp]),
        "fvar_select_topr": (i, [vp, i, i, i, vp, vp, vp]),
        "fvar_ln_modulate": (i, [vp, i, i, i, vp, vp, ll, f, vp, vp]),
        "fvar_gemm_bf16": (i, [vp, vp, vp, i, i, i, vp, vp]),
        "fvar_gemm_bf16_form": (i, [vp, vp, vp, i, i, i, i, i, vp, vp]),
        "fvar_gemm_bf16_wt": (i, [vp, vp, vp, i, i, i, i, vp, vp]),
        "fvar_attention": (i, [vp, vp, vp, i, i, i, i, i, i, vp, vp]),
        "fvar_rtr_fill": (i, [vp, i, i, i, i, i, i, vp, vp, vp]),
        "fvar_select_rows_static": (i, [vp, i, i, i, i, vp, vp, vp]),
        "fvar_l2_prefetch": (i, [vp, ct.c_size_t, vp]),
        "fvar_selftest_wait_timeout": (i, [vp, ll, vp]),
        "fvar_rank_from_keep_ratio": (i, [i, f]),
        "fvar_rank_from_table_ratio": (i, [i, i, ct.c_double]),
        "fvar_infinity_rank_ratio": (i, [i, i, P(ct.c_double)]),
        "fvar_infinity_group_ranks": (i, [i, i, i, P(i)]),
        "fvar_infinity_schedule": (i, [i, i, P(i), P(i), P(i)]),
    }
    for name, (res, args) in sigs.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


EXPORTED = ("fvar_workspace_bytes", "fvar_init", "fvar_set_cond", "fvar_set_projection", "fvar_generate_projection",
            "fvar_get_projection", "fvar_set_codebook", "fvar_scale_transition", "fvar_scale_transition_pairs", "fvar_get_feature", "fvar_scale_step",
            "fvar_scale_step_host", "fvar_scale_step_host_async", "fvar_host_sync", "fvar_kv_append", "fvar_get_indices", "fvar_get_group_output", "fvar_load_kv",
            "fvar_load_group_cache", "fvar_cache_len", "fvar_launch_count", "fvar_poll_status", "fvar_reset",
            "fvar_destroy", "fvar_last_error", "fvar_restore_loaded", "fvar_set_option", "fvar_profile_enable", "fvar_profile_read", "fvar_profile_dump",
            "fvar_row_scores", "fvar_row_keys", "fvar_select_topr", "fvar_ln_modulate",
            "fvar_gemm_bf16", "fvar_gemm_bf16_form", "fvar_gemm_bf16_wt", "fvar_cfg_combine", "fvar_attention", "fvar_rtr_fill", "fvar_select_rows_static", "fvar_l2_prefetch", "fvar_selftest_wait_timeout",
            "fvar_rank_from_keep_ratio", "fvar_rank_from_table_ratio", "fvar_infinity_rank_ratio", "fvar_infinity_group_ranks",
            "fvar_infinity_schedule")


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _check_kernel(status: int):
    if status != OK:
        raise FvarError(status, (load_library().fvar_last_error(None) or b"").decode())


def _dev(t: torch.Tensor, dtype) -> torch.Tensor:
    assert t.is_cuda and t.dtype == dtype and t.is_contiguous(), (t.device, t.dtype, t.is_contiguous())
    return t


# ------------------------------------------------------------------------------------ kernel-level calls

def fvar_row_scores(x: torch.Tensor) -> torch.Tensor:
    """x fp32 [B][M][C] -> scores fp32 [B][M]."""
    _dev(x, torch.float32)
    B, M, C = x.shape
    s = torch.empty((B, M), dtype=torch.float32, device=x.device)
    _check_kernel(load_library().fvar_row_scores(x.data_ptr(), B, M, C, s.data_ptr(), _stream()))
    return s


def fvar_row_keys(x: torch.Tensor, noise: torch.Tensor) -> torch.Tensor:
    """x fp32 [B][M][C], noise fp32 [B][M] (Exp(1) variates) -> sampling keys fp32 [B][M] = score / noise."""
    _dev(x, torch.float32), _dev(noise, torch.float32)
    B, M, C = x.shape
    k = torch.empty((B, M), dtype=torch.float32, device=x.device)
    _check_kernel(load_library().fvar_row_keys(x.data_ptr(), noise.data_ptr(), B, M, C, k.data_ptr(), _stream()))
    return k


def fvar_select_topr(scores: torch.Tensor, r: int):
    """scores fp32 [B][M] -> (idx int32 [B][r] ascending, inv int32 [B][M])."""
    _dev(scores, torch.float32)
    B, M = scores.shape
    idx = torch.empty((B, r), dtype=torch.int32, device=scores.device)
    inv = torch.empty((B, M), dtype=torch.int32, device=scores.device)
    _check_kernel(load_library().fvar_select_topr(scores.data_ptr(), B, M, r, idx.data_ptr(), inv.data_ptr(), _stream()))
    return idx, inv


def fvar_ln_modulate(x: torch.Tensor, shift: torch.Tensor, scale: torch.Tensor, eps: float) -> torch.Tensor:
    """x fp32 [B][n][C], shift/scale fp32 [B][C] -> bf16 [B][n][C]."""
    _dev(x, torch.float32), _dev(shift, torch.float32), _dev(scale, torch.float32)
    B, n, C = x.shape
    y = torch.empty((B, n, C), dtype=torch.bfloat16, device=x.device)
    _check_kernel(load_library().fvar_ln_modulate(x.data_ptr(), B * n, C, n, shift.data_ptr(), scale.data_ptr(), C,
                                                  eps, y.data_ptr(), _stream()))
    return y


def fvar_gemm_bf16(A: torch.Tensor, W: torch.Tensor, bias: Optional[torch.Tensor] = None) -> torch.Tensor:
    """A bf16 [R][K], W bf16 [N][K], bias bf16 [N] -> fp32 [R][N] = A W^T + bias."""
    return fvar_gemm_bf16_form(A, W, bias, GEMM_AUTO, 0)


def fvar_gemm_bf16_form(A: torch.Tensor, W: torch.Tensor, bias: Optional[torch.Tensor], form: int, block_n: int) -> torch.Tensor:
    """fvar_gemm_bf16 with the launch form (GEMM_AUTO / GEMM_SINGLE / GEMM_PAIR) and tile width given."""
    _dev(A, torch.bfloat16), _dev(W, torch.bfloat16)
    R, K = A.shape
    N = W.shape[0]
    out = torch.empty((R, N), dtype=torch.float32, device=A.device)
    _check_kernel(load_library().fvar_gemm_bf16_form(A.data_ptr(), W.data_ptr(), _ptr(bias), R, N, K, form, block_n,
                                                     out.data_ptr(), _stream()))
    return out


def fvar_gemm_bf16_wt(A: torch.Tensor, Wt: torch.Tensor, bias: Optional[torch.Tensor] = None, block_n: int = 0) -> torch.Tensor:
    """A bf16 [R][K], Wt bf16 [K][N] (the second operand transposed, row-major) -> fp32 [R][N] = A Wt + bias."""
    _dev(A, torch.bfloat16), _dev(Wt, torch.bfloat16)
    R, K = A.shape
    N = Wt.shape[1]
    out = torch.empty((R, N), dtype=torch.float32, device=A.device)
    _check_kernel(load_library().fvar_gemm_bf16_wt(A.data_ptr(), Wt.data_ptr(), _ptr(bias), R, N, K, block_n, out.data_ptr(), _stream()))
    return out


def fvar_cfg_combine(pair: torch.Tensor, guidance: float) -> torch.Tensor:
    """pair bf16 [B][...] with elements (2p, 2p + 1) = (prompt, null) -> bf16 [B / 2][...] = null + guidance (prompt - null)."""
    _dev(pair, torch.bfloat16)
    B = pair.shape[0]
    per = pair[0].numel()
    out = torch.empty((B // 2,) + tuple(pair.shape[1:]), dtype=torch.bfloat16, device=pair.device)
    _check_kernel(load_library().fvar_cfg_combine(pair.data_ptr(), B, per, float(guidance), out.data_ptr(), _stream()))
    return out


def fvar_attention(q: torch.Tensor, Kc: torch.Tensor, Vt: torch.Tensor, L: int) -> torch.Tensor:
    """q bf16 [B][r][H*D], Kc bf16 [B][H][L_cap][D], Vt bf16 [B][H][D][L_cap] -> bf16 [B][r][H*D]."""
    _dev(q, torch.bfloat16), _dev(Kc, torch.bfloat16), _dev(Vt, torch.bfloat16)
    B, H, L_cap, D = Kc.shape
    r = q.shape[1]
    out = torch.empty_like(q)
    _check_kernel(load_library().fvar_attention(q.data_ptr(), Kc.data_ptr(), Vt.data_ptr(), B, H, r, D, L, L_cap,
                                                out.data_ptr(), _stream()))
    return out


def fvar_rtr_fill(prev: torch.Tensor, hw_in, hw_out, inv: Optional[torch.Tensor], out: torch.Tensor) -> torch.Tensor:
    """Fills rows of out fp32 [B][h1*w1][C] whose inv < 0 with the upsampled rows of prev fp32 [B][h0*w0][C]."""
    _dev(prev, torch.float32), _dev(out, torch.float32)
    B, _, C = prev.shape
    _check_kernel(load_library().fvar_rtr_fill(prev.data_ptr(), B, hw_in[0], hw_in[1], hw_out[0], hw_out[1], C,
                                               _ptr(inv), out.data_ptr(), _stream()))
    return out


def fvar_select_rows_static(x: torch.Tensor, r: int, idx: torch.Tensor, inv: torch.Tensor):
    """Top-r row selection of x fp32 [B][M][C] into caller-provided idx int32 [B][r] and inv int32 [B][M],
    with the intermediate scores kept in the library's built-in array: nothing is allocated, here or in
    the library.  For callers whose device memory is fully planned by someone else."""
    _dev(x, torch.float32), _dev(idx, torch.int32), _dev(inv, torch.int32)
    B, M, C = x.shape
    assert idx.shape == (B, r) and inv.shape == (B, M)
    _check_kernel(load_library().fvar_select_rows_static(x.data_ptr(), B, M, C, r, idx.data_ptr(), inv.data_ptr(), _stream()))


def kernel_poll_status() -> int:
    """Synchronises and returns the status of the kernel-level calls (FVAR_OK / FVAR_ETIMEOUT)."""
    return load_library().fvar_poll_status(None)


# ------------------------------------------------------------------------------------ the context

class Fvar:
    """One block stack on one GPU.  `weights` is a list (per block) of dicts of bf16 CUDA tensors
    named as in include/fvar.h; `scale_hw` a list of (h, w)."""

    def __init__(self, weights: List[Dict[str, torch.Tensor]], *, blocks_per_group: int, n_heads: int, head_dim: int,
                 ffn_dim: int, scale_hw: Sequence, max_batch: int, ctx_len: int = 0, ctx_width: int = 0,
                 ln_eps: float = 1e-6):
        self.lib = load_library()
        self.ctx = ct.c_void_p(None)
        self.weights = weights                       # keeps the tensors alive
        width = weights[0]["w_o"].shape[0]
        cross = "w_cq" in weights[0]
        hw = [int(v) for pair in scale_hw for v in pair]
        self._hw = (ct.c_int * len(hw))(*hw)
        self.scale_hw = [tuple(p) for p in scale_hw]
        self.n_groups = len(weights) // blocks_per_group
        self.width, self.max_batch = width, max_batch
        self._cfg = _Cfg(len(weights), blocks_per_group, width, n_heads, head_dim, ffn_dim, len(scale_hw),
                         ct.cast(self._hw, ct.POINTER(ct.c_int)), max_batch, int(cross), ctx_len, ctx_width, ln_eps)
        nbytes = self.lib.fvar_workspace_bytes(ct.byref(self._cfg))
        if nbytes == 0:
            raise FvarError(EINVAL, "unsupported shape")
        self.workspace = torch.empty(nbytes + 1024, dtype=torch.uint8, device="cuda")
        base = (self.workspace.data_ptr() + 1023) // 1024 * 1024
        w = _Weights()
        self._arrays = []
        for name in _WEIGHT_FIELDS:
            if name in weights[0]:
                for blk in weights:
                    _dev(blk[name], torch.bfloat16)
                arr = (ct.c_void_p * len(weights))(*[blk[name].data_ptr() for blk in weights])
                self._arrays.append(arr)
                setattr(w, name, ct.cast(arr, ct.POINTER(ct.c_void_p)))
        self._stream = _stream()
        st = self.lib.fvar_init(ct.byref(w), ct.byref(self._cfg), base, nbytes, self._stream, ct.byref(self.ctx))
        if st != OK:
            raise FvarError(st, (self.lib.fvar_last_error(None) or b"").decode())
        self.B = 0

    def _check(self, st: int):
        if st != OK:
            raise FvarError(st, (self.lib.fvar_last_error(self.ctx) or b"").decode())

    def close(self):
        if self.ctx:
            self.lib.fvar_destroy(self.ctx)
            self.ctx = ct.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_cond(self, cond: torch.Tensor, context: Optional[torch.Tensor] = None):
        _dev(cond, torch.bfloat16)
        self.B = cond.shape[0]
        self._check(self.lib.fvar_set_cond(self.ctx, self.B, cond.data_ptr(), _ptr(context)))

    def set_projection(self, scale_idx: int, group: int, Qt: torch.Tensor):
        """Qt bf16 [r][M]: the projection matrix of Sec. 3.3, transposed."""
        _dev(Qt, torch.bfloat16)
        self._check(self.lib.fvar_set_projection(self.ctx, scale_idx, group, Qt.data_ptr(), Qt.shape[0]))

    def generate_projection(self, scale_idx: int, group: int, r: int, seed: int):
        """Draws the projection of (scale, group) on the device from a 64-bit seed (Philox4x32-10 + Box-Muller)."""
        self._check(self.lib.fvar_generate_projection(self.ctx, scale_idx, group, r, seed & 0xFFFFFFFFFFFFFFFF))

    def get_projection(self, scale_idx: int, group: int, M: int) -> torch.Tensor:
        """The stored projection of (scale, group), transposed: bf16 [r][M] (M = tokens of that scale)."""
        buf = torch.empty((M, M), dtype=torch.bfloat16, device="cuda")
        r = ct.c_int(0)
        self._check(self.lib.fvar_get_projection(self.ctx, scale_idx, group, buf.data_ptr(), ct.byref(r)))
        return buf.view(-1)[: r.value * M].view(r.value, M)

    def set_codebook(self, Z: torch.Tensor):
        """Z bf16 [V][C]: the quantizer's codebook (kept by reference)."""
        _dev(Z, torch.bfloat16)
        self._codebook = Z
        self._check(self.lib.fvar_set_codebook(self.ctx, Z.data_ptr(), Z.shape[0]))

    def scale_transition(self, fo: torch.Tensor, scale_idx: int, next_M: Optional[int], pairs: bool = False):
        """fo bf16 [B][M_k][C] -> (codes int32 [B][M_k], next tokens bf16 [B][next_M][C] or None at the last scale).
        pairs: the next tokens come out as [2 B][next_M][C], every image's rows twice (both branches of its CFG pair)."""
        _dev(fo, torch.bfloat16)
        B, M, C = fo.shape
        codes = torch.empty((B, M), dtype=torch.int32, device=fo.device)
        nxt = torch.empty(((2 * B if pairs else B), next_M, C), dtype=torch.bfloat16, device=fo.device) if next_M else None
        fn = self.lib.fvar_scale_transition_pairs if pairs else self.lib.fvar_scale_transition
        self._check(fn(self.ctx, fo.data_ptr(), scale_idx, B, codes.data_ptr(), _ptr(nxt)))
        return codes, nxt

    def get_feature(self, B: int, M_last: int, C: int) -> torch.Tensor:
        """The accumulated feature map F_k: fp32 [B][M_last][C]."""
        out = torch.empty((B, M_last, C), dtype=torch.float32, device="cuda")
        self._check(self.lib.fvar_get_feature(self.ctx, out.data_ptr()))
        return out

    def _policy(self, mode, cfg_mode, keep_ratio, rank_per_group, forced_indices, sample_noise=None, restore=RESTORE_RTR):
        pol = _Policy(mode, cfg_mode, None, float(keep_ratio), None, SELECT_TOPR, None, int(restore))
        if sample_noise is not None:
            _dev(sample_noise, torch.float32)
            pol.select, pol.sample_noise = SELECT_SAMPLE, sample_noise.data_ptr()
        keep = []
        if rank_per_group is not None:
            arr = (ct.c_int * len(rank_per_group))(*[int(r) for r in rank_per_group])
            keep.append(arr)
            pol.rank_per_group = ct.cast(arr, ct.POINTER(ct.c_int))
        if forced_indices is not None:
            _dev(forced_indices, torch.int32)
            pol.forced_indices = forced_indices.data_ptr()
        return pol, keep

    def out_shape(self, scale_idx: int, cfg_mode: int):
        if not 0 <= scale_idx < len(self.scale_hw):
            return (1,)                                  # the library rejects the index
        h, w = self.scale_hw[scale_idx]
        return (self.B // 2 if cfg_mode == CFG_NULL_ONLY else self.B, h * w, self.width)

    def scale_step(self, tokens: torch.Tensor, scale_idx: int, *, mode: int = DENSE, cfg_mode: int = CFG_PAIR,
                   keep_ratio: float = 1.0, rank_per_group=None, forced_indices=None, sample_noise=None,
                   out: Optional[torch.Tensor] = None, restore: int = RESTORE_RTR) -> Optional[torch.Tensor]:
        _dev(tokens, torch.bfloat16)
        pol, _keep = self._policy(mode, cfg_mode, keep_ratio, rank_per_group, forced_indices, sample_noise, restore)
        if mode == SKIP:
            self._check(self.lib.fvar_scale_step(self.ctx, tokens.data_ptr(), scale_idx, ct.byref(pol), None))
            return None
        if out is None:
            out = torch.empty(self.out_shape(scale_idx, cfg_mode), dtype=torch.bfloat16, device=tokens.device)
        self._check(self.lib.fvar_scale_step(self.ctx, tokens.data_ptr(), scale_idx, ct.byref(pol), out.data_ptr()))
        return out

    def scale_step_host(self, tokens_host: torch.Tensor, scale_idx: int, out_host: torch.Tensor, *, mode: int = DENSE,
                        cfg_mode: int = CFG_PAIR, keep_ratio: float = 1.0, rank_per_group=None):
        assert not tokens_host.is_cuda and not out_host.is_cuda
        pol, _keep = self._policy(mode, cfg_mode, keep_ratio, rank_per_group, None)
        self._check(self.lib.fvar_scale_step_host(self.ctx, tokens_host.data_ptr(), scale_idx, ct.byref(pol),
                                                  out_host.data_ptr()))
        return out_host

    def scale_step_host_async(self, tokens_host: torch.Tensor, scale_idx: int, out_host: torch.Tensor, *, mode: int = DENSE,
                              cfg_mode: int = CFG_PAIR, keep_ratio: float = 1.0, rank_per_group=None, restore: int = RESTORE_RTR):
        """Pipelined host entry point: enqueues upload, step and download and returns; host_sync() waits for them."""
        assert not tokens_host.is_cuda and not out_host.is_cuda
        pol, _keep = self._policy(mode, cfg_mode, keep_ratio, rank_per_group, None, None, restore)
        self._check(self.lib.fvar_scale_step_host_async(self.ctx, tokens_host.data_ptr(), scale_idx, ct.byref(pol),
                                                        out_host.data_ptr()))
        return out_host

    def host_sync(self):
        self._check(self.lib.fvar_host_sync(self.ctx))

    def kv_append(self, scale_idx: int):
        self._check(self.lib.fvar_kv_append(self.ctx, scale_idx))

    def get_indices(self, group: int, B_eff: int, r_cap: int) -> torch.Tensor:
        buf = torch.empty((B_eff * r_cap,), dtype=torch.int32, device="cuda")
        cnt = ct.c_int(0)
        self._check(self.lib.fvar_get_indices(self.ctx, group, buf.data_ptr(), ct.byref(cnt)))
        return buf[:B_eff * cnt.value].view(B_eff, cnt.value)

    def get_group_output(self, group: int, M: int) -> torch.Tensor:
        out = torch.empty((self.B, M, self.width), dtype=torch.float32, device="cuda")
        self._check(self.lib.fvar_get_group_output(self.ctx, group, out.data_ptr()))
        return out

    def load_kv(self, K: torch.Tensor, V: torch.Tensor):
        """K, V bf16 [n_blocks][B][L][C]: committed rows of the earlier scales."""
        _dev(K, torch.bfloat16), _dev(V, torch.bfloat16)
        self._check(self.lib.fvar_load_kv(self.ctx, K.data_ptr(), V.data_ptr(), K.shape[2]))

    def load_group_cache(self, scale_idx: int, cache: torch.Tensor):
        """cache fp32 [n_groups][B][M][C]: block-group outputs of scale scale_idx."""
        _dev(cache, torch.float32)
        self._check(self.lib.fvar_load_group_cache(self.ctx, scale_idx, cache.data_ptr()))

    def cache_len(self, block: int) -> int:
        return self.lib.fvar_cache_len(self.ctx, block)

    def launch_count(self) -> int:
        return self.lib.fvar_launch_count(self.ctx)

    def poll_status(self) -> int:
        return self.lib.fvar_poll_status(self.ctx)

    def selftest_wait_timeout(self, cycles: int):
        """Launches the one-CTA kernel whose bounded wait runs out after `cycles` clock cycles."""
        self._check(self.lib.fvar_selftest_wait_timeout(self.ctx, int(cycles), None))

    def reset(self):
        self._check(self.lib.fvar_reset(self.ctx))

    def set_option(self, option: int, value: int):
        self._check(self.lib.fvar_set_option(self.ctx, option, value))

    def restore_loaded(self):
        self._check(self.lib.fvar_restore_loaded(self.ctx))

    def profile_enable(self, on: bool):
        self._check(self.lib.fvar_profile_enable(self.ctx, int(on)))

    def profile_dump(self, kclass: int, capacity: int = 4096):
        """Per-launch times in ms of one kernel class, in launch order."""
        buf = (ct.c_float * capacity)()
        n = ct.c_int(0)
        self._check(self.lib.fvar_profile_dump(self.ctx, kclass, buf, capacity, ct.byref(n)))
        return [buf[j] for j in range(min(n.value, capacity))]

    def profile_read(self, kclass: int):
        """(total ms, launches, algorithmic flops, algorithmic bytes) of one kernel class."""
        ms, n, fl, by = ct.c_double(0), ct.c_longlong(0), ct.c_double(0), ct.c_double(0)
        self._check(self.lib.fvar_profile_read(self.ctx, kclass, ct.byref(ms), ct.byref(n), ct.byref(fl), ct.byref(by)))
        return ms.value, n.value, fl.value, by.value
