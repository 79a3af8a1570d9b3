"""Shared by the GPU tests: moving seeded numpy inputs to the device and comparing results."""
import numpy as np
import torch

import synth_inputs as si


def to_bf16_cuda(a: np.ndarray) -> torch.Tensor:
    """fp32 array holding bf16-representable values -> bf16 CUDA tensor with the same bits."""
    bits = si.bf16_bits(a)
    t = torch.from_numpy(bits.view(np.int16).reshape(a.shape))
    return t.view(torch.bfloat16).cuda()


def bf16_to_numpy(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def weights_to_cuda(weights):
    return [{k: to_bf16_cuda(v) for k, v in blk.items()} for blk in weights]


def rel_err(got: np.ndarray, ref: np.ndarray):
    """(max-abs error / RMS of the reference, cosine similarity)."""
    got, ref = np.asarray(got, np.float64).ravel(), np.asarray(ref, np.float64).ravel()
    rms = float(np.sqrt(np.mean(ref ** 2))) + 1e-30
    cos = float(got @ ref / (np.linalg.norm(got) * np.linalg.norm(ref) + 1e-30))
    return float(np.max(np.abs(got - ref))) / rms, cos


def assert_close(got, ref, max_rel=2e-2, min_cos=0.999, what=""):
    """The acceptance bar of the block outputs: max-abs error <= 2e-2 x output RMS, cosine >= 0.999."""
    e, c = rel_err(got, ref)
    assert e <= max_rel and c >= min_cos, "%s: max-abs/RMS %.3e (bar %.1e), cosine %.6f (bar %.4f)" % (
        what, e, max_rel, c, min_cos)
    return e, c


def assert_out_close(got_bf16, ref, what="", max_rel=2e-2):
    """bf16 output of the step: the block-output bar (2e-2 x output RMS, cosine >= 0.999) plus the one
    rounding of the returned value to bf16.  bf16 keeps 8 significant bits (1 implicit + 7 stored), so round to
    nearest moves x by at most half a unit in the last place = 2^(e-8) for 2^e <= |x| < 2^(e+1), i.e. by at most
    2^-8 |x| (reached just above a power of two); |x| <= |ref| + the bar.  The fp32 group outputs carry no such
    term and are held to the plain bar (assert_close) in every step test."""
    got, ref = np.asarray(got_bf16, np.float64), np.asarray(ref, np.float64)
    rms = float(np.sqrt(np.mean(ref ** 2)))
    excess = np.abs(got - ref) - (max_rel * rms + 2.0 ** -8 * (np.abs(ref) + max_rel * rms))
    _, c = rel_err(got, ref)
    assert excess.max() <= 0 and c >= 0.999, "%s: worst excess over the bound %.3e (RMS %.3e), cosine %.6f" % (
        what, excess.max(), rms, c)
