"""Stand-alone timings of the library's kernels through the C ABI (CUDA events, one GPU).

    python microbench.py gemm [single|pair <64|128|256>]   # the library's choice, or a given launch form and tile width
    python microbench.py skinny      # the weight-streaming form on the Infinity-2B-shaped late GEMMs
    python microbench.py skinny_one R N K [S]  # eight launches of that form on one shape (for ncu)
    python microbench.py attention_one B H D r L   # four attention launches on one shape (for ncu)
    python microbench.py gemmk [single|pair <width>]       # the same over K at fixed R x N: fixed cost and cost per K step
    python microbench.py attention
    python microbench.py memory      # score, LayerNorm + modulate, restoration fill, selection
    python microbench.py transition  # between two scale steps: codeword search, Up-accumulate, Down

GEMM calls rotate over several weight copies (more than L2 holds) and are captured in one CUDA graph so
that host launch cost does not enter the time.
"""
from __future__ import annotations

import sys

import torch

from paper_2512_16483_b200 import binding as fv


def _time(fn, n=20, warm=3):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / n          # microseconds


def _form_args():
    """Optional launch form after the sub-command: `single|pair <tile width>`; default: the library's cost model."""
    if len(sys.argv) > 3 and sys.argv[2] in ("single", "pair"):
        return (fv.GEMM_SINGLE if sys.argv[2] == "single" else fv.GEMM_PAIR), int(sys.argv[3]), "%s %s" % (sys.argv[2], sys.argv[3])
    return fv.GEMM_AUTO, 0, "picked"


def gemm():
    lib = fv.load_library()
    form, block_n, bn = _form_args()
    shapes = [(1024, 3072, 1024), (1024, 1024, 1024), (1024, 4096, 1024), (1024, 1024, 4096), (400, 3072, 1024),
              (16, 2048, 2048), (16, 2048, 8192), (336, 8192, 2048), (4096, 4096, 1024), (8192, 8192, 2048),
              (16384, 4096, 4096)]
    for R, N, K in shapes:
        if form == fv.GEMM_PAIR and R <= 128:
            continue                                     # a single row tile has no partner
        us = _gemm_form_graph_us(lib, R, N, K, form, block_n)
        print("form %s R=%d N=%d K=%d: %.2f us  %.1f TFLOP/s  weights %.0f GB/s" % (
            bn, R, N, K, us, 2 * R * N * K / us / 1e6, N * K * 2 / us / 1e3))


def _gemm_form_graph_us(lib, R, N, K, form, block_n):
    ncopy = max(2, min(32, int(300e6 // (N * K * 2))))
    A = torch.randn(R, K, device="cuda").bfloat16()
    Ws = [torch.randn(N, K, device="cuda").bfloat16() * 0.02 for _ in range(ncopy)]
    out = torch.empty(R, N, device="cuda", dtype=torch.float32)

    def call(i):
        st = lib.fvar_gemm_bf16_form(A.data_ptr(), Ws[i % ncopy].data_ptr(), None, R, N, K, form, block_n, out.data_ptr(),
                                     torch.cuda.current_stream().cuda_stream)
        assert st == 0, st
    for i in range(ncopy):
        call(i)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(ncopy):
            call(i)
    return _time(g.replay, n=5, warm=1) / ncopy


def skinny():
    """The weight-streaming form against the picked form on the GEMM shapes of the Infinity-2B-shaped late steps."""
    lib = fv.load_library()
    for R in (16, 64, 111, 170, 256, 336, 410):
        for N, K in ((6144, 2048), (2048, 2048), (8192, 2048), (2048, 8192)):
            auto = _gemm_form_graph_us(lib, R, N, K, fv.GEMM_AUTO, 0)
            sk = _gemm_form_graph_us(lib, R, N, K, fv.GEMM_SKINNY, 0)
            print("R=%d N=%d K=%d: picked form %.2f us | weight-streaming %.2f us  weights %.0f GB/s  %.0f TFLOP/s" % (
                R, N, K, auto, sk, N * K * 2 / sk / 1e3, 2 * R * N * K / sk / 1e6), flush=True)


def skinny_one():
    """A few launches of the weight-streaming form over rotating weight copies (for a profiler): R N K [ranges]."""
    lib = fv.load_library()
    R, N, K = (int(x) for x in sys.argv[2:5])
    S = int(sys.argv[5]) if len(sys.argv) > 5 else 0
    A = torch.randn(R, K, device="cuda").bfloat16()
    Ws = [torch.randn(N, K, device="cuda").bfloat16() * 0.02 for _ in range(8)]
    out = torch.empty(R, N, device="cuda", dtype=torch.float32)
    for W in Ws:
        assert lib.fvar_gemm_bf16_form(A.data_ptr(), W.data_ptr(), None, R, N, K, fv.GEMM_SKINNY, S, out.data_ptr(),
                                       torch.cuda.current_stream().cuda_stream) == 0
    torch.cuda.synchronize()
    print("launched 8 weight-streaming GEMMs R=%d N=%d K=%d" % (R, N, K))


def attention_one():
    """A few launches of the attention kernel over rotating caches (for a profiler): B H D r L."""
    B, H, D, r, L = (int(x) for x in sys.argv[2:7])
    Lc = (L + 127) // 128 * 128
    q = torch.randn(B, r, H * D, device="cuda").bfloat16()
    caches = [(torch.randn(B, H, Lc, D, device="cuda").bfloat16(), torch.randn(B, H, D, Lc, device="cuda").bfloat16()) for _ in range(4)]
    for Kc, Vt in caches:
        fv.fvar_attention(q, Kc, Vt, L)
    torch.cuda.synchronize()
    print("launched 4 attention calls B=%d H=%d D=%d r=%d L=%d" % (B, H, D, r, L))


def ksplit():
    """128 x 128 tiles with the K range over a cluster against the picked form and the weight-streaming form."""
    lib = fv.load_library()
    for R in (111, 170, 256, 336, 410, 479):
        for N, K in ((2048, 2048), (2048, 8192), (6144, 2048), (8192, 2048)):
            auto = _gemm_form_graph_us(lib, R, N, K, fv.GEMM_AUTO, 0)
            sk = _gemm_form_graph_us(lib, R, N, K, fv.GEMM_SKINNY, 0)
            ks = _gemm_form_graph_us(lib, R, N, K, fv.GEMM_KSPLIT, 0)
            print("R=%d N=%d K=%d: picked %.2f us | weight-streaming %.2f us | 128x128 cluster-split %.2f us (%.0f TFLOP/s)" % (
                R, N, K, auto, sk, ks, 2 * R * N * K / ks / 1e6), flush=True)


def gemmk():
    lib = fv.load_library()
    form, block_n, tag = _form_args()
    for R, N in [(1024, 3072), (1024, 1024), (4096, 4096)]:
        res = ["K=%d: %.2f us" % (K, _gemm_form_graph_us(lib, R, N, K, form, block_n)) for K in (128, 256, 512, 1024, 2048, 4096)]
        print("form", tag, "R=%d N=%d |" % (R, N), "  ".join(res), flush=True)


def attention():
    lib = fv.load_library()
    cases = [(2, 16, 128, 4096, 10521, 10624), (2, 16, 128, 1600, 4121, 4224), (2, 16, 128, 4096, 256, 256),
             (16, 16, 64, 256, 680, 768), (32, 30, 64, 256, 680, 768), (8, 16, 64, 128, 552, 768),
             (1, 16, 128, 170, 6595, 10624)]
    for B, H, D, r, L, Lc in cases:
        C = H * D
        q = torch.randn(B, r, C, device="cuda").bfloat16()
        Kc = torch.randn(B, H, Lc, D, device="cuda").bfloat16()
        Vt = torch.randn(B, H, D, Lc, device="cuda").bfloat16()
        out = torch.empty_like(q)
        us = _time(lambda: lib.fvar_attention(q.data_ptr(), Kc.data_ptr(), Vt.data_ptr(), B, H, r, D, L, Lc,
                                              out.data_ptr(), torch.cuda.current_stream().cuda_stream), n=10)
        print("B=%d H=%d D=%d r=%d L=%d: %.1f us  %.1f TFLOP/s  K/V %.0f GB/s" % (
            B, H, D, r, L, us, 4.0 * B * r * L * C / us / 1e6, 4.0 * B * L * C / us / 1e3))
    assert fv.kernel_poll_status() == fv.OK


def memory():
    for B, M, C in [(2, 4096, 2048), (32, 4096, 2048), (32, 1600, 1024)]:
        xs = [torch.randn(B, M, C, device="cuda") for _ in range(2)]
        k = [0]

        def nxt():
            k[0] += 1
            return xs[k[0] % 2]
        us = _time(lambda: fv.fvar_row_scores(nxt()))
        print("row_scores   B=%d M=%d C=%d: %.1f us  %.0f GB/s" % (B, M, C, us, B * M * C * 4 / us / 1e3))
        sh, sc = torch.randn(B, C, device="cuda"), torch.randn(B, C, device="cuda")
        us = _time(lambda: fv.fvar_ln_modulate(nxt(), sh, sc, 1e-6))
        print("ln_modulate  B=%d M=%d C=%d: %.1f us  %.0f GB/s" % (B, M, C, us, B * M * C * 6 / us / 1e3))
        if M == 4096:
            prev = torch.randn(B, 2304, C, device="cuda")
            out = torch.empty(B, M, C, device="cuda")
            inv = torch.full((B, M), -1, dtype=torch.int32, device="cuda")
            inv[:, ::24] = 1
            us = _time(lambda: fv.fvar_rtr_fill(prev, (48, 48), (64, 64), inv, out))
            nfill = int((inv < 0).sum().item())
            print("rtr_fill     B=%d M=%d C=%d: %.1f us  %.0f GB/s (rows written once + cache read once)" % (
                B, M, C, us, (nfill * C * 4 + B * 2304 * C * 4) / us / 1e3))
        s = torch.rand(B, M, device="cuda")
        us = _time(lambda: fv.fvar_select_topr(s, M // 4))
        print("select_topr  B=%d M=%d r=%d: %.1f us (includes ~10 us of host call overhead)" % (B, M, M // 4, us))


def transition():
    """Transitions of an Infinity-2B-shaped schedule tail (32 x 32, 48 x 48, 64 x 64 tokens; accumulation at
    64 x 64; C = 2048, 8192 codewords) for 8 elements, timed per kernel by the library's profile pass."""
    C, V, B = 2048, 8192, 8
    hw = [(32, 32), (48, 48), (64, 64)]
    Ms = [h * w_ for h, w_ in hw]
    dims = {"w_qkv": (3 * C, C), "b_qkv": (3 * C,), "w_o": (C, C), "b_o": (C,), "w_fc1": (4 * C, C), "b_fc1": (4 * C,),
            "w_fc2": (C, 4 * C), "b_fc2": (C,), "w_ada": (6 * C, C), "b_ada": (6 * C,)}
    w = [{n: torch.zeros(shape, dtype=torch.bfloat16, device="cuda") for n, shape in dims.items()}]
    ctx = fv.Fvar(w, blocks_per_group=1, n_heads=16, head_dim=128, ffn_dim=4 * C, scale_hw=hw, max_batch=B)
    ctx.set_codebook(torch.randn(V, C, device="cuda").bfloat16())
    fo = [torch.randn(B, m, C, device="cuda").bfloat16() for m in Ms]

    def chain():
        ctx.scale_transition(fo[0], 0, Ms[1])
        ctx.scale_transition(fo[1], 1, Ms[2])
    chain()
    ctx.profile_enable(True)
    for _ in range(5):
        chain()
    gemm_t = ctx.profile_dump(fv.KCLASSES.index("gemm"))          # per pass: search of scale 0, of scale 1
    up_t = ctx.profile_dump(fv.KCLASSES.index("rtr_fill"))        # per pass: Up of scale 0 (write), of scale 1 (accumulate)
    cv_t = ctx.profile_dump(fv.KCLASSES.index("convert"))         # per pass: unpack, Down 64->48, unpack, Down 64->64
    t_g, t_u, t_d = 1e3 * min(gemm_t[1::2]), 1e3 * min(up_t[1::2]), 1e3 * min(cv_t[1::4])
    print("codeword search  R=%d V=%d K=%d: %.1f us  %.0f TFLOP/s" % (B * Ms[1], V, C, t_g, 2.0 * B * Ms[1] * V * C / t_g / 1e6))
    print("up_accumulate    B=%d 48x48 -> 64x64 C=%d: %.1f us  %.0f GB/s (fp32 map read and written once)" % (
        B, C, t_u, 8.0 * B * Ms[2] * C / t_u / 1e3))
    print("down_area        B=%d 64x64 -> 48x48 C=%d: %.1f us  %.0f GB/s (map read once, bf16 tokens written once)" % (
        B, C, t_d, (4.0 * B * Ms[2] * C + 2.0 * B * Ms[1] * C) / t_d / 1e3))
    ctx.profile_enable(False)


if __name__ == "__main__":
    which = sys.argv[1] if len(sys.argv) > 1 else "gemm"
    {"gemm": gemm, "gemmk": gemmk, "attention": attention, "memory": memory, "transition": transition, "skinny": skinny,
     "ksplit": ksplit, "skinny_one": skinny_one, "attention_one": attention_one}[which]()
