"""Single-kernel cases for timing and profiling.

    python -m paper_1908_05033_b200.cases gemm --size 4096 --bits 4 --iters 5
    python -m paper_1908_05033_b200.cases conv --cin 64 --cout 64 --hw 56 --batch 64 --ksize 3
    python -m paper_1908_05033_b200.cases quant --mb 1024 --bits 4
    python -m paper_1908_05033_b200.cases dw --c 192 --hw 56 --batch 64
    python -m paper_1908_05033_b200.cases soft --mb 1024 --bits 4

Each runs the named kernel `--iters` times on seeded synthetic inputs (an L2
flush between launches) and prints the median CUDA-event time with the
derived rate.  Small enough to sit under a profiler.
"""
import argparse
import json
import statistics
import sys

import numpy as np
import torch

from . import binding as B


def _timeit(fn, iters, flush):
    times = []
    for i in range(iters):
        if flush is not None:
            flush.zero_()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    keep = times[min(2, len(times) - 1):]
    return statistics.median(keep), times


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["gemm", "bgemm", "wgemm", "conv", "quant", "dw", "soft"])
    ap.add_argument("--size", type=int, default=4096)
    ap.add_argument("--bits", type=int, default=4)
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--cin", type=int, default=64)
    ap.add_argument("--cout", type=int, default=64)
    ap.add_argument("--c", type=int, default=192)
    ap.add_argument("--hw", type=int, default=56)
    ap.add_argument("--batch", type=int, default=64)
    ap.add_argument("--ksize", type=int, default=3)
    ap.add_argument("--stride", type=int, default=1)
    ap.add_argument("--mb", type=int, default=1024, help="fp32 input size in MiB")
    ap.add_argument("--no-flush", action="store_true")
    ap.add_argument("--f32-out", action="store_true")
    ap.add_argument("--tile-n", type=int, default=0)
    ap.add_argument("--round-k", type=int, default=0)
    ap.add_argument("--pairs", type=int, default=0, help="0 auto, 1 never, 2 wherever possible")
    ap.add_argument("--window", type=int, default=1,
                    help="3x3 stride-1 convolutions: 1 shared-memory window kernel, 0 im2col kernel")
    ap.add_argument("--residual", action="store_true")
    ap.add_argument("--fused", action="store_true",
                    help="gemm: the single fused kernel (small workspace) instead of two passes")
    a = ap.parse_args(argv)
    dev = "cuda"
    ws = B.new_workspace(dev)
    flush = None if a.no_flush else torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(1908)
    bits = a.bits
    B.dsq_set_tile_n(a.tile_n)
    B.dsq_set_round_k_steps(a.round_k)
    B.dsq_set_cta_pairs(a.pairs)
    B.dsq_set_conv3_window(a.window)
    out = {"case": a.case, "bits": bits, "tile_n": a.tile_n}
    if a.case == "gemm":
        n = a.size
        pitch = B.dsq_row_pitch(n, bits)
        A = torch.randint(0, 256, (n, pitch), dtype=torch.uint8, device=dev, generator=gen)
        Bm = torch.randint(0, 256, (n, pitch), dtype=torch.uint8, device=dev, generator=gen)
        Cm = torch.empty((n, n), dtype=torch.int32, device=dev)
        if not a.fused:
            ws = B.new_gemm_workspace(n, n, n, bits, dev)
        ms, all_ms = _timeit(lambda: B.dsq_gemm(A, Bm, n, n, n, bits, ws, out_i32=Cm),
                             a.iters, flush)
        out.update(size=n, ms=ms, tops=2.0 * n ** 3 / (ms * 1e-3) / 1e12, all_ms=all_ms)
    elif a.case == "bgemm":
        # binary GEMM: 1-bit rows, values -1 / +1
        n = a.size
        pitch = B.dsq_row_pitch(n, 1)
        A = torch.randint(0, 256, (n, pitch), dtype=torch.uint8, device=dev, generator=gen)
        Bm = torch.randint(0, 256, (n, pitch), dtype=torch.uint8, device=dev, generator=gen)
        Cm = torch.empty((n, n), dtype=torch.int32, device=dev)
        ws = torch.zeros(B.lib.dsq_binary_gemm_workspace_bytes(n, n, n), dtype=torch.uint8, device=dev)
        ms, all_ms = _timeit(lambda: B._check(B.lib.dsq_binary_gemm(
            A.data_ptr(), Bm.data_ptr(), n, n, n, Cm.data_ptr(), None, None, ws.data_ptr(),
            ws.numel(), torch.cuda.current_stream().cuda_stream), "dsq_binary_gemm"), a.iters, flush)
        out.update(size=n, ms=ms, tops=2.0 * n ** 3 / (ms * 1e-3) / 1e12, all_ms=all_ms)
    elif a.case == "wgemm":
        # weight-only: bf16 activations [size, size] x b-bit weights [size, size]
        n = a.size
        X = torch.randn((n, n), device=dev, generator=gen).to(torch.bfloat16)
        W = torch.randint(0, 256, (n, B.dsq_row_pitch(n, bits)), dtype=torch.uint8, device=dev,
                          generator=gen)
        sc = torch.full((n,), 0.01, device=dev)
        Y = torch.empty((n, n), dtype=torch.float32, device=dev)
        ws = torch.zeros(B.lib.dsq_wgemm_workspace_bytes(n, n), dtype=torch.uint8, device=dev)
        ms, all_ms = _timeit(lambda: B.dsq_wgemm_bf16(X, W, n, n, n, bits, sc, ws=ws, out=Y),
                             a.iters, flush)
        out.update(size=n, ms=ms, tflops=2.0 * n ** 3 / (ms * 1e-3) / 1e12, all_ms=all_ms)
    elif a.case == "conv":
        shape = (a.batch, a.hw, a.hw, a.cin)
        pitch = B.dsq_row_pitch(a.cin, bits)
        act = torch.randint(0, 256, shape[:3] + (pitch,), dtype=torch.uint8, device=dev,
                            generator=gen)
        w = torch.randn((a.cout, a.ksize, a.ksize, a.cin), device=dev, generator=gen) * 0.05
        blob, conv = B.dsq_pack_weights(w, bits, -0.1, 0.1, ws, stride=a.stride,
                                        pad=a.ksize // 2)
        scale = torch.full((a.cout,), 1e-3, device=dev)
        bias = torch.zeros((a.cout,), device=dev)
        ho = (a.hw + 2 * (a.ksize // 2) - a.ksize) // a.stride + 1
        codes = torch.empty((a.batch, ho, ho, B.dsq_row_pitch(a.cout, bits)),
                            dtype=torch.uint8, device=dev)
        res = torch.randint(0, 256, codes.shape, dtype=torch.uint8, device=dev,
                            generator=gen) if a.residual else None
        fn = lambda: B.dsq_conv2d(act, shape, (bits, 0.0, 2.0), blob, conv, scale, bias, ws,
                                  w_offset=0.5, requant=(bits, 0.0, 2.0), out_codes=codes,
                                  want_f32=a.f32_out, residual=res,
                                  residual_q=(bits, 0.0, 2.0) if a.residual else None)
        ms, all_ms = _timeit(fn, a.iters, flush)
        macs = a.batch * ho * ho * a.cout * a.ksize * a.ksize * a.cin
        out.update(shape=list(shape), cout=a.cout, ksize=a.ksize, stride=a.stride, ms=ms,
                   tops=2.0 * macs / (ms * 1e-3) / 1e12, all_ms=all_ms)
    elif a.case == "quant":
        n = a.mb * (1 << 20) // 4
        rows = n // 64
        x = torch.randn((1, 1, rows, 64), device=dev, generator=gen)
        o = torch.empty((1, 1, rows, B.dsq_row_pitch(64, bits)), dtype=torch.uint8, device=dev)
        ms, all_ms = _timeit(lambda: B.dsq_quantize_act(x, bits, 0.0, 2.0, out=o), a.iters,
                             flush)
        nbytes = rows * 64 * 4 + o.numel()
        out.update(elements=rows * 64, ms=ms, gbs=nbytes / (ms * 1e-3) / 1e9, all_ms=all_ms)
    elif a.case == "soft":
        # training-side soft quantiser: forward (8 B / element) and backward (12 B / element)
        n = a.mb * (1 << 20) // 4
        x = torch.randn(n, device=dev, generator=gen)
        g = torch.randn(n, device=dev, generator=gen)
        y = torch.empty_like(x)
        gp = torch.empty(3, dtype=torch.float64, device=dev)
        ms, all_ms = _timeit(lambda: B.dsq_soft_quantize_fwd(x, bits, -1.0, 2.0, 0.2, out=y),
                             a.iters, flush)
        msb, all_b = _timeit(lambda: B.dsq_soft_quantize_bwd(x, g, bits, -1.0, 2.0, 0.2, out=y,
                                                             grad_params=gp), a.iters, flush)
        out.update(elements=n, fwd_ms=ms, fwd_gbs=8.0 * n / (ms * 1e-3) / 1e9, bwd_ms=msb,
                   bwd_gbs=12.0 * n / (msb * 1e-3) / 1e9, all_ms=all_ms + all_b)
    else:
        shape = (a.batch, a.hw, a.hw, a.c)
        pitch = B.dsq_row_pitch(a.c, bits)
        act = torch.randint(0, 256, shape[:3] + (pitch,), dtype=torch.uint8, device=dev,
                            generator=gen)
        w = torch.randn((a.c, 3, 3), device=dev, generator=gen) * 0.3
        blob, conv = B.dsq_pack_weights(w, bits, -1.0, 1.0, ws, depthwise=True,
                                        stride=a.stride, pad=1)
        scale = torch.full((a.c,), 1e-2, device=dev)
        bias = torch.zeros((a.c,), device=dev)
        ho = (a.hw + 2 - 3) // a.stride + 1
        codes = torch.empty((a.batch, ho, ho, pitch), dtype=torch.uint8, device=dev)
        fn = lambda: B.dsq_dwconv2d(act, shape, (bits, 0.0, 6.0), blob, conv, scale, bias,
                                    w_offset=0.5, requant=(bits, 0.0, 6.0), out_codes=codes)
        ms, all_ms = _timeit(fn, a.iters, flush)
        nbytes = act.numel() + codes.numel()
        out.update(shape=list(shape), stride=a.stride, ms=ms,
                   gbs=nbytes / (ms * 1e-3) / 1e9, all_ms=all_ms)
    B.check_workspace(ws, a.case)
    print(json.dumps(out))
    return 0


if __name__ == "__main__":
    sys.exit(main())
