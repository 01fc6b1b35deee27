"""Per-configuration timing report: ``python -m paper_1804_01526_b200.report [--out FILE]``.

For every GEMM of the benchmark configurations (single 256-cube, MLP step, ResNet im2col
convolutions, transformer layer, large sweep) it times, with CUDA events on the current stream,
the conversion of each FP32 operand to block floating point and the BFP GEMM on already-packed
operands, and prints one markdown table row per GEMM. Weights in shared tiles are converted once
per layer (both views) and re-used by forward and backward-data, as in training. Calls shorter
than 0.3 ms are timed as the per-call device time of 20 calls captured in one CUDA graph (their
operands then sit in L2), since one event-timed call would measure the binding's host time.
"""
from __future__ import annotations

import argparse
import statistics
import sys

import torch

from . import binding as hb
from . import workloads as wl


def _time(fn, iters=10, warm=3):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    ts = []
    for _ in range(iters):
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        fn()
        e.record()
        torch.cuda.synchronize()
        ts.append(s.elapsed_time(e))
    return statistics.median(ts)


GRAPH_BELOW_MS = 0.3      # calls shorter than this are timed as a CUDA-graph replay
GRAPH_CALLS = 20


def _time_graph(fn, calls=GRAPH_CALLS, iters=10):
    """Device time per call of ``calls`` back-to-back calls captured in one CUDA graph. For calls of
    a few microseconds this leaves out the host time the Python binding spends per launch, which a
    single event-timed call would measure instead of the kernels."""
    fn()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for _ in range(calls):
            fn()
    return _time(g.replay, iters=iters) / calls


def _time_auto(fn):
    t = _time(fn)
    return _time_graph(fn) if t < GRAPH_BELOW_MS else t


def mlp_step_lines():
    """The nine GEMMs of the MLP step, each with its conversions, as one captured graph."""
    specs = wl.config_mlp()
    t = wl.materialize(specs, seed=1)
    dev = {k: torch.from_numpy(v).cuda() for k, v in t.items()}
    outs = [torch.empty((sp.M, sp.N), dtype=torch.float32, device="cuda") for sp in specs]
    fmts = [(hb.Format(**sp.fmt_a), hb.Format(**sp.fmt_b)) for sp in specs]
    wss = [torch.empty(max(hb.gemm_workspace(sp.transA, sp.transB, sp.M, sp.N, sp.K, fa, fb), 1), dtype=torch.int8,
                       device="cuda") for sp, (fa, fb) in zip(specs, fmts)]

    def step():
        for sp, (fa, fb), C, ws in zip(specs, fmts, outs, wss):
            hb.gemm(sp.transA, sp.transB, dev[sp.a_key], dev[sp.b_key], fa, fb, out=C, workspace=ws)

    t_eager = _time(step)
    t_graph = _time_graph(step, calls=1)
    ops = sum(sp.ops for sp in specs)

    # The same step as training issues it: every weight matrix converted once into its two shared views, forward
    # and backward-data read them (hbfp_gemm_q), and each backward-weight GEMM, which nothing later in the step
    # waits for, goes to a second stream that the graph joins at the end.
    layers = [specs[i:i + 3] for i in range(0, len(specs), 3)]          # (forward, backward-data, backward-weight)
    views = []
    for fwd, _, _ in layers:
        c0, c1, _g = hb.quantize_tiles(dev[fwd.b_key], hb.Format(**fwd.fmt_b))
        views.append((c0, c1))
    by_name = {sp.name: (C, ws) for sp, C, ws in zip(specs, outs, wss)}
    side = torch.cuda.Stream()

    def steady():
        main = torch.cuda.current_stream()
        for (fwd, _, _), (c0, c1) in zip(layers, views):
            hb.quantize_tiles(dev[fwd.b_key], hb.Format(**fwd.fmt_b), out=(c0, c1), want_grid=False)
        for (fwd, _, _), (c0, c1) in zip(layers, views):
            C, ws = by_name[fwd.name]
            hb.gemm_q(fwd.M, fwd.N, fwd.K, dev[fwd.a_key], c1 if fwd.transB else c0, transA=fwd.transA,
                      fmtA=hb.Format(**fwd.fmt_a), out=C, workspace=ws)
        for (_, dg, wg), (c0, c1) in reversed(list(zip(layers, views))):
            C, ws = by_name[dg.name]
            hb.gemm_q(dg.M, dg.N, dg.K, dev[dg.a_key], c1 if dg.transB else c0, transA=dg.transA,
                      fmtA=hb.Format(**dg.fmt_a), out=C, workspace=ws)
            side.wait_stream(main)
            with torch.cuda.stream(side):
                C, ws = by_name[wg.name]
                hb.gemm(wg.transA, wg.transB, dev[wg.a_key], dev[wg.b_key], hb.Format(**wg.fmt_a), hb.Format(**wg.fmt_b),
                        out=C, workspace=ws)
        main.wait_stream(side)

    t_steady = _time_graph(steady, calls=1)
    return [f"MLP step, 9 x hbfp_gemm (27 launches + memsets): {t_eager*1e3:.1f} us issued call by call from Python, "
            f"{t_graph*1e3:.1f} us as one CUDA-graph replay ({ops/(t_graph*1e-3)/1e12:.2f} TOPS); weights converted once per "
            f"layer into shared views, backward-weight GEMMs on a second stream of the same graph: {t_steady*1e3:.1f} us "
            f"({ops/(t_steady*1e-3)/1e12:.2f} TOPS)"]


def wide_lines(hbm_gbs):
    """Wide weight storage on the weight matrices of the configurations: first conversion, in-place
    FP32 update (with the narrow views of the new weights) and the narrow views alone."""
    out = ["", "| weights | format | wide quantise µs | wide update + views µs (GB/s, % HBM) | narrow views only µs | FP32 -> views (`hbfp_quantize_tiles`) µs (GB/s, % HBM) |",
           "|---|---|---|---|---|---|"]
    for name, shape, fd in (("c1.l1.W", (1024, 1024), dict(mant_bits=8, block=24, tile=24, rounding=1, seed=1)),
                            ("c3.up.W", (1024, 4096), dict(mant_bits=12, block=64, tile=64, rounding=1, seed=7)),
                            ("8192 x 8192", (8192, 8192), dict(mant_bits=8, block=64, tile=64, rounding=0)),
                            ("16384 x 16384", (16384, 16384), dict(mant_bits=8, block=64, tile=64, rounding=0)),
                            ("16384 x 16384", (16384, 16384), dict(mant_bits=8, block=128, tile=128, rounding=0))):
        fmt = hb.Format(**fd)
        w = torch.from_numpy(wl.draw("he_weight", shape, seed=3, fan_in=shape[0])).cuda()
        dw = torch.from_numpy(wl.draw("grad", shape, seed=4)).cuda()
        wide, views = hb.wide_quantize(w, fmt)
        t_q = _time_auto(lambda: hb.wide_quantize(w, fmt, out=wide, views=views))
        t_u = _time_auto(lambda: hb.wide_update(wide, dw, fmt, views=views))
        t_n = _time_auto(lambda: hb.wide_narrow(wide, fmt, views=views))
        t_t = _time_auto(lambda: hb.quantize_tiles(w, fmt, out=views, want_grid=False))
        planes = 1 if fd["mant_bits"] <= 8 else 2
        n = shape[0] * shape[1]
        bytes_u = n * (2 + 4 + 2 + 2 * planes)          # read wide + delta, write wide + both views
        gbs = bytes_u / (t_u * 1e-3) / 1e9
        gbs_t = n * (4 + 2 * planes) / (t_t * 1e-3) / 1e9      # read FP32, write both views
        f = f"m{fd['mant_bits']} t{fd['tile']}" + (" SR" if fd["rounding"] else " RNE")
        out.append(f"| {name} {shape[0]}x{shape[1]} | {f} | {t_q*1e3:.1f} | {t_u*1e3:.1f} ({gbs:.0f}, {100*gbs/hbm_gbs:.0f} %) | "
                   f"{t_n*1e3:.1f} | {t_t*1e3:.1f} ({gbs_t:.0f}, {100*gbs_t/hbm_gbs:.0f} %) |")
        del w, dw, wide, views
    torch.cuda.empty_cache()
    return out


def conv_lines():
    """Forward GEMM operand of the two 3x3 convolutions: converting the FP32 im2col matrix against
    converting the activations once per pixel and gathering the packed operand."""
    out = ["", "| convolution | im2col matrix FP32 MB | forward: convert im2col matrix µs | convert pixels µs | gather packed operand µs | GEMM µs | "
           "implicit GEMM (`hbfp_conv_forward`) µs (GB/s of output) | backward-weight: convert im2col matrix (column blocks) µs | operand from the activations µs |",
           "|---|---|---|---|---|---|---|---|---|"]
    for name, n, hw, c, f in (("c2.conv64", 128, 32, 64, 64), ("c2.conv128", 128, 16, 128, 128)):
        fmt = hb.Format(mant_bits=8, block=c)          # one block per pixel; the configuration's 64 for the first
        x = torch.from_numpy(wl.draw("half_normal", (n * hw * hw, c), seed=5)).cuda()
        wt = torch.from_numpy(wl.draw("he_weight", (9 * c, f), seed=6, fan_in=9 * c)).cuda()
        px = hb.quantize(x, 1, fmt)
        pa = hb.im2col_packed(px, n, hw, hw, c, 3, 3, 1)
        pw = hb.quantize(wt, 0, fmt)
        cols = hb.dequantize(pa) * 0 + 1.0              # an FP32 matrix of the im2col shape, for timing its conversion
        pc = hb.quantize(cols, 1, fmt)
        M, K = n * hw * hw, 9 * c
        t_c = _time_auto(lambda: hb.quantize(cols, 1, fmt, out=pc))
        t_p = _time_auto(lambda: hb.quantize(x, 1, fmt, out=px))
        t_g = _time_auto(lambda: hb.im2col_packed(px, n, hw, hw, c, 3, 3, 1, out=pa))
        C = torch.empty((M, f), dtype=torch.float32, device="cuda")
        ws = torch.empty(max(hb.gemm_q_workspace(M, f, K, pa, pw), 1), dtype=torch.int8, device="cuda")
        t_m = _time_auto(lambda: hb.gemm_q(M, f, K, pa, pw, out=C, workspace=ws))
        t_i = _time_auto(lambda: hb.conv_forward(px, pw, n, hw, hw, c, 3, 3, 1, out=C))
        fb = hb.Format(mant_bits=8, block=64)           # backward-weight: blocks of 64 output pixels
        pt = hb.quantize(cols, 0, fb)
        t_ct = _time_auto(lambda: hb.quantize(cols, 0, fb, out=pt))
        x4 = x.view(n, hw, hw, c)
        pt2 = hb.im2col_packed_t(x4, 3, 3, 1, fb)
        t_t = _time_auto(lambda: hb.im2col_packed_t(x4, 3, 3, 1, fb, out=pt2))
        out.append(f"| {name} {M}x{f}x{K} | {M*K*4/1e6:.0f} | {t_c*1e3:.1f} | {t_p*1e3:.1f} | {t_g*1e3:.1f} | {t_m*1e3:.1f} | {t_i*1e3:.1f} ({M*f*4/(t_i*1e-3)/1e9:.0f}) | {t_ct*1e3:.1f} | {t_t*1e3:.1f} |")
        del x, x4, wt, px, pa, pw, cols, pc, C, ws, pt, pt2
    torch.cuda.empty_cache()
    # backward-data: the product dY x W^T in the im2col shape (its FP32 result still has to be folded back onto the
    # pixels) against the convolution of the packed dY with the regrouped forward weights, which yields dX itself
    out += ["", "| convolution | convert dY (one block per pixel) µs | weights tiled over the feature maps µs | dY·Wᵀ GEMM, im2col-shaped FP32 result µs (MB written) | "
            "regroup filters (`hbfp_conv_dgrad_filters`) µs | implicit backward-data µs (MB written) |", "|---|---|---|---|---|---|"]
    for name, n, hw, c, f in (("c2.conv64", 128, 32, 64, 64), ("c2.conv128", 128, 16, 128, 128)):
        M = n * hw * hw
        fg = hb.Format(mant_bits=8, block=f, rounding=1, seed=3)
        fw = hb.Format(mant_bits=8, block=f, tile=f)
        dy = torch.from_numpy(wl.draw("normal", (M, f), seed=7)).cuda()
        wt = torch.from_numpy(wl.draw("he_weight", (9 * c, f), seed=6, fan_in=9 * c)).cuda()
        pg = hb.quantize(dy, 1, fg)
        t_g = _time_auto(lambda: hb.quantize(dy, 1, fg, out=pg))
        c0, c1, _ = hb.quantize_conv_weights(wt, 9, fw)
        t_w = _time_auto(lambda: hb.quantize_conv_weights(wt, 9, fw, out=(c0, c1)))
        dcols = torch.empty((M, 9 * c), dtype=torch.float32, device="cuda")
        ws = torch.empty(max(hb.gemm_q_workspace(M, 9 * c, f, pg, c1), 1), dtype=torch.int8, device="cuda")
        t_m = _time_auto(lambda: hb.gemm_q(M, 9 * c, f, pg, c1, out=dcols, workspace=ws))
        d = hb.conv_dgrad_filters(c1, 3, 3, c, f)
        t_d = _time_auto(lambda: hb.conv_dgrad_filters(c1, 3, 3, c, f, out=d))
        dx = torch.empty((M, c), dtype=torch.float32, device="cuda")
        t_i = _time_auto(lambda: hb.conv_forward(pg, d, n, hw, hw, f, 3, 3, 1, out=dx))
        out.append(f"| {name} dX {M}x{c}, K = {9*f} | {t_g*1e3:.1f} | {t_w*1e3:.1f} | {t_m*1e3:.1f} ({M*9*c*4/1e6:.0f}) | {t_d*1e3:.1f} | {t_i*1e3:.1f} ({M*c*4/1e6:.0f}) |")
        del dy, wt, pg, c0, c1, dcols, ws, d, dx
    torch.cuda.empty_cache()
    return out


def rows_for(specs, tensors_np, peak_tops, hbm_gbs):
    dev = {k: torch.from_numpy(v).cuda() for k, v in tensors_np.items()}
    out = []
    for sp in specs:
        A, B = dev[sp.a_key], dev[sp.b_key]
        fa, fb = hb.Format(**sp.fmt_a), hb.Format(**sp.fmt_b)
        a_axis = 0 if sp.transA else 1           # contraction axis of the stored A
        b_axis = 1 if sp.transB else 0
        pa = hb.quantize(A, a_axis, fa)
        t_qa = _time_auto(lambda: hb.quantize(A, a_axis, fa, out=pa))
        if fb.tile > 0:
            c0, c1, _ = hb.quantize_tiles(B, fb)
            t_qb = _time_auto(lambda: hb.quantize_tiles(B, fb, out=(c0, c1), want_grid=False))
            pb = c1 if sp.transB else c0
        else:
            pb = hb.quantize(B, b_axis, fb)
            t_qb = _time_auto(lambda: hb.quantize(B, b_axis, fb, out=pb))
        C = torch.empty((sp.M, sp.N), dtype=torch.float32, device="cuda")
        ws = torch.empty(max(hb.gemm_q_workspace(sp.M, sp.N, sp.K, pa, pb), 1), dtype=torch.int8, device="cuda")
        t_g = _time_auto(lambda: hb.gemm_q(sp.M, sp.N, sp.K, pa, pb, out=C, workspace=ws))
        ops = sp.ops
        planes = 1 if fa.mant_bits <= 8 else 2
        qa_bytes = A.numel() * (4 + planes + 1.0 / (fa.block if fa.block > 0 else sp.K))
        tops_g = ops / (t_g * 1e-3) / 1e12
        tops_all = ops / ((t_qa + t_qb + t_g) * 1e-3) / 1e12
        fmt = f"m{fa.mant_bits} b{fa.block}" + (f" t{fb.tile}" if fb.tile else "") + (" SR" if fa.rounding else " RNE")
        out.append(f"| {sp.name} | {sp.M}x{sp.N}x{sp.K} | {fmt} | {t_qa*1e3:.1f} | {t_qb*1e3:.1f} | {t_g*1e3:.1f} | "
                   f"{qa_bytes/(t_qa*1e-3)/1e9:.0f} ({100*qa_bytes/(t_qa*1e-3)/1e9/hbm_gbs:.0f} %) | {tops_g:.1f} | "
                   f"{tops_all:.1f} ({100*tops_all/peak_tops:.1f} % / {100*tops_all/4500:.1f} %) |")
        del pa, pb, C, ws
    del dev
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default=None)
    ap.add_argument("--peak-tops", type=float, default=3266.6, help="int8 dense peak used for the % column")
    ap.add_argument("--hbm-gbs", type=float, default=6550.1)
    ap.add_argument("--sweep", type=int, nargs="*", default=[4096, 8192, 16384])
    ap.add_argument("--only", default=None, help="time only the GEMMs whose name contains this text (e.g. for a profiler)")
    args = ap.parse_args()
    hb.lib()
    lines = ["| GEMM | M x N x K | format | quantise A µs | quantise B µs | GEMM µs | quantise A GB/s (% HBM) | GEMM-only TOPS | "
             "quantise+GEMM TOPS (% of measured int8 proxy / % of nominal 4500) |", "|---|---|---|---|---|---|---|---|---|"]
    for name, specs, seed in (("single", wl.config_single_256(), 0), ("mlp", wl.config_mlp(), 1),
                              ("resnet", wl.config_resnet_im2col(), 2), ("transformer", wl.config_transformer(), 7)):
        if args.only:
            specs = [sp for sp in specs if args.only in sp.name]
        if specs:
            lines += rows_for(specs, wl.materialize(specs, seed=seed), args.peak_tops, args.hbm_gbs)
    for n in args.sweep:
        # the design points of Sec. 6: 8- and 12-bit mantissas, the 4-bit end of the mantissa range, and one
        # exponent per whole row / column (block 0: BFP without tiles)
        for (m, b, r) in ((8, 128, 0), (8, 64, 0), (8, 32, 0), (8, 128, 1), (12, 64, 1), (4, 128, 0), (8, 0, 0)):
            specs = wl.config_sweep(n, m, b, r)
            if args.only and args.only not in specs[0].name:
                continue
            t = {specs[0].a_key: wl.draw("lognormal", (n, n), seed=3, salt=0),
                 specs[0].b_key: wl.draw("lognormal", (n, n), seed=3, salt=1)}
            lines += rows_for(specs, t, args.peak_tops, args.hbm_gbs)
    if not args.only or args.only == "mlp":
        lines += [""] + mlp_step_lines()
    if not args.only or args.only == "wide":
        lines += wide_lines(args.hbm_gbs)
    if not args.only or args.only == "conv":
        lines += conv_lines()
    text = "\n".join(lines) + "\n"
    if args.out:
        with open(args.out, "w") as f:
            f.write(text)
    sys.stdout.write(text)
    if hb.device_status() != 0:
        raise SystemExit("device status non-zero")


if __name__ == "__main__":
    main()
