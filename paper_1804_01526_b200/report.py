"""Per-configuration timing report: ``python -m paper_1804_01526_b200.report [--out FILE]``.

For every GEMM of the benchmark configurations (single 256-cube, MLP step, ResNet im2col
convolutions, transformer layer, large sweep) it times, with CUDA events on the current stream,
the conversion of each FP32 operand to block floating point and the BFP GEMM on already-packed
operands, and prints one markdown table row per GEMM. Weights in shared tiles are converted once
per layer (both views) and re-used by forward and backward-data, as in training.
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


def rows_for(specs, tensors_np, peak_tops, hbm_gbs):
    dev = {k: torch.from_numpy(v).cuda() for k, v in tensors_np.items()}
    out = []
    for sp in specs:
        A, B = dev[sp.a_key], dev[sp.b_key]
        fa, fb = hb.Format(**sp.fmt_a), hb.Format(**sp.fmt_b)
        a_axis = 0 if sp.transA else 1           # contraction axis of the stored A
        b_axis = 1 if sp.transB else 0
        pa = hb.quantize(A, a_axis, fa)
        t_qa = _time(lambda: hb.quantize(A, a_axis, fa, out=pa))
        if fb.tile > 0:
            c0, c1, _ = hb.quantize_tiles(B, fb)
            t_qb = _time(lambda: hb.quantize_tiles(B, fb, out=(c0, c1), want_grid=False))
            pb = c1 if sp.transB else c0
        else:
            pb = hb.quantize(B, b_axis, fb)
            t_qb = _time(lambda: hb.quantize(B, b_axis, fb, out=pb))
        C = torch.empty((sp.M, sp.N), dtype=torch.float32, device="cuda")
        ws = torch.empty(max(hb.gemm_q_workspace(sp.M, sp.N, sp.K, pa, pb), 1), dtype=torch.int8, device="cuda")
        t_g = _time(lambda: hb.gemm_q(sp.M, sp.N, sp.K, pa, pb, out=C, workspace=ws))
        ops = sp.ops
        planes = 1 if fa.mant_bits <= 8 else 2
        qa_bytes = A.numel() * (4 + planes + 1.0 / max(fa.block, 1))
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
    args = ap.parse_args()
    hb.lib()
    lines = ["| GEMM | M x N x K | format | quantise A µs | quantise B µs | GEMM µs | quantise A GB/s (% HBM) | GEMM-only TOPS | "
             "quantise+GEMM TOPS (% of measured int8 proxy / % of nominal 4500) |", "|---|---|---|---|---|---|---|---|---|"]
    for name, specs, seed in (("single", wl.config_single_256(), 0), ("mlp", wl.config_mlp(), 1),
                              ("resnet", wl.config_resnet_im2col(), 2), ("transformer", wl.config_transformer(), 7)):
        lines += rows_for(specs, wl.materialize(specs, seed=seed), args.peak_tops, args.hbm_gbs)
    for n in args.sweep:
        for (m, b, r) in ((8, 128, 0), (8, 64, 0), (8, 32, 0), (8, 128, 1), (12, 64, 1)):
            specs = wl.config_sweep(n, m, b, r)
            t = {specs[0].a_key: wl.draw("lognormal", (n, n), seed=3, salt=0),
                 specs[0].b_key: wl.draw("lognormal", (n, n), seed=3, salt=1)}
            lines += rows_for(specs, t, args.peak_tops, args.hbm_gbs)
    text = "\n".join(lines) + "\n"
    if args.out:
        with open(args.out, "w") as f:
            f.write(text)
    sys.stdout.write(text)
    if hb.device_status() != 0:
        raise SystemExit("device status non-zero")


if __name__ == "__main__":
    main()
