"""The paper's kernel benchmark grid (appendix "Kernel Benchmarks"): tokens 2^12..2^16 x the 17 hidden
sizes {k * 2^r, k in 1,3,5,7} within [2^10, 2^14] x block sizes, Gaussian input, forward only, norm gain
folded away; speed-up of `mxnorm_fwd` over the fused conventional path `rmsnorm_mxfp8_fwd`, geometric mean
over the grid.  Both sides are this library's hand-written kernels on the same GPU (the paper compares two
torch.compile kernels on a GB200).

Each case is timed as the replay of a CUDA graph of back-to-back launches over rotating buffer sets (3x L2).

    python -m paper_2603_13180_b200.sweep [--blocks 32] [--elem e4m3|e2m1|nvfp4] [--tokens 4096 16384 65536] [--json out.json] [--md out.md]

`--md` appends compact tables (one row per token count, one column per hidden size) to a Markdown file: bandwidth of
`mxnorm_fwd` as a fraction of the measured copy peak, its speed-up over the conventional kernel, and - as a yardstick
for the small cases, where a launch is too short to reach the peak whatever it does - the bandwidth of a plain
device-to-device copy that moves the same number of bytes, timed the same way.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import time

import torch


TOKENS = [2 ** 12, 2 ** 13, 2 ** 14, 2 ** 15, 2 ** 16]
HIDDEN = sorted({k * 2 ** r for k in (1, 3, 5, 7) for r in range(4, 15) if 2 ** 10 <= k * 2 ** r <= 2 ** 14})
EPS = 1e-5


def _time(fn, sets, steps, warmup, stream, graph=True):
    """Microseconds per launch over `steps` back-to-back launches that rotate over `sets` buffer sets.
    With graph=True the launches are captured once into a CUDA graph and the replay is timed, so that
    kernels of a few microseconds are not limited by the host's launch rate."""
    for i in range(warmup):
        fn(i % sets)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if graph:
        g = torch.cuda.CUDAGraph()
        torch.cuda.synchronize()
        with torch.cuda.graph(g, stream=stream):
            for i in range(steps):
                fn(i % sets)
        g.replay()                     # untimed: uploads the graph
        torch.cuda.synchronize()
        a.record(stream)
        g.replay()
        b.record(stream)
    else:
        torch.cuda.synchronize()
        a.record(stream)
        for i in range(steps):
            fn(i % sets)
        b.record(stream)
    torch.cuda.synchronize()
    return a.elapsed_time(b) / steps * 1e3   # microseconds


REST_S = 0.25   # idle time before each case: every case is a burst measurement (like the measured copy peak), not a
                # point in one long uninterrupted load, which on this pool runs the same kernels up to 8 % slower


def run(tokens, hidden, blocks, steps=30, warmup=5, l2_bytes=126 << 20, elem="e4m3", graph=True):
    stream = torch.cuda.Stream()       # a side stream: the default stream cannot be captured
    stream.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(stream):
        return _run(stream, tokens, hidden, blocks, steps, warmup, l2_bytes, elem, graph)


def _run(stream, tokens, hidden, blocks, steps, warmup, l2_bytes, elem, graph):
    from . import binding as mx   # needs the compiled library and a GPU; the table formatting below does not
    sh = stream.cuda_stream
    L = mx.lib
    rows = []
    for B in blocks:
        for T in tokens:
            for D in hidden:
                nv4 = elem == "nvfp4"
                if nv4 and B != 16:
                    continue
                fp4 = elem == "e2m1" or nv4
                per_set = T * D * 2 + (T * D // 2 if fp4 else T * D) + T * (D // B) + 4 * T
                sets = max(2, min(8, -(-3 * l2_bytes // per_set)))        # working set of at least 3x L2
                g = torch.Generator(device="cuda").manual_seed(T + D)
                xs = [torch.randn(T, D, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16) for _ in range(sets)]
                outs = [mx.alloc_outputs(T, D, B, mx.SCALES_SWIZZLE_128x4, nvfp4=fp4) for _ in range(sets)]

                def mxn(i):
                    c, s, r = outs[i]
                    if nv4:
                        st = L.mxnorm_nvfp4_fwd(xs[i].data_ptr(), T, D, 2, 0.0, EPS, 1.0, c.data_ptr(), s.data_ptr(), r.data_ptr(),
                                                mx.SCALES_SWIZZLE_128x4, sh)
                        assert st == 0, mx.status_string(st)
                        return
                    if fp4:
                        st = L.mxnorm_mxfp4_fwd(xs[i].data_ptr(), T, D, B, 2, 0.0, EPS, c.data_ptr(), s.data_ptr(), r.data_ptr(),
                                                mx.SCALES_SWIZZLE_128x4, sh)
                        assert st == 0, mx.status_string(st)
                        return
                    st = L.mxnorm_fwd(xs[i].data_ptr(), None, T, D, B, 2, 0.0, EPS, c.data_ptr(), s.data_ptr(), r.data_ptr(),
                                      0, mx.SCALES_SWIZZLE_128x4, sh)
                    assert st == 0, mx.status_string(st)

                def rms(i):
                    c, s, r = outs[i]
                    if nv4:
                        st = L.rmsnorm_nvfp4_fwd(xs[i].data_ptr(), T, D, EPS, 1.0, c.data_ptr(), s.data_ptr(), r.data_ptr(),
                                                 mx.SCALES_SWIZZLE_128x4, sh)
                        assert st == 0, mx.status_string(st)
                        return
                    if fp4:
                        st = L.rmsnorm_mxfp4_fwd(xs[i].data_ptr(), T, D, B, EPS, c.data_ptr(), s.data_ptr(), r.data_ptr(),
                                                 mx.SCALES_SWIZZLE_128x4, sh)
                        assert st == 0, mx.status_string(st)
                        return
                    st = L.rmsnorm_mxfp8_fwd(xs[i].data_ptr(), None, T, D, B, EPS, c.data_ptr(), s.data_ptr(), r.data_ptr(),
                                             0, mx.SCALES_SWIZZLE_128x4, sh)
                    assert st == 0, mx.status_string(st)

                torch.cuda.synchronize()
                time.sleep(REST_S)
                t_mx = min(_time(mxn, sets, steps, warmup, stream, graph) for _ in range(2))
                t_rms = min(_time(rms, sets, steps, warmup, stream, graph) for _ in range(2))
                # yardstick: an elementwise copy kernel over per_set / 2 bytes (it reads and writes them: per_set bytes of
                # traffic), as 32-bit words so that it is a plain vectorised kernel and not a copy-engine transfer
                half = per_set // 2 // 16 * 16
                src = [torch.zeros(half // 4, dtype=torch.int32, device="cuda") for _ in range(sets)]
                dst = [torch.empty(half // 4, dtype=torch.int32, device="cuda") for _ in range(sets)]

                def cpy(i):
                    torch.add(src[i], 1, out=dst[i])

                t_cp = min(_time(cpy, sets, steps, warmup, stream, graph) for _ in range(2))
                rows.append({"elem": elem, "block": B, "tokens": T, "hidden": D, "mxnorm_us": t_mx, "rmsnorm_us": t_rms,
                             "speedup": t_rms / t_mx, "mxnorm_gbs": per_set / t_mx / 1e3, "rmsnorm_gbs": per_set / t_rms / 1e3,
                             "copy_us": t_cp, "copy_gbs": 2 * half / t_cp / 1e3})
                del xs, outs, src, dst
    return rows


def summarise(rows):
    out = {}
    for B in sorted({r["block"] for r in rows}):
        sel = [r for r in rows if r["block"] == B]
        out[f"B={B}"] = {
            "cases": len(sel),
            "geomean_speedup": math.exp(sum(math.log(r["speedup"]) for r in sel) / len(sel)),
            "max_speedup": max(r["speedup"] for r in sel),
            "min_speedup": min(r["speedup"] for r in sel),
            "geomean_mxnorm_gbs": math.exp(sum(math.log(r["mxnorm_gbs"]) for r in sel) / len(sel)),
            "min_mxnorm_gbs": min(r["mxnorm_gbs"] for r in sel),
        }
    return out


def measured_peak_gbs() -> float:
    """The machine's measured copy bandwidth (generated file at the repository root), else the stated fallback."""
    path = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"])
    except Exception:
        return 6650.0


def markdown_tables(rows, peak: float, compact: bool = False) -> str:
    """Compact tables per (element format, block size): rows = tokens, columns = hidden sizes
    (compact: only the two bandwidth-fraction tables)."""
    out = []
    for elem in sorted({r["elem"] for r in rows}):
        for B in sorted({r["block"] for r in rows if r["elem"] == elem}):
            sel = [r for r in rows if r["elem"] == elem and r["block"] == B]
            hidden = sorted({r["hidden"] for r in sel})
            tokens = sorted({r["tokens"] for r in sel})
            cell = {(r["tokens"], r["hidden"]): r for r in sel}
            big = [r for r in sel if r["tokens"] >= 16384]
            gm = math.exp(sum(math.log(r["speedup"]) for r in sel) / len(sel))
            out.append(f"### {elem}, block {B}: {len(sel)} cases, geometric-mean speed-up {gm:.3f} "
                       f"(max {max(r['speedup'] for r in sel):.3f}, min {min(r['speedup'] for r in sel):.3f})\n")
            if big:
                worst = min(big, key=lambda r: r["mxnorm_gbs"])
                out.append(f"Lowest `mxnorm` bandwidth at 16384 tokens and more: {worst['mxnorm_gbs']:.0f} GB/s = {worst['mxnorm_gbs'] / peak:.2f} of the "
                           f"measured peak at T = {worst['tokens']}, D = {worst['hidden']} (a copy of the same bytes: {worst['copy_gbs']:.0f} GB/s).\n")
            for title, fn in (("`mxnorm` bandwidth / measured copy peak", lambda r: f"{r['mxnorm_gbs'] / peak:.2f}"),
                              ("`mxnorm` microseconds per launch", lambda r: f"{r['mxnorm_us']:.1f}"),
                              ("speed-up over the conventional kernel", lambda r: f"{r['speedup']:.2f}"),
                              ("`mxnorm` bandwidth / bandwidth of a copy of the same bytes", lambda r: f"{r['mxnorm_gbs'] / r['copy_gbs']:.2f}")):
                if compact and ("microseconds" in title or "speed-up" in title):
                    continue
                out.append(f"{title}:\n")
                out.append("| tokens \\ hidden | " + " | ".join(str(h) for h in hidden) + " |")
                out.append("|---|" + "---|" * len(hidden))
                for T in tokens:
                    out.append(f"| {T} | " + " | ".join(fn(cell[(T, h)]) if (T, h) in cell else "" for h in hidden) + " |")
                out.append("")
    return "\n".join(out) + "\n"


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--blocks", type=int, nargs="+", default=[32])
    ap.add_argument("--tokens", type=int, nargs="+", default=TOKENS)
    ap.add_argument("--hidden", type=int, nargs="+", default=HIDDEN)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--elem", default="e4m3", choices=["e4m3", "e2m1", "nvfp4"],
                    help="element format: e4m3/e2m1 with E8M0 scales, or nvfp4 (E2M1 codes, E4M3 scales, block 16)")
    ap.add_argument("--no-graph", action="store_true", help="time direct launches instead of a CUDA-graph replay")
    ap.add_argument("--json", default="")
    ap.add_argument("--md", default="", help="append compact Markdown tables to this file")
    ap.add_argument("--compact", action="store_true", help="with --md: only the two bandwidth-fraction tables per format")
    ap.add_argument("--from-json", nargs="+", default=[], help="render --md from result files written by --json (no GPU needed)")
    args = ap.parse_args()
    if args.from_json:
        rows = []
        for path in args.from_json:
            with open(path) as f:
                rows += json.load(f)["rows"]
        with open(args.md, "a") as f:
            f.write(markdown_tables(rows, measured_peak_gbs(), args.compact))
        return
    rows = run(args.tokens, args.hidden, args.blocks, steps=args.steps, elem=args.elem, graph=not args.no_graph)
    summary = summarise(rows)
    for r in rows:
        print(f"{r['elem']} B={r['block']:2d} T={r['tokens']:6d} D={r['hidden']:6d}  mxnorm {r['mxnorm_us']:9.2f} us {r['mxnorm_gbs']:6.0f} GB/s   "
              f"rmsnorm+cast {r['rmsnorm_us']:9.2f} us {r['rmsnorm_gbs']:6.0f} GB/s   speedup {r['speedup']:.3f}")
    print(json.dumps(summary))
    if args.json:
        with open(args.json, "w") as f:
            json.dump({"rows": rows, "summary": summary}, f)
    if args.md:
        with open(args.md, "a") as f:
            f.write(markdown_tables(rows, measured_peak_gbs(), args.compact))


if __name__ == "__main__":
    main()
