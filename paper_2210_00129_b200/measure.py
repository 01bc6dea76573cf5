"""Per-call timing sweep over the paper's layer shapes, against the roofline of each call.

    python -m paper_2210_00129_b200.measure [--group vit|convnext|detection|forward|blocks|sampler|all] [--iters 24]

For every layer of the chosen groups (ViT-B/16 MLP and attention projections at four keep ratios,
ConvNeXt-B point-wise layers of the four stages with random and grid masks, the detection-resolution
map; Sec. 5 of the paper gives the models) it times `sbp_sample_keep`, `sbp_forward_cache` and
`sbp_linear_backward` (dW alone, dX alone, db alone, both products, all three) on one GPU and prints a markdown table:
microseconds, the lower bound `t_min = max(FLOP / peak, bytes / bandwidth)` of the call's algorithmic
work, `t_min / t`, and the speed-up of the whole backward over keep ratio 1.0.

Timing: each call is captured `iters` times into a CUDA graph over rotating buffer sets whose total
size exceeds the L2 cache (so every launch reads its inputs from HBM and no host launch gap is inside the
timed region), the graph is replayed once untimed and once between two CUDA events.  All arithmetic runs
in the library's kernels; torch only holds the buffers.
"""
import argparse
import json
import os
import sys

import torch

import paper_2210_00129_b200 as sbp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FALLBACK = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK), "fallback"


def layers(group):
    """(name, B, H, W, C_in, C_out, keep ratio, mask mode) of every layer of a group."""
    out = []
    if group in ("vit", "all"):
        out.append(("vit_b16 fc1 B=64", 64, 14, 14, 768, 3072, 0.5, 0))
        for r in (0.25, 0.5, 0.75, 1.0):
            for nm, ci, co in (("qkv", 768, 2304), ("proj", 768, 768), ("fc1", 768, 3072), ("fc2", 3072, 768)):
                out.append((f"vit_b16 {nm} B=128 r={r}", 128, 14, 14, ci, co, r, 0))
    if group in ("convnext", "all"):
        for mode in (0, 1):
            for st, (dim, hw) in enumerate(((128, 56), (256, 28), (512, 14), (1024, 7)), 1):
                for nm, ci, co in (("pw1", dim, 4 * dim), ("pw2", 4 * dim, dim)):
                    out.append((f"convnext_b s{st} {nm} {'grid' if mode else 'random'}", 64, hw, hw, ci, co, 0.5, mode))
    if group in ("detection", "all"):
        for nm, ci, co in (("128->512", 128, 512), ("512->128", 512, 128)):
            out.append((f"detection 200x334 {nm}", 2, 200, 334, ci, co, 0.5, 0))
    return out


class Bench:
    def __init__(self, iters):
        self.iters = iters
        self.stream = torch.cuda.Stream()
        self.sid = self.stream.cuda_stream

    def time_us(self, fn, n_sets):
        """fn(set index, step) enqueues one call on self.stream; returns microseconds per call."""
        with torch.cuda.stream(self.stream):
            for i in range(3):
                fn(i % n_sets, i)
            self.stream.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=self.stream):
                for i in range(self.iters):
                    fn(i % n_sets, i)
        g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / self.iters * 1e3


def measure_layer(bench, spec, pk):
    name, B, H, W_, C_in, C_out, r, mode = spec
    es = 2
    M = B * H * W_
    cap = B * sbp.sbp_keep_count(mode, H, W_, r)
    set_bytes = (2 * M * C_in + M * C_out + C_in * C_out + cap * C_in) * es + C_in * C_out * 4
    n_sets = max(3, int(400e6 // set_bytes) + 1)
    gen = torch.Generator(device="cuda").manual_seed(1234)
    sets = []
    for _ in range(n_sets):
        sets.append(dict(
            X=torch.randn(M, C_in, device="cuda", generator=gen).bfloat16(),
            dY=(torch.randn(M, C_out, device="cuda", generator=gen) * 0.01).bfloat16(),
            W=(torch.randn(C_in, C_out, device="cuda", generator=gen) * 0.02).bfloat16(),
            rows=torch.zeros(cap, dtype=torch.int32, device="cuda"),
            offs=torch.zeros(B + 1, dtype=torch.int32, device="cuda"),
            Xk=torch.zeros(cap, C_in, device="cuda", dtype=torch.bfloat16),
            dW=torch.zeros(C_in, C_out, device="cuda"), db=torch.zeros(C_out, device="cuda"),
            dX=torch.zeros(M, C_in, device="cuda", dtype=torch.bfloat16)))
    nb = sbp.sbp_linear_backward_workspace_bytes(sbp.SBP_BF16, M, cap, C_in, C_out)
    ws = torch.empty(max(nb, 16), dtype=torch.uint8, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    sid = bench.sid
    torch.cuda.synchronize()      # the buffers were filled on torch's stream; the calls below run on another

    def cnt(s):          # device-side row count (grid masks on odd maps keep 24 or 25 of 49)
        return s["offs"][B:] if mode == 1 else None

    def sample(k, i):
        s = sets[k]
        sbp.sbp_sample_keep(mode, B, H, W_, r, 0, i, 0, 0, s["rows"], s["offs"], stream=sid)

    def cache(k, i):
        s = sets[k]
        sbp.sbp_forward_cache(sbp.SBP_BF16, s["X"], M, C_in, s["rows"], cnt(s), cap, s["Xk"], stream=sid)

    def bw(k, dW, db, dX):
        s = sets[k]
        sbp.sbp_linear_backward(sbp.SBP_BF16, s["Xk"], s["dY"], s["W"], s["rows"], cnt(s), M, cap, C_in, C_out,
                                s["dW"] if dW else None, s["db"] if db else None, s["dX"] if dX else None, 0, ws, nb,
                                st, stream=sid)

    with torch.cuda.stream(bench.stream):
        for k in range(n_sets):
            sample(k, 0)
            cache(k, 0)
    bench.stream.synchronize()
    M_keep = int(sets[0]["offs"][B].item())

    t = {
        "sample": bench.time_us(sample, n_sets),
        "cache": bench.time_us(cache, n_sets),
        "db": bench.time_us(lambda k, i: bw(k, 0, 1, 0), n_sets),
        "dW": bench.time_us(lambda k, i: bw(k, 1, 0, 0), n_sets),
        "dX": bench.time_us(lambda k, i: bw(k, 0, 0, 1), n_sets),
        "dW+dX": bench.time_us(lambda k, i: bw(k, 1, 0, 1), n_sets),
        "bwd": bench.time_us(lambda k, i: bw(k, 1, 1, 1), n_sets),
    }
    assert int(st.item()) == 0, f"status word {int(st.item())} on {name}"
    flop = 2.0 * M_keep * C_in * C_out
    tf, bw_ = pk["bf16_tflops_sustained"] * 1e12, pk["hbm_gbs"] * 1e9
    by = {   # algorithmic HBM bytes of each call
        "sample": 4.0 * M_keep + 4 * (B + 1),
        "cache": 2.0 * M_keep * C_in * es + 4 * M_keep,
        "db": M_keep * C_out * es + 4.0 * M_keep,
        "dW": M_keep * (C_in + C_out) * es + 4.0 * C_in * C_out,
        "dX": M_keep * C_out * es + C_in * C_out * es + M * C_in * es,
    }
    by["bwd"] = M_keep * (C_in + C_out) * es + C_in * C_out * es + 4.0 * C_in * C_out + M * C_in * es + 4 * C_out
    by["dW+dX"] = by["bwd"] - 4 * C_out
    fl = {"sample": 0.0, "cache": 0.0, "db": 0.0, "dW": flop, "dX": flop, "dW+dX": 2 * flop, "bwd": 2 * flop}
    tmin = {k: max(fl[k] / tf, by[k] / bw_) * 1e6 for k in t}
    bound = {k: ("tensor" if fl[k] / tf > by[k] / bw_ else "hbm") for k in t}
    del sets
    torch.cuda.empty_cache()
    return dict(name=name, M=M, M_keep=M_keep, t=t, tmin=tmin, bound=bound, flop=flop, bytes=by)


def mlp_block(bench, B, H, W_, d, h, r):
    """Backward of a two-layer block d -> h -> d (a ViT MLP, a ConvNeXt block's point-wise pair; upper layer first)
    with the same keep set on both layers: the gradient between the layers scattered to all rows and gathered
    again, against kept packed (Eq. 9)."""
    M = B * H * W_
    cap = B * sbp.sbp_keep_count(0, H, W_, r)
    gen = torch.Generator(device="cuda").manual_seed(99)
    rn = lambda *sh: torch.randn(*sh, device="cuda", generator=gen)
    n_sets = 3
    sets = []
    for _ in range(n_sets):
        sets.append(dict(X0k=rn(cap, d).bfloat16(), X1k=rn(cap, h).bfloat16(), dY=(rn(M, d) * 0.01).bfloat16(),
                         W1=(rn(d, h) * 0.02).bfloat16(), W2=(rn(h, d) * 0.02).bfloat16(),
                         dW1=torch.zeros(d, h, device="cuda"), db1=torch.zeros(h, device="cuda"),
                         dW2=torch.zeros(h, d, device="cuda"), db2=torch.zeros(d, device="cuda"),
                         dX1=torch.zeros(M, h, device="cuda", dtype=torch.bfloat16),
                         dX0=torch.zeros(M, d, device="cuda", dtype=torch.bfloat16),
                         rows=torch.zeros(cap, dtype=torch.int32, device="cuda"),
                         offs=torch.zeros(B + 1, dtype=torch.int32, device="cuda")))
    nb = max(sbp.sbp_linear_backward_workspace_bytes(sbp.SBP_BF16, M, cap, d, h),
             sbp.sbp_linear_backward_workspace_bytes(sbp.SBP_BF16, M, cap, h, d))
    ws = torch.empty(nb, dtype=torch.uint8, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    with torch.cuda.stream(bench.stream):
        for s in sets:
            sbp.sbp_sample_keep(0, B, H, W_, r, 0, 0, 0, 0, s["rows"], s["offs"], stream=bench.sid)
    bench.stream.synchronize()

    def block(k, packed):
        s = sets[k]
        up, low = (sbp.SBP_FLAG_DX_COMPACT, sbp.SBP_FLAG_DY_COMPACT) if packed else (0, 0)
        sbp.sbp_linear_backward(sbp.SBP_BF16, s["X1k"], s["dY"], s["W2"], s["rows"], None, M, cap, h, d, s["dW2"], s["db2"],
                                s["dX1"], up, ws, nb, st, stream=bench.sid)
        sbp.sbp_linear_backward(sbp.SBP_BF16, s["X0k"], s["dX1"], s["W1"], s["rows"], None, M, cap, d, h, s["dW1"], s["db1"],
                                s["dX0"], low, ws, nb, st, stream=bench.sid)

    t_scatter = bench.time_us(lambda k, i: block(k, False), n_sets)
    t_packed = bench.time_us(lambda k, i: block(k, True), n_sets)
    assert int(st.item()) == 0
    flop = 8.0 * cap * d * h
    return cap, t_scatter, t_packed, flop


def forward_layers(bench, pk):
    """sbp_linear_forward with the cache fused in, against the forward alone followed by sbp_forward_cache."""
    rows = []
    for name, B, H, W_, C_in, C_out, r in (("vit_b16 fc1 B=64", 64, 14, 14, 768, 3072, 0.5), ("vit_b16 fc2 B=64", 64, 14, 14, 3072, 768, 0.5),
                                           ("vit_b16 fc1 B=128", 128, 14, 14, 768, 3072, 0.5), ("vit_b16 qkv B=128", 128, 14, 14, 768, 2304, 0.5),
                                           ("convnext_b s1 pw1", 64, 56, 56, 128, 512, 0.5), ("convnext_b s1 pw2", 64, 56, 56, 512, 128, 0.5),
                                           ("convnext_b s3 pw1", 64, 14, 14, 512, 2048, 0.5)):
        M = B * H * W_
        cap = B * sbp.sbp_keep_count(0, H, W_, r)
        gen = torch.Generator(device="cuda").manual_seed(7)
        set_bytes = (M * C_in + M * C_out + C_in * C_out + cap * C_in) * 2
        n_sets = max(3, int(400e6 // set_bytes) + 1)
        sets = [dict(X=torch.randn(M, C_in, device="cuda", generator=gen).bfloat16(),
                     W=(torch.randn(C_in, C_out, device="cuda", generator=gen) * 0.02).bfloat16(),
                     b=torch.randn(C_out, device="cuda", generator=gen), Y=torch.zeros(M, C_out, device="cuda", dtype=torch.bfloat16),
                     Xk=torch.zeros(cap, C_in, device="cuda", dtype=torch.bfloat16), rows=torch.zeros(cap, dtype=torch.int32, device="cuda"),
                     offs=torch.zeros(B + 1, dtype=torch.int32, device="cuda")) for _ in range(n_sets)]
        torch.cuda.synchronize()
        with torch.cuda.stream(bench.stream):
            for s in sets:
                sbp.sbp_sample_keep(0, B, H, W_, r, 0, 0, 0, 0, s["rows"], s["offs"], stream=bench.sid)
        bench.stream.synchronize()

        def fused(k, i):
            s = sets[k]
            sbp.sbp_linear_forward(sbp.SBP_BF16, s["X"], s["W"], s["b"], M, C_in, C_out, s["Y"], s["rows"], None, cap, s["Xk"],
                                   stream=bench.sid)

        def separate(k, i):
            s = sets[k]
            sbp.sbp_linear_forward(sbp.SBP_BF16, s["X"], s["W"], s["b"], M, C_in, C_out, s["Y"], stream=bench.sid)
            sbp.sbp_forward_cache(sbp.SBP_BF16, s["X"], M, C_in, s["rows"], None, cap, s["Xk"], stream=bench.sid)

        tf, ts = bench.time_us(fused, n_sets), bench.time_us(separate, n_sets)
        flop = 2.0 * M * C_in * C_out
        by = (M * C_in + C_in * C_out + M * C_out + cap * C_in) * 2.0
        tmin = max(flop / (pk["bf16_tflops_sustained"] * 1e12), by / (pk["hbm_gbs"] * 1e9)) * 1e6
        rows.append((name, M, tf, ts, tmin, flop / tf / 1e6))
        del sets
        torch.cuda.empty_cache()
    return rows


def sampler_stress(bench, pk):
    """Sampler alone on a shape whose index stream is large enough to read as bandwidth."""
    rows = []
    for B, H, W_, r in ((4096, 56, 56, 0.5), (4096, 14, 14, 0.5), (2, 200, 334, 0.5)):
        cap = B * sbp.sbp_keep_count(0, H, W_, r)
        bufs = [(torch.zeros(cap, dtype=torch.int32, device="cuda"), torch.zeros(B + 1, dtype=torch.int32, device="cuda"))
                for _ in range(3)]
        torch.cuda.synchronize()
        us = bench.time_us(lambda k, i: sbp.sbp_sample_keep(0, B, H, W_, r, 0, i, 0, 0, bufs[k][0], bufs[k][1],
                                                            stream=bench.sid), 3)
        rows.append((B, H, W_, cap, us, 4.0 * cap / us / 1e3, B * H * W_ / us / 1e3))
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--group", default="all", choices=["vit", "convnext", "detection", "forward", "blocks", "sampler", "all"])
    ap.add_argument("--iters", type=int, default=24)
    ap.add_argument("--compact", action="store_true", help="one table row per layer: us (t_min / t) per call")
    args = ap.parse_args()
    sbp.load_library()
    pk, kind = peaks()
    bench = Bench(args.iters)
    print(f"peaks ({kind}): bf16 {pk['bf16_tflops_sustained']:.0f} TFLOP/s sustained, HBM {pk['hbm_gbs']:.0f} GB/s; "
          f"{args.iters} graph-replayed launches per figure, rotating buffer sets larger than L2\n")
    if args.group not in ("sampler", "blocks", "forward"):
        if args.compact:
            print("us (t_min / t) per call; bound of the whole backward in the last column\n")
            print("| layer | M_keep | sample | cache | db | dW | dX | dW+dX (one launch) | backward (dW+db+dX) | TFLOP/s | bound |")
            print("|---|---|---|---|---|---|---|---|---|---|---|")
        else:
            print("| layer | M_keep | call | us | t_min us | t_min/t | bound | achieved |")
            print("|---|---|---|---|---|---|---|---|")
        full = {}
        res = []
        for spec in layers(args.group):
            m = measure_layer(bench, spec, pk)
            res.append((spec, m))
            if args.compact:
                cells = " | ".join(f"{m['t'][k]:.1f} ({m['tmin'][k] / m['t'][k]:.2f})" for k in ("cache", "db", "dW", "dX", "dW+dX", "bwd"))
                print(f"| {m['name']} | {m['M_keep']} | {m['t']['sample']:.1f} | {cells} | "
                      f"{2 * m['flop'] / m['t']['bwd'] / 1e6:.0f} | {m['bound']['bwd']} |")
            for k in (() if args.compact else ("sample", "cache", "db", "dW", "dX", "dW+dX", "bwd")):
                us = m["t"][k]
                if k in ("dW", "dX", "dW+dX", "bwd"):
                    ach = f"{(2 if k in ('bwd', 'dW+dX') else 1) * m['flop'] / us / 1e6:.0f} TFLOP/s"
                else:
                    ach = f"{m['bytes'][k] / us / 1e3:.0f} GB/s"
                print(f"| {m['name']} | {m['M_keep']} | {k} | {us:.1f} | {m['tmin'][k]:.1f} | {m['tmin'][k] / us:.2f} | "
                      f"{m['bound'][k]} | {ach} |")
            sys.stdout.flush()
            if spec[6] == 1.0:
                full[(spec[1], spec[2], spec[3], spec[4], spec[5], spec[7])] = m["t"]["bwd"]
        lines = []
        for spec, m in res:
            key = (spec[1], spec[2], spec[3], spec[4], spec[5], spec[7])
            if key in full and spec[6] != 1.0:
                lines.append(f"| {m['name']} | {spec[6]} | {m['t']['bwd']:.1f} | {full[key]:.1f} | {full[key] / m['t']['bwd']:.2f} | {1 / spec[6]:.2f} |")
        if lines:
            print("\n| layer | keep ratio | backward us | at keep 1.0 us | speed-up | 1/r |")
            print("|---|---|---|---|---|---|")
            print("\n".join(lines))
    if args.group in ("forward", "all"):
        print("\n| forward Y = XW + b with the cache (sbp_linear_forward) | M | fused us | forward + sbp_forward_cache us | "
              "t_min us | t_min/t | TFLOP/s |")
        print("|---|---|---|---|---|---|---|")
        for name, M, tf, ts, tmin, tfl in forward_layers(bench, pk):
            print(f"| {name} | {M} | {tf:.1f} | {ts:.1f} | {tmin:.1f} | {tmin / tf:.2f} | {tfl:.0f} |")
    if args.group in ("blocks", "all"):
        print("\n| two-layer block backward, d -> 4d -> d (both layers, dW + db + dX each) | M_keep | gradient between "
              "the layers scattered, us | packed, us | gain | packed TFLOP/s |")
        print("|---|---|---|---|---|---|")
        blocks = [("vit_b16 MLP B=64 r=0.5", 64, 14, 14, 768, 0.5), ("vit_b16 MLP B=128 r=0.25", 128, 14, 14, 768, 0.25),
                  ("vit_b16 MLP B=128 r=0.5", 128, 14, 14, 768, 0.5), ("vit_b16 MLP B=128 r=0.75", 128, 14, 14, 768, 0.75),
                  ("convnext_b s1 block", 64, 56, 56, 128, 0.5), ("convnext_b s2 block", 64, 28, 28, 256, 0.5),
                  ("convnext_b s3 block", 64, 14, 14, 512, 0.5), ("detection 200x334 block", 2, 200, 334, 128, 0.5)]
        for nm, B, H, W_, d, r in blocks:
            cap, ts, tp, flop = mlp_block(bench, B, H, W_, d, 4 * d, r)
            print(f"| {nm} | {cap} | {ts:.1f} | {tp:.1f} | {ts / tp:.2f} | {flop / tp / 1e6:.0f} |")
    if args.group in ("sampler", "all"):
        print("\n| sampler shape | kept ids | us | index stream GB/s | positions per ns |")
        print("|---|---|---|---|---|")
        for B, H, W_, cap, us, gbs, pos in sampler_stress(bench, pk):
            print(f"| B={B}, {H}x{W_} | {cap} | {us:.1f} | {gbs:.1f} | {pos:.2f} |")


if __name__ == "__main__":
    main()
