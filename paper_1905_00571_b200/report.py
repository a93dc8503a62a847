"""Measurement report: whole-network and per-layer times of the synthetic pruned networks, the
fraction of the sparse roofline they reach, and the same layers run dense.

    python -m paper_1905_00571_b200.report --workload resnet50 --batch 1 8 --density 0.125 1.0 [--layers]

Everything timed here runs through the C ABI (argument marshalling only in Python).  The dense
comparison is (i) this library at density 1.0 and (ii), as labelled context, torch's cuDNN
convolutions on the same shapes (fp32 with TF32 off, and TF32 on) - library calls only.
Prints markdown.
"""
import argparse
import sys

import numpy as np
import torch

from workloads import models
from . import binding as B
from . import roofline
from .network import PackedModel


def build(workload, density):
    if workload == "resnet50":
        fc = 0.10 if density < 1.0 else 1.0
        return models.resnet50(density=density, fc_density=fc)
    if workload == "mobilenet_v2":
        return models.mobilenet_v2(density=density)
    if workload == "vgg16":
        return models.vgg16(density=density, fc_density=min(1.0, density / 2))
    if workload == "resnet50_int8":
        return models.resnet50_int8(density=density, fc_density=0.10 if density < 1.0 else 1.0)
    if workload == "mobilenet_v1":
        return models.mobilenet_v1(density=density)
    if workload == "inception_v3":
        return models.inception_v3(density=density, fc_density=0.10 if density < 1.0 else 1.0)
    if workload == "vgg16_block":   # block-structured pruning: `density` is the fraction of 64 x 64 blocks kept
        return models.vgg16_block(block_density=density)
    raise SystemExit("unknown workload " + workload)


def time_forward(pm, x, y, reps=50):
    pm.forward(x, y)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        pm.forward(x, y)
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / reps


def torch_dense_ms(model, batch, tf32, reps=20):
    """cuDNN convolutions / matmuls on the same layer shapes (dense weights), layer by layer."""
    if model.dtype != "f32":
        return None
    torch.backends.cudnn.allow_tf32 = tf32
    torch.backends.cuda.matmul.allow_tf32 = tf32
    layers = []
    for op in model.ops:
        if op.kind == "conv":
            kh, kw = int(op.w.shape[1]), int(op.w.shape[2])
            pad = (op.pad, op.pad if getattr(op, "pad_w", -1) < 0 else op.pad_w)
            w = torch.randn(op.c_out, op.c_in // op.groups, kh, kw, device="cuda").contiguous(memory_format=torch.channels_last)
            xin = torch.randn(batch, op.c_in, op.in_hw[0], op.in_hw[1], device="cuda").contiguous(memory_format=torch.channels_last)
            layers.append((lambda xin=xin, w=w, op=op, pad=pad: torch.nn.functional.conv2d(xin, w, None, op.stride, pad, 1, op.groups)))
        elif op.kind == "fc":
            w = torch.randn(op.c_out, op.c_in, device="cuda")
            xin = torch.randn(batch, op.c_in, device="cuda")
            layers.append((lambda xin=xin, w=w: xin @ w.t()))
    for f in layers:
        f()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for f in layers:
            f()
    g.replay()
    torch.cuda.synchronize()
    a.record()
    for _ in range(reps):
        g.replay()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / reps


def block_crossover(batches):
    """Block-structured int8 layer (a VGG conv3 shape, 256 -> 256, 3x3, 56x56): the tensor-core route for its
    64 x 64 blocks against the sparse CUDA-core kernel on the same mask, by the density INSIDE the blocks (all blocks
    present; the tensor-core time does not depend on it, the sparse kernel's does), and by the fraction of
    blocks kept (blocks whole)."""
    import os
    from workloads import gen
    dev = "cuda:0"
    c, hw = 256, 56
    g = gen.rng(99)
    q = gen.int8_weights(g, (c, 3, 3, c))
    m = torch.full((c,), 2e-5, device=dev)
    b = torch.zeros(c, device=dev)

    def time_it(fn, reps=20):
        # the calls are captured into one CUDA graph, so that the host's launch cost stays out of the figure
        fn()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for _ in range(reps):
                fn()
        graph.replay()
        torch.cuda.synchronize()
        best = 1e9
        for _ in range(3):
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record()
            graph.replay()
            a1.record()
            torch.cuda.synchronize()
            best = min(best, a0.elapsed_time(a1) / reps * 1e3)
        return best

    def both(mask, batch, threshold):
        x = torch.from_numpy(gen.int8_image(g, (batch, hw, hw, c))).to(dev)
        y1 = torch.zeros((batch, hw, hw, c), dtype=torch.int8, device=dev)
        y2 = torch.zeros_like(y1)
        os.environ["CADNN_BLOCK_DENSITY"] = str(threshold)
        wg = B.cadnn_pack_q8(B.make_desc(c, c, 3, 3, 1, 1, 1, hw, hw, batch, "s8", fmt=B.FMT_GROUPED), q, mask)
        os.environ.pop("CADNN_BLOCK_DENSITY", None)
        ws = torch.empty(B.cadnn_weights_workspace_bytes(wg, batch), dtype=torch.uint8, device=dev)
        wsp = B.cadnn_pack_q8(B.make_desc(c, c, 3, 3, 1, 1, 1, hw, hw, batch, "s8"), q, mask)
        t_g = time_it(lambda: B.cadnn_conv2d_workspace(wg, x, y1, ws, m, b, None, "relu", out_dtype="s8"))
        t_s = time_it(lambda: B.cadnn_conv2d(wsp, x, y2, m, b, None, "relu", out_dtype="s8"))
        torch.cuda.synchronize()
        assert torch.equal(y1, y2), "the two routes disagree"
        return t_g, t_s, B.cadnn_weights_block_info(wg)["blocks"]

    print("# Block-structured int8 conv 256->256 3x3 56x56: tensor-core blocks + sparse remainder vs sparse kernel alone\n")
    print("## by density inside the blocks (every block present, all of them taken as dense blocks)\n")
    print("| batch | density in block | blocks | tensor-core route µs | sparse kernel µs | ratio sparse / tc |")
    print("|---|---|---|---|---|---|")
    for batch in batches:
        for rho in (0.05, 0.1, 0.2, 0.3, 0.5, 0.75, 1.0):
            mask = (g.random(q.shape) < rho).astype(np.uint8) if rho < 1.0 else np.ones(q.shape, np.uint8)
            t_g, t_s, nb = both(mask, batch, 0.0)
            print("| %d | %.2f | %d | %.1f | %.1f | %.2f |" % (batch, rho, nb, t_g, t_s, t_s / t_g))
            sys.stdout.flush()
    print("\n## by fraction of blocks kept (kept blocks whole, nothing else)\n")
    print("| batch | blocks kept | blocks | tensor-core route µs | sparse kernel µs | ratio sparse / tc |")
    print("|---|---|---|---|---|---|")
    for batch in batches:
        for bd in (0.05, 0.1, 0.25, 0.5, 1.0):
            mask = gen.block_mask(g, q.shape, bd)
            t_g, t_s, nb = both(mask, batch, 0.5)
            print("| %d | %.2f | %d | %.1f | %.1f | %.2f |" % (batch, bd, nb, t_g, t_s, t_s / t_g))
            sys.stdout.flush()


def persistent_profile(workload, batch):
    """Per-phase clock profile of the persistent whole-network kernel (CADNN_PERSIST=1): wall clocks of the
    phase, busiest and mean block, clocks until the first copy was issued and until its bytes had landed,
    and what the host planner chose for every layer of the phase."""
    import os
    os.environ["CADNN_PERSIST"] = "1"
    os.environ["CADNN_PERSIST_PROFILE"] = "1"
    dev = "cuda:0"
    m = build(workload, 0.125)
    x = models.make_input(m, batch)
    pm = PackedModel(m, batch, dev)
    xd = torch.from_numpy(x).to(dev)
    y = pm.new_output()
    for _ in range(10):
        pm.forward(xd, y)
    torch.cuda.synchronize()
    prof = B.cadnn_net_persistent_profile(pm.net)
    names = {}
    for i, op in enumerate(m.ops):
        pl = B.cadnn_net_persistent_plan(pm.net, i)
        if pl is not None:
            names.setdefault(pl["phase"], []).append((op.name, pl))
    print("# persistent kernel, %s batch %d: clocks per phase (last of 10 forwards)\n" % (workload, batch))
    print("| phase | wall | busiest block | mean block | first copy issued | first bytes landed | layers (tile bands T, filters per item G, tiles, groups, passes) |")
    print("|---|---|---|---|---|---|---|")
    tot = 0.0
    for ph, (w, bm, ba, ti, tl) in enumerate(prof):
        tot += w
        desc = "; ".join("%s T%d G%d t%d g%d p%d" % (n, p["T"], p["G"], p["tiles"], p["groups"], p["passes"]) for n, p in names.get(ph, []))
        print("| %d | %.0f | %.0f | %.0f | %.0f | %.0f | %s |" % (ph, w, bm, ba, ti, tl, desc))
    print("\ntotal %.0f clocks" % tot)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--block-crossover", action="store_true",
                    help="time the tensor-core block route against the sparse kernel on one block-structured int8 layer")
    ap.add_argument("--persistent-profile", action="store_true",
                    help="per-phase clock profile of the persistent kernel on the workload (first --batch value)")
    ap.add_argument("--workload", default="resnet50")
    ap.add_argument("--batch", type=int, nargs="+", default=[1])
    ap.add_argument("--density", type=float, nargs="+", default=[0.125])
    ap.add_argument("--layers", action="store_true", help="also print the per-layer table")
    ap.add_argument("--no-autotune", action="store_true")
    ap.add_argument("--torch-dense", action="store_true", help="add cuDNN dense timings (context)")
    args = ap.parse_args()
    if args.persistent_profile:
        persistent_profile(args.workload, args.batch[0])
        return
    if args.block_crossover:
        block_crossover(args.batch)
        return
    peaks = roofline.measured_peaks()
    r_alu = roofline.alu_peak_tflops(peaks["sm_max_mhz"])
    print("# %s: sparse-roofline report (ALU peak %.1f TFLOP/s, HBM %.0f GB/s nominal / %.0f measured)\n"
          % (args.workload, r_alu, roofline.HBM_NOMINAL_GBS, peaks["hbm_gbs"]))
    print("| batch | density | latency ms | images/s | roofline µs | fraction | k×k frac | 1×1 frac | nnz stored |")
    print("|---|---|---|---|---|---|---|---|---|")
    layer_tables = []
    for dens in args.density:
        model = build(args.workload, dens)
        for batch in args.batch:
            pm = PackedModel(model, batch, "cuda:0", autotune=not args.no_autotune)
            x = torch.from_numpy(models.make_input(model, batch)).cuda()
            y = pm.new_output()
            ms = time_forward(pm, x, y)
            rows = roofline.network_roofline(model, batch, r_alu, roofline.HBM_NOMINAL_GBS)
            per = np.zeros(len(model.ops))
            for _ in range(2):
                per += np.array(pm.layer_times(x, y, reps=10)) / 2
            t_roof = sum(r["t_roof_us"] for r in rows)
            fam = {}
            for r, t in zip(rows, per):
                f = fam.setdefault(r["family"], [0.0, 0.0])
                f[0] += r["t_roof_us"]
                f[1] += t * 1e3
            frac = lambda k: ("%.3f" % (fam[k][0] / fam[k][1])) if k in fam and fam[k][1] > 0 else "-"
            print("| %d | %.3g | %.4f | %.0f | %.1f | %.4f | %s | %s | %d |" % (
                batch, dens, ms, batch / ms * 1e3, t_roof, t_roof / (ms * 1e3), frac("sconv_kxk"), frac("sconv_1x1"),
                sum(o.nnz for o in model.weight_ops())))
            sys.stdout.flush()
            if args.layers:
                lines = ["\n## per layer: batch %d, density %.3g\n" % (batch, dens),
                         "| layer | kernel | in | c_in→c_out | k/s | nnz | µs | roofline µs | fraction | schedule |", "|---|---|---|---|---|---|---|---|---|---|"]
                planar = B.cadnn_net_layout(pm.net)["planar"]
                parity_ops = set(B.cadnn_net_parity_layers(pm.net, ops=True))
                for i, (op, r, t) in enumerate(zip(model.ops, rows, per)):
                    s = B.cadnn_weights_schedule(pm.weights[i]) if i in pm.weights else None
                    ss = ("T%d rpw%d nw%d cic%d ks%d" % (s["T"], s["RPW"], s["NW"], s["CIc"], s["ksplit"])) if s and s["kind"] in (1, 2) else ""
                    wh = pm.weights.get(i) if op.kind == "conv" else None
                    if wh is not None and i in parity_ops:   # the stride-1 form over the input's parity planes runs
                        wh = B.cadnn_weights_parity_form(wh)
                    ps = B.cadnn_weights_planar_schedule(wh) if (planar and wh is not None) else None
                    if ps and ps["variant"] == 1:
                        ss = "planar direct T%d nw%d ksw%d rpw%d d%d" % (ps["T"], ps["NW"], ps["KS"], ps["RPW"], ps["stages"])
                    elif ps and ps["variant"] == 2:
                        ss = "planar %s T%d nw%d ks%d rpw%d cic%d st%d kc%d" % ("tma" if ps["tma"] else "cp.async", ps["T"], ps["NW"], ps["KS"],
                                                                               ps["RPW"], ps["CIc"], ps["stages"], ps["KC"])
                    if i in parity_ops:
                        ss = "parity planes, " + ss
                    lines.append("| %s | %s | %dx%d | %d→%d | %d/%d | %d | %.1f | %.2f | %.3f | %s |" % (
                        op.name, r["family"], op.in_hw[0], op.in_hw[1], op.c_in, op.c_out, op.k, op.stride, r["nnz"],
                        t * 1e3, r["t_roof_us"], r["t_roof_us"] / (t * 1e3), ss))
                layer_tables.append("\n".join(lines))
            del pm
            torch.cuda.empty_cache()
    for t in layer_tables:
        print(t)
    if args.torch_dense:
        print("\n## dense context: torch / cuDNN on the same layer shapes (library calls, channels-last)\n")
        print("| batch | fp32 (TF32 off) ms | TF32 on ms |")
        print("|---|---|---|")
        model = build(args.workload, 1.0) if args.workload != "vgg16" else None
        for batch in args.batch:
            if model is None:
                break
            a = torch_dense_ms(model, batch, False)
            b = torch_dense_ms(model, batch, True)
            print("| %d | %.4f | %.4f |" % (batch, a, b))


if __name__ == "__main__":
    main()
