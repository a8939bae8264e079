"""Bandwidth sweep of the fused entry point over one synthetic activation set.

    python -m paper_2503_18339_b200.sweep --config 5            # ResNet-50 shapes, fp32 + bf16, b = 2..8

Per tensor, element type, bit-width and mode (forward only / forward + backward) it prints the
CUDA-event time of one call (median of `--iters`, after warm-up, an L2-sized scratch write between
calls), the algorithmic GB/s (fp32: 8 / 16 B per element, bf16: 4 / 8) and its fraction of the
measured copy bandwidth.  Inputs come from `workloads.py`; bf16 inputs are the round-to-nearest-even
of the fp32 sample.

    python -m paper_2503_18339_b200.sweep --config 2 --distortion --bits 3,4

prints instead the statistics of the paper's Table 2 (cosine similarity and relative error of the
fake-quantized activations) for layer-wise against channel-wise quantization of the same tensors.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics

import torch

from . import binding as b
from . import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _peak() -> float:
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
            return float(json.load(fh)["hbm_gbs"])
    except Exception:
        return 6650.0


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=5)
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--bits", default="", help="comma list; default: the config's own")
    ap.add_argument("--dtypes", default="", help="comma list of f32,bf16; default: the config's own")
    ap.add_argument("--modes", default="fwd,fwd+bwd")
    ap.add_argument("--only", default="", help="keep tensors whose name contains this")
    ap.add_argument("--tune", default="", help="planner knobs, e.g. l2_wave_kb=32768,l2_upl=2")
    ap.add_argument("--distortion", action="store_true",
                    help="instead of the bandwidth sweep: the statistics of Table 2 (cosine similarity, relative "
                         "error) of layer-wise against channel-wise quantization on the config's tensors")
    ap.add_argument("--table5", action="store_true",
                    help="instead of the bandwidth sweep: the three rows of the paper's Table 5 in kind - forward "
                         "fake-quantization of all 19 ResNet-20 activation tensors at batch 16, 3 bits: layer-wise, "
                         "channel-wise by the per-channel loop, channel-wise by the default plan")
    ap.add_argument("--packed", action="store_true",
                    help="instead of the bandwidth sweep: quantize to packed b-bit codes and dequantize from them")
    ap.add_argument("--weights", default="", choices=["", "resnet20", "resnet18"],
                    help="instead of the bandwidth sweep: all weight tensors of the network in one batched "
                         "launch against one fused call per tensor")
    args = ap.parse_args()
    b.lib()
    if args.weights:
        weights_table(args)
        return
    if args.packed:
        packed_table(args)
        return
    if args.table5:
        table5(args)
        return
    if args.distortion:
        distortion_table(args)
        return
    knobs = {"l2_wave_kb": b.KNOB_L2_WAVE_KB, "l2_upl": b.KNOB_L2_UPL, "l2_ctas_per_sm": b.KNOB_L2_CTAS_PER_SM}
    for item in filter(None, args.tune.split(",")):
        name, val = item.split("=")
        b.tune(knobs[name], int(val))
    peak = _peak()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    seen = set()
    print("tensor dtype bits mode us GB/s frac_of_measured")
    for spec in wl.config_tensors(args.config):
        if spec.shape in seen or args.only not in spec.name:
            continue
        seen.add(spec.shape)
        x32 = torch.from_numpy(wl.make_activation(spec)).cuda()
        g32 = torch.from_numpy(wl.make_upstream_grad(spec)).cuda()
        for dt in (args.dtypes.split(",") if args.dtypes else spec.dtypes):
            x = x32 if dt == "f32" else x32.to(torch.bfloat16)
            gy = g32 if dt == "f32" else g32.to(torch.bfloat16)
            out = b.FakeQuantOut(y=torch.empty_like(x), gx=torch.empty_like(x))
            esize = x.element_size()
            for bits in ([int(v) for v in args.bits.split(",")] if args.bits else spec.bits):
                for mode in args.modes.split(","):
                    g = gy if mode == "fwd+bwd" else None
                    for _ in range(2):
                        b.granq_fakequant_fused(x, bits, gy=g, out=out)
                    times = []
                    for _ in range(args.iters):
                        flush.fill_(1)
                        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        e0.record()
                        b.granq_fakequant_fused(x, bits, gy=g, out=out)
                        e1.record()
                        torch.cuda.synchronize()
                        times.append(e0.elapsed_time(e1) * 1e3)
                    assert b.workspace_status(out.workspace) == b.OK
                    us = statistics.median(times)
                    nbytes = x.numel() * esize * (4 if g is not None else 2)
                    gbs = nbytes / us / 1e3
                    print(f"{spec.name} {dt} {bits} {mode} {us:.1f} {gbs:.0f} {gbs / peak:.3f}", flush=True)
            del x, gy, out
        del x32, g32


def table5(args) -> None:
    """Quantization latency of one forward pass over the ResNet-20 activation set at batch 16 (the setting of
    Table 5): wall time of the 19 calls including their launches, median of `--iters` repetitions."""
    import dataclasses
    import time
    specs = [dataclasses.replace(s, shape=(16,) + tuple(s.shape[1:])) for s in wl.config_tensors(2)]
    xs = [torch.from_numpy(wl.make_activation(s)).cuda() for s in specs]
    rows = (("layer-wise (one range per tensor)", b.GROUP_TENSOR, 0),
            ("channel-wise, per-channel loop (3 launches per channel)", b.GROUP_CHANNEL, b.FLAG_FORCE_NAIVE),
            ("channel-wise, default plan (1 launch per tensor)", b.GROUP_CHANNEL, 0))
    print("scheme ms_per_pass launches")
    for name, group, flags in rows:
        outs = [b.FakeQuantOut(y=torch.empty_like(x), workspace=b.make_workspace(x, 1, group)) for x in xs]
        launches = sum(b.fused_plan(b.F32, x.shape, group=group, with_backward=False, flags=flags)[1] for x in xs)

        def one_pass():
            for x, o in zip(xs, outs):
                b.granq_fakequant_fused(x, 3, group=group, out=o, flags=flags)
        one_pass()
        torch.cuda.synchronize()
        times = []
        for _ in range(max(args.iters, 5)):
            t0 = time.perf_counter()
            one_pass()
            torch.cuda.synchronize()
            times.append((time.perf_counter() - t0) * 1e3)
        print(f"{name}: {statistics.median(times):.3f} {launches}", flush=True)


def packed_table(args) -> None:
    """Packed b-bit codes: time and algorithmic GB/s (fp32: 4 + b/8 bytes per element each way) of
    granq_quantize_packed (range given) and granq_dequantize_packed on the config's tensors."""
    peak = _peak()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    print("tensor bits op us GB/s frac_of_measured")
    seen = set()
    for spec in wl.config_tensors(args.config):
        if spec.shape in seen or args.only not in spec.name:
            continue
        seen.add(spec.shape)
        x = torch.from_numpy(wl.make_activation(spec)).cuda()
        lo, hi = b.granq_range(x)
        y = torch.empty_like(x)
        for bits in ([int(v) for v in args.bits.split(",")] if args.bits else spec.bits):
            pc = torch.empty(b.packed_codes_bytes(x.shape, bits) // 4, dtype=torch.int32, device="cuda")
            out = b.granq_quantize_packed(x, bits, lo, hi, packed_codes=pc)
            ops = (("quantize_packed", lambda: b.granq_quantize_packed(x, bits, lo, hi, packed_codes=pc)),
                   ("dequantize_packed", lambda: b.granq_dequantize_packed(pc, x.shape, x.dtype, bits, out.s, out.z, y=y)))
            for name, fn in ops:
                fn()
                times = []
                for _ in range(args.iters):
                    flush.fill_(1)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    fn()
                    e1.record()
                    torch.cuda.synchronize()
                    times.append(e0.elapsed_time(e1) * 1e3)
                us = statistics.median(times)
                gbs = x.numel() * (4 + bits / 8) / us / 1e3
                print(f"{spec.name} {bits} {name} {us:.1f} {gbs:.0f} {gbs / peak:.3f}", flush=True)
        del x, y


def weights_table(args) -> None:
    """Channel-wise fake-quantization (forward + STE backward) of every weight tensor of a network:
    one batched launch against a loop of fused calls with channel_axis = 0."""
    ws = [torch.from_numpy(w).cuda() for w in wl.make_weights(args.weights)]
    gs = [torch.from_numpy(g).cuda() for g in wl.make_weights(args.weights, grads=True)]
    elems = sum(w.numel() for w in ws)
    ws4 = [w.reshape(w.shape[0], -1, 1, 1) for w in ws]
    gs4 = [g.reshape(g.shape[0], -1, 1, 1) for g in gs]
    outs = [b.FakeQuantOut(y=torch.empty_like(w), gx=torch.empty_like(w), workspace=b.make_workspace(w, 0)) for w in ws4]
    batch = b.WeightBatch(ws, 4, grads=gs)

    def batched():
        batch.run()

    def looped():
        for w, g, o in zip(ws4, gs4, outs):
            b.granq_fakequant_fused(w, 4, gy=g, channel_axis=0, out=o)

    print("network tensors elements variant us GB/s(16 B/element)")
    for name, fn in (("batched", batched), ("one call per tensor", looped)):
        for _ in range(3):
            fn()
        times = []
        for _ in range(max(args.iters, 5)):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1) * 1e3)
        us = statistics.median(times)
        print(f"{args.weights} {len(ws)} {elems} {name} {us:.1f} {elems * 16 / us / 1e3:.0f}", flush=True)


def distortion_table(args) -> None:
    """Table 2 in kind: per tensor and averaged, layer-wise (one range per tensor) against channel-wise
    (one range per channel) at the given bit-widths, with the time of the pass that gathers the sums."""
    bits_list = [int(v) for v in args.bits.split(",")] if args.bits else [3]
    print("tensor bits grouping cosine rel_error us")
    seen = set()
    avg = {}
    for spec in wl.config_tensors(args.config):
        if spec.shape in seen or args.only not in spec.name:
            continue
        seen.add(spec.shape)
        x = torch.from_numpy(wl.make_activation(spec)).cuda()
        for bits in bits_list:
            for name, group in (("layer-wise", b.GROUP_TENSOR), ("channel-wise", b.GROUP_CHANNEL)):
                out = b.FakeQuantOut(y=torch.empty_like(x))
                b.granq_fakequant_fused_stats(x, bits, group=group, out=out)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                b.granq_fakequant_fused_stats(x, bits, group=group, out=out)
                e1.record()
                torch.cuda.synchronize()
                assert b.workspace_status(out.workspace) == b.OK
                cos, rel = b.distortion_from_sums(out.sums.cpu().tolist())
                avg.setdefault((bits, name), []).append((cos, rel))
                print(f"{spec.name} {bits} {name} {cos:.4f} {rel:.4f} {e0.elapsed_time(e1) * 1e3:.1f}", flush=True)
        del x
    for (bits, name), rows in avg.items():
        print(f"average {bits} {name} {sum(r[0] for r in rows) / len(rows):.4f} "
              f"{sum(r[1] for r in rows) / len(rows):.4f} -")


if __name__ == "__main__":
    main()
