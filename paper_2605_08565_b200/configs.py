"""The five benchmark configurations of this library, timed one recipe at a time.

    python -m paper_2605_08565_b200.configs [--configs 1,2,3,4,5] [--out results.json] [--hash-inputs]

For every (configuration, block size, scale format, recipe) the quantize pass is timed with CUDA
events over the whole synthetic workload (launches back to back; tensors larger than L2 or rotated
so that inputs come from HBM), the tensor MSE is computed with ``mxq_tensor_mse`` after each pass
(outside the quantize timing), and the result is reported as GElem/s together with the fraction of
the bounding roofline: HBM copy bandwidth for abs-max / prevent-zero / 4-over-6 (algorithmic bytes
``b_in + 0.5 + 5/B`` per element), the 128-lanes-per-SM issue peak at the maximum SM clock for brute
force (4 lane-ops per element and scale code).  Inputs are seeded stand-ins for the LLM tensors the
paper measures on (shapes and rough value distributions only).  Every step runs in the CUDA
kernels; there is no CPU fallback.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os

import torch

from . import binding as mxq
from . import inputs

RECIPE_NAMES = {mxq.MXQ_ABSMAX: "absmax", mxq.MXQ_ABSMAX_PZ: "absmax_pz", mxq.MXQ_4O6: "4o6", mxq.MXQ_4O6_PZ: "4o6_pz",
                mxq.MXQ_BRUTE: "brute", mxq.MXQ_BRUTE_PZ: "brute_pz"}
FMT_NAMES = {mxq.MXQ_SF_UE8M0: "ue8m0", mxq.MXQ_SF_UE4M3: "ue4m3", mxq.MXQ_SF_UE5M3: "ue5m3"}
N_CODES = {mxq.MXQ_SF_UE8M0: 255, mxq.MXQ_SF_UE4M3: 127, mxq.MXQ_SF_UE5M3: 255}


def _peaks():
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    path = os.path.join(root, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), float(p.get("sm_max_mhz", 1965.0)), "measured"
    return 6650.0, 1965.0, "fallback"


class _Acc:
    """CUDA-event time and elements per (B, fmt, recipe, tensor-scale) key.  A key's tensors are
    quantized back to back inside one event pair (after one untimed launch that takes the kernel's
    first-use costs), `rounds` times over; the tensor MSE is taken afterwards, untimed."""

    def __init__(self):
        self.ms, self.elems, self.mse = {}, {}, {}

    def run(self, key, xs, B, fmt, recipe, g, dgs, bufs, rounds=1):
        self._run(key, xs, B, fmt, recipe, g, dgs, bufs, rounds)
        if recipe in (mxq.MXQ_BRUTE, mxq.MXQ_BRUTE_PZ):   # the same pass with the pruned sweep, as a row of its own
            mxq.mxq_set_option(mxq.MXQ_OPT_BRUTE_PRUNE, 1)
            try:
                self._run(key + ("pruned",), xs, B, fmt, recipe, g, dgs, bufs, rounds)
            finally:
                mxq.mxq_set_option(mxq.MXQ_OPT_BRUTE_PRUNE, 0)

    def _run(self, key, xs, B, fmt, recipe, g, dgs, bufs, rounds):
        codes, scales, sse, mse_out, ws = bufs
        dgs = dgs if dgs is not None else [None] * len(xs)
        mxq.mxq_quantize_ex(xs[0], xs[0].numel(), B, fmt, recipe, g, dgs[0], codes, scales, sse)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(rounds):
            for x, dg in zip(xs, dgs):
                mxq.mxq_quantize_ex(x, x.numel(), B, fmt, recipe, g, dg, codes, scales, sse)
        e1.record()
        tot, cnt = 0.0, 0
        for x, dg in zip(xs, dgs):
            mxq.mxq_quantize_ex(x, x.numel(), B, fmt, recipe, g, dg, codes, scales, sse)
            mxq.mxq_tensor_mse(sse, x.numel() // B, x.numel(), mse_out, ws)
            tot += float(mse_out.cpu()[0]) * x.numel()
            cnt += x.numel()
        torch.cuda.synchronize()
        self.ms[key] = self.ms.get(key, 0.0) + e0.elapsed_time(e1)
        self.elems[key] = self.elems.get(key, 0) + cnt * rounds
        m = self.mse.setdefault(key, [0.0, 0])
        m[0] += tot
        m[1] += cnt

    def rows(self, cfg, elem_bytes, hbm_gbs, alu_peak):
        out = []
        for key, ms in self.ms.items():
            B, fmt, recipe, gk = key[:4]
            pruned = len(key) > 4
            n = self.elems[key]
            ge = n / ms / 1e6
            row = {"config": cfg, "block": B, "scale_fmt": FMT_NAMES[fmt],
                   "recipe": RECIPE_NAMES[recipe] + ("+prune" if pruned else ""), "tensor_scale": gk,
                   "elements": n, "ms": ms, "gelem_s": ge, "mse": self.mse[key][0] / self.mse[key][1]}
            if pruned:
                # codes left out are not work done: no roofline fraction, only the speed-up over the full sweep
                full = self.elems[key[:4]] / self.ms[key[:4]] / 1e6
                row.update(bound="alu", speedup_over_full_sweep=ge / full, frac=None)
            elif recipe in (mxq.MXQ_BRUTE, mxq.MXQ_BRUTE_PZ):
                ach = ge * 1e9 * N_CODES[fmt] * 4 / 1e12
                row.update(bound="alu", achieved_tlaneop_s=ach, frac=ach / alu_peak)
            else:
                ach = ge * (elem_bytes + 0.5 + 5.0 / B)
                row.update(bound="hbm", achieved_gb_s=ach, frac=ach / hbm_gbs, frac_of_8tbs=ach / 8000.0)
            out.append(row)
        return out


class _InputDigest:
    """SHA-256 over the bytes of a configuration's input tensors, in generation order (so that a run
    can be tied to the exact inputs it quantized); computed on the host, only when asked for."""

    def __init__(self, enabled):
        self.h = hashlib.sha256() if enabled else None
        self.tensors, self.elements = 0, 0

    def add(self, x):
        self.tensors += 1
        self.elements += x.numel()
        if self.h is not None:
            self.h.update(x.view(torch.uint8).cpu().numpy().tobytes())

    def result(self):
        return {"tensors": self.tensors, "elements": self.elements,
                "sha256": self.h.hexdigest() if self.h is not None else None}


def _bufs(n, B, dev):
    codes, scales, sse = mxq.alloc_outputs(n, B, dev)
    return (codes, scales, sse, torch.empty(1, dtype=torch.float64, device=dev),
            torch.empty(mxq.mxq_tensor_mse_workspace_bytes(n // B) // 8, dtype=torch.float64, device=dev))


def _tensor_scale(x):
    amax = torch.empty(1, dtype=torch.float32, device=x.device)
    dg = torch.empty(1, dtype=torch.float32, device=x.device)
    mxq.mxq_tensor_amax(x, x.numel(), amax, dg)
    return dg


def run(configs=(1, 2, 3, 4, 5), device="cuda", hash_inputs=False):
    if not torch.cuda.is_available():
        raise mxq.MxqError("needs a CUDA device (no CPU fallback)")
    dev = torch.device(device)
    hbm, mhz, src = _peaks()
    n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
    alu_peak = n_sm * 128 * mhz * 1e6 / 1e12
    A, P, R4, BR = mxq.MXQ_ABSMAX, mxq.MXQ_ABSMAX_PZ, mxq.MXQ_4O6, mxq.MXQ_BRUTE
    U4, U5, U8 = mxq.MXQ_SF_UE4M3, mxq.MXQ_SF_UE5M3, mxq.MXQ_SF_UE8M0
    rows = []
    digests = {}
    warm = inputs.normal(1 << 20, 0, 1.0, torch.float32, dev)          # first-launch costs out of the way
    for r in (A, R4, BR):
        mxq.quantize(warm, 16, U4, r)

    if 1 in configs:   # 1024 x 1024 fp32 N(0,1), B=16, UE4M3 + tensor scale; 4 MB: L2-resident, launch-bound
        x = inputs.normal(1024 * 1024, 1, 1.0, torch.float32, dev)
        digests["C1"] = _InputDigest(hash_inputs)
        digests["C1"].add(x)
        dg = _tensor_scale(x)
        acc, bufs = _Acc(), _bufs(x.numel(), 16, dev)
        for r in (A, R4, BR):
            acc.run((16, U4, r, "amax/2688"), [x], 16, U4, r, 1.0, [dg], bufs, rounds=50)
        rows += acc.rows("C1 1024x1024 fp32 N(0,1)", 4, hbm, alu_peak)

    if 2 in configs:   # 4096 x 4096 bf16 0.02 * t5, all block sizes, UE4M3, no tensor scale; 8 rotating tensors
        xs = [inputs.student_t(4096 * 4096, 5, 0.02, 2 * 1_000_003 + i, torch.bfloat16, dev) for i in range(8)]
        digests["C2"] = _InputDigest(hash_inputs)
        for x in xs:
            digests["C2"].add(x)
        acc = _Acc()
        for B in (2, 4, 8, 16, 32, 64):
            bufs = _bufs(xs[0].numel(), B, dev)
            for r in (A, P, R4, BR):
                acc.run((B, U4, r, "none"), xs, B, U4, r, 1.0, None, bufs, rounds=4 if r != BR else 1)
        rows += acc.rows("C2 4096x4096 bf16 0.02*t5", 2, hbm, alu_peak)
        del xs

    if 3 in configs:   # 8192 x 4096 bf16 N(0,1) with 1 % outlier columns x50, B=16; 4 rotating tensors
        xs = [inputs.outlier_columns(8192, 4096, 3 + i, dtype=torch.bfloat16, device=dev) for i in range(4)]
        digests["C3"] = _InputDigest(hash_inputs)
        for x in xs:
            digests["C3"].add(x)
        dgs = [_tensor_scale(x) for x in xs]
        acc, bufs = _Acc(), _bufs(xs[0].numel(), 16, dev)
        for r in (A, R4):
            acc.run((16, U4, r, "amax/2688"), xs, 16, U4, r, 1.0, dgs, bufs, rounds=4)
            acc.run((16, U5, r, "none"), xs, 16, U5, r, 1.0, None, bufs, rounds=4)
        rows += acc.rows("C3 8192x4096 bf16 outlier columns", 2, hbm, alu_peak)
        del xs

    if 4 in configs:   # Llama-3-8B-shaped weight set, 224 matrices, one at a time
        acc = _Acc()
        digests["C4"] = _InputDigest(hash_inputs)
        for layer in range(inputs.LLAMA8B_LAYERS):
            for idx, (name, rows_, cols) in enumerate(inputs.LLAMA8B_LAYER_SHAPES):
                x = inputs.student_t(rows_ * cols, 4, 1.0 / math.sqrt(cols), 4 + layer * 7 + idx, torch.bfloat16, dev)
                digests["C4"].add(x)
                for B in (8, 16):
                    bufs = _bufs(x.numel(), B, dev)
                    for fmt in (U4, U5):
                        for r in RECIPE_NAMES:
                            acc.run((B, fmt, r, "none"), [x], B, fmt, r, 1.0, None, bufs)
                del x
        rows += acc.rows("C4 Llama-3-8B-shaped set (224 matrices, 6.98 G elements)", 2, hbm, alu_peak)

    if 5 in configs:   # 16384 x 16384 fp32 Laplace, brute force, tensor scale
        x = inputs.laplace(16384 * 16384, 5, torch.float32, dev)
        digests["C5"] = _InputDigest(hash_inputs)
        digests["C5"].add(x)
        dg = _tensor_scale(x)
        acc = _Acc()
        for B in (2, 4, 8, 16, 32):
            bufs = _bufs(x.numel(), B, dev)
            for fmt in (U8, U4, U5):
                acc.run((B, fmt, BR, "amax/2688"), [x], B, fmt, BR, 1.0, [dg], bufs)
        rows += acc.rows("C5 16384x16384 fp32 Laplace", 4, hbm, alu_peak)
    return {"hbm_gbs": hbm, "alu_peak_tlaneop_s": alu_peak, "peak_source": src, "rows": rows,
            "inputs": {k: d.result() for k, d in digests.items()}}


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--configs", default="1,2,3,4,5")
    ap.add_argument("--out", default=None)
    ap.add_argument("--hash-inputs", action="store_true",
                    help="record the SHA-256 of every configuration's input bytes (copies each tensor to the host once)")
    args = ap.parse_args()
    res = run(tuple(int(c) for c in args.configs.split(",")), hash_inputs=args.hash_inputs)
    for r in res["rows"]:
        head = (f'{r["config"][:28]:28s} B={r["block"]:<2d} {r["scale_fmt"]:5s} {r["recipe"]:14s} g={r["tensor_scale"]:9s} '
                f'{r["gelem_s"]:9.1f} GElem/s  ')
        if r["frac"] is None:
            print(head + f'{r["speedup_over_full_sweep"]:8.2f} x the full sweep{"":14s}  mse={r["mse"]:.4e}')
            continue
        ach = r.get("achieved_gb_s", r.get("achieved_tlaneop_s"))
        unit = "GB/s" if r["bound"] == "hbm" else "Tlop/s"
        print(head + f'{ach:8.1f} {unit:6s} {100 * r["frac"]:5.1f}% of {r["bound"]}  mse={r["mse"]:.4e}')
    for cfg, d in res["inputs"].items():
        print(f'{cfg}: {d["tensors"]} tensors, {d["elements"]} elements' + (f', sha256 {d["sha256"]}' if d["sha256"] else ""))
    if args.out:
        with open(args.out, "w") as f:
            json.dump(res, f, indent=1)


if __name__ == "__main__":
    main()
