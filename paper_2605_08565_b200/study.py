"""Numerical study of the paper (Results, "Numerical Study"; Appendix, clipping-only MSE and
histograms) on the GPU library: MSE against the standard deviation of N(0, sigma^2) samples for
block sizes {4, 8, 16, 32} and the recipes abs-max, prevent-zero, 4-over-6, prevent-zero + 4-over-6
and brute force, with UE4M3 block scales and FP4 (E2M1) entries.

All 151 sigmas of one block size are one tensor (segments of 50,000 blocks): one quantize launch
per recipe, one ``mxq_segment_mse`` launch for the 151 MSE values, one ``mxq_block_clip_sse`` +
``mxq_segment_mse`` for the clipping-only part, one ``mxq_histograms`` per region of interest.

    python -m paper_2605_08565_b200.study [--out study.json] [--blocks-per-sigma 50000]

Every arithmetic step runs in the CUDA kernels; this module only draws inputs, calls the C-ABI
binding and collects the curves.  There is no CPU fallback.
"""
from __future__ import annotations

import argparse
import json
import time

import torch

from . import binding as mxq
from . import inputs

RECIPES = {"absmax": mxq.MXQ_ABSMAX, "absmax_pz": mxq.MXQ_ABSMAX_PZ, "4o6": mxq.MXQ_4O6, "4o6_pz": mxq.MXQ_4O6_PZ,
           "brute": mxq.MXQ_BRUTE}
BLOCK_SIZES = (4, 8, 16, 32)


def run(block_sizes=BLOCK_SIZES, n_sigma: int = 151, sigma_lo: float = 0.0005, sigma_hi: float = 0.05,
        blocks_per_sigma: int = 50_000, scale_fmt: int = mxq.MXQ_SF_UE4M3, seed: int = 0, device="cuda",
        recipes=RECIPES, histogram_sigmas=(), keep_block_sse: bool = False):
    """Returns {"sigma": [...], "mse": {recipe: {B: [...]}}, "clip_mse": {...}, "hist": {...}, "seconds": ...}.

    histogram_sigmas: indices into the sigma grid for which the 16-bin entry histogram and the
    256-bin scale histogram are collected per recipe and block size.
    keep_block_sse: also return the per-block SSE tensors (device, one row of blocks_per_sigma values
    per sigma) under "block_sse", for callers that want more than the mean (e.g. its sampling error).
    """
    if not torch.cuda.is_available():
        raise mxq.MxqError("the numerical study needs a CUDA device (no CPU fallback)")
    dev = torch.device(device)
    sig = inputs.sigma_grid(n_sigma, sigma_lo, sigma_hi)
    res = {"sigma": [float(s) for s in sig], "blocks_per_sigma": blocks_per_sigma, "scale_fmt": scale_fmt,
           "mse": {r: {} for r in recipes}, "clip_mse": {r: {} for r in recipes}, "hist": {}, "elements": 0}
    if keep_block_sse:
        res["block_sse"] = {r: {} for r in recipes}
    torch.cuda.synchronize(dev)
    t0 = time.perf_counter()
    gpu_s = 0.0
    for B in block_sizes:
        per_sigma = blocks_per_sigma * B
        x = inputs.sigma_sweep(per_sigma, seed * 1000 + B, n_sigma, sigma_lo, sigma_hi, torch.float32, dev)
        n = x.numel()
        nb = n // B
        codes, scales, sse = mxq.alloc_outputs(n, B, dev)
        clip = torch.empty(nb, dtype=torch.float32, device=dev)
        mse = torch.empty(n_sigma, dtype=torch.float64, device=dev)
        cmse = torch.empty(n_sigma, dtype=torch.float64, device=dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for name, rid in recipes.items():
            mxq.mxq_quantize_ex(x, n, B, scale_fmt, rid, 1.0, None, codes, scales, sse)
            mxq.mxq_segment_mse(sse, nb, blocks_per_sigma, per_sigma, mse)
            mxq.mxq_block_clip_sse(x, n, B, scale_fmt, 1.0, None, scales, clip)
            mxq.mxq_segment_mse(clip, nb, blocks_per_sigma, per_sigma, cmse)
            res["mse"][name][B] = mse.cpu().tolist()
            if keep_block_sse:
                res["block_sse"][name][B] = sse.view(n_sigma, blocks_per_sigma).clone()
            res["clip_mse"][name][B] = cmse.cpu().tolist()
            for k in histogram_sigmas:
                ch = torch.zeros(16, dtype=torch.int64, device=dev)
                sh = torch.zeros(256, dtype=torch.int64, device=dev)
                lo_b = k * blocks_per_sigma
                mxq.mxq_histograms(codes[lo_b * B // 2:(lo_b + blocks_per_sigma) * B // 2],
                                   scales[lo_b:lo_b + blocks_per_sigma], per_sigma, B, ch, sh)
                res["hist"][f"{name}/B{B}/sigma{k}"] = {"codes": ch.cpu().tolist(), "scales": sh.cpu().tolist()}
            res["elements"] += n
        e1.record()
        torch.cuda.synchronize(dev)
        gpu_s += e0.elapsed_time(e1) / 1e3
        del x, codes, scales, sse, clip
    res["seconds_wall"] = time.perf_counter() - t0
    res["seconds_gpu_quantize_and_score"] = gpu_s
    return res


def findings(res) -> dict:
    """The qualitative statements of the numerical study, evaluated on the curves."""
    sig = res["sigma"]
    bs = sorted(int(b) for b in next(iter(res["mse"].values())).keys())
    get = lambda r, b: res["mse"][r][b] if b in res["mse"][r] else res["mse"][r][str(b)]
    small, large = bs[0], bs[-1]
    out = {}
    # Region A: the zero-scale spike of abs-max and its removal by prevent-zero
    ratio = [get("absmax", small)[k] / max(get("absmax_pz", small)[k], 1e-300) for k in range(len(sig))]
    out["region_a_peak_ratio_absmax_over_pz"] = max(ratio)
    out["region_a_sigma_of_peak"] = sig[ratio.index(max(ratio))]
    out["pz_never_worse"] = all(get("absmax_pz", b)[k] <= get("absmax", b)[k] for b in bs for k in range(len(sig)))
    # Region B: smaller blocks worse than larger ones (inversion)
    for r in ("absmax_pz", "4o6_pz", "brute"):
        # different block sizes see different samples: 1 % covers the sampling noise of 50,000 blocks
        inv = [k for k in range(len(sig)) if get(r, small)[k] > 1.01 * get(r, large)[k]]
        out[f"inversion_points_{r}"] = len(inv)
        out[f"inversion_sigma_range_{r}"] = [sig[inv[0]], sig[inv[-1]]] if inv else None
    out["brute_monotone_in_block_size"] = all(
        get("brute", a)[k] <= get("brute", b)[k] * 1.01 for a, b in zip(bs[:-1], bs[1:]) for k in range(len(sig)))
    return out


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default=None)
    ap.add_argument("--blocks-per-sigma", type=int, default=50_000)
    ap.add_argument("--n-sigma", type=int, default=151)
    ap.add_argument("--seed", type=int, default=0)
    args = ap.parse_args()
    res = run(n_sigma=args.n_sigma, blocks_per_sigma=args.blocks_per_sigma, seed=args.seed)
    res["findings"] = findings(res)
    summary = {k: res[k] for k in ("elements", "seconds_wall", "seconds_gpu_quantize_and_score", "findings")}
    summary["gelem_s_quantize_and_score"] = res["elements"] / res["seconds_gpu_quantize_and_score"] / 1e9
    print(json.dumps(summary))
    if args.out:
        with open(args.out, "w") as f:
            json.dump(res, f)


if __name__ == "__main__":
    main()
