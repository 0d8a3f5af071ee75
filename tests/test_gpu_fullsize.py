"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration the
benchmark times (whole tensors, persistent grids).  Where the CPU oracle gets through a whole
tensor in seconds (every recipe on the 16.8 M element benchmark tensor, the one-pass recipes on
the 33.5 M element activation tensor and on the weight-shaped matrices) every output byte is
compared; elsewhere (brute force on the larger tensors) it computes sampled blocks one by one (blocks are independent given the tensor scale) and the rest is covered by
properties that hold at any size."""
import os

import numpy as np
import pytest
import torch

from oracle import mxq_oracle as orc
from paper_2605_08565_b200 import binding as mxq
from paper_2605_08565_b200 import dist, inputs

pytestmark = pytest.mark.gpu

ABSMAX, ABSMAX_PZ, R4O6, BRUTE = mxq.MXQ_ABSMAX, mxq.MXQ_ABSMAX_PZ, mxq.MXQ_4O6, mxq.MXQ_BRUTE


def _sample_blocks(n_blocks, k, seed):
    rng = np.random.default_rng(seed)
    edge = np.concatenate([np.arange(min(96, n_blocks)), np.arange(max(0, n_blocks - 96), n_blocks)])
    pick = rng.integers(0, n_blocks, size=k)
    return np.unique(np.concatenate([edge, pick]))


def _check_sampled(x, B, fmt, recipe, g, codes, scales, sse, k, seed):
    """Oracle on the sampled blocks (gathered into one short tensor) against the GPU outputs."""
    n_blocks = x.numel() // B
    idx = _sample_blocks(n_blocks, k, seed)
    t_idx = torch.from_numpy(idx).cuda()
    xs = x.view(n_blocks, B)[t_idx].contiguous().view(-1)
    oc, os_, oe = orc.quantize(inputs.to_numpy_bits(xs), B, fmt, recipe, g, threads=8)
    gc = codes.view(n_blocks, B // 2)[t_idx].cpu().numpy().reshape(-1)
    gs = scales[t_idx].cpu().numpy()
    ge = sse[t_idx].cpu().numpy()
    bad = np.flatnonzero(gs != os_)
    assert bad.size == 0, f"scale bytes differ at sampled blocks {idx[bad[:8]]}: gpu={gs[bad[:8]]} oracle={os_[bad[:8]]}"
    bad = np.flatnonzero(gc != oc)
    assert bad.size == 0, f"code bytes differ in sampled blocks {idx[bad[:8] // (B // 2)]}"
    bad = np.flatnonzero(ge.view(np.uint32) != oe.view(np.uint32))
    assert bad.size == 0, f"block SSE differs at sampled blocks {idx[bad[:8]]}"


def _check_full(x, B, fmt, recipe, g, codes, scales, sse):
    """Oracle on the whole tensor against the GPU outputs, every byte."""
    oc, os_, oe = orc.quantize(inputs.to_numpy_bits(x), B, fmt, recipe, g, threads=os.cpu_count() or 8)
    gs = scales.cpu().numpy()
    bad = np.flatnonzero(gs != os_)
    assert bad.size == 0, f"scale bytes differ at blocks {bad[:8]}: gpu={gs[bad[:8]]} oracle={os_[bad[:8]]}"
    bad = np.flatnonzero(codes.cpu().numpy() != oc)
    assert bad.size == 0, f"code bytes differ in blocks {bad[:8] // (B // 2)}"
    bad = np.flatnonzero(sse.cpu().numpy().view(np.uint32) != oe.view(np.uint32))
    assert bad.size == 0, f"block SSE differs at blocks {bad[:8]}"


def _pruned_sweep_equals(x, B, fmt, recipe, g, dg, codes, scales, sse):
    """The pruned brute-force sweep must reproduce the full sweep on every byte of the tensor."""
    mxq.mxq_set_option(mxq.MXQ_OPT_BRUTE_PRUNE, 1)
    try:
        c2, s2, e2 = mxq.quantize(x, B, fmt, recipe, g, dg)
        torch.cuda.synchronize()
    finally:
        mxq.mxq_set_option(mxq.MXQ_OPT_BRUTE_PRUNE, 0)
    assert torch.equal(s2, scales), f"scale bytes differ in {int((s2 != scales).sum())} blocks"
    assert torch.equal(c2, codes)
    assert torch.equal(e2.view(torch.int32), sse.view(torch.int32))


def _mse_matches_sum(sse, n):
    got = float(mxq.tensor_mse(sse, n).cpu()[0])
    want = float(sse.double().sum().cpu()) / n       # another binary64 summation order
    assert abs(got - want) <= 1e-6 * want
    return got


def test_weight_sweep_tensor_4096x4096_bf16_all_block_sizes():
    """The tensor and the passes of the default benchmark step (seeded exactly as bench.py does)."""
    n = 4096 * 4096
    x = inputs.student_t(n, 5, 0.02, dist.rank_seed(2, 0, 0), torch.bfloat16, "cuda")
    mse = {}
    for B in (2, 4, 8, 16, 32, 64):
        out = {}
        for recipe in (ABSMAX, ABSMAX_PZ, R4O6, BRUTE):
            codes, scales, sse = mxq.quantize(x, B, mxq.MXQ_SF_UE4M3, recipe)
            torch.cuda.synchronize()
            _check_full(x, B, mxq.MXQ_SF_UE4M3, recipe, 1.0, codes, scales, sse)
            out[recipe] = sse
            mse[(B, recipe)] = _mse_matches_sum(sse, n)
            if recipe == BRUTE:
                _pruned_sweep_equals(x, B, mxq.MXQ_SF_UE4M3, recipe, 1.0, None, codes, scales, sse)
        # candidate sets nest, and the SSE is one function of (block, code): bitwise orderings
        assert bool((out[BRUTE] <= out[R4O6]).all()) and bool((out[R4O6] <= out[ABSMAX]).all())
        assert bool((out[ABSMAX_PZ] <= out[ABSMAX]).all())
    # finer is better for the optimal scale (Results, numerical study): exact arithmetic would make it
    # monotone; binary32 sums of different lengths get a little slack
    bs = (2, 4, 8, 16, 32, 64)
    for a, b in zip(bs[:-1], bs[1:]):
        assert mse[(a, BRUTE)] <= mse[(b, BRUTE)] * (1 + 1e-6)


def test_hierarchical_leg_of_the_benchmark_step():
    n = 4096 * 4096
    x = inputs.student_t(n, 5, 0.02, dist.rank_seed(2, 0, 1), torch.bfloat16, "cuda")
    amax = torch.empty(1, dtype=torch.float32, device="cuda")
    dg = torch.empty(1, dtype=torch.float32, device="cuda")
    mxq.mxq_tensor_amax(x, n, amax, dg)
    torch.cuda.synchronize()
    assert float(amax.cpu()[0]) == float(x.float().abs().max().cpu())
    g = float(dg.cpu()[0])
    assert g == mxq.mxq_global_scale_from_amax(float(amax.cpu()[0]))
    for recipe in (ABSMAX, R4O6):
        codes, scales, sse = mxq.quantize(x, 16, mxq.MXQ_SF_UE4M3, recipe, 1.0, dg)
        torch.cuda.synchronize()
        _check_full(x, 16, mxq.MXQ_SF_UE4M3, recipe, g, codes, scales, sse)
        _mse_matches_sum(sse, n)
    # de-quantization of the whole tensor: every element is grid value times decode scale
    xh = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    mxq.mxq_dequantize(codes, scales, n, 16, mxq.MXQ_SF_UE4M3, g, xh)
    torch.cuda.synchronize()
    idx = _sample_blocks(n // 16, 2000, 5)
    t_idx = torch.from_numpy(idx).cuda()
    want = orc.dequantize(codes.view(-1, 8)[t_idx].cpu().numpy().reshape(-1), scales[t_idx].cpu().numpy(), idx.size * 16,
                          16, orc.UE4M3, g, orc.BF16)
    got = inputs.to_numpy_bits(xh.view(-1, 16)[t_idx].contiguous())
    assert np.array_equal(got, want.view(np.uint16))


def test_activation_shaped_8192x4096_bf16_outlier_columns():
    x = inputs.outlier_columns(8192, 4096, 3, dtype=torch.bfloat16, device="cuda")
    n = x.numel()
    amax = torch.empty(1, dtype=torch.float32, device="cuda")
    dg = torch.empty(1, dtype=torch.float32, device="cuda")
    mxq.mxq_tensor_amax(x, n, amax, dg)
    torch.cuda.synchronize()
    g = float(dg.cpu()[0])
    for fmt, gg, d in ((mxq.MXQ_SF_UE4M3, g, dg), (mxq.MXQ_SF_UE5M3, 1.0, None)):
        sses = {}
        for recipe in (ABSMAX, R4O6):
            codes, scales, sse = mxq.quantize(x, 16, fmt, recipe, 1.0, d)
            torch.cuda.synchronize()
            _check_full(x, 16, fmt, recipe, gg, codes, scales, sse)
            _mse_matches_sum(sse, n)
            sses[recipe] = sse
        assert bool((sses[R4O6] <= sses[ABSMAX]).all())


@pytest.mark.parametrize("name,rows,cols", [s for s in inputs.LLAMA8B_LAYER_SHAPES if s[0] in ("q", "k", "gate", "down")])
def test_llama_shaped_weight_matrices_bf16(name, rows, cols):
    """One matrix of each distinct shape of the Llama-3-8B-shaped set, all recipes, both FP8 scale formats."""
    index = [s[0] for s in inputs.LLAMA8B_LAYER_SHAPES].index(name)
    x = inputs.student_t(rows * cols, 4, 1.0 / np.sqrt(cols), 4 + index, torch.bfloat16, "cuda")
    n = x.numel()
    for fmt in (mxq.MXQ_SF_UE4M3, mxq.MXQ_SF_UE5M3):
        best = {}
        for B in (8, 16):
            out = {}
            for recipe in (ABSMAX, ABSMAX_PZ, R4O6, BRUTE):
                codes, scales, sse = mxq.quantize(x, B, fmt, recipe)
                torch.cuda.synchronize()
                if recipe != BRUTE:
                    _check_full(x, B, fmt, recipe, 1.0, codes, scales, sse)
                else:
                    _check_sampled(x, B, fmt, recipe, 1.0, codes, scales, sse, 1000, B + fmt + recipe + index)
                out[recipe] = sse
                if recipe == BRUTE:
                    _pruned_sweep_equals(x, B, fmt, recipe, 1.0, None, codes, scales, sse)
            assert bool((out[BRUTE] <= out[R4O6]).all()) and bool((out[R4O6] <= out[ABSMAX]).all())
            best[B] = _mse_matches_sum(out[BRUTE], n)
        assert best[8] <= best[16] * (1 + 1e-6)


@pytest.fixture(scope="module")
def laplace_16384x16384():
    n = 16384 * 16384
    x = inputs.laplace(n, 5, torch.float32, "cuda")
    amax = torch.empty(1, dtype=torch.float32, device="cuda")
    dg = torch.empty(1, dtype=torch.float32, device="cuda")
    mxq.mxq_tensor_amax(x, n, amax, dg)
    torch.cuda.synchronize()
    return x, dg, float(dg.cpu()[0])


@pytest.mark.parametrize("fmt", [mxq.MXQ_SF_UE8M0, mxq.MXQ_SF_UE4M3, mxq.MXQ_SF_UE5M3])
def test_bulk_brute_force_16384x16384_fp32_laplace_with_tensor_scale(laplace_16384x16384, fmt):
    """The bulk scale-search case at full size: every block size, full code sweep per block."""
    x, dg, g = laplace_16384x16384
    n = x.numel()
    prev = None
    for B in (2, 4, 8, 16, 32):
        codes, scales, sse = mxq.quantize(x, B, fmt, BRUTE, 1.0, dg)
        torch.cuda.synchronize()
        _check_sampled(x, B, fmt, BRUTE, g, codes, scales, sse, 1000, 900 + B + fmt)
        _pruned_sweep_equals(x, B, fmt, BRUTE, 1.0, dg, codes, scales, sse)
        m = _mse_matches_sum(sse, n)
        assert int(scales.max().cpu()) < (127 if fmt == mxq.MXQ_SF_UE4M3 else 255)
        if prev is not None:
            assert prev <= m * (1 + 1e-6)
        prev = m
        del codes, scales, sse


def test_more_than_two_to_the_32_elements():
    """A tensor whose element index, byte offsets and block count need more than 32 bits where they
    are formed (2^32 + 3 * 2^20 bf16 elements, 8.6 GB): one-pass recipes, brute force, tensor abs-max,
    tensor MSE and de-quantization, compared with the oracle on the first and last blocks and on random ones."""
    n = (1 << 32) + (3 << 20)
    B, fmt = 16, mxq.MXQ_SF_UE4M3
    x = inputs.student_t(n, 5, 0.02, 99, torch.bfloat16, "cuda")
    x[-5] = 96.0                                       # the tensor maximum sits beyond element 2^32
    amax = torch.empty(1, dtype=torch.float32, device="cuda")
    mxq.mxq_tensor_amax(x, n, amax)
    torch.cuda.synchronize()
    assert float(amax.cpu()[0]) == 96.0 == float(x.abs().max().float().cpu())
    codes, scales, sse = mxq.alloc_outputs(n, B, "cuda")
    for recipe in (ABSMAX, R4O6):
        mxq.mxq_quantize_ex(x, n, B, fmt, recipe, 1.0, None, codes, scales, sse)
        torch.cuda.synchronize()
        _check_sampled(x, B, fmt, recipe, 1.0, codes, scales, sse, 4000, 4242 + recipe)
        got = float(mxq.tensor_mse(sse, n).cpu()[0])
        want = sum(float(part.double().sum().cpu()) for part in sse.split(1 << 26)) / n
        assert abs(got - want) <= 1e-6 * want
    # brute force at this size, both sweeps
    mxq.mxq_quantize_ex(x, n, B, fmt, BRUTE, 1.0, None, codes, scales, sse)
    torch.cuda.synchronize()
    _check_sampled(x, B, fmt, BRUTE, 1.0, codes, scales, sse, 1500, 4250)
    _pruned_sweep_equals(x, B, fmt, BRUTE, 1.0, None, codes, scales, sse)
    xh = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    mxq.mxq_dequantize(codes, scales, n, B, fmt, 1.0, xh)
    torch.cuda.synchronize()
    idx = _sample_blocks(n // B, 3000, 17)
    t_idx = torch.from_numpy(idx).cuda()
    want = orc.dequantize(codes.view(-1, B // 2)[t_idx].cpu().numpy().reshape(-1), scales[t_idx].cpu().numpy(), idx.size * B,
                          B, orc.UE4M3, 1.0, orc.BF16)
    got = inputs.to_numpy_bits(xh.view(-1, B)[t_idx].contiguous())
    assert np.array_equal(got, want.view(np.uint16))
