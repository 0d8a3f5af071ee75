"""GPU parity of the analysis entry points (clipping-only SSE, histograms, segment MSE) and of a
reduced numerical study against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import mxq_oracle as orc
from paper_2605_08565_b200 import binding as mxq
from paper_2605_08565_b200 import inputs, study

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("B", [2, 4, 16, 64])
def test_clip_sse_and_histograms_bit_exact(dtype, B):
    n = 3 * 256 * max(B, 8) + 5 * 64 + (B if B < 8 else 0)
    x = (inputs.adversarial(n, 3 + B, torch.float32) * 0.5).to(dtype).contiguous()
    for fmt, g, recipe in ((mxq.MXQ_SF_UE4M3, 1.0, mxq.MXQ_ABSMAX), (mxq.MXQ_SF_UE4M3, 0.0131, mxq.MXQ_ABSMAX_PZ),
                           (mxq.MXQ_SF_UE5M3, 1.0, mxq.MXQ_4O6), (mxq.MXQ_SF_UE8M0, 1.0, mxq.MXQ_ABSMAX)):
        xg = x.cuda()
        codes, scales, sse = mxq.quantize(xg, B, fmt, recipe, g)
        clip = torch.empty_like(sse)
        mxq.mxq_block_clip_sse(xg, n, B, fmt, g, None, scales, clip)
        ch = torch.zeros(16, dtype=torch.int64, device="cuda")
        sh = torch.zeros(256, dtype=torch.int64, device="cuda")
        mxq.mxq_histograms(codes, scales, n, B, ch, sh)
        mxq.mxq_histograms(codes, scales, n, B, ch, sh)      # counts accumulate
        torch.cuda.synchronize()
        xb = inputs.to_numpy_bits(x)
        oc, os_, oe = orc.quantize(xb, B, fmt, recipe, g)
        want = orc.block_clip_sse(xb, os_, B, fmt, g)
        assert np.array_equal(clip.cpu().numpy().view(np.uint32), want.view(np.uint32))
        och, osh = orc.histograms(oc, os_, n, B)
        assert np.array_equal(ch.cpu().numpy().astype(np.uint64), 2 * och)
        assert np.array_equal(sh.cpu().numpy().astype(np.uint64), 2 * osh)


def test_segment_mse_matches_oracle():
    rng = np.random.default_rng(8)
    for nseg, per in ((1, 1), (7, 50), (151, 1000), (3, 70001)):
        sse = (rng.random(nseg * per) * np.exp2(rng.integers(-30, 4, nseg * per))).astype(np.float32)
        d = torch.from_numpy(sse).cuda()
        out = torch.empty(nseg, dtype=torch.float64, device="cuda")
        mxq.mxq_segment_mse(d, nseg * per, per, per * 16, out)
        mxq_out = out.cpu().numpy()
        want = orc.segment_mse(sse, per, per * 16)
        assert np.all(np.abs(mxq_out - want) <= 1e-12 * want)
        out2 = torch.empty_like(out)
        mxq.mxq_segment_mse(d, nseg * per, per, per * 16, out2)
        assert torch.equal(out, out2)


def test_reduced_numerical_study_against_oracle():
    """16 sigmas x 2000 blocks, all five recipes, block sizes 4 and 16: every MSE and clipping-MSE
    point against the oracle on the very same samples."""
    n_sigma, per_blocks = 16, 2000
    res = study.run(block_sizes=(4, 16), n_sigma=n_sigma, blocks_per_sigma=per_blocks, seed=3, histogram_sigmas=(0, 9))
    for B in (4, 16):
        x = inputs.sigma_sweep(per_blocks * B, 3 * 1000 + B, n_sigma, device="cuda").cpu()
        xb = inputs.to_numpy_bits(x)
        for name, rid in study.RECIPES.items():
            oc, os_, oe = orc.quantize(xb, B, orc.UE4M3, rid, 1.0, threads=8)
            want = orc.segment_mse(oe, per_blocks, per_blocks * B)
            got = np.array(res["mse"][name][B])
            assert np.all(np.abs(got - want) <= 1e-6 * want), (name, B)
            wclip = orc.segment_mse(orc.block_clip_sse(xb, os_, B, orc.UE4M3), per_blocks, per_blocks * B)
            gclip = np.array(res["clip_mse"][name][B])
            assert np.all(np.abs(gclip - wclip) <= 1e-6 * wclip + 1e-300), (name, B)
            for k in (0, 9):
                lo = k * per_blocks
                och, osh = orc.histograms(oc[lo * B // 2:(lo + per_blocks) * B // 2], os_[lo:lo + per_blocks],
                                          per_blocks * B, B)
                h = res["hist"][f"{name}/B{B}/sigma{k}"]
                assert np.array_equal(np.array(h["codes"], dtype=np.uint64), och)
                assert np.array_equal(np.array(h["scales"], dtype=np.uint64), osh)
    f = study.findings(res)
    assert f["pz_never_worse"]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("B", [2, 4, 8, 16, 32, 64])
@pytest.mark.parametrize("recipe", [mxq.MXQ_ABSMAX_OCP, mxq.MXQ_ABSMAX_CLIP7])
def test_alternative_power_of_two_recipes_bit_exact(dtype, B, recipe):
    n = 3 * 256 * max(B, 8) + 5 * 64 + (B if B < 8 else 0)
    x = inputs.adversarial(n, 21 + B, dtype)
    if recipe == mxq.MXQ_ABSMAX_CLIP7:      # block maxima on both sides of the 1.75 * 2^k edges of the rule
        xb = x.view(-1, B)
        k = torch.arange(xb.shape[0] // 3)
        edge = torch.tensor([1.75, 1.7421875, 1.765625])[k % 3] * torch.exp2(((k // 3) % 24 - 12).float())
        xb[::3][:k.numel(), 0] = edge.to(dtype)
    for g in (1.0, 0.0131, 2.0 ** -100):
        xg = x.cuda()
        codes, scales, sse = mxq.quantize(xg, B, mxq.MXQ_SF_UE8M0, recipe, g)
        torch.cuda.synchronize()
        oc, os_, oe = orc.quantize(inputs.to_numpy_bits(x), B, orc.UE8M0, recipe, g)
        assert np.array_equal(scales.cpu().numpy(), os_)
        assert np.array_equal(codes.cpu().numpy(), oc)
        assert np.array_equal(sse.cpu().numpy().view(np.uint32), oe.view(np.uint32))
    with pytest.raises(mxq.MxqError):
        mxq.quantize(x.cuda(), B, mxq.MXQ_SF_UE4M3, recipe)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("B", [2, 4, 8, 16, 32, 64])
def test_fake_quantize_equals_quantize_then_dequantize(dtype, B):
    n = 3 * 256 * max(B, 8) + 5 * 64 + (B if B < 8 else 0)
    x = (inputs.adversarial(n, 33 + B, torch.float32) * 0.25).to(dtype).contiguous()
    xg = x.cuda()
    for fmt, recipe, g in ((mxq.MXQ_SF_UE4M3, mxq.MXQ_ABSMAX, 1.0), (mxq.MXQ_SF_UE4M3, mxq.MXQ_4O6_PZ, 0.0131),
                           (mxq.MXQ_SF_UE5M3, mxq.MXQ_4O6, 1.0), (mxq.MXQ_SF_UE8M0, mxq.MXQ_ABSMAX_OCP, 1.0),
                           (mxq.MXQ_SF_UE8M0, mxq.MXQ_ABSMAX, 3.0e-37)):
        for odt, oid in ((torch.float32, orc.F32), (torch.bfloat16, orc.BF16)):
            out = torch.empty(n, dtype=odt, device="cuda")
            mxq.mxq_fake_quantize(xg, n, B, fmt, recipe, g, None, out)
            codes, scales, _ = mxq.quantize(xg, B, fmt, recipe, g)
            two_step = torch.empty(n, dtype=odt, device="cuda")
            mxq.mxq_dequantize(codes, scales, n, B, fmt, g, two_step)
            torch.cuda.synchronize()
            got = inputs.to_numpy_bits(out)
            view = np.uint32 if odt == torch.float32 else np.uint16
            assert np.array_equal(got.view(view), inputs.to_numpy_bits(two_step).view(view))
            want = orc.fake_quantize(inputs.to_numpy_bits(x), B, fmt, recipe, g, oid)
            assert np.array_equal(got.view(view), want.view(view))
    out = torch.empty(n, dtype=torch.float32, device="cuda")
    with pytest.raises(mxq.MxqError):
        mxq.mxq_fake_quantize(xg, n, B, mxq.MXQ_SF_UE4M3, mxq.MXQ_BRUTE, 1.0, None, out)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_mask_interval_matches_definition(dtype):
    for n in (1, 7, 8, 4096 + 5):
        x = (inputs.normal(max(n, 8), 4 + n, 0.02, torch.float32)[:n]).to(dtype).contiguous()
        xg = x.cuda()
        out = torch.empty_like(xg)
        for lo, hi in ((0.0, 0.0), (0.005, 0.015), (0.0, 0.035), (0.02, 1.0e9)):
            mxq.mxq_mask_interval(xg, n, lo, hi, out)
            torch.cuda.synchronize()
            want = orc.mask_interval(inputs.to_numpy_bits(x), lo, hi)
            got = inputs.to_numpy_bits(out)
            view = np.uint32 if dtype == torch.float32 else np.uint16
            assert np.array_equal(got.view(view), want.view(view)), (n, lo, hi)
    y = xg.clone()
    mxq.mxq_mask_interval(y, n, 0.005, 0.015, y)             # in place
    mxq.mxq_mask_interval(xg, n, 0.005, 0.015, out)
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.int16 if dtype == torch.bfloat16 else torch.int32),
                       out.view(torch.int16 if dtype == torch.bfloat16 else torch.int32))
    with pytest.raises(mxq.MxqError):
        mxq.mxq_mask_interval(xg, n, 0.02, 0.01, out)


def test_numerical_study_at_the_papers_size_shows_the_papers_findings():
    """The full protocol of the numerical study (Results, "Numerical Study" and its MSE-versus-sigma
    figure): N(0, sigma^2) samples, 151 sigmas evenly spaced in [0.0005, 0.05], 50,000 blocks per sigma,
    block sizes 4, 8, 16, 32, FP4 entries, UE4M3 scales.  Asserted, with the sampling error of every MSE
    estimate taken into account (mean of 50,000 block SSEs; different block sizes see different samples):
      * Region A: where every abs-max scale underflows to zero the MSE is the signal power itself, the
        abs-max curve peaks far above prevent-zero's at small sigma, and prevent-zero is never worse;
      * Region B: with abs-max + prevent-zero the smallest block is significantly WORSE than the largest
        over a range of sigmas (the inversion), and most of that error is clipping;
      * 4-over-6 + prevent-zero and brute force show no significant inversion at any sigma, and the
        brute-force optimum never gets significantly worse when blocks get finer."""
    res = study.run(keep_block_sse=True)
    sig = np.array(res["sigma"])
    assert len(sig) == 151 and res["blocks_per_sigma"] == 50_000
    bs = (4, 8, 16, 32)
    mean, se = {}, {}
    for name in study.RECIPES:
        for B in bs:
            s = res["block_sse"][name][B].double()
            mean[name, B] = (s.mean(dim=1) / B).cpu().numpy()
            se[name, B] = (s.std(dim=1) / (s.shape[1] ** 0.5) / B).cpu().numpy()
            got = np.array(res["mse"][name][B])
            assert np.all(np.abs(got - mean[name, B]) <= 1e-9 * mean[name, B] + 1e-300)   # the library's tree = the plain mean

    def worse(name, b_small, b_large, z=5.0):
        """sigmas at which b_small's MSE exceeds b_large's by more than z combined standard errors"""
        d = mean[name, b_small] - mean[name, b_large]
        return np.flatnonzero(d > z * np.sqrt(se[name, b_small] ** 2 + se[name, b_large] ** 2))

    # Region A
    k0 = 0                                                       # sigma = 0.0005: every block maximum / 6 rounds to scale 0
    assert abs(mean["absmax", 4][k0] / sig[k0] ** 2 - 1.0) < 0.02
    ratio = mean["absmax", 4] / mean["absmax_pz", 4]
    kpk = int(np.argmax(ratio))
    assert ratio[kpk] > 10.0 and sig[kpk] < 0.005
    for B in bs:
        assert np.all(mean["absmax_pz", B] <= mean["absmax", B])
        assert np.all(mean["4o6_pz", B] <= mean["4o6", B])
    # Region B
    inv = worse("absmax_pz", 4, 32)
    assert inv.size >= 20 and 0.004 < sig[inv].min() < 0.01 and sig[inv].max() < 0.03
    mid = inv[inv.size // 2]
    clip_share = np.array(res["clip_mse"]["absmax_pz"][4])[mid] / mean["absmax_pz", 4][mid]
    assert clip_share > 0.4
    # no inversion for 4-over-6 + prevent-zero beyond the zero-scale region, none at all for brute force
    assert np.all(sig[worse("4o6_pz", 4, 32)] < 0.004)
    assert worse("brute", 4, 32).size == 0
    for a, b in ((4, 8), (8, 16), (16, 32)):
        assert worse("brute", a, b).size == 0
    # the recipes order as the paper has them, at every sigma and block size
    for B in bs:
        assert np.all(mean["brute", B] <= mean["4o6_pz", B] * (1 + 1e-12))
        assert np.all(mean["4o6_pz", B] <= mean["absmax_pz", B] * (1 + 1e-12))
