"""GPU parity: the CUDA library, called through its C-ABI binding, against the CPU oracle on the
same seeded inputs.  Codes, scale bytes and block SSE must be bit-identical; tensor MSE within 1e-6
relative (binary64 sums in a different order)."""
import numpy as np
import pytest
import torch

from oracle import mxq_oracle as orc
from paper_2605_08565_b200 import binding as mxq
from paper_2605_08565_b200 import inputs

pytestmark = pytest.mark.gpu

FMTS = [mxq.MXQ_SF_UE8M0, mxq.MXQ_SF_UE4M3, mxq.MXQ_SF_UE5M3]
RECIPES = [mxq.MXQ_ABSMAX, mxq.MXQ_ABSMAX_PZ, mxq.MXQ_4O6, mxq.MXQ_4O6_PZ, mxq.MXQ_BRUTE, mxq.MXQ_BRUTE_PZ]
BLOCKS = [2, 4, 8, 16, 32, 64]
MSE_RTOL = 1e-6


def _mixed(n, seed, dtype):
    """Normals at several magnitudes interleaved with tie-prone / zero / denormal / huge runs."""
    a = inputs.adversarial(n, seed, torch.float32)
    b = inputs.normal(n, seed + 1, 1.0, torch.float32) * torch.exp2(torch.randint(-14, 8, (n // 64 + 1,), generator=torch.Generator().manual_seed(seed)).float()).repeat_interleave(64)[:n]
    pick = (torch.arange(n) // 64) % 3 == 0
    return torch.where(pick, a, b).to(dtype).contiguous()


def gpu_quantize(x_cpu, B, fmt, recipe, g=1.0, device_g=False):
    x = x_cpu.cuda()
    dg = torch.tensor([g], dtype=torch.float32, device="cuda") if device_g else None
    codes, scales, sse = mxq.quantize(x, B, fmt, recipe, 1.0 if device_g else g, dg)
    mse = mxq.tensor_mse(sse, x.numel())
    torch.cuda.synchronize()
    return codes.cpu().numpy(), scales.cpu().numpy(), sse.cpu().numpy(), float(mse.cpu()[0])


def check_parity(x_cpu, B, fmt, recipe, g=1.0, device_g=False):
    gc, gs, ge, gm = gpu_quantize(x_cpu, B, fmt, recipe, g, device_g)
    oc, os_, oe = orc.quantize(inputs.to_numpy_bits(x_cpu), B, fmt, recipe, g, threads=8)
    bad = np.flatnonzero(gs != os_)
    assert bad.size == 0, f"scale bytes differ at blocks {bad[:8]} gpu={gs[bad[:8]]} oracle={os_[bad[:8]]}"
    bad = np.flatnonzero(gc != oc)
    assert bad.size == 0, f"code bytes differ at {bad[:8]} gpu={gc[bad[:8]]} oracle={oc[bad[:8]]}"
    bad = np.flatnonzero(ge.view(np.uint32) != oe.view(np.uint32))
    assert bad.size == 0, f"block SSE differs at {bad[:8]} gpu={ge[bad[:8]]} oracle={oe[bad[:8]]}"
    om = orc.tensor_mse(oe, x_cpu.numel())
    assert abs(gm - om) <= MSE_RTOL * abs(om) + 1e-300, (gm, om)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("B", BLOCKS)
@pytest.mark.parametrize("fmt", FMTS)
def test_one_pass_recipes_bit_exact(dtype, B, fmt):
    # several CTAs' worth of chunks plus a ragged end (not a multiple of 8 for the small blocks)
    n = 3 * 256 * max(B, 8) + 5 * 64 + (B if B < 8 else 0)
    x = _mixed(n, 10 + B + fmt, dtype)
    for recipe in (mxq.MXQ_ABSMAX, mxq.MXQ_ABSMAX_PZ, mxq.MXQ_4O6, mxq.MXQ_4O6_PZ):
        check_parity(x, B, fmt, recipe, 1.0)
        check_parity(x, B, fmt, recipe, 0.0131)


@pytest.fixture(params=[0, 1], ids=["full_sweep", "pruned_sweep"])
def sweep_mode(request):
    """Both ways of running the brute-force kernels: every code evaluated, and the codes that provably
    tie with the all-zero quantization left out.  The outputs must not depend on it."""
    mxq.mxq_set_option(mxq.MXQ_OPT_BRUTE_PRUNE, request.param)
    assert mxq.mxq_get_option(mxq.MXQ_OPT_BRUTE_PRUNE) == request.param
    yield request.param
    mxq.mxq_set_option(mxq.MXQ_OPT_BRUTE_PRUNE, 0)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("B", BLOCKS)
@pytest.mark.parametrize("fmt", FMTS)
def test_brute_force_bit_exact(dtype, B, fmt, sweep_mode):
    n = 2 * 256 * B + 7 * B
    x = _mixed(n, 40 + B + fmt, dtype)
    check_parity(x, B, fmt, mxq.MXQ_BRUTE, 1.0)
    check_parity(x, B, fmt, mxq.MXQ_BRUTE_PZ, 0.0131)


@pytest.mark.parametrize("B", BLOCKS)
@pytest.mark.parametrize("fmt", FMTS)
def test_brute_force_on_small_magnitudes_and_quarter_scale_ties(B, fmt, sweep_mode):
    """Inputs on which most codes quantize a whole warp's elements to zero: weight-like small values,
    all-zero stretches as long as a warp's share, and magnitudes that are exactly a quarter of a
    decode scale (the tie that still rounds to zero)."""
    n = 3 * 256 * max(B, 32) + 11 * B
    gen = torch.Generator().manual_seed(900 + B + fmt)
    x = inputs.student_t(n, 5, 0.02, 70 + B, torch.float32)
    span = 32 * max(B, 32)                                   # elements one warp holds per trip
    x[span:2 * span] = 0.0
    x[4 * span:5 * span] *= 2.0 ** -20
    quarter = torch.exp2(torch.randint(-12, 3, (span,), generator=gen).float()) * (1.0 + torch.randint(0, 8, (span,), generator=gen).float() / 8)
    sign = torch.where(torch.rand(span, generator=gen) < 0.5, -1.0, 1.0)
    x[6 * span:7 * span] = 0.25 * quarter * sign
    for dtype in (torch.float32, torch.bfloat16):
        xd = x.to(dtype).contiguous()
        check_parity(xd, B, fmt, mxq.MXQ_BRUTE, 1.0)
        check_parity(xd, B, fmt, mxq.MXQ_BRUTE_PZ, 1.0)
        check_parity(xd, B, fmt, mxq.MXQ_BRUTE, 3.7e-3)


@pytest.mark.parametrize("B", [8, 16, 32, 64])
@pytest.mark.parametrize("fmt", FMTS)
def test_brute_force_on_warps_of_unlike_blocks(B, fmt, sweep_mode):
    """Blocks of very different magnitude side by side in one warp's share (one tiny block, one huge
    block, blocks of equal elements, a block with a single nonzero element among ordinary ones): the
    cases in which bounds taken from some blocks must not decide for the others."""
    span = 32 * max(B, 32)
    n = 8 * span
    x = inputs.normal(n, 500 + B + fmt, 1.0, torch.float32)
    xb = x.view(-1, B)
    nb = xb.shape[0]
    xb[1::37] *= 2.0 ** -9            # tiny blocks among ordinary ones
    xb[5::41] *= 2.0 ** 7             # huge blocks
    xb[7::43] = 0.75                  # constant blocks (zero error at the right scale)
    xb[11::47] = 0.0
    xb[11::47, 0] = -3.0              # one nonzero element
    xb[13::53] = 0.0                  # all-zero blocks
    xb[nb // 2:nb // 2 + 3] *= 2.0 ** -30
    for g in (1.0, 0.0173):
        check_parity(x, B, fmt, mxq.MXQ_BRUTE, g)
    check_parity(x.to(torch.bfloat16), B, fmt, mxq.MXQ_BRUTE_PZ, 1.0)


def test_option_calls_reject_bad_arguments():
    with pytest.raises(mxq.MxqError):
        mxq.mxq_set_option(99, 1)
    with pytest.raises(mxq.MxqError):
        mxq.mxq_set_option(mxq.MXQ_OPT_BRUTE_PRUNE, 2)
    with pytest.raises(mxq.MxqError):
        mxq.mxq_get_option(99)
    assert mxq.mxq_get_option(mxq.MXQ_OPT_BRUTE_PRUNE) == 0


@pytest.mark.parametrize("recipe", RECIPES)
def test_extreme_global_scales(recipe, sweep_mode):
    x = _mixed(4096, 77, torch.float32)
    for g in (2.0 ** -30, 2.0 ** 20, 3.0e-37, 1.0e30):
        check_parity(x, 16, mxq.MXQ_SF_UE4M3, recipe, g)
    check_parity(x, 8, mxq.MXQ_SF_UE8M0, recipe, 2.0 ** -100)
    check_parity(x, 8, mxq.MXQ_SF_UE8M0, recipe, 2.0 ** 100)
    check_parity(x, 8, mxq.MXQ_SF_UE5M3, recipe, 5.0e-33)


def _ulp_neighbours(center, span):
    """float32 values from `span` units in the last place below `center` to `span` above."""
    c = np.float32(center)
    out = [c]
    lo = hi = c
    for _ in range(span):
        lo = np.nextafter(lo, np.float32(-np.inf), dtype=np.float32)
        hi = np.nextafter(hi, np.float32(np.inf), dtype=np.float32)
        out += [lo, hi]
    return out


@pytest.mark.parametrize("fmt", [mxq.MXQ_SF_UE4M3, mxq.MXQ_SF_UE5M3])
@pytest.mark.parametrize("g", [1.0, 0.0371, 1.0 / 3.0, 0.7, 1.9e-3])
def test_elements_and_maxima_next_to_rounding_midpoints(fmt, g):
    """Blocks built so that quotients fall within a few units in the last place of an FP4 midpoint of
    the block's own decode scale, and block maxima within a few units of a scale-code midpoint (for
    both 4-over-6 targets): the inputs on which a quotient that is not correctly rounded, or a target
    computed with one division instead of two, picks the neighbouring code."""
    B = 16
    mids = [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]
    blocks = []
    n_codes = orc.num_codes(fmt)
    for code in range(9, n_codes - 8, 7):
        S = np.float32(orc.scale_value(fmt, code))
        a = np.float32(np.float32(6.0) * np.float32(S * np.float32(g)))        # a block maximum that selects about this scale
        head = np.zeros(B, dtype=np.float32)
        head[0] = a
        _, sc, _ = orc.quantize(head, B, fmt, orc.ABSMAX, g)
        D = np.float32(np.float32(orc.scale_value(fmt, int(sc[0]))) * np.float32(g))
        near = [v for m in mids for v in _ulp_neighbours(np.float32(m) * D, 2)]   # 35 values, all below the maximum
        for i in range(0, len(near), B - 1):
            blk = np.zeros(B, dtype=np.float32)
            part = near[i:i + B - 1]
            blk[1:1 + len(part)] = part
            blk[1::2] *= -1
            blk[0] = a
            blocks.append(blk)
        # maxima next to the midpoint between this scale code and the next, for M = 6 and M = 4
        mid = (np.float64(orc.scale_value(fmt, code)) + np.float64(orc.scale_value(fmt, code + 1))) / 2
        for M in (6.0, 4.0):
            for a2 in _ulp_neighbours(np.float32(mid * M * g), 3):
                blk = np.zeros(B, dtype=np.float32)
                blk[5] = -a2
                blk[9] = a2 * np.float32(0.37)
                blocks.append(blk)
    x = torch.from_numpy(np.concatenate(blocks))
    if not np.all(np.isfinite(x.numpy())):
        x = torch.nan_to_num(x, nan=0.0, posinf=0.0, neginf=0.0)
    for recipe in (mxq.MXQ_ABSMAX, mxq.MXQ_ABSMAX_PZ, mxq.MXQ_4O6, mxq.MXQ_4O6_PZ):
        check_parity(x, B, fmt, recipe, g)
        check_parity(x, B, fmt, recipe, g, device_g=True)
    check_parity(x[: 64 * B], B, fmt, mxq.MXQ_BRUTE, g)


def _to_bf16_floor(p64):
    """Largest bf16 value not above the positive binary64 number p64, as float32."""
    f = np.float32(p64)
    if np.float64(f) > p64:
        f = np.nextafter(f, np.float32(0), dtype=np.float32)
    return (np.array([f], dtype=np.float32).view(np.uint32) & np.uint32(0xFFFF0000)).view(np.float32)[0]


def _bf16_step(v, k):
    """The bf16 value k steps above (k < 0: below) the bf16 value v."""
    return (np.array([v], dtype=np.float32).view(np.uint32).astype(np.int64) + (k << 16)).astype(np.uint32).view(np.float32)[0]


def _one_multiply_code_differs(v, D):
    """True if rounding RZ(v * RN(1 / D)) to the FP4 grid gives another magnitude than rounding fl32(v / D)
    (a single multiply by the reciprocal, rounded toward zero, against the correctly rounded quotient)."""
    R = np.float32(np.float32(1) / D)
    p = np.float64(v) * np.float64(R)                 # exact: 8 x 24 significant bits
    h = np.float32(p)
    if np.float64(h) > p:
        h = np.nextafter(h, np.float32(0), dtype=np.float32)
    f = np.float32(v / D)
    return orc.e2m1_index(float(h)) != orc.e2m1_index(float(f))


def test_bf16_elements_next_to_midpoints_of_long_decode_scales():
    """bf16 input under tensor scales g chosen so that, for the decode scale D = fl(1.0 * g) of code 0x38,
    M * D lies within a few 2^-24 of a bf16 value for one FP4 midpoint M: there a single multiply by 1 / D
    can round to the other side of M although bf16 values are 2^-8 apart.  Each block holds a maximum
    that selects code 0x38 and, for all seven midpoints, the bf16 values just below and above M * D.  The
    test first shows (on the host) that for several of these scales the one-multiply quotient is wrong
    for an element of the block, so a kernel that took that shortcut unchecked fails here."""
    B, fmt = 16, mxq.MXQ_SF_UE4M3
    mids = [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]
    rng = np.random.default_rng(77)
    wrong_somewhere = 0
    cases = []
    for _ in range(400):
        vb = _bf16_step(np.float32(2.0 ** int(rng.integers(-12, 3))), int(rng.integers(0, 128)))
        m = mids[int(rng.integers(0, 7))]
        D = np.float32(np.float64(vb) / m)
        for _k in range(int(rng.integers(0, 4))):
            D = np.nextafter(D, np.float32(np.inf if rng.integers(0, 2) else 0), dtype=np.float32)
        g = D                                          # code 0x38 has scale value 1.0: D = fl(1.0 * g) = g
        near = []
        for mm in mids:
            v0 = _to_bf16_floor(np.float64(mm) * np.float64(D))
            near += [v0, _bf16_step(v0, 1)]
        a = None                                       # a bf16 maximum above every other element that selects code 0x38
        for cand in (_to_bf16_floor(6.0 * np.float64(D)), _bf16_step(_to_bf16_floor(6.0 * np.float64(D)), 1),
                     _bf16_step(_to_bf16_floor(6.0 * np.float64(D)), -1)):
            head = np.zeros(B, dtype=np.float32)
            head[0] = cand
            if cand > max(near) and orc.quantize(head, B, fmt, orc.ABSMAX, float(g))[1][0] == 0x38:
                a = cand
                break
        if a is None:
            continue
        wrong = any(_one_multiply_code_differs(v, D) for v in near)
        wrong_somewhere += int(wrong)
        if wrong or len(cases) < 12:
            blk = np.zeros(B, dtype=np.float32)
            blk[0] = a
            blk[1:15] = near
            blk[2::2] *= -1
            cases.append((float(g), blk))
        if wrong_somewhere >= 12 and len(cases) >= 24:
            break
    assert wrong_somewhere >= 5, "the generator no longer produces scales that defeat the one-multiply quotient"
    filler = inputs.normal(64 * B, 3, 1.0, torch.float32).numpy()
    for g, blk in cases:
        x = torch.from_numpy(np.concatenate([blk, filler * np.float32(g), blk[::-1].copy()])).to(torch.bfloat16)
        for recipe in (mxq.MXQ_ABSMAX, mxq.MXQ_4O6_PZ):
            check_parity(x, B, fmt, recipe, g, device_g=True)
    # the same blocks walked as parts of longer blocks and as small ones
    g, blk = cases[0]
    x = torch.from_numpy(np.concatenate([blk] * 8 + [filler * np.float32(g)])).to(torch.bfloat16)
    for Bx in (4, 8, 32, 64):
        check_parity(x, Bx, fmt, mxq.MXQ_4O6, g)
        check_parity(x, Bx, mxq.MXQ_SF_UE5M3, mxq.MXQ_ABSMAX, g)


def test_bf16_under_the_tensor_scale_of_every_bf16_amax_significand():
    """Hierarchical scaling of a bf16 tensor: g = amax / 2688 with amax a bf16 value.  Quotients v / D are
    then ratios of small integers and hit FP4 rounding midpoints exactly in real arithmetic, for every
    amax, while the binary32 g and D carry rounding errors: the inputs on which a reciprocal multiply is
    most likely to round to the wrong side.  One launch per amax significand (128 of them), the tensor
    scale taken on the device from the tensor itself, data drawn as bf16 values over four binades below
    the maximum so that every (significand, midpoint) meeting occurs thousands of times."""
    B, n = 16, 64 * 1024
    gen = torch.Generator().manual_seed(2688)
    for s in range(128, 256):
        amax = np.float32(s / 128.0 * 2.0 ** ((s % 7) - 3))
        sig = torch.randint(128, 256, (n,), generator=gen).float() / 128.0
        ex = torch.randint(-6, 0, (n,), generator=gen).float()
        sign = torch.randint(0, 2, (n,), generator=gen).float() * 2 - 1
        x = (sig * torch.exp2(ex) * sign * float(amax)).to(torch.bfloat16)
        x[int(s) * 17] = float(amax)
        xg = x.cuda()
        a = torch.empty(1, dtype=torch.float32, device="cuda")
        dg = torch.empty(1, dtype=torch.float32, device="cuda")
        mxq.mxq_tensor_amax(xg, n, a, dg)
        g = float(dg.cpu()[0])
        assert float(a.cpu()[0]) == float(amax) and g == float(orc.global_scale_from_amax(amax))
        fmt = mxq.MXQ_SF_UE4M3 if s % 2 == 0 else mxq.MXQ_SF_UE5M3
        check_parity(x, B, fmt, mxq.MXQ_4O6 if s % 4 < 2 else mxq.MXQ_ABSMAX, g, device_g=True)


@pytest.mark.parametrize("g", [1.3 * 2.0 ** -40, 0.0131, 1.7 * 2.0 ** 19, 1.1 * 2.0 ** -41, 1.2 * 2.0 ** 20])
def test_bf16_block_maxima_over_the_whole_exponent_range_under_tensor_scales(g):
    """bf16 blocks whose maxima run through the binades from the bf16 denormals up to 2^60 under
    tensor scales at and just outside the range for which the kernels use their lean loop: maxima far above
    the saturation point of the scale format, maxima so small that the quotient by g underflows, zero
    blocks, and everything in between, for both FP8 formats and every one-pass recipe."""
    B = 8
    gen = torch.Generator().manual_seed(41)
    blocks = []
    for e in range(-133, 61):                      # block SSEs stay finite in binary32
        blk = (torch.rand(4, B, generator=gen) * 2 - 1) * 2.0 ** e
        blk[:, e % B] = 2.0 ** e * (1.0 + (e % 7) / 8.0)
        blocks.append(blk.reshape(-1))
    blocks.append(torch.zeros(4 * B))
    x = torch.cat(blocks).to(torch.bfloat16)
    x = torch.cat([x, x.flip(0)])
    for fmt in (mxq.MXQ_SF_UE4M3, mxq.MXQ_SF_UE5M3):
        for recipe in (mxq.MXQ_ABSMAX, mxq.MXQ_ABSMAX_PZ, mxq.MXQ_4O6, mxq.MXQ_4O6_PZ):
            check_parity(x, B, fmt, recipe, g)
    check_parity(x, 16, mxq.MXQ_SF_UE4M3, mxq.MXQ_4O6_PZ, g, device_g=True)
    check_parity(x, 32, mxq.MXQ_SF_UE5M3, mxq.MXQ_4O6, g)
    check_parity(x, 2, mxq.MXQ_SF_UE4M3, mxq.MXQ_4O6_PZ, g)


@pytest.mark.parametrize("g", [1.0, 0.0131, 0.75])
def test_bf16_block_maxima_next_to_every_ue5m3_scale_midpoint(g):
    """4-over-6 on bf16 with UE5M3 scales: block maxima placed at the bf16 values around M * g * (midpoint of
    two neighbouring scale values) for every pair of neighbouring codes and both targets M = 4 and 6, i.e.
    where the rounding of either candidate's scale is decided, across the whole code range (the kernels
    round both candidates with one UE4M3 conversion of a scaled pair; see the oracle-side test of that
    identity).  UE4M3 runs on the same data for comparison."""
    B = 8
    blocks = []
    for fmt in (mxq.MXQ_SF_UE5M3,):
        for c in range(0, orc.num_codes(fmt) - 1):
            mid = (orc.scale_value(fmt, c) + orc.scale_value(fmt, c + 1)) / 2
            for M in (4.0, 6.0):
                a0 = _to_bf16_floor(np.float64(mid) * M * g)
                if not (0 < a0 < 1e30):
                    continue
                for k in (-1, 0, 1, 2):
                    a = _bf16_step(a0, k)
                    blk = np.zeros(B, dtype=np.float32)
                    blk[(c + k) % B] = a if c % 2 else -a
                    blk[(c + k + 3) % B] = a * np.float32(0.4375)
                    blocks.append(blk)
    x = torch.from_numpy(np.concatenate(blocks)).to(torch.bfloat16)
    for fmt in (mxq.MXQ_SF_UE5M3, mxq.MXQ_SF_UE4M3):
        for recipe in (mxq.MXQ_4O6, mxq.MXQ_4O6_PZ, mxq.MXQ_ABSMAX):
            check_parity(x, B, fmt, recipe, g)
    check_parity(x, 16, mxq.MXQ_SF_UE5M3, mxq.MXQ_4O6, g, device_g=True)
    check_parity(x, 2, mxq.MXQ_SF_UE5M3, mxq.MXQ_4O6_PZ, g)
    check_parity(x, 32, mxq.MXQ_SF_UE5M3, mxq.MXQ_4O6, g)


@pytest.mark.parametrize("B", [4, 16, 32])
def test_bf16_under_many_tensor_scales(B):
    """The per-launch check of the decode-scale table runs for every tensor scale that is not a power of
    two: many scales, both FP8 formats, bf16 data at the magnitudes the scales imply."""
    rng = np.random.default_rng(5 + B)
    base = _mixed(4 * 256 * max(B, 8) + 3 * 64, 90 + B, torch.float32)
    for i in range(24):
        g = float(np.float32(np.exp(rng.uniform(np.log(1e-6), np.log(30.0)))))
        x = (base * np.float32(g * 300.0)).to(torch.bfloat16)
        fmt = mxq.MXQ_SF_UE4M3 if i % 2 == 0 else mxq.MXQ_SF_UE5M3
        check_parity(x, B, fmt, mxq.MXQ_4O6 if i % 3 else mxq.MXQ_ABSMAX_PZ, g, device_g=bool(i % 2))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("B", [2, 16, 32])
def test_non_finite_elements_stay_inside_their_own_blocks(dtype, B, sweep_mode):
    """NaN and infinite elements are outside the contract: the outputs of a block that holds one are
    unspecified.  What the library does promise is that nothing else suffers: the call returns normally,
    every block WITHOUT such an element still comes out bit for bit as the oracle has it (the oracle sees a
    copy with the offending blocks zeroed), and the next call on the same context is exact again."""
    n = 2 * 256 * 64 + 7 * 64
    x = _mixed(n, 400 + B, torch.float32)
    x = torch.nan_to_num(x, nan=0.0, posinf=0.0, neginf=0.0)
    gen = torch.Generator().manual_seed(9 + B)
    where = torch.randperm(n, generator=gen)[:60]
    x[where[:20]] = float("nan")
    x[where[20:40]] = float("inf")
    x[where[40:]] = float("-inf")
    x = x.to(dtype)
    bad_block = (~torch.isfinite(x.float())).reshape(-1, B).any(dim=1).numpy()
    clean = x.clone().reshape(-1, B)
    clean[torch.from_numpy(bad_block)] = 0
    clean = clean.reshape(-1).contiguous()
    good = ~bad_block
    for fmt in FMTS:
        for recipe in (mxq.MXQ_ABSMAX_PZ, mxq.MXQ_4O6, mxq.MXQ_BRUTE):
            if recipe == mxq.MXQ_BRUTE and fmt == mxq.MXQ_SF_UE5M3 and B == 32:
                continue                                  # the same kernels as UE4M3; keeps the oracle time down
            gc, gs, ge, _ = gpu_quantize(x, B, fmt, recipe, 1.0)
            oc, os_, oe = orc.quantize(inputs.to_numpy_bits(clean), B, fmt, recipe, 1.0, threads=8)
            assert np.array_equal(gs[good], os_[good]), (fmt, recipe)
            assert np.array_equal(gc.reshape(-1, B // 2)[good], oc.reshape(-1, B // 2)[good]), (fmt, recipe)
            assert np.array_equal(ge.view(np.uint32)[good], oe.view(np.uint32)[good]), (fmt, recipe)
    check_parity(clean, B, mxq.MXQ_SF_UE4M3, mxq.MXQ_4O6_PZ, 1.0)


def test_device_resident_global_scale_matches_host_scale():
    x = _mixed(8192, 5, torch.bfloat16)
    for recipe in (mxq.MXQ_ABSMAX, mxq.MXQ_4O6, mxq.MXQ_BRUTE):
        check_parity(x, 16, mxq.MXQ_SF_UE4M3, recipe, 0.0421, device_g=True)


def test_all_zero_and_single_block_tensors():
    for B in BLOCKS:
        z = torch.zeros(B, dtype=torch.float32)
        for fmt in FMTS:
            for recipe in RECIPES:
                check_parity(z, B, fmt, recipe)
        one = inputs.normal(B, B, 0.3)
        check_parity(one, B, mxq.MXQ_SF_UE4M3, mxq.MXQ_4O6)
        check_parity(one, B, mxq.MXQ_SF_UE4M3, mxq.MXQ_BRUTE)


def test_fp4_rounding_boundaries_through_the_kernel():
    # a block whose maximum is 6*S makes the block scale exactly S, so every other element v
    # is divided by S: sweep v across all seven rounding midpoints and one float either side
    S = 0.40625  # 1.625 * 2^-2, a UE4M3 value
    mids = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0], dtype=np.float32) * np.float32(S)
    pts = np.concatenate([np.nextafter(mids, 0), mids, np.nextafter(mids, np.float32(10))]).astype(np.float32)
    pts = np.concatenate([pts, -pts, [0.0, -0.0, 1e-30, -1e-30, 1e-45, -1e-45]]).astype(np.float32)
    blocks = []
    for i in range(0, len(pts), 15):
        chunk = list(pts[i:i + 15])
        chunk += [0.0] * (15 - len(chunk))
        blocks.append(chunk + [6 * S])
    x = torch.tensor(np.array(blocks, dtype=np.float32).reshape(-1))
    check_parity(x, 16, mxq.MXQ_SF_UE4M3, mxq.MXQ_ABSMAX)
    check_parity(x, 16, mxq.MXQ_SF_UE5M3, mxq.MXQ_ABSMAX)


# ------------------------------------------------------------------------------------------------
# Workload-shaped cases (small versions of the benchmark configurations)
# ------------------------------------------------------------------------------------------------
def test_config_normal_1024x1024_fp32_hierarchical():
    x = inputs.normal(1024 * 1024, 1, 1.0, torch.float32)
    xg = x.cuda()
    amax = torch.empty(1, dtype=torch.float32, device="cuda")
    dg = torch.empty(1, dtype=torch.float32, device="cuda")
    mxq.mxq_tensor_amax(xg, xg.numel(), amax, dg)
    torch.cuda.synchronize()
    o_amax = orc.tensor_amax(x.numpy())
    assert float(amax.cpu()[0]) == float(o_amax)
    g = float(orc.global_scale_from_amax(o_amax))
    assert float(dg.cpu()[0]) == g == mxq.mxq_global_scale_from_amax(float(o_amax))
    for recipe in (mxq.MXQ_ABSMAX, mxq.MXQ_4O6, mxq.MXQ_BRUTE):
        check_parity(x, 16, mxq.MXQ_SF_UE4M3, recipe, g, device_g=True)


@pytest.mark.parametrize("B", BLOCKS)
def test_config_weight_student_t_bf16(B):
    x = inputs.student_t(512 * 1024, 5, 0.02, 2, torch.bfloat16)
    for recipe in (mxq.MXQ_ABSMAX, mxq.MXQ_ABSMAX_PZ):
        check_parity(x, B, mxq.MXQ_SF_UE4M3, recipe)
    check_parity(x[: 64 * 1024], B, mxq.MXQ_SF_UE4M3, mxq.MXQ_BRUTE)


def test_config_activation_outlier_columns_bf16():
    x = inputs.outlier_columns(256, 4096, 3, dtype=torch.bfloat16)
    g = float(orc.global_scale_from_amax(orc.tensor_amax(inputs.to_numpy_bits(x))))
    for recipe in (mxq.MXQ_ABSMAX, mxq.MXQ_4O6):
        check_parity(x, 16, mxq.MXQ_SF_UE4M3, recipe, g)
        check_parity(x, 16, mxq.MXQ_SF_UE5M3, recipe, 1.0)


@pytest.mark.parametrize("fmt", FMTS)
def test_config_laplace_fp32_brute_force_with_tensor_scale(fmt, sweep_mode):
    x = inputs.laplace(96 * 1024, 5, torch.float32)
    g = float(orc.global_scale_from_amax(orc.tensor_amax(x.numpy())))
    for B in (2, 4, 8, 16, 32):
        check_parity(x[: 1024 * B], B, fmt, mxq.MXQ_BRUTE, g)


# ------------------------------------------------------------------------------------------------
# The smaller entry points
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_tensor_amax(dtype):
    for n in (1, 7, 8, 1000, 256 * 1024 + 3):
        x = _mixed(max(n, 64), n, dtype)[:n].contiguous()
        xg = x.cuda()
        out = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
        mxq.mxq_tensor_amax(xg, n, out)
        torch.cuda.synchronize()
        assert float(out.cpu()[0]) == float(orc.tensor_amax(inputs.to_numpy_bits(x)))
    # with the tensor scale: the last CTA to finish writes it, whatever the grid size (one CTA to the
    # full persistent grid), and buffers that held something else before are overwritten
    for n in (5, 4096, 1024 * 1024 + 16, 24 * 1024 * 1024 + 5):
        x = (inputs.normal(n, 7 + n, 3.0, torch.float32) * (1.0 + (n % 5))).clamp(-50.0, 50.0).to(dtype).contiguous()
        x[n // 3] = -77.5
        xg = x.cuda()
        out = torch.full((1,), 1.0e30, dtype=torch.float32, device="cuda")
        dg = torch.full((1,), -3.0, dtype=torch.float32, device="cuda")
        for _ in range(3):
            mxq.mxq_tensor_amax(xg, n, out, dg)
        torch.cuda.synchronize()
        want = orc.tensor_amax(inputs.to_numpy_bits(x))
        assert float(out.cpu()[0]) == float(want) == 77.5
        assert float(dg.cpu()[0]) == float(orc.global_scale_from_amax(want))
    z = torch.zeros(4096, dtype=dtype, device="cuda")
    out = torch.full((1,), 5.0, dtype=torch.float32, device="cuda")
    dg = torch.full((1,), 5.0, dtype=torch.float32, device="cuda")
    mxq.mxq_tensor_amax(z, 4096, out, dg)
    assert float(out.cpu()[0]) == 0.0 and float(dg.cpu()[0]) == 1.0      # an all-zero tensor: scale 1


def test_tensor_mse_is_deterministic_and_accurate():
    rng = np.random.default_rng(3)
    for nb in (1, 255, 256, 257, 100_000, 1024 * 256 + 17):
        sse = (rng.random(nb) * np.exp2(rng.integers(-30, 4, nb))).astype(np.float32)
        d = torch.from_numpy(sse).cuda()
        a = float(mxq.tensor_mse(d, nb * 16).cpu()[0])
        b = float(mxq.tensor_mse(d, nb * 16).cpu()[0])
        want = orc.tensor_mse(sse, nb * 16)
        assert a == b
        assert abs(a - want) <= 1e-12 * want


@pytest.mark.parametrize("fmt,g", [(mxq.MXQ_SF_UE4M3, 1.0), (mxq.MXQ_SF_UE5M3, 0.37), (mxq.MXQ_SF_UE8M0, 1.0)])
@pytest.mark.parametrize("B", [2, 4, 16, 64])
def test_dequantize(fmt, g, B):
    n = 256 * 64 * 2 + (B if B < 8 else 0)
    x = _mixed(n, 90 + B, torch.float32)
    codes, scales, _ = orc.quantize(x.numpy(), B, fmt, mxq.MXQ_ABSMAX, g)
    dc, ds = torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda()
    for odt, oid in ((torch.float32, orc.F32), (torch.bfloat16, orc.BF16)):
        out = torch.empty(n, dtype=odt, device="cuda")
        mxq.mxq_dequantize(dc, ds, n, B, fmt, g, out)
        torch.cuda.synchronize()
        want = orc.dequantize(codes, scales, n, B, fmt, g, oid)
        got = inputs.to_numpy_bits(out)
        assert np.array_equal(got.view(np.uint32 if odt == torch.float32 else np.uint16),
                              want.view(np.uint32 if odt == torch.float32 else np.uint16))


def test_sse_output_is_optional_and_launches_are_counted():
    x = inputs.normal(4096, 1).cuda()
    before = mxq.mxq_launch_count()
    codes, scales, sse = mxq.quantize(x, 16, mxq.MXQ_SF_UE4M3, mxq.MXQ_4O6)
    c2, s2, none = mxq.quantize(x, 16, mxq.MXQ_SF_UE4M3, mxq.MXQ_4O6, with_sse=False)
    torch.cuda.synchronize()
    assert none is None and torch.equal(codes, c2) and torch.equal(scales, s2)
    assert mxq.mxq_launch_count() == before + 2


@pytest.mark.parametrize("dtype,B,recipe", [
    (torch.bfloat16, 16, mxq.MXQ_ABSMAX),        # thread-private staging
    (torch.bfloat16, 64, mxq.MXQ_4O6),           # cooperative staging, block walked in parts
    (torch.float32, 32, mxq.MXQ_4O6),            # cooperative staging, whole block in registers
    (torch.float32, 64, mxq.MXQ_ABSMAX_PZ),      # cooperative staging, 16 pieces per chunk
    (torch.bfloat16, 2, mxq.MXQ_BRUTE),
    (torch.float32, 32, mxq.MXQ_BRUTE),
])
def test_repeated_launches_give_the_same_bytes(dtype, B, recipe, sweep_mode):
    """The staging rings hand data from copies to readers (across lanes for the long chunks): a missing
    wait would show as outputs that change from launch to launch.  Sixty launches over several trips of
    the persistent grid, two streams' worth of back-to-back work, all compared with the first."""
    n = 148 * 8 * 256 * max(B, 32) * 2 + 7 * 64          # more chunks than one wave of the grid holds
    x = inputs.student_t(n, 5, 0.02, 321 + B, dtype, "cuda")
    ref = [t.clone() for t in mxq.quantize(x, B, mxq.MXQ_SF_UE4M3, recipe)]
    codes, scales, sse = mxq.alloc_outputs(n, B, "cuda")
    for it in range(60):
        mxq.mxq_quantize_ex(x, n, B, mxq.MXQ_SF_UE4M3, recipe, 1.0, None, codes, scales, sse)
        if it % 20 == 19:
            torch.cuda.synchronize()
            assert torch.equal(codes, ref[0]) and torch.equal(scales, ref[1])
            assert torch.equal(sse.view(torch.int32), ref[2].view(torch.int32))
    check_parity(x[: 4096 * B].cpu(), B, mxq.MXQ_SF_UE4M3, recipe)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("B", BLOCKS)
def test_fused_quantize_mse_equals_quantize_then_tensor_mse(dtype, B, sweep_mode):
    """``mxq_quantize_mse`` (tensor MSE from partial sums formed inside the quantization kernel) against the
    two-call path and the oracle: same codes, scale bytes and block SSEs bit for bit; MSE within 1e-12 of
    the two-call tree and within 1e-6 of the oracle; identical bits when repeated; block SSE output optional.
    Sizes: only a ragged tail (less than one thread's chunk), whole chunks only, and several CTAs plus a tail."""
    cases = [(mxq.MXQ_SF_UE4M3, mxq.MXQ_ABSMAX, 1.0), (mxq.MXQ_SF_UE4M3, mxq.MXQ_4O6_PZ, 0.0131),
             (mxq.MXQ_SF_UE8M0, mxq.MXQ_ABSMAX, 1.0), (mxq.MXQ_SF_UE5M3, mxq.MXQ_BRUTE, 1.0)]
    chunk = max(B, 64)
    for n in (B, 256 * chunk, 3 * 256 * chunk + 5 * 64 + (B if B < 8 else 0)):
        x = _mixed(max(n, 64), 300 + B, dtype)[:n].contiguous()
        xg = x.cuda()
        for fmt, recipe, g in cases:
            codes, scales, sse = mxq.quantize(xg, B, fmt, recipe, g)
            mse2 = mxq.tensor_mse(sse, n)
            c1, s1, e1 = mxq.alloc_outputs(n, B, xg.device)
            ws = torch.full((mxq.mxq_tensor_mse_workspace_bytes(n // B) // 8,), float("nan"), dtype=torch.float64, device="cuda")
            m1 = torch.empty(1, dtype=torch.float64, device="cuda")
            mxq.mxq_quantize_mse(xg, n, B, fmt, recipe, g, None, c1, s1, e1, m1, ws)
            m2 = torch.empty(1, dtype=torch.float64, device="cuda")
            c2, s2, _ = mxq.alloc_outputs(n, B, xg.device, with_sse=False)
            mxq.mxq_quantize_mse(xg, n, B, fmt, recipe, g, None, c2, s2, None, m2, ws)       # no SSE output
            torch.cuda.synchronize()
            assert torch.equal(codes, c1) and torch.equal(codes, c2)
            assert torch.equal(scales, s1) and torch.equal(scales, s2)
            assert torch.equal(sse.view(torch.int32), e1.view(torch.int32))
            a, b, c = float(mse2.cpu()[0]), float(m1.cpu()[0]), float(m2.cpu()[0])
            assert b == c                                            # deterministic
            assert abs(a - b) <= 1e-12 * abs(a) + 1e-300, (n, fmt, recipe, a, b)
            om = orc.tensor_mse(sse.cpu().numpy(), n)
            assert abs(b - om) <= MSE_RTOL * abs(om) + 1e-300


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("B", BLOCKS)
def test_multi_tensor_launch_equals_one_launch_per_tensor(dtype, B):
    """``mxq_quantize_batch`` over tensors of very different sizes (one 64-element tensor, sizes that end in the
    middle of a warp's row of chunks, one that spans many CTAs) against ``mxq_quantize_ex`` on each tensor and,
    for the first recipe, against the oracle: every output byte identical, the optional SSE output included."""
    sizes = [64, 64 * 37, 64 * 1024 + 64, 64, 64 * 5000, 64 * 33, 64 * 20000 + 64 * 7]
    xs = [_mixed(n, 400 + i + B, dtype).cuda() for i, n in enumerate(sizes)]
    dt = mxq.MXQ_F32 if dtype == torch.float32 else mxq.MXQ_BF16
    cases = [(mxq.MXQ_SF_UE4M3, mxq.MXQ_ABSMAX, 1.0), (mxq.MXQ_SF_UE4M3, mxq.MXQ_4O6_PZ, 1.0),
             (mxq.MXQ_SF_UE5M3, mxq.MXQ_4O6, 0.0131), (mxq.MXQ_SF_UE8M0, mxq.MXQ_ABSMAX_OCP, 1.0)]
    for ci, (fmt, recipe, g) in enumerate(cases):
        outs = [mxq.alloc_outputs(x.numel(), B, x.device, with_sse=(i % 3 != 1)) for i, x in enumerate(xs)]
        for c, s_, e in outs:
            c.fill_(0xAA); s_.fill_(0xAA)
        h, d = mxq.make_tensor_descs([(x, c, s_, e) for x, (c, s_, e) in zip(xs, outs)])
        mxq.mxq_quantize_batch(h, d, len(xs), dt, B, fmt, recipe, g)
        torch.cuda.synchronize()
        for i, (x, (c, s_, e)) in enumerate(zip(xs, outs)):
            c1, s1, e1 = mxq.quantize(x, B, fmt, recipe, g)
            assert torch.equal(c, c1) and torch.equal(s_, s1), (i, fmt, recipe)
            if e is not None:
                assert torch.equal(e.view(torch.int32), e1.view(torch.int32)), (i, fmt, recipe)
            if ci == 0:
                oc, os_, oe = orc.quantize(inputs.to_numpy_bits(x), B, fmt, recipe, g)
                assert np.array_equal(c.cpu().numpy(), oc) and np.array_equal(s_.cpu().numpy(), os_)
    # argument checks happen on the host, before any launch
    with pytest.raises(mxq.MxqError):
        mxq.mxq_quantize_batch(h, d, len(xs), dt, B, mxq.MXQ_SF_UE4M3, mxq.MXQ_BRUTE)
    bad = mxq.alloc_outputs(96, B, xs[0].device)
    hb, db = mxq.make_tensor_descs([(xs[2][:96], *bad)])
    with pytest.raises(mxq.MxqError):
        mxq.mxq_quantize_batch(hb, db, 1, dt, B, mxq.MXQ_SF_UE4M3, mxq.MXQ_ABSMAX)      # 96 is not a multiple of 64


def test_multi_tensor_launch_with_hundreds_of_small_tensors():
    """777 tensors of 256 to 2560 elements in one launch (the prefix sums over the tensor list span several
    warps of the scan; most tensors end inside a warp's row), and the largest list the entry point takes.
    Lengths are multiples of 256 so that every slice of the shared output buffers is 16-byte aligned."""
    gen = torch.Generator().manual_seed(5)
    B = 16
    for count in (777, 1024):
        sizes = (256 * torch.randint(1, 11, (count,), generator=gen)).tolist()
        big = _mixed(sum(sizes), 600 + count, torch.bfloat16).cuda()
        xs, o = [], 0
        for n in sizes:
            xs.append(big[o:o + n])
            o += n
        codes = torch.zeros(sum(sizes) // 2, dtype=torch.uint8, device="cuda")
        scales = torch.zeros(sum(sizes) // B, dtype=torch.uint8, device="cuda")
        sse = torch.zeros(sum(sizes) // B, dtype=torch.float32, device="cuda")
        items, o = [], 0
        for n, x in zip(sizes, xs):
            items.append((x, codes[o // 2:(o + n) // 2], scales[o // B:(o + n) // B], sse[o // B:(o + n) // B]))
            o += n
        h, d = mxq.make_tensor_descs(items)
        mxq.mxq_quantize_batch(h, d, count, mxq.MXQ_BF16, B, mxq.MXQ_SF_UE4M3, mxq.MXQ_4O6)
        # blocks never straddle tensors here (every length is a multiple of 64), so the whole buffer quantized as
        # one tensor must give the same bytes
        c1, s1, e1 = mxq.quantize(big, B, mxq.MXQ_SF_UE4M3, mxq.MXQ_4O6)
        torch.cuda.synchronize()
        assert torch.equal(codes, c1) and torch.equal(scales, s1) and torch.equal(sse.view(torch.int32), e1.view(torch.int32))
    with pytest.raises(mxq.MxqError):
        mxq.mxq_quantize_batch(h, d, 1025, mxq.MXQ_BF16, B, mxq.MXQ_SF_UE4M3, mxq.MXQ_4O6)
