"""GPU tests of the entry points and launch paths that the parity matrix does not reach: the plain
``mxq_quantize`` call (float32, legacy default stream), the whole path on an explicit non-default
stream ordered against a producer on another stream, and the row-sharded hierarchical wrapper run
as two ranks."""
import os
import socket
import subprocess
import sys

import numpy as np
import pytest
import torch

from oracle import mxq_oracle as orc
from paper_2605_08565_b200 import binding as mxq
from paper_2605_08565_b200 import inputs

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.mark.parametrize("fmt,recipe,B,g", [
    (mxq.MXQ_SF_UE4M3, mxq.MXQ_ABSMAX, 16, 1.0), (mxq.MXQ_SF_UE4M3, mxq.MXQ_4O6_PZ, 8, 0.0131),
    (mxq.MXQ_SF_UE8M0, mxq.MXQ_ABSMAX, 32, 1.0), (mxq.MXQ_SF_UE5M3, mxq.MXQ_BRUTE, 4, 0.37),
    (mxq.MXQ_SF_UE4M3, mxq.MXQ_BRUTE_PZ, 64, 1.0)])
def test_mxq_quantize_itself_on_the_default_stream(fmt, recipe, B, g):
    """`mxq_quantize` (float32 input, stream 0) against the oracle: codes, scale bytes, block SSE bit for
    bit, tensor MSE within 1e-6."""
    n = 3 * 256 * max(B, 16) + 7 * B
    x = (inputs.adversarial(n, 90 + B, torch.float32) * 0.5 + inputs.normal(n, 91 + B, 0.01)).contiguous()
    xg = x.cuda()
    codes, scales, sse = mxq.alloc_outputs(n, B, xg.device)
    torch.cuda.synchronize()
    mxq.mxq_quantize(xg, n, B, fmt, recipe, g, codes, scales, sse)     # legacy default stream
    mse = torch.empty(1, dtype=torch.float64, device="cuda")
    ws = torch.empty(mxq.mxq_tensor_mse_workspace_bytes(n // B) // 8, dtype=torch.float64, device="cuda")
    mxq.mxq_tensor_mse(sse, n // B, n, mse, ws, stream=torch.cuda.default_stream())
    torch.cuda.synchronize()
    oc, os_, oe = orc.quantize(x.numpy(), B, fmt, recipe, g, threads=8)
    assert np.array_equal(scales.cpu().numpy(), os_)
    assert np.array_equal(codes.cpu().numpy(), oc)
    assert np.array_equal(sse.cpu().numpy().view(np.uint32), oe.view(np.uint32))
    om = orc.tensor_mse(oe, n)
    assert abs(float(mse.cpu()[0]) - om) <= 1e-6 * om


def test_whole_path_on_an_explicit_stream_ordered_after_a_producer_on_another_stream():
    """The input is produced on stream A behind a long delay; stream B waits for A's event and then runs
    tensor abs-max -> quantize -> tensor MSE -> de-quantize, every call given stream B explicitly.  If a
    call ran on another stream than the one it was handed, it would read the still-zero input (or
    unfinished outputs) and the comparison with the oracle would fail."""
    n, B = 1 << 20, 16
    src = inputs.student_t(n, 5, 0.02, 7, torch.bfloat16).cuda()
    x = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    codes, scales, sse = mxq.alloc_outputs(n, B, x.device)
    amax = torch.empty(1, dtype=torch.float32, device="cuda")
    dg = torch.empty(1, dtype=torch.float32, device="cuda")
    mse = torch.full((1,), -1.0, dtype=torch.float64, device="cuda")
    ws = torch.empty(mxq.mxq_tensor_mse_workspace_bytes(n // B) // 8, dtype=torch.float64, device="cuda")
    xh = torch.zeros(n, dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    a, b = torch.cuda.Stream(), torch.cuda.Stream()
    ready = torch.cuda.Event()
    with torch.cuda.stream(a):
        torch.cuda._sleep(60_000_000)          # tens of milliseconds: the consumer is enqueued long before this ends
        x.copy_(src, non_blocking=True)
        ready.record(a)
    b.wait_event(ready)
    mxq.mxq_tensor_amax(x, n, amax, dg, stream=b)
    mxq.mxq_quantize_ex(x, n, B, mxq.MXQ_SF_UE4M3, mxq.MXQ_4O6, 1.0, dg, codes, scales, sse, stream=b)
    mxq.mxq_tensor_mse(sse, n // B, n, mse, ws, stream=b)
    mxq.mxq_dequantize_ex(codes, scales, n, B, mxq.MXQ_SF_UE4M3, 1.0, dg, xh, stream=b)   # g stays on the device
    b.synchronize()
    g = float(dg.cpu()[0])
    xb = inputs.to_numpy_bits(src)
    og = float(orc.global_scale_from_amax(orc.tensor_amax(xb)))
    assert g == og and g != 1.0
    oc, os_, oe = orc.quantize(xb, B, orc.UE4M3, orc.R4O6, og, threads=8)
    assert np.array_equal(scales.cpu().numpy(), os_)
    assert np.array_equal(codes.cpu().numpy(), oc)
    assert np.array_equal(sse.cpu().numpy().view(np.uint32), oe.view(np.uint32))
    om = orc.tensor_mse(oe, n)
    assert abs(float(mse.cpu()[0]) - om) <= 1e-6 * om
    want = orc.dequantize(oc, os_, n, B, orc.UE4M3, og, orc.F32)
    assert np.array_equal(xh.cpu().numpy().view(np.uint32), want.view(np.uint32))
    xh2 = torch.empty_like(xh)
    mxq.mxq_dequantize(codes, scales, n, B, mxq.MXQ_SF_UE4M3, g, xh2, stream=b)               # host g: same bits
    b.synchronize()
    assert torch.equal(xh.view(torch.int32), xh2.view(torch.int32))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("recipe", [mxq.MXQ_ABSMAX, mxq.MXQ_4O6])
def test_row_sharded_hierarchical_quantize_as_two_ranks(tmp_path, recipe):
    """A 384 x 4096 bf16 tensor with outlier columns is split by rows over two ranks (two processes, gloo,
    both on cuda:0; no kernel of one rank waits for the other).  Each runs
    ``dist.sharded_hierarchical_quantize`` on its rows; the concatenated codes, scale bytes and block SSE,
    the shared tensor scale and the tensor MSE must equal the oracle's result on the whole tensor."""
    rows, cols, B = 384, 4096, 16
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK="0", WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.join(HERE, "sharded_worker.py"), str(rows), str(cols),
                                       str(B), str(recipe), str(tmp_path)], env=env, cwd=os.path.dirname(HERE)))
    for p in procs:
        assert p.wait(timeout=300) == 0
    x = inputs.outlier_columns(rows, cols, 11, dtype=torch.bfloat16)
    xb = inputs.to_numpy_bits(x)
    g = float(orc.global_scale_from_amax(orc.tensor_amax(xb)))
    oc, os_, oe = orc.quantize(xb, B, orc.UE4M3, recipe, g, threads=8)
    om = orc.tensor_mse(oe, rows * cols)
    parts = [np.load(os.path.join(tmp_path, f"rank{r}.npz")) for r in range(2)]
    assert all(float(p["g"]) == g for p in parts)
    assert np.array_equal(np.concatenate([p["codes"] for p in parts]), oc)
    assert np.array_equal(np.concatenate([p["scales"] for p in parts]), os_)
    assert np.array_equal(np.concatenate([p["sse"] for p in parts]).view(np.uint32), oe.view(np.uint32))
    for p in parts:
        assert abs(float(p["mse"]) - om) <= 1e-6 * om
    assert float(parts[0]["mse"]) == float(parts[1]["mse"])        # rank-order sum: the same bits on every rank
    # the sharded MSE is exactly (sum of the two ranks' binary64 tree sums) / n
    s = [float(p["local_sum"]) for p in parts]
    assert float(parts[0]["mse"]) == (s[0] + s[1]) / (rows * cols)


def test_entry_points_called_from_four_host_threads_at_once():
    """Four host threads, each with its own stream and tensors, run abs-max -> quantize + MSE -> de-quantize
    sixteen times over while a fifth flips the process-wide brute-force option: every thread must get the
    bytes that a quiet single-threaded run gets (the header's statement on threads)."""
    import threading
    n, B = 1 << 18, 16
    xs = [inputs.student_t(n, 5, 0.02, 50 + i, torch.bfloat16).cuda() for i in range(4)]
    recipes = [mxq.MXQ_ABSMAX, mxq.MXQ_4O6, mxq.MXQ_BRUTE, mxq.MXQ_ABSMAX_PZ]
    want = []
    for x, r in zip(xs, recipes):
        c, s_, e = mxq.quantize(x, B, mxq.MXQ_SF_UE4M3, r)
        want.append((c.clone(), s_.clone(), e.clone(), mxq.tensor_mse(e, n).clone()))
    torch.cuda.synchronize()
    errors = []
    stop = threading.Event()

    def worker(i):
        try:
            torch.cuda.set_device(0)
            st = torch.cuda.Stream()
            c, s_, e = mxq.alloc_outputs(n, B, xs[i].device)
            m = torch.empty(1, dtype=torch.float64, device="cuda")
            ws = torch.empty(1024, dtype=torch.float64, device="cuda")
            for _ in range(16):
                mxq.mxq_quantize_mse(xs[i], n, B, mxq.MXQ_SF_UE4M3, recipes[i], 1.0, None, c, s_, e, m, ws, stream=st)
                st.synchronize()
                ok = (torch.equal(c, want[i][0]) and torch.equal(s_, want[i][1])
                      and torch.equal(e.view(torch.int32), want[i][2].view(torch.int32))
                      and abs(float(m.cpu()[0]) - float(want[i][3].cpu()[0])) <= 1e-12 * float(want[i][3].cpu()[0]))
                if not ok:
                    errors.append(i)
        except Exception as ex:      # noqa: BLE001
            errors.append((i, repr(ex)))

    def flipper():
        v = 0
        while not stop.is_set():
            v ^= 1
            mxq.mxq_set_option(mxq.MXQ_OPT_BRUTE_PRUNE, v)

    ths = [threading.Thread(target=worker, args=(i,)) for i in range(4)]
    fl = threading.Thread(target=flipper)
    fl.start()
    for t in ths:
        t.start()
    for t in ths:
        t.join()
    stop.set()
    fl.join()
    mxq.mxq_set_option(mxq.MXQ_OPT_BRUTE_PRUNE, 0)
    assert not errors, errors
