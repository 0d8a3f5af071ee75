"""One rank of tests/test_gpu_streams.py::test_row_sharded_hierarchical_quantize_as_two_ranks: quantizes its
rows of a seeded tensor with ``dist.sharded_hierarchical_quantize`` and writes its outputs to a file."""
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2605_08565_b200 import binding as mxq  # noqa: E402
from paper_2605_08565_b200 import dist, inputs  # noqa: E402


def main():
    rows, cols, B, recipe, out_dir = int(sys.argv[1]), int(sys.argv[2]), int(sys.argv[3]), int(sys.argv[4]), sys.argv[5]
    torch.cuda.set_device(0)
    rank, _, world = dist.init("gloo")
    x = inputs.outlier_columns(rows, cols, 11, dtype=torch.bfloat16).view(rows, cols)
    r0, r1 = dist.row_shard(rows, rank, world)
    x_local = x[r0:r1].contiguous().reshape(-1).cuda()
    codes, scales, sse, dg, mse = dist.sharded_hierarchical_quantize(x_local, rows * cols, B, mxq.MXQ_SF_UE4M3, recipe)
    local_sum = mxq.tensor_mse(sse, 1)
    torch.cuda.synchronize()
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), codes=codes.cpu().numpy(), scales=scales.cpu().numpy(),
             sse=sse.cpu().numpy(), g=dg.cpu().numpy()[0], mse=np.float64(mse), local_sum=local_sum.cpu().numpy()[0])
    dist.barrier()
    dist.shutdown()


if __name__ == "__main__":
    main()
