"""One gloo rank of the height-split test (launched by torch.distributed.run): computes its band of two streamed
chunks with the neighbour exchange over the process group, the layer itself by the oracle; rank 0 gathers the
bands and compares them with the unsplit oracle."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import oracle  # noqa: E402
from _hsplit_cpu import OracleConv, TorchRowOps, case_tensors  # noqa: E402
from paper_2609_31938_b200.hsplit import DistTransport, HSplitCausalConv3d, band  # noqa: E402


def main():
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    k, dil, pad = (3, 5, 3), (1, 2, 1), (1, 4, 1)          # halo: 4 rows on either side
    N, Cin, Cout, T, H, W = 1, 3, 4, 2, 37, 8
    x, w, b = case_tensors(5, N, Cin, Cout, 2 * T, H, W, k)
    layer = HSplitCausalConv3d(w, b, H, rank, world, transport=DistTransport(), ops=TorchRowOps(),
                               conv=OracleConv(w, b, pad[2], dilation=dil), dilation=dil, pad=pad)
    r0, r1 = band(H, world, rank)
    cache, outs = None, []
    for c in range(2):
        xb = torch.from_numpy(np.ascontiguousarray(x[:, :, c * T:(c + 1) * T, r0:r1]))
        o, cache = layer(xb, cache)
        outs.append(o)
    mine = torch.cat(outs, dim=2).contiguous()
    sizes = [band(H, world, r)[1] - band(H, world, r)[0] for r in range(world)]
    if rank == 0:
        parts = [mine] + [torch.empty((N, Cout, 2 * T, s, mine.shape[-1]), dtype=torch.float64) for s in sizes[1:]]
        for r in range(1, world):
            dist.recv(parts[r], r)
        got = torch.cat(parts, dim=3).numpy()
        ref, _ = oracle.forward_general(x, None, w, b, pad=(pad[1], pad[2]), dil=(dil[1], dil[2]), dil_t=dil[0])
        assert got.shape == ref.shape, (got.shape, ref.shape)
        assert np.array_equal(got, ref), float(np.abs(got - ref).max())
        print(f"HSPLIT_OK world={world} rows={sizes}")
    else:
        dist.send(mine, 0)
    dist.barrier()
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
