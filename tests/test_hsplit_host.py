"""Height-split of a layer across ranks, host logic only (no GPU): the row partition, the halo plan, the
neighbour exchange over gloo with 2 and 3 ranks, slab assembly and the cache slabs across streamed chunks.  The
layer inside is the oracle, so a band must equal the same rows of the unsplit oracle exactly."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import oracle
from _hsplit_cpu import OracleConv, TorchRowOps, case_tensors
from paper_2609_31938_b200.hsplit import HSplitCausalConv3d, band, forward_all_local, halo_plan

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("H,world", [(16, 1), (16, 4), (17, 4), (352, 8), (5, 5), (7, 3)])
def test_bands_partition_the_rows(H, world):
    edges = [band(H, world, r) for r in range(world)]
    assert edges[0][0] == 0 and edges[-1][1] == H
    assert all(a[1] == b[0] for a, b in zip(edges, edges[1:]))
    sizes = [b - a for a, b in edges]
    assert max(sizes) - min(sizes) <= 1 and sorted(sizes, reverse=True) == sizes


def test_halo_plan_follows_the_taps():
    p = halo_plan(352, 2, 1, kh=3, pad_h=1)
    assert (p.top, p.bot, p.r0, p.r1, p.slab_rows, p.up, p.down) == (1, 1, 176, 352, 178, 0, None)
    p = halo_plan(64, 4, 0, kh=5, pad_h=4, dil_h=2)                    # reach 8: 4 rows on either side
    assert (p.top, p.bot, p.up, p.down) == (4, 4, None, 1)
    p = halo_plan(64, 4, 2, kh=1, pad_h=0)                             # no taps in h: nothing to exchange
    assert (p.top, p.bot, p.slab_rows) == (0, 0, 16)
    with pytest.raises(ValueError):
        halo_plan(64, 4, 4, kh=3, pad_h=1)                             # rank out of range
    with pytest.raises(ValueError):
        halo_plan(64, 4, 0, kh=3, pad_h=0)                             # the layer would shrink the height
    with pytest.raises(ValueError):
        halo_plan(8, 4, 0, kh=3, pad_h=1, dil_h=3)                     # bands of 2 rows, halo of 3


CASES = [
    # k, dilation, pad, stride, H, W, worlds
    ((3, 3, 3), (1, 1, 1), (1, 1, 1), (1, 1, 1), 13, 6, (1, 2, 3)),
    ((3, 5, 3), (1, 2, 1), (1, 4, 1), (1, 1, 1), 29, 5, (2, 3)),      # dilated 5 taps in h: halo of 4 rows
    ((2, 1, 3), (2, 1, 1), (1, 0, 1), (1, 1, 1), 12, 4, (2, 4)),      # no taps in h: nothing exchanged; d_t = 2
    ((3, 3, 3), (1, 1, 1), (1, 1, 1), (2, 1, 2), 11, 8, (2,)),        # stride in t and w is the layer's own
]


@pytest.mark.parametrize("k,dil,pad,stride,H,W,worlds", CASES)
def test_bands_equal_the_unsplit_layer(k, dil, pad, stride, H, W, worlds):
    N, Cin, Cout, T = 2, 3, 4, 3
    x, w, b = case_tensors(11, N, Cin, Cout, 2 * T, H, W, k)
    kw = dict(stride=(1, stride[2]), pad=(pad[1], pad[2]), dil=(dil[1], dil[2]), dil_t=dil[0], stride_t=stride[0])
    ref0, c0 = oracle.forward_general(x[:, :, :T], None, w, b, **kw)
    ref1, _ = oracle.forward_general(x[:, :, T:], c0, w, b, **kw)
    for world in worlds:
        layers = [HSplitCausalConv3d(w, b, H, r, world, ops=TorchRowOps(), transport=None,
                                     conv=OracleConv(w, b, pad[2], stride, dil), stride=stride, dilation=dil, pad=pad)
                  for r in range(world)]
        caches, got = None, []
        for c in range(2):
            xs = [torch.from_numpy(np.ascontiguousarray(x[:, :, c * T:(c + 1) * T, l.plan.r0:l.plan.r1])) for l in layers]
            outs, caches = forward_all_local(layers, xs, caches)
            assert all(cs.shape[-2] == l.plan.slab_rows for cs, l in zip(caches, layers))
            got.append(torch.cat(outs, dim=3).numpy())
        assert np.array_equal(got[0], ref0) and np.array_equal(got[1], ref1)


def test_stride_in_h_is_refused():
    x, w, b = case_tensors(1, 1, 2, 2, 1, 8, 8, (3, 3, 3))
    with pytest.raises(ValueError):
        HSplitCausalConv3d(w, b, 8, 0, 2, ops=TorchRowOps(), conv=lambda *a: None, stride=(1, 2, 1))


@pytest.mark.parametrize("world", [2, 3])
def test_neighbour_exchange_over_gloo(world):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={world}", "--master-addr",
           "127.0.0.1", "--master-port", str(29650 + world), os.path.join(ROOT, "tests", "_hsplit_worker.py")]
    r = subprocess.run(cmd, cwd=ROOT, env=dict(os.environ, OMP_NUM_THREADS="2"), capture_output=True, text=True,
                       timeout=600)
    assert r.returncode == 0, (r.stdout[-1500:], r.stderr[-3000:])
    assert f"HSPLIT_OK world={world}" in r.stdout


def test_ring_frame_runs_wrap_around():
    """Slots slot0 .. slot0+T-1 (mod F) as contiguous runs: the row copies of a ring's halo rows go run by run."""
    from paper_2609_31938_b200.hsplit import _frame_runs
    assert _frame_runs(0, 4, 6) == [(0, 4, 0)]
    assert _frame_runs(4, 4, 6) == [(4, 2, 0), (0, 2, 2)]
    assert _frame_runs(5, 1, 6) == [(5, 1, 0)]
    assert _frame_runs(7, 3, 6) == [(1, 3, 0)]                    # a slot given beyond F is taken mod F
    for F in (3, 5, 6):
        for slot0 in range(F):
            for T in range(1, F + 1):
                runs = _frame_runs(slot0, T, F)
                slots = [s + i for s, n, _ in runs for i in range(n)]
                assert slots == [(slot0 + t) % F for t in range(T)]
                assert [t0 for _, _, t0 in runs] == [0] + ([runs[0][1]] if len(runs) == 2 else [])
