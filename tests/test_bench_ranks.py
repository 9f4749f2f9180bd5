"""The multi-rank path of bench.py without GPUs: two gloo ranks on 127.0.0.1 run the same rendezvous, barrier,
max-over-ranks and rank-0 reporting code the NCCL run uses (replicas only: no collective on the data path), and
the reference arm prints from rank 0 only."""
import json
import os
import subprocess
import sys

import synth_inputs as si

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _torchrun(extra, nproc=2, port=29641):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={nproc}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py")] + extra
    env = dict(os.environ, OMP_NUM_THREADS="2")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)


def test_two_ranks_aggregate_to_one_line():
    r = _torchrun(["--gpus", "2", "--steps", "4", "--selftest-dist"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout                         # rank 0 alone reports
    d = json.loads(lines[0])
    flops = si.conv_flops(**{k: v for k, v in si.CONFIGS["cfg3_bf16_192"].items() if k in "N Cin Cout T H W k".split()})
    assert d["n_gpus"] == 2 and d["scaling"] == "weak"
    assert abs(d["ms_per_step"] - 1.25) < 1e-9                # the slower rank's time
    assert abs(d["value"] - 2 * flops / 1.25e-3 / 1e12) < 1e-6 * d["value"]


def test_single_process_selftest():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--selftest-dist", "--steps", "2"], cwd=ROOT,
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    d = json.loads(r.stdout.strip().splitlines()[-1])
    assert d["n_gpus"] == 1 and abs(d["ms_per_step"] - 1.0) < 1e-9


def test_gpus_flag_starts_its_own_ranks():
    """`python bench.py --gpus 2` without torchrun: the script starts two ranks itself (here on CPU, gloo, through the
    same self-test as above) and rank 0 prints the one line with n_gpus = 2."""
    env = dict(os.environ, OMP_NUM_THREADS="2")
    for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK"):
        env.pop(k, None)
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "4", "--selftest-dist"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and abs(d["ms_per_step"] - 1.25) < 1e-9


def test_useful_tap_fraction_matches_the_interval_algebra():
    """The bench's useful-FLOP count of a first-chunk call: the (output frame, temporal tap) pairs whose source frame
    exists, 1/3, 3/6 and 9/12 of them at T = 1, 2, 4 with kt = 3 and no history (the worked cases of Eq. (4)), all of
    them with a full cache; and the same count from the oracle's interval routine."""
    sys.path.insert(0, ROOT)
    import bench
    import oracle
    assert abs(bench.useful_tap_fraction(1, 3, 0) - 1 / 3) < 1e-12
    assert abs(bench.useful_tap_fraction(2, 3, 0) - 3 / 6) < 1e-12
    assert abs(bench.useful_tap_fraction(4, 3, 0) - 9 / 12) < 1e-12
    assert bench.useful_tap_fraction(4, 3, 2) == 1.0 and bench.useful_tap_fraction(3, 1, 0) == 1.0
    for kt in (1, 2, 3):
        for cf in range(kt):
            for T in (1, 2, 4, 5):
                _, taps = oracle.tap_intervals(kt, cf, T)
                pairs = sum(max(0, oh - ol) for (_, ol, oh, _, _) in taps)
                assert abs(bench.useful_tap_fraction(T, kt, cf) - pairs / (T * kt)) < 1e-12
