"""Host-side pieces of bench.py that need no GPU: the reference arm must run without touching
the CUDA library, the scattered support must be a valid assignment, the sampled pack blocks of the
parity check must be valid and include the ends."""
import json
import os
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from oracle import design as od  # noqa: E402


def test_reference_arm_runs_without_importing_the_cuda_package():
    """`bench.py --impl reference` times the oracle alone: its bits and weights come from
    oracle/design.py and no module of the package (hence no libagc.so) is loaded."""
    prog = ("import sys, runpy\n"
            "sys.argv = ['bench.py', '--impl', 'reference', '--workload', 'cfg1', '--steps', '2', '--warmup', '1']\n"
            "runpy.run_path('bench.py', run_name='__main__')\n"
            "bad = [m for m in sys.modules if m.startswith('paper_2605_15890_b200')]\n"
            "assert not bad, bad\n")
    out = subprocess.run([sys.executable, "-c", prog], cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["gpu_launches"] == 0 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["host_cores"] >= 1
    assert line["cpu_baseline"]["encode"]["value"] > 0 and line["cpu_baseline"]["decode"]["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0


def test_reference_arm_code_is_unbiased_on_the_configurations_support():
    for name in ("cfg1", "cfg2", "cfg3"):
        wl = bench.workload(name)
        (rp, ci, a, w), bits = bench.oracle_build_code(wl, 512)
        assert bits.sum() == (wl.z_tot if wl.bits is None else int(np.sum(wl.bits)))
        A = od.csr_to_dense(rp, ci, a.astype(np.float64), wl.k)
        assert od.unbiasedness_residual(A, w.astype(np.float64), wl.p) < 1e-5
        sup = od.cyclic_support(wl.n, wl.k, wl.s)
        for i in range(wl.n):
            assert set(ci[rp[i]:rp[i + 1]]) <= set(sup[i])


def test_scattered_support_is_a_valid_assignment():
    for name in ("cfg3", "cfg5", "cfg1"):
        wl = bench.workload(name)
        sup = bench.workload_support(wl, "scattered")
        assert len(sup) == wl.n
        held = set()
        for cols in sup:
            assert cols == sorted(set(cols)) and 1 <= len(cols) <= wl.s and all(0 <= j < wl.k for j in cols)
            held |= set(cols)
        assert held == set(range(wl.k))
        assert sup == bench.workload_support(wl, "scattered")       # seeded
        assert sup != bench.workload_support(wl, "cyclic")


def test_parity_sample_blocks():
    wl = bench.workload("cfg3")
    nblk = (wl.d + 511) // 512
    qs = bench.parity_blocks(wl, nblk)
    assert len(qs) == 64 and qs == sorted(set(qs)) and qs[0] == 0 and qs[-1] == nblk - 1
    assert all(0 <= q < nblk for q in qs)
    small = bench.workload("cfg4")
    assert bench.parity_blocks(small, 8) == list(range(8))
    assert bench.sample_size(wl, 10) == 5120 and bench.sample_size(small, 100) == small.d
