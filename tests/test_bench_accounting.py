"""The roofline numerator: bytes a step must move, per element and worker, for the five workloads.

g is read (4 B), x read and written (8 B), m read and written when there is momentum (8 B), e read and
written only where it is touched: everywhere but the update-selected blocks on a plain step (fraction
1 - 1/R1), and on a reset step also on the reset-selected ones (1 - (1/R1)(1 - 1/R2)).
"""
import pytest

import bench
from paper_2007_13221_b200 import synth


@pytest.mark.parametrize("cfg,per_elt,gb_per_step", [(1, 18.125, 0.1520), (2, 27.751, 7.9365), (3, 27.969, 11.4370),
                                                     (4, 27.992, 5.7232), (5, 27.875, 74.7373)])
def test_algorithmic_bytes_per_workload(cfg, per_elt, gb_per_step):
    w = synth.CONFIGS[cfg]
    mean = bench.mean_algorithmic_bytes(w, 1, w.H)           # one reset in H steps
    assert abs(mean / (w.n_workers * w.d) - per_elt) < 5e-4
    assert abs(mean / 1e9 - gb_per_step) < 5e-4 * gb_per_step + 1e-4


def test_variants_change_the_count_as_stated():
    w = synth.CONFIGS[2]
    assert bench.algorithmic_bytes(w, 1.0) == w.n_workers * w.d * 28
    bench.NO_ERROR_ARRAY = True
    try:
        assert bench.algorithmic_bytes(w, 1.0) == w.n_workers * w.d * 20
    finally:
        bench.NO_ERROR_ARRAY = False
    from dataclasses import replace
    assert bench.expected_e_fraction(replace(w, R1=0), False) == 1.0      # C2 = 0: e touched everywhere
    assert bench.expected_e_fraction(replace(w, R1=1, R2=1), True) == 1.0
    assert bench.expected_e_fraction(replace(w, R1=1), False) == 0.0      # everything synchronized: e idle


def test_overall_compression_ratio_matches_the_papers_formula_and_table():
    """Section 5.1: R_C = 1 / (1/R_C2 + 1/(R_C1 H)); Appendix C lists (R_C2, R_C1, H) = (512, 16, 32) for an
    overall ratio of 256 and (2048, 32, 64) for 1024 (R1 here is the paper's R_C2, R2 its R_C1)."""
    import os
    from dataclasses import replace
    w = synth.CONFIGS[2]
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "table3_cser_hyperparameters.txt")
    rows = [tuple(int(v) for v in ln.split()) for ln in open(path) if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 6
    for overall, R1, R2, H in rows:
        assert abs(replace(w, R1=R1, R2=R2, H=H).overall_ratio - overall) < 1e-9, (overall, R1, R2, H)
    assert abs(w.overall_ratio - 1.0 / (1 / 32 + 1 / 256)) < 1e-12
    assert replace(w, R1=0, R2=4, H=2).overall_ratio == 8.0            # CSER-PL: only the reset is exchanged


def test_reference_arm_prints_the_contract_line_and_says_what_it_measured():
    """`bench.py --impl reference` times the oracle on the host: one JSON line with the same metric, unit and
    config object as the GPU arm's, `impl: reference`, a `cpu_baseline` describing the run, an `e2e` object
    with no copies, and, when only a slab of the vector was timed, the measured slab and wall time beside the
    extrapolated value."""
    import json
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--config", "1",
                          "--steps", "2", "--warmup", "3"], capture_output=True, text=True, timeout=600,
                         env={**os.environ, "CUDA_VISIBLE_DEVICES": ""})
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    w = synth.CONFIGS[1]
    assert line["impl"] == "reference" and line["metric"] == bench.METRIC and line["unit"] == bench.UNIT
    assert line["config"] == bench.config_of(w, 1)
    assert line["higher_is_better"] is True and line["vs_baseline"] is None and line["steps"] == 2
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] == 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    # workload 1 runs real full-d steps: nothing is extrapolated, and value is the measured rate
    assert line["extrapolated"] is False and line["measured_cols"] == w.d
    assert abs(line["value"] - 1e3 / line["ms_per_step"]) < 1e-9 * line["value"] + 1e-12
    # the larger workloads time a slab beyond the host caches and scale by columns
    cols = bench.oracle_sample_cols(synth.CONFIGS[5])
    assert cols % synth.CONFIGS[5].block_size == 0 and 8 * synth.CONFIGS[5].n_workers * cols >= 256 << 20
    assert bench.oracle_sample_cols(synth.CONFIGS[1]) == w.d
