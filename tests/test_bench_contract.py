"""Host-side pieces of the benchmark that need no GPU: the byte accounting that every GB/s figure
rests on, the workload table, the defaults of the command line, and the key that ties the ncu
traffic figure to the kernel sources it was captured from."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench
from fixtures import synth


def test_algorithmic_bytes_per_element():
    # read a (2) + read m (2) + write m (2) + codes (b/8) + one fp32 step per group (4/G)
    assert bench.bytes_per_element(4, 64) == 6.5625            # GPT2-shaped boundary
    assert bench.bytes_per_element(2, 128) == 6.28125          # DeBERTa-shaped boundary
    assert bench.bytes_per_element(3, 64) == 6.4375            # forward half of the pipeline sweep
    # m kept in z bits: a (2) + m read and written (2 * (z/8 + 4/G)) + codes + step
    assert bench.bytes_per_element(4, 64, 8) == 2 + 2 * (1 + 0.0625) + 0.5 + 0.0625
    assert bench.bytes_per_element(4, 64, 32) == 2 + 8 + 0.5 + 0.0625
    # one launch of the headline workload
    cfg = synth.GPT2_XL
    assert 32 * cfg.elems * bench.bytes_per_element(cfg.bits, cfg.group) == 344064000


def test_workload_table_names_recipes_that_exist():
    for name, (recipe, macro, label) in bench.WORKLOADS.items():
        cfg = getattr(synth, recipe)
        assert cfg.n_samples % macro == 0 and macro % cfg.n_batch == 0, name
        assert "configs[" in label
    assert bench.WORKLOADS["gpt2"][1] == 32 and bench.WORKLOADS["deberta"][1] == 64 and bench.WORKLOADS["sweep"][1] == 16


def test_command_line_defaults(monkeypatch):
    monkeypatch.setattr(sys, "argv", ["bench.py"])
    args = bench.parse_args()
    assert args.gpus == 1 and args.impl == "b200" and args.workload == "gpt2" and args.topology == "replicas"
    assert args.warmup >= 3 and args.steps >= 1
    assert args.min_timed_ms >= 100                            # a timed region of a few ms is repeated


def test_traffic_figure_is_keyed_to_the_kernel_sources():
    h = bench.kernel_source_hash()
    assert len(h) == 16 and int(h, 16) >= 0
    assert bench.kernel_source_hash() == h                     # a pure function of the files
    for name, rec in bench.NCU_TRAFFIC.items():
        assert name in bench.WORKLOADS
        assert len(rec["kernel_hash"]) == 16
        # between the algorithmic reads alone and the algorithmic bytes: no re-reads, some writes still in L2
        cfg = getattr(synth, bench.WORKLOADS[name][0])
        assert 4.0 <= rec["encode_bytes_per_element"] <= bench.bytes_per_element(cfg.bits, cfg.group)


def test_peak_falls_back_when_no_measurement_is_at_hand(monkeypatch, tmp_path):
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    assert bench.measured_peak() == (bench.FALLBACK_HBM_GBS, "fallback")
    (tmp_path / "MEASURED_PEAKS.json").write_text('{"hbm_gbs": 6543.7}')
    assert bench.measured_peak() == (6543.7, "measured")
