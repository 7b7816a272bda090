"""Host-side pieces of bench.py that need no GPU: the algorithmic byte counts behind the roofline
numbers and the reader of the recorded DRAM traffic."""
import hashlib
import importlib
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2412_12639_b200 import synth  # noqa: E402

bench = importlib.import_module("bench")


def test_attention_bytes_per_layer_match_the_formula():
    # per sequence: K and V rows of prefix + tree once, q read and out written, the parent array
    for name, want in (("v7b", 18_743_536), ("l13b", 45_220_160), ("l70b", 19_136_768)):
        spec = synth.SPECS[name]
        tb = synth.make_trees(spec)
        L, T = int(tb.prefix_len[0]), tb.tree_size(0)
        by_hand = 2 * spec.n_kv_heads * (L + T) * spec.head_dim * 2 + 2 * T * spec.n_q_heads * spec.head_dim * 2 + 4 * T
        assert bench.attn_bytes_per_layer(spec, tb) == by_hand == want


def test_accept_bytes():
    spec = synth.SPECS["v7b"]
    tb = synth.make_trees(spec)
    assert bench.accept_bytes(spec, tb) == 4 * 60 * 32000 + 12 * 60


def test_recorded_traffic_is_tied_to_the_kernel_source(tmp_path, monkeypatch):
    src_dir = tmp_path / "paper_2412_12639_b200" / "csrc"
    src_dir.mkdir(parents=True)
    (tmp_path / "profiles").mkdir()
    (src_dir / "tree_attn_tc.cu").write_bytes(b"kernel v1")
    sha = hashlib.sha256(b"kernel v1").hexdigest()
    (tmp_path / "profiles" / "tree_attn_tc_v7b_ncu.md").write_text(
        "| x |\n\ndram_bytes_per_launch: 18317312\nkernel_source_sha256: %s\n" % sha)
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    assert bench.recorded_traffic("v7b", "tc") == 18317312
    assert bench.recorded_traffic("l13b", "tc") is None           # no summary for that workload
    assert bench.recorded_traffic("v7b", "tck") is None           # nor for the other kernel
    (src_dir / "tree_attn_tc.cu").write_bytes(b"kernel v2")        # the kernel changed since the capture
    assert bench.recorded_traffic("v7b", "tc") is None


def test_reference_arm_prints_one_line_on_the_small_workload():
    import json
    import subprocess
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600)
    assert p.returncode == 0, p.stderr[-2000:]
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == "tree-verify steps/sec" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    # the same description of the workload as the GPU arm prints, and whole steps (no extrapolation) when they fit
    assert line["extrapolated"] is False and "one whole step" in line["cpu_baseline"]["sample"]
    spec = synth.SPECS["tiny"]
    assert line["config"]["workload"] == "tiny" and line["config"]["n_layers"] == spec.n_layers
    assert set(line["config"]) == set(bench.config_of(type("A", (), {"workload": "tiny"})(), spec, synth.make_trees(spec), 1))
