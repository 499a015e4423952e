"""Host-side helpers of bench.py that need no GPU: the table printer of the `all_configs` block, the
look-up of recorded DRAM traffic, and the launch count the bench line claims."""

import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def test_traffic_record_matches_workload_and_chunk_only():
    import bench
    t = bench.load_traffic("c4", 16384)
    assert t is not None and t["bytes_per_step"] > 4.0e9 and t["launches_per_step"] == 31
    assert abs(t["bytes_per_launch_avg"] * t["launches_per_step"] - t["bytes_per_step"]) < 1.0
    assert bench.load_traffic("c4", 8192) is None          # no capture at that chunk width: no number
    assert bench.load_traffic("c2", 37888) is None


def test_table_of_a_saved_line(tmp_path, capsys):
    import bench
    row = dict(workload="c5", dtype="bf16", beam=8.0, frozen_head=False, M_frames=9602, K_selected=1066, D=5120,
               V=151936, chunk=16384, ms_per_step=48.4, frames_per_s=198000.0, tflops=1234.1,
               frac_of_bf16_peak=dict(burst=0.74, sustained=0.876), dp_ms=6.64, workspace_bytes=942431488,
               workspace_bytes_at_half_V=942108672, one_fp32_MxV_array=5835558912)
    broken = dict(workload="g16k", beam=0.0, error="RuntimeError('x')")
    fp32 = dict(row, workload="c1", beam=0.0, frac_of_bf16_peak=None)
    p = tmp_path / "line.log"
    p.write_text("noise\n" + json.dumps(dict(metric="m", all_configs=[row, broken, fp32])) + "\n")
    assert bench.print_table(str(p)) == 0
    out = capsys.readouterr().out.splitlines()
    assert out[2].startswith("| c5, beam 8 | 9602 | 1066 | 16384 | 48.400 | 198k | 1234.1 | 74.0% / 87.6% | 6.64 |")
    assert "failed" in out[3] and out[4].startswith("| c1 |") and "n/a" in out[4]
    (tmp_path / "empty.log").write_text("{}\n")
    assert bench.print_table(str(tmp_path / "empty.log")) == 1
