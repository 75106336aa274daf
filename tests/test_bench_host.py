"""Host-side pieces of the bench: the DRAM-traffic table (written from an ncu capture, read by
bench.py, void once the kernel's sources change) and the fp32 build of the oracle's loops that the
all-cores CPU leg times."""
import os
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _csv(path):
    rows = [["ID", "Kernel Name", "dram__bytes_read.sum", "dram__bytes_write.sum"],
            ["", "", "Mbyte", "Kbyte"],
            ["0", "void fwd_bf16_cs_kernel<64, 2, 4, 0, 1>(ScanArgs)", "100.5", "2,000.0"],
            ["1", "void reduce_slabs_kernel<bf16>(float const*)", "7.0", "7.0"],
            ["2", "void fwd_bf16_cs_kernel<64, 2, 4, 0, 1>(ScanArgs)", "101.5", "4,000.0"]]
    with open(path, "w") as f:
        for r in rows:
            f.write(",".join(f'"{x}"' for x in r) + "\n")


def test_traffic_table_round_trip(tmp_path, monkeypatch):
    from paper_2603_14360_b200 import ncu_traffic
    import bench
    _csv(tmp_path / "cap.csv")
    rd, wr, n = ncu_traffic.dram_bytes(str(tmp_path / "cap.csv"), "fwd_bf16_cs_kernel")
    assert (rd, wr, n) == (101.0e6, 3.0e6, 2)
    table = tmp_path / "dram_traffic.txt"
    monkeypatch.setattr(ncu_traffic, "TABLE", str(table))
    monkeypatch.setattr(sys, "argv", ["ncu_traffic", str(tmp_path / "cap.csv"), "--workload", "fwd_bf16", "--kernel",
                                      "fwd_bf16_cs_kernel", "--source", "scan_fwd_bf16_cs.cu", "--units", "1000"])
    ncu_traffic.main()
    monkeypatch.setattr(bench, "TRAFFIC_TABLE", str(table))
    t = bench.profiled_traffic("fwd_bf16", 4000)         # a launch four times the captured one
    assert t["bytes"] == 4 * 104.0e6 and "x4" in t["source"]
    assert bench.profiled_traffic("bptt_bf16", 4000) is None      # no row
    # a row whose digest no longer matches the sources is void
    table.write_text(table.read_text().replace(ncu_traffic.source_digest("scan_fwd_bf16_cs.cu"), "0" * 16))
    assert bench.profiled_traffic("fwd_bf16", 4000) is None
    assert bench.kernel_source_digest("api.cu") == ncu_traffic.source_digest("api.cu")


def test_committed_traffic_table_parses():
    import bench
    if os.path.exists(bench.TRAFFIC_TABLE):
        for ln in open(bench.TRAFFIC_TABLE):
            f = ln.split()
            if f and not f[0].startswith("#"):
                assert len(f) >= 6 and float(f[3]) > 0 and int(f[4]) > 0
                assert os.path.exists(os.path.join(bench.CSRC, f[2]))


def test_fp32_build_of_the_oracle_loops_tracks_the_fp64_oracle(oracle):
    from paper_2603_14360_b200 import inputs
    from paper_2603_14360_b200.inputs import ScanConfig
    f = inputs.to_f64
    cfg = ScanConfig("t", B=2, T=24, N=2, K=16, V=32, dtype="f32", seed=77)
    d = inputs.make_inputs(cfg, backward=True)
    a = [f(d[x]) for x in ("q", "k", "v", "gate", "W", "h0")]
    y, hT = oracle.fwd(*a)
    y32, hT32 = oracle.fwd_f32(*a)
    assert y32.dtype == np.float32
    assert np.abs(y32 - y).max() <= 1e-5 * np.abs(y).max() and np.abs(hT32 - hT).max() <= 1e-5 * np.abs(hT).max()
    ref, got = oracle.bwd(*a, f(d["dy"])), oracle.bwd_f32(*a, f(d["dy"]))
    for x in ref:
        assert np.abs(got[x] - ref[x]).max() <= 1e-5 * np.abs(ref[x]).max(), x


def test_all_cores_leg_runs_on_a_small_workload():
    import bench
    from paper_2603_14360_b200.inputs import ScanConfig
    cfg = ScanConfig("small", B=2, T=64, N=4, K=16, V=16, seed=5)
    rate, cores, desc, dt = bench.oracle_all_cores_rate(cfg, "fwd+bwd", seconds_target=0.2)
    assert rate > 0 and 1 <= cores <= (os.cpu_count() or 1) and "fp32" in desc
