"""Host-side logic of bench.py that needs no GPU: the byte accounting of the roofline figures, the DRAM-traffic file
written from an ncu log and read back (with the source hash that voids it), and the command-line surface."""
import importlib.util
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench():
    spec = importlib.util.spec_from_file_location("bench_under_test", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_algorithmic_bytes_follow_the_pass_table():
    b = _bench()
    for n, C in [(4, 4096), (3, 1536), (5, 1536), (2, 8)]:
        per = b.algorithmic_bytes_per_token(n, C)
        assert per == {"pre_fwd": (2 * n + 2) * C, "post_fwd": (4 * n + 2) * C, "post_bwd": (4 * n + 4) * C,
                       "tail_bwd": (6 * n + 2) * C}
        assert sum(per.values()) == (16 * n + 10) * C
        assert sum(b.algorithmic_bytes_per_token(n, C, backward=False).values()) == (6 * n + 4) * C
        # the kernels of the fused sequence move x twice in two stages: (20 n + 12) C
        assert sum(b.kernel_bytes_per_token(n, C).values()) == (20 * n + 12) * C


def test_rates_of_a_known_time():
    b = _bench()
    r = b.rates(4, 4096, 131072, 8.0, 6398.3)
    assert r["tokens_per_s"] == pytest.approx(131072 / 8e-3)
    assert r["algorithmic_gbs"] == pytest.approx(303104 * 131072 / 8e-3 / 1e9)
    assert r["frac_of_measured_peak"] == pytest.approx(r["algorithmic_gbs"] / 6398.3)
    assert r["frac_of_8TBs"] == pytest.approx(r["algorithmic_gbs"] / 8000.0)
    s = b.rates(4, 2048, 16384, 12.0, 6398.3, layers=24)
    assert s["token_layers_per_s"] == pytest.approx(24 * 16384 / 12e-3)


NCU_LOG = '''==PROF== Connected to process 1 (/usr/bin/python3.12)
"ID","Process ID","Process Name","Host Name","Kernel Name","Context","Stream","Block Size","Grid Size","Device","CC","Section Name","Metric Name","Metric Unit","Metric Value"
"0","1","python3.12","127.0.0.1","mhcl::proj_fwd_tc_k(CUtensorMap_st, CUtensorMap_st, long)","1","7","(192, 1, 1)","(64, 1, 1)","0","10.0","Command line profiler metrics","dram__bytes_read.sum","byte","270,000,000"
"0","1","python3.12","127.0.0.1","mhcl::proj_fwd_tc_k(CUtensorMap_st, CUtensorMap_st, long)","1","7","(192, 1, 1)","(64, 1, 1)","0","10.0","Command line profiler metrics","dram__bytes_write.sum","byte","1,000,000"
"1","1","python3.12","127.0.0.1","void mhcl::tail_ftc_k<4, 1>(CUtensorMap_st)","1","7","(352, 1, 1)","(64, 2, 1)","0","10.0","Command line profiler metrics","dram__bytes_read.sum","byte","600,000,000"
"1","1","python3.12","127.0.0.1","void mhcl::tail_ftc_k<4, 1>(CUtensorMap_st)","1","7","(352, 1, 1)","(64, 2, 1)","0","10.0","Command line profiler metrics","dram__bytes_write.sum","byte","240,000,000"
"2","1","python3.12","127.0.0.1","void mhcl::tail_ftc_k<4, 1>(CUtensorMap_st)","1","7","(352, 1, 1)","(64, 2, 1)","0","10.0","Command line profiler metrics","dram__bytes_read.sum","byte","999"
'''


def test_traffic_file_round_trip_and_hash_guard(tmp_path, monkeypatch):
    b = _bench()
    # a scratch repository root with the two source files the entries point at
    csrc = tmp_path / "paper_2601_05732_b200" / "csrc"
    csrc.mkdir(parents=True)
    (tmp_path / "profiles").mkdir()
    for name in ("proj_tc.cu", "tail_ftc.cu"):
        (csrc / name).write_text("// " + name)
    monkeypatch.setattr(b, "ROOT", str(tmp_path))
    log = tmp_path / "ncu.csv"
    log.write_text(NCU_LOG)
    b.write_ncu_traffic("cfgX", 8192, str(log))
    # the first launch of each kernel counts; bytes scale with the tokens of the timed launch
    assert b.ncu_traffic("proj_fwd", "cfgX", 8192) == 271_000_000
    assert b.ncu_traffic("tail_dx", "cfgX", 131072) == 840_000_000 * 16
    assert b.ncu_traffic("act_premix", "cfgX", 8192) is None          # not in the log
    assert b.ncu_traffic("tail_dx", "other", 8192) is None            # no file for that workload
    (csrc / "tail_ftc.cu").write_text("// edited since the capture")
    assert b.ncu_traffic("tail_dx", "cfgX", 8192) is None             # the kernel's source changed: figure void
    assert b.ncu_traffic("proj_fwd", "cfgX", 8192) == 271_000_000


def test_command_line_surface():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--help"], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0
    for flag in ("--gpus", "--steps", "--warmup", "--impl", "--workload", "--T", "--layers", "--permutations",
                 "--no-e2e", "--no-cpu-baseline", "--no-sk", "--no-table", "--no-graph", "--traffic-from-ncu"):
        assert flag in out.stdout, flag
