"""Host-side logic of bench.py, on CPU: workload parsing, the flop / byte models, the clock
parser, and the max-over-ranks reduction of the multi-rank launch (two gloo ranks)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2504_05295_b200 import inputs  # noqa: E402


def test_workloads_match_the_configurations():
    sweep = bench.parse_cases("", inputs, "sweep")
    assert len(sweep) == 9 and (8192, 8192, 512) in sweep and (2048, 2048, 2048) in sweep
    large = bench.parse_cases("", inputs, "large")
    assert (32768, 32768, 8192) in large and (16384, 16384, 256) in large and len(large) == 6
    l8 = bench.parse_cases("", inputs, "llama8b")
    assert len(l8) == 224 and l8.count((14336, 4096, 1024, "bf16")) == 64 and l8.count((4096, 14336, 1024, "bf16")) == 32
    l405 = bench.parse_cases("", inputs, "llama405b")
    assert (53248, 16384, 4096, "bf16") in l405 and (16384, 53248, 1024, "bf16") in l405 and len(l405) == 14
    assert bench.parse_cases("4096:1024,1024x4096:256:bf16", inputs) == [(4096, 4096, 1024), (1024, 4096, 256, "bf16")]
    assert bench.case_gbytes((1, 1, 1, "bf16")) == 2 and bench.case_gbytes((1, 1, 1)) == 4
    assert bench.parse_cases("", inputs, "config1") == [(256, 512, 64)]
    assert bench.ALL_WORKLOADS[-1] == bench.HEADLINE == "llama8b" and len(bench.ALL_WORKLOADS) == 5
    # the oracle's bounded samples: the three 2048^2 cases of the sweep, else the cheapest distinct case(s)
    assert sorted(bench.oracle_sample_cases(sweep, "sweep")) == [(2048, 2048, 128), (2048, 2048, 512), (2048, 2048, 2048)]
    assert bench.oracle_sample_cases(l8, "llama8b") == [(1024, 4096, 256), (4096, 4096, 1024)]
    assert bench.oracle_sample_cases(large, "large") == [(16384, 16384, 256)]
    assert bench.traffic_variant(4096, 4096, 1024, 0) == "fp32_sum_in_scratch"
    assert bench.traffic_variant(4096, 4096, 256, 0) == "fp32_sum_in_scratch_low_rank" and bench.traffic_variant(16384, 16384, 128, 0) == "fp32_fused_add"
    assert bench.traffic_variant(14336, 4096, 1024, 0, 2) == "fp32_sum_in_scratch_bf16_g"
    assert bench.traffic_variant(4096, 4096, 256, 1) == "bf16_arrays"


def test_flop_and_byte_models():
    m, n, r = 4096, 2048, 256
    fl = bench.phase_flops(m, n, r, orth=0)
    assert fl["P"] == fl["R"] == fl["EF"] == fl["X"] == 2.0 * m * n * r          # 8 m n r in all (paper's count)
    assert fl["ORTH"] == 2 * (2.0 * m * r * r + r ** 3 / 3.0)                     # CholeskyQR2 at rank fraction <= 1/4
    assert bench.phase_flops(m, n, n, orth=0, rounds=3)["ORTH"] == 3 * (2.0 * m * n * n + n ** 3 / 3.0)
    by = bench.phase_bytes(m, n, r, orth=0)
    assert by["P"] == m * n * 8 + 4.0 * (n * r + m * r)
    assert by["EF"] == m * n * 12 + 4.0 * (m * r + n * r)
    assert bench.phase_bytes(m, n, r, orth=0, gbytes=2)["EF"] == m * n * 10 + 4.0 * (m * r + n * r)
    assert bench.orth_mode(m, n, r, 0) == 1 and bench.orth_mode(m, n, n, 0) == 2 and bench.orth_mode(m, n, r, 3) == 3


def test_clock_parser():
    lines = ["1965, 1965, 410.2, Not Active, Not Active, Not Active, Not Active",
             "1320, 1965, 998.0, Not Active, Not Active, Not Active, Active",
             "1335, 1965, 1001.3, Not Active, Not Active, Not Active, Active",
             "garbage"]
    res = bench.ClockSampler.parse(lines)
    assert res["sm_mhz"] == 1335.0 and res["sm_max_mhz"] == 1965.0 and res["reasons"] == ["sw_power_cap"]
    assert res["samples"] == 3
    assert bench.ClockSampler.parse([])["sm_mhz"] is None


_RANK_SCRIPT = r"""
import os, sys, json
sys.path.insert(0, %r)
import torch.distributed as dist
import bench
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%%s" %% os.environ["PORT"],
                        rank=int(os.environ["RANK"]), world_size=2)
mine = 10.0 + 5.0 * int(os.environ["RANK"])          # rank 1 is the slow one
print(json.dumps({"rank": int(os.environ["RANK"]), "max": bench.max_over_ranks(mine)}))
dist.destroy_process_group()
""" % ROOT


def test_max_over_ranks_with_two_gloo_ranks():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", _RANK_SCRIPT], env=env, stdout=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs)
    got = sorted((json.loads(o.strip().splitlines()[-1]) for o in outs), key=lambda d: d["rank"])
    assert got[0]["max"] == 15.0 and got[1]["max"] == 15.0      # every rank reports the slowest rank's time
    assert bench.max_over_ranks(3.5) == 3.5                     # no process group: identity


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--cases", "128:32,128:8",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "ms" and line["higher_is_better"] is False
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["vs_baseline"] is None
    # the value is a timing of the sample; the flop-scaled figure has its own field
    assert line["value"] == line["workloads"]["custom"]["value"] and line["projected_ms"] >= line["value"] * 0.999
