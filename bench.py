#!/usr/bin/env python
"""Benchmark of the Dion step (C-ABI CUDA library) on one B200.

One "step" is one pass of the whole hot path (P, Orthonormalize, R, error feedback, ColNorm, X
update) over one batch of synthetic input.  A default run times five workloads one after another
in one process, each for the same --steps / --warmup, building and freeing one at a time:

  config1    one 256 x 512 fp32 matrix, r = 64; a step = its ten consecutive dion_step calls
  sweep      nine fp32 squares 2048^2, 4096^2, 8192^2 at rank fractions 1, 1/4, 1/16 (one dion_step each)
  large      16384^2 and 32768^2 at rank fractions 1/4, 1/16, 1/64
  llama405b  one Llama-3-405B-shaped block at rank fractions 1/4 and 1/16, bf16 gradients (one dion_step_grouped call)
  llama8b    Llama-3-8B-shaped list, 224 matrices, bf16 gradients, rank fraction 1/4 (ONE dion_step_grouped call)

The top-level metric is the device time of the llama8b step in milliseconds (lower is better);
every workload's record, with its own roofline, end-to-end time and per-case table, is under
"workloads".  --workload NAME times that workload alone.

  python bench.py [--gpus N] [--steps K] [--warmup W]          # this library
  python bench.py --impl reference ...                          # float64 CPU oracle, bounded samples

For N > 1 launch with torch.distributed.run: every rank runs the same workloads on its own GPU
(independent replicas, no collective on the data path; weak scaling); times are the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "dion_step_time"
UNIT = "ms"
MU, ETA, EPS = 0.95, 0.01, 1e-8
HEADLINE = "llama8b"
ALL_WORKLOADS = ["config1", "sweep", "large", "llama405b", "llama8b"]
FFMA_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12     # 148 SMs x 128 FMA lanes x 2 flop x max clock
# DRAM bytes (read + write, ncu dram__bytes_*.sum) of the contraction kernel's four large launches over their
# algorithmic bytes, one ratio per way the kernel is fed.  `roofline.traffic` is the algorithmic bytes of each
# case times the ratio of its variant: a scaled figure, not a per-run counter (traffic grows in proportion to
# the matrix sizes).  Each entry names the capture it came from.
TRAFFIC_RATIOS = {
    # M + G kept in scratch: P, R and the error feedback read 4 bytes per element where the algorithmic model
    # counts M and G (the elementwise pass that forms the sum is another kernel)
    "fp32_sum_in_scratch": (0.574, "ncu --set full, one step on 4096^2 r=1024, fp32 G, fp32 mode: P 90.9 + R 91.6 + error "
                                   "feedback 144.8 + X 95.8 = 423.6 MB / 738.3 MB"),
    "fp32_sum_in_scratch_bf16_g": (0.817, "the same on 14336x4096 r=1024 with bf16 G (the dominant shape of the Llama lists; the "
                                          "model counts 2 bytes for G there): 368 + 317 + 549 + 451 = 1685 MB / 2063.6 MB"),
    "fp32_sum_in_scratch_low_rank": (0.718, "the same on 16384^2 r=256 (rank fraction 1/64), fp32 G: 1.30 + 1.30 + 2.32 + 2.12 = "
                                            "7.03 GB / 9.80 GB"),
    "fp32_fused_add": (0.885, "same capture with M + G formed inside P and R (the path below rank fraction 1/64)"),
    "bf16_arrays": (0.99, "ncu --set full, 8192^2 r=512, bf16-operand mode: error feedback 0.98, X update 0.93, P 1.07"),
}


def traffic_variant(m, n, r, precision, gbytes=4):
    if precision == 1:
        return "bf16_arrays"
    if 64 * r < min(m, n):
        return "fp32_fused_add"
    if gbytes == 2:
        return "fp32_sum_in_scratch_bf16_g"
    return "fp32_sum_in_scratch" if 8 * r >= min(m, n) else "fp32_sum_in_scratch_low_rank"


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_burst": float(d["bf16_tflops"]),
                "bf16_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


def parse_cases(spec, inputs, workload="sweep"):
    """Cases are (m, n, r) for fp32 gradients or (m, n, r, "bf16").  --cases takes d:r or mxn:r[:bf16]."""
    if spec:
        out = []
        for tok in spec.split(","):
            f = tok.split(":")
            if "x" in f[0]:
                m, n = (int(v) for v in f[0].split("x"))
            else:
                m = n = int(f[0])
            case = (m, n, int(f[1]))
            if len(f) > 2 and f[2] == "bf16":
                case = case + ("bf16",)
            out.append(case)
        return out
    if workload == "config1":
        m, n, r, _ = inputs.config1()
        return [(m, n, r)]
    if workload == "large":
        return inputs.config3_cases()
    if workload == "llama8b":
        return [(m, n, min(m, n) // 4, "bf16") for _, m, n in inputs.config4_shapes()]
    if workload == "llama405b":
        return ([(m, n, min(m, n) // 4, "bf16") for _, m, n in inputs.config5_shapes()] +
                [(m, n, min(m, n) // 16, "bf16") for _, m, n in inputs.config5_shapes()])
    return inputs.config2_cases()


def case_gbytes(c):
    return 2 if len(c) > 3 and c[3] == "bf16" else 4


# ---------------------------------------------------------------------------
# flop / byte models (algorithmic: what the method must compute and move, whatever the kernels do)
# ---------------------------------------------------------------------------

def orth_mode(m, n, r, orth):
    if orth == 0:
        return 1 if 4 * r <= min(m, n) else 2
    return orth


def phase_flops(m, n, r, orth, rounds=None):
    if rounds is None:
        rounds = {1: 2, 2: 4}.get(orth_mode(m, n, r, orth), 0)
    if orth == 4:
        # randomized Cholesky QR: sketch product 2.5 m r^2, ~2 rounds on the stacked panel [S P; P] (Gram matrix
        # from the 1.25 r sketch rows, factor, solve over 1.25 r + m rows), then one Cholesky-QR round on B
        # plus the Gram matrix of its check
        k = 1.25 * r
        rnd = 2.0 * (k * r * r + r ** 3 / 3.0 + (k + m) * r * r)
        o = 2.5 * m * r * r + rnd + 3.0 * m * r * r + r ** 3 / 3.0
        g = 2.0 * m * n * r
        return {"P": g, "ORTH": o, "R": g, "EF": g, "COLNORM": 3.0 * n * r, "X": g, "ORTH_GEMM": o}
    if rounds == 1 and orth_mode(m, n, r, orth) == 1:
        # CholeskyQR2 whose second round was skipped on the device: one round plus the Gram matrix of the check
        o = 3.0 * m * r * r + r ** 3 / 3.0
        g = 2.0 * m * n * r
        og = 3.0 * m * r * r + 2.0 / 3.0 * r ** 3
        return {"P": g, "ORTH": o, "R": g, "EF": g, "COLNORM": 3.0 * n * r, "X": g, "ORTH_GEMM": og}
    if rounds:
        o = rounds * (2.0 * m * r * r + r ** 3 / 3.0)     # Gram (symmetric half) + Cholesky + solve
    else:
        o = 4.0 * m * r * r - 4.0 / 3.0 * r ** 3          # Householder incl. forming the factor
    g = 2.0 * m * n * r
    # tensor-engine products inside the orthonormalization: Gram half + solve + blocked Cholesky
    # updates + triangular inverse ~ 2 m r^2 + 2/3 r^3 per round
    og = rounds * (2.0 * m * r * r + 2.0 / 3.0 * r ** 3) if rounds else 0.0
    return {"P": g, "ORTH": o, "R": g, "EF": g, "COLNORM": 3.0 * n * r, "X": g, "ORTH_GEMM": og}


def phase_bytes(m, n, r, orth, gbytes=4, rounds=None):
    if rounds is None:
        rounds = {1: 2, 2: 4}.get(orth_mode(m, n, r, orth), 2)
    mn = float(m) * n
    return {"P": mn * (4 + gbytes) + 4.0 * (n * r + m * r),
            "ORTH": rounds * 4.0 * (3 * m * r),
            "R": mn * (4 + gbytes) + 4.0 * (m * r + n * r),
            "EF": mn * (8 + gbytes) + 4.0 * (m * r + n * r),
            "COLNORM": 4.0 * 3 * n * r,
            "X": mn * 8 + 4.0 * (m * r + n * r),
            "ORTH_GEMM": rounds * 4.0 * (3 * m * r + 4 * r * r)}


def pairs_apply(m, n, r):
    """Shapes whose R and error-feedback products run on bf16 (hi, lo) pairs in fp32 mode (the library's own rule:
    M + G kept in scratch, i.e. rank fraction >= 1/64, and dimensions that are multiples of 8)."""
    return r >= 64 and 64 * r >= min(m, n) and m % 8 == 0 and n % 8 == 0 and r % 8 == 0 and m >= 128 and n >= 128


def p_pairs_apply(m, n, r, orth):
    """Shapes whose P = (M + G) Q runs on bf16 pairs first (the library's rule: pairs in use, CholeskyQR2, and
    m n r >= 1.5e10; the accurate product is recomputed on the device only if the orthogonality probe asks)."""
    return pairs_apply(m, n, r) and float(m) * n * r >= 1.5e10 and orth_mode(m, n, r, orth) == 1


def case_report(c, ms, rounds, args, peaks, binding):
    """Per-case line: time and the roofline that binds it.  t_hbm: the 7-pass model (read M and G twice,
    read-modify-write M, read-modify-write X) at the measured copy bandwidth; t_tensor: every product at the
    tensor peak of the arithmetic it runs in -- fp32 mode: the orthonormalization 3xTF32 (three TF32 passes, TF32
    taken as half the measured bf16 peak), P, R and the error feedback three bf16 passes on (hi, lo) pairs where
    the library uses them (else 3xTF32), the X update one pass on IEEE half factors at the 16-bit rate where every
    dimension is a multiple of 8 (else one TF32 pass); bf16-operand mode: one bf16 pass for the four products."""
    m, n, r = c[:3]
    out = {"m": m, "n": n, "r": r, "ms": ms,
           "orth_mode": ["auto", "cholqr2", "adaptive", "householder", "rcqr"][orth_mode(m, n, r, args.orth)], "orth_rounds": rounds}
    if ms is None or args.engine == binding.ENGINE_SIMT or args.lazy:
        return out
    gb = case_gbytes(c)
    fl = phase_flops(m, n, r, args.orth, rounds=rounds)
    model_bytes = float(m) * n * (20 + 2 * gb) + 4.0 * (3 * n * r + 3 * m * r)
    bf16 = peaks["bf16_sustained"]
    tf32 = 0.5 * bf16
    t_hbm = model_bytes / (peaks["hbm_gbs"] * 1e9) * 1e3
    if args.precision == binding.PREC_BF16_OPERANDS:
        t_prod = sum(fl[p] for p in ("P", "R", "EF", "X")) / (bf16 * 1e12)
    else:
        pair_peak = bf16 / 3.0 if pairs_apply(m, n, r) else tf32 / 3.0
        ef_peak = bf16 / 3.0 if (m % 8 == 0 and n % 8 == 0 and r % 8 == 0 and r >= 64) else tf32 / 3.0
        p_peak = bf16 / 3.0 if p_pairs_apply(m, n, r, args.orth) else tf32 / 3.0
        x_peak = bf16 if (m % 8 == 0 and n % 8 == 0 and r % 8 == 0 and r >= 64 and m >= 128 and n >= 64) else tf32
        t_prod = fl["P"] / (p_peak * 1e12) + fl["R"] / (pair_peak * 1e12) + fl["EF"] / (ef_peak * 1e12) + fl["X"] / (x_peak * 1e12)
    t_tensor = (t_prod + fl["ORTH"] / (tf32 / 3.0 * 1e12)) * 1e3
    bound = "hbm" if t_hbm >= t_tensor else "tensor"
    out.update({"t_hbm_ms": t_hbm, "t_tensor_ms": t_tensor, "bound": bound,
                "roofline_frac": max(t_hbm, t_tensor) / ms, "model_gbs": model_bytes / (ms * 1e-3) / 1e9})
    return out


def oracle_flops(m, n, r):
    return 8.0 * m * n * r + 4.0 * m * r * r - 4.0 / 3.0 * r ** 3


def max_over_ranks(value: float, device=None) -> float:
    """Max of a per-rank scalar over the default process group (identity without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# ---------------------------------------------------------------------------
# clocks sampler
# ---------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.proc = None
        self.path = None
        self.dev = device_index

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(prefix="dion_clocks_", suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.dev)], stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        res = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return res
        try:
            self.proc.terminate()
            self.proc.wait(timeout=5)
        except Exception:
            pass
        try:
            self.out.close()
            lines = open(self.path).read().splitlines()
            os.unlink(self.path)
            res = self.parse(lines)
        except Exception:
            pass
        return res

    @staticmethod
    def parse(lines):
        """Median SM clock, max clock and the throttle reasons seen in nvidia-smi CSV lines."""
        res = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if True:
            rows = [l.strip().split(",") for l in lines if l.strip()]
            sm, mx, reasons = [], [], set()
            names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
            for row in rows:
                if len(row) < 7:
                    continue
                try:
                    sm.append(float(row[0])); mx.append(float(row[1]))
                except ValueError:
                    continue
                for nm, v in zip(names, row[3:7]):
                    if v.strip().lower() == "active":
                        reasons.add(nm)
            if sm:
                res = {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                       "samples": len(sm)}
        return res


# ---------------------------------------------------------------------------
# reference arm: the float64 oracle on host cores, bounded samples
# ---------------------------------------------------------------------------

def oracle_sample_cases(cases, wid):
    """The bounded sample of a workload the oracle is timed on: the three 2048^2 cases of the sweep (full rank
    included); otherwise the smallest distinct case (two for the headline list: its two cheapest shape classes)."""
    uniq = sorted(set(tuple(c[:3]) for c in cases), key=lambda c: oracle_flops(*c))
    if wid == "sweep":
        return [c for c in uniq if c[0] == 2048]
    if wid == HEADLINE:
        return uniq[:2]
    return uniq[:1]


def time_oracle(sample, steps, warmup, bf16=False):
    """Times the oracle as it stands: one step on each sample case per pass.  Returns (ms per pass, cores)."""
    import torch
    from oracle import dion_oracle as orc
    from paper_2504_05295_b200 import inputs
    probs = []
    for k, (m, n, r) in enumerate(sample):
        pb = inputs.make_problem(m, n, r, seed=0, k=k, ks=min(64, m, n),
                                 g_dtype=torch.bfloat16 if bf16 else torch.float32)
        probs.append([pb, pb.X.double().numpy(), pb.M.double().numpy(), pb.Q.double().numpy(),
                      pb.grad(0).double().numpy()])
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        for p in probs:
            res = orc.step(p[1], p[2], p[4], p[3], MU, ETA, EPS)
            p[1], p[2], p[3] = res.X, res.M, res.Q
        dt = (time.perf_counter() - t0) * 1e3
        if it >= warmup:
            times.append(dt)
    return sum(times) / len(times), orc.num_threads()


def sample_text(sample):
    return ", ".join(f"{m}x{n} r={r}" for m, n, r in sample)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2504_05295_b200 import inputs
    steps, warmup = max(1, min(args.steps, 2)), min(args.warmup, 1)
    wids = [args.workload] if (args.workload != "all" or args.cases) else ALL_WORKLOADS
    if args.cases:
        wids = ["custom"]
    records, cores = {}, 1
    for wid in wids:
        cases = parse_cases(args.cases, inputs, wid)
        sample = [tuple(c[:3]) for c in cases] if args.cases else oracle_sample_cases(cases, wid)
        bf16 = any(case_gbytes(c) == 2 for c in cases)
        ms, cores = time_oracle(sample, steps, warmup, bf16)
        f_sample = sum(oracle_flops(*c) for c in sample)
        f_full = sum(oracle_flops(*c[:3]) for c in cases)
        records[wid] = {"value": ms, "unit": UNIT, "sample": sample_text(sample), "steps": steps, "warmup": warmup,
                        "projected_ms": ms * f_full / f_sample,
                        "projected_note": "the measured sample time scaled to the whole workload by the oracle's flop "
                                          "count 8mnr + 4mr^2 - 4/3 r^3; not a timing",
                        "workload": workload_name(cases)}
    top = HEADLINE if HEADLINE in records else wids[-1]
    rec = records[top]
    desc = (f"float64 CPU oracle, one step each on {rec['sample']} (a bounded sample of the workload), "
            f"{steps} timed passes; value = the measured time of that sample")
    line = {"impl": "reference", "metric": METRIC, "value": rec["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": rec["value"], "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": rec["workload"], "workload_id": top, "sample": rec["sample"]},
            "projected_ms": rec["projected_ms"],
            "cpu_baseline": {"value": rec["value"], "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": rec["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "workloads": records, "gpu_launches": 0}
    print(json.dumps(line))


def workload_name(cases):
    import collections
    cnt = collections.Counter((c[0], c[1], c[2], "bf16 G" if case_gbytes(c) == 2 else "fp32 G") for c in cases)
    return ("; ".join(f"{k}x {m}x{n} r={r} {g}" if k > 1 else f"{m}x{n} r={r} {g}" for (m, n, r, g), k in cnt.items()) +
            "; fp32 X, M, Q; seeded low-rank (rank 64, s_i=2^-i/2) + 0.1 N(0,1) gradients")


# ---------------------------------------------------------------------------
# this library
# ---------------------------------------------------------------------------

def measure_tf32_peak(torch, binding, n=8192, reps=5):
    """TFLOP/s of the library's own single-pass TF32 contraction (one kind::tf32 MMA per K step, operands by
    TMA) on an n^3 product, through the library's internal one-product hook: the measured counterpart of the
    1/2 x bf16 figure the TF32 roofline assumes."""
    import ctypes

    class GemmArgs(ctypes.Structure):     # dion_debug_gemm_args of csrc/dion_internal.h
        _fields_ = [("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                    ("A", ctypes.c_void_p), ("a_si", ctypes.c_int64), ("a_sk", ctypes.c_int64),
                    ("A2", ctypes.c_void_p), ("a2_si", ctypes.c_int64), ("a2_sk", ctypes.c_int64), ("a2_mode", ctypes.c_int),
                    ("B", ctypes.c_void_p), ("b_sk", ctypes.c_int64), ("b_sn", ctypes.c_int64),
                    ("C", ctypes.c_void_p), ("ldc", ctypes.c_int64), ("epi", ctypes.c_int),
                    ("C2", ctypes.c_void_p), ("ldc2", ctypes.c_int64), ("c2_mode", ctypes.c_int),
                    ("alpha", ctypes.c_float), ("tri", ctypes.c_int), ("klimit", ctypes.c_int), ("precise", ctypes.c_int),
                    ("ab16", ctypes.c_int), ("tf32x1", ctypes.c_int), ("variant", ctypes.c_int),
                    ("A16lo", ctypes.c_void_p), ("B16lo", ctypes.c_void_p)]
    lib = binding.load_library()
    lib.dion_debug_gemm.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.POINTER(GemmArgs), ctypes.c_void_p,
                                    ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
    lib.dion_debug_gemm.restype = ctypes.c_int
    A = torch.randn(n, n, device="cuda").to(torch.bfloat16).float()    # values that fit TF32
    B = torch.randn(n, n, device="cuda").to(torch.bfloat16).float()
    C = torch.zeros(n, n, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    a = GemmArgs()
    a.M = a.N = a.K = n
    a.A, a.a_si, a.a_sk = A.data_ptr(), n, 1
    a.B, a.b_sk, a.b_sn = B.data_ptr(), 1, n
    a.C, a.ldc, a.epi, a.alpha, a.tf32x1 = C.data_ptr(), n, 0, 1.0, 1
    sptr = int(torch.cuda.current_stream().cuda_stream)
    best = None
    for i in range(reps + 2):
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        rc = lib.dion_debug_gemm(2, 0, ctypes.byref(a), None, 0, status.data_ptr(), sptr)
        e1.record()
        torch.cuda.synchronize()
        if rc != 0 or int(status.item()) != 0:
            return None
        if i >= 2:
            ms = e0.elapsed_time(e1)
            best = ms if best is None else min(best, ms)
    return 2.0 * n ** 3 / (best * 1e-3) / 1e12


def run_workload(wid, cases, grouped, args, ctx):
    """Builds one workload in HBM, times `steps` steps of it after `warmup`, its end-to-end form and its
    roofline, frees it.  Returns the workload's record (every rank calls this; the times are maxima over ranks)."""
    import torch
    from paper_2504_05295_b200 import binding, inputs
    world, rank, local, dev, peaks = ctx["world"], ctx["rank"], ctx["local"], ctx["dev"], ctx["peaks"]
    stream = torch.cuda.current_stream()
    sptr = int(stream.cuda_stream)
    reps_per_step = 10 if wid == "config1" else 1       # config 1 is a ten-step sequence on one small matrix
    ks = inputs.config1()[3] if wid == "config1" else 64

    dp_sync = args.sync == "dp"
    state = []
    for k, c in enumerate(cases):
        m, n, r = c[:3]
        # data-parallel ranks share X and Q (one seed) and see their own gradients (noise seeded per rank below)
        pb = inputs.make_problem(m, n, r, seed=0 if dp_sync else rank, k=k, ks=ks, device=dev, keep_signal=False,
                                 g_dtype=torch.bfloat16 if case_gbytes(c) == 2 else torch.float32)
        gs = [pb.grad(t + (2 * rank if dp_sync else 0)) for t in range(2)]
        d = torch.zeros(r, device=dev)
        # --form short-side: the transposed form wherever it shortens the orthonormalized panel
        tr = args.form == "short-side" and m > n
        if tr:
            pb.Q = inputs.row_side_factor(pb)
        sk = inputs.sketch_matrix(pb, transposed=tr) if args.orth == 4 else None   # Algorithm 4's S, 1.25 r rows
        descs = [binding.matrix_desc(pb.X, pb.M, g, pb.Q, d, tr, sk) for g in gs]
        state.append({"pb": pb, "G": gs, "d": d, "descs": descs, "transposed": tr, "sketch": sk})
    torch.cuda.synchronize()

    opt = binding.Dion(mu=MU, eps=EPS, precision=args.precision, orth=args.orth, engine=args.engine, device=local)
    need = max(opt.workspace_bytes(*c[:3]) for c in cases)
    packed = [binding.Dion.pack([st["descs"][i] for st in state]) for i in range(2)]

    steppers = None
    if dp_sync:
        from paper_2504_05295_b200 import dp
        steppers = [dp.DpStepper(opt, [st["descs"][i] for st in state], dev) for i in range(2)]

    def one_step(t, per_case_events=None):
        for rep in range(reps_per_step):
            tt = t * reps_per_step + rep
            if dp_sync:     # project all, all-reduce P, factor all, all-reduce W, finish all
                steppers[tt % 2].step(ETA, stream)
                continue
            if grouped:     # one dion_step_grouped call over the whole list
                opt.step_grouped_packed(packed[tt % 2], len(state), ETA, sptr)
                continue
            for ci, st in enumerate(state):
                if per_case_events is not None:
                    e0 = torch.cuda.Event(enable_timing=True); e0.record(stream)
                if args.lazy:   # Lazy-Dion: the right factor is refreshed every K-th step only
                    opt.lazy_step_desc(st["descs"][tt % 2], ETA, tt % args.lazy == 0, sptr)
                else:
                    opt.step_desc(st["descs"][tt % 2], ETA, sptr)
                if per_case_events is not None:
                    e1 = torch.cuda.Event(enable_timing=True); e1.record(stream)
                    per_case_events[ci].append((e0, e1))

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for t in range(args.warmup):
        one_step(t)
    torch.cuda.synchronize()
    status, skipped = opt.get_status()

    # ---- timed region: exactly K steps --------------------------------------------------
    sampler = ClockSampler(local)
    case_events = [[] for _ in cases]
    launches0 = opt.launch_count()
    barrier()
    sampler.start()
    e_start = torch.cuda.Event(enable_timing=True); e_end = torch.cuda.Event(enable_timing=True)
    e_start.record(stream)
    for t in range(args.steps):
        one_step(args.warmup + t, case_events)
    e_end.record(stream)
    barrier()
    clocks = sampler.stop()
    ms_total = e_start.elapsed_time(e_end)
    launches = opt.launch_count() - launches0
    if clocks.get("samples", 0) == 0 and not dp_sync:
        # a timed region shorter than nvidia-smi's first sample (config 1: ~20 ms): the same steps once more,
        # untimed, for about a second under a fresh sampler, so that the record still says what clocks this load sees
        sampler = ClockSampler(local)
        sampler.start()
        t_end = time.time() + 1.0
        t_extra = 0
        while time.time() < t_end:
            one_step(args.warmup + args.steps + t_extra)
            t_extra += 1
            if t_extra % 8 == 0:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        clocks = sampler.stop()
        clocks["note"] = "timed region shorter than one sampling interval: sampled over the same steps repeated untimed right after it"
    status2, skipped2 = opt.get_status()
    ms_step = max_over_ranks(ms_total / args.steps, dev)
    case_ms = [sum(a.elapsed_time(b) for a, b in ev) / len(ev) if ev else None for ev in case_events]

    # ---- per-phase times: a second, profiled pass (the library's own events around every phase).  Kept out of
    # the timed region: with profiling on, small steps are launched kernel by kernel instead of as one graph. ----
    prof_steps = max(1, min(args.steps, 3))
    opt.profile_enable(True)
    for t in range(prof_steps):
        one_step(args.warmup + args.steps + t)
    torch.cuda.synchronize()
    phase_ms, phase_launches = opt.profile_read()
    opt.profile_enable(False)
    phase_ms = {k: v * args.steps / prof_steps for k, v in phase_ms.items()}             # scaled to the timed steps
    phase_launches = {k: v * args.steps / prof_steps for k, v in phase_launches.items()}
    s2b, k2b = opt.get_status()
    status2 |= s2b; skipped2 += k2b

    # ---- end to end: host gradients in, column norms out, through the same C-ABI call ----
    host_g = [st["G"][0].cpu().pin_memory() for st in state]
    host_d = [torch.zeros(st["d"].shape, dtype=torch.float32).pin_memory() for st in state]
    h2d = sum(g.numel() * g.element_size() for g in host_g) * reps_per_step
    d2h = sum(d.numel() * d.element_size() for d in host_d) * reps_per_step

    # The gradients arrive matrix by matrix on a copy stream; a matrix is stepped as soon as its
    # gradient has landed, so the copy of the next one overlaps the kernels of this one (within a
    # step only: a step's gradients cannot exist before the previous step's update).  A grouped
    # workload is stepped in up to E2E_GROUPS dion_step_grouped calls, one per group of consecutive
    # matrices (whole layers), each as soon as its group's gradients have landed: with one call for the
    # whole list the 14 GB of gradients of the 8B list would have to land before the first kernel.
    copy_stream = torch.cuda.Stream(device=dev)
    done_ev = [None] * len(state)       # matrix k's kernels of the previous step (they read G_k)
    E2E_GROUPS = 4
    ngroups = min(E2E_GROUPS, max(1, len(state) // 7)) if grouped else 1
    bounds = [len(state) * i // ngroups for i in range(ngroups + 1)]
    group_packed = [binding.Dion.pack([st["descs"][0] for st in state[bounds[i]:bounds[i + 1]]]) for i in range(ngroups)] if grouped else []

    def e2e_once(after=None):
        landed = []
        with torch.cuda.stream(copy_stream):
            if after is not None:
                copy_stream.wait_event(after)
            for k, (st, hg) in enumerate(zip(state, host_g)):
                if done_ev[k] is not None:
                    copy_stream.wait_event(done_ev[k])
                st["G"][0].copy_(hg, non_blocking=True)
                ev = torch.cuda.Event(); ev.record(copy_stream)
                landed.append(ev)
        if grouped:
            for gi in range(ngroups):
                lo, hi = bounds[gi], bounds[gi + 1]
                stream.wait_event(landed[hi - 1])
                opt.step_grouped_packed(group_packed[gi], hi - lo, ETA, sptr)
                ev = torch.cuda.Event(); ev.record(stream)
                for k in range(lo, hi):
                    host_d[k].copy_(state[k]["d"], non_blocking=True)
                    done_ev[k] = ev
        elif dp_sync:
            stream.wait_event(landed[-1])
            steppers[0].step(ETA, stream)
            ev = torch.cuda.Event(); ev.record(stream)
            for k, (st, hd) in enumerate(zip(state, host_d)):
                hd.copy_(st["d"], non_blocking=True)
                done_ev[k] = ev
        else:
            for k, (st, hd) in enumerate(zip(state, host_d)):
                stream.wait_event(landed[k])
                if args.lazy:
                    opt.lazy_step_desc(st["descs"][0], ETA, False, sptr)
                else:
                    opt.step_desc(st["descs"][0], ETA, sptr)
                ev = torch.cuda.Event(); ev.record(stream)
                done_ev[k] = ev
                hd.copy_(st["d"], non_blocking=True)

    def e2e_step(after=None):
        for rep in range(reps_per_step):
            e2e_once(after if rep == 0 else None)

    e2e_step()
    barrier()
    e2e_steps = max(1, min(args.steps, 3))
    f0 = torch.cuda.Event(enable_timing=True); f1 = torch.cuda.Event(enable_timing=True)
    f0.record(stream)
    for i in range(e2e_steps):
        e2e_step(after=f0 if i == 0 else None)
    f1.record(stream)
    barrier()
    e2e_ms = max_over_ranks(f0.elapsed_time(f1) / e2e_steps, dev)
    status3, _ = opt.get_status()
    del host_g

    # Cholesky-QR rounds the device ran per case, read on one more (untimed) step
    opt.orth_rounds()
    case_rounds = []
    for ci, st in enumerate(state):
        m_, n_, r_ = cases[ci][:3]
        if orth_mode(m_, n_, r_, args.orth) not in (1, 2) or (grouped and ci >= 8):
            case_rounds.append(None)
            continue
        opt.step_desc(st["descs"][1], ETA, sptr)
        case_rounds.append(opt.orth_rounds())
    if grouped:     # matrices of one shape class behave alike: reuse the first one's count
        seen = {}
        for ci, c in enumerate(cases):
            if case_rounds[ci] is not None:
                seen.setdefault(tuple(c[:3]), case_rounds[ci])
        case_rounds = [seen.get(tuple(c[:3])) for c in cases]

    # the cases of the oracle's bounded sample, stepped alone (for the CPU-baseline comparison)
    sample_gpu_ms = None
    if ctx.get("want_cpu") and wid == ctx.get("cpu_wid"):
        sample = oracle_sample_cases(cases, wid)
        keys = [tuple(c[:3]) for c in cases]
        tot = 0.0
        for c in sample:
            st = state[keys.index(c)]
            opt.step_desc(st["descs"][1], ETA, sptr)
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record(stream)
            opt.step_desc(st["descs"][0], ETA, sptr)
            b.record(stream)
            torch.cuda.synchronize()
            tot += a.elapsed_time(b)
        sample_gpu_ms = tot

    rec = None
    e2e_calls = (ngroups if grouped else len(state)) * reps_per_step
    if rank == 0:
        rec = workload_record(wid, cases, grouped, args, peaks, binding, ms_step, e2e_ms, e2e_steps, e2e_calls, h2d, d2h,
                              launches, clocks, phase_ms, phase_launches, case_ms, case_rounds, need,
                              (status, status2, status3, skipped + skipped2), reps_per_step, world,
                              sum(1 for st in state if st["transposed"]))
        rec["sample_gpu_ms"] = sample_gpu_ms
    opt.close()
    del state, packed, steppers, host_d, group_packed
    torch.cuda.empty_cache()
    return rec


def workload_record(wid, cases, grouped, args, peaks, binding, ms_step, e2e_ms, e2e_steps, e2e_calls, h2d, d2h, launches, clocks,
                    phase_ms, phase_launches, case_ms, case_rounds, need, stat, reps_per_step, world, n_transposed):
    # ---- roofline of the dominant phase ---------------------------------------------------
    # Algorithmic work: the four products, 8 m n r flops, plus the orthonormalization counted as CholeskyQR2
    # (6 p r^2 + 2/3 r^3 on the p x r panel) whatever rounds the device ran; the executed rounds are reported beside.
    tot_fl = {p: 0.0 for p in binding.PHASES}
    tot_by = {p: 0.0 for p in binding.PHASES}
    exe_fl = {p: 0.0 for p in binding.PHASES}
    traffic = 0.0
    for c, nr in zip(cases, case_rounds):
        m, n, r = c[:3]
        fl = phase_flops(m, n, r, args.orth, rounds=None)
        fx = phase_flops(m, n, r, args.orth, rounds=nr)
        by = phase_bytes(m, n, r, args.orth, gbytes=case_gbytes(c), rounds=None)
        if orth_mode(m, n, r, args.orth) in (1, 2):
            prow = n if (args.form == "short-side" and m > n) else m
            fl["ORTH"] = fl["ORTH_GEMM"] = 6.0 * prow * r * r + 2.0 / 3.0 * r ** 3
        if args.lazy:
            # per step: W = B Q, the M update and the X update (2 m n r each); per refresh two more passes
            # over B (T = B Q, Z = B^T T) and the orthonormalization of an n x r panel
            refresh = sum(1 for t in range(args.warmup, args.warmup + args.steps) if t % args.lazy == 0) / args.steps
            flo = phase_flops(n, m, r, args.orth)
            for f in (fl, fx):
                f["R"] = 0.0
                f["ORTH"] = refresh * (4.0 * m * n * r + flo["ORTH"]); f["ORTH_GEMM"] = refresh * flo["ORTH_GEMM"]
                f["COLNORM"] = 3.0 * m * r
            by["R"] = 0.0
            by["ORTH"] = refresh * (2.0 * by["P"] + by["ORTH"]); by["ORTH_GEMM"] = refresh * by["ORTH_GEMM"]
        ratio = TRAFFIC_RATIOS[traffic_variant(m, n, r, args.precision, case_gbytes(c))][0]
        for p in binding.PHASES:
            tot_fl[p] += fl[p] * reps_per_step; tot_by[p] += by[p] * reps_per_step; exe_fl[p] += fx[p] * reps_per_step
        traffic += ratio * sum(by[p] for p in ("P", "R", "EF", "X")) * reps_per_step
    # The dominant kernel is the tcgen05 contraction kernel: the four large products plus the
    # products inside the orthonormalization.  Its roofline uses their summed algorithmic
    # flops / bytes and summed event times.  (With --engine 1 the same phases run on the FMA kernel.)
    gemm_phases = ["P", "R", "EF", "X", "ORTH_GEMM"]
    dom_ms = sum(phase_ms[p] for p in gemm_phases) / args.steps
    dom_fl = sum(tot_fl[p] for p in gemm_phases)
    dom_fx = sum(exe_fl[p] for p in gemm_phases)
    dom_by = sum(tot_by[p] for p in gemm_phases)
    dom_launches = sum(phase_launches[p] for p in gemm_phases) / args.steps
    total_phase_ms = sum(phase_ms[p] for p in binding.PHASES if p != "ORTH_GEMM")
    tensor_engine = (args.engine != binding.ENGINE_SIMT)
    if args.precision == binding.PREC_BF16_OPERANDS:
        flop_peak, flop_bound, peak_note = peaks["bf16_sustained"], "tensor", "bf16 sustained, of " + peaks["source"]
    elif tensor_engine:
        flop_peak, flop_bound = peaks["bf16_sustained"] * 0.5, "tensor"
        peak_note = ("tf32 = 1/2 x bf16 sustained, of " + peaks["source"] + " (nominal ratio); a 3xTF32 product counts "
                     "once although it issues three MMAs (four with split accumulators)")
    else:
        flop_peak, flop_bound, peak_note = FFMA_PEAK_TFLOPS, "alu", "fp32 FMA: 148 SM x 128 lanes x 2 x 1.965 GHz"
    t_flop = dom_fl / (flop_peak * 1e12) * 1e3
    t_hbm = dom_by / (peaks["hbm_gbs"] * 1e9) * 1e3
    if dom_ms <= 0:
        roof = {"bound": None, "achieved": None, "peak": None, "unit": None, "frac": None, "traffic": None}
    elif t_hbm >= t_flop:
        achieved = dom_by / (dom_ms * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": None, "peak_note": "copy bandwidth, of " + peaks["source"]}
    else:
        achieved = dom_fl / (dom_ms * 1e-3) / 1e12
        roof = {"bound": flop_bound, "achieved": achieved, "peak": flop_peak, "unit": "TFLOP/s",
                "frac": achieved / flop_peak, "traffic": None, "peak_note": peak_note,
                "achieved_executed": dom_fx / (dom_ms * 1e-3) / 1e12,
                "executed_note": "flops of the Cholesky-QR rounds the device actually ran (implementation work) in "
                                 "place of the CholeskyQR2 count"}
    roof.update({"kernel": "k_gemm_umma" if tensor_engine else "k_gemm_simt",
                 "phases": gemm_phases, "ms_per_step": dom_ms,
                 "share_of_step": dom_ms * args.steps / max(total_phase_ms, 1e-9),
                 "launches_per_step": dom_launches,
                 "algorithmic_flops_per_step": dom_fl, "algorithmic_bytes_per_step": dom_by,
                 "traffic_is_scaled": True,
                 "traffic_note": "algorithmic bytes of the four large products of each case x the measured DRAM / "
                                 "algorithmic ratio of the way that case feeds the kernel; ratios and their captures: " +
                                 "; ".join(f"{k} {v[0]} ({v[1]})" for k, v in TRAFFIC_RATIOS.items())})
    if tensor_engine and dom_ms > 0:
        roof["traffic"] = traffic
    # The four large products alone (never overlapped with other work; the products inside the
    # orthonormalization run partly beside its serial chain on a second stream, so their event
    # durations include waiting for SMs).
    big = ["P", "R", "EF", "X"]
    big_ms = sum(phase_ms[p] for p in big) / args.steps
    if big_ms > 0 and roof.get("unit") == "TFLOP/s":
        big_tf = sum(tot_fl[p] for p in big) / (big_ms * 1e-3) / 1e12
        roof["large_products"] = {"phases": big, "ms_per_step": big_ms, "achieved": big_tf, "frac": big_tf / flop_peak,
                                  "gbs": sum(tot_by[p] for p in big) / (big_ms * 1e-3) / 1e9}
    phases = {}
    for p in binding.PHASES:
        ms_p = phase_ms[p] / args.steps
        phases[p] = {"ms": ms_p, "share": phase_ms[p] / max(total_phase_ms, 1e-9),
                     "tflops": tot_fl[p] / (ms_p * 1e-3) / 1e12 if ms_p > 0 else None,
                     "gbs": tot_by[p] / (ms_p * 1e-3) / 1e9 if ms_p > 0 else None}
    status, status2, status3, skipped = stat
    rec = {"value": ms_step, "unit": UNIT, "ms_per_step": ms_step, "steps": args.steps, "warmup": args.warmup,
           "config": {"workload": workload_name(cases), "workload_id": wid, "n_matrices": len(cases),
                      "call": ("one dion_step_grouped call per step" if grouped else
                               "ten consecutive dion_step calls per step" if reps_per_step > 1 else
                               "one dion_step call per matrix per step"),
                      "engine": ["auto", "simt", "tensor"][args.engine],
                      "precision": ["fp32 (Orthonormalize 3xTF32; R, the error feedback and, on large matrices, P on bf16 "
                                    "(hi, lo) pairs, 16 significant bits, where M + G is kept in scratch, P recomputed in "
                                    "3xTF32 when the orthogonality probe asks; the X update one pass on factors rounded to "
                                    "IEEE half (11 significant bits); FMA for ragged shapes)", "bf16 operands"][args.precision],
                      "orth": ["auto", "cholqr2", "shifted3", "householder", "rcqr"][args.orth],
                      "sync": ("compressed data-parallel sync: P and W all-reduced (mean) over the ranks"
                               if args.sync == "dp" else "none (independent replicas)"),
                      "rule": ("Lazy-Dion (Algorithm 6), refresh every %d steps" % args.lazy) if args.lazy else "Dion (Algorithm 1 + 2)",
                      "form": args.form, "n_transposed": n_transposed,
                      "l2": ("inputs larger than L2: the workload's X, M, G (GBs) cycle through between repeats"
                             if wid != "config1" else
                             "1.5 MB of state: L2 resident by nature (launch-latency bound case)"),
                      "replicas": world, "workspace_bytes": need},
           "cases": ([] if len(cases) > 32 else
                     [case_report(c, ms, nr, args, peaks, binding) for c, ms, nr in zip(cases, case_ms, case_rounds)]),
           "phases": phases, "roofline": roof,
           "e2e": {"value": e2e_ms, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                   "calls_per_step": e2e_calls},
           "gpu_launches": launches, "launches_per_step": launches / args.steps, "clocks": clocks,
           "device_status": {"warmup": status, "timed": status2, "e2e": status3, "steps_skipped": skipped}}
    if reps_per_step > 1:
        rec["us_per_dion_step"] = ms_step * 1e3 / reps_per_step
        rec["launches_per_dion_step"] = launches / args.steps / reps_per_step
    return rec


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2504_05295_b200 import binding, build, inputs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    build.build()
    dev = torch.device("cuda", local)
    if args.cases:
        wids = ["custom"]
    elif args.workload == "all":
        wids = list(ALL_WORKLOADS)
    else:
        wids = [args.workload]
    if (args.sync == "dp" or args.lazy) and (args.form != "standard" or args.orth == 4):
        raise SystemExit("--sync dp and --lazy step single matrices in the standard form")
    top = HEADLINE if HEADLINE in wids else wids[-1]
    want_cpu = world == 1 and not args.no_cpu
    ctx = {"world": world, "rank": rank, "local": local, "dev": dev, "peaks": load_peaks(), "want_cpu": want_cpu,
           "cpu_wid": top}
    records = {}
    for wid in wids:
        cases = parse_cases(args.cases, inputs, wid)
        grouped = wid in ("llama8b", "llama405b") and not args.cases and args.sync != "dp" and not args.lazy
        if (args.sync == "dp" or args.lazy) and wid in ("llama8b", "llama405b"):
            continue
        records[wid] = run_workload(wid, cases, grouped, args, ctx)
    if top not in records:
        top = list(records)[-1]
    tf32_measured = measure_tf32_peak(torch, binding) if (rank == 0 and args.engine != binding.ENGINE_SIMT) else None
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- CPU baseline: the oracle on a bounded sample of the headline workload (rank 0, N = 1 only) ----
    cpu = None
    if want_cpu:
        cases = parse_cases(args.cases, inputs, top)
        sample = oracle_sample_cases(cases, top)
        ms_o, cores = time_oracle(sample, 1, 0, any(case_gbytes(c) == 2 for c in cases))
        cpu = {"value": ms_o, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": "one float64 oracle step each on " + sample_text(sample) + " (the two cheapest shape classes of "
                         "the workload when it has several); value = their summed host time",
               "gpu_ms_same_cases": records[top].get("sample_gpu_ms")}

    rec = records[top]
    peaks = ctx["peaks"]
    line = {"metric": METRIC, "value": rec["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": rec["value"], "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if args.precision == binding.PREC_BF16_OPERANDS else "f32",
            "data": "synthetic", "config": rec["config"], "cases": rec["cases"], "phases": rec["phases"],
            "roofline": rec["roofline"], "cpu_baseline": cpu, "e2e": rec["e2e"], "gpu_launches": rec["gpu_launches"],
            "clocks": rec["clocks"], "device_status": rec["device_status"],
            "peaks": {"hbm_gbs": peaks["hbm_gbs"], "bf16_tflops_sustained": peaks["bf16_sustained"],
                      "tf32_assumed_tflops": 0.5 * peaks["bf16_sustained"],
                      "tf32_single_pass_measured_tflops": tf32_measured, "source": peaks["source"],
                      "tf32_note": "measured: this library's single-pass TF32 contraction on 8192^3 (burst, best of 5); "
                                   "the roofline fractions use the assumed figure"},
            "workloads": {w: {k: v for k, v in r.items() if k != "sample_gpu_ms"} for w, r in records.items()}}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="all", choices=["all"] + ALL_WORKLOADS,
                    help="all (default): the five workloads one after another, the headline being llama8b; or one of them")
    ap.add_argument("--cases", default="", help="a custom list of single matrices instead: d:r or mxn:r[:bf16], comma separated")
    ap.add_argument("--engine", type=int, default=0, help="0 auto, 1 simt, 2 tensor")
    ap.add_argument("--precision", type=int, default=0, help="0 fp32, 1 bf16 operands")
    ap.add_argument("--orth", type=int, default=0, help="0 auto, 1 cholqr2, 2 shifted3, 3 householder, 4 randomized Cholesky QR")
    ap.add_argument("--form", default="standard", choices=["standard", "short-side"],
                    help="short-side: matrices with m > n take the transposed form (panel n x r instead of m x r)")
    ap.add_argument("--lazy", type=int, default=0,
                    help="K > 0: Lazy-Dion (Algorithm 6): dion_lazy_step with a SymPowerIter1 refresh every K-th step "
                         "instead of dion_step; single matrices, standard form")
    ap.add_argument("--sync", default="replicas", choices=["replicas", "dp"],
                    help="dp: compressed data-parallel sync (P and W all-reduced over the ranks, same X and Q on "
                         "every rank) instead of independent replicas; standard form, not for the grouped workloads")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-baseline leg")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
