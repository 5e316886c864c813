"""Parity of the CUDA library (through the C-ABI) with the float64 CPU oracle on
the same seeded inputs.  Needs a B200; run with ``-m gpu``.

Tolerances: relative Frobenius error <= 1e-4 on X, M and Q for the fp32 path and
<= 3e-2 for the bf16-operand path, after 1 and after 10 steps.
"""
import numpy as np
import pytest
import torch

from helpers import (EPS, ETA, MU, TOL_BF16, TOL_FP32, check_conditioned, device_state, movement_tol, one_step_movement,
                     oracle_steps, oracle_steps_fp32_panel, rel, to_np64)
from paper_2504_05295_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available(), "GPU tests selected but no CUDA device is visible"
    binding.load_library()


def run_gpu(pb, steps, grads=None, **cfg):
    X, M, Q = device_state(pb)
    d = torch.zeros(pb.r, device="cuda")
    snaps = []
    with binding.Dion(mu=MU, eps=EPS, **cfg) as opt:
        for t in range(steps):
            G = (grads[t] if grads is not None else pb.grad(t)).to("cuda")
            opt.step(X, M, G, Q, ETA, colnorm_out=d)
            snaps.append((to_np64(X), to_np64(M), to_np64(Q), to_np64(d)))
        status, skipped = opt.get_status()
        launches = opt.launch_count()
    assert launches > 0
    return snaps, status, skipped


def check(snap, res, tol, tag=""):
    ex, em, eq = rel(snap[0], res.X), rel(snap[1], res.M), rel(snap[2], res.Q)
    ed = rel(snap[3], res.d)
    assert ex <= tol and em <= tol and eq <= tol and ed <= tol, \
        f"{tag}: X {ex:.2e} M {em:.2e} Q {eq:.2e} d {ed:.2e} (tol {tol:.0e})"


ENGINES = [binding.ENGINE_SIMT, binding.ENGINE_AUTO]


@pytest.mark.parametrize("engine", ENGINES)
@pytest.mark.parametrize("orth", [binding.ORTH_AUTO, binding.ORTH_CHOLQR2, binding.ORTH_SHIFTED3,
                                  binding.ORTH_HOUSEHOLDER])
def test_config1_after_1_and_10_steps(engine, orth):
    m, n, r, ks = inputs.config1()
    pb = inputs.make_problem(m, n, r, seed=0, ks=ks)
    ref = oracle_steps(pb, 10)
    snaps, status, skipped = run_gpu(pb, 10, engine=engine, orth=orth)
    assert status == 0 and skipped == 0
    check(snaps[0], ref[0], TOL_FP32, "step 1")
    check(snaps[9], ref[9], TOL_FP32, "step 10")


@pytest.mark.parametrize("engine", ENGINES)
@pytest.mark.parametrize("m,n,r", [(1, 1, 1), (5, 3, 2), (3, 5, 3), (130, 70, 1), (257, 129, 33),
                                   (200, 333, 65), (129, 1000, 129), (640, 384, 160)])
def test_ragged_shapes_all_tiles_and_tails(engine, m, n, r):
    pb = inputs.make_problem(m, n, r, seed=3, ks=min(8, m, n))
    ref = oracle_steps(pb, 3)
    snaps, status, skipped = run_gpu(pb, 3, engine=engine)        # AUTO at every rank fraction
    assert status == 0 and skipped == 0
    if r < min(m, n):
        check(snaps[0], ref[0], TOL_FP32, "step 1")
        check(snaps[2], ref[2], TOL_FP32, "step 3")
    else:
        # full-rank panels are ill conditioned: the bar is 1e-4 or what the float64 rule itself moves by
        # under a float32 panel, whichever is larger (helpers.py)
        moved = oracle_steps_fp32_panel(pb, 3)
        check_conditioned(snaps[0], ref[0], moved[0], f"{m}x{n} r={r} step 1")
        check_conditioned(snaps[2], ref[2], moved[2], f"{m}x{n} r={r} step 3")


@pytest.mark.parametrize("engine", ENGINES)
def test_strided_leading_dimensions(engine):
    m, n, r = 192, 320, 48
    pb = inputs.make_problem(m, n, r, seed=4, ks=8)
    ref = oracle_steps(pb, 2)
    def padded(t, pad):
        buf = torch.full((t.shape[0], t.shape[1] + pad), 7.0, device="cuda", dtype=t.dtype)
        v = buf[:, :t.shape[1]]
        v.copy_(t)
        return buf, v
    Xb, X = padded(pb.X, 4); Mb, M = padded(pb.M, 8); Qb, Q = padded(pb.Q, 12)
    with binding.Dion(mu=MU, eps=EPS, engine=engine) as opt:
        for t in range(2):
            Gb, G = padded(pb.grad(t), 16)
            opt.step(X, M, G, Q, ETA)
        assert opt.get_status() == (0, 0)
    assert rel(to_np64(X), ref[1].X) <= TOL_FP32 and rel(to_np64(M), ref[1].M) <= TOL_FP32
    assert rel(to_np64(Q), ref[1].Q) <= TOL_FP32
    # the padding columns were never written
    assert torch.all(Xb[:, n:] == 7.0) and torch.all(Mb[:, n:] == 7.0) and torch.all(Qb[:, r:] == 7.0)


@pytest.mark.parametrize("shape", [(512, 768, 128), (2048, 2048, 512)])
def test_grouped_chain_with_mixed_leading_dimensions_equals_single_calls(shape):
    # three matrices of one shape in a chain, one of them with padded leading dimensions (and one with only its Q
    # padded): the chain-wide launches need common leading dimensions, so these chains fall back to one launch per
    # matrix where they must -- same bits as single calls, padding untouched
    m, n, r = shape
    pbs = [inputs.make_problem(m, n, r, seed=81, k=k, ks=16) for k in range(3)]

    def padded(t, pad):
        buf = torch.full((t.shape[0], t.shape[1] + pad), 7.0, device="cuda", dtype=t.dtype)
        v = buf[:, :t.shape[1]]
        v.copy_(t)
        return buf, v

    def make_state():
        out = []
        for k, pb in enumerate(pbs):
            px, pm, pq, pg = [(0, 0, 0, 0), (8, 4, 12, 16), (0, 0, 8, 0)][k]
            Xb, X = padded(pb.X, px); Mb, M = padded(pb.M, pm); Qb, Q = padded(pb.Q, pq); Gb, G = padded(pb.grad(0), pg)
            out.append((X, M, G, Q, (Xb, Mb, Qb)))
        return out

    with binding.Dion(mu=MU, eps=EPS) as opt:
        single = make_state()
        for X, M, G, Q, _ in single:
            opt.step(X, M, G, Q, ETA)
        grouped = make_state()
        opt.step_grouped([(X, M, G, Q) for X, M, G, Q, _ in grouped], ETA)
        assert opt.get_status() == (0, 0)
    for k, (a, b) in enumerate(zip(single, grouped)):
        for name, u, v in zip("XMQ", (a[0], a[1], a[3]), (b[0], b[1], b[3])):
            assert torch.equal(u, v), f"matrix {k}: {name} differs between dion_step and dion_step_grouped"
        Xb, Mb, Qb = b[4]
        assert torch.all(Xb[:, n:] == 7.0) and torch.all(Mb[:, n:] == 7.0) and torch.all(Qb[:, r:] == 7.0)
    ref = oracle_steps(pbs[1], 1)[0]
    assert rel(to_np64(grouped[1][0]), ref.X) <= TOL_FP32 and rel(to_np64(grouped[1][3]), ref.Q) <= TOL_FP32


@pytest.mark.parametrize("engine", ENGINES)
def test_bf16_gradient_storage(engine):
    m, n, r = 512, 384, 96
    pb = inputs.make_problem(m, n, r, seed=5, ks=16, g_dtype=torch.bfloat16)
    ref = oracle_steps(pb, 3)       # the oracle consumes the bf16-rounded values, up-cast exactly
    snaps, status, skipped = run_gpu(pb, 3, engine=engine)
    assert status == 0 and skipped == 0
    check(snaps[2], ref[2], TOL_FP32, "bf16 G, fp32 arithmetic")


@pytest.mark.parametrize("m,n,r,gdt", [(1024, 768, 192, torch.bfloat16), (768, 1024, 192, torch.float32),
                                       (2048, 2048, 512, torch.bfloat16), (1000, 776, 100, torch.bfloat16),
                                       (644, 388, 68, torch.float32)])
def test_bf16_operand_mode_within_its_bar(m, n, r, gdt):
    # shapes whose dimensions are multiples of 8 run the four products on bf16 arrays formed once per
    # step; the others round fp32 tiles to bf16 inside the kernel
    pb = inputs.make_problem(m, n, r, seed=6, ks=32, g_dtype=gdt)
    ref = oracle_steps(pb, 10)
    snaps, status, skipped = run_gpu(pb, 10, precision=binding.PREC_BF16_OPERANDS)
    assert status == 0 and skipped == 0
    check(snaps[0], ref[0], TOL_BF16, "step 1")
    check(snaps[9], ref[9], TOL_BF16, "step 10")


def test_bf16_operand_mode_grouped_equals_single_calls():
    shapes = [(512, 256, 64), (256, 512, 64), (512, 256, 64), (384, 384, 96)]
    pbs = [inputs.make_problem(m, n, r, seed=8, k=k, ks=16, g_dtype=torch.bfloat16) for k, (m, n, r) in enumerate(shapes)]
    with binding.Dion(mu=MU, eps=EPS, precision=binding.PREC_BF16_OPERANDS) as opt:
        single = []
        for pb in pbs:
            X, M, Q = device_state(pb)
            opt.step(X, M, pb.grad(0).cuda(), Q, ETA)
            single.append((X, M, Q))
        grouped = [device_state(pb) for pb in pbs]
        opt.step_grouped([(X, M, pb.grad(0).cuda(), Q) for pb, (X, M, Q) in zip(pbs, grouped)], ETA)
        assert opt.get_status() == (0, 0)
    for k, (a, b) in enumerate(zip(single, grouped)):
        for name, u, v in zip("XMQ", a, b):
            assert torch.equal(u, v), f"matrix {k}: {name} differs"


@pytest.mark.parametrize("engine", ENGINES)
@pytest.mark.parametrize("m,n,r", [(2048, 2048, 512), (2048, 2048, 128), (1024, 4096, 256), (4096, 1024, 256)])
def test_multi_tile_sizes(engine, m, n, r):
    pb = inputs.make_problem(m, n, r, seed=7, ks=64)
    ref = oracle_steps(pb, 2)
    snaps, status, skipped = run_gpu(pb, 2, engine=engine)
    assert status == 0 and skipped == 0
    check(snaps[0], ref[0], TOL_FP32, "step 1")
    check(snaps[1], ref[1], TOL_FP32, "step 2")


@pytest.mark.parametrize("engine", ENGINES)
def test_full_rank_square_shifted_cholqr3(engine):
    d = 1024
    pb = inputs.make_problem(d, d, d, seed=8, ks=64)
    ref = oracle_steps(pb, 3)
    snaps, status, skipped = run_gpu(pb, 3, engine=engine)      # AUTO picks the shifted rounds
    assert status == 0 and skipped == 0
    check(snaps[0], ref[0], TOL_FP32, "step 1")
    check(snaps[2], ref[2], TOL_FP32, "step 3")
    # closed form at full rank: M_new = mu (M + G)
    B = to_np64(pb.M) + to_np64(pb.grad(0))
    assert rel(snaps[0][1], MU * B) <= TOL_FP32


def test_grouped_equals_single_calls():
    shapes = [(256, 512, 64), (512, 256, 64), (384, 384, 96), (256, 512, 64), (130, 70, 10)]
    pbs = [inputs.make_problem(m, n, r, seed=9, k=k, ks=8) for k, (m, n, r) in enumerate(shapes)]
    single, grouped = [], []
    with binding.Dion(mu=MU, eps=EPS) as opt:
        for pb in pbs:
            X, M, Q = device_state(pb)
            for t in range(2):
                opt.step(X, M, pb.grad(t).cuda(), Q, ETA)
            single.append((X, M, Q))
        states = [device_state(pb) for pb in pbs]
        for t in range(2):
            opt.step_grouped([(X, M, pb.grad(t).cuda(), Q) for pb, (X, M, Q) in zip(pbs, states)], ETA)
        opt.step_grouped([], ETA)      # empty list is a no-op
        assert opt.get_status() == (0, 0)
    for (X1, M1, Q1), (X2, M2, Q2), pb in zip(single, states, pbs):
        assert torch.equal(X1, X2) and torch.equal(M1, M2) and torch.equal(Q1, Q2)
        ref = oracle_steps(pb, 2)
        assert rel(to_np64(X2), ref[1].X) <= TOL_FP32 and rel(to_np64(Q2), ref[1].Q) <= TOL_FP32


@pytest.mark.parametrize("shape,count", [((1024, 4096, 256), 5), ((4096, 4096, 1024), 3), ((2560, 1536, 640), 3),
                                         ((1280, 1280, 1280), 2), ((1400, 1100, 700), 3), ((512, 2048, 512), 4)])
def test_chain_products_in_one_launch_equal_one_launch_per_matrix(shape, count):
    # the tensor-engine products of a grouped chain run as one launch over (matrix, tile) pairs; with the test hook
    # that turns this off they run matrix by matrix: same bits, fewer launches
    import ctypes
    m, n, r = shape
    pbs = [inputs.make_problem(m, n, r, seed=41, k=k, ks=32) for k in range(count)]
    lib = binding.load_library()
    lib.dion_debug_chain_batch.argtypes = [ctypes.c_void_p, ctypes.c_int]
    lib.dion_debug_chain_batch.restype = ctypes.c_int
    results, launches = [], []
    for on in (1, 0):
        with binding.Dion(mu=MU, eps=EPS) as opt:
            assert lib.dion_debug_chain_batch(opt._ctx, on) == 0
            states = [device_state(pb) for pb in pbs]
            for t in range(2):
                l0 = opt.launch_count()
                opt.step_grouped([(X, M, pb.grad(t).cuda(), Q) for pb, (X, M, Q) in zip(pbs, states)], ETA)
            launches.append(opt.launch_count() - l0)
            assert opt.get_status() == (0, 0)
        results.append(states)
    for k, ((X1, M1, Q1), (X2, M2, Q2)) in enumerate(zip(*results)):
        assert torch.equal(X1, X2) and torch.equal(M1, M2) and torch.equal(Q1, Q2), k
    print(f"{shape} x {count}: {launches[0]} launches batched, {launches[1]} per matrix")
    assert launches[0] < launches[1]


@pytest.mark.parametrize("shape,orth", [((2560, 1536, 640), binding.ORTH_AUTO), ((1280, 1280, 1280), binding.ORTH_AUTO),
                                        # ragged: a second square of 188 columns (blocks of 64, 64, 60)
                                        ((1400, 1100, 700), binding.ORTH_AUTO), ((3000, 2900, 700), binding.ORTH_AUTO)])
def test_grouped_chain_above_512_columns_equals_single_calls(shape, orth):
    # r > 512: two-level Cholesky, blocked solves on the second stream, three matrices sharing every small launch
    m, n, r = shape
    pbs = [inputs.make_problem(m, n, r, seed=12, k=k, ks=32) for k in range(3)]
    with binding.Dion(mu=MU, eps=EPS, orth=orth) as opt:
        single = []
        for pb in pbs:
            X, M, Q = device_state(pb)
            opt.step(X, M, pb.grad(0).cuda(), Q, ETA)
            single.append((X, M, Q))
        states = [device_state(pb) for pb in pbs]
        opt.step_grouped([(X, M, pb.grad(0).cuda(), Q) for pb, (X, M, Q) in zip(pbs, states)], ETA)
        assert opt.get_status() == (0, 0)
    for k, ((X1, M1, Q1), (X2, M2, Q2)) in enumerate(zip(single, states)):
        assert torch.equal(X1, X2) and torch.equal(M1, M2) and torch.equal(Q1, Q2), k
    ref = oracle_steps(pbs[0], 1)[0]
    tol = TOL_FP32
    if r == min(m, n):      # ill-conditioned panel: the conditioned bar of helpers.py
        pb = pbs[0]
        tol = movement_tol(one_step_movement(to_np64(pb.X), to_np64(pb.M), to_np64(pb.grad(0)), to_np64(pb.Q)))["X"]
    assert rel(to_np64(states[0][1]), ref.M) <= TOL_FP32 and rel(to_np64(states[0][0]), ref.X) <= tol


@pytest.mark.parametrize("m,n,r,precision", [(2048, 2048, 2048, binding.PREC_FP32), (3072, 2048, 1024, binding.PREC_FP32),
                                             (2048, 2048, 768, binding.PREC_BF16_OPERANDS)])
def test_repeated_runs_are_bit_identical(m, n, r, precision):
    # the look-ahead on the library's second stream and the dependent launches must not make a step
    # depend on timing: the same two steps from the same state give the same bits every time
    pb = inputs.make_problem(m, n, r, seed=13, ks=64, device="cuda", keep_signal=False)
    gs = [pb.grad(t) for t in range(2)]
    ref = None
    with binding.Dion(mu=MU, eps=EPS, precision=precision) as opt:
        for rep in range(3):
            X, M, Q = pb.X.clone(), pb.M.clone(), pb.Q.clone()
            for t in range(2):
                opt.step(X, M, gs[t], Q, ETA)
            torch.cuda.synchronize()
            if ref is None:
                ref = (X, M, Q)
            else:
                assert all(torch.equal(a, b) for a, b in zip(ref, (X, M, Q))), rep
        assert opt.get_status() == (0, 0)


@pytest.mark.parametrize("shape", [(2048, 1536, 256), (1024, 768, 100), (4096, 4096, 1024)])
def test_orthogonality_probe_estimates_the_frobenius_deviation(shape):
    # the device's estimate of |U1^T U1 - I|_F^2 (8 fixed sign vectors, two passes over the panel) against the same
    # quantity computed in float64 from the U the step used (one round passed, so U = U1).  r a multiple of 4 from
    # 128 up takes the kernel with the sign table in shared memory, smaller or odd r the plain one.
    import ctypes
    m, n, r = shape
    pb = inputs.make_problem(m, n, r, seed=71, ks=32, device="cuda")
    lib = binding.load_library()
    lib.dion_debug_orth_measure.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(ctypes.c_float)]
    lib.dion_debug_orth_measure.restype = ctypes.c_int
    P = torch.empty(m, r, device="cuda")
    W = torch.empty(n, r, device="cuda")
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    with binding.Dion(mu=MU, eps=EPS, orth=binding.ORTH_CHOLQR2) as opt:
        desc = binding.matrix_desc(pb.X, pb.M, pb.grad(0), pb.Q)
        opt.dp_project(desc, P, flag)
        opt.dp_factor(desc, P, W, flag)
        assert opt.get_status() == (0, 0) and opt.orth_rounds() == 1
        est = ctypes.c_float(0.0)
        assert lib.dion_debug_orth_measure(opt._ctx, ctypes.c_void_p(int(torch.cuda.current_stream().cuda_stream)),
                                           ctypes.byref(est)) == 0
    U = P.double()
    true = float(((U.t() @ U - torch.eye(r, device="cuda", dtype=torch.float64)) ** 2).sum())
    print(f"{shape}: estimate {est.value:.3e}, |U^T U - I|_F^2 {true:.3e}")
    assert 0.4 * true <= est.value <= 2.5 * true
    assert est.value <= (3e-5) ** 2 * r          # what let the device skip the second round


def test_cholqr2_takes_its_second_round_only_when_the_first_is_not_enough():
    m, n, r = 1024, 768, 128
    pb = inputs.make_problem(m, n, r, seed=15, ks=16)
    G = pb.grad(0)
    # (i) the workload's own warm start: cond(P) of a few units -> one round passes the device's check
    X, M, Q = device_state(pb)
    with binding.Dion(mu=MU, eps=EPS, orth=binding.ORTH_CHOLQR2) as opt:
        opt.step(X, M, G.cuda(), Q, ETA)
        assert opt.get_status() == (0, 0) and opt.orth_rounds() == 1
    ref = oracle_steps(pb, 1)[0]
    assert rel(to_np64(Q), ref.Q) <= TOL_FP32 and rel(to_np64(M), ref.M) <= TOL_FP32 and rel(to_np64(X), ref.X) <= TOL_FP32
    # (ii) a warm start whose columns are nearly parallel (every column = the first one + 3 % of its own:
    # cond(P) in the hundreds, not curable by column scaling): the first round's result fails the check,
    # the second round runs, and the outputs still meet the bar
    Qbad = pb.Q[:, :1] + 0.03 * pb.Q
    Qbad = Qbad / Qbad.norm(dim=0)
    from oracle import dion_oracle as orc
    want = orc.step(to_np64(pb.X), to_np64(pb.M), to_np64(G), to_np64(Qbad), MU, ETA, EPS)
    X, M, Q = pb.X.cuda().clone(), pb.M.cuda().clone(), Qbad.cuda().clone()
    with binding.Dion(mu=MU, eps=EPS, orth=binding.ORTH_CHOLQR2) as opt:
        opt.step(X, M, G.cuda(), Q, ETA)
        assert opt.get_status() == (0, 0) and opt.orth_rounds() == 2
    assert rel(to_np64(M), want.M) <= TOL_FP32 and rel(to_np64(X), want.X) <= TOL_FP32
    # cond(P) is in the hundreds here: Q is held to 1e-4 or to what the float64 rule moves by under a float32
    # panel on this input, whichever is larger
    tolq = movement_tol(one_step_movement(to_np64(pb.X), to_np64(pb.M), to_np64(G), to_np64(Qbad)))["Q"]
    eq = rel(to_np64(Q), want.Q)
    print(f"nearly parallel warm start: Q {eq:.2e} / {tolq:.1e}")
    assert eq <= tolq


def test_checkpoint_resume_is_bit_identical():
    m, n, r, ks = inputs.config1()
    pb = inputs.make_problem(m, n, r, seed=0, ks=ks)
    grads = [pb.grad(t).cuda() for t in range(10)]
    X, M, Q = device_state(pb)
    with binding.Dion(mu=MU, eps=EPS) as opt:
        for t in range(10):
            opt.step(X, M, grads[t], Q, ETA)
        torch.cuda.synchronize()
    X2, M2, Q2 = device_state(pb)
    with binding.Dion(mu=MU, eps=EPS) as opt:
        for t in range(5):
            opt.step(X2, M2, grads[t], Q2, ETA)
        torch.cuda.synchronize()
    saved = [t.cpu().clone() for t in (X2, M2, Q2)]          # "checkpoint": state is X, M, Q only
    X3, M3, Q3 = [t.cuda() for t in saved]
    with binding.Dion(mu=MU, eps=EPS) as opt:                # a fresh context: the library is stateless
        for t in range(5, 10):
            opt.step(X3, M3, grads[t], Q3, ETA)
        torch.cuda.synchronize()
    assert torch.equal(X, X3) and torch.equal(M, M3) and torch.equal(Q, Q3)


def test_breakdown_is_flagged_and_leaves_state_untouched():
    # a rank-deficient right factor (two equal columns) makes P = B Q rank deficient:
    # outside the contract for parity, but it must be reported, finite and transactional
    m, n, r = 256, 320, 32
    pb = inputs.make_problem(m, n, r, seed=11, ks=8)
    X, M, Q = device_state(pb)
    Q[:, 5] = Q[:, 4]
    Q[:, 9] = 0.0
    X0, M0, Q0 = X.clone(), M.clone(), Q.clone()
    G = pb.grad(0).cuda()
    with binding.Dion(mu=MU, eps=EPS, orth=binding.ORTH_CHOLQR2) as opt:
        opt.step(X, M, G, Q, ETA)
        status, skipped = opt.get_status()
        assert status & binding.STATUS_BREAKDOWN and skipped == 1
        assert torch.equal(X, X0) and torch.equal(M, M0) and torch.equal(Q, Q0)
        assert opt.get_status() == (0, 0)                    # reading clears the latch
        # the context stays usable: a healthy step afterwards matches the oracle
        Xh, Mh, Qh = device_state(pb)
        opt.step(Xh, Mh, G, Qh, ETA)
        assert opt.get_status() == (0, 0)
    ref = oracle_steps(pb, 1)
    assert rel(to_np64(Xh), ref[0].X) <= TOL_FP32 and rel(to_np64(Qh), ref[0].Q) <= TOL_FP32


def test_zero_gradient_and_momentum_is_finite():
    m, n, r = 128, 96, 8
    pb = inputs.make_problem(m, n, r, seed=12, ks=4)
    X, M, Q = device_state(pb)
    G = torch.zeros(m, n, device="cuda")
    for orth in (binding.ORTH_CHOLQR2, binding.ORTH_HOUSEHOLDER):
        with binding.Dion(mu=MU, eps=EPS, orth=orth) as opt:
            opt.step(X, M, G, Q, ETA)
            opt.get_status()
        assert all(bool(torch.isfinite(t).all()) for t in (X, M, Q))


def test_argument_errors():
    pb = inputs.make_problem(64, 48, 8, seed=13, ks=4)
    X, M, Q = device_state(pb)
    G = pb.grad(0).cuda()
    with binding.Dion() as opt:
        with pytest.raises(binding.DionError) as e:
            opt.step(X, M, G, Q[:, :0], ETA)                 # r = 0 (an empty view has a NULL pointer)
        assert e.value.code in (-1, -2)
        with pytest.raises(binding.DionError) as e:
            opt.step(X, X, G, Q, ETA)                        # aliasing
        assert e.value.code == -4
        big = torch.zeros(48, 49, device="cuda")
        with pytest.raises(binding.DionError) as e:
            opt.step(X, M, G, big, ETA)                      # r > min(m, n)
        assert e.value.code == -2
        opt.step(X, M, G, Q, ETA)
        assert opt.get_status() == (0, 0)


@pytest.mark.parametrize("m,n,r,precision", [(384, 256, 32, binding.PREC_FP32), (1536, 1024, 128, binding.PREC_FP32),
                                             (1536, 1024, 128, binding.PREC_BF16_OPERANDS),
                                             (1000, 776, 100, binding.PREC_BF16_OPERANDS)])
def test_lazy_dion_steps_match_oracle(m, n, r, precision):
    from oracle import dion_oracle as orc
    pb = inputs.make_problem(m, n, r, seed=14, ks=8)
    X, M, Q = device_state(pb)
    Xo, Mo, Qo = to_np64(pb.X), to_np64(pb.M), to_np64(pb.Q)
    d = torch.zeros(r, device="cuda")
    tol = TOL_FP32 if precision == binding.PREC_FP32 else TOL_BF16
    with binding.Dion(mu=MU, eps=EPS, precision=precision) as opt:
        for t in range(6):
            refresh = (t % 3 == 0)
            G = pb.grad(t)
            opt.lazy_step(X, M, G.cuda(), Q, ETA, refresh, colnorm_out=d)
            Xo, Mo, Qo, do = orc.lazy_step(Xo, Mo, to_np64(G), Qo, MU, ETA, EPS, refresh=refresh)
        assert opt.get_status() == (0, 0)
    assert rel(to_np64(X), Xo) <= tol and rel(to_np64(M), Mo) <= tol
    assert rel(to_np64(Q), Qo) <= tol and rel(to_np64(d), do) <= tol


# ---------------------------------------------------------------------------
# Benchmark-size cases.  One full-size element-wise comparison that the oracle
# finishes in tens of seconds, then properties that hold at any size, evaluated in
# float64 on the device (test-side arithmetic; the step itself is the library's).
# ---------------------------------------------------------------------------

def test_4096_square_quarter_rank_against_oracle():
    m = n = 4096
    r = 1024
    pb = inputs.make_problem(m, n, r, seed=15, ks=64)
    ref = oracle_steps(pb, 1)
    snaps, status, skipped = run_gpu(pb, 1)
    assert status == 0 and skipped == 0
    check(snaps[0], ref[0], TOL_FP32, "4096^2 r=1024, step 1")


def step_properties(m, n, r, g_dtype, tol=TOL_FP32, precision=binding.PREC_FP32, steps=2):
    """Runs `steps` library steps on device-generated inputs and checks, in float64, what the rule fixes for
    the last one.  U is the one the library computes for that step (handed out by the data-parallel entry
    points from the same state); R is read back from the outputs, R = Q' diag(d + eps)."""
    pb = inputs.make_problem(m, n, r, seed=16, ks=64, g_dtype=g_dtype, device="cuda", keep_signal=False)
    X, M, Q = pb.X, pb.M, pb.Q
    d = torch.zeros(r, device="cuda")
    Pbuf = torch.empty(m, r, device="cuda")
    Wbuf = torch.empty(n, r, device="cuda")
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    with binding.Dion(mu=MU, eps=EPS, precision=precision) as opt:
        for t in range(steps):
            G = pb.grad(t)
            if t == steps - 1:
                X0, M0 = X.clone(), M.clone()
                desc = binding.matrix_desc(X, M, G, Q)
                opt.dp_project(desc, Pbuf, flag)
                opt.dp_factor(desc, Pbuf, Wbuf, flag)          # Pbuf <- U
            opt.step(X, M, G, Q, ETA, colnorm_out=d)
        assert opt.get_status() == (0, 0)
    del Wbuf
    s = ETA * (m / n) ** 0.5
    B = M0.double() + G.double()
    Qn = Q.double()
    U = Pbuf.double()
    R = Qn * (d.double() + EPS)
    eye = torch.eye(r, device="cuda", dtype=torch.float64)
    # in bf16-operand mode the data-parallel calls form their products from fp32 tiles while dion_step reads
    # bf16 copies made once: the two U agree to the mode's bar only
    tol_u = tol
    assert float((U.t() @ U - eye).abs().max()) <= TOL_FP32
    assert float(torch.linalg.norm(B.t() @ U - R) / torch.linalg.norm(R)) <= tol_u
    assert float(torch.linalg.norm(B - (1 - MU) * (U @ R.t()) - M.double()) / torch.linalg.norm(M.double())) <= tol
    nq = torch.linalg.norm(Qn, dim=0)
    assert float((nq - 1).abs().max()) <= 1e-5
    upd = float(torch.linalg.norm(X0.double() - X.double()))
    assert abs(upd - s * r ** 0.5) <= 1e-3 * s * r ** 0.5
    assert float(torch.linalg.norm(d.double() - torch.linalg.norm(B.t() @ U, dim=0)) / torch.linalg.norm(d.double())) <= tol_u
    # the update is built from this U and the Q' the step wrote (single-pass TF32 on rounded factors in fp32
    # mode, bf16 operands in bf16 mode; read back from fp32 X by subtraction)
    delta = (X0.double() - X.double()) / s
    assert float(torch.linalg.norm(delta - U @ Qn.t()) / torch.linalg.norm(delta)) <= max(10 * tol, 1e-3)


@pytest.mark.parametrize("m,n,r", [(8192, 8192, 512), (8192, 8192, 2048), (2048, 2048, 2048), (4096, 4096, 4096)])
def test_properties_on_the_square_sweep_sizes(m, n, r):
    step_properties(m, n, r, torch.float32)


@pytest.mark.parametrize("m,n,r", [(4096, 4096, 1024), (1024, 4096, 256), (14336, 4096, 1024), (4096, 14336, 1024)])
def test_properties_on_llama8b_shapes_bf16_gradients(m, n, r):
    step_properties(m, n, r, torch.bfloat16)


@pytest.mark.parametrize("m,n,r,gdt", [(8192, 8192, 512, torch.float32), (4096, 4096, 4096, torch.float32),
                                       (14336, 4096, 1024, torch.bfloat16), (16384, 16384, 1024, torch.float32)])
def test_properties_in_bf16_operand_mode_at_bench_sizes(m, n, r, gdt):
    step_properties(m, n, r, gdt, tol=TOL_BF16, precision=binding.PREC_BF16_OPERANDS, steps=2 if m < 16384 else 1)
    torch.cuda.empty_cache()


@pytest.mark.parametrize("m,n,r", [(16384, 16384, 1024), (32768, 32768, 512)])
def test_properties_on_the_large_square_sizes(m, n, r):
    step_properties(m, n, r, torch.float32, steps=1)
    torch.cuda.empty_cache()


@pytest.mark.parametrize("m,n,r", [(1024, 16384, 256), (53248, 16384, 1024), (16384, 53248, 1024)])
def test_properties_on_llama405b_shapes_bf16_gradients(m, n, r):
    step_properties(m, n, r, torch.bfloat16, steps=1)
    torch.cuda.empty_cache()


@pytest.mark.parametrize("m,n,r", [(1792, 512, 128), (512, 1792, 128), (128, 512, 32)])
def test_llama_aspect_ratios_bf16_gradients_against_oracle(m, n, r):
    pb = inputs.make_problem(m, n, r, seed=17, ks=32, g_dtype=torch.bfloat16)
    ref = oracle_steps(pb, 3)
    snaps, status, skipped = run_gpu(pb, 3)
    assert status == 0 and skipped == 0
    check(snaps[0], ref[0], TOL_FP32, "step 1")
    check(snaps[2], ref[2], TOL_FP32, "step 3")


def test_grouped_llama_like_block_list_against_oracle():
    # two "layers" of the seven block shapes, scaled down by 8, rank fraction 1/4, bf16 gradients
    shapes = [(nm, m // 8, n // 8) for nm, m, n in inputs.llama_block_shapes(4096, 1024, 14336)] * 2
    pbs = [inputs.make_problem(m, n, min(m, n) // 4, seed=18, k=k, ks=16, g_dtype=torch.bfloat16)
           for k, (nm, m, n) in enumerate(shapes)]
    states = [device_state(pb) for pb in pbs]
    with binding.Dion(mu=MU, eps=EPS) as opt:
        for t in range(2):
            opt.step_grouped([(X, M, pb.grad(t).cuda(), Q) for pb, (X, M, Q) in zip(pbs, states)], ETA)
        assert opt.get_status() == (0, 0)
    for pb, (X, M, Q) in zip(pbs, states):
        ref = oracle_steps(pb, 2)
        assert rel(to_np64(X), ref[1].X) <= TOL_FP32 and rel(to_np64(M), ref[1].M) <= TOL_FP32
        assert rel(to_np64(Q), ref[1].Q) <= TOL_FP32


# ---------------------------------------------------------------------------
# Failure handling on the device: Cholesky QR breakdown -> fallback; non-finite inputs
# ---------------------------------------------------------------------------

def _nearly_parallel(Q, delta):
    Qb = Q[:, :1] + delta * Q
    return (Qb / Qb.norm(dim=0)).contiguous()


@pytest.mark.parametrize("scale_exp", [-40, 20])
def test_gradient_scale_does_not_matter_to_the_16_bit_paths(scale_exp):
    # The Gram matrix of a tall panel runs on a pair of IEEE HALF arrays (5 exponent bits) after scaling the panel
    # by a power of two found on the device, and the X update on half factors whose entries are at most 1: neither
    # may depend on the scale of the gradient.  4096 x 4096 at r = 1024 takes both paths (and P on bf16 pairs);
    # gradients scaled by 2^-40 and 2^20 must give the oracle's X, M, Q on the same scaled inputs.
    from oracle import dion_oracle as orc
    m = n = 4096
    r = 1024
    pb = inputs.make_problem(m, n, r, seed=61, ks=64)
    sc = 2.0 ** scale_exp
    G = pb.grad(0) * sc
    M0 = (0.5 * pb.grad(1)) * sc                      # a non-zero momentum of the same scale
    want = orc.step(to_np64(pb.X), to_np64(M0), to_np64(G), to_np64(pb.Q), MU, ETA, EPS)
    X, M, Q = pb.X.cuda().clone(), M0.cuda().clone(), pb.Q.cuda().clone()
    d = torch.zeros(r, device="cuda")
    with binding.Dion(mu=MU, eps=EPS) as opt:
        opt.step(X, M, G.cuda(), Q, ETA, colnorm_out=d)
        assert opt.get_status() == (0, 0) and opt.orth_rounds() == 1 and opt.fallbacks() == 0
    errs = {"X": rel(to_np64(X), want.X), "M": rel(to_np64(M), want.M), "Q": rel(to_np64(Q), want.Q),
            "d": rel(to_np64(d), want.d)}
    print(f"gradient scale 2^{scale_exp}: " + " ".join(f"{k} {v:.2e}" for k, v in errs.items()))
    assert all(v <= TOL_FP32 for v in errs.values()), errs


def test_fast_panel_is_recomputed_when_the_probe_rejects_it():
    # 4096^2 at r = 1024 is large enough for P = (M + G) Q to run on bf16 operand pairs first (~1e-5).
    # (i) the workload's own warm start: well conditioned, the probe accepts the first round, one round of work,
    # the 1e-4 bar holds; (ii) a warm start with nearly parallel columns (cond(P) in the hundreds): the probe
    # rejects the round, the device recomputes P with the accurate product and repeats it (three rounds of work
    # counted), and the outputs meet the same conditioned bar as everywhere else; (iii) a grouped call mixing both
    # equals the single calls bit for bit
    from oracle import dion_oracle as orc
    m = n = 4096
    r = 1024
    pb = inputs.make_problem(m, n, r, seed=51, ks=64)
    G = pb.grad(0)
    Qbad = _nearly_parallel(pb.Q, 0.03)
    outs = []
    with binding.Dion(mu=MU, eps=EPS) as opt:
        for q0, rounds in ((pb.Q, 1), (Qbad, 3)):
            X, M, Q = pb.X.cuda().clone(), pb.M.cuda().clone(), q0.cuda().clone()
            opt.step(X, M, G.cuda(), Q, ETA)
            assert opt.get_status() == (0, 0) and opt.fallbacks() == 0
            assert opt.orth_rounds() == rounds
            want = orc.step(to_np64(pb.X), to_np64(pb.M), to_np64(G), to_np64(q0), MU, ETA, EPS)
            tol = movement_tol(one_step_movement(to_np64(pb.X), to_np64(pb.M), to_np64(G), to_np64(q0)))
            errs = {"X": rel(to_np64(X), want.X), "M": rel(to_np64(M), want.M), "Q": rel(to_np64(Q), want.Q)}
            print(f"rounds {rounds}: " + " ".join(f"{k} {v:.2e}/{tol[k]:.1e}" for k, v in errs.items()))
            assert all(errs[k] <= tol[k] for k in errs)
            if rounds == 1:
                assert errs["Q"] <= TOL_FP32
            outs.append((X, M, Q))
        grouped = [(pb.X.cuda().clone(), pb.M.cuda().clone(), q0.cuda().clone()) for q0 in (pb.Q, Qbad)]
        opt.step_grouped([(X, M, G.cuda(), Q) for X, M, Q in grouped], ETA)
        assert opt.get_status() == (0, 0)
    for a, b in zip(outs, grouped):
        for u, v in zip(a, b):
            assert torch.equal(u, v)


def test_cholesky_breakdown_falls_back_on_the_device():
    # rank fraction 1/8 through AUTO (CholeskyQR2) with a warm start whose columns are nearly parallel: the
    # Gram matrix of P is not positive definite in fp32, a pivot fails, and the same call redoes the panel with
    # the Gram-Schmidt fallback: no breakdown reported, no step skipped, outputs on the conditioned bar
    m, n, r = 1024, 1024, 128
    pb = inputs.make_problem(m, n, r, seed=41, ks=16)
    G = pb.grad(0)
    Qbad = _nearly_parallel(pb.Q, 1e-4)
    from oracle import dion_oracle as orc
    want = orc.step(to_np64(pb.X), to_np64(pb.M), to_np64(G), to_np64(Qbad), MU, ETA, EPS)
    cond = np.linalg.cond(want.P)
    X, M, Q = pb.X.cuda().clone(), pb.M.cuda().clone(), Qbad.cuda().clone()
    d = torch.zeros(r, device="cuda")
    with binding.Dion(mu=MU, eps=EPS) as opt:
        opt.step(X, M, G.cuda(), Q, ETA, colnorm_out=d)
        assert opt.get_status() == (0, 0)
        assert opt.fallbacks() == 1
        # a healthy step afterwards takes no fallback
        Xh, Mh, Qh = device_state(pb)
        opt.step(Xh, Mh, G.cuda(), Qh, ETA)
        assert opt.get_status() == (0, 0) and opt.fallbacks() == 0
    tol = movement_tol(one_step_movement(to_np64(pb.X), to_np64(pb.M), to_np64(G), to_np64(Qbad)))
    errs = {"X": rel(to_np64(X), want.X), "M": rel(to_np64(M), want.M), "Q": rel(to_np64(Q), want.Q),
            "d": rel(to_np64(d), want.d)}
    print(f"fallback, cond(P) {cond:.1e}: " + " ".join(f"{k} {errs[k]:.2e}/{tol[k]:.1e}" for k in errs))
    assert all(errs[k] <= tol[k] for k in errs), (errs, tol)


def test_fallback_inside_a_grouped_chain_touches_only_the_failed_matrix():
    m, n, r = 768, 512, 64
    pbs = [inputs.make_problem(m, n, r, seed=42, k=k, ks=16) for k in range(3)]
    Q0 = [pb.Q for pb in pbs]
    Q0[1] = _nearly_parallel(pbs[1].Q, 1e-4)
    with binding.Dion(mu=MU, eps=EPS) as opt:
        single = []
        for pb, q in zip(pbs, Q0):
            X, M, Q = pb.X.cuda().clone(), pb.M.cuda().clone(), q.cuda().clone()
            opt.step(X, M, pb.grad(0).cuda(), Q, ETA)
            single.append((X, M, Q))
        assert opt.get_status() == (0, 0) and opt.fallbacks() == 1
        grouped = [(pb.X.cuda().clone(), pb.M.cuda().clone(), q.cuda().clone()) for pb, q in zip(pbs, Q0)]
        opt.step_grouped([(X, M, pb.grad(0).cuda(), Q) for pb, (X, M, Q) in zip(pbs, grouped)], ETA)
        assert opt.get_status() == (0, 0) and opt.fallbacks() == 1
    for k, (a, b) in enumerate(zip(single, grouped)):
        for name, u, v in zip("XMQ", a, b):
            assert torch.equal(u, v), f"matrix {k}: {name} differs between dion_step and dion_step_grouped"
    ref = oracle_steps(pbs[0], 1)[0]
    assert rel(to_np64(grouped[0][2]), ref.Q) <= TOL_FP32


@pytest.mark.parametrize("m,n,r", [(512, 384, 64), (512, 512, 512)])
def test_non_finite_gradient_is_flagged_and_cancels_the_step(m, n, r):
    pb = inputs.make_problem(m, n, r, seed=43, ks=8)
    X, M, Q = device_state(pb)
    X0, M0, Q0 = X.clone(), M.clone(), Q.clone()
    G = pb.grad(0).cuda()
    G[17, 5] = float("nan")
    with binding.Dion(mu=MU, eps=EPS) as opt:
        opt.step(X, M, G, Q, ETA)
        status, skipped = opt.get_status()
        assert status & binding.STATUS_NONFINITE and skipped == 1
        assert torch.equal(X, X0) and torch.equal(M, M0) and torch.equal(Q, Q0)
        G[17, 5] = float("inf")
        opt.step(X, M, G, Q, ETA)
        status, skipped = opt.get_status()
        assert status & binding.STATUS_NONFINITE and skipped == 1
        assert torch.equal(X, X0) and torch.equal(M, M0) and torch.equal(Q, Q0)
        # the context stays usable
        opt.step(X, M, pb.grad(0).cuda(), Q, ETA)
        assert opt.get_status() == (0, 0)
    ref = oracle_steps(pb, 1)
    if r < min(m, n):
        assert rel(to_np64(X), ref[0].X) <= TOL_FP32 and rel(to_np64(Q), ref[0].Q) <= TOL_FP32


# ---------------------------------------------------------------------------
# Graph replay of launch-bound steps: small matrices are stepped by replaying a captured CUDA graph
# ---------------------------------------------------------------------------

def test_graph_replay_equals_the_plain_launch_chain_and_follows_the_learning_rate():
    m, n, r = 512, 384, 64
    pb = inputs.make_problem(m, n, r, seed=44, ks=16)
    grads = [pb.grad(t).cuda() for t in range(4)]
    lrs = [0.01, 0.02, 0.005, 0.01]
    # plain chain: profiling on keeps the library from replaying graphs
    Xa, Ma, Qa = device_state(pb)
    with binding.Dion(mu=MU, eps=EPS) as opt:
        opt.profile_enable(True)
        G = grads[0].clone()
        for t in range(4):
            G.copy_(grads[t])
            opt.step(Xa, Ma, G, Qa, lrs[t])
        opt.profile_enable(False)
        assert opt.get_status() == (0, 0)
    # replayed: the same descriptor every step (one gradient buffer, refilled), a different learning rate each time
    Xb, Mb, Qb = device_state(pb)
    with binding.Dion(mu=MU, eps=EPS) as opt:
        G = grads[0].clone()
        n0 = opt.launch_count()
        for t in range(4):
            G.copy_(grads[t])
            opt.step(Xb, Mb, G, Qb, lrs[t])
        assert opt.get_status() == (0, 0) and opt.launch_count() > n0
        # a second matrix and a non-default stream go through their own graph
        side = torch.cuda.Stream()
        Xc, Mc, Qc = device_state(pb)
        torch.cuda.synchronize()
        for t in range(4):
            G.copy_(grads[t])
            torch.cuda.synchronize()
            opt.step(Xc, Mc, G, Qc, lrs[t], stream=side)
            side.synchronize()
        assert opt.get_status(side) == (0, 0)
    for name, u, v, w in zip("XMQ", (Xa, Ma, Qa), (Xb, Mb, Qb), (Xc, Mc, Qc)):
        assert torch.equal(u, v), f"{name}: graph replay differs from the plain launch chain"
        assert torch.equal(u, w), f"{name}: graph replay on a side stream differs"
    ref = oracle_steps(pb, 1)
    # (the oracle comparison with eta = 0.01 after one step is covered elsewhere; here: finite and moved)
    assert torch.isfinite(Xb).all() and not torch.equal(Xb, pb.X.cuda())
