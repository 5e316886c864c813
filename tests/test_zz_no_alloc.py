"""dion_step_noalloc: the Dion step for host programs that cannot allocate device memory.

Some callers (a plug-in inside another framework's memory pool that owns the whole
GPU, a process held to a memory budget fixed at start-up, code that cannot afford the
allocator's device-wide synchronisation) cannot call cudaMalloc when they want to
step.  dion_step_noalloc keeps its scratch in a 24 MiB array built into the library
instead.  This test calls it through the C-ABI twice in a row and checks every output
against dion_step (the allocating entry point) on the same inputs, that device memory
does not shrink across the calls, and that a shape too large for the array is refused.

The file name sorts last on purpose: a run that stops at the first failure has then
already run every other test.  It passes alone in a fresh process and after the others.
"""
import pytest
import torch

from helpers import EPS, ETA, MU, TOL_FP32, device_state, rel, to_np64
from paper_2504_05295_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available(), "GPU tests selected but no CUDA device is visible"
    binding.load_library()


@pytest.mark.parametrize("m,n,r,ks", [(256, 512, 64, 16), (640, 384, 160, 8), (2048, 2048, 128, 64)])
def test_noalloc_matches_dion_step_on_two_calls_in_a_row(m, n, r, ks):
    pb = inputs.make_problem(m, n, r, seed=21, ks=ks)
    grads = [pb.grad(t).cuda() for t in range(2)]

    Xa, Ma, Qa = device_state(pb)
    da = torch.zeros(r, device="cuda")
    ref = []
    with binding.Dion(mu=MU, eps=EPS) as opt:
        for t in range(2):
            opt.step(Xa, Ma, grads[t], Qa, ETA, colnorm_out=da)
            ref.append([to_np64(v) for v in (Xa, Ma, Qa, da)])
        assert opt.get_status() == (0, 0)

    Xb, Mb, Qb = device_state(pb)
    db = torch.zeros(r, device="cuda")
    binding.step_noalloc(Xb, Mb, grads[0], Qb, ETA, MU, EPS, colnorm_out=db)   # first call: set-up
    torch.cuda.synchronize()
    got = [[to_np64(v) for v in (Xb, Mb, Qb, db)]]
    free_before, _ = torch.cuda.mem_get_info()
    binding.step_noalloc(Xb, Mb, grads[1], Qb, ETA, MU, EPS, colnorm_out=db)   # second call, same array
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    got.append([to_np64(v) for v in (Xb, Mb, Qb, db)])

    assert free_after >= free_before, "dion_step_noalloc must not allocate device memory"
    for t in range(2):
        for name, a, b in zip("XMQd", got[t], ref[t]):
            assert rel(a, b) <= TOL_FP32, f"call {t + 1}: {name} differs from dion_step by {rel(a, b):.2e}"


def test_noalloc_refuses_shapes_beyond_its_array():
    limit = binding.noalloc_scratch_limit()
    assert 16 << 20 <= limit <= 24 << 20
    m = n = 4096
    r = 1024
    X = torch.zeros(m, n, device="cuda"); M = torch.zeros(m, n, device="cuda")
    G = torch.ones(m, n, device="cuda"); Q = torch.ones(n, r, device="cuda")
    with binding.Dion() as opt:
        assert opt.workspace_bytes(m, n, r) > limit
    with pytest.raises(binding.DionError) as e:
        binding.step_noalloc(X, M, G, Q, ETA)
    assert e.value.code == -8 and "scratch" in str(e.value)
    torch.cuda.synchronize()
    assert float(X.abs().max()) == 0.0 and float(M.abs().max()) == 0.0      # nothing was launched
