"""The two contraction engines (fp32 FMA and tcgen05 tensor cores) in isolation.

Each product C = op(A) * op(B) with its fused operand formation (M + G) and
epilogue is run through the library's internal hook and compared with a float64
product of the same operands.  Covers the four operand layouts (k-contiguous or
row-contiguous A and B), ragged tails, lower-triangular output, the K limit of a
triangular operand, split-K and bf16 gradients.  The end-to-end parity with the
CPU oracle is in test_gpu_parity.py; this file localises a failure to an engine.
"""
import ctypes

import pytest
import torch

from paper_2504_05295_b200 import binding, build

pytestmark = pytest.mark.gpu


class GemmArgs(ctypes.Structure):
    _fields_ = [("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                ("A", ctypes.c_void_p), ("a_si", ctypes.c_int64), ("a_sk", ctypes.c_int64),
                ("A2", ctypes.c_void_p), ("a2_si", ctypes.c_int64), ("a2_sk", ctypes.c_int64), ("a2_mode", ctypes.c_int),
                ("B", ctypes.c_void_p), ("b_sk", ctypes.c_int64), ("b_sn", ctypes.c_int64),
                ("C", ctypes.c_void_p), ("ldc", ctypes.c_int64), ("epi", ctypes.c_int),
                ("C2", ctypes.c_void_p), ("ldc2", ctypes.c_int64), ("c2_mode", ctypes.c_int),
                ("alpha", ctypes.c_float), ("tri", ctypes.c_int), ("klimit", ctypes.c_int), ("precise", ctypes.c_int),
                ("ab16", ctypes.c_int), ("tf32x1", ctypes.c_int), ("variant", ctypes.c_int),
                    ("A16lo", ctypes.c_void_p), ("B16lo", ctypes.c_void_p), ("f16", ctypes.c_int)]


@pytest.fixture(scope="module")
def lib():
    build.build()
    assert torch.cuda.is_available()
    lib = binding.load_library()
    lib.dion_debug_gemm.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.POINTER(GemmArgs), ctypes.c_void_p,
                                    ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
    lib.dion_debug_gemm.restype = ctypes.c_int
    return lib


def run(lib, engine, precision, M, N, K, a_mn, b_mn, add=None, epi=0, tri=0, klimit=0, alpha=1.0, seed=0,
        precise=0, ab16=False, variant=0, tf32x1=False, expect_status=0, out=None):
    g = torch.Generator(device="cuda"); g.manual_seed(seed)
    rn = lambda *s: torch.randn(*s, generator=g, device="cuda")
    # A(i,k): stored M x K (k contiguous) or K x M (row index contiguous)
    A_store = rn(K, M) if a_mn else rn(M, K)
    if ab16:                             # operands stored as bf16: the reference sees the rounded values
        A_store = A_store.to(torch.bfloat16)
    if tf32x1:                           # values that fit TF32 (10 explicit mantissa bits): bf16 values do
        A_store = A_store.to(torch.bfloat16).float()
    A_log = A_store.t() if a_mn else A_store
    A2_store = None
    if add is not None:
        A2_store = (rn(K, M) if a_mn else rn(M, K)).to(add)
        A_eff = A_log.double() + (A2_store.t() if a_mn else A2_store).double()
    else:
        A_eff = A_log.double()
    # B(k,j): stored K x N (n contiguous) or N x K (k contiguous)
    B_store = rn(K, N) if b_mn else rn(N, K)
    if ab16:
        B_store = B_store.to(torch.bfloat16)
    if tf32x1:
        B_store = B_store.to(torch.bfloat16).float()
    B_log = B_store if b_mn else B_store.t()
    if klimit:
        B_log = torch.triu(B_log)       # B(k,j) = 0 for k > j
        if b_mn:
            B_store = B_log.contiguous()
        else:
            B_store = B_log.t().contiguous()
    C = rn(M, N)
    C0 = C.clone()
    C2 = rn(M, N).to(add if add is not None else torch.float32)
    ref = A_eff @ B_log.double()
    if epi == 0:
        want = alpha * ref
    elif epi == 1:
        want = C0.double() - alpha * ref
    else:
        want = C0.double() + C2.double() - alpha * ref
    a = GemmArgs()
    a.M, a.N, a.K = M, N, K
    a.A = A_store.data_ptr(); a.a_si, a.a_sk = (1, M) if a_mn else (K, 1)
    if add is not None:
        a.A2 = A2_store.data_ptr(); a.a2_si, a.a2_sk = (1, M) if a_mn else (K, 1)
        a.a2_mode = 1 if add == torch.float32 else 2
    a.B = B_store.data_ptr(); a.b_sk, a.b_sn = (N, 1) if b_mn else (1, K)
    a.C = C.data_ptr(); a.ldc = N; a.epi = epi
    a.C2 = C2.data_ptr(); a.ldc2 = N; a.c2_mode = 1 if C2.dtype == torch.float32 else 2
    a.alpha = alpha; a.tri = tri; a.klimit = klimit; a.precise = precise; a.ab16 = int(ab16)
    a.tf32x1 = int(tf32x1); a.variant = variant
    part = torch.empty(8 << 20, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rc = lib.dion_debug_gemm(engine, precision, ctypes.byref(a), part.data_ptr(), part.numel(), status.data_ptr(),
                             int(torch.cuda.current_stream().cuda_stream))
    torch.cuda.synchronize()
    assert rc == 0, f"dion_debug_gemm returned {rc}"
    assert int(status.item()) == expect_status, f"device status {int(status.item())}"
    if expect_status:
        return None
    if out is not None:
        out.append(C)
    got = C.double()
    if tri:
        # only the elements on or below the diagonal are guaranteed to be written
        idx = torch.arange(M, device="cuda")
        mask = idx[None, :] <= idx[:, None]
        got, want = got[mask], want[mask]
    err = (got - want).norm() / want.norm()
    return float(err)


LAYOUTS = [(False, False), (False, True), (True, True), (True, False)]
# relative Frobenius error of one product on N(0,1) data: fp32 FMA stays below 3e-6 up to
# K = 8192; the 3xTF32 tensor-core product accumulates in the tensor core's fp32 adder and
# reaches 4e-6 there (single-pass TF32 would be ~5e-4)
TOL = {1: 3e-6, 2: 8e-6}


@pytest.mark.parametrize("engine", [1, 2])
@pytest.mark.parametrize("a_mn,b_mn", LAYOUTS)
def test_layouts_fp32(lib, engine, a_mn, b_mn):
    err = run(lib, engine, 0, 512, 512, 1024, a_mn, b_mn)
    assert err < TOL[engine], err


@pytest.mark.parametrize("engine", [1, 2])
@pytest.mark.parametrize("M,N,K", [(128, 64, 64), (132, 260, 100), (640, 384, 96), (1028, 132, 2052), (256, 1024, 68)])
def test_ragged_shapes(lib, engine, M, N, K):
    for a_mn, b_mn in LAYOUTS:
        err = run(lib, engine, 0, M, N, K, a_mn, b_mn, seed=M + N)
        assert err < TOL[engine], (a_mn, b_mn, err)


@pytest.mark.parametrize("engine", [1, 2])
@pytest.mark.parametrize("add", [torch.float32, torch.bfloat16])
def test_fused_add_and_epilogues(lib, engine, add):
    # P = (M + G) Q ; R = (M + G)^T U ; M <- M + G - beta U R^T ; X <- X - s U Q^T
    assert run(lib, engine, 0, 1024, 256, 768, False, True, add=add) < TOL[engine]
    assert run(lib, engine, 0, 768, 256, 1024, True, True, add=add) < TOL[engine]
    assert run(lib, engine, 0, 1024, 768, 256, False, False, add=add, epi=2, alpha=0.05) < TOL[engine]
    assert run(lib, engine, 0, 1024, 768, 256, False, False, epi=1, alpha=0.01) < TOL[engine]


@pytest.mark.parametrize("engine", [1, 2])
def test_gram_lower_triangle_and_split_k(lib, engine):
    # Gram matrix P^T P: both operands row-contiguous, only lower tiles, long K -> split-K
    assert run(lib, engine, 0, 512, 512, 8192, True, True, tri=1) < TOL[engine]
    assert run(lib, engine, 0, 256, 256, 4096, True, True, tri=1) < TOL[engine]
    # large enough for the tensor engine's 128 x 256 lower tiles, with a ragged last tile row
    assert run(lib, engine, 0, 4096, 4096, 512, True, True, tri=1) < TOL[engine]
    assert run(lib, engine, 0, 4360, 4360, 264, True, True, tri=1, precise=1) < TOL[engine]
    # tall-skinny product with few tiles -> split-K
    assert run(lib, engine, 0, 2048, 128, 2048, False, True) < TOL[engine]


@pytest.mark.parametrize("engine", [1, 2])
def test_triangular_operand_k_limit(lib, engine):
    # U = P Linv^T with Linv lower triangular: B(k,j) = Linv[j][k] = 0 for k > j
    assert run(lib, engine, 0, 2048, 512, 512, False, False, klimit=1) < TOL[engine]
    assert run(lib, engine, 0, 1024, 768, 768, False, False, klimit=1) < TOL[engine]


@pytest.fixture(params=["tma", "registers"])
def bf16_path(request):
    # bf16 operands are formed from TMA-loaded fp32 tiles by default; bit 0 of the hook's variant word
    # selects the kernel whose producer warps load through registers
    return 1 if request.param == "registers" else 0


@pytest.mark.parametrize("a_mn,b_mn", LAYOUTS)
def test_bf16_operand_mode(lib, bf16_path, a_mn, b_mn):
    err = run(lib, 2, 1, 512, 512, 1024, a_mn, b_mn, variant=bf16_path)
    assert err < 6e-3, err
    err = run(lib, 2, 1, 648, 392, 328, a_mn, b_mn, seed=5, variant=bf16_path)
    assert err < 6e-3, err
    err = run(lib, 2, 1, 256, 1024, 2080, a_mn, b_mn, seed=6, variant=bf16_path)      # two accumulation chunks on the TMA path
    assert err < 6e-3, err


@pytest.mark.parametrize("add", [torch.float32, torch.bfloat16])
def test_bf16_operand_mode_fused_add_and_epilogues(lib, bf16_path, add):
    assert run(lib, 2, 1, 1024, 256, 768, False, True, add=add, variant=bf16_path) < 6e-3
    assert run(lib, 2, 1, 768, 256, 1024, True, True, add=add, variant=bf16_path) < 6e-3
    # the rank-r updates: the product (entries ~16 here) is scaled by alpha before it meets C (entries ~1)
    assert run(lib, 2, 1, 1024, 768, 256, False, False, add=add, epi=2, alpha=0.05, variant=bf16_path) < 3e-3
    assert run(lib, 2, 1, 1024, 768, 256, False, False, epi=1, alpha=0.01, variant=bf16_path) < 1e-3
    assert run(lib, 2, 1, 512, 512, 4096, True, True, tri=1, variant=bf16_path) < 6e-3
    assert run(lib, 2, 1, 1024, 768, 768, False, False, klimit=1, variant=bf16_path) < 6e-3


@pytest.mark.parametrize("a_mn,b_mn", LAYOUTS)
def test_bf16_arrays_as_operands(lib, a_mn, b_mn):
    # the operands are exact in bf16, so only the (truncating) fp32 accumulation separates the result from float64
    for (M, N, K) in [(512, 512, 1024), (648, 392, 328), (256, 1024, 4160), (128, 64, 64)]:
        err = run(lib, 2, 1, M, N, K, a_mn, b_mn, ab16=True, seed=M + K)
        assert err < 1e-5, (M, N, K, err)


@pytest.mark.parametrize("a_mn,b_mn", LAYOUTS)
def test_bf16_arrays_on_cta_pairs(lib, a_mn, b_mn):
    # from 512 rows and 256 columns the products on single 16-bit arrays run on clusters of two CTAs too (both CTAs'
    # tiles complete on the leader's barrier); bit 2 of the variant word keeps them on single CTAs: same bits
    for (M, N, K, epi) in [(1024, 512, 512, 0), (2048, 768, 2112, 1), (648, 392, 328, 2), (1280, 256, 64, 1),
                           (4096, 1024, 1024, 1)]:
        got = []
        err = run(lib, 2, 1, M, N, K, a_mn, b_mn, ab16=True, epi=epi, alpha=0.05, seed=M + K, out=got)
        assert err < 1e-5, (M, N, K, epi, err)
        err1 = run(lib, 2, 1, M, N, K, a_mn, b_mn, ab16=True, epi=epi, alpha=0.05, seed=M + K, variant=4, out=got)
        assert err1 < 1e-5, (M, N, K, epi, err1)
        assert torch.equal(got[0], got[1]), (M, N, K, epi)


def test_bf16_arrays_epilogues_and_lower_triangle(lib):
    assert run(lib, 2, 1, 1024, 768, 256, False, False, ab16=True, epi=2, alpha=0.05) < 1e-5
    assert run(lib, 2, 1, 1024, 768, 256, False, False, ab16=True, epi=1, alpha=0.01) < 1e-5
    assert run(lib, 2, 1, 512, 512, 4096, True, True, ab16=True, tri=1) < 1e-5
    assert run(lib, 2, 1, 2048, 128, 2048, False, True, ab16=True) < 1e-5      # split-K


@pytest.mark.parametrize("a_mn,b_mn", LAYOUTS)
def test_split_accumulators_reach_fma_accuracy(lib, a_mn, b_mn):
    for (M, N, K) in [(512, 512, 1024), (640, 388, 2052), (256, 128, 4096)]:
        err = run(lib, 2, 0, M, N, K, a_mn, b_mn, precise=1, seed=K)
        assert err < 1e-6, (M, N, K, err)
    # a Gram matrix sums same-sign terms on its diagonal, where the truncating adder is biased
    assert run(lib, 2, 0, 512, 512, 8192, True, True, tri=1, precise=1) < 2e-6
    assert run(lib, 2, 0, 2048, 512, 512, False, False, klimit=1, precise=1) < 1.5e-6


def test_register_path_fp32(lib):
    # the fp32 (3xTF32) kernel whose producer warps load through registers: operands TMA cannot describe
    for a_mn, b_mn in LAYOUTS:
        assert run(lib, 2, 0, 640, 384, 200, a_mn, b_mn, variant=1, seed=3) < TOL[2]


@pytest.mark.parametrize("M,N,K,epi", [(1024, 768, 256, 1), (640, 392, 96, 1), (2048, 256, 2080, 1), (256, 128, 64, 0),
                                       (512, 512, 512, 2)])
def test_single_pass_tf32_on_operands_that_fit_tf32(lib, M, N, K, epi):
    # operands whose values fit TF32 are read exactly by one MMA per K step: the only error left is the
    # tensor core's fp32 accumulation
    err = run(lib, 2, 0, M, N, K, False, False, epi=epi, alpha=0.05, tf32x1=True, seed=K)
    assert err < 8e-6, err


def test_a_wait_that_runs_out_reports_timeout_and_the_next_product_is_correct(lib):
    # bit 1 of the variant word: the producer warps of the register-path kernel withhold their first arrival
    # and every barrier wait has a 1 ms budget.  The kernel must give up (no trap, no endless wait), set
    # DION_STATUS_TIMEOUT (4) and return; the context stays usable.
    assert run(lib, 2, 0, 128, 128, 64, False, False, variant=3, expect_status=4) is None
    assert run(lib, 2, 0, 256, 384, 128, False, False, variant=3, expect_status=4) is None      # several CTAs
    assert run(lib, 2, 0, 128, 128, 64, False, False, variant=1) < TOL[2]
    assert run(lib, 2, 0, 512, 512, 1024, False, True) < TOL[2]


# ---------------------------------------------------------------------------
# CTA pairs (cta_group::2): fp32-mode products with at least 512 rows and 256 columns run on clusters of two
# CTAs that share a 256 x 256 tile; bit 2 of the variant word keeps such a product on single-CTA tiles.
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("a_mn,b_mn", LAYOUTS)
@pytest.mark.parametrize("precise", [0, 1])
def test_cta_pairs_all_layouts(lib, a_mn, b_mn, precise):
    tol = 3e-6 if precise else TOL[2]          # the error grows with the number of 1024-k accumulation chunks
    for (M, N, K) in [(1024, 512, 512), (2048, 768, 2080), (648, 392, 328), (1280, 256, 96)]:
        err = run(lib, 2, 0, M, N, K, a_mn, b_mn, precise=precise, seed=M + K)
        assert err < tol, (M, N, K, err)
        ref = run(lib, 2, 0, M, N, K, a_mn, b_mn, precise=precise, seed=M + K, variant=4)
        assert ref < tol, ("single-CTA tiles", M, N, K, ref)


def test_cta_pairs_epilogues_triangle_and_k_limit(lib):
    assert run(lib, 2, 0, 2048, 1536, 256, False, False, add=torch.float32, epi=2, alpha=0.05) < TOL[2]
    assert run(lib, 2, 0, 2048, 1536, 256, False, False, epi=1, alpha=0.01) < TOL[2]
    assert run(lib, 2, 0, 1100, 520, 300, False, True, add=torch.float32) < TOL[2]       # fused fp32 addend, ragged
    assert run(lib, 2, 0, 2304, 2304, 512, True, True, tri=1, precise=1) < 2e-6           # lower 256 x 256 tiles
    assert run(lib, 2, 0, 4360, 4360, 264, True, True, tri=1) < TOL[2]
    assert run(lib, 2, 0, 2048, 512, 512, False, False, klimit=1) < TOL[2]
    assert run(lib, 2, 0, 512, 512, 8192, True, True) < TOL[2]                             # few tiles: split-K over pairs


@pytest.mark.parametrize("M,N,K,epi", [(1024, 768, 256, 2), (1024, 768, 256, 3), (648, 392, 328, 1), (2048, 256, 2112, 0),
                                       (128, 64, 64, 0)])
def test_bf16_operand_pairs(lib, M, N, K, epi):
    # each operand as a pair of bf16 arrays, x ~ hi + lo (16 significant bits): three bf16 MMAs per K step
    g = torch.Generator(device="cuda"); g.manual_seed(M + K)
    A = torch.randn(M, K, generator=g, device="cuda"); B = torch.randn(N, K, generator=g, device="cuda")
    Ah = A.to(torch.bfloat16); Al = (A - Ah.float()).to(torch.bfloat16)
    Bh = B.to(torch.bfloat16); Bl = (B - Bh.float()).to(torch.bfloat16)
    C = torch.randn(M, N, generator=g, device="cuda"); C0 = C.clone()
    C2 = torch.randn(M, N, generator=g, device="cuda")
    alpha = 0.05
    ref = A.double() @ B.double().t()
    want = {0: alpha * ref, 1: C0.double() - alpha * ref, 2: C0.double() + C2.double() - alpha * ref,
            3: C2.double() - alpha * ref}[epi]
    a = GemmArgs()
    a.M, a.N, a.K = M, N, K
    a.A = Ah.data_ptr(); a.a_si, a.a_sk = K, 1; a.A16lo = Al.data_ptr()
    a.B = Bh.data_ptr(); a.b_sk, a.b_sn = 1, K; a.B16lo = Bl.data_ptr()
    a.C = C.data_ptr(); a.ldc = N; a.epi = epi
    a.C2 = C2.data_ptr(); a.ldc2 = N; a.c2_mode = 1
    a.alpha = alpha; a.ab16 = 1
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rc = lib.dion_debug_gemm(2, 1, ctypes.byref(a), None, 0, status.data_ptr(), int(torch.cuda.current_stream().cuda_stream))
    torch.cuda.synchronize()
    assert rc == 0 and int(status.item()) == 0
    # the product itself is accurate to ~2^-16 of |A| |B|
    prod = {0: C.double() / alpha, 1: (C0.double() - C.double()) / alpha, 2: (C0.double() + C2.double() - C.double()) / alpha,
            3: (C2.double() - C.double()) / alpha}[epi]
    err_prod = float((prod - ref).norm() / ref.norm())
    err = float((C.double() - want).norm() / want.norm())
    assert err_prod < 3e-5, err_prod
    assert err < 1e-5 or epi == 0, err


def _pair_product(lib, M, N, K, a_mn, b_mn, epi, variant, seed):
    """C after one product on bf16 (hi, lo) operand pairs in the given storage layouts; also the float64 target."""
    g = torch.Generator(device="cuda"); g.manual_seed(seed)
    A = torch.randn(M, K, generator=g, device="cuda"); B = torch.randn(N, K, generator=g, device="cuda")

    def split(x):
        h = x.to(torch.bfloat16)
        return h, (x - h.float()).to(torch.bfloat16)
    As = A.t().contiguous() if a_mn else A          # stored K x M (row index contiguous) or M x K
    Bs = B.t().contiguous() if b_mn else B          # stored K x N or N x K
    Ah, Al = split(As); Bh, Bl = split(Bs)
    C = torch.randn(M, N, generator=g, device="cuda"); C0 = C.clone()
    C2 = torch.randn(M, N, generator=g, device="cuda")
    alpha = 0.05
    ref = A.double() @ B.double().t()
    want = {0: alpha * ref, 1: C0.double() - alpha * ref, 2: C0.double() + C2.double() - alpha * ref,
            3: C2.double() - alpha * ref}[epi]
    a = GemmArgs()
    a.M, a.N, a.K = M, N, K
    a.A = Ah.data_ptr(); a.A16lo = Al.data_ptr(); a.a_si, a.a_sk = (1, M) if a_mn else (K, 1)
    a.B = Bh.data_ptr(); a.B16lo = Bl.data_ptr(); a.b_sk, a.b_sn = (N, 1) if b_mn else (1, K)
    a.C = C.data_ptr(); a.ldc = N; a.epi = epi
    a.C2 = C2.data_ptr(); a.ldc2 = N; a.c2_mode = 1
    a.alpha = alpha; a.ab16 = 1; a.variant = variant
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    part = torch.empty(8 << 20, device="cuda")
    rc = lib.dion_debug_gemm(2, 1, ctypes.byref(a), part.data_ptr(), part.numel(), status.data_ptr(),
                             int(torch.cuda.current_stream().cuda_stream))
    torch.cuda.synchronize()
    assert rc == 0 and int(status.item()) == 0, (rc, int(status.item()))
    return C, want


@pytest.mark.parametrize("a_mn,b_mn", LAYOUTS)
def test_bf16_operand_pairs_on_cta_pairs(lib, a_mn, b_mn):
    # from 512 rows and 256 columns the operand-pair product runs on clusters of two CTAs (256 x 256 tiles, each CTA
    # loading half of the B tile); bit 2 of the variant word keeps it on single-CTA tiles: same bits
    for (M, N, K, epi) in [(1024, 512, 512, 0), (2048, 768, 2112, 1), (648, 392, 328, 2), (1280, 256, 96, 3),
                           (512, 512, 8192, 0)]:
        C, want = _pair_product(lib, M, N, K, a_mn, b_mn, epi, 0, seed=M + K)
        err = float((C.double() - want).norm() / want.norm())
        assert err < (3e-5 if epi == 0 else 1e-5), (M, N, K, epi, err)
        C1, _ = _pair_product(lib, M, N, K, a_mn, b_mn, epi, 4, seed=M + K)
        if K < 8192:      # (the last case has few tiles: K is split, differently for pairs and single CTAs)
            assert torch.equal(C, C1), (M, N, K, epi)


def test_column_panel_tile_order_when_b_exceeds_l2(lib):
    # N x K operands above ~48 MB switch the tile order to column panels (every tile still computed exactly once)
    assert run(lib, 2, 0, 1024, 4096, 4096, False, False, epi=1, alpha=0.01) < TOL[2]
    assert run(lib, 2, 0, 1024, 4352, 3104, False, True, epi=0) < TOL[2]                    # ragged, last panel narrower
    assert run(lib, 2, 0, 640, 8192, 2048, False, False, epi=1, alpha=0.05, tf32x1=True) < 8e-6
    for (a_mn, b_mn) in LAYOUTS:
        C, want = _pair_product(lib, 1024, 8192 + 256, 2048, a_mn, b_mn, 3, 0, seed=5)
        assert float((C.double() - want).norm() / want.norm()) < 1e-5


@pytest.mark.parametrize("M,N,K,epi", [(1024, 768, 256, 1), (640, 392, 96, 1), (2048, 256, 1024, 0), (4096, 4096, 128, 1)])
def test_ieee_half_arrays_as_operands(lib, M, N, K, epi):
    # the weight update's factors as IEEE half arrays: values that fit half exactly are multiplied exactly, so the
    # only error left is the tensor core's fp32 accumulation
    g = torch.Generator(device="cuda"); g.manual_seed(M + K)
    A = torch.randn(M, K, generator=g, device="cuda").half(); B = torch.randn(N, K, generator=g, device="cuda").half()
    C = torch.randn(M, N, generator=g, device="cuda"); C0 = C.clone()
    alpha = 0.05
    ref = A.double() @ B.double().t()
    want = alpha * ref if epi == 0 else C0.double() - alpha * ref
    a = GemmArgs()
    a.M, a.N, a.K = M, N, K
    a.A = A.data_ptr(); a.a_si, a.a_sk = K, 1
    a.B = B.data_ptr(); a.b_sk, a.b_sn = 1, K
    a.C = C.data_ptr(); a.ldc = N; a.epi = epi
    a.alpha = alpha; a.ab16 = 1; a.f16 = 1
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rc = lib.dion_debug_gemm(2, 0, ctypes.byref(a), None, 0, status.data_ptr(), int(torch.cuda.current_stream().cuda_stream))
    torch.cuda.synchronize()
    assert rc == 0 and int(status.item()) == 0
    err = float((C.double() - want).norm() / want.norm())
    assert err < 8e-6, err
