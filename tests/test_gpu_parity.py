"""GPU parity: the CUDA path (through the C-ABI) against the CPU oracle, element by element, on
the same seeded inputs.  Sizes span several tiles and ragged tails; the categories follow the
paper's test list (Appendix "Testing")."""
import dataclasses
import itertools

import numpy as np
import pytest
import torch

import helpers
import oracle
from paper_2601_07827_b200 import inputs

pytestmark = pytest.mark.gpu

REAL_AND_COMPLEX = [torch.float32, torch.float64, torch.complex64, torch.complex128]


@pytest.fixture(scope="module")
def api():
    return helpers.api()


@pytest.fixture(scope="module")
def handle(api):
    return api.Handle()


def small_workloads():
    W = inputs.workloads()
    out = {
        "cfg1": W["cfg1_f64_small"],
        "cfg2s": inputs.scaled_down(W["cfg2_f64_ccsd_ladder"], {"a": 12, "b": 12, "c": 10, "d": 10, "i": 7, "j": 6}),
        "cfg3s": inputs.scaled_down(W["cfg3_f32_batched_permuted"], {"z": 3, "a": 20, "b": 12, "j": 24, "k": 6, "l": 8}),
        "cfg4s": inputs.scaled_down(W["cfg4_c64_conj"], {"p": 40, "q": 24, "r": 5, "s": 12, "t": 8}),
        "cfg5": W["cfg5_f32_tensor_network"],
        "cfg5b": W["cfg5b_f32_tensor_network_rev"],
    }
    return out


@pytest.mark.parametrize("name", list(small_workloads()))
@pytest.mark.parametrize("kernel", ["auto", "generic", "tiled"])
def test_workload_shapes(api, handle, name, kernel):
    w = small_workloads()[name]
    code = {"auto": api.KERNEL_AUTO, "generic": api.KERNEL_GENERIC, "tiled": api.KERNEL_TILED}[kernel]
    try:
        worst, status, _ = helpers.workload_case(handle, w, kernel=code, want_status=True)
    except api.BtcError as e:
        if kernel == "tiled" and e.code == api.ERR_NOT_SUPPORTED:
            pytest.skip("no tiled kernel for this element type yet")
        raise
    assert worst <= 1.0, worst
    if kernel != "auto":
        assert status["kernel"] == code


@pytest.mark.parametrize("split_k", [1, 2, 3, 4, 7, 8])
@pytest.mark.parametrize("name", ["cfg1", "cfg4s"])
def test_split_k_slices(api, handle, name, split_k):
    w = small_workloads()[name]
    worst, status, first = helpers.workload_case(handle, w, kernel=api.KERNEL_TILED, split_k=split_k, want_status=True)
    # the library may lower the request so that no slice is empty
    assert worst <= 1.0 and (split_k > 1) == (status["split_k"] > 1) and status["split_k"] <= split_k
    # 64-bit element types: 2, 4 or 8 slices add up inside a thread-block cluster (one launch); other
    # counts go through scratch and a second kernel
    assert status["launches"] == (1 if status["split_k"] in (1, 2, 4, 8) else 2)
    _, _, second = helpers.workload_case(handle, w, kernel=api.KERNEL_TILED, split_k=split_k)
    assert torch.equal(first.view(torch.int64), second.view(torch.int64))   # run-to-run bit identical


def _ext(labels, table):
    return tuple(table[l] for l in labels)


CATEGORIES = {
    # name: (labelsA, labelsB, labelsD, extents)
    "hadamard": ("ij", "ij", "ij", dict(i=37, j=29)),
    "basic": ("ikl", "ljk", "ji", dict(i=70, j=45, k=9, l=11)),
    "equal_extents": ("aibj", "jcia", "cb", dict(a=6, b=6, c=6, i=6, j=6)),
    "outer_product": ("ij", "kl", "kijl", dict(i=13, j=5, k=9, l=7)),
    "all_contracted": ("ijk", "kji", "", dict(i=17, j=9, k=33)),
    "zero_mode_A": ("", "ij", "ji", dict(i=40, j=33)),
    "one_mode": ("k", "kj", "j", dict(k=300, j=70)),
    "hadamard_free": ("hik", "hkj", "ijh", dict(h=5, i=33, j=18, k=40)),
    "hadamard_contracted": ("hk", "hk", "h", dict(h=77, k=130)),
    "repeated": ("kik", "kjj", "ij", dict(i=35, j=21, k=19)),
    "isolated": ("ikx", "kyj", "ij", dict(i=33, j=20, k=17, x=3, y=4)),
    "gemv_like": ("ik", "k", "i", dict(i=1000, k=333)),
    "big_ragged": ("ik", "kj", "ij", dict(i=257, j=131, k=67)),
}


@pytest.mark.parametrize("dtype", REAL_AND_COMPLEX)
@pytest.mark.parametrize("cat", list(CATEGORIES))
def test_paper_test_categories(api, handle, cat, dtype):
    la, lb, ld, ext = CATEGORIES[cat]
    A = helpers.random_tensor(11, _ext(la, ext), None, dtype)
    B = helpers.random_tensor(12, _ext(lb, ext), None, dtype)
    C = helpers.random_tensor(13, _ext(ld, ext), None, dtype)
    D = inputs.place(None, _ext(ld, ext), None, dtype)
    cplx = dtype.is_complex
    alpha = complex(0.75, -1.25) if cplx else 0.75
    beta = complex(-0.5, 0.25) if cplx else -0.5
    worst, status, _ = helpers.run_case(handle, A, la, B, lb, C, D, ld, alpha, beta, conjA=cplx, conjC=cplx, want_status=True)
    assert worst <= 1.0, worst
    if cat in ("hadamard", "outer_product", "zero_mode_A"):
        # no contracted label: the bandwidth-bound streaming kernel (Appendix "Testing" items 1, 6, 8)
        assert status["variant"] == 100 and status["launches"] == 1, status


def test_strict_fp32_precision_runs_the_fma_kernels(api, handle):
    """BTC_ATTR_COMPUTE_PRECISION = STRICT: the planner must leave the TF32-split tensor-core variants (6 and up)
    for the FFMA variants (0-5); the result meets the same tolerance, and on small integers it is bit exact
    either way."""
    ext = dict(i=300, j=200, k=150)
    A = helpers.random_tensor(71, _ext("ik", ext), None, torch.float32)
    B = helpers.random_tensor(72, _ext("kj", ext), None, torch.float32)
    D = inputs.place(None, _ext("ij", ext), None, torch.float32)
    dt = api.dtype_code(torch.float32)
    tA, tB, tD = (api.TensorInfo(handle, dt, x.extents, x.strides) for x in (A, B, D))
    op = api.Contraction(handle, tA, "ik", tB, "kj", None, "ij", tD, "ij", 1.0, 0.0)
    assert op.variant >= 6
    op.set_attr(api.ATTR_COMPUTE_PRECISION, api.PRECISION_STRICT)
    assert 0 <= op.variant <= 5
    dA, dB, dD = A.to("cuda"), B.to("cuda"), D.to("cuda")
    need = op.workspace_size()
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device="cuda")
    op.execute(torch.cuda.current_stream().cuda_stream, dA.data_ptr(), dB.data_ptr(), 0, dD.data_ptr(), workspace=ws.data_ptr(),
               workspace_bytes=need)
    torch.cuda.synchronize()
    want = D.clone()
    scale = oracle.contract(A.numpy(), "ik", B.numpy(), "kj", None, "ij", want.numpy(), "ij", 1.0, 0.0)
    pos = D.offsets()
    assert helpers.compare(dD.buffer.cpu()[pos].numpy(), want.buffer[pos].numpy(), scale, torch.float32) <= 1.0
    op.set_attr(api.ATTR_COMPUTE_PRECISION, api.PRECISION_DEFAULT)
    assert op.variant >= 6


@pytest.mark.parametrize("seed", range(64))
def test_seeded_random_contractions(api, handle, seed):
    """Randomized set (the paper plans randomized benchmarks; these are seeded stand-ins): random numbers
    of batch, free and contracted labels (rank 0-8), mixed extents including 1, every tensor in its own
    memory order with padding, negative strides in A and B, all four element types in turn, whatever
    kernel the planner picks; padding bytes of D must stay untouched."""
    la, lb, ld, ext, sA, sB, sD = inputs.random_contraction(9000 + seed)
    dtype = REAL_AND_COMPLEX[seed % len(REAL_AND_COMPLEX)]
    A = helpers.random_tensor(3 * seed + 1, _ext(la, ext), sA, dtype)
    B = helpers.random_tensor(3 * seed + 2, _ext(lb, ext), sB, dtype)
    C = helpers.random_tensor(3 * seed + 3, _ext(ld, ext), sD, dtype)
    D = inputs.place(None, _ext(ld, ext), sD, dtype)
    cplx = dtype.is_complex
    alpha = complex(1.25, -0.5) if cplx else 1.25
    beta = (complex(0.5, 0.75) if cplx else 0.5) if seed % 3 else 0.0
    worst, _, _ = helpers.run_case(handle, A, la, B, lb, C if seed % 3 else None, D, ld, alpha, beta,
                                   conjA=cplx and seed % 2 == 0, conjB=cplx and seed % 4 == 1)
    assert worst <= 1.0, (worst, la, lb, ld, ext)


@pytest.mark.parametrize("dtype", [torch.float64, torch.complex128, torch.float32])
@pytest.mark.parametrize("kernel", ["auto", "generic"])
def test_strides_negative_zero_padded_subtensor(api, handle, dtype, kernel):
    code = {"auto": api.KERNEL_AUTO, "generic": api.KERNEL_GENERIC}[kernel]
    ext = dict(i=70, j=45, k=40, l=6)
    # A: negative stride on i, padded; B: zero stride on l (broadcast), mixed signs; D: padded + negative
    A = helpers.random_tensor(21, _ext("ikl", ext), (-1, 75, 75 * 41), dtype)
    B = helpers.random_tensor(22, _ext("lkj", ext), (0, -3, 130), dtype)
    C = helpers.random_tensor(23, _ext("ji", ext), (2, -95), dtype)
    D = inputs.place(None, _ext("ji", ext), (2, -95), dtype)
    worst, _, _ = helpers.run_case(handle, A, "ikl", B, "lkj", C, D, "ji", 1.5, 0.5, kernel=code)
    assert worst <= 1.0, worst
    # sub-tensor with fewer modes than its parent: a slice of a rank-4 buffer used as a rank-2 operand
    A2 = helpers.random_tensor(24, (70, 40), (7, 7 * 80), dtype)
    D2 = inputs.place(None, (70, 45), (1, 72), dtype)
    worst, _, _ = helpers.run_case(handle, A2, "ik", B, "lkj", None, D2, "ij", kernel=code)
    assert worst <= 1.0, worst


@pytest.mark.parametrize("dtype", [torch.complex64, torch.complex128])
def test_conjugation_flags(api, handle, dtype):
    ext = dict(i=40, j=36, k=50)
    A = helpers.random_tensor(31, _ext("ki", ext), None, dtype)
    B = helpers.random_tensor(32, _ext("kj", ext), None, dtype)
    C = helpers.random_tensor(33, _ext("ij", ext), None, dtype)
    D = inputs.place(None, _ext("ij", ext), None, dtype)
    for ca, cb, cc in itertools.product([False, True], repeat=3):
        worst, _, _ = helpers.run_case(handle, A, "ki", B, "kj", C, D, "ij", complex(0.5, -0.25), complex(1, 2),
                                       conjA=ca, conjB=cb, conjC=cc)
        assert worst <= 1.0, (ca, cb, cc, worst)


@pytest.mark.parametrize("dtype", REAL_AND_COMPLEX)
def test_small_integers_bit_exact(api, handle, dtype):
    """Exactly representable inputs: every summation order gives the same bits."""
    ext = dict(i=70, j=66, k=40, l=5)
    A = helpers.random_tensor(41, _ext("ikl", ext), None, dtype, ("smallint", 8))
    B = helpers.random_tensor(42, _ext("lkj", ext), None, dtype, ("smallint", 8))
    C = helpers.random_tensor(43, _ext("ji", ext), None, dtype, ("smallint", 8))
    D = inputs.place(None, _ext("ji", ext), None, dtype)
    for kernel in (api.KERNEL_AUTO, api.KERNEL_GENERIC):
        worst, _, _ = helpers.run_case(handle, A, "ikl", B, "lkj", C, D, "ji", 2.0, -3.0, kernel=kernel)
        assert worst == 0.0


def test_alpha_zero_and_beta_zero_never_read(api, handle):
    ext = dict(i=130, j=70, k=64)
    A = helpers.random_tensor(51, _ext("ik", ext), None, torch.float64)
    B = helpers.random_tensor(52, _ext("kj", ext), None, torch.float64)
    C = helpers.random_tensor(53, _ext("ij", ext), None, torch.float64)
    D = inputs.place(None, _ext("ij", ext), None, torch.float64)
    nanA = inputs.place(None, _ext("ik", ext), None, torch.float64)   # all NaN
    worst, _, _ = helpers.run_case(handle, nanA, "ik", B, "kj", C, D, "ij", 0.0, 2.0)
    assert worst == 0.0
    nanC = inputs.place(None, _ext("ij", ext), None, torch.float64)
    worst, _, _ = helpers.run_case(handle, A, "ik", B, "kj", nanC, D, "ij", 1.0, 0.0)
    assert worst <= 1.0


def test_in_place_update(api, handle):
    w = small_workloads()["cfg2s"]
    assert w.in_place
    worst, _, _ = helpers.workload_case(handle, w)
    assert worst <= 1.0


@pytest.mark.parametrize("name", ["cfg1", "cfg3s", "cfg4s"])
def test_host_buffer_entry_point(api, handle, name):
    worst, _, _ = helpers.workload_case(handle, small_workloads()[name], host_path=True)
    assert worst <= 1.0


def test_execute_argument_errors(api, handle):
    w = small_workloads()["cfg1"]
    A, B, C, D = (t.to("cuda") for t in inputs.make_workload_tensors(w))
    dt = api.F64
    tA, tB = api.TensorInfo(handle, dt, A.extents), api.TensorInfo(handle, dt, B.extents)
    tD = api.TensorInfo(handle, dt, D.extents)
    op = api.Contraction(handle, tA, w.labelsA, tB, w.labelsB, tD, w.labelsD, tD, w.labelsD, 1.0, 0.5)
    ws = torch.empty(op.workspace_size(), dtype=torch.uint8, device="cuda")

    def code(fn):
        with pytest.raises(api.BtcError) as ei:
            fn()
        return ei.value.code
    assert op.workspace_size() > 0
    assert code(lambda: op.execute(0, A.data_ptr(), B.data_ptr(), C.data_ptr(), D.data_ptr())) == api.ERR_WORKSPACE_TOO_SMALL
    assert code(lambda: op.execute(0, A.data_ptr(), B.data_ptr(), C.data_ptr(), D.data_ptr(),
                                   workspace=ws.data_ptr(), workspace_bytes=16)) == api.ERR_WORKSPACE_TOO_SMALL
    assert code(lambda: op.execute(0, A.data_ptr() + 4, B.data_ptr(), C.data_ptr(), D.data_ptr(),
                                   workspace=ws.data_ptr(), workspace_bytes=ws.numel())) == api.ERR_MISALIGNED
    assert code(lambda: op.execute(0, A.data_ptr(), B.data_ptr(), 0, D.data_ptr(),
                                   workspace=ws.data_ptr(), workspace_bytes=ws.numel())) == api.ERR_INVALID_ARGUMENT
    op.execute(0, A.data_ptr(), B.data_ptr(), 0, D.data_ptr(), beta=0.0, workspace=ws.data_ptr(), workspace_bytes=ws.numel())
    torch.cuda.synchronize()


def test_unaligned_base_pointer_falls_back_to_element_copies(api, handle):
    """Operands whose strides allow 16-byte copies but whose base pointer is only 8-byte aligned."""
    ext = dict(i=128, j=64, k=32)
    A = helpers.random_tensor(61, (4200,), None, torch.float64)
    A_view = inputs.StridedTensor(A.buffer, (128, 32), (1, 130), 1)   # starts at element 1, ld 130
    B = helpers.random_tensor(62, _ext("kj", ext), None, torch.float64)
    D = inputs.place(None, _ext("ij", ext), None, torch.float64)
    worst, _, _ = helpers.run_case(handle, A_view, "ik", B, "kj", None, D, "ij", kernel=api.KERNEL_TILED)
    assert worst <= 1.0


@pytest.mark.parametrize("dtype,variant", [(torch.float64, v) for v in range(5)] + [(torch.float32, v) for v in range(23)]
                         + [(torch.complex128, v) for v in range(3)] + [(torch.complex64, v) for v in range(2)])
def test_every_tile_variant(api, handle, dtype, variant):
    """Each tile variant of the tiled kernels, forced through the attribute, on a ragged multi-tile case
    with one operand contiguous along its free index and the other along k."""
    ext = dict(i=300, j=200, k=150)
    A = helpers.random_tensor(71, _ext("ik", ext), None, dtype)
    B = helpers.random_tensor(72, _ext("kj", ext), None, dtype)
    C = helpers.random_tensor(73, _ext("ij", ext), None, dtype)
    D = inputs.place(None, _ext("ij", ext), None, dtype)
    worst, status, _ = helpers.run_case(handle, A, "ik", B, "kj", C, D, "ij", 1.25, -0.5, kernel=api.KERNEL_TILED,
                                        variant=variant, want_status=True)
    assert worst <= 1.0 and status["kernel"] == api.KERNEL_TILED
    # both operands contiguous along k / both along the free index
    A2 = helpers.random_tensor(74, _ext("ki", ext), None, dtype)
    B2 = helpers.random_tensor(75, _ext("jk", ext), None, dtype)
    worst, _, _ = helpers.run_case(handle, A2, "ki", B, "kj", None, D, "ij", kernel=api.KERNEL_TILED, variant=variant)
    assert worst <= 1.0
    worst, _, _ = helpers.run_case(handle, A, "ik", B2, "jk", None, D, "ij", kernel=api.KERNEL_TILED, variant=variant)
    assert worst <= 1.0


@pytest.mark.parametrize("variant", [10, 11, 12, 13, 14, 15, 16])
def test_persistent_tensor_memory_kernel_walks_many_tiles(api, handle, variant):
    """The tcgen05 kernels are persistent: with more tiles than SMs every CTA takes several tiles in
    turn, re-using both accumulators, the stage rings and the double-buffered offset arrays.  Ragged
    extents, a batch label, beta != 0 and a strided (non-vector) operand are all in play."""
    ext = dict(i=128 * 17 + 5, j=96 * 6 + 7, k=70, z=3)
    A = helpers.random_tensor(81, _ext("kiz", ext), None, torch.float32)
    B = helpers.random_tensor(82, _ext("zkj", ext), None, torch.float32)
    C = helpers.random_tensor(83, _ext("ijz", ext), None, torch.float32)
    D = inputs.place(None, _ext("ijz", ext), None, torch.float32)
    worst, status, _ = helpers.run_case(handle, A, "kiz", B, "zkj", C, D, "ijz", 0.75, 1.5, kernel=api.KERNEL_TILED,
                                        variant=variant, want_status=True)
    assert worst <= 1.0 and status["kernel"] == api.KERNEL_TILED
    bn = {10: 96, 11: 128, 12: 256, 13: 96, 14: 128, 15: 96, 16: 128}[variant]
    assert status["grid"][0] < -(-ext["i"] // 128) * -(-ext["j"] // bn) * ext["z"]   # fewer CTAs than tiles


BULK = {
    # name: (labelsA, labelsB, labelsD, extents, strides of D or None); the operand that ends up on the M side
    # is a tensor of boxes for stages of 24 and of 32 contracted indices
    "rows_contiguous_ragged": ("ik", "kj", "ij", dict(i=128 * 3 + 44, j=200, k=150), None),
    "k_contiguous_ragged": ("ki", "kj", "ij", dict(i=128 * 2 + 20, j=150, k=152), None),
    "k_contiguous_two_k_modes": ("kiq", "jqk", "ij", dict(i=256, j=100, k=96, q=3), None),
    # workload 3 scaled down: rows of a tile = 8 j x 16 b, stage = all 24 l, batch z
    "blocked_free_modes": ("akzl", "lbkjz", "jbza", dict(z=3, a=40, b=32, j=24, k=5, l=24), (1, 28, 28 * 32, 28 * 32 * 3)),
    "many_tiles_batch": ("kiz", "zkj", "ijz", dict(i=128 * 17 + 5, j=96 * 3 + 7, k=72, z=2), None),
}


@pytest.mark.parametrize("variant", [17, 18, 19, 20, 21])
@pytest.mark.parametrize("name", list(BULK))
def test_bulk_tensor_copy_variants(api, handle, name, variant):
    """The tcgen05 variants that fetch the M-side tile of every stage with one bulk tensor copy: boxes with
    rows or k contiguous, ragged last tiles in M and in K (zero-filled by the copy), several contracted
    modes, blocked free modes with a batch label, and more tiles than SMs.  Where a stage of that
    variant's length is no box of the operand the planner must hand the work to the gathering twin."""
    la, lb, ld, ext, sD = BULK[name]
    A = helpers.random_tensor(91, _ext(la, ext), None, torch.float32)
    B = helpers.random_tensor(92, _ext(lb, ext), None, torch.float32)
    C = helpers.random_tensor(93, _ext(ld, ext), sD, torch.float32)
    D = inputs.place(None, _ext(ld, ext), sD, torch.float32)
    worst, status, _ = helpers.run_case(handle, A, la, B, lb, C, D, ld, 0.75, 1.5, kernel=api.KERNEL_TILED,
                                        variant=variant, want_status=True)
    assert worst <= 1.0 and status["kernel"] == api.KERNEL_TILED
    bk = 24 if variant in (17, 20, 21) else 32
    boxes = not (name == "blocked_free_modes" and bk == 32)      # 24 l, then k: a stage of 32 is no box
    assert status["variant"] == (variant if boxes else (13 if variant in (17, 18, 21) else 14))


CASE4 = {
    # name: (labelsA, labelsB, labelsD, extents, stridesA or None)
    "x_slowest_in_A": ("ikx", "kj", "ij", dict(i=150, j=90, k=70, x=6), None),
    "x_fastest_in_A": ("xik", "kj", "ij", dict(i=150, j=90, k=70, x=40), None),          # one warp per element of A'
    "both_inputs": ("ixk", "ykjz", "ij", dict(i=130, j=70, k=50, x=5, y=3, z=4), None),
    "trace_of_repeated_isolated": ("xikx", "kj", "ij", dict(i=60, j=50, k=40, x=9), None),
    "all_of_B_isolated": ("ik", "xy", "ik", dict(i=80, k=60, x=7, y=5), None),            # B' is a scalar
    "padded_negative": ("ikx", "kj", "ij", dict(i=100, j=64, k=48, x=5), (-1, 104, 104 * 50)),
    "with_batch": ("hixk", "khj", "ijh", dict(h=3, i=70, j=66, k=40, x=4), None),
}


@pytest.mark.parametrize("dtype", REAL_AND_COMPLEX)
@pytest.mark.parametrize("name", list(CASE4))
def test_case4_isolated_labels_are_summed_first(api, handle, name, dtype):
    """Case 4: labels that occur in one input only.  The default plan sums that input over them in
    a kernel of its own (workspace) and contracts the result with the tiled kernel; with the
    pre-reduction switched off the generic kernel sums them inside the contraction.  Both must
    match the oracle, which follows the definition."""
    la, lb, ld, ext, sA = CASE4[name]
    A = helpers.random_tensor(91, _ext(la, ext), sA, dtype)
    B = helpers.random_tensor(92, _ext(lb, ext), None, dtype)
    C = helpers.random_tensor(93, _ext(ld, ext), None, dtype)
    D = inputs.place(None, _ext(ld, ext), None, dtype)
    cplx = dtype.is_complex
    alpha = complex(0.5, 0.25) if cplx else 0.5
    worst, status, _ = helpers.run_case(handle, A, la, B, lb, C, D, ld, alpha, 1.0, conjA=cplx, conjB=cplx, want_status=True)
    assert worst <= 1.0, worst
    sums = 2 if name == "both_inputs" else 1
    assert status["launches"] >= 1 + sums
    worst, status, _ = helpers.run_case(handle, A, la, B, lb, C, D, ld, alpha, 1.0, conjA=cplx, conjB=cplx,
                                        pre_reduce=False, want_status=True)
    assert worst <= 1.0 and status["launches"] == 1 and status["kernel"] == api.KERNEL_GENERIC
    if name == "x_slowest_in_A":
        worst, _, _ = helpers.run_case(handle, A, la, B, lb, C, D, ld, alpha, 1.0, conjA=cplx, conjB=cplx, host_path=True)
        assert worst <= 1.0


def test_bounded_wait_gives_up_and_the_context_stays_usable(api, handle):
    """Failure detection on the device: a wait on a barrier that nothing signals must run out of
    polls, record its code and let the kernel return; afterwards the same context still computes."""
    code, gave_up = api.selftest_bounded_wait(handle, torch.cuda.current_stream().cuda_stream, polls=500)
    assert code == 7 and gave_up == 64
    torch.cuda.synchronize()
    ext = dict(i=70, j=45, k=40)
    A = helpers.random_tensor(101, _ext("ik", ext), None, torch.float64)
    B = helpers.random_tensor(102, _ext("kj", ext), None, torch.float64)
    D = inputs.place(None, _ext("ij", ext), None, torch.float64)
    worst, _, _ = helpers.run_case(handle, A, "ik", B, "kj", None, D, "ij")
    assert worst <= 1.0


SHORT_K = {
    # name: (labelsA, labelsB, labelsD, extents, strides of D or None, beta)
    "rows_rows": ("ik", "jk", "ij", dict(i=300, j=200, k=64), None, 0.0),
    "k_k_ragged_k": ("ki", "kj", "ij", dict(i=300, j=200, k=36), None, -0.5),
    "rows_k": ("ik", "kj", "ij", dict(i=132, j=260, k=20), None, 1.5),
    "k_rows_outer_product": ("ki", "jk", "ij", dict(i=256, j=128, k=4), None, 0.0),
    "transposed_output": ("ik", "kj", "ji", dict(i=260, j=136, k=48), None, 0.5),
    "strided_output_element_stores": ("ik", "kj", "ij", dict(i=256, j=130, k=32), (2, 520), 0.25),
    "padded_output": ("ik", "kj", "ij", dict(i=256, j=130, k=64), (1, 260), 0.0),
    "batch_label_many_tiles": ("kiz", "jkz", "ijz", dict(i=128 * 9 + 4, j=128 * 6 + 8, k=24, z=3), None, 2.0),
    "interleaved_small_modes": ("axbycw", "wfygxh", "afbgch", dict(a=4, b=8, c=8, f=4, g=8, h=4, x=4, y=4, w=4), None, 0.0),
}


@pytest.mark.parametrize("name", list(SHORT_K))
def test_short_k_streaming_kernel(api, handle, name):
    """The fp32 streaming kernel for contracted extents up to 64 (tcgen05, piece-order loads and stores),
    forced through the attribute: both memory orders of either operand, K that is no multiple of 8 (zero
    padded), ragged last tiles, beta != 0, a batch label with more tiles than SMs, an output written in
    16-byte pieces or element by element, and interleaved modes of extent 4 to 8."""
    la, lb, ld, ext, sD, beta = SHORT_K[name]
    A = helpers.random_tensor(111, _ext(la, ext), None, torch.float32)
    B = helpers.random_tensor(112, _ext(lb, ext), None, torch.float32)
    C = helpers.random_tensor(113, _ext(ld, ext), sD, torch.float32)
    D = inputs.place(None, _ext(ld, ext), sD, torch.float32)
    worst, status, _ = helpers.run_case(handle, A, la, B, lb, C if beta else None, D, ld, 0.75, beta, kernel=api.KERNEL_TILED,
                                        variant=23, want_status=True)
    assert worst <= 1.0, worst
    assert status["variant"] == 23 and status["launches"] == 1


def test_short_k_streaming_kernel_is_the_default_for_the_tensor_network_workload(api, handle):
    for name in ("cfg5", "cfg5b"):
        worst, status, _ = helpers.workload_case(handle, small_workloads()[name], want_status=True)
        assert worst <= 1.0 and status["variant"] == 23, (name, worst, status)


def test_short_k_streaming_kernel_declines_what_it_cannot_fetch_in_16_byte_pieces(api, handle):
    """K above 64, or an operand whose strides or base pointer rule out 16-byte pieces: the mma.sync
    kernel with the same tiles runs instead, and the result is the same."""
    ext = dict(i=256, j=128, k=72)
    A = helpers.random_tensor(121, _ext("ik", ext), None, torch.float32)
    B = helpers.random_tensor(122, _ext("kj", ext), None, torch.float32)
    D = inputs.place(None, _ext("ij", ext), None, torch.float32)
    worst, status, _ = helpers.run_case(handle, A, "ik", B, "kj", None, D, "ij", kernel=api.KERNEL_TILED, variant=23, want_status=True)
    assert worst <= 1.0 and status["variant"] == 6
    buf = helpers.random_tensor(123, (256 * 32 + 8,), None, torch.float32)
    A_off = inputs.StridedTensor(buf.buffer, (256, 32), (1, 256), 1)      # base pointer 4 bytes past a 16-byte boundary
    B2 = helpers.random_tensor(124, (32, 128), None, torch.float32)
    worst, status, _ = helpers.run_case(handle, A_off, "ik", B2, "kj", None, D, "ij", kernel=api.KERNEL_TILED, variant=23, want_status=True)
    assert worst <= 1.0 and status["variant"] == 6


@pytest.mark.parametrize("limit", [0, 1])
@pytest.mark.parametrize("dtype,variant", [(torch.float64, 2), (torch.float64, 1), (torch.complex128, 0), (torch.float32, 7),
                                           (torch.float32, 13), (torch.float32, 21), (torch.float32, 23)])
def test_waits_that_run_out_are_reported_and_the_operation_recovers(api, handle, dtype, variant, limit):
    """Failure detection in the real kernels.  With a poll limit of zero every device-side wait gives up at
    once; with a limit of one, waits on shared-memory stages may run out while their copies are still in
    flight (that depends on timing; when none did, the result must simply be right).  Either way the kernel
    must return (nothing traps or hangs), the operation's device error word must tell, bytes outside D's
    elements must stay untouched, and after the limit is put back and the word cleared the same operation
    computes the right result."""
    ext = dict(i=128 * 3 + 8, j=128 * 2 + 4, k=64 if variant == 23 else 200)
    A = helpers.random_tensor(131, _ext("ki", ext), None, dtype)
    B = helpers.random_tensor(132, _ext("kj", ext), None, dtype)
    D = inputs.place(None, _ext("ij", ext), (1, ext["i"] + 4), dtype)
    dt = api.dtype_code(dtype)
    tA, tB, tD = (api.TensorInfo(handle, dt, x.extents, x.strides) for x in (A, B, D))
    op = api.Contraction(handle, tA, "ki", tB, "kj", None, "ij", tD, "ij", 1.0, 0.0)
    op.set_attr(api.ATTR_KERNEL, api.KERNEL_TILED)
    op.set_attr(api.ATTR_VARIANT, variant)
    assert op.variant == variant
    dA, dB, dD = A.to("cuda"), B.to("cuda"), D.to("cuda")
    need = op.workspace_size()
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device="cuda")
    run = lambda: op.execute(torch.cuda.current_stream().cuda_stream, dA.data_ptr(), dB.data_ptr(), 0, dD.data_ptr(),
                             workspace=ws.data_ptr(), workspace_bytes=need)
    op.set_attr(api.ATTR_POLL_LIMIT, limit)
    run()
    torch.cuda.synchronize()
    word = op.device_error
    if limit == 0:
        assert word != 0
        assert torch.equal(dD.buffer.cpu().view(torch.uint8), D.buffer.view(torch.uint8))   # nothing was written
    pos = D.offsets()
    assert helpers.canary_intact(D.buffer, dD.buffer.cpu(), pos)
    want = D.clone()
    scale = oracle.contract(A.numpy(), "ki", B.numpy(), "kj", None, "ij", want.numpy(), "ij", 1.0, 0.0)
    if word == 0:
        assert helpers.compare(dD.buffer.cpu()[pos].numpy(), want.buffer[pos].numpy(), scale, dtype) <= 1.0
    else:
        assert 1 <= word <= 11
    op.set_attr(api.ATTR_POLL_LIMIT, 1 << 22)
    op.set_attr(api.ATTR_DEVICE_ERROR, 0)
    assert op.device_error == 0
    run()
    torch.cuda.synchronize()
    assert op.device_error == 0
    assert helpers.compare(dD.buffer.cpu()[pos].numpy(), want.buffer[pos].numpy(), scale, dtype) <= 1.0
    assert helpers.canary_intact(D.buffer, dD.buffer.cpu(), pos)


def test_host_buffer_entry_point_reports_a_device_timeout(api, handle):
    """btc_execute_host synchronises, so it can and does return DEVICE_TIMEOUT when a wait gave up."""
    ext = dict(i=256, j=256, k=256)
    A = helpers.random_tensor(141, _ext("ki", ext), None, torch.float64)
    B = helpers.random_tensor(142, _ext("kj", ext), None, torch.float64)
    D = inputs.place(None, _ext("ij", ext), None, torch.float64)
    tA, tB, tD = (api.TensorInfo(handle, api.F64, x.extents, x.strides) for x in (A, B, D))
    op = api.Contraction(handle, tA, "ki", tB, "kj", None, "ij", tD, "ij", 1.0, 0.0)
    op.set_attr(api.ATTR_KERNEL, api.KERNEL_TILED)
    op.set_attr(api.ATTR_POLL_LIMIT, 1)
    hD = D.clone()
    try:
        op.execute_host(0, A.data_ptr(), B.data_ptr(), 0, hD.data_ptr())
        timed_out = False
    except api.BtcError as e:
        assert e.code == api.ERR_DEVICE_TIMEOUT
        timed_out = True
    assert timed_out == (op.device_error != 0)
    op.set_attr(api.ATTR_POLL_LIMIT, 1 << 22)
    op.set_attr(api.ATTR_DEVICE_ERROR, 0)
    op.execute_host(0, A.data_ptr(), B.data_ptr(), 0, hD.data_ptr())
    want = D.clone()
    scale = oracle.contract(A.numpy(), "ki", B.numpy(), "kj", None, "ij", want.numpy(), "ij", 1.0, 0.0)
    pos = D.offsets()
    assert helpers.compare(hD.buffer[pos].numpy(), want.buffer[pos].numpy(), scale, torch.float64) <= 1.0


STREAM = {
    # name: (labelsA, labelsB, labelsD, extents, strides of D or None)
    "outer_product_vector_rows": ("ij", "kl", "ijkl", dict(i=64, j=9, k=7, l=5), None),
    "outer_product_odd_rows": ("ij", "kl", "ijkl", dict(i=37, j=9, k=7, l=5), None),
    "rank_two_update": ("ik", "kj", "ij", dict(i=260, j=130, k=2), None),
    "four_contracted_batch": ("kiz", "jkz", "ijz", dict(i=72, j=50, k=4, z=6), None),
    "three_contracted_rows_strided_in_A": ("ki", "kj", "ij", dict(i=128, j=33, k=3), None),
    "scalar_times_tensor_permuted": ("", "ijk", "kji", dict(i=20, j=12, k=36), None),
    "hadamard_three_labels": ("ijk", "ijk", "ijk", dict(i=32, j=11, k=9), None),
    "padded_output": ("i", "j", "ij", dict(i=96, j=40), (1, 100)),
}


@pytest.mark.parametrize("dtype", REAL_AND_COMPLEX)
@pytest.mark.parametrize("name", list(STREAM))
def test_streaming_kernel_for_at_most_four_contracted_indices(api, handle, name, dtype):
    """Outer products, rank-k updates with k <= 4, a scalar operand, Hadamard products: the streaming kernel
    (one thread per 16 bytes of D) for every element type, with and without 16-byte rows in D and A, beta != 0,
    conjugation, a batch label, padding in D."""
    la, lb, ld, ext, sD = STREAM[name]
    A = helpers.random_tensor(151, _ext(la, ext), None, dtype)
    B = helpers.random_tensor(152, _ext(lb, ext), None, dtype)
    C = helpers.random_tensor(153, _ext(ld, ext), sD, dtype)
    D = inputs.place(None, _ext(ld, ext), sD, dtype)
    cplx = dtype.is_complex
    alpha = complex(0.75, -1.25) if cplx else 0.75
    beta = complex(-0.5, 0.25) if cplx else -0.5
    worst, status, _ = helpers.run_case(handle, A, la, B, lb, C, D, ld, alpha, beta, conjA=cplx, conjB=cplx, conjC=cplx,
                                        want_status=True)
    assert worst <= 1.0, worst
    assert status["variant"] == 100 and status["launches"] == 1, status
