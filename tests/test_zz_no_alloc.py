"""nm_spmm_static_scratch: the split-K GEMM for callers that cannot allocate device memory
(a server whose memory was handed out at start-up, a loop where cudaMalloc would stall the
device).  Its partial sums go to the library's built-in scratch array; the result must equal
what nm_spmm produces with a caller-provided workspace, call after call."""
import numpy as np
import pytest
import torch

from paper_2607_12505_b200 import binding as nm
from paper_2607_12505_b200 import inputs
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", ["i8", "f16"])
def test_static_scratch_matches_workspace_entry_point_twice(dtype):
    T, O, K, n, m = 197, 1024, 4096, 2, 4
    od = nm.NM_OUT_I32 if dtype == "i8" else nm.NM_OUT_F32
    W = (inputs.w_i8 if dtype == "i8" else inputs.w_f16)(O, K, n, m, "noalloc")
    w = nm.nm_compress(W, n, m)
    plan = gu.make_plan(T, w, od, path=nm.NM_PATH_UMMA_SP24, split_k=8, tile_t=128)
    assert 0 < plan.workspace_bytes <= nm.NM_STATIC_SCRATCH_BYTES
    stream = torch.cuda.current_stream().cuda_stream
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    for call in range(2):                      # two calls in a row share the same scratch array
        X = (inputs.x_i8 if dtype == "i8" else inputs.x_f16)(T, K, "noalloc", call)
        Xd = torch.from_numpy(X).cuda()
        want = nm.nm_spmm(Xd, w, plan=plan, out_dtype=od)          # existing entry point, caller workspace
        got = torch.full_like(want, 77)
        st = nm.nm_spmm_static_scratch_raw(Xd.data_ptr(), K, T, w, plan, got.data_ptr(), O, od,
                                           status.data_ptr(), stream)
        assert st == nm.NM_OK, nm.lib().nm_status_string(st)
        torch.cuda.synchronize()
        assert int(status[0]) == 0
        if dtype == "i8":
            assert torch.equal(got, want)                           # INT8: bit-exact
            gu.check_against_oracle(X, W, n, m, got.cpu().numpy())  # ... and equal to the CPU oracle
        else:
            gu.check_against_oracle(X, W, n, m, got.cpu().numpy())  # FP16: the tests' 1e-3 * sum|x||w| bound
            assert torch.equal(got, want)                           # and the same plan sums in the same order


def test_static_scratch_rejects_plans_that_need_more():
    T, O, K = 2048, 1024, 4096
    w = nm.nm_compress(inputs.w_i8(O, K, 2, 4, "noalloc_big"), 2, 4)
    plan = gu.make_plan(T, w, nm.NM_OUT_I32, path=nm.NM_PATH_UMMA_SP24, split_k=8, tile_t=128)
    assert plan.workspace_bytes > nm.NM_STATIC_SCRATCH_BYTES
    X = torch.zeros((T, K), dtype=torch.int8, device="cuda")
    Y = torch.empty((T, O), dtype=torch.int32, device="cuda")
    st = nm.nm_spmm_static_scratch_raw(X.data_ptr(), K, T, w, plan, Y.data_ptr(), O, nm.NM_OUT_I32)
    assert st == nm.NM_ERR_WORKSPACE
    # a plan without split-K needs no scratch and goes through
    plan1 = gu.make_plan(T, w, nm.NM_OUT_I32, path=nm.NM_PATH_UMMA_SP24, split_k=1)
    assert nm.nm_spmm_static_scratch_raw(X.data_ptr(), K, T, w, plan1, Y.data_ptr(), O, nm.NM_OUT_I32) == nm.NM_OK
    torch.cuda.synchronize()
    assert int(Y.abs().max()) == 0


def _static(Xd, ldx, T, w, plan, od, O):
    """One call of the allocation-free entry point; returns (Y, status word)."""
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    Y = torch.full((T, O), 55, dtype=nm._out_torch_dtype(od), device="cuda")
    st = nm.nm_spmm_static_scratch_raw(Xd.data_ptr(), ldx, T, w, plan, Y.data_ptr(), O, od, status.data_ptr(),
                                       torch.cuda.current_stream().cuda_stream)
    assert st == nm.NM_OK, nm.lib().nm_status_string(st)
    torch.cuda.synchronize()
    return Y, int(status[0])


def test_static_scratch_without_a_plan_never_fails_on_alignment():
    """No plan given and an X pitch that TMA cannot address: like nm_spmm, the call falls back to
    the CUDA-core path instead of returning NM_ERR_ALIGN."""
    T, O, K, n, m = 64, 256, 512, 2, 4
    X = inputs.x_i8(T, K, "noalloc_unaligned")
    W = inputs.w_i8(O, K, n, m, "noalloc_unaligned")
    w = nm.nm_compress(W, n, m)
    Xwide = torch.zeros((T, K + 1), dtype=torch.int8, device="cuda")     # pitch K + 1 bytes: not a 16-byte multiple
    Xwide[:, :K] = torch.from_numpy(X).cuda()
    Xd = Xwide[:, :K]
    for _ in range(2):
        got, status = _static(Xd, K + 1, T, w, None, nm.NM_OUT_I32, O)
        assert status == 0
        want = torch.empty_like(got)
        ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
        assert nm.nm_spmm_raw(Xd.data_ptr(), K + 1, T, w, None, want.data_ptr(), O, nm.NM_OUT_I32, ws.data_ptr(), ws.numel()) == nm.NM_OK
        torch.cuda.synchronize()
        assert torch.equal(got, want)
        gu.check_against_oracle(X, W, n, m, got.cpu().numpy())


def test_static_scratch_without_a_plan_degrades_when_the_dense_copy_does_not_fit():
    """Canonical image only (4:8) and a weight whose zero-filled dense copy is larger than the fixed
    array: the automatic plan decodes on chip instead of refusing the call."""
    T, O, K, n, m = 64, 4096, 4608, 4, 8
    assert O * K > nm.NM_STATIC_SCRATCH_BYTES
    X = inputs.x_i8(T, K, "noalloc_decode")
    W = inputs.w_i8(O, K, n, m, "noalloc_decode")
    w = nm.nm_compress(W, n, m, images=nm.NM_IMG_CANONICAL)
    assert nm.nm_plan_create(T, w, nm.NM_OUT_I32, 0).path == nm.NM_PATH_UMMA_EXPAND
    Xd = torch.from_numpy(X).cuda()
    for _ in range(2):
        got, status = _static(Xd, K, T, w, None, nm.NM_OUT_I32, O)
        assert status == 0
        gu.check_against_oracle(X, W, n, m, got.cpu().numpy())
        want = nm.nm_spmm(Xd, w, out_dtype=nm.NM_OUT_I32)              # planner's choice with all the scratch it asks for
        torch.cuda.synchronize()
        assert torch.equal(got, want)


@pytest.mark.parametrize("dtype", ["i8", "f16"])
def test_static_scratch_holds_the_dense_copy_and_the_slices_of_an_expand_plan(dtype):
    """Canonical image only: the dense copy (head of the scratch) and the split-K slices behind it
    both live in the fixed array."""
    T, O, K, n, m = 197, 1024, 2048, 4, 8
    od = nm.NM_OUT_I32 if dtype == "i8" else nm.NM_OUT_F32
    W = (inputs.w_i8 if dtype == "i8" else inputs.w_f16)(O, K, n, m, "noalloc_expand")
    w = nm.nm_compress(W, n, m, images=nm.NM_IMG_CANONICAL)
    plan = gu.make_plan(T, w, od, path=nm.NM_PATH_UMMA_EXPAND, split_k=4, tile_t=64, cta_group=1)
    head = O * K * (1 if dtype == "i8" else 2)
    assert head < plan.workspace_bytes <= nm.NM_STATIC_SCRATCH_BYTES
    for call in range(2):
        X = (inputs.x_i8 if dtype == "i8" else inputs.x_f16)(T, K, "noalloc_expand", call)
        Xd = torch.from_numpy(X).cuda()
        got, status = _static(Xd, K, T, w, plan, od, O)
        assert status == 0
        gu.check_against_oracle(X, W, n, m, got.cpu().numpy())
        want = nm.nm_spmm(Xd, w, plan=plan, out_dtype=od)
        torch.cuda.synchronize()
        assert torch.equal(got, want)
