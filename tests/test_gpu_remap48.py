"""The three-chunk K remap (NM_PATH_UMMA_REMAP48): weights with up to 4 nonzeros per 8 k run on the 2:4
sparse tensor core over K + K/2, the extra K range reading gathered copies of the activations
k+0, k+1, k+4, k+5 of every group.  Same result as every other path: bit-exact INT8, FP16 within
1e-3 * sum|x||w| of the CPU oracle."""
import numpy as np
import pytest

from paper_2607_12505_b200 import binding as nm
from paper_2607_12505_b200 import inputs
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

REMAP = nm.NM_PATH_UMMA_REMAP48


@pytest.mark.parametrize("n,m", [(4, 8), (3, 8), (2, 8)])
@pytest.mark.parametrize("dtype", ["i8", "f16"])
def test_remap_ragged(n, m, dtype):
    # ragged in every dimension; K is not a multiple of the sparse K step, so the main range is padded
    gu.run_case(300, 330, 1008, n, m, dtype=dtype, at_most=True, key="remap", path=REMAP)


@pytest.mark.parametrize("T,O,K", [(197, 1024, 4096), (1576, 3072, 1024), (64, 128, 128), (640, 256, 16)])
@pytest.mark.parametrize("dtype", ["i8", "f16"])
def test_remap_shapes(T, O, K, dtype):
    gu.run_case(T, O, K, 4, 8, dtype=dtype, key="remap_shape", path=REMAP)


def test_remap_all_four_nonzeros_in_one_chunk():
    """The worst case of the remap: both excess elements of a chunk move to the third chunk."""
    T, O, K = 96, 130, 512
    rng = np.random.default_rng(11)
    W = np.zeros((O, K), dtype=np.int8)
    for o in range(O):
        for g in range(K // 8):
            half = int(rng.integers(0, 2))
            W[o, g * 8 + half * 4: g * 8 + half * 4 + 4] = rng.integers(1, 128, size=4) * rng.choice([-1, 1], size=4)
    X = inputs.x_i8(T, K, "remap_worst")
    Y, plan, w = gu.gpu_spmm(X, W, 4, 8, path=REMAP)
    assert w.desc.images & nm.NM_IMG_REMAP48
    gu.check_against_oracle(X, W, 4, 8, Y)
    # and the identity probe: Y = W~^T exactly
    Xi = np.eye(K, dtype=np.int8)
    Yi, _, _ = gu.gpu_spmm(Xi, W, 4, 8, path=REMAP)
    assert np.array_equal(Yi, W.T.astype(np.int32))


def test_remap_needs_its_image_and_a_plain_plan():
    import torch
    W = inputs.w_i8(256, 512, 4, 8, "remap_err")
    w = nm.nm_compress(W, 4, 8)                                       # no remap image
    X = torch.zeros((64, 512), dtype=torch.int8, device="cuda")
    plan = gu.make_plan(64, w, nm.NM_OUT_I32, path=REMAP)
    with pytest.raises(nm.NMError) as e:
        nm.nm_spmm(X, w, plan=plan, out_dtype=nm.NM_OUT_I32)
    assert e.value.status == nm.NM_ERR_UNSUPPORTED
    w2 = nm.nm_compress(W, 4, 8, images=nm.NM_IMG_AUTO | nm.NM_IMG_REMAP48)
    plan = gu.make_plan(64, w2, nm.NM_OUT_I32, path=REMAP)
    plan.workspace_bytes = 0                                           # the gathered activations need the workspace
    Y = torch.empty((64, 256), dtype=torch.int32, device="cuda")
    st = nm.nm_spmm_raw(X.data_ptr(), 512, 64, w2, plan, Y.data_ptr(), 256, nm.NM_OUT_I32)
    assert st == nm.NM_ERR_WORKSPACE
    # the automatic plan never selects the remap
    assert nm.nm_plan_create(64, w2, nm.NM_OUT_I32, 0).path != REMAP
