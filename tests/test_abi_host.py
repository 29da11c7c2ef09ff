"""CPU-only checks of the C-ABI library: it loads, exports what include/nm.h declares,
packs byte-identically to the oracle, plans deterministically, and rejects bad input.
No kernel is launched here."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import nm_oracle as orc
from paper_2607_12505_b200 import binding as nm
from paper_2607_12505_b200 import inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
NM_SET = [(2, 4), (1, 4), (2, 8), (1, 8), (4, 8), (3, 8), (4, 4), (8, 8), (1, 2), (3, 16)]


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "nm.h")).read()
    declared = re.findall(r"^NM_API\s+[\w\s\*]+?\b(nm_\w+)\s*\(", header, flags=re.M)
    assert set(declared) == set(nm.EXPORTS), (sorted(declared), sorted(nm.EXPORTS))
    L = nm.lib()
    for name in declared:
        assert hasattr(L, name), f"{name} not exported"
    assert L.nm_status_string(nm.NM_ERR_TIMEOUT) == b"NM_ERR_TIMEOUT"
    c0 = nm.launch_count()
    assert isinstance(c0, int) and c0 >= 0
    nm.nm_plan_shape(197, 384, 384, 2, 4, nm.NM_I8, nm.NM_OUT_I32, nm.NM_IMG_CANONICAL | nm.NM_IMG_HW24)
    assert nm.launch_count() == c0, "host-only calls launch nothing"


@pytest.mark.parametrize("n,m", NM_SET)
@pytest.mark.parametrize("dtype", ["i8", "f16"])
def test_canonical_bytes_equal_oracle(n, m, dtype):
    O, K = 37, 12 * m
    W = (inputs.w_i8 if dtype == "i8" else inputs.w_f16)(O, K, n, m, "abi", at_most=True)
    pw = nm.nm_compress_host(W, n, m)
    canon = pw.buf[pw.desc.off_canonical:pw.desc.off_canonical + orc.packed_bytes(O, K, n, m, pw.desc.dtype)]
    assert np.array_equal(canon, orc.compress(W, n, m))


def _decode_hw24(pw, dtype, remap=False):
    """Test-side reader of the hardware 2:4 image: rebuilds W~ from compressed values and
    the 4-bit-per-chunk metadata (two ascending 2-bit positions, low slot first).  remap=True reads
    the 2:4 image of the K-remapped weight instead (same format, longer K)."""
    d = pw.desc
    O, K = d.O, (d.remap_k if remap else d.K)
    off_v, off_m, row_bytes, kblocks = ((d.off_remap_values, d.off_remap_meta, d.remap_row_bytes, d.remap_meta_kblocks) if remap else
                                        (d.off_hw24_values, d.off_hw24_meta, d.hw24_row_bytes, d.hw24_meta_kblocks))
    eb = 1 if dtype == "i8" else 2
    chunks = (K + 3) // 4
    vals = pw.buf[off_v:off_v + O * row_bytes].reshape(O, row_bytes)
    vals = vals.view(np.int8 if dtype == "i8" else np.float16)
    meta = pw.buf[off_m:]
    W = np.zeros((O, chunks * 4), dtype=vals.dtype)
    for o in range(O):
        ot, r = divmod(o, 128)
        for c in range(chunks):
            kb, cc = divmod(c, 32)
            blk = (ot * kblocks + kb) * 2048
            if eb == 1:
                byte, shift = r * 16 + cc // 2, (cc & 1) * 4
            else:
                k = cc * 4
                byte = (r & 7) * 16 + ((r >> 3) & 1) * 2 + (r >> 4) * 256 + ((k >> 4) & 1) * 128 + (k >> 5) * 4 + (k & 15) // 8
                shift = k & 7
            nib = (int(meta[blk + byte]) >> shift) & 0xF
            i0, i1 = nib & 3, nib >> 2
            assert i0 < i1
            W[o, 4 * c + i0] = vals[o, 2 * c]
            W[o, 4 * c + i1] = vals[o, 2 * c + 1]
    return W[:, :K]


@pytest.mark.parametrize("n,m", [(2, 4), (1, 4), (2, 8), (1, 8), (1, 2)])
@pytest.mark.parametrize("dtype", ["i8", "f16"])
def test_hw24_image_roundtrip(n, m, dtype):
    O, K = 150, 264 if m != 8 else 272          # two 128-row tiles, ragged K blocks
    W = (inputs.w_i8 if dtype == "i8" else inputs.w_f16)(O, K, n, m, "hw24", at_most=True)
    pw = nm.nm_compress_host(W, n, m)
    assert pw.desc.images & nm.NM_IMG_HW24 and not pw.desc.images & nm.NM_IMG_DENSE
    assert np.array_equal(_decode_hw24(pw, dtype), W)


@pytest.mark.parametrize("n,m", [(4, 8), (3, 8), (2, 8)])
@pytest.mark.parametrize("dtype", ["i8", "f16"])
def test_remap48_image_folds_back_to_the_weight(n, m, dtype):
    """Three-chunk K remap: the remapped weight is 2:4-clean (the 2:4 packer accepted it), holds the
    moved elements in the third chunks, and folding those back onto k + {0,1,4,5} restores W."""
    O, K = 150, 264 if dtype == "i8" else 136          # K is not a multiple of the sparse K step: the main range is padded
    W = (inputs.w_i8 if dtype == "i8" else inputs.w_f16)(O, K, n, m, "remap", at_most=True)
    if n == 4:                                          # worst cases: all four nonzeros of a group in one 4-chunk
        W[0, :] = 0
        W[0, 0:4] = 3
        W[1, :] = 0
        W[1, 12:16] = -5
    pw = nm.nm_compress_host(W, n, m, images=nm.NM_IMG_AUTO | nm.NM_IMG_REMAP48)
    d = pw.desc
    assert d.images & nm.NM_IMG_REMAP48
    eb = 1 if dtype == "i8" else 2
    assert d.remap_k_main == -(-K * eb // 256) * 256 // eb and d.remap_k == d.remap_k_main + K // 2
    Wr = _decode_hw24(pw, dtype, remap=True)
    assert (np.count_nonzero(Wr.reshape(O, -1, 4), axis=2) <= 2).all()
    assert not Wr[:, K:d.remap_k_main].any()
    back = Wr[:, :K].copy()
    third = Wr[:, d.remap_k_main:].reshape(O, K // 8, 4)
    for j, pos in enumerate((0, 1, 4, 5)):
        cols = np.arange(K // 8) * 8 + pos
        assert not (back[:, cols] != 0)[third[:, :, j] != 0].any(), "a moved element must leave its original place"
        back[:, cols] += third[:, :, j]
    assert np.array_equal(back, W)
    if n == 4:
        assert np.count_nonzero(third) > 0
    # a weight with more than 4 nonzeros in a group of 8 cannot be remapped; dense weights need no image
    W58 = inputs.w_i8(8, 64, 5, 8, "remap58")
    with pytest.raises(nm.NMError) as e:
        nm.nm_compress_host(W58, 5, 8, images=nm.NM_IMG_AUTO | nm.NM_IMG_REMAP48)
    assert e.value.status == nm.NM_ERR_UNSUPPORTED
    # never built unless asked for
    assert not nm.nm_compress_host(W, n, m).desc.images & nm.NM_IMG_REMAP48


def test_image_selection():
    W48 = inputs.w_i8(16, 64, 4, 8, "sel")                 # random 4:8 is not 2:4-clean
    pw = nm.nm_compress_host(W48, 4, 8)
    assert pw.desc.images == nm.NM_IMG_CANONICAL | nm.NM_IMG_DENSE
    with pytest.raises(nm.NMError) as e:
        nm.nm_compress_host(W48, 4, 8, images=nm.NM_IMG_HW24)
    assert e.value.status == nm.NM_ERR_UNSUPPORTED
    # a 4:8 weight that happens to be 2:4-clean gets the sparse image ...
    W24 = inputs.w_i8(16, 256, 2, 4, "sel")
    pw = nm.nm_compress_host(W24, 4, 8)
    assert pw.desc.images == nm.NM_IMG_CANONICAL | nm.NM_IMG_HW24
    # ... unless a row fits in one dense K step (128 bytes): the dense MMA then serves it, and the
    # planner prefers the dense image when both exist
    W24s = inputs.w_i8(16, 64, 2, 4, "sel")
    assert nm.nm_compress_host(W24s, 2, 4).desc.images == nm.NM_IMG_CANONICAL | nm.NM_IMG_DENSE
    assert nm.nm_compress_host(W24s, 2, 4, images=nm.NM_IMG_AUTO | nm.NM_IMG_HW24).desc.images == \
        nm.NM_IMG_CANONICAL | nm.NM_IMG_DENSE | nm.NM_IMG_HW24
    both = nm.NM_IMG_CANONICAL | nm.NM_IMG_DENSE | nm.NM_IMG_HW24
    assert nm.nm_plan_shape(5000, 96, 96, 2, 4, nm.NM_I8, nm.NM_OUT_I32, both).path == nm.NM_PATH_UMMA_DENSE
    assert nm.nm_plan_shape(5000, 96, 256, 2, 4, nm.NM_I8, nm.NM_OUT_I32, both).path == nm.NM_PATH_UMMA_SP24
    assert nm.nm_plan_shape(5000, 96, 64, 2, 4, nm.NM_F16, nm.NM_OUT_F16, both).path == nm.NM_PATH_UMMA_DENSE
    pw = nm.nm_compress_host(inputs.w_i8(16, 64, 4, 4, "sel"), 4, 4)
    assert pw.desc.images == nm.NM_IMG_CANONICAL
    # dense image rows equal W
    pw = nm.nm_compress_host(W48, 4, 8)
    d = pw.desc
    rows = pw.buf[d.off_dense:d.off_dense + 16 * d.dense_row_bytes].reshape(16, d.dense_row_bytes)
    assert np.array_equal(rows[:, :64].view(np.int8), W48)


def test_compress_errors():
    W = inputs.w_i8(8, 32, 2, 4, "err")
    W[5, 8:12] = 1
    with pytest.raises(nm.NMError) as e:
        nm.nm_compress_host(W, 2, 4)
    assert e.value.status == nm.NM_ERR_NOT_NM and "row 5, group 2" in str(e.value)
    L = nm.lib()
    plan = nm.NMPlan()
    assert L.nm_plan_shape(10, 8, 30, 2, 4, 0, 0, 1, 0, ctypes.byref(plan)) == nm.NM_ERR_SHAPE      # K % m
    assert L.nm_plan_shape(10, 8, 32, 5, 4, 0, 0, 1, 0, ctypes.byref(plan)) == nm.NM_ERR_INVALID_ARG  # n > m
    assert L.nm_plan_shape(10, 8, 32, 2, 4, 0, 1, 1, 0, ctypes.byref(plan)) == nm.NM_ERR_INVALID_ARG  # i8 -> f32
    assert L.nm_plan_shape(10, 8, 131072, 2, 4, 0, 0, 1, 0, ctypes.byref(plan)) == nm.NM_ERR_SHAPE    # int32 bound
    assert L.nm_packed_size(8, 30, 2, 4, 0, nm.NM_IMG_AUTO) == 0
    # nm_spmm validates before touching the device
    assert L.nm_spmm(None, 32, 4, None, None, None, 8, 0, None, 0, None, None) == nm.NM_ERR_INVALID_ARG


def test_prune_matches_oracle_and_is_legal():
    rng = np.random.default_rng(3)
    for n, m in [(2, 4), (1, 4), (2, 8), (4, 8)]:
        W = rng.integers(-128, 128, size=(9, 48), dtype=np.int8)
        assert np.array_equal(nm.nm_prune_magnitude(W, n, m), orc.prune_magnitude(W, n, m))
        Wf = rng.standard_normal((9, 48)).astype(np.float16)
        P = nm.nm_prune_magnitude(Wf, n, m)
        assert np.array_equal(P, orc.prune_magnitude(Wf, n, m))
        nm.nm_compress_host(P, n, m)


def test_plan_is_deterministic_and_follows_the_split_rule():
    imgs = nm.NM_IMG_CANONICAL | nm.NM_IMG_HW24
    a = nm.nm_plan_shape(12608, 1152, 384, 2, 4, nm.NM_I8, nm.NM_OUT_I32, imgs).as_dict()
    b = nm.nm_plan_shape(12608, 1152, 384, 2, 4, nm.NM_I8, nm.NM_OUT_I32, imgs).as_dict()
    assert a == b and a["path"] == nm.NM_PATH_UMMA_SP24 and a["split_k"] == 1 and a["workspace_bytes"] == 0
    # plenty of tiles -> no split; few tiles and a long K -> split grows (parallelism priority)
    small = nm.nm_plan_shape(197, 1024, 4096, 2, 4, nm.NM_I8, nm.NM_OUT_I32, imgs, 148)
    assert small.split_k > 1 and small.workspace_bytes > 0
    # The split rule of Section 4.3 on this shape (16 K steps of 128 compressed bytes per row):
    T, O, K, ksteps = 197, 1024, 4096, 16
    tiles = -(-O // 128) * -(-T // small.tile_t)
    in_bytes = T * K + O * (K // 2)
    assert tiles < 148, "K is split only where one round of tiles leaves SMs idle"
    assert ksteps // small.split_k >= 2, "controlled reduction: every slice keeps two K steps"
    assert small.split_k * T * O * 4 <= 2 * in_bytes, "controlled reduction: partial sums do not dominate the traffic"
    # parallelism priority: the split grows until the grid fills the SMs or the next candidate of the
    # set {1, 2, 4, 8, 16} breaks one of the two conditions above
    nxt = 2 * small.split_k
    assert tiles * small.split_k >= 148 or nxt > 16 or ksteps // nxt < 2 or nxt * T * O * 4 > 2 * in_bytes
    # short K -> split stays 1 (controlled reduction)
    shortk = nm.nm_plan_shape(197, 384, 128, 2, 4, nm.NM_I8, nm.NM_OUT_I32, imgs, 148)
    assert shortk.split_k == 1
    # path follows the images present
    assert nm.nm_plan_shape(64, 128, 128, 4, 8, nm.NM_I8, nm.NM_OUT_I32, nm.NM_IMG_CANONICAL).path == nm.NM_PATH_UMMA_EXPAND
    assert nm.nm_plan_shape(64, 128, 128, 4, 8, nm.NM_I8, nm.NM_OUT_I32,
                            nm.NM_IMG_CANONICAL | nm.NM_IMG_DENSE).path == nm.NM_PATH_UMMA_DENSE
    assert nm.nm_plan_shape(64, 128, 128, 8, 8, nm.NM_I8, nm.NM_OUT_I32, nm.NM_IMG_CANONICAL).path == nm.NM_PATH_UMMA_DENSE
    for T in (1, 31, 197, 12608, 200704):
        p = nm.nm_plan_shape(T, 96, 96, 2, 4, nm.NM_I8, nm.NM_OUT_I32, imgs)
        assert p.tile_t % 32 == 0 and 32 <= p.tile_t <= 256 and 1 <= p.stages <= 8


def test_plan_fields_stay_within_what_the_kernels_accept():
    """Every plan the planner can return over a grid of shapes: CTA pairs never split K, keep at
    least two rounds of tiles and need more than one 128-row tile; two issuers only on single-CTA
    tensor-core paths with room for two accumulators next to the sparse metadata."""
    imgs24 = nm.NM_IMG_CANONICAL | nm.NM_IMG_HW24
    imgsd = nm.NM_IMG_CANONICAL | nm.NM_IMG_DENSE
    seen_pair = seen_dual = False
    for T in (1, 64, 197, 788, 1576, 12608, 50432):
        for (K, O) in ((96, 96), (384, 1152), (1024, 3072), (4096, 1024), (1536, 384)):
            for (n, m, dt, imgs) in ((2, 4, nm.NM_I8, imgs24), (4, 8, nm.NM_I8, imgsd), (2, 4, nm.NM_F16, imgs24),
                                     (4, 8, nm.NM_F16, imgsd), (4, 8, nm.NM_I8, nm.NM_IMG_CANONICAL)):
                od = nm.NM_OUT_I32 if dt == nm.NM_I8 else nm.NM_OUT_F16
                p = nm.nm_plan_shape(T, O, K, n, m, dt, od, imgs, 148)
                assert p.cta_group in (1, 2) and p.issuers in (1, 2) and p.split_k in (1, 2, 4, 8, 16)
                assert p.tile_t % 32 == 0 and 32 <= p.tile_t <= 256
                sparse = p.path == nm.NM_PATH_UMMA_SP24
                if p.cta_group == 2:
                    seen_pair = True
                    assert p.split_k == 1 and p.issuers == 1 and O > 128 and p.path != nm.NM_PATH_UMMA_DECODE
                    items = -(-O // 256) * -(-T // p.tile_t)
                    assert -(-items // 74) >= 2
                if p.issuers == 2:
                    seen_dual = True
                    assert p.path in (nm.NM_PATH_UMMA_SP24, nm.NM_PATH_UMMA_DENSE, nm.NM_PATH_UMMA_EXPAND)
                    assert 2 * p.tile_t + (64 if sparse else 0) <= 512
                assert p.merge == nm.NM_MERGE_WORKSPACE and p.reserved == 0     # the on-chip merge is opt-in
                # scratch: the dense copy of a canonical-only weight first, then the split-K slices
                eb = 1 if dt == nm.NM_I8 else 2
                head = -(-(O * (-(-(K * eb) // 16) * 16)) // 256) * 256 if p.path == nm.NM_PATH_UMMA_EXPAND else 0
                if p.split_k > 1:
                    assert p.workspace_bytes == head + p.split_k * (-(-T // p.tile_t) * p.tile_t) * O * 4
                else:
                    assert p.workspace_bytes == head
                assert (p.path == nm.NM_PATH_UMMA_EXPAND) == (imgs == nm.NM_IMG_CANONICAL)
    assert seen_pair and seen_dual
