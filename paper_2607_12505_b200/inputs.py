"""Seeded synthetic inputs with the shapes of the ViT / Swin linear layers.

This module draws random tensors and names layer shapes.  It holds none of the
method's arithmetic (no packing, no GEMM): both the CPU oracle's tests and the
CUDA library's tests feed from it so that they see identical inputs.

Recipe (stand-ins for DeiT / Swin / ViT-L activations and pruned weights; no
dataset or trained weight is involved):
  * int8 X: uniform on [-128, 127].
  * int8 W: every aligned group of m consecutive k in a row gets exactly n
    nonzero positions (uniform over the C(m,n) masks, drawn as the n smallest of
    m random keys); kept values uniform on {-127..-1, 1..127}.
  * fp16 X, W: N(0, 0.02^2) rounded to binary16 (a few values are subnormal);
    kept weights that round to zero are replaced by the smallest subnormal so
    the mask keeps exactly n nonzeros.
  * ``at_most=True`` additionally zeroes ~25 % of the kept weights (groups with
    fewer than n nonzeros), and int8 weights may then include -128.
"""
from __future__ import annotations

import zlib

import numpy as np

BASE_SEED = 260712505


def tensor_seed(*key) -> int:
    """Stable 63-bit seed from the base seed and a readable key."""
    text = "/".join(str(k) for k in key)
    return (BASE_SEED * 1000003 + zlib.crc32(text.encode())) & 0x7FFFFFFFFFFFFFFF


def _rng(*key) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(tensor_seed(*key)))


def nm_mask(rng: np.random.Generator, O: int, K: int, n: int, m: int) -> np.ndarray:
    """Boolean [O, K] mask with exactly n True per aligned group of m."""
    assert K % m == 0 and 1 <= n <= m
    G = K // m
    if n == m:
        return np.ones((O, K), dtype=bool)
    keys = rng.random((O, G, m), dtype=np.float32)
    pick = np.argpartition(keys, n - 1, axis=2)[:, :, :n]      # tie-safe: exactly n indices
    mask = np.zeros((O, G, m), dtype=bool)
    np.put_along_axis(mask, pick, True, axis=2)
    return mask.reshape(O, K)


def x_i8(T: int, K: int, *key) -> np.ndarray:
    return _rng("x_i8", T, K, *key).integers(-128, 128, size=(T, K), dtype=np.int8)


def w_i8(O: int, K: int, n: int, m: int, *key, at_most: bool = False) -> np.ndarray:
    rng = _rng("w_i8", O, K, n, m, at_most, *key)
    mask = nm_mask(rng, O, K, n, m)
    mag = rng.integers(1, 128, size=(O, K), dtype=np.int16)
    sign = rng.integers(0, 2, size=(O, K), dtype=np.int16) * 2 - 1
    W = (mag * sign).astype(np.int8)
    if at_most:
        W[rng.random((O, K)) < 0.05] = -128
        mask &= rng.random((O, K)) >= 0.25
    return np.where(mask, W, np.int8(0)).astype(np.int8)


def x_f16(T: int, K: int, *key, std: float = 0.02) -> np.ndarray:
    return (_rng("x_f16", T, K, *key).standard_normal((T, K), dtype=np.float32) * std).astype(np.float16)


def w_f16(O: int, K: int, n: int, m: int, *key, std: float = 0.02, at_most: bool = False) -> np.ndarray:
    rng = _rng("w_f16", O, K, n, m, at_most, *key)
    mask = nm_mask(rng, O, K, n, m)
    W = (rng.standard_normal((O, K), dtype=np.float32) * std).astype(np.float16)
    tiny = np.float16(5.9604645e-08)              # smallest positive subnormal
    W = np.where(W == 0, tiny, W)
    if at_most:
        mask &= rng.random((O, K)) >= 0.25
    return np.where(mask, W, np.float16(0)).astype(np.float16)


def small_int_f16(shape, *key, lo: int = -8, hi: int = 8) -> np.ndarray:
    """fp16 tensor of small integers: every partial sum is exact in fp32."""
    return _rng("small_int", *shape, *key).integers(lo, hi + 1, size=shape).astype(np.float16)


# ---------------------------------------------------------------------------
# Layer shapes (K -> O) of the benchmark configurations.
# ---------------------------------------------------------------------------

def vit_block_layers(dim: int, mlp_ratio: int = 4):
    """(name, K, O) of the four linear layers of one transformer block."""
    return [("qkv", dim, 3 * dim), ("proj", dim, dim),
            ("fc1", dim, mlp_ratio * dim), ("fc2", mlp_ratio * dim, dim)]


def cfg0():
    """Single INT8 2:4 GEMM: T=197, K=384, O=384."""
    return dict(T=197, K=384, O=384, n=2, m=4, dtype="i8")


def cfg1_layers():
    """DeiT-Small linear stack, batch 64: T = 64*197; W at 2:4, 1:4 and 2:8."""
    T = 64 * 197
    out = []
    for (n, m) in [(2, 4), (1, 4), (2, 8)]:
        for (name, K, O) in vit_block_layers(384):
            out.append(dict(name=f"deit_s.{name}.{n}:{m}", T=T, K=K, O=O, n=n, m=m, dtype="i8"))
    return out


CFG2_CHOICES = [(4, 4), (2, 4), (1, 4), (2, 8), (1, 8)]     # (4,4) = dense


def cfg2_layers(dtype: str = "i8", blocks: int = 12):
    """DeiT-Base, 12 blocks, batch 128: per-layer n:m drawn by seed."""
    T = 128 * 197
    rng = _rng("cfg2_nm")
    out = []
    for blk in range(blocks):
        for (name, K, O) in vit_block_layers(768):
            n, m = CFG2_CHOICES[int(rng.integers(0, len(CFG2_CHOICES)))]
            out.append(dict(name=f"deit_b.{blk}.{name}.{n}:{m}", T=T, K=K, O=O, n=n, m=m, dtype=dtype))
    return out


def cfg3_layers():
    """Swin-T-shaped layers, batch 64: 4 stages, W at 2:4 and 4:8."""
    out = []
    for stage, (tok, C) in enumerate([(3136, 96), (784, 192), (196, 384), (49, 768)]):
        T = 64 * tok
        for (n, m) in [(2, 4), (4, 8)]:
            for (name, K, O) in vit_block_layers(C):
                out.append(dict(name=f"swin_t.s{stage + 1}.{name}.{n}:{m}", T=T, K=K, O=O, n=n, m=m, dtype="i8"))
    return out


def cfg4_layers(dtypes=("i8", "f16"), batches=(1, 8, 64, 256)):
    """ViT-Large/16 layers swept over batch and n:m."""
    out = []
    for dt in dtypes:
        for B in batches:
            for (n, m) in [(2, 4), (4, 8), (2, 8), (1, 8)]:
                for (name, K, O) in [("qkv", 1024, 3072), ("fc1", 1024, 4096), ("fc2", 4096, 1024)]:
                    out.append(dict(name=f"vit_l.b{B}.{name}.{n}:{m}.{dt}", T=197 * B, K=K, O=O, n=n, m=m, dtype=dt))
    return out


MODELS = {
    # name: (blocks, hidden, tokens per image)
    "deit_s": (12, 384, 197),
    "deit_b": (12, 768, 197),
    "vit_l": (24, 1024, 197),
}


def layer_shapes(model: str):
    """(name, K, O) of every linear layer of a ViT-family model, block by block."""
    blocks, d, _ = MODELS[model]
    return [(f"b{b}.{name}", K, O) for b in range(blocks) for (name, K, O) in vit_block_layers(d)]


def make_layer(spec: dict, *key, at_most: bool = False):
    """(X, W) numpy arrays for one layer spec."""
    k = (spec.get("name", ""),) + key
    if spec["dtype"] == "i8":
        return (x_i8(spec["T"], spec["K"], *k),
                w_i8(spec["O"], spec["K"], spec["n"], spec["m"], *k, at_most=at_most))
    return (x_f16(spec["T"], spec["K"], *k),
            w_f16(spec["O"], spec["K"], spec["n"], spec["m"], *k, at_most=at_most))
