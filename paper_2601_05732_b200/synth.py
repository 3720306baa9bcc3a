"""Seeded synthetic inputs for the mHC-lite mixing path.

This module only *draws numbers*: it holds none of the method's arithmetic, so
both the CPU oracle's tests and the CUDA path's tests may feed from it.

Every tensor of a workload is drawn from its own counter-based stream
(Philox-4x64 keyed by ``(seed, tensor_index)``), as fp64 normals, and then
rounded to the storage format the layer takes:

* activations (``x_l``, ``y``, upstream gradients) -> bf16, round-to-nearest-even,
  returned as ``uint16`` bit patterns (``bf16_bits``) so that every consumer
  sees the same bits;
* parameters (``W``, ``b``, ``alpha``, ``gain``) -> fp32.

The shapes and value distributions are the ones of the paper's models (n = 4
residual streams, hidden sizes of a few hundred to a few thousand channels,
1024-2048 token sequences; Section 4 and Appendix A), with the weights of the
dynamic mappings small (std 0.02) and alpha = 0.01 as at the paper's
initialisation (Section 4, "Initialization").
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

__all__ = [
    "Workload", "WORKLOADS", "normal", "to_bf16_bits", "bf16_bits_to_f64",
    "bf16_bits_to_f32", "n_logits", "make_layer_inputs", "make_layer_params", "paper_init_bias", "normal_bf16",
    "normal_bf16_rows", "sample_perm_table",
]


# --------------------------------------------------------------------------- #
# random streams and storage formats
# --------------------------------------------------------------------------- #
def normal(seed: int, stream: int, shape, std: float = 1.0) -> np.ndarray:
    """fp64 N(0, std^2) samples from the counter-based stream (seed, stream)."""
    bitgen = np.random.Philox(key=[int(seed) & (2**64 - 1), int(stream) & (2**64 - 1)])
    return np.random.Generator(bitgen).standard_normal(size=shape, dtype=np.float64) * std


_BLOCK = 1 << 22      # elements per independently keyed block of a large bf16 tensor


def _block_gen(seed: int, stream: int, block: int):
    # block 0 continues the plain stream (seed, stream); later blocks take the block index in the key's high bits
    key = [int(seed) & (2**64 - 1), (int(stream) + (int(block) << 32)) & (2**64 - 1)]
    return np.random.Generator(np.random.Philox(key=key))


def normal_bf16(seed: int, stream: int, shape, std: float = 1.0, first: int = 0, count: int | None = None) -> np.ndarray:
    """bf16 bit patterns of N(0, std^2) samples of stream (seed, stream).

    The flat tensor is cut into blocks of 2^22 elements; block b is drawn from its own counter-based
    stream keyed by (seed, stream, b), so the blocks are drawn in parallel on the host threads and any
    range of the tensor can be drawn without the rest.  `first` / `count` select flat elements
    [first, first + count) of the tensor of `shape` (the result is then 1-D).
    """
    total = int(np.prod(shape))
    whole = count is None
    lo = int(first)
    hi = total if whole else lo + int(count)
    assert 0 <= lo <= hi <= total
    out = np.empty(hi - lo, dtype=np.uint16)

    def fill(b):
        b0, b1 = b * _BLOCK, min(total, (b + 1) * _BLOCK)
        v = _block_gen(seed, stream, b).standard_normal(size=b1 - b0, dtype=np.float64)
        if std != 1.0:
            v *= std
        a, z = max(lo, b0), min(hi, b1)
        out[a - lo:z - lo] = to_bf16_bits(v[a - b0:z - b0])

    blocks = range(lo // _BLOCK, (max(hi, lo + 1) - 1) // _BLOCK + 1) if hi > lo else range(0)
    if len(blocks) > 1:
        import concurrent.futures as cf
        import os
        with cf.ThreadPoolExecutor(max_workers=min(len(blocks), os.cpu_count() or 1)) as ex:
            list(ex.map(fill, blocks))
    else:
        for b in blocks:
            fill(b)
    return out.reshape(shape) if whole and lo == 0 else out


def normal_bf16_rows(seed: int, stream: int, shape, rows, std: float = 1.0) -> np.ndarray:
    """Rows `rows` (indices along the first axis) of the tensor normal_bf16(seed, stream, shape), drawn
    without the rest of it: [len(rows), *shape[1:]] bf16 bit patterns."""
    row_elems = int(np.prod(shape[1:]))
    out = np.empty((len(rows),) + tuple(shape[1:]), dtype=np.uint16)
    for i, r in enumerate(rows):
        out[i] = normal_bf16(seed, stream, shape, std, first=int(r) * row_elems, count=row_elems).reshape(shape[1:])
    return out


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp64/fp32 values to bf16 (nearest, ties to even); returns uint16 bits.

    fp64 input whose every value lies in bf16's normal range is rounded directly on its bit pattern
    (one rounding of the 52-bit mantissa to 7 bits, the carry running into the exponent).  Anything
    else (zeros, subnormals, overflow, fp32 input) goes through fp32: the value is first rounded to
    fp32; where that first rounding lands exactly on a bf16 tie, the tie is broken by the sign of the
    first rounding's error so that the result equals a single direct rounding of the input.
    """
    a = np.asarray(a)
    if a.dtype == np.float64 and a.size:
        u = np.ascontiguousarray(a).view(np.uint64)
        mag = u & np.uint64(0x7FFFFFFFFFFFFFFF)
        # exponent field in [897, 1150]: 2^-126 <= |v| < 2^128 minus the top binade (kept clear of overflow)
        if mag.min() >= (np.uint64(897) << np.uint64(52)) and mag.max() < (np.uint64(1150) << np.uint64(52)):
            r = (mag >> np.uint64(45)) & np.uint64(1)
            r += mag
            r += np.uint64((1 << 44) - 1)
            r >>= np.uint64(45)
            r -= np.uint64(896 << 7)
            r |= (u >> np.uint64(48)) & np.uint64(0x8000)
            return r.astype(np.uint16)
    a64 = np.asarray(a, dtype=np.float64)
    f32 = a64.astype(np.float32)
    bits = f32.view(np.uint32).astype(np.uint64)
    low = bits & 0xFFFF
    trunc = bits >> 16
    up = low > 0x8000
    tie = low == 0x8000
    # on a tie after the first rounding: compare the original magnitude
    err = np.abs(a64) - np.abs(f32.astype(np.float64))
    tie_up = tie & ((err > 0) | ((err == 0) & ((trunc & 1) == 1)))
    out = trunc + (up | tie_up).astype(np.uint64)
    return out.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(bits).astype(np.float64)


# --------------------------------------------------------------------------- #
# workloads
# --------------------------------------------------------------------------- #
def n_logits(n: int, kind: str = "lite") -> int:
    """Number of projection columns: n! + 2n (mHC-lite) or n^2 + 2n (mHC / SK)."""
    if kind == "lite":
        return math.factorial(n) + 2 * n
    if kind == "sk":
        return n * n + 2 * n
    raise ValueError(kind)


@dataclass(frozen=True)
class Workload:
    name: str
    n: int
    C: int
    T: int
    seed: int
    bias_std: float = 0.0          # 0 -> zeros
    alpha: float = 0.01
    w_std: float = 0.02
    layers: int = 1
    backward: bool = True
    note: str = ""
    extra: dict = field(default_factory=dict)


WORKLOADS = {
    # small case the oracle finishes in seconds; forward only
    "cfg1": Workload("cfg1", n=4, C=256, T=4096, seed=0, backward=False,
                     note="n=4, C=256, T=4096, b=0, fwd only"),
    # the headline configuration: 8 sequences x 2048 tokens, hidden 1024
    "cfg2": Workload("cfg2", n=4, C=1024, T=16384, seed=1, bias_std=0.1,
                     note="n=4, C=1024, T=16384 (8x2048), b~N(0,0.1), fwd+bwd"),
    "cfg3": Workload("cfg3", n=4, C=2048, T=16384, seed=2, layers=24,
                     note="24-layer stack, stand-in sublayer y=RMSNorm(u)"),
    "cfg4a": Workload("cfg4a", n=3, C=1536, T=32768, seed=3, bias_std=0.1,
                      note="n=3 (6 permutations)"),
    "cfg4b": Workload("cfg4b", n=5, C=1536, T=32768, seed=4, bias_std=0.1,
                      note="n=5 (120 permutations)"),
    "cfg5": Workload("cfg5", n=4, C=4096, T=131072, seed=5, bias_std=0.1,
                     note="SK comparison / bandwidth sweep, T = 4096 ... 131072"),
}

# stream indices of the tensors of one layer (layer l uses offset 16*l)
_S_X, _S_Y, _S_G, _S_DU, _S_W, _S_B, _S_WSK, _S_BSK, _S_GAIN = range(9)


def paper_init_bias(n: int, kind: str = "lite") -> np.ndarray:
    """Bias pattern of the paper's initialisation (Section 4, "Initialization").

    b_res = -8 everywhere except 0 at the identity (permutation 0 for mHC-lite,
    the diagonal for mHC); b_pre and b_post = -1 except a single +1 (taken here
    at stream 0).
    """
    if kind == "lite":
        res = np.full(math.factorial(n), -8.0, dtype=np.float32)
        res[0] = 0.0
    else:
        res = np.full((n, n), -8.0, dtype=np.float32)
        res[np.arange(n), np.arange(n)] = 0.0
        res = res.reshape(-1)
    gate = np.full(n, -1.0, dtype=np.float32)
    gate[0] = 1.0
    return np.concatenate([res, gate, gate]).astype(np.float32)


def sample_perm_table(n: int, K: int, seed: int) -> np.ndarray:
    """A table of K distinct permutations of (0..n-1) for the subset variant of the paper's Section 5:
    row 0 is the identity (so that the paper's initialisation, which puts the weight on the identity,
    keeps its meaning), the other rows are drawn without repetition from stream (seed, 77).  uint8 [K, n]."""
    if not 1 <= K <= math.factorial(n):
        raise ValueError("K must be in [1, n!]")
    gen = np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), 77]))
    rows = [tuple(range(n))]
    seen = set(rows)
    while len(rows) < K:
        r = tuple(int(v) for v in gen.permutation(n))
        if r not in seen:
            seen.add(r)
            rows.append(r)
    return np.array(rows, dtype=np.uint8)


def make_layer_inputs(n: int, C: int, T: int, seed: int, *, layer: int = 0,
                      bias_std: float = 0.0, alpha=0.01, w_std: float = 0.02,
                      kind: str = "lite", gain_std: float = 0.0,
                      shard: int = 0, n_res: int | None = None) -> dict:
    """All inputs of one layer, fwd and bwd, as host arrays.

    Returns a dict with
      x  [T,n,C] uint16 (bf16 bits)    residual streams x_l
      y  [T,C]   uint16                sublayer output  f(H_pre x_l)
      g  [T,n,C] uint16                upstream gradient dL/dx_{l+1}
      du [T,C]   uint16                gradient the sublayer's backward returns, dL/du
      W  [nC,N]  float32, b [N] float32, alpha [3] float32 (res, pre, post),
      gain [nC]  float32 (ones, or 1 + N(0, gain_std^2))
    ``shard`` selects the token streams, so that the ranks of a sharded run draw
    different tokens (rank r passes shard=r) while sharing the parameters.  ``n_res`` overrides
    the number of residual columns (K for a table of K sampled permutations).
    """
    N = n_logits(n, kind) if n_res is None else n_res + 2 * n
    base = 16 * layer
    tok = 4096 * int(shard)                    # token tensors: one stream per shard
    x = normal_bf16(seed, base + _S_X + tok, (T, n, C))
    y = normal_bf16(seed, base + _S_Y + tok, (T, C))
    g = normal_bf16(seed, base + _S_G + tok, (T, n, C))
    du = normal_bf16(seed, base + _S_DU + tok, (T, C))
    p = make_layer_params(n, C, seed, layer=layer, bias_std=bias_std, alpha=alpha, w_std=w_std, kind=kind,
                          gain_std=gain_std, n_res=n_res)
    return dict(x=x, y=y, g=g, du=du, W=p["W"], b=p["b"], alpha=p["alpha"], gain=p["gain"],
                n=n, C=C, T=T, N=N, kind=kind)


def make_layer_params(n: int, C: int, seed: int, *, layer: int = 0, bias_std: float = 0.0, alpha=0.01,
                      w_std: float = 0.02, kind: str = "lite", gain_std: float = 0.0, n_res: int | None = None) -> dict:
    """The parameters of layer `layer` alone (W, b, alpha, gain), as make_layer_inputs draws them."""
    N = n_logits(n, kind) if n_res is None else n_res + 2 * n
    base = 16 * layer
    sw, sb = (_S_W, _S_B) if kind == "lite" else (_S_WSK, _S_BSK)
    W = normal(seed, base + sw, (n * C, N), w_std).astype(np.float32)
    if bias_std > 0:
        b = normal(seed, base + sb, (N,), bias_std).astype(np.float32)
    else:
        b = np.zeros(N, dtype=np.float32)
    a = np.asarray(alpha, dtype=np.float32)
    alpha3 = np.full(3, a, dtype=np.float32) if a.ndim == 0 else a.astype(np.float32).reshape(3)
    if gain_std > 0:
        gain = (1.0 + normal(seed, base + _S_GAIN, (n * C,), gain_std)).astype(np.float32)
    else:
        gain = np.ones(n * C, dtype=np.float32)
    return dict(W=W, b=b, alpha=alpha3, gain=gain, n=n, C=C, N=N, kind=kind)
