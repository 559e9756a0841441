"""Seeded synthetic inputs for the MUXQ linear layer (shared by the oracle tests, the GPU parity
tests and the benchmark).  This module holds NONE of the method's arithmetic: it only draws
activations and weights with the structure the paper describes (a handful of channels of the
activation matrix carry the outliers, Fig. 1) at GPT-2 layer shapes (Section IV-B).

Generator: counter based and independent of any library RNG state.  Element i of tensor t under
seed s hashes the counter (s, t, i) with splitmix64 to two uniforms and applies Box-Muller, so
any slice can be regenerated on its own.  Values are rounded to fp16 (round to nearest even).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Tuple

import numpy as np

_MASK = np.uint64(0xFFFFFFFFFFFFFFFF)


def _splitmix64(z: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = (z + np.uint64(0x9E3779B97F4A7C15)) & _MASK
        z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _MASK
        z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _MASK
        return z ^ (z >> np.uint64(31))


def _key(seed: int, tensor_id: int, stream: int) -> np.uint64:
    k = np.array([(seed * 0x1000003 + tensor_id) & 0xFFFFFFFFFFFFFFFF], np.uint64)
    k = _splitmix64(k)
    k = _splitmix64(k ^ np.uint64(stream * 0x632BE59BD9B4E019 & 0xFFFFFFFFFFFFFFFF))
    return k[0]


def _uniform(seed: int, tensor_id: int, stream: int, start: int, n: int) -> np.ndarray:
    """n uniforms in (0,1), element counters start..start+n-1."""
    ctr = np.arange(start, start + n, dtype=np.uint64)
    with np.errstate(over="ignore"):
        h = _splitmix64(ctr * np.uint64(0xD1342543DE82EF95) ^ _key(seed, tensor_id, stream))
    return ((h >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(seed: int, tensor_id: int, n: int, start: int = 0, stream: int = 0) -> np.ndarray:
    u1 = _uniform(seed, tensor_id, 2 * stream, start, n)
    u2 = _uniform(seed, tensor_id, 2 * stream + 1, start, n)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def student_t4(seed: int, tensor_id: int, n: int, start: int = 0) -> np.ndarray:
    """Student-t with 4 degrees of freedom: z / sqrt(chi2_4 / 4), chi2_4 = -2 ln(u1 u2)."""
    z = normal(seed, tensor_id, n, start, stream=0)
    ua = _uniform(seed, tensor_id, 10, start, n)
    ub = _uniform(seed, tensor_id, 11, start, n)
    chi2 = -2.0 * (np.log(ua) + np.log(ub))
    return z / np.sqrt(chi2 / 4.0)


def outlier_channels(seed: int, tensor_id: int, K: int, r: int) -> np.ndarray:
    """First r entries of a seeded Fisher-Yates shuffle of 0..K-1."""
    perm = np.arange(K, dtype=np.int64)
    u = _uniform(seed, tensor_id, 20, 0, max(r, 1))
    for i in range(min(r, K - 1)):
        j = i + int(u[i] * (K - i))
        perm[i], perm[j] = perm[j], perm[i]
    return perm[:r].copy()


def make_x(seed: int, tensor_id: int, M: int, K: int, n_outliers: int, mult_lo: float,
           mult_hi: float, bulk: str = "normal", bulk_scale: float = 1.0,
           chunk_rows: int = 2048) -> Tuple[np.ndarray, np.ndarray]:
    """X [M,K] fp16: bulk draw times a per-channel multiplier (constant down the column).

    Returns (X, injected channel indices sorted ascending)."""
    ch = outlier_channels(seed, tensor_id, K, n_outliers)
    mult = np.full(K, bulk_scale, np.float64)
    if n_outliers:
        um = _uniform(seed, tensor_id, 21, 0, n_outliers)
        mult[ch] = bulk_scale * (mult_lo + (mult_hi - mult_lo) * um)
    x = np.empty((M, K), np.float16)
    for r0 in range(0, M, chunk_rows):
        r1 = min(M, r0 + chunk_rows)
        n = (r1 - r0) * K
        if bulk == "normal":
            v = normal(seed, tensor_id, n, start=r0 * K)
        elif bulk == "t4":
            v = student_t4(seed, tensor_id, n, start=r0 * K)
        else:
            raise ValueError(bulk)
        x[r0:r1] = (v.reshape(r1 - r0, K) * mult[None, :]).astype(np.float16)
    return x, np.sort(ch)


def make_w(seed: int, tensor_id: int, K: int, N: int, sigma: float = 0.02) -> np.ndarray:
    """W [K,N] fp16 with N(0, sigma) entries (GPT-2's initialisation width)."""
    v = normal(seed, tensor_id + 1_000_000, K * N)
    return (v.reshape(K, N) * sigma).astype(np.float16)


@dataclass(frozen=True)
class LayerSpec:
    name: str
    M: int
    K: int
    N: int
    n_outliers: int
    mult_lo: float
    mult_hi: float
    bulk: str
    bulk_scale: float
    seed: int
    tensor_id: int

    def x(self):
        return make_x(self.seed, self.tensor_id, self.M, self.K, self.n_outliers, self.mult_lo,
                      self.mult_hi, self.bulk, self.bulk_scale)

    def w(self):
        return make_w(self.seed, self.tensor_id, self.K, self.N)


def _gpt2_linears(d: int) -> List[Tuple[str, int, int]]:
    return [("c_attn", d, 3 * d), ("attn_c_proj", d, d), ("c_fc", d, 4 * d),
            ("mlp_c_proj", 4 * d, d)]


def config_layers(cfg: int, M: int | None = None, n_outliers: int | None = None,
                  layers: int = 1) -> List[LayerSpec]:
    """The five benchmark workloads, as LayerSpecs.

    0: one 128x768x768 layer, 4 outlier channels x50, seed 0.
    1: GPT-2-small linears at M=8192, 6 outlier channels x U(40,80), seed 1.
    2: GPT-2-medium linears at M=8192, bulk 0.05*t4, 8 outlier channels x60, seed 2.
    3: GPT-2-large linears at M=16384 (or decode M), 8 outlier channels x60, seed 3.
    4: `layers` x GPT-2-large linears at M=8192, fresh X per layer, n_outliers x60, seed 4.
    """
    if cfg == 0:
        return [LayerSpec("cfg0", M or 128, 768, 768, 4, 50.0, 50.0, "normal", 1.0, 0, 0)]
    if cfg == 1:
        return [LayerSpec(n, M or 8192, k, nn, 6, 40.0, 80.0, "normal", 1.0, 1, i)
                for i, (n, k, nn) in enumerate(_gpt2_linears(768))]
    if cfg == 2:
        return [LayerSpec(n, M or 8192, k, nn, 8, 60.0, 60.0, "t4", 0.05, 2, i)
                for i, (n, k, nn) in enumerate(_gpt2_linears(1024))]
    if cfg == 3:
        return [LayerSpec(n, M or 16384, k, nn, 8, 60.0, 60.0, "normal", 1.0, 3, i)
                for i, (n, k, nn) in enumerate(_gpt2_linears(1280))]
    if cfg == 4:
        r = 8 if n_outliers is None else n_outliers
        out = []
        for layer in range(layers):
            for i, (n, k, nn) in enumerate(_gpt2_linears(1280)):
                out.append(LayerSpec(f"L{layer}.{n}", M or 8192, k, nn, r, 60.0, 60.0, "normal",
                                     1.0, 4, layer * 4 + i))
        return out
    raise ValueError(cfg)


def buffer_hash64(a: np.ndarray) -> str:
    """64-bit hash of a buffer, for reports."""
    b = np.ascontiguousarray(a).view(np.uint8).reshape(-1)
    # fold 8 bytes at a time with a multiplicative mix (fast, order-sensitive)
    pad = (-b.size) % 8
    if pad:
        b = np.concatenate([b, np.zeros(pad, np.uint8)])
    w = b.view(np.uint64)
    idx = np.arange(1, w.size + 1, dtype=np.uint64)
    with np.errstate(over="ignore"):
        h = np.bitwise_xor.reduce(_splitmix64(w ^ (idx * np.uint64(0x100000001B3))))
    return f"{int(h):016x}"
