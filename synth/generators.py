"""Seeded operand matrices and fault-site tables for the five benchmark workloads.

Everything here is input preparation: draw numbers from a counter-based
generator (Philox), shape them like the workloads (LayerNorm-like, GELU, ReLU
activations; small-variance weights), round them to the storage format with
round-to-nearest-even and draw uniformly distributed fault sites. The operand
bits produced here are handed unchanged to whichever implementation consumes
them, so every implementation sees identical inputs.

Layouts
-------
A  : M x K row-major (K contiguous).
Bt : N x K row-major, i.e. B stored K-major (the layout of a Linear weight).
FP16/BF16 are returned as uint16 bit patterns, TF32 as uint32 FP32 words whose
low 13 bits are zero.

Fault-site table: numpy structured array, 32 bytes per entry,
(kind, row, col, k, xor_mask, trial, pad0, pad1), all uint32.
"""
from __future__ import annotations

import dataclasses

import numpy as np

DTYPE_FP16, DTYPE_BF16, DTYPE_TF32 = 0, 1, 2
KIND_A, KIND_B, KIND_ACC, KIND_OUT, KIND_TERM = 0, 1, 2, 3, 4

SITE_DTYPE = np.dtype([
    ("kind", "<u4"), ("row", "<u4"), ("col", "<u4"), ("k", "<u4"),
    ("xor_mask", "<u4"), ("trial", "<u4"), ("pad0", "<u4"), ("pad1", "<u4"),
])
assert SITE_DTYPE.itemsize == 32

BASE_SEED = 231105782

# detect_mode values carried by the configs: technique in bits 1:0
# (1 = BoundCheck), bit 4 = correction enabled.
_DET_BOUND = 1
_DET_BOUND_CORRECT = 1 | 16

CONFIGS = {
    # FP16 256^3, 64 output-element single-bit trials, detection only
    "c1": dict(index=1, dtype=DTYPE_FP16, M=256, N=256, K=256,
               a=("normal", 1.0 / 16.0), b=("normal", 1.0 / 16.0),
               trials=64, mix="out", detect_mode=_DET_BOUND),
    # BF16 4096^3, 1024 operand single-bit trials, detection + correction
    "c2": dict(index=2, dtype=DTYPE_BF16, M=4096, N=4096, K=4096,
               a=("normal", 1.0 / 64.0), b=("normal", 1.0 / 64.0),
               trials=1024, mix="operand", detect_mode=_DET_BOUND_CORRECT),
    # transformer-layer FP16 GEMMs, batch 32 x seq 512
    "c3a": dict(index=3, dtype=DTYPE_FP16, M=16384, N=4096, K=1024,
                a=("normal", 1.0), b=("normal", 0.02),
                trials=4096, mix="out", detect_mode=_DET_BOUND),
    "c3b": dict(index=3, dtype=DTYPE_FP16, M=16384, N=1024, K=4096,
                a=("gelu", 1.0), b=("normal", 0.02), seed_shift=10,
                trials=4096, mix="out", detect_mode=_DET_BOUND),
    # TF32 8192^3, 2048 accumulator trials with two adjacent bits
    "c4": dict(index=4, dtype=DTYPE_TF32, M=8192, N=8192, K=8192,
               a=("uniform", 1.0), b=("uniform", 1.0),
               trials=2048, mix="acc2", detect_mode=_DET_BOUND),
    # conv-as-GEMM (im2col of a 3x3, 64->64 conv, 56x56, batch 256), FP16
    "c5": dict(index=5, dtype=DTYPE_FP16, M=802816, N=64, K=576,
               a=("relu", 1.0), b=("normal", float(np.sqrt(2.0 / 576.0))),
               trials=100000, mix="mixed", detect_mode=_DET_BOUND_CORRECT),
}


def kstep(dtype: int) -> int:
    """Number of k elements between two accumulator boundaries (one 128-byte row)."""
    return 32 if dtype == DTYPE_TF32 else 64


def storage_dtype(dtype: int):
    return np.uint32 if dtype == DTYPE_TF32 else np.uint16


def operand_bits(dtype: int) -> int:
    """Width of an operand's storage format in bits (TF32 uses 19)."""
    return 19 if dtype == DTYPE_TF32 else 16


def round_to_storage(x: np.ndarray, dtype: int) -> np.ndarray:
    """Round FP32 values to the storage format, ties to even; return the bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if dtype == DTYPE_FP16:
        return x.astype(np.float16).view(np.uint16)
    u = x.view(np.uint32)
    if dtype == DTYPE_BF16:
        r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
        return r.astype(np.uint16)
    if dtype == DTYPE_TF32:
        r = u + np.uint32(0xFFF) + ((u >> np.uint32(13)) & np.uint32(1))
        return r & np.uint32(0xFFFFE000)
    raise ValueError(f"unknown dtype {dtype}")


def _draw(rng: np.random.Generator, shape, spec) -> np.ndarray:
    law, scale = spec
    if law == "uniform":
        x = rng.random(shape, dtype=np.float32) * np.float32(2.0) - np.float32(1.0)
        return x * np.float32(scale)
    x = rng.standard_normal(shape, dtype=np.float32)
    if law == "normal":
        pass
    elif law == "relu":
        np.maximum(x, np.float32(0.0), out=x)
    elif law == "gelu":
        from scipy.special import erf  # exact erf form of GELU
        x = (x * np.float32(0.5) * (np.float32(1.0) + erf(x / np.float32(np.sqrt(2.0))))).astype(np.float32)
    else:
        raise ValueError(law)
    return x * np.float32(scale)


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=int(seed)))


def config_seed(name: str) -> int:
    cfg = CONFIGS[name]
    return BASE_SEED + 1000 * cfg["index"] + cfg.get("seed_shift", 0)


def make_operands(name: str, M=None, N=None, K=None, seed=None, dtype=None):
    """Return (A_bits[M,K], Bt_bits[N,K]) for a config, optionally at reduced sizes and, with `dtype`, with the same
    draws rounded to another storage format."""
    cfg = CONFIGS[name]
    if dtype is not None:
        cfg = dict(cfg, dtype=dtype)
    M = cfg["M"] if M is None else M
    N = cfg["N"] if N is None else N
    K = cfg["K"] if K is None else K
    seed = config_seed(name) if seed is None else seed
    a = round_to_storage(_draw(_rng(seed), (M, K), cfg["a"]), cfg["dtype"])
    bt = round_to_storage(_draw(_rng(seed + 1), (N, K), cfg["b"]), cfg["dtype"])
    return a, bt


def adjacent_mask(start: np.ndarray, nbits: int) -> np.ndarray:
    """Mask of `nbits` adjacent bits whose lowest bit is `start`."""
    return (np.uint32((1 << nbits) - 1) << start.astype(np.uint32)).astype(np.uint32)


def make_sites(mix: str, dtype: int, M: int, N: int, K: int, n: int, seed: int,
               nbits: int = 1) -> np.ndarray:
    """Draw `n` independent single-fault trials.

    mix: "out"     one output element, bit(s) uniform in the 32-bit word
         "operand" A or B with probability 1/2, element uniform, bit(s) uniform in the storage word
         "acc"     one accumulator element after a uniformly chosen k boundary
         "acc2"    as "acc" with two adjacent bits
         "term"    one product term (i, j, k), bit(s) uniform in the 32-bit product
         "term_op" the same with the bit(s) uniform in a word of the operand format (16 bits; 19 for TF32), for the
                   reading in which the product is held in that format
         "mixed"   kind uniform over {operand, acc, out}
    """
    rng = _rng(seed)
    s = np.zeros(n, dtype=SITE_DTYPE)
    s["trial"] = np.arange(n, dtype=np.uint32)
    if mix == "acc2":
        mix, nbits = "acc", 2
    kt = kstep(dtype)
    nb = (K + kt - 1) // kt
    obits = operand_bits(dtype)

    u_kind = rng.integers(0, 3, size=n)
    u_ab = rng.integers(0, 2, size=n)
    row = rng.integers(0, M, size=n, dtype=np.int64)
    col = rng.integers(0, N, size=n, dtype=np.int64)
    kk = rng.integers(0, K, size=n, dtype=np.int64)
    bnd = rng.integers(1, nb + 1, size=n, dtype=np.int64)
    u_bit = rng.random(size=n)

    if mix == "out":
        kind = np.full(n, KIND_OUT)
    elif mix == "operand":
        kind = np.where(u_ab == 0, KIND_A, KIND_B)
    elif mix == "acc":
        kind = np.full(n, KIND_ACC)
    elif mix in ("term", "term_op"):
        kind = np.full(n, KIND_TERM)
    elif mix == "mixed":
        kind = np.where(u_kind == 0, np.where(u_ab == 0, KIND_A, KIND_B),
                        np.where(u_kind == 1, KIND_ACC, KIND_OUT))
    else:
        raise ValueError(mix)

    is_op = (kind == KIND_A) | (kind == KIND_B)
    width = np.where(is_op | (mix == "term_op"), obits, 32)
    start = np.floor(u_bit * (width - nbits + 1)).astype(np.uint32)
    s["kind"] = kind
    s["row"] = np.where(kind == KIND_B, 0, row)
    s["col"] = np.where(kind == KIND_A, 0, col)
    s["k"] = np.where(kind == KIND_ACC, np.minimum(bnd * kt, K),
                      np.where(kind == KIND_OUT, 0, kk))
    s["xor_mask"] = adjacent_mask(start, nbits)
    return s


@dataclasses.dataclass
class Workload:
    name: str
    dtype: int
    M: int
    N: int
    K: int
    A: np.ndarray
    Bt: np.ndarray
    sites: np.ndarray
    detect_mode: int


def make_workload(name: str, M=None, N=None, K=None, trials=None, mix=None) -> Workload:
    """Operands plus the trial table of a config (optionally at reduced sizes)."""
    cfg = CONFIGS[name]
    M = cfg["M"] if M is None else M
    N = cfg["N"] if N is None else N
    K = cfg["K"] if K is None else K
    trials = cfg["trials"] if trials is None else trials
    mix = cfg["mix"] if mix is None else mix
    a, bt = make_operands(name, M, N, K)
    sites = make_sites(mix, cfg["dtype"], M, N, K, trials, config_seed(name) + 2)
    return Workload(name, cfg["dtype"], M, N, K, a, bt, sites, cfg["detect_mode"])
