"""ctypes binding of the CPU oracle (test infrastructure, not the product path).

Only tests, the smoke check and the benchmark's CPU-baseline leg import this.
It never touches the CUDA library. `build()` compiles the C file with gcc;
the binding builds it on first use when the shared object is missing or older
than the source.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mpgemmfi_oracle.c")
_LIB = os.path.join(_HERE, "libmpgemmfi_oracle.so")

FP16, BF16, TF32 = 0, 1, 2
KIND_A, KIND_B, KIND_ACC, KIND_OUT, KIND_TERM = 0, 1, 2, 3, 4
T_NONE, T_BOUND, T_RMAX, T_RFLIP = 0, 1, 2, 3
CORRECT = 16
OUTPUT_RANGE = 64
TERM_IN_FORMAT = 128

SITE = np.dtype([("kind", "<u4"), ("row", "<u4"), ("col", "<u4"), ("k", "<u4"),
                 ("xor_mask", "<u4"), ("trial", "<u4"), ("pad0", "<u4"), ("pad1", "<u4")])
SITE_LOG = np.dtype([("before_bits", "<u4"), ("after_bits", "<u4"), ("final_bits", "<u4"), ("status", "<u4")])
RECORD = np.dtype([("status", "<u4"), ("kind", "<u4"), ("primary_index", "<u4"), ("before_bits", "<u4"),
                   ("after_bits", "<u4"), ("final_bits", "<u4"), ("n_affected", "<u4"), ("n_detected", "<u4"),
                   ("idx_hash", "<u8"), ("first_detected", "<u4"), ("max_abs_dev", "<f4")])
assert SITE.itemsize == 32 and SITE_LOG.itemsize == 16 and RECORD.itemsize == 48


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no FMA contraction, OpenMP across independent elements)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-mavx2", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        L = _lib
        L.orc_widen_bits.restype = C.c_uint32
        L.orc_widen_bits.argtypes = [C.c_int, C.c_uint32]
        L.orc_widen.restype = C.c_float
        L.orc_widen.argtypes = [C.c_int, C.c_uint32]
        L.orc_flip_operand.restype = C.c_uint32
        L.orc_flip_operand.argtypes = [C.c_int, C.c_uint32, C.c_uint32]
        L.orc_boundcheck_detect.restype = C.c_int
        L.orc_boundcheck_detect.argtypes = [C.c_uint32]
        L.orc_boundcheck_correct.restype = C.c_uint32
        L.orc_boundcheck_correct.argtypes = [C.c_uint32]
        L.orc_rangecheck_bound.restype = C.c_int
        L.orc_rangecheck_bound.argtypes = [C.c_uint32, C.c_uint32]
        L.orc_rangecheck_detect.restype = C.c_int
        L.orc_rangecheck_detect.argtypes = [C.c_uint32, C.c_int]
        L.orc_rangecheck_max.restype = C.c_uint32
        L.orc_rangecheck_max.argtypes = [C.c_uint32, C.c_int]
        L.orc_rangecheck_flip.restype = C.c_uint32
        L.orc_rangecheck_flip.argtypes = [C.c_uint32, C.c_int]
        L.orc_num_threads.restype = C.c_int
        vp = C.c_void_p
        L.orc_gemm.restype = C.c_int
        L.orc_gemm.argtypes = [C.c_int] * 4 + [vp, vp, vp, vp, C.c_int, C.c_int, C.c_int, vp, vp, vp]
        L.orc_gemm_addend.restype = C.c_int
        L.orc_gemm_addend.argtypes = [C.c_int] * 4 + [vp, vp, vp, vp, vp, C.c_int, C.c_int, C.c_int, vp, vp, vp]
        L.orc_campaign.restype = C.c_int
        L.orc_campaign.argtypes = [C.c_int] * 4 + [vp, vp, vp, vp, C.c_int, C.c_int, C.c_int, vp]
        L.orc_campaign_form.restype = C.c_int
        L.orc_campaign_form.argtypes = [C.c_int] * 4 + [vp, vp, vp, vp, C.c_int, C.c_int, C.c_int, C.c_int, vp]
        L.orc_operand_trial_values.restype = C.c_int
        L.orc_operand_trial_values.argtypes = [C.c_int] * 4 + [vp, vp, vp, vp, C.c_int, vp]
        L.orc_round_to_operand.restype = C.c_uint32
        L.orc_round_to_operand.argtypes = [C.c_int, C.c_uint32]
        L.orc_round_output.restype = C.c_uint32
        L.orc_round_output.argtypes = [C.c_int, C.c_uint32]
        L.orc_gemm_out16.restype = C.c_int
        L.orc_gemm_out16.argtypes = [C.c_int] * 4 + [vp, vp, vp, C.c_int, vp, vp, C.c_int, C.c_int, C.c_int, vp, vp, vp]
        L.orc_sample.restype = C.c_int
        L.orc_sample.argtypes = [C.c_int] * 4 + [vp, vp, vp, C.c_int, vp, vp, C.c_int, vp, vp]
        L.orc_sample_addend.restype = C.c_int
        L.orc_sample_addend.argtypes = [C.c_int] * 4 + [vp, vp, vp, C.c_int, vp, vp, vp, C.c_int, vp, vp]
        L.orc_operand_exponents.restype = None
        L.orc_operand_exponents.argtypes = [C.c_int, C.c_int, C.c_int, vp, vp]
        L.orc_output_range_bound.restype = C.c_int
        L.orc_output_range_bound.argtypes = [C.c_uint32, C.c_uint32, C.c_int]
        L.orc_summary.restype = None
        L.orc_summary.argtypes = [vp, C.c_int, vp]
        L.orc_absprod.restype = C.c_int
        L.orc_absprod.argtypes = [C.c_int] * 4 + [vp, vp, vp]
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _storage(a, dtype):
    want = np.uint32 if dtype == TF32 else np.uint16
    a = np.ascontiguousarray(a)
    assert a.dtype == want, (a.dtype, want)
    return a


def _sites(sites):
    if sites is None:
        return np.zeros(0, dtype=SITE)
    s = np.ascontiguousarray(sites)
    assert s.dtype.itemsize == 32
    return s.view(SITE) if s.dtype != SITE else s


# ---------------------------------------------------------------- scalar entry points

def widen_bits(dtype, s):
    return int(lib().orc_widen_bits(dtype, int(s)))


def widen(dtype, s):
    return float(lib().orc_widen(dtype, int(s)))


def flip_operand(dtype, s, mask):
    return int(lib().orc_flip_operand(dtype, int(s), int(mask)))


def boundcheck_detect(bits):
    return int(lib().orc_boundcheck_detect(int(bits)))


def boundcheck_correct(bits):
    return int(lib().orc_boundcheck_correct(int(bits)))


def rangecheck_bound(a_bits, b_bits):
    return int(lib().orc_rangecheck_bound(int(a_bits), int(b_bits)))


def rangecheck_detect(p_bits, bound):
    return int(lib().orc_rangecheck_detect(int(p_bits), int(bound)))


def rangecheck_max(p_bits, bound):
    return int(lib().orc_rangecheck_max(int(p_bits), int(bound)))


def rangecheck_flip(p_bits, bound):
    return int(lib().orc_rangecheck_flip(int(p_bits), int(bound)))


def num_threads():
    return int(lib().orc_num_threads())


# ---------------------------------------------------------------- matrix entry points

def gemm(dtype, A, Bt, sites=None, detect_mode=0, kstep=None, addend=None):
    """Full-recompute fault-injected GEMM. Returns (C, header[16], site_log, bitmap[M, ceil(N/32)]).

    addend: optional M x N FP32 matrix, the C of D = A x B + C (Section II-B): every running sum starts from it."""
    A = _storage(A, dtype)
    Bt = _storage(Bt, dtype)
    M, K = A.shape
    N, K2 = Bt.shape
    assert K == K2
    kstep = (32 if dtype == TF32 else 64) if kstep is None else kstep
    s = _sites(sites)
    Cm = np.empty((M, N), dtype=np.float32)
    hdr = np.zeros(16, dtype=np.uint32)
    log = np.zeros(len(s), dtype=SITE_LOG)
    bitmap = np.zeros((M, (N + 31) // 32), dtype=np.uint32)
    if addend is None:
        rc = lib().orc_gemm(dtype, M, N, K, _ptr(A), _ptr(Bt), _ptr(Cm), _ptr(s), len(s), detect_mode, kstep,
                            _ptr(hdr), _ptr(log), _ptr(bitmap))
    else:
        Cin = np.ascontiguousarray(addend, dtype=np.float32)
        assert Cin.shape == (M, N)
        rc = lib().orc_gemm_addend(dtype, M, N, K, _ptr(A), _ptr(Bt), _ptr(Cin), _ptr(Cm), _ptr(s), len(s),
                                   detect_mode, kstep, _ptr(hdr), _ptr(log), _ptr(bitmap))
    assert rc == 0
    return Cm, hdr, log, bitmap


def campaign(dtype, A, Bt, C_clean, sites, detect_mode=0, kstep=None, operand_form=0):
    """One record per single-site trial (incremental evaluation of the affected elements).
    operand_form: 0 = an operand trial's row / column is accumulated again with the faulty operand (the definition);
    1 = Eq. 1-2 applied to the finished sums of C_clean."""
    A = _storage(A, dtype)
    Bt = _storage(Bt, dtype)
    M, K = A.shape
    N, _ = Bt.shape
    kstep = (32 if dtype == TF32 else 64) if kstep is None else kstep
    s = _sites(sites)
    Cc = np.ascontiguousarray(C_clean, dtype=np.float32)
    assert Cc.shape == (M, N)
    rec = np.zeros(len(s), dtype=RECORD)
    rc = lib().orc_campaign_form(dtype, M, N, K, _ptr(A), _ptr(Bt), _ptr(Cc), _ptr(s), len(s), detect_mode, kstep,
                                 operand_form, _ptr(rec))
    assert rc == 0
    return rec


def operand_trial_values(dtype, A, Bt, C_clean, site, form=0):
    """Unchecked values of the row (A site) or column (B site) of C that one operand site reaches; form as in campaign()."""
    A = _storage(A, dtype)
    Bt = _storage(Bt, dtype)
    M, K = A.shape
    N, _ = Bt.shape
    s = _sites(np.asarray(site).reshape(1))
    Cc = np.ascontiguousarray(C_clean, dtype=np.float32)
    assert Cc.shape == (M, N)
    out = np.empty(N if int(s["kind"][0]) == KIND_A else M, dtype=np.float32)
    n = lib().orc_operand_trial_values(dtype, M, N, K, _ptr(A), _ptr(Bt), _ptr(Cc), _ptr(s), form, _ptr(out))
    assert n == len(out), n
    return out


OUT_FP16, OUT_BF16 = 0, 1


def round_to_operand(dtype, bits):
    """FP32 word -> storage word of the operand format (round to nearest even)."""
    return int(lib().orc_round_to_operand(dtype, int(bits) & 0xFFFFFFFF))


def round_output(out_fmt, bits):
    """FP32 word -> 16-bit word of the output format, round to nearest even."""
    return int(lib().orc_round_output(out_fmt, int(bits) & 0xFFFFFFFF))


def gemm_out16(dtype, A, Bt, out_fmt, sites=None, detect_mode=0, kstep=None, addend=None):
    """orc.gemm with the checked FP32 result rounded to a 16-bit format. Returns (D16 uint16[M,N], header, log, bitmap)."""
    A = _storage(A, dtype)
    Bt = _storage(Bt, dtype)
    M, K = A.shape
    N, _ = Bt.shape
    kstep = (32 if dtype == TF32 else 64) if kstep is None else kstep
    s = _sites(sites)
    D = np.empty((M, N), dtype=np.uint16)
    hdr = np.zeros(16, dtype=np.uint32)
    log = np.zeros(len(s), dtype=SITE_LOG)
    bitmap = np.zeros((M, (N + 31) // 32), dtype=np.uint32)
    Cin = None if addend is None else np.ascontiguousarray(addend, dtype=np.float32)
    rc = lib().orc_gemm_out16(dtype, M, N, K, _ptr(A), _ptr(Bt), _ptr(Cin), out_fmt, _ptr(D), _ptr(s), len(s),
                              detect_mode, kstep, _ptr(hdr), _ptr(log), _ptr(bitmap))
    assert rc == 0
    return D, hdr, log, bitmap


def sample(dtype, A, Bt, si, sj, sites=None, start=None):
    """Clean (operand-faulted) C[i,j] and (|A||B|)_ij at sampled positions, any matrix size.
    start: optional float32 value per sample that its running sum begins with (the addend c_ij of D = A x B + C);
    its magnitude is added to the second result."""
    A = _storage(A, dtype)
    Bt = _storage(Bt, dtype)
    M, K = A.shape
    N, _ = Bt.shape
    si = np.ascontiguousarray(si, dtype=np.uint32)
    sj = np.ascontiguousarray(sj, dtype=np.uint32)
    s = _sites(sites)
    out = np.empty(len(si), dtype=np.float32)
    ap = np.empty(len(si), dtype=np.float64)
    if start is None:
        rc = lib().orc_sample(dtype, M, N, K, _ptr(A), _ptr(Bt), _ptr(s), len(s), _ptr(si), _ptr(sj), len(si), _ptr(out), _ptr(ap))
    else:
        st = np.ascontiguousarray(start, dtype=np.float32)
        assert st.shape == (len(si),)
        rc = lib().orc_sample_addend(dtype, M, N, K, _ptr(A), _ptr(Bt), _ptr(s), len(s), _ptr(st), _ptr(si), _ptr(sj), len(si),
                                     _ptr(out), _ptr(ap))
    assert rc == 0
    return out, ap


def operand_exponents(dtype, X):
    """Largest FP32 exponent field per row of an operand matrix (uint32[rows])."""
    X = _storage(X, dtype)
    out = np.zeros(X.shape[0], dtype=np.uint32)
    lib().orc_operand_exponents(dtype, X.shape[0], X.shape[1], _ptr(X), _ptr(out))
    return out


def output_range_bound(EA, EB, K):
    return int(lib().orc_output_range_bound(int(EA), int(EB), int(K)))


def summary(records):
    """Deviation summary of trial records: 272 uint32 words (6 counts, 5 + 5 per-kind counts, 256 histogram bins)."""
    rec = np.ascontiguousarray(records)
    assert rec.dtype.itemsize == 48
    out = np.zeros(272, dtype=np.uint32)
    lib().orc_summary(_ptr(rec), len(rec), _ptr(out))
    return out


def absprod(dtype, A, Bt):
    A = _storage(A, dtype)
    Bt = _storage(Bt, dtype)
    M, K = A.shape
    N, _ = Bt.shape
    out = np.empty((M, N), dtype=np.float64)
    rc = lib().orc_absprod(dtype, M, N, K, _ptr(A), _ptr(Bt), _ptr(out))
    assert rc == 0
    return out
