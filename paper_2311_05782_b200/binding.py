"""ctypes binding of libmpgemmfi.so.

`mpgemmfi_*` functions mirror the C ABI one to one (raw pointers and sizes).
`gemm` and `campaign` are convenience wrappers that take torch CUDA tensors,
allocate the output buffers with torch and pass `data_ptr()`s and the current
stream; they do no arithmetic.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

FP16, BF16, TF32 = 0, 1, 2
SITE_A, SITE_B, SITE_ACC, SITE_OUT, SITE_TERM = 0, 1, 2, 3, 4
DETECT_NONE, DETECT_BOUNDCHECK, DETECT_RANGE_MAX, DETECT_RANGE_FLIP = 0, 1, 2, 3
CORRECT = 16
TERM_HMMA_STEP = 32
OUT_FP32, OUT_FP16, OUT_BF16 = 0, 1, 2
OUTPUT_RANGE = 64
TERM_IN_FORMAT = 128
STATUS_SITE_SKIPPED, STATUS_WAIT_LIMIT = 1, 2
MAX_FAULTS = 4096
INLINE_FAULTS = 8
STATIC_MAX_TRIALS = 65536
TILES_AUTO, TILES_SINGLE, TILES_PAIR = 0, 1, 2
SPLIT_AUTO, SPLIT_OFF, SPLIT_ON = 0, 1, 2
HEADER_WORDS = 16

SITE_DTYPE = np.dtype([("kind", "<u4"), ("row", "<u4"), ("col", "<u4"), ("k", "<u4"),
                       ("xor_mask", "<u4"), ("trial", "<u4"), ("pad0", "<u4"), ("pad1", "<u4")])
SITE_LOG_DTYPE = np.dtype([("before_bits", "<u4"), ("after_bits", "<u4"), ("final_bits", "<u4"), ("status", "<u4")])
RECORD_DTYPE = np.dtype([("status", "<u4"), ("kind", "<u4"), ("primary_index", "<u4"), ("before_bits", "<u4"),
                         ("after_bits", "<u4"), ("final_bits", "<u4"), ("n_affected", "<u4"), ("n_detected", "<u4"),
                         ("idx_hash", "<u8"), ("first_detected", "<u4"), ("max_abs_dev", "<f4")])

SUMMARY_DTYPE = np.dtype([("n_trials", "<u4"), ("n_invalid", "<u4"), ("n_zero_diff", "<u4"), ("n_detected", "<u4"),
                          ("n_corrected", "<u4"), ("n_nonfinite", "<u4"), ("kind_trials", "<u4", (5,)),
                          ("kind_zero_diff", "<u4", (5,)), ("dev_exponent_hist", "<u4", (256,))])

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libmpgemmfi.so")
_lib = None

_SYMBOLS = [
    "mpgemmfi_gemm", "mpgemmfi_campaign", "mpgemmfi_kstep", "mpgemmfi_flags_bytes",
    "mpgemmfi_flags_bitmap_offset", "mpgemmfi_campaign_workspace_bytes", "mpgemmfi_validate_sites",
    "mpgemmfi_strerror", "mpgemmfi_last_cuda_error", "mpgemmfi_version", "mpgemmfi_campaign_static",
    "mpgemmfi_set_tile_policy", "mpgemmfi_set_split_policy", "mpgemmfi_campaign_summary", "mpgemmfi_operand_exponents", "mpgemmfi_gemm_ranged",
    "mpgemmfi_gemm_addend", "mpgemmfi_set_wait_limit_ms", "mpgemmfi_debug_break_handover", "mpgemmfi_debug_launch_slot",
    "mpgemmfi_gemm_out16", "mpgemmfi_debug_segments", "mpgemmfi_null_launch",
]


class MpgemmfiError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        detail = ""
        if code == -7:
            detail = f" (cudaError {mpgemmfi_last_cuda_error()})"
        super().__init__(f"{where}: {mpgemmfi_strerror(code)} [{code}]{detail}")


def library_path() -> str:
    return _LIB_PATH


def exported_symbols():
    """Names every build of the library must export (the declarations of include/mpgemmfi.h)."""
    return list(_SYMBOLS)


def load_library():
    """Load libmpgemmfi.so; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2311_05782_b200.build`")
    L = C.CDLL(_LIB_PATH)
    vp, i, sz = C.c_void_p, C.c_int, C.c_size_t
    L.mpgemmfi_gemm.restype = i
    L.mpgemmfi_gemm.argtypes = [i, i, i, i, vp, vp, vp, vp, i, i, vp, vp]
    L.mpgemmfi_gemm_addend.restype = i
    L.mpgemmfi_gemm_addend.argtypes = [i, i, i, i, vp, vp, vp, vp, vp, i, i, vp, vp]
    L.mpgemmfi_gemm_out16.restype = i
    L.mpgemmfi_gemm_out16.argtypes = [i, i, i, i, vp, vp, vp, i, vp, vp, i, i, vp, vp]
    L.mpgemmfi_campaign.restype = i
    L.mpgemmfi_campaign.argtypes = [i, i, i, i, vp, vp, vp, vp, i, i, vp, vp, sz, vp]
    L.mpgemmfi_campaign_static.restype = i
    L.mpgemmfi_campaign_static.argtypes = [i, i, i, i, vp, vp, vp, vp, i, i, vp, vp]
    L.mpgemmfi_operand_exponents.restype = i
    L.mpgemmfi_operand_exponents.argtypes = [i, i, i, vp, vp, vp]
    L.mpgemmfi_gemm_ranged.restype = i
    L.mpgemmfi_gemm_ranged.argtypes = [i, i, i, i, vp, vp, vp, vp, i, i, vp, vp, vp, vp]
    L.mpgemmfi_campaign_summary.restype = i
    L.mpgemmfi_campaign_summary.argtypes = [vp, i, vp, vp]
    L.mpgemmfi_set_tile_policy.restype = i
    L.mpgemmfi_set_tile_policy.argtypes = [i]
    L.mpgemmfi_set_split_policy.restype = i
    L.mpgemmfi_set_split_policy.argtypes = [i]
    L.mpgemmfi_set_wait_limit_ms.restype = i
    L.mpgemmfi_set_wait_limit_ms.argtypes = [i]
    L.mpgemmfi_null_launch.restype = i
    L.mpgemmfi_null_launch.argtypes = [vp]
    L.mpgemmfi_debug_break_handover.restype = i
    L.mpgemmfi_debug_break_handover.argtypes = [i]
    L.mpgemmfi_debug_launch_slot.restype = i
    L.mpgemmfi_debug_launch_slot.argtypes = [C.c_uint32, C.POINTER(C.c_uint32)]
    L.mpgemmfi_debug_segments.restype = i
    L.mpgemmfi_debug_segments.argtypes = [i, i, i, i, vp, i]
    L.mpgemmfi_kstep.restype = i
    L.mpgemmfi_kstep.argtypes = [i]
    L.mpgemmfi_flags_bytes.restype = sz
    L.mpgemmfi_flags_bytes.argtypes = [i, i, i]
    L.mpgemmfi_flags_bitmap_offset.restype = sz
    L.mpgemmfi_flags_bitmap_offset.argtypes = [i]
    L.mpgemmfi_campaign_workspace_bytes.restype = sz
    L.mpgemmfi_campaign_workspace_bytes.argtypes = [i, i, i, i, i]
    L.mpgemmfi_validate_sites.restype = i
    L.mpgemmfi_validate_sites.argtypes = [vp, i, i, i, i, i, C.POINTER(C.c_int)]
    L.mpgemmfi_strerror.restype = C.c_char_p
    L.mpgemmfi_strerror.argtypes = [i]
    L.mpgemmfi_last_cuda_error.restype = i
    L.mpgemmfi_version.restype = i
    _lib = L
    return L


# ---------------------------------------------------------------- raw C ABI

def mpgemmfi_gemm(dtype, M, N, K, A, Bt, C_out, fault_sites, n_faults, detect_mode, flags_out, stream):
    """Raw call: every matrix argument is a device address (int), `stream` a cudaStream_t handle (int)."""
    return load_library().mpgemmfi_gemm(dtype, M, N, K, A, Bt, C_out, fault_sites, n_faults, detect_mode,
                                        flags_out, stream)


def mpgemmfi_gemm_addend(dtype, M, N, K, A, Bt, C_in, D, fault_sites, n_faults, detect_mode, flags_out, stream):
    """Raw call of D = A x B + C_in (device addresses; C_in may be D itself)."""
    return load_library().mpgemmfi_gemm_addend(dtype, M, N, K, A, Bt, C_in, D, fault_sites, n_faults, detect_mode,
                                               flags_out, stream)


def mpgemmfi_gemm_out16(dtype, M, N, K, A, Bt, C_in, out_format, D16, fault_sites, n_faults, detect_mode, flags_out, stream):
    """Raw call of the GEMM with a 16-bit result (OUT_FP16 / OUT_BF16); C_in is None or the FP32 addend."""
    return load_library().mpgemmfi_gemm_out16(dtype, M, N, K, A, Bt, C_in, out_format, D16, fault_sites, n_faults,
                                              detect_mode, flags_out, stream)


def mpgemmfi_campaign(dtype, M, N, K, A, Bt, C_clean, sites, n_trials, detect_mode, records, workspace,
                      workspace_bytes, stream):
    return load_library().mpgemmfi_campaign(dtype, M, N, K, A, Bt, C_clean, sites, n_trials, detect_mode, records,
                                            workspace, workspace_bytes, stream)


def mpgemmfi_campaign_static(dtype, M, N, K, A, Bt, C_clean, sites, n_trials, detect_mode, records, stream):
    """Raw call of the campaign variant that keeps its schedule in the library's built-in device array,
    for callers that are not allowed to allocate device memory. At most STATIC_MAX_TRIALS trials per call."""
    return load_library().mpgemmfi_campaign_static(dtype, M, N, K, A, Bt, C_clean, sites, n_trials, detect_mode,
                                                   records, stream)


def mpgemmfi_operand_exponents(dtype, rows, K, X, out, stream):
    """Raw call: out[r] = largest FP32 exponent field of row r of the rows x K operand matrix X (device pointers)."""
    return load_library().mpgemmfi_operand_exponents(dtype, rows, K, X, out, stream)


def mpgemmfi_gemm_ranged(dtype, M, N, K, A, Bt, C_out, fault_sites, n_faults, detect_mode, flags_out, exp_a, exp_bt, stream):
    """Raw call: mpgemmfi_gemm with the operands' exponent maxima for the output-level range check (OUTPUT_RANGE)."""
    return load_library().mpgemmfi_gemm_ranged(dtype, M, N, K, A, Bt, C_out, fault_sites, n_faults, detect_mode,
                                               flags_out, exp_a, exp_bt, stream)


def mpgemmfi_campaign_summary(records, n_trials, summary, stream):
    """Raw call: reduce n_trials device records into a device mpgemmfi_summary (SUMMARY_DTYPE.itemsize bytes)."""
    return load_library().mpgemmfi_campaign_summary(records, n_trials, summary, stream)


def campaign_summary(records, stream=None):
    """Deviation summary of a records tensor ([n, 12] int32 on CUDA); returns a host numpy record of SUMMARY_DTYPE."""
    torch = _torch()
    out = torch.empty(SUMMARY_DTYPE.itemsize // 4, dtype=torch.int32, device=records.device)
    stream_h = (torch.cuda.current_stream(records.device) if stream is None else stream).cuda_stream
    rc = mpgemmfi_campaign_summary(records.data_ptr() if records.shape[0] else None, records.shape[0], out.data_ptr(), stream_h)
    if rc != 0:
        raise MpgemmfiError(rc, "mpgemmfi_campaign_summary")
    return out.cpu().numpy().view(np.uint32).view(SUMMARY_DTYPE)[0]


def mpgemmfi_set_tile_policy(policy):
    """TILES_AUTO (0), TILES_SINGLE (1) or TILES_PAIR (2); process-wide."""
    return load_library().mpgemmfi_set_tile_policy(policy)


def mpgemmfi_set_split_policy(policy):
    """SPLIT_AUTO (0), SPLIT_OFF (1) or SPLIT_ON (2); process-wide."""
    return load_library().mpgemmfi_set_split_policy(policy)


def mpgemmfi_set_wait_limit_ms(ms):
    """How long a device-side wait of the GEMM kernel may last before the launch gives up (1..60000 ms, default 4000)."""
    return load_library().mpgemmfi_set_wait_limit_ms(ms)


def mpgemmfi_null_launch(stream):
    """Queue a kernel that does nothing (what a launch costs by itself when timed like a GEMM)."""
    return load_library().mpgemmfi_null_launch(stream)


def mpgemmfi_debug_break_handover(on):
    """Test hook: make the continuation of a cut tile wait for a hand-over that never comes."""
    return load_library().mpgemmfi_debug_break_handover(int(bool(on)))


def mpgemmfi_debug_launch_slot(counter):
    """(slot, tag) of the launch with the given counter value."""
    tag = C.c_uint32(0)
    slot = load_library().mpgemmfi_debug_launch_slot(int(counter) & 0xFFFFFFFF, C.byref(tag))
    return slot, tag.value


def mpgemmfi_debug_segments(num_tiles, num_kt, walkers, policy):
    """The tile schedule as the kernel's walkers will run it: uint32 array [n, 8] of
    (walker, index, tile, kt0, kt1, part, load, save)."""
    L = load_library()
    n = L.mpgemmfi_debug_segments(num_tiles, num_kt, walkers, policy, None, 0)
    if n < 0:
        raise MpgemmfiError(n, "mpgemmfi_debug_segments")
    out = np.zeros((n, 8), dtype=np.uint32)
    L.mpgemmfi_debug_segments(num_tiles, num_kt, walkers, policy, out.ctypes.data_as(C.c_void_p), n)
    return out


def mpgemmfi_kstep(dtype):
    return load_library().mpgemmfi_kstep(dtype)


def mpgemmfi_flags_bytes(M, N, n_faults):
    return load_library().mpgemmfi_flags_bytes(M, N, n_faults)


def mpgemmfi_flags_bitmap_offset(n_faults):
    return load_library().mpgemmfi_flags_bitmap_offset(n_faults)


def mpgemmfi_campaign_workspace_bytes(dtype, M, N, K, n_trials):
    return load_library().mpgemmfi_campaign_workspace_bytes(dtype, M, N, K, n_trials)


def mpgemmfi_validate_sites(host_sites: np.ndarray, dtype, M, N, K):
    """Returns (code, first_bad_index). host_sites: numpy array of 32-byte site entries."""
    s = np.ascontiguousarray(host_sites)
    assert s.dtype.itemsize == 32
    bad = C.c_int(-1)
    rc = load_library().mpgemmfi_validate_sites(s.ctypes.data_as(C.c_void_p), len(s), dtype, M, N, K, C.byref(bad))
    return rc, bad.value


def mpgemmfi_strerror(code):
    return load_library().mpgemmfi_strerror(code).decode()


def mpgemmfi_last_cuda_error():
    return load_library().mpgemmfi_last_cuda_error()


def mpgemmfi_version():
    return load_library().mpgemmfi_version()


# ---------------------------------------------------------------- torch-tensor convenience wrappers

def _torch():
    import torch
    return torch


def _check_operand(t, dtype, name):
    torch = _torch()
    want = torch.int32 if dtype == TF32 else torch.int16
    ok = {TF32: (torch.int32, torch.float32), FP16: (torch.int16, torch.float16),
          BF16: (torch.int16, torch.bfloat16)}[dtype]
    if not t.is_cuda or not t.is_contiguous() or t.dim() != 2 or t.dtype not in ok:
        raise ValueError(f"{name}: expected a contiguous 2-D CUDA tensor of dtype in {ok} (storage {want})")


class _HostSites:
    """A small site table kept in host memory (it travels in the launch parameters); quacks like a tensor here."""

    def __init__(self, arr):
        self.arr = arr

    def data_ptr(self):
        return self.arr.ctypes.data


def _sites_tensor(sites, device, inline=True):
    """numpy structured array (or None) -> the table to pass and its length. Up to INLINE_FAULTS entries stay in
    host memory (inline=False: copied to the device like a longer table); a longer table becomes an int32 CUDA
    tensor [n, 8]; CUDA tensors pass through."""
    torch = _torch()
    if sites is None:
        return None, 0
    if isinstance(sites, np.ndarray):
        s = np.ascontiguousarray(sites)
        assert s.dtype.itemsize == 32
        if len(s) == 0:
            return None, 0
        if inline and len(s) <= INLINE_FAULTS:
            host = np.empty(len(s) * 8 + 4, dtype=np.int32)          # room to start on a 16-byte boundary
            off = (-host.ctypes.data % 16) // 4
            host = host[off:off + len(s) * 8]
            host[:] = s.view(np.int32).reshape(-1)
            return _HostSites(host), len(s)
        t = torch.from_numpy(s.view(np.int32).reshape(len(s), 8)).to(device)
        return t, len(s)
    assert sites.is_cuda and sites.is_contiguous() and sites.dtype == torch.int32 and sites.shape[-1] == 8
    return (sites, sites.shape[0]) if sites.shape[0] else (None, 0)


def gemm(dtype, A, Bt, sites=None, detect_mode=DETECT_NONE, C_out=None, flags_out=None, stream=None, addend=None,
         out_format=OUT_FP32, inline_sites=True):
    """Fault-injected GEMM on CUDA tensors. Returns (C, flags) where flags is the raw uint32 buffer
    (as an int32 tensor) laid out as documented in include/mpgemmfi.h; see split_flags().
    addend: optional M x N float32 CUDA tensor, the C_in of D = A x B + C_in (it may be C_out itself).
    out_format: OUT_FP16 / OUT_BF16 give an M x N float16 / bfloat16 result (mpgemmfi_gemm_out16).
    sites: numpy structured array (up to INLINE_FAULTS entries are handed over in host memory unless
    inline_sites=False; more are copied to the device) or an int32 CUDA tensor [n, 8]."""
    torch = _torch()
    _check_operand(A, dtype, "A")
    _check_operand(Bt, dtype, "Bt")
    M, K = A.shape
    N, K2 = Bt.shape
    if K != K2:
        raise ValueError("A and Bt disagree on K")
    st, n_faults = _sites_tensor(sites, A.device, inline_sites)
    out_dtype = {OUT_FP32: torch.float32, OUT_FP16: torch.float16, OUT_BF16: torch.bfloat16}[out_format]
    if C_out is None:
        C_out = torch.empty((M, N), dtype=out_dtype, device=A.device)
    if flags_out is None:
        flags_out = torch.empty(mpgemmfi_flags_bytes(M, N, n_faults) // 4, dtype=torch.int32, device=A.device)
    stream_h = (torch.cuda.current_stream(A.device) if stream is None else stream).cuda_stream
    if out_format != OUT_FP32:
        if detect_mode & OUTPUT_RANGE:
            raise ValueError("the output-level range check writes FP32 only")
        if C_out.dtype != out_dtype or tuple(C_out.shape) != (M, N) or not C_out.is_contiguous():
            raise ValueError("C_out must be a contiguous M x N tensor of the output format")
        rc = mpgemmfi_gemm_out16(dtype, M, N, K, A.data_ptr(), Bt.data_ptr(), None if addend is None else addend.data_ptr(),
                                 out_format, C_out.data_ptr(), st.data_ptr() if st is not None else None, n_faults,
                                 detect_mode, flags_out.data_ptr(), stream_h)
        if rc != 0:
            raise MpgemmfiError(rc, "mpgemmfi_gemm_out16")
        return C_out, flags_out
    if detect_mode & OUTPUT_RANGE:
        if addend is not None:
            raise ValueError("the output-level range check takes no addend")
        # output-level range check: the exponent maxima of the (clean) operands come first
        ea = torch.empty(M, dtype=torch.int32, device=A.device)
        eb = torch.empty(N, dtype=torch.int32, device=A.device)
        for X, rows, e in ((A, M, ea), (Bt, N, eb)):
            rc = mpgemmfi_operand_exponents(dtype, rows, K, X.data_ptr(), e.data_ptr(), stream_h)
            if rc != 0:
                raise MpgemmfiError(rc, "mpgemmfi_operand_exponents")
        rc = mpgemmfi_gemm_ranged(dtype, M, N, K, A.data_ptr(), Bt.data_ptr(), C_out.data_ptr(),
                                  st.data_ptr() if st is not None else None, n_faults, detect_mode,
                                  flags_out.data_ptr(), ea.data_ptr(), eb.data_ptr(), stream_h)
        if rc != 0:
            raise MpgemmfiError(rc, "mpgemmfi_gemm_ranged")
        return C_out, flags_out
    if addend is not None:
        if addend.dtype != torch.float32 or tuple(addend.shape) != (M, N) or not addend.is_contiguous() or not addend.is_cuda:
            raise ValueError("addend must be a contiguous M x N float32 CUDA tensor")
        rc = mpgemmfi_gemm_addend(dtype, M, N, K, A.data_ptr(), Bt.data_ptr(), addend.data_ptr(), C_out.data_ptr(),
                                  st.data_ptr() if st is not None else None, n_faults, detect_mode,
                                  flags_out.data_ptr(), stream_h)
        if rc != 0:
            raise MpgemmfiError(rc, "mpgemmfi_gemm_addend")
        return C_out, flags_out
    rc = mpgemmfi_gemm(dtype, M, N, K, A.data_ptr(), Bt.data_ptr(), C_out.data_ptr(),
                       st.data_ptr() if st is not None else None, n_faults, detect_mode,
                       flags_out.data_ptr(), stream_h)
    if rc != 0:
        raise MpgemmfiError(rc, "mpgemmfi_gemm")
    return C_out, flags_out


def split_flags(flags, M, N, n_faults):
    """Copy a flags buffer to the host and split it into (header[16], site_log[n_faults], bitmap[M, ceil(N/32)])."""
    raw = flags.cpu().numpy().view(np.uint32)
    off = HEADER_WORDS + 4 * n_faults
    hdr = raw[:HEADER_WORDS].copy()
    log = raw[HEADER_WORDS:off].copy().view(SITE_LOG_DTYPE)
    wpr = (N + 31) // 32
    bitmap = raw[off:off + M * wpr].reshape(M, wpr).copy()
    return hdr, log, bitmap


def campaign(dtype, A, Bt, sites, detect_mode=DETECT_NONE, C_clean=None, records=None, workspace=None, stream=None):
    """Injection campaign on CUDA tensors. Returns (C_clean, records) with records an int32 tensor [n_trials, 12]
    (view the host copy as RECORD_DTYPE)."""
    torch = _torch()
    _check_operand(A, dtype, "A")
    _check_operand(Bt, dtype, "Bt")
    M, K = A.shape
    N, _ = Bt.shape
    st, n_trials = _sites_tensor(sites, A.device, inline=False)      # the campaign reads its table on the device
    if C_clean is None:
        C_clean = torch.empty((M, N), dtype=torch.float32, device=A.device)
    if records is None:
        records = torch.empty((max(n_trials, 1), 12), dtype=torch.int32, device=A.device)
    ws_bytes = mpgemmfi_campaign_workspace_bytes(dtype, M, N, K, n_trials)
    if workspace is None:
        workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=A.device)
    stream_h = (torch.cuda.current_stream(A.device) if stream is None else stream).cuda_stream
    rc = mpgemmfi_campaign(dtype, M, N, K, A.data_ptr(), Bt.data_ptr(), C_clean.data_ptr(),
                           st.data_ptr() if st is not None else None, n_trials, detect_mode,
                           records.data_ptr(), workspace.data_ptr(), workspace.numel(), stream_h)
    if rc != 0:
        raise MpgemmfiError(rc, "mpgemmfi_campaign")
    return C_clean, records[:n_trials]
