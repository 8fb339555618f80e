"""Shared helpers of the GPU parity tests: run the CUDA path and the oracle on the same inputs and compare.

Comparison rules
  * untouched elements and elements reached only through a faulty operand:
        |C_gpu - C_oracle| <= 1e-3 * (|A'||B'|)_ij   with the operands actually multiplied;
    an infinite or NaN bound (the faulty operand is Inf/NaN) admits anything.
  * elements carrying an OUT / ACC / TERM site: the value the mask was applied to must agree
    within the tolerance above, the flip itself must be bit-exact (after == before ^ mask), and
    the stored element must be what the checks make of the GPU's own flipped value.
  * flags, counts and indices are bit-exact, except on "fragile" sites where the two `before`
    values (both within tolerance) differ in sign or exponent field, so that the flip lands on
    different bits; those are counted and must stay rare.
"""
import numpy as np
import torch

import oracle as orc
import paper_2311_05782_b200 as mpg

TOL = 1e-3
ELEMENT_KINDS = (orc.KIND_ACC, orc.KIND_OUT, orc.KIND_TERM)


def to_dev(bits: np.ndarray, dtype: int) -> torch.Tensor:
    if dtype == orc.TF32:
        return torch.from_numpy(bits.view(np.int32)).cuda()
    return torch.from_numpy(bits.view(np.int16)).cuda()


def faulted_operands(dtype, A, Bt, sites):
    A2, B2 = A.copy(), Bt.copy()
    M, K = A.shape
    N = Bt.shape[0]
    for s in sites:
        if s["kind"] == orc.KIND_A and s["row"] < M and s["k"] < K:
            A2[s["row"], s["k"]] = orc.flip_operand(dtype, int(A2[s["row"], s["k"]]), int(s["xor_mask"]))
        elif s["kind"] == orc.KIND_B and s["col"] < N and s["k"] < K:
            B2[s["col"], s["k"]] = orc.flip_operand(dtype, int(B2[s["col"], s["k"]]), int(s["xor_mask"]))
    return A2, B2


def close(x, y, tol):
    """|x-y| <= tol, NaN matches NaN, equal infinities match, unbounded tolerance admits anything."""
    x = np.asarray(x, dtype=np.float64); y = np.asarray(y, dtype=np.float64); tol = np.asarray(tol, dtype=np.float64)
    with np.errstate(invalid="ignore"):
        ok = np.abs(x - y) <= tol
    ok |= np.isnan(x) & np.isnan(y)
    ok |= (x == y)
    ok |= ~np.isfinite(tol)
    return ok


def bits_f32(u):
    return np.array([u], dtype=np.uint32).view(np.float32)[0]


def run_gpu_gemm(dtype, A, Bt, sites, mode, addend=None, in_place=False):
    M, K = A.shape
    N = Bt.shape[0]
    n = 0 if sites is None else len(sites)
    if addend is None:
        Cg, flags = mpg.gemm(dtype, to_dev(A, dtype), to_dev(Bt, dtype), sites, mode)
    else:
        cin = torch.from_numpy(addend).cuda()
        Cg, flags = mpg.gemm(dtype, to_dev(A, dtype), to_dev(Bt, dtype), sites, mode, addend=cin,
                             C_out=cin if in_place else None)
    torch.cuda.synchronize()
    hdr, log, bm = mpg.split_flags(flags, M, N, n)
    return Cg.cpu().numpy(), hdr, log, bm


def check_gemm_against_oracle(dtype, A, Bt, sites, mode, max_fragile=0, addend=None, in_place=False):
    """Full element-by-element comparison at sizes the oracle finishes quickly. Returns the number of fragile sites.
    addend: the C_in of D = A x B + C_in (its magnitude joins the tolerance); in_place: D is written over it."""
    sites = np.zeros(0, dtype=orc.SITE) if sites is None else sites
    M, K = A.shape
    N = Bt.shape[0]
    Cg, hdr_g, log_g, bm_g = run_gpu_gemm(dtype, A, Bt, sites, mode, addend, in_place)
    Co, hdr_o, log_o, bm_o = orc.gemm(dtype, A, Bt, sites, mode, addend=addend)
    assert not (hdr_g[0] & mpg.STATUS_WAIT_LIMIT), "device wait limit hit"
    A2, B2 = faulted_operands(dtype, A, Bt, sites)
    tol = TOL * orc.absprod(dtype, A2, B2)
    if addend is not None:
        tol = tol + TOL * np.abs(addend).astype(np.float64)

    touched = np.zeros((M, N), dtype=bool)
    fragile = 0
    valid = log_o["status"] != 2
    assert np.array_equal(log_g["status"] == 2, ~valid), "the two sides skip different sites"
    assert hdr_g[3] == hdr_o[3] and hdr_g[4] == hdr_o[4]
    assert bool(hdr_g[0] & 1) == bool(hdr_o[0] & 1)
    fragile_elems = set()
    seen = {}
    for t, s in enumerate(sites):
        if not valid[t]:
            continue
        kind = int(s["kind"])
        lg, lo = log_g[t], log_o[t]
        if kind in (orc.KIND_A, orc.KIND_B):
            assert lg["before_bits"] == lo["before_bits"] and lg["after_bits"] == lo["after_bits"]
            assert lg["final_bits"] == lo["final_bits"] and lg["status"] == 1
            continue
        i, j = int(s["row"]), int(s["col"])
        touched[i, j] = True
        assert lg["after_bits"] == lg["before_bits"] ^ s["xor_mask"], "flip is not bit-exact"
        if kind == orc.KIND_TERM:
            # products of two low-precision operands are exact: bit-equal on both sides
            assert lg["before_bits"] == lo["before_bits"] and lg["final_bits"] == lo["final_bits"]
            assert lg["status"] == lo["status"]
        elif (i, j) not in seen:
            # first site on this element: the value it meets is a (partial) clean sum
            assert close(bits_f32(lg["before_bits"]), bits_f32(lo["before_bits"]), tol[i, j])
            if (lg["before_bits"] ^ lo["before_bits"]) & 0xFF800000:
                fragile += 1
                fragile_elems.add((i, j))
        elif kind == orc.KIND_OUT and seen[(i, j)][0] == orc.KIND_OUT:
            # later output sites continue from the previous flip, bit for bit
            assert lg["before_bits"] == log_g[seen[(i, j)][1]]["after_bits"]
        seen[(i, j)] = (kind, t)
    # stored values
    ok = close(Cg, Co, tol) | touched
    assert ok.all(), f"{(~ok).sum()} elements out of tolerance, first at {np.argwhere(~ok)[:5].tolist()}"
    # elements with sites: the stored value is what the checks make of the GPU's own value
    tech = mode & 3
    for (i, j) in zip(*np.nonzero(touched)):
        g = int(Cg[i, j].view(np.uint32))
        flagged = bool((bm_g[i, j // 32] >> (j % 32)) & 1)
        if tech == 1:
            if mode & orc.CORRECT:
                assert orc.boundcheck_detect(g) == 0
            else:
                assert flagged == bool(orc.boundcheck_detect(g))
        else:
            assert not flagged
        # OUT-only elements: final is exactly check(before ^ masks)
        mine = [t for t, s in enumerate(sites) if valid[t] and int(s["kind"]) in ELEMENT_KINDS
                and int(s["row"]) == i and int(s["col"]) == j]
        if all(int(sites[t]["kind"]) == orc.KIND_OUT for t in mine):
            v = int(log_g[mine[0]]["before_bits"])
            for t in mine:
                v ^= int(sites[t]["xor_mask"])
            if tech == 1 and (mode & orc.CORRECT):
                v = orc.boundcheck_correct(v)
            assert g == v
            for t in mine:
                assert int(log_g[t]["final_bits"]) == g
    # flags: bit-exact outside fragile elements
    diff = bm_g ^ bm_o
    for (i, j) in fragile_elems:
        diff[i, j // 32] &= ~np.uint32(1 << (j % 32))
    assert not diff.any(), f"flag bitmaps differ at {np.argwhere(diff)[:5].tolist()}"
    if not fragile_elems:
        assert hdr_g[1] == hdr_o[1] and hdr_g[2] == hdr_o[2]
    assert sum(bin(int(w)).count("1") for w in bm_g.reshape(-1)) == hdr_g[1]
    assert fragile <= max_fragile, f"{fragile} fragile sites"
    return fragile


def run_gpu_campaign(dtype, A, Bt, sites, mode):
    Cg, rec = mpg.campaign(dtype, to_dev(A, dtype), to_dev(Bt, dtype), sites, mode)
    torch.cuda.synchronize()
    return Cg.cpu().numpy(), rec.cpu().numpy().view(np.uint32).reshape(-1).view(mpg.RECORD_DTYPE)


def check_campaign_against_oracle(dtype, A, Bt, sites, mode, max_fragile=0):
    """Trial records against the oracle's incremental evaluation."""
    M, K = A.shape
    N = Bt.shape[0]
    Cg, rg = run_gpu_campaign(dtype, A, Bt, sites, mode)
    Cclean, *_ = orc.gemm(dtype, A, Bt)
    ro = orc.campaign(dtype, A, Bt, Cclean, sites, mode)
    ro_raw = orc.campaign(dtype, A, Bt, Cclean, sites, mode & ~orc.CORRECT) if mode & orc.CORRECT else ro
    ap = orc.absprod(dtype, A, Bt)
    assert close(Cg, Cclean, TOL * ap).all()
    fragile = 0
    for t, s in enumerate(sites):
        g, o = rg[t], ro[t]
        kind = int(s["kind"])
        assert g["kind"] == o["kind"] == kind
        if o["status"] & 0x100:
            assert g["status"] & 0x100
            continue
        assert g["primary_index"] == o["primary_index"] and g["n_affected"] == o["n_affected"]
        assert g["after_bits"] == g["before_bits"] ^ (s["xor_mask"] if kind in ELEMENT_KINDS else 0) or kind in (orc.KIND_A, orc.KIND_B)
        if kind in (orc.KIND_ACC, orc.KIND_TERM):
            # recomputed in k order on both sides: everything is bit-exact
            # ... except the payload of a NaN that the fault created and later additions carried along:
            # IEEE 754 leaves it to the platform, so what a correction makes of it is not unique
            nan_made = bool(np.isnan(bits_f32(ro_raw[t]["final_bits"])))
            for f in g.dtype.names:
                if nan_made and f in ("final_bits", "max_abs_dev"):
                    continue
                assert g[f] == o[f] or (f == "max_abs_dev" and np.isnan(g[f]) and np.isnan(o[f])), (t, f, g, o)
        elif kind == orc.KIND_OUT:
            i, j = int(s["row"]), int(s["col"])
            assert g["before_bits"] == Cg[i, j].view(np.uint32)
            assert close(bits_f32(g["before_bits"]), bits_f32(o["before_bits"]), TOL * ap[i, j])
            if (int(g["before_bits"]) ^ int(o["before_bits"])) & 0xFF800000:
                fragile += 1
                continue
            for f in ("status", "n_detected", "idx_hash", "first_detected"):
                assert g[f] == o[f], (t, f, g, o)
            fin = int(g["after_bits"])
            if (mode & 3) == 1 and (mode & orc.CORRECT):
                fin = orc.boundcheck_correct(fin)
            assert g["final_bits"] == fin
            dev_tol = TOL * ap[i, j] * max(1.0, abs(float(bits_f32(g["final_bits"]))) / max(abs(float(Cg[i, j])), 1e-30))
            assert close(g["max_abs_dev"], o["max_abs_dev"], max(dev_tol, 1e-6 * abs(float(o["max_abs_dev"]))))
        else:
            assert g["before_bits"] == o["before_bits"] and g["after_bits"] == o["after_bits"]
            assert g["final_bits"] == o["final_bits"]
            # the affected row/column: detection decided element by element on values within tolerance
            if g["n_detected"] != o["n_detected"] or g["idx_hash"] != o["idx_hash"]:
                fragile += 1
                continue
            assert g["first_detected"] == o["first_detected"]
            assert (g["status"] & 6) == (o["status"] & 6)
            od = float(o["max_abs_dev"])
            # a faulty operand that is Inf or NaN makes NaNs whose payloads (and what a correction makes of them) are
            # not part of parity
            special = not np.isfinite(orc.widen(dtype, int(o["after_bits"])))
            assert special or close(g["max_abs_dev"], od, max(1e-3 * abs(od), 1e-3 * float(ap.max()))) or not np.isfinite(od), (t, g, o)
    assert fragile <= max_fragile, f"{fragile} fragile trials"
    return fragile
