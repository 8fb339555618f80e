"""Shared helpers of the GPU parity tests: run the CUDA path and the oracle on the same inputs and compare.

Comparison rules
  * untouched elements and elements reached only through a faulty operand:
        |C_gpu - C_oracle| <= 1e-3 * (|A'||B'|)_ij   with the operands actually multiplied;
    an infinite or NaN bound (the faulty operand is Inf/NaN) admits anything.
  * elements carrying an OUT / ACC / TERM site: the value the mask was applied to must agree
    within the tolerance above, the flip itself must be bit-exact (after == before ^ mask), and
    the stored element must be what the checks make of the GPU's own flipped value.
  * flags, counts and indices are bit-exact, except (a) on "fragile" OUT / ACC sites where the two
    `before` values (both checked to be within tolerance) differ in sign or exponent field, so that
    the flip lands on different bits (counted, bounded per test), and (b) on elements whose
    unflagged value sits within tolerance of the BoundCheck edge 131072: there the two sides may
    decide differently, and the test checks that every disagreement is of that kind.
  * operand trials of a campaign: bit for bit against the oracle's Eq. 1-2 form on the device's clean
    C, and against the oracle's recompute under rule (b).
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


def absprod_fast(dtype, A, Bt):
    """(|A||B|)_ij by a library matrix product (float32 is plenty for a tolerance): for sizes where the oracle's
    double-precision triple loop would take minutes."""
    def widen(bits):
        if dtype == orc.FP16:
            return np.abs(bits.view(np.float16).astype(np.float32))
        if dtype == orc.BF16:
            return np.abs((bits.astype(np.uint32) << 16).view(np.float32))
        return np.abs((bits & np.uint32(0xFFFFE000)).view(np.float32))
    return (widen(A) @ widen(Bt).T).astype(np.float64)


def check_gemm_against_oracle(dtype, A, Bt, sites, mode, max_fragile=0, addend=None, in_place=False, fast_tol=False):
    """Full element-by-element comparison. Returns the number of fragile sites.
    addend: the C_in of D = A x B + C_in (its magnitude joins the tolerance); in_place: D is written over it;
    fast_tol: take (|A||B|) from a library matrix product (the benchmark's full sizes)."""
    sites = np.zeros(0, dtype=orc.SITE) if sites is None else sites
    M, K = A.shape
    N = Bt.shape[0]
    Cg, hdr_g, log_g, bm_g = run_gpu_gemm(dtype, A, Bt, sites, mode, addend, in_place)
    Co, hdr_o, log_o, bm_o = orc.gemm(dtype, A, Bt, sites, mode, addend=addend)
    assert not (hdr_g[0] & mpg.STATUS_WAIT_LIMIT), "device wait limit hit"
    A2, B2 = faulted_operands(dtype, A, Bt, sites)
    tol = TOL * (absprod_fast(dtype, A2, B2) if fast_tol else orc.absprod(dtype, A2, B2))
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
    # flags: bit-exact outside fragile elements
    diff = bm_g ^ bm_o
    for (i, j) in fragile_elems:
        diff[i, j // 32] &= ~np.uint32(1 << (j % 32))
    edge = 0
    edge_mask = np.zeros((M, N), dtype=bool)
    for (i, w) in np.argwhere(diff):
        for j in range(32 * w, min(N, 32 * w + 32)):
            if (int(diff[i, w]) >> (j % 32)) & 1:
                # exactly one side left the element unflagged, so it still holds the unchecked value there: it must
                # sit within tolerance below the BoundCheck edge
                raw = float(Co[i, j]) if (int(bm_g[i, w]) >> (j % 32)) & 1 else float(Cg[i, j])
                assert 0.0 <= BOUND_EDGE - abs(raw) <= tol[i, j], f"flags differ at ({i},{j}) away from the edge: {raw}"
                edge += 1
                edge_mask[i, j] = True
    if not fragile_elems and not edge:
        assert hdr_g[1] == hdr_o[1] and hdr_g[2] == hdr_o[2]
    # stored values (an element at the edge that only one side corrected is compared through its flag above)
    ok = close(Cg, Co, tol) | touched | edge_mask
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
    assert int(np.bitwise_count(bm_g).sum()) == hdr_g[1]
    assert fragile <= max_fragile, f"{fragile} fragile sites"
    return fragile


BOUND_EDGE = 131072.0        # BoundCheck flags |v| >= 2^17 (exponent field 0x90 and above)


def trial_values(dtype, A, Bt, C, s, form):
    """orc.operand_trial_values on the slice of the problem that the site reaches (one row of A and of C, or one row of
    Bt and one column of C), so that the oracle does not widen matrices it will not read."""
    one = np.array(s, dtype=orc.SITE).reshape(1).copy()
    if int(s["kind"]) == orc.KIND_A:
        i = int(s["row"]); one["row"] = 0
        return orc.operand_trial_values(dtype, A[i:i + 1], Bt, C[i:i + 1], one[0], form)
    j = int(s["col"]); one["col"] = 0
    return orc.operand_trial_values(dtype, A, Bt[j:j + 1], np.ascontiguousarray(C[:, j:j + 1]), one[0], form)


def check_operand_trial(dtype, A, Bt, s, mode, Cg, Cclean, g, o, w, deep=True):
    """One A / B trial: device record g, oracle record o (row / column accumulated again with the faulty operand on the
    oracle's clean C: the definition), oracle record w (Eq. 1-2 on the finished sums of the DEVICE's clean C).

    g against w: every field bit for bit (both apply the same four rounded operations to the same words; only a NaN's
    payload is left open). g against o: the two forms differ by rounding, so counts and indices must agree except on
    elements whose value sits within tolerance of the BoundCheck edge, and the "changed" bit except where the fault
    moves every element by less than the tolerance. deep=False skips the element-by-element part when the two
    records agree outright (the benchmark's full sizes, where it costs seconds per trial)."""
    is_a = int(s["kind"]) == orc.KIND_A
    special = not np.isfinite(orc.widen(dtype, int(o["after_bits"])))
    exact = all(g[f] == w[f] or (f == "max_abs_dev" and np.isnan(g[f]) and np.isnan(w[f])) for f in g.dtype.names)
    v_w = None
    if not exact:
        v_w = trial_values(dtype, A, Bt, Cg, s, 1)
        has_nan = bool(np.isnan(v_w).any())
        for f in g.dtype.names:
            if has_nan and f in ("max_abs_dev", "status"):
                continue
            assert g[f] == w[f], ("write-back form", f, g, w)
    if special:
        return          # a faulty operand that is Inf or NaN: the finished sum cannot give it back (reading R17)
    same_sets = all(g[f] == o[f] for f in ("n_detected", "idx_hash", "first_detected")) and (g["status"] & 6) == (o["status"] & 6)
    same_changed = (g["status"] & 1) == (o["status"] & 1)
    od = float(o["max_abs_dev"])
    if not deep and same_sets and same_changed and close(g["max_abs_dev"], od, 1e-4 * abs(od) + 1e-7):
        return
    if v_w is None:
        v_w = trial_values(dtype, A, Bt, Cg, s, 1)
    v_o = trial_values(dtype, A, Bt, Cclean, s, 0)
    # tolerance of each affected element, with the operand actually multiplied
    A2, B2 = faulted_operands(dtype, A, Bt, [s])
    if is_a:
        i = int(s["row"])
        tol = TOL * absprod_fast(dtype, A2[i:i + 1], B2)[0]
        clean_tol = TOL * absprod_fast(dtype, A[i:i + 1], Bt)[0]
    else:
        j = int(s["col"])
        tol = TOL * absprod_fast(dtype, A2, B2[j:j + 1])[:, 0]
        clean_tol = TOL * absprod_fast(dtype, A, Bt[j:j + 1])[:, 0]
    assert close(v_w, v_o, tol + clean_tol).all(), "write-back values leave the tolerance of the recomputed ones"
    differ = np.zeros(len(v_o), dtype=bool)
    if (mode & 3) == 1:
        det_w = ~(np.abs(v_w) < BOUND_EDGE)
        det_o = ~(np.abs(v_o) < BOUND_EDGE)
        differ = det_w != det_o
        assert (np.abs(np.abs(v_o[differ].astype(np.float64)) - BOUND_EDGE) <= (tol + clean_tol)[differ]).all(), \
            "detected sets differ on elements that are not at the BoundCheck edge"
    if not differ.any():
        assert same_sets, (g, o)
    if not same_changed:
        # "changed" is ill-posed only when the fault moves no element by more than the tolerance
        x = orc.widen(dtype, int(o["before_bits"])); xf = orc.widen(dtype, int(o["after_bits"]))
        other = Bt[:, int(s["k"])] if is_a else A[:, int(s["k"])]
        y = np.array([orc.widen(dtype, int(v)) for v in other], dtype=np.float64)
        assert (np.abs((xf - x) * y) <= tol + clean_tol).all(), "the changed bits differ although the fault moves an element visibly"
    if not differ.any():
        # largest deviation: each side's final and clean values are within their tolerances of the other side's
        assert close(g["max_abs_dev"], od, float((tol + 2 * clean_tol).max())), (g, o)


def run_gpu_campaign(dtype, A, Bt, sites, mode):
    Cg, rec = mpg.campaign(dtype, to_dev(A, dtype), to_dev(Bt, dtype), sites, mode)
    torch.cuda.synchronize()
    return Cg.cpu().numpy(), rec.cpu().numpy().view(np.uint32).reshape(-1).view(mpg.RECORD_DTYPE)


def check_campaign_against_oracle(dtype, A, Bt, sites, mode, max_fragile=0, Cclean=None, ap=None, deep_every=1):
    """Trial records against the oracle's incremental evaluation. Cclean / ap: the oracle's clean product and
    (|A||B|) when the caller has them already; deep_every: operand trials t with t % deep_every == 0 take the
    element-by-element comparison even when their records agree outright (0: only those that disagree)."""
    M, K = A.shape
    N = Bt.shape[0]
    Cg, rg = run_gpu_campaign(dtype, A, Bt, sites, mode)
    if Cclean is None:
        Cclean, *_ = orc.gemm(dtype, A, Bt)
    ro = orc.campaign(dtype, A, Bt, Cclean, sites, mode)
    ro_raw = orc.campaign(dtype, A, Bt, Cclean, sites, mode & ~orc.CORRECT) if mode & orc.CORRECT else ro
    if ap is None:
        ap = orc.absprod(dtype, A, Bt)
    assert close(Cg, Cclean, TOL * ap).all()
    # operand trials once more in the oracle, in the form the device uses: Eq. 1-2 on the finished sums of the clean C
    # that the device itself produced
    rw = orc.campaign(dtype, A, Bt, Cg, sites, mode, operand_form=1)
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
            check_operand_trial(dtype, A, Bt, s, mode, Cg, Cclean, g, o, rw[t],
                                deep=bool(deep_every) and t % deep_every == 0)
    assert fragile <= max_fragile, f"{fragile} fragile trials"
    return fragile
