"""Shared plumbing of the GPU parity tests: upload a seeded workload, run it through the
C-ABI binding, evaluate the oracle on the checked rows / columns and compare.

Acceptance (per checked element, against the UNROUNDED fp64 oracle value y):
    |D_gpu - y| <= 2e-3 * (|alpha| * sum_k |a||b| + |beta| * |C_in| + |bias_j|) + 1e-5  (+ u_out * |y| for a 16-bit
    output: when there is no cancellation, |y| equals the sum in the first term and rounding y to bf16 alone can
    move it by 2^-8 |y| = 3.9e-3 |y|, more than the 2e-3 allows)
and, over each checked block, the relative Frobenius error
    fp32 output  : ||D_gpu - y||_F / ||y||_F <= 1e-4
    16-bit output: every element within one unit in the last place of RNE(y -> output dtype)
                   (or within the absolute 1e-5 of y: values that small are governed by the
                   absolute term), at least 99 % of the elements with |y| >= 1e-4 bit-identical
                   to it, and
                   ||D_gpu - RNE(y)||_F / ||RNE(y)||_F <= max(1e-4, 0.1 * u_out),
                   u_out = 2^-8 (bf16) or 2^-11 (fp16).
Rounding y to bf16 alone moves it by ~1.7e-3 relative (fp16: ~2e-4), so the 1e-4 bar cannot be
applied to a 16-bit output against y; against the rounded oracle the only differences are
elements whose fp32 accumulator landed on the other side of a rounding boundary.  With a
fraction f of such one-ulp flips the Frobenius distance is about u_out * sqrt(f); fp32
accumulation over K = 8192 terms with heavy cancellation (config c2) flips about 0.5 % of the
elements, so the bar is set at f = 1 %, i.e. 0.1 * u_out.  The accumulator itself is held to 1e-4
against y by re-running the same plan with fp32 output.
A transcendental activation (GELU, SiLU) is evaluated in fp32 with the hardware's approximate exp2 and
reciprocal, or erff() with the cancellation of 1 + erf(x) in its negative half: a relative error d_act of
up to about 1e-5 in the value that is then rounded.  A rounding boundary of the output format lies within
that distance of a fraction 2 * d_act / u_out of the values (4 % for fp16, 0.5 % for bf16), so for those
epilogues the share of bit-identical elements is required to be 99 % minus that fraction; the one-ulp,
per-element and Frobenius bars are unchanged.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2512_16465_b200 as bg
import workloads as wl

REL_TOL, ABS_TOL, FROB_TOL = 2e-3, 1e-5, 1e-4
D_ACT = 1e-5   # relative fp32 error allowed to a transcendental activation before the output rounding (see above)
U_OUT = {wl.BF16: 2.0 ** -8, wl.F16: 2.0 ** -11, wl.F32: 0.0}


def frob_tol_for(c_dtype: int) -> float:
    return max(FROB_TOL, 0.1 * U_OUT[c_dtype])


def ulp_distance(a_bits: np.ndarray, b_bits: np.ndarray) -> np.ndarray:
    """Distance in representable values between two arrays of 16-bit float patterns."""
    def key(x):
        x = x.astype(np.int32)
        return np.where(x & 0x8000, -(x & 0x7FFF), x)
    return np.abs(key(a_bits) - key(b_bits))
_TORCH_DT = {wl.BF16: torch.bfloat16, wl.F16: torch.float16, wl.F32: torch.float32}


def to_device(arr: np.ndarray, dtype: int) -> torch.Tensor:
    if dtype == wl.F32 or arr.dtype == np.uint8:      # fp32 values, or the bytes of 8-bit floats
        return torch.from_numpy(arr).cuda()
    return torch.from_numpy(arr.view(np.int16)).cuda().view(_TORCH_DT[dtype])


def to_host_bits(t: torch.Tensor, dtype: int) -> np.ndarray:
    if dtype == wl.F32:
        return t.cpu().numpy()
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def desc_of(w: wl.Workload, flags: int = 0, c_dtype=None, options: int = 0) -> bg.Desc:
    cd = w.c_dtype if c_dtype is None else c_dtype
    return bg.make_desc(w.M, w.N, w.K, w.transa, w.transb, w.ab_dtype, cd, w.lda, w.ldb, w.ldc, w.batch,
                        w.stride_a, w.stride_b, w.stride_c, w.epilogue, flags | bg.make_flags(bias_per_row=w.bias_per_row, a_lower=w.a_tri == 1, a_upper=w.a_tri == 2,
                                                                                           d_lower=w.d_tri == 1, d_upper=w.d_tri == 2),
                        structure=w.b_tri | (4 if w.d_mirror else 0), options=options)


def problem_of(w: wl.Workload, c_dtype=None) -> oracle.Problem:
    cd = w.c_dtype if c_dtype is None else c_dtype
    return oracle.Problem(w.M, w.N, w.K, w.transa, w.transb, w.ab_dtype, cd, w.lda, w.ldb, w.ldc, w.batch,
                          w.stride_a, w.stride_b, w.stride_c, w.epilogue, w.bias_per_row)


def c_in_as(inputs: dict, w: wl.Workload, c_dtype: int):
    """C_in converted to another output dtype (for the fp32-output re-run of a 16-bit config)."""
    c = inputs["C"]
    if c is None or c_dtype == w.c_dtype:
        return c
    vals = oracle.decode(c, w.c_dtype)
    return oracle.round_to(vals, c_dtype)


_NAN_BITS = {wl.BF16: 0x7FC0, wl.F16: 0x7E00, wl.FP8_E4M3: 0x7F, wl.FP8_E5M2: 0x7F}


def poison_operand_padding(arr: np.ndarray, dtype: int, rows: int, row_len: int, ld: int, batch: int, stride: int) -> np.ndarray:
    """A copy of a stored operand (``batch`` matrices of ``rows`` x ``row_len`` elements, pitch ``ld``, ``stride`` apart)
    in which every element that is not part of a matrix -- the padding behind each row and the gaps between batches --
    holds a NaN.  A kernel that reads any of them (a tensor map with the pitch as its extent, a box that runs past
    the row's end) turns its result into NaN."""
    if ld == row_len and (batch == 1 or stride == rows * ld) and arr.size == batch * rows * ld:
        return arr                                   # tightly packed: there is no padding
    out = np.full_like(arr, _NAN_BITS[dtype])
    idx = (np.arange(batch, dtype=np.int64)[:, None, None] * stride + np.arange(rows, dtype=np.int64)[None, :, None] * ld +
           np.arange(row_len, dtype=np.int64)[None, None, :]).ravel()
    out[idx] = arr[idx]
    return out


def run_gpu(w: wl.Workload, inputs: dict, flags: int = 0, c_dtype=None, poison: bool = True, repeats: int = 1, options: int = 0):
    """Run the workload through the binding; returns (host bit array of the whole C buffer, plan info).  The device
    copies of A and B carry NaN in every padding element (the oracle sees the plain inputs)."""
    cd = w.c_dtype if c_dtype is None else c_dtype
    plan = bg.Plan(desc_of(w, flags, cd, options))
    try:
        a_rows, a_len = (w.K, w.M) if w.transa else (w.M, w.K)
        b_rows, b_len = (w.N, w.K) if w.transb else (w.K, w.N)
        A = to_device(poison_operand_padding(inputs["A"], w.ab_dtype, a_rows, a_len, w.lda, w.batch, w.stride_a), w.ab_dtype)
        B = to_device(poison_operand_padding(inputs["B"], w.ab_dtype, b_rows, b_len, w.ldb, w.batch, w.stride_b), w.ab_dtype)
        bias = None if inputs["bias"] is None else to_device(inputs["bias"], wl.F32)
        cin = c_in_as(inputs, w, cd)
        outs = []
        for _ in range(repeats):
            if cin is not None:
                C = to_device(cin, cd).clone()
            else:
                C = torch.empty(w.elems_c(), dtype=_TORCH_DT[cd], device="cuda")
                if poison:   # beta == 0 must never read C: NaN would propagate
                    C.fill_(float("nan"))
            plan.run(A, B, C, bias, w.alpha, w.beta)
            torch.cuda.synchronize()
            st = plan.status()
            if st != bg.OK:
                raise bg.GemmError(st, "gemm_plan_status")
            outs.append(to_host_bits(C, cd))
        for o in outs[1:]:
            assert o.tobytes() == outs[0].tobytes(), "run-to-run results differ bitwise"   # (NaN-poisoned padding included)
        return outs[0], plan.info
    finally:
        plan.close()


def gather(cbits: np.ndarray, w: wl.Workload, batches, rows, cols) -> np.ndarray:
    idx = (np.asarray(batches)[:, None, None] * w.stride_c + np.asarray(rows)[None, :, None] * w.ldc +
           np.asarray(cols)[None, None, :])
    return cbits[idx]


def compare_block(got_bits: np.ndarray, y: np.ndarray, bound: np.ndarray, c_dtype: int) -> dict:
    got = oracle.decode(got_bits, c_dtype)
    err = np.abs(got - y)
    # a 16-bit output may sit half an ulp (relative 2^-8 / 2^-11 at the bottom of a binade) from y by rounding alone
    tol = REL_TOL * bound + ABS_TOL + U_OUT[c_dtype] * np.abs(y)
    ref_bits = oracle.round_to(y, c_dtype)
    ref = oracle.decode(ref_bits, c_dtype) if c_dtype != wl.F32 else y
    denom = float(np.linalg.norm(ref.ravel()))
    frob = float(np.linalg.norm((got - ref).ravel())) / max(denom, 1e-300)
    frob_unrounded = float(np.linalg.norm((got - y).ravel())) / max(float(np.linalg.norm(y.ravel())), 1e-300)
    same = got_bits == ref_bits
    big = np.abs(y) >= 1e-4
    exact = float(np.mean(same[big])) if big.any() else 1.0
    finite = bool(np.all(np.isfinite(got)))
    max_ulp = 0
    if c_dtype != wl.F32 and err.size:
        ulps = ulp_distance(got_bits, ref_bits)
        ulps = np.where(err <= ABS_TOL, np.minimum(ulps, 1), ulps)
        max_ulp = int(ulps.max())
    worst = float(np.max(err / tol)) if err.size else 0.0
    return {"max_err_over_tol": worst, "frob": frob, "frob_unrounded": frob_unrounded, "bit_identical": exact,
            "finite": finite, "n": int(err.size), "max_ulp": max_ulp, "c_dtype": c_dtype, "argmax": np.unravel_index(int(np.argmax(err / tol)), err.shape) if err.size else None}


def check_blocks(w: wl.Workload, inputs: dict, cbits: np.ndarray, blocks, c_dtype=None) -> list:
    """blocks: list of (batches, rows, cols) index arrays.  Returns one report per block."""
    cd = w.c_dtype if c_dtype is None else c_dtype
    p = problem_of(w, cd)
    cin = c_in_as(inputs, w, cd)
    reports = []
    for batches, rows, cols in blocks:
        y, bound = oracle.gemm(p, inputs["A"], inputs["B"], C_in=cin, bias=inputs["bias"], alpha=w.alpha, beta=w.beta,
                               batches=batches, rows=rows, cols=cols)
        got_bits = gather(cbits, w, batches, rows, cols)
        if not w.d_tri:
            reports.append(compare_block(got_bits, y, bound, cd))
            reports[-1]["transcendental"] = w.epilogue >= 4
            continue
        # one triangle of D wanted: its elements are held to the usual bars; every other element must either be
        # untouched (still the NaN poison, or C_in when beta != 0) or hold its value of the plain product
        keep = np.broadcast_to(oracle.wanted(rows, cols, w.d_tri)[None, :, :], y.shape)
        rep = compare_block(got_bits[keep], y[keep], bound[keep], cd)
        out_bits, out_y, out_bound = got_bits[~keep], y[~keep], bound[~keep]
        out_val = oracle.decode(out_bits, cd)
        untouched = np.isnan(out_val) if cin is None else out_bits == gather(cin, w, batches, rows, cols)[~keep]
        with np.errstate(invalid="ignore"):
            plain = np.abs(out_val - out_y) <= REL_TOL * out_bound + ABS_TOL + U_OUT[cd] * np.abs(out_y)
        if w.d_mirror:   # symmetric result: every other element holds the bits of its mirror image
            image = np.swapaxes(gather(cbits, w, batches, cols, rows), 1, 2)
            rep["outside_ok"] = bool(np.array_equal(out_bits, image[~keep]))
            rep["outside_untouched"], rep["outside_n"], rep["transcendental"] = 0, int(out_bits.size), w.epilogue >= 4
            reports.append(rep)
            continue
        rep["outside_ok"] = bool(np.all(untouched | plain))
        rep["outside_untouched"] = int(np.sum(untouched))
        rep["outside_n"] = int(untouched.size)
        rep["transcendental"] = w.epilogue >= 4
        reports.append(rep)
    return reports


def default_blocks(w: wl.Workload) -> list:
    """Everything for small problems; seeded rows x all columns and all rows x seeded columns
    (plus whole batches where the config asks) for the large ones."""
    allb = np.arange(w.batch, dtype=np.int64)
    allr = np.arange(w.M, dtype=np.int64)
    allc = np.arange(w.N, dtype=np.int64)
    if not w.sample_rows and not w.sample_cols:
        return [(allb, allr, allc)]
    blocks = []
    if w.full_batches:
        fb = sorted(set([0, w.batch - 1] + wl.sample_indices(w.batch, w.full_batches, w.seed, 3)[:w.full_batches].tolist()))
        fb = fb[:max(w.full_batches, 2)]
        blocks.append((np.array(fb, dtype=np.int64), allr, allc))
    rows = wl.sample_indices(w.M, w.sample_rows, w.seed, 1)
    cols = wl.sample_indices(w.N, w.sample_cols, w.seed, 2)
    blocks.append((allb, rows, allc))
    blocks.append((allb, allr, cols))
    return blocks


def assert_reports(reports, what=""):
    for r in reports:
        assert r["finite"], f"{what}: non-finite output {r}"
        assert r.get("outside_ok", True), f"{what}: an element outside the wanted triangle is neither untouched nor right {r}"
        assert r["max_err_over_tol"] <= 1.0, f"{what}: per-element tolerance exceeded {r}"
        assert r["frob"] <= frob_tol_for(r["c_dtype"]), f"{what}: Frobenius error {r}"
        if r["c_dtype"] != wl.F32:
            assert r["max_ulp"] <= 1, f"{what}: more than one ulp from the rounded oracle {r}"
            floor = 0.99 - (2.0 * D_ACT / U_OUT[r["c_dtype"]] if r.get("transcendental") else 0.0)
            assert r["bit_identical"] >= floor, f"{what}: too many one-ulp flips {r}"


def assert_padding_untouched(w: wl.Workload, inputs: dict, cbits: np.ndarray, c_dtype=None):
    """Everything in the C buffer that is not an element of D -- the row padding behind column N - 1 when ldc > N, the
    gaps between batches -- must still hold what it held before the run (C_in, or the NaN poison).  A matrix that is a
    column block of a larger one has its neighbours' data there."""
    cd = w.c_dtype if c_dtype is None else c_dtype
    if w.elems_c() == w.batch * w.M * w.N:
        return
    mask = np.ones(w.elems_c(), bool)
    for b in range(w.batch):
        idx = b * w.stride_c + np.arange(w.M, dtype=np.int64)[:, None] * w.ldc + np.arange(w.N, dtype=np.int64)[None, :]
        mask[idx.ravel()] = False
    cin = c_in_as(inputs, w, cd)
    if cin is not None:
        assert np.array_equal(cbits[mask], cin[mask]), f"{w.name}: bytes outside D were overwritten"
    else:
        assert np.all(np.isnan(oracle.decode(cbits[mask].copy(), cd))), f"{w.name}: bytes outside D were overwritten"


def check_workload(w: wl.Workload, flags: int = 0, exact: bool = False, c_dtype=None, repeats: int = 1, inputs=None, options: int = 0):
    """Run + compare.  exact=True additionally requires bit equality with the rounded oracle
    (for integer-valued inputs whose every partial sum is exactly representable)."""
    inputs = wl.make_inputs(w) if inputs is None else inputs
    cbits, info = run_gpu(w, inputs, flags, c_dtype, repeats=repeats, options=options)
    reports = check_blocks(w, inputs, cbits, default_blocks(w), c_dtype)
    assert_reports(reports, what=w.name)
    assert_padding_untouched(w, inputs, cbits, c_dtype)
    if exact:
        for r in reports:
            assert r["bit_identical"] == 1.0, f"{w.name}: not bit-exact {r} {info}"
    return reports, info
