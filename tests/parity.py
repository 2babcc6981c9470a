"""Comparison of the CUDA library's outputs with the fp64 oracle.

Tolerances (stated once, used by every parity test):
  * row max, safe-set size, membership flags, packed mask: bit-exact on every
    row.  Rows that hold a logit within 1e-6 relative of the threshold are
    counted and reported, but they get no allowance: the library decides
    membership exactly as the double comparison does, so none is needed;
  * log-probabilities (logp, logp_mp, log_ratio): 1e-4 absolute, infinities
    and NaNs must coincide;
  * lse, lse_safe: 1e-4 absolute plus one float32 rounding of the value (they
    are float32 outputs whose magnitude can reach the hundreds);
  * log_cov = ln Z: 1e-4 absolute, never positive, and the pruned mass 1 - Z
    (the total variation distance of the proof of Prop. 5.5) within 1e-3 relative
    plus 2e-5: Z is a ratio of two float32 sums of up to 2^18 exponentials, whose
    per-thread chains (a few thousand additions with 64-thread blocks) leave
    relative errors of up to about 1e-5 on each sum;
  * importance weights (weight_kind): 2e-4 relative (two log-probabilities of
    1e-4 each in the exponent), infinities and NaNs must coincide; rows whose
    ratio lies within 5e-4 relative of a masking bound, where the weight jumps,
    are counted and left out of the weight and gradient comparison;
  * gradients: per row, ||G - G_oracle||_2 <= (1e-3 + u) ||G_oracle||_2 with u
    the unit roundoff of the gradient's storage type (0 for float32, 2^-8 for
    bfloat16, 2^-11 for float16): round-to-nearest storage alone contributes
    up to u (errors below half the spacing of the storage type's subnormals are
    not counted).  Rows where both are zero pass.  In addition every element must
    sit within (1e-3 + u) |G_oracle| + a of the oracle's element, a being half
    the spacing of the storage type's subnormals (2^-25 for float16) or 1e-30.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle

LOGP_TOL = 1e-4
GRAD_TOL = 1e-3
UNIT_ROUNDOFF = {torch.float32: 0.0, torch.bfloat16: 2.0 ** -8, torch.float16: 2.0 ** -11}
SUBNORMAL_HALF_STEP = {torch.float32: 1e-30, torch.bfloat16: 1e-30, torch.float16: 2.0 ** -25}
ORACLE_DTYPE = {torch.float32: oracle.F32, torch.bfloat16: oracle.BF16, torch.float16: oracle.F16}


def to_oracle_storage(x: torch.Tensor) -> np.ndarray:
    """Host copy of stored logits in the form the oracle reads (same bits)."""
    x = x.detach().cpu()
    if x.dtype == torch.float32:
        return x.numpy()
    return x.view(torch.int16).numpy().view(np.uint16)


def run_oracle(train, infer, ids, rho, upstream=None, want_mask=False, threads=8, weight=None):
    kw = {} if weight is None else dict(weight_kind=weight[0], weight_lo=weight[1], weight_hi=weight[2])
    return oracle.dvp_rows(
        to_oracle_storage(train), ids.detach().cpu().numpy().astype(np.int64), rho,
        dtype=ORACLE_DTYPE[train.dtype],
        infer=to_oracle_storage(infer) if infer is not None else None,
        upstream=upstream.detach().cpu().numpy().astype(np.float64) if upstream is not None else None,
        want_grad=upstream is not None, want_mask=want_mask, threads=threads, **kw)


def near_threshold_rows(stored: torch.Tensor, side) -> np.ndarray:
    """Rows that hold a logit within 1e-6 relative of the threshold."""
    z = stored.detach().cpu().to(torch.float64).numpy()
    tau = side.tau[:, None]
    with np.errstate(invalid="ignore"):
        close = np.abs(z - tau) <= 1e-6 * np.abs(tau)
    return close.any(axis=1)


def _same_special(got: np.ndarray, want: np.ndarray, name: str):
    assert np.array_equal(np.isnan(got), np.isnan(want)), f"{name}: NaN pattern differs"
    assert np.array_equal(np.isposinf(got), np.isposinf(want)), f"{name}: +inf pattern differs"
    assert np.array_equal(np.isneginf(got), np.isneginf(want)), f"{name}: -inf pattern differs"


def _close(got, want, tol, name, rows=None):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    if rows is not None:
        got, want = got[rows], want[rows]
    _same_special(got, want, name)
    fin = np.isfinite(want)
    err = np.abs(got[fin] - want[fin])
    bound = tol(want[fin]) if callable(tol) else tol
    worst = float((err - bound).max()) if err.size else -1.0
    assert worst <= 0, f"{name}: max error {err.max():.3e} beyond tolerance"
    return float(err.max()) if err.size else 0.0


def unpack_mask(mask: torch.Tensor, V: int) -> np.ndarray:
    words = mask.detach().cpu().numpy().view(np.uint32)
    bits = np.unpackbits(words.view(np.uint8), axis=1, bitorder="little")
    assert not bits[:, V:].any(), "padding bits of the packed mask must be zero"
    return bits[:, :V]


def check_side(got, want, stored, V, label, report):
    """got: namespace of device tensors; want: oracle.Side."""
    near = near_threshold_rows(stored, want)
    ok = np.ones_like(near)
    report[f"{label}_near_threshold_rows"] = int(near.sum())
    assert np.array_equal(got.max.cpu().numpy().astype(np.float64), want.max), f"{label}.max"
    cnt = got.count.cpu().numpy().astype(np.int64)
    assert np.array_equal(cnt[ok], want.count[ok]), f"{label}.count"
    report[f"{label}_count_mismatch_near"] = int((cnt[near] != want.count[near]).sum())
    lse_tol = lambda w: LOGP_TOL + 2.0 ** -23 * np.abs(w)
    report[f"{label}_lse_err"] = _close(got.lse.cpu(), want.lse, lse_tol, f"{label}.lse")
    report[f"{label}_lse_safe_err"] = _close(got.lse_safe.cpu(), want.lse_safe, lse_tol,
                                             f"{label}.lse_safe", ok)
    report[f"{label}_logp_err"] = _close(got.logp.cpu(), want.logp, LOGP_TOL, f"{label}.logp")
    report[f"{label}_logp_mp_err"] = _close(got.logp_mp.cpu(), want.logp_mp, LOGP_TOL,
                                            f"{label}.logp_mp", ok)
    comp_want = np.where(want.member == 1, want.sum_safe_x / want.sum_safe, 1.0)
    comp_want = np.where(np.isnan(want.logp), np.nan, comp_want)
    _close(got.comp_mp.cpu(), comp_want, lambda w: 1e-6 + 1e-4 * np.abs(w), f"{label}.comp_mp", ok)
    # coverage: ln Z within 1e-4, and the pruned mass 1 - Z within 1e-3 relative plus the 2e-5
    # that float32 sums of up to 2^18 terms leave on Z itself
    lc = got.log_cov.cpu().numpy().astype(np.float64)
    assert (lc <= 0).all(), f"{label}.log_cov must not be positive"
    report[f"{label}_log_cov_err"] = _close(lc, want.log_cov, LOGP_TOL, f"{label}.log_cov", ok)
    pruned_got, pruned_want = -np.expm1(lc[ok]), -np.expm1(want.log_cov[ok])
    assert (np.abs(pruned_got - pruned_want) <= 1e-3 * pruned_want + 2e-5).all(), f"{label}: 1 - Z"
    if got.mask is not None and want.mask is not None:
        bits = unpack_mask(got.mask, V)
        assert np.array_equal(bits[ok], want.mask[ok]), f"{label}.mask"


def check_flags(flags: torch.Tensor, res, ids: np.ndarray, V: int, ok_rows=None):
    f = flags.cpu().numpy()
    want = (res.train.member.astype(np.uint8) * 1)
    if res.infer is not None:
        want = want | (res.infer.member.astype(np.uint8) * 2)
    want = want | np.where(ids < 0, 64, 0).astype(np.uint8) | np.where(ids >= V, 128, 0).astype(np.uint8)
    if ok_rows is None:
        ok_rows = np.ones(len(f), dtype=bool)
    assert np.array_equal(f[ok_rows], want[ok_rows]), "flags"


def check_grad(grad: torch.Tensor, want: np.ndarray, report, rows=None, label="grad"):
    u = UNIT_ROUNDOFF[grad.dtype]
    got = grad.detach().cpu().to(torch.float64).numpy()
    if rows is not None:
        got, want = got[rows], want[rows]
    assert np.isfinite(got).all(), "gradient holds a non-finite value"
    err = got - want
    floor = SUBNORMAL_HALF_STEP[grad.dtype]
    excess = np.maximum(np.abs(err) - floor, 0.0)      # what the storage grid cannot hold is not an error
    num = np.sqrt((excess * excess).sum(axis=1))
    den = np.sqrt((want * want).sum(axis=1))
    both_zero = (den == 0) & (np.abs(got).sum(axis=1) == 0)
    rel = np.where(both_zero, 0.0, num / np.maximum(den, 1e-300))
    assert (rel <= GRAD_TOL + u).all(), f"{label}: worst row relative L2 {rel.max():.3e}"
    assert (np.abs(err) <= (GRAD_TOL + u) * np.abs(want) + floor).all(), f"{label}: element bound"
    assert ((want == 0) <= (got == 0)).all(), f"{label}: pruned entries must be exactly zero"
    report[f"{label}_worst_row_rel_l2"] = float(rel.max()) if rel.size else 0.0
    report[f"{label}_frac_rows_above_1e-3"] = float((rel > GRAD_TOL).mean()) if rel.size else 0.0
    report[f"{label}_zero_rows"] = int(both_zero.sum())


def check_forward(res_gpu, batch, rho, V, want_grad, report=None, threads=8):
    """Full element-by-element comparison of one dvp_forward result."""
    report = {} if report is None else report
    want = run_oracle(batch.train, batch.infer, batch.ids, rho,
                      upstream=batch.upstream if want_grad else None,
                      want_mask=res_gpu.train.mask is not None, threads=threads)
    check_side(res_gpu.train, want.train, batch.train, V, "train", report)
    near = near_threshold_rows(batch.train, want.train)
    if want.infer is not None:
        check_side(res_gpu.infer, want.infer, batch.infer, V, "infer", report)
        near = near | near_threshold_rows(batch.infer, want.infer)
        report["log_ratio_err"] = _close(res_gpu.log_ratio.cpu(), want.log_ratio, LOGP_TOL,
                                         "log_ratio")
    report["near_threshold_rows"] = int(near.sum())
    check_flags(res_gpu.flags, want, batch.ids.cpu().numpy(), V)
    if want_grad:
        check_grad(res_gpu.grad_train, want.grad, report)
    report["mean_safe_set_size"] = float(want.train.count.mean())
    report["frac_sampled_in_train_set"] = float(want.train.member.mean())
    return report, want


def check_weighted(res_gpu, batch, rho, V, weight, report=None, threads=8):
    """dvp_forward with an in-kernel importance weight against the oracle's weighted gradient."""
    report = {} if report is None else report
    kind, lo, hi = weight
    want = run_oracle(batch.train, batch.infer, batch.ids, rho, upstream=batch.upstream, threads=threads,
                      weight=weight)
    ratio = np.exp(want.log_ratio)
    near = np.zeros(len(ratio), dtype=bool)
    if kind == oracle.WEIGHT_MASK:
        with np.errstate(invalid="ignore"):
            near = (np.abs(ratio - lo) <= 5e-4 * lo) | (np.abs(ratio - hi) <= 5e-4 * hi)
    ok = ~near
    report["near_weight_bound_rows"] = int(near.sum())
    report["weight_err"] = _close(res_gpu.weight.cpu(), want.weight, lambda w: 2e-4 * np.abs(w), "weight", ok)
    # an unbounded plain ratio (token pruned on the inference side only) has no finite gradient row
    unbounded = np.isinf(want.weight)
    report["unbounded_weight_rows"] = int(unbounded.sum())
    ok = ok & ~unbounded
    check_grad(res_gpu.grad_train, want.grad, report, rows=ok, label="weighted_grad")
    report["zero_weight_rows"] = int((want.weight[ok] == 0).sum())
    report["live_rows"] = int(((want.weight[ok] != 0) & (want.train.member[ok] == 1)).sum())
    return report, want
