"""Parity of the row kernel that keeps the candidates of the safe set on chip
(launch_hint stage byte 3 or 4; 2-byte logits) with the fp64 oracle, through the
C ABI.  Same tolerances as the other row tests (tests/parity.py)."""
import dataclasses
import math

import numpy as np
import pytest
import torch

from paper_2512_23087_b200 import binding, inputs

import oracle
import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
W = inputs.WORKLOADS
STORE3, STORE4 = 3 << 16, 4 << 16


def _forward(batch, rho, backward, hint, want_mask=True, grad_dtype=None, **kw):
    return binding.dvp_forward(batch.train, batch.ids, rho, infer_logits=batch.infer,
                               upstream=batch.upstream if backward else None,
                               grad_dtype=grad_dtype, want_mask=want_mask, launch_hint=hint, **kw)


@pytest.mark.parametrize("hint", [STORE3, STORE4], ids=["three_blocks", "four_blocks"])
@pytest.mark.parametrize("rho", [1e-4, 1e-3, 2.3e-6])
def test_bf16_full_vocabulary_rows(rho, hint):
    """V = 151,936 bf16: 19 steps of a 256-thread block, a ragged last step; light rows, rows
    whose lists fill before the head tokens are met, and (rho = e^-13) rows whose warps
    give their lists up."""
    w = W["c2_bf16_fwdbwd"]
    batch = inputs.make_rows(w, seed=2, device=DEV, T=96)
    res = _forward(batch, rho, True, hint)
    again = _forward(batch, rho, True, hint)
    plain = _forward(batch, rho, True, 0)
    torch.cuda.synchronize()
    report, want = parity.check_forward(res, batch, rho, w.V, True)
    assert report["mean_safe_set_size"] > 5
    # which warps keep their lists depends on timing; the results must not
    for name in ("max", "lse", "lse_safe", "logp", "logp_mp", "comp_mp", "count", "mask"):
        assert torch.equal(getattr(res.train, name), getattr(again.train, name)), name
        assert torch.equal(getattr(res.infer, name), getattr(again.infer, name)), name
    assert torch.equal(res.grad_train, again.grad_train)
    assert torch.equal(res.log_ratio.nan_to_num(), again.log_ratio.nan_to_num())
    # and the exact outputs agree with the default kernel's
    assert torch.equal(res.train.count, plain.train.count) and torch.equal(res.flags, plain.flags)


@pytest.mark.parametrize("hint", [STORE3, STORE4])
@pytest.mark.parametrize("dtype", ["bf16", "f16"])
@pytest.mark.parametrize("V,ld", [(1, 16), (7, 16), (1000, 1008), (1003, 1008), (4097, 4112), (33000, 33008),
                                  (999, 1001)])
def test_ragged_sizes_strides_and_alignment(dtype, V, ld, hint):
    """Short rows (the block shrinks), ragged last granules, padded strides whose padding
    must never be read; the unaligned layout takes the scalar kernel."""
    w = dataclasses.replace(W["c0_small_f32"], dtype=dtype, head_boost=6.0)
    batch = inputs.make_rows(w, seed=V, device=DEV, T=9, V=V, ld=ld)
    for rho in (1e-2, 1e-4, 0.0):
        res = _forward(batch, rho, True, hint)
        torch.cuda.synchronize()
        parity.check_forward(res, batch, rho, V, True)


@pytest.mark.parametrize("grad_dtype", [torch.float32, torch.bfloat16, torch.float16])
def test_gradient_storage_types(grad_dtype):
    w = dataclasses.replace(W["c0_small_f32"], dtype="bf16")
    batch = inputs.make_rows(w, seed=11, device=DEV, T=33, V=5000)
    res = _forward(batch, 1e-3, True, STORE3, grad_dtype=grad_dtype)
    torch.cuda.synchronize()
    assert res.grad_train.dtype == grad_dtype
    parity.check_forward(res, batch, 1e-3, 5000, True)


def _rows(z, zi, ids, g=None):
    z = torch.as_tensor(z, dtype=torch.float32, device=DEV).to(torch.bfloat16)
    zi = z.clone() if zi is None else torch.as_tensor(zi, dtype=torch.float32, device=DEV).to(torch.bfloat16)
    T = z.shape[0]
    g = torch.ones(T, device=DEV) if g is None else torch.as_tensor(g, dtype=torch.float32, device=DEV)
    return inputs.RowBatch(z, zi, torch.as_tensor(ids, dtype=torch.int64, device=DEV), g)


@pytest.mark.parametrize("hint", [STORE3, STORE4])
def test_rows_built_to_stress_the_running_bound(hint):
    """Row 0: logits rise along the row, so the bound keeps rising and earlier entries are
    dropped again and again; the sampled token is the lowest one.  Row 1: everything but the
    last element is a candidate until the very end (the only large logit comes last).
    Row 2: all equal (every token safe, lists overflow).  Row 3: the maximum comes first.
    Row 4: no sampled token.  Row 5: ties at the maximum in different warps' shares."""
    V = 40000
    rng = np.random.default_rng(0)
    z = np.zeros((6, V), dtype=np.float32)
    z[0] = np.linspace(-30.0, 30.0, V)
    z[1] = rng.normal(size=V) * 0.5
    z[1, V - 1] = 25.0
    z[2] = 0.75
    z[3] = rng.normal(size=V) * 2.0
    z[3, 0] = 22.0
    z[4] = rng.normal(size=V) * 3.0
    z[5] = rng.normal(size=V)
    z[5, [5, 9000, 21000, 39999]] = 12.0
    zi = z + rng.normal(size=z.shape).astype(np.float32) * 0.02
    ids = [0, 17, 5, 0, -1, 9000]
    batch = _rows(z, zi, ids, g=[1.0, -1.0, 2.0, 0.5, 1.0, -3.0])
    for rho in (1e-4, 1e-2, 0.5, 1.0):
        res = _forward(batch, rho, True, hint)
        torch.cuda.synchronize()
        report, want = parity.check_forward(res, batch, rho, V, True)
    assert res.train.count.tolist()[5] == 4 and res.train.count.tolist()[2] == V


@pytest.mark.parametrize("weight", [(oracle.WEIGHT_RATIO, 0.0, math.inf), (oracle.WEIGHT_TRUNCATE, 0.0, 1.02),
                                    (oracle.WEIGHT_MASK, 0.97, 1.03)], ids=["ratio", "truncate", "mask"])
def test_importance_weights_in_the_kernel(weight):
    """The weighted form sweeps the inference row first."""
    w = W["c2_bf16_fwdbwd"]
    batch = inputs.make_rows(w, seed=5, device=DEV, T=96)
    res = binding.dvp_forward(batch.train, batch.ids, 1e-3, infer_logits=batch.infer, upstream=batch.upstream,
                              weight_kind=weight[0], weight_lo=weight[1], weight_hi=weight[2], launch_hint=STORE3)
    torch.cuda.synchronize()
    report, want = parity.check_weighted(res, batch, 1e-3, w.V, weight)
    assert report["live_rows"] >= 20


@pytest.mark.parametrize("in_dtype_threshold", [True, False])
def test_finite_mask_value_mode(in_dtype_threshold):
    w = W["c2_bf16_fwdbwd"]
    batch = inputs.make_rows(w, seed=7, device=DEV, T=24)
    rho, mv = 1e-3, -50.0
    res = binding.dvp_forward(batch.train, batch.ids, rho, infer_logits=batch.infer, upstream=batch.upstream,
                              mask_value=mv, threshold_in_logits_dtype=in_dtype_threshold, launch_hint=STORE3)
    plain = binding.dvp_forward(batch.train, batch.ids, rho, infer_logits=batch.infer, upstream=batch.upstream,
                                mask_value=mv, threshold_in_logits_dtype=in_dtype_threshold)
    torch.cuda.synchronize()
    ids = batch.ids.cpu().numpy()
    up = batch.upstream.cpu().numpy().astype(np.float64)
    out, grad, thr = oracle.dvp_rows_listing(batch.train.cpu().to(torch.float64).numpy(), ids, rho, mv,
                                             dtype=oracle.BF16, upstream=up,
                                             threshold_in_storage_type=in_dtype_threshold)
    assert np.array_equal(res.train.count.cpu().numpy(), out["count"])
    np.testing.assert_allclose(res.train.lse_safe.cpu().numpy(), out["lse_masked"], atol=1e-4, rtol=1e-7)
    np.testing.assert_allclose(res.train.logp_mp.cpu().numpy(), out["logp_masked"], atol=1e-4, rtol=0)
    parity.check_grad(res.grad_train, grad, {}, label="listing")
    assert torch.equal(res.infer.count, plain.infer.count) and torch.equal(res.flags, plain.flags)


def test_hints_the_kernel_cannot_take_fall_back():
    """fp32 logits and unaligned rows take the other kernels, same results."""
    w = W["c0_small_f32"]
    batch = inputs.make_rows(w, seed=3, device=DEV, T=8)
    res = _forward(batch, 1e-3, True, STORE3)
    torch.cuda.synchronize()
    parity.check_forward(res, batch, 1e-3, w.V, True)
