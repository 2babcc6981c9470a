"""Parity of the finite-mask-value mode (the App. A listing taken literally)
with its oracle: kept set and counts exact, log-probabilities within 1e-4,
gradients within (1e-3 + u) relative L2 per row as in the other parity tests."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2512_23087_b200 import binding, inputs

import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
CODE = {"f32": oracle.F32, "bf16": oracle.BF16, "f16": oracle.F16}


@pytest.mark.parametrize("dtype,V,ld", [("bf16", 151936, 151936), ("f32", 20000, 20000), ("f16", 4099, 4112),
                                        ("bf16", 1003, 1003)])
@pytest.mark.parametrize("in_dtype_threshold", [True, False])
def test_listing_mode_matches_its_oracle(dtype, V, ld, in_dtype_threshold):
    w = dataclasses.replace(inputs.WORKLOADS["c2_bf16_fwdbwd"], dtype=dtype)
    batch = inputs.make_rows(w, seed=V, device=DEV, T=24, V=V, ld=ld)
    rho, mv = 1e-3, -50.0
    res = binding.dvp_forward(batch.train, batch.ids, rho, infer_logits=batch.infer, upstream=batch.upstream,
                              mask_value=mv, threshold_in_logits_dtype=in_dtype_threshold)
    grad2 = binding.dvp_backward(batch.train, batch.ids, rho, batch.upstream, res, mask_value=mv,
                                 threshold_in_logits_dtype=in_dtype_threshold)
    torch.cuda.synchronize()
    ids = batch.ids.cpu().numpy()
    up = batch.upstream.cpu().numpy().astype(np.float64)
    sides = {}
    for name, logits, got in (("train", batch.train, res.train), ("infer", batch.infer, res.infer)):
        z = logits.cpu().to(torch.float64).numpy()
        out, grad, thr = oracle.dvp_rows_listing(z, ids, rho, mv, dtype=CODE[dtype],
                                                 upstream=up if name == "train" else None,
                                                 threshold_in_storage_type=in_dtype_threshold)
        sides[name] = (out, grad)
        assert np.array_equal(got.max.cpu().numpy().astype(np.float64), out["max"])
        assert np.array_equal(got.count.cpu().numpy(), out["count"])
        np.testing.assert_allclose(got.lse.cpu().numpy(), out["lse_full"], atol=1e-4, rtol=1e-7)
        np.testing.assert_allclose(got.lse_safe.cpu().numpy(), out["lse_masked"], atol=1e-4, rtol=1e-7)
        np.testing.assert_allclose(got.logp_mp.cpu().numpy(), out["logp_masked"], atol=1e-4, rtol=0)
        np.testing.assert_allclose(got.comp_mp.cpu().numpy(), out["comp"], atol=1e-6, rtol=1e-4)
    flags = res.flags.cpu().numpy()
    assert np.array_equal(flags & 1, sides["train"][0]["member"])
    assert np.array_equal((flags >> 1) & 1, sides["infer"][0]["member"])
    want_lr = sides["train"][0]["logp_masked"] - sides["infer"][0]["logp_masked"]
    np.testing.assert_allclose(res.log_ratio.cpu().numpy(), want_lr, atol=1e-4, rtol=0)
    rep = {}
    parity.check_grad(res.grad_train, sides["train"][1], rep, label="fused")
    parity.check_grad(grad2, sides["train"][1], rep, label="standalone")


def test_listing_mode_pruned_sampled_token_keeps_a_gradient():
    z = np.full((2, 512), 0.0, dtype=np.float32)
    z[:, 0] = 10.0
    z[:, 1] = 9.0
    z[:, 2] = -30.0
    ids = torch.tensor([2, 1], device=DEV)
    zt = torch.from_numpy(z).to(DEV)
    g = torch.tensor([1.5, -0.5], device=DEV)
    res = binding.dvp_forward(zt, ids, 1e-3, upstream=g, mask_value=-50.0)
    exact = binding.dvp_forward(zt, ids, 1e-3, upstream=g)
    torch.cuda.synchronize()
    assert res.flags.tolist()[0] & 1 == 0 and torch.isfinite(res.train.logp_mp[0])
    assert res.grad_train[0].abs().sum().item() > 0 and res.grad_train[0, 2].item() == 0.0
    assert torch.isneginf(exact.train.logp_mp[0]) and exact.grad_train[0].abs().sum().item() == 0.0
    out, grad, _ = oracle.dvp_rows_listing(z.astype(np.float64), ids.cpu().numpy(), 1e-3, -50.0,
                                           upstream=g.cpu().numpy().astype(np.float64),
                                           threshold_in_storage_type=False)
    parity.check_grad(res.grad_train, grad, {})
    with pytest.raises(binding.DvpError):
        binding.dvp_forward(zt, ids, 1e-3, mask_value=float("inf"))
