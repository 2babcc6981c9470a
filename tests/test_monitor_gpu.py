"""Parity of dvp_monitor with the oracle: entropies within 1e-4 nats, divergences
within 5e-6 + 1e-3 of their value (they are small differences of fp32 sums)."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2512_23087_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("dtype,V,ld,sigma", [("bf16", 151936, 151936, 0.02), ("f32", 40000, 40000, 0.05),
                                              ("f16", 4099, 4112, 0.3), ("bf16", 1003, 1003, 0.02),
                                              ("f32", 7, 8, 0.5)])
def test_monitor_matches_the_oracle(dtype, V, ld, sigma):
    w = dataclasses.replace(inputs.WORKLOADS["c2_bf16_fwdbwd"], dtype=dtype, infer_sigma=sigma)
    batch = inputs.make_rows(w, seed=V + 1, device=DEV, T=20, V=V, ld=ld)
    got = binding.dvp_monitor(batch.train, batch.infer)
    torch.cuda.synchronize()
    want = oracle.dvp_monitor(batch.train.cpu().double().numpy(), batch.infer.cpu().double().numpy())
    for i, name in enumerate(("kl_infer_train", "kl_train_infer")):
        g = getattr(got, name).cpu().numpy().astype(np.float64)
        assert (np.abs(g - want[:, i]) <= 5e-6 + 1e-3 * want[:, i]).all(), (name, g, want[:, i])
    for i, name in ((2, "entropy_train"), (3, "entropy_infer")):
        g = getattr(got, name).cpu().numpy().astype(np.float64)
        assert np.abs(g - want[:, i]).max() <= 1e-4, name


def test_monitor_identical_rows_and_errors():
    z = torch.randn(5, 3000, device=DEV) * 4
    got = binding.dvp_monitor(z, z.clone())
    torch.cuda.synchronize()
    assert got.kl_infer_train.abs().max().item() <= 1e-6 and got.kl_train_infer.abs().max().item() <= 1e-6
    assert torch.equal(got.entropy_train, got.entropy_infer)
    with pytest.raises(ValueError):
        binding.dvp_monitor(z, z[:, :100])
