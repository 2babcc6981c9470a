"""Token-level importance weights applied to the upstream gradient inside
dvp_forward (Thm. 5.3 per token, App. A protocol 4), against the fp64 oracle."""
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
KINDS = [(oracle.WEIGHT_RATIO, 0.0, math.inf), (oracle.WEIGHT_TRUNCATE, 0.0, 1.02), (oracle.WEIGHT_MASK, 0.97, 1.03)]
assert (binding.DVP_WEIGHT_RATIO, binding.DVP_WEIGHT_TRUNCATE, binding.DVP_WEIGHT_MASK) == \
    (oracle.WEIGHT_RATIO, oracle.WEIGHT_TRUNCATE, oracle.WEIGHT_MASK)


def _forward(batch, rho, weight, **kw):
    res = binding.dvp_forward(batch.train, batch.ids, rho, infer_logits=batch.infer, upstream=batch.upstream,
                              weight_kind=weight[0], weight_lo=weight[1], weight_hi=weight[2], **kw)
    assert binding.dvp_row_wait_status() == 0
    return res


@pytest.mark.parametrize("hint", [0, 0x11 << 16], ids=["streaming", "resident"])
@pytest.mark.parametrize("weight", KINDS, ids=["ratio", "truncate", "mask"])
def test_bf16_full_vocabulary_rows(weight, hint):
    w = W["c2_bf16_fwdbwd"]
    batch = inputs.make_rows(w, seed=5, device=DEV, T=160)
    rho = 1e-3
    res = _forward(batch, rho, weight, launch_hint=hint)
    report, want = parity.check_weighted(res, batch, rho, w.V, weight)
    assert report["live_rows"] >= 40
    if weight[0] == oracle.WEIGHT_MASK:
        assert report["zero_weight_rows"] > report["live_rows"] // 50      # the bounds do cut
    # the other outputs are those of the unweighted call
    plain = binding.dvp_forward(batch.train, batch.ids, rho, infer_logits=batch.infer, upstream=batch.upstream,
                                launch_hint=hint)
    assert torch.equal(plain.train.logp_mp, res.train.logp_mp) and torch.equal(plain.infer.logp_mp, res.infer.logp_mp)
    assert torch.equal(plain.log_ratio.isnan(), res.log_ratio.isnan())
    assert torch.equal(plain.flags, res.flags) and torch.equal(plain.train.count, res.train.count)


@pytest.mark.parametrize("dtype,V,ld", [("f32", 4096, 4096), ("f16", 5000, 5008), ("bf16", 1003, 1003), ("f32", 999, 1001)])
@pytest.mark.parametrize("weight", KINDS, ids=["ratio", "truncate", "mask"])
def test_small_rows_vector_and_scalar_kernels(weight, dtype, V, ld):
    w = dataclasses.replace(W["c0_small_f32"], dtype=dtype, infer_sigma=0.03)
    batch = inputs.make_rows(w, seed=V, device=DEV, T=64, V=V, ld=ld)
    res = _forward(batch, 1e-2, weight)
    report, _ = parity.check_weighted(res, batch, 1e-2, V, weight)
    assert report["live_rows"] >= 20


def test_pruned_tokens_missing_ids_and_identical_policies():
    z = np.full((6, 512), -30.0, dtype=np.float32)
    z[:, 3] = 5.0
    z[:, 9] = 4.0
    zi = z.copy()
    zi[1, 9] = -30.0            # a = 9 is pruned on the inference side only: ratio +inf
    z[2, 9] = -30.0             # a = 9 is pruned on the training side: ratio zero
    zi[3, 9] = 4.5              # a plain ratio below one
    ids = np.array([3, 9, 9, 9, -1, 600])
    g = torch.ones(6, device=DEV)
    batch = inputs.RowBatch(torch.from_numpy(z).to(DEV), torch.from_numpy(zi).to(DEV),
                            torch.from_numpy(ids).to(DEV), g)
    for weight in [(oracle.WEIGHT_TRUNCATE, 0.0, 2.0), (oracle.WEIGHT_MASK, 0.5, 2.0)]:
        res = _forward(batch, 1e-3, weight)
        report, want = parity.check_weighted(res, batch, 1e-3, 512, weight)
        wt = res.weight.cpu().numpy()
        assert wt[0] == pytest.approx(1.0, rel=1e-6)
        assert wt[1] == (2.0 if weight[0] == oracle.WEIGHT_TRUNCATE else 0.0)
        assert wt[2] == 0.0 and res.grad_train[2].abs().max().item() == 0.0
        assert 0.5 < wt[3] < 1.0
        assert np.isnan(wt[4]) and np.isnan(wt[5])
        assert res.grad_train[4:].abs().max().item() == 0.0


def test_argument_errors():
    w = W["c0_small_f32"]
    batch = inputs.make_rows(w, seed=1, device=DEV, T=8)
    with pytest.raises(binding.DvpError):      # a weight needs the inference logits
        binding.dvp_forward(batch.train, batch.ids, 1e-3, upstream=batch.upstream, weight_kind=binding.DVP_WEIGHT_RATIO)
    with pytest.raises(binding.DvpError):      # and a gradient to apply it to
        binding.dvp_forward(batch.train, batch.ids, 1e-3, infer_logits=batch.infer, weight_kind=binding.DVP_WEIGHT_RATIO)
    with pytest.raises(binding.DvpError):      # bounds out of order
        binding.dvp_forward(batch.train, batch.ids, 1e-3, infer_logits=batch.infer, upstream=batch.upstream,
                            weight_kind=binding.DVP_WEIGHT_MASK, weight_lo=2.0, weight_hi=1.0)
    with pytest.raises(binding.DvpError):      # unknown kind
        binding.dvp_forward(batch.train, batch.ids, 1e-3, infer_logits=batch.infer, upstream=batch.upstream,
                            weight_kind=7)
