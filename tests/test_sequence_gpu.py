"""Parity of dvp_sequence_aggregate with the oracle: sums within 1e-4 + 1e-6 sum|r|
(float32 inputs summed in double on both sides), counts, minima, infinities and
veto flags exact."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2512_23087_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _compare(lr, off, thr):
    got = binding.dvp_sequence_aggregate(lr, off, thr)
    torch.cuda.synchronize()
    want = oracle.dvp_sequences(lr.cpu().numpy().astype(np.float64), off.cpu().numpy(), thr)
    g = got.seq_log_ratio.cpu().numpy().astype(np.float64)
    assert np.array_equal(np.isposinf(g), np.isposinf(want.seq_log_ratio))
    assert np.array_equal(np.isneginf(g), np.isneginf(want.seq_log_ratio))
    fin = np.isfinite(want.seq_log_ratio)
    lrn = np.nan_to_num(lr.cpu().numpy().astype(np.float64), nan=0.0, posinf=0.0, neginf=0.0)
    mass = np.array([np.abs(lrn[a:b]).sum() for a, b in zip(off.cpu().numpy()[:-1], off.cpu().numpy()[1:])])
    assert (np.abs(g[fin] - want.seq_log_ratio[fin]) <= 1e-4 + 1e-6 * mass[fin]).all()
    assert np.array_equal(got.min_log_ratio.cpu().numpy().astype(np.float64), want.min_log_ratio)
    assert np.array_equal(got.n_valid.cpu().numpy(), want.n_valid)
    assert np.array_equal(got.n_zero_weight.cpu().numpy(), want.n_zero_weight)
    assert np.array_equal(got.veto.cpu().numpy(), want.veto)
    return got, want


def test_sequences_of_a_forward_pass():
    """64 sequences of ragged length over the per-token log-ratios of a real forward."""
    w = inputs.WORKLOADS["c2_bf16_fwdbwd"]
    batch = inputs.make_rows(w, seed=5, device=DEV, T=4096, V=8192)
    res = binding.dvp_forward(batch.train, batch.ids, 1e-3, infer_logits=batch.infer)
    g = torch.Generator().manual_seed(1)
    cuts = torch.sort(torch.randint(0, 4097, (63,), generator=g)).values
    off = torch.cat([torch.tensor([0]), cuts, torch.tensor([4096])]).to(DEV)
    got, want = _compare(res.log_ratio, off, 1e-4)
    assert want.veto.sum() >= 1 and (want.veto == 0).sum() >= 1


def test_coverage_minimum_and_mean_per_sequence():
    """Z_min and mean Z over each sequence (Def. 5.2; Prop. 5.5's bound uses Z_min) from the
    per-token ln Z of a forward pass, against the oracle's ln Z and its coverage statistics."""
    w = inputs.WORKLOADS["c2_bf16_fwdbwd"]
    batch = inputs.make_rows(w, seed=6, device=DEV, T=3000, V=8192)
    batch.ids[7] = -1                                  # a state without a sampled token still counts
    res = binding.dvp_forward(batch.train, batch.ids, 1e-3, infer_logits=batch.infer)
    off = torch.tensor([0, 0, 1, 700, 3000, 3000], device=DEV)
    got = binding.dvp_sequence_aggregate(res.log_ratio, off, 1e-4, log_cov=res.train.log_cov)
    torch.cuda.synchronize()
    import parity
    want_rows = parity.run_oracle(batch.train, batch.infer, batch.ids, 1e-3)
    lo, mean = oracle.dvp_coverage(want_rows.train.log_cov, off.cpu().numpy())
    g_lo, g_mean = got.min_cov.cpu().numpy().astype(np.float64), got.mean_cov.cpu().numpy().astype(np.float64)
    assert np.isposinf(g_lo[[0, 4]]).all() and np.isnan(g_mean[[0, 4]]).all()
    np.testing.assert_allclose(g_lo[1:4], lo[1:4], atol=1e-4, rtol=0)
    np.testing.assert_allclose(g_mean[1:4], mean[1:4], atol=1e-4, rtol=0)
    assert (g_lo[1:4] <= g_mean[1:4] + 1e-7).all() and (g_mean[1:4] <= 1.0).all() and g_lo[3] < 1.0
    # the other outputs do not change when the coverage is asked for
    plain = binding.dvp_sequence_aggregate(res.log_ratio, off, 1e-4)
    assert torch.equal(plain.veto, got.veto) and torch.equal(plain.n_valid, got.n_valid)
    with pytest.raises(binding.DvpError):              # coverage outputs without the input
        a = binding.SequenceArgs()
        import ctypes
        a.struct_size = ctypes.sizeof(binding.SequenceArgs)
        a.T, a.S = 8, 1
        a.seq_offsets, a.log_ratio, a.min_cov = off.data_ptr(), res.log_ratio.data_ptr(), got.min_cov.data_ptr()
        st = binding.load_library().dvp_sequence_aggregate(ctypes.byref(a))
        if st != binding.DVP_OK:
            raise binding.DvpError(st, "dvp_sequence_aggregate")


def test_special_values_empty_and_long_sequences():
    T = 40000
    g = torch.Generator().manual_seed(2)
    lr = (torch.randn(T, generator=g) * 0.05)
    lr[5] = float("nan")
    lr[100] = -math.inf
    lr[200] = math.inf
    lr[300] = math.log(0.99e-4)
    lr[400] = math.log(1.01e-4)
    lr[20000] = -math.inf
    lr[20001] = math.inf
    off = torch.tensor([0, 0, 50, 150, 250, 350, 450, 19000, 40000, 40000])
    for thr in (1e-4, 0.0, 0.5):
        _compare(lr.to(DEV), off.to(DEV), thr)
    got, _ = _compare(lr.to(DEV), off.to(DEV), 1e-4)
    assert got.veto.tolist() == [0, 0, 1, 0, 1, 0, 0, 1, 0]
    assert got.n_valid.tolist()[1] == 49


def test_sequence_argument_errors():
    lr = torch.zeros(8, device=DEV)
    off = torch.tensor([0, 8], device=DEV)
    with pytest.raises(binding.DvpError):
        binding.dvp_sequence_aggregate(lr, off, -1.0)
    with pytest.raises(binding.DvpError):
        binding.dvp_sequence_aggregate(lr, off, float("nan"))
