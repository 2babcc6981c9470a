"""Parity of the resident-row kernel (one block per row; the row, or its last 120 KB,
stays in shared memory between the sweeps, the rest is re-read through a small
ring) with the fp64 oracle, through the C ABI.  The kernel is selected with the
stage byte 0x11 of ``launch_hint``."""
import dataclasses
import math

import numpy as np
import pytest
import torch

from paper_2512_23087_b200 import binding, inputs

import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
W = inputs.WORKLOADS


RESIDENT = 0x11 << 16
SLOT = 30720         # bytes of one shared-memory slot (480 threads x 4 vectors x 16 bytes)


def _forward(batch, rho, backward, want_mask=True, grad_dtype=None, **kw):
    res = binding.dvp_forward(batch.train, batch.ids, rho, infer_logits=batch.infer,
                              upstream=batch.upstream if backward else None,
                              grad_dtype=grad_dtype, want_mask=want_mask, **kw)
    assert binding.dvp_row_wait_status() == 0
    return res


@pytest.mark.parametrize("rho", [1e-4, 1e-3])
def test_bf16_full_vocabulary_rows(rho):
    """V = 151,936 bf16 (304 KB) does not fit one SM: 4 slots (120 KB) stay resident, 6 are
    streamed once per sweep; more rows than blocks, so every block walks several
    tokens through its rings."""
    w = W["c2_bf16_fwdbwd"]
    batch = inputs.make_rows(w, seed=2, device=DEV, T=400)
    res = _forward(batch, rho, True, launch_hint=RESIDENT)
    report, want = parity.check_forward(res, batch, rho, w.V, True)
    assert report["mean_safe_set_size"] > 5


def test_fp32_heavy_tail_262144():
    """A 1 MiB fp32 row is too long for the resident kernel (64 slots at most): the
    hint falls back to the streaming kernel; a 400 KB fp32 row is served."""
    w = W["c3_f32_heavy"]
    batch = inputs.make_rows(w, seed=3, device=DEV, T=40, chunk_rows=8)
    res = _forward(batch, 1e-4, True, launch_hint=RESIDENT)
    report, want = parity.check_forward(res, batch, 1e-4, w.V, True)
    assert report["mean_safe_set_size"] < 50
    batch = inputs.make_rows(w, seed=4, device=DEV, T=40, V=100000, chunk_rows=8)
    res = _forward(batch, 1e-4, True, launch_hint=RESIDENT)
    parity.check_forward(res, batch, 1e-4, 100000, True)


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("slots,extra,pad", [(0, 8, 8), (0, 64, 0), (0, 1000, 8), (0, 1928, 0), (1, 0, 0), (1, 8, 8),
                                             (2, -8, 16), (4, 0, 0), (4, 8, 8), (5, 0, 16), (6, 8, 0), (7, 0, 8),
                                             (7, 16, 0), (8, -16, 16), (10, 8, 8), (16, 0, 0), (16, 8, 8)])
def test_slot_and_residency_boundaries(dtype, slots, extra, pad):
    """Row lengths around a slot (1920 vectors), around the longest row that is
    resident as a whole (4 slots), around the point where the streamed part wraps
    the stream ring (3 slots) and around the longest row the kernel takes (16
    slots; longer ones fall back to the streaming kernel); ragged last slots; rows
    of a few vectors; padded strides whose padding holds huge logits."""
    size = 4 if dtype == "f32" else 2
    V = slots * SLOT // size + extra
    w = dataclasses.replace(W["c0_small_f32"], dtype=dtype, head_boost=6.0)
    batch = inputs.make_rows(w, seed=V, device=DEV, T=37 if V < 50000 else 13, V=V, ld=V + pad)
    for rho in (1e-2, 1e-4):
        res = _forward(batch, rho, True, launch_hint=RESIDENT)
        parity.check_forward(res, batch, rho, V, True)


@pytest.mark.parametrize("grad_dtype", [torch.float32, torch.bfloat16, torch.float16])
@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_gradient_storage_types(dtype, grad_dtype):
    w = dataclasses.replace(W["c0_small_f32"], dtype=dtype)
    batch = inputs.make_rows(w, seed=11, device=DEV, T=33, V=5000)
    res = _forward(batch, 1e-3, True, grad_dtype=grad_dtype, launch_hint=RESIDENT)
    assert res.grad_train.dtype == grad_dtype
    parity.check_forward(res, batch, 1e-3, 5000, True)


def _manual_batch(z, zi, ids, g=None):
    z = torch.as_tensor(z, dtype=torch.float32, device=DEV)
    zi = z.clone() if zi is None else torch.as_tensor(zi, dtype=torch.float32, device=DEV)
    T = z.shape[0]
    g = torch.ones(T, device=DEV) if g is None else torch.as_tensor(g, dtype=torch.float32, device=DEV)
    return inputs.RowBatch(z, zi, torch.as_tensor(ids, dtype=torch.int64, device=DEV), g)


def test_degenerate_thresholds_ties_and_ids():
    rng = np.random.default_rng(5)
    V = 776
    z = (rng.normal(size=(8, V)) * 3).astype(np.float32)
    z[1, 100] = z[1, 700] = z[1].max() + 1.0          # exact tie for the maximum
    ids = [int(z[0].argmax()), 100, 5, 6, -1, V, V + 5, 8]
    batch = _manual_batch(z, z + 0.01, ids)
    for rho in (0.0, 1.0, 0.25):
        res = _forward(batch, rho, True, launch_hint=RESIDENT)
        parity.check_forward(res, batch, rho, V, True)
    res = _forward(batch, 0.0, True, launch_hint=RESIDENT)
    assert (res.train.count == V).all()
    res = _forward(batch, 1.0, True, launch_hint=RESIDENT)
    assert res.train.count.tolist()[:2] == [1, 2]
    assert res.train.logp_mp[1].item() == pytest.approx(-math.log(2.0), abs=1e-6)
    assert res.grad_train[0].abs().max().item() == 0.0   # single-element safe set
    flags = res.flags.cpu().numpy()
    assert flags[4] & binding.DVP_FLAG_NO_ID and flags[5] & binding.DVP_FLAG_BAD_ID
    assert res.grad_train[4:7].abs().max().item() == 0.0


def test_tie_exactly_at_the_threshold_is_kept():
    rho = 0.25
    z = np.full((2, 4096), -20.0, dtype=np.float32)
    z[:, 7] = 3.0
    tau = np.float32(3.0 + math.log(rho))              # not exact: place logits at fl(tau) and below
    up = np.nextafter(tau, np.float32(np.inf))
    z[0, 3000] = up
    z[1, 3000] = np.nextafter(tau, np.float32(-np.inf))
    batch = _manual_batch(z, None, [7, 7])
    res = _forward(batch, rho, True, launch_hint=RESIDENT)
    parity.check_forward(res, batch, rho, 4096, True)


def test_train_only_forward_only_and_modes():
    w = dataclasses.replace(W["c0_small_f32"], dtype="bf16")
    batch = inputs.make_rows(w, seed=21, device=DEV, T=50, V=20000)
    h = RESIDENT
    res = binding.dvp_forward(batch.train, batch.ids, 1e-3, launch_hint=h)          # train side only
    full = _forward(batch, 1e-3, False, launch_hint=h)                              # both, no gradient
    assert binding.dvp_row_wait_status() == 0
    assert torch.equal(res.train.logp_mp, full.train.logp_mp)
    parity.check_forward(full, batch, 1e-3, 20000, False)
    ref = binding.dvp_forward(batch.train, batch.ids, 1e-3, infer_logits=batch.infer, upstream=batch.upstream,
                              mask_value=-50.0, threshold_in_logits_dtype=True, launch_hint=256 | (2 << 16))
    got = binding.dvp_forward(batch.train, batch.ids, 1e-3, infer_logits=batch.infer, upstream=batch.upstream,
                              mask_value=-50.0, threshold_in_logits_dtype=True, launch_hint=h)
    assert binding.dvp_row_wait_status() == 0
    assert torch.equal(ref.train.count, got.train.count) and torch.equal(ref.flags, got.flags)
    assert (ref.train.logp_mp - got.train.logp_mp).abs().max().item() < 1e-5
    assert (ref.log_ratio - got.log_ratio).abs().max().item() < 1e-5
    num = (ref.grad_train.float() - got.grad_train.float()).norm(dim=1)
    den = ref.grad_train.float().norm(dim=1).clamp_min(1e-20)
    assert (num / den).max().item() < 2.0 ** -7


def test_reruns_are_bit_identical_and_agree_with_the_streaming_kernel():
    w = W["c2_bf16_fwdbwd"]
    batch = inputs.make_rows(w, seed=9, device=DEV, T=300, V=100000)
    runs = [_forward(batch, 1e-4, True, launch_hint=RESIDENT) for _ in range(2)]
    assert torch.equal(runs[0].grad_train, runs[1].grad_train)
    assert torch.equal(runs[0].train.lse_safe, runs[1].train.lse_safe)
    other = _forward(batch, 1e-4, True, launch_hint=256 | (2 << 16))
    assert torch.equal(other.train.count, runs[0].train.count)
    assert torch.equal(other.train.mask, runs[0].train.mask)
    fin = torch.isfinite(other.train.logp_mp)
    assert torch.equal(fin, torch.isfinite(runs[0].train.logp_mp))
    assert (other.train.logp_mp[fin] - runs[0].train.logp_mp[fin]).abs().max().item() < 1e-5


def test_a_wait_that_runs_out_ends_the_launch_and_is_reported():
    """Stage byte 0x1e: block 0 of the resident-row kernel withholds its first bulk
    copy, so the consumers' wait for it reaches its limit (about a second).  The
    launch must end by itself, `dvp_row_wait_status` must report it once (code 1, a
    copy did not land, or code 2, the producer found no free slot behind the stuck
    consumers: whichever wait gives up first), and the next launch on the same
    context must be correct."""
    w = dataclasses.replace(W["c0_small_f32"], dtype="bf16")
    batch = inputs.make_rows(w, seed=31, device=DEV, T=300, V=40000)
    assert binding.dvp_row_wait_status() == 0
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    binding.dvp_forward(batch.train, batch.ids, 1e-3, infer_logits=batch.infer, upstream=batch.upstream,
                        launch_hint=0x1e << 16)
    t1.record()
    status = binding.dvp_row_wait_status()          # synchronises
    assert status in (1, 2, 3), status
    assert t0.elapsed_time(t1) < 20000.0             # it gave up, in seconds at most
    assert binding.dvp_row_wait_status() == 0        # the word is cleared by the read
    res = _forward(batch, 1e-3, True, launch_hint=RESIDENT)
    parity.check_forward(res, batch, 1e-3, 40000, True)
