"""Parity of the CUDA row kernels with the fp64 oracle, through the C ABI."""
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


def _forward(batch, rho, backward, want_mask=True, grad_dtype=None, **kw):
    return binding.dvp_forward(batch.train, batch.ids, rho, infer_logits=batch.infer,
                               upstream=batch.upstream if backward else None,
                               grad_dtype=grad_dtype, want_mask=want_mask, **kw)


def test_config0_small_fp32_forward_backward():
    w = W["c0_small_f32"]
    batch = inputs.make_rows(w, seed=1, device=DEV)
    res = _forward(batch, 1e-3, True)
    torch.cuda.synchronize()
    report, want = parity.check_forward(res, batch, 1e-3, w.V, True)
    assert report["train_near_threshold_rows"] == 0
    assert 1 <= report["mean_safe_set_size"] < 200


@pytest.mark.parametrize("cluster", [0, 2, 4])
@pytest.mark.parametrize("rho", [1e-4, 1e-3])
def test_bf16_full_vocabulary_rows(rho, cluster):
    """V = 151,936 bf16: several sweeps of a 256-thread block plus a ragged tail;
    one block per row, or a cluster of 2 or 4 blocks sharing each row."""
    w = W["c2_bf16_fwdbwd"]
    batch = inputs.make_rows(w, seed=2, device=DEV, T=96)
    res = _forward(batch, rho, True, launch_hint=(256 | (2 << 16) | (cluster << 24)) if cluster else 0)
    torch.cuda.synchronize()
    report, want = parity.check_forward(res, batch, rho, w.V, True)
    assert report["mean_safe_set_size"] > 5


@pytest.mark.parametrize("cluster", [0, 4])
def test_fp32_heavy_tail_262144(cluster):
    w = W["c3_f32_heavy"]
    batch = inputs.make_rows(w, seed=3, device=DEV, T=24, chunk_rows=8)
    res = _forward(batch, 1e-4, True, launch_hint=(256 | (2 << 16) | (cluster << 24)) if cluster else 0)
    torch.cuda.synchronize()
    report, want = parity.check_forward(res, batch, 1e-4, w.V, True)
    assert report["mean_safe_set_size"] < 50


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("V,ld", [(1, 8), (7, 8), (1000, 1000), (1003, 1008), (4097, 4104),
                                  (1003, 1003), (999, 1001), (33000, 33000)])
def test_ragged_sizes_strides_and_alignment(dtype, V, ld):
    """Row lengths that are not a multiple of the vector width, padded row
    strides (the padding holds huge logits that must never be read) and rows
    that do not start on 16-byte boundaries (scalar kernel)."""
    w = dataclasses.replace(W["c0_small_f32"], dtype=dtype, head_boost=6.0)
    batch = inputs.make_rows(w, seed=V, device=DEV, T=9, V=V, ld=ld)
    for rho in (1e-2, 1e-4):
        res = _forward(batch, rho, True)
        torch.cuda.synchronize()
        parity.check_forward(res, batch, rho, V, True)


@pytest.mark.parametrize("grad_dtype", [torch.float32, torch.bfloat16, torch.float16])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_gradient_storage_types(dtype, grad_dtype):
    w = dataclasses.replace(W["c0_small_f32"], dtype=dtype)
    batch = inputs.make_rows(w, seed=11, device=DEV, T=33, V=5000)
    res = _forward(batch, 1e-3, True, grad_dtype=grad_dtype)
    torch.cuda.synchronize()
    assert res.grad_train.dtype == grad_dtype
    parity.check_forward(res, batch, 1e-3, 5000, True)


def _manual_batch(z, zi, ids, g=None):
    z = torch.as_tensor(z, dtype=torch.float32, device=DEV)
    zi = z.clone() if zi is None else torch.as_tensor(zi, dtype=torch.float32, device=DEV)
    T = z.shape[0]
    g = torch.ones(T, device=DEV) if g is None else torch.as_tensor(g, dtype=torch.float32, device=DEV)
    return inputs.RowBatch(z, zi, torch.as_tensor(ids, dtype=torch.int64, device=DEV), g)


def test_degenerate_thresholds_rho_zero_and_one():
    rng = np.random.default_rng(5)
    z = (rng.normal(size=(6, 777)) * 3).astype(np.float32)
    z[1, 100] = z[1, 200] = z[1].max() + 1.0          # exact tie for the maximum
    ids = [int(z[0].argmax()), 100, 5, 6, 7, 8]
    batch = _manual_batch(z, z + 0.01, ids)
    for rho in (0.0, 1.0):
        res = _forward(batch, rho, True)
        torch.cuda.synchronize()
        parity.check_forward(res, batch, rho, 777, True)
    res = _forward(batch, 0.0, True)
    assert (res.train.count == 777).all()
    ref = torch.log_softmax(batch.train.double(), dim=-1)[torch.arange(6), batch.ids]
    assert (res.train.logp_mp.double() - ref).abs().max() < 1e-4
    res = _forward(batch, 1.0, True)
    assert res.train.count.tolist()[:2] == [1, 2]
    assert res.train.logp_mp[1].item() == pytest.approx(-math.log(2.0), abs=1e-6)
    assert res.grad_train[0].abs().max().item() == 0.0   # single-element safe set


def test_rho_zero_with_a_ragged_row_on_the_vector_path():
    """The fill of the ragged last granule must not be counted when every logit is safe."""
    w = dataclasses.replace(W["c0_small_f32"], dtype="bf16")
    batch = inputs.make_rows(w, seed=77, device=DEV, T=7, V=1003, ld=1008)
    for rho in (0.0, 1e-30):
        res = _forward(batch, rho, True)
        torch.cuda.synchronize()
        assert (res.train.count == 1003).all() and (res.infer.count == 1003).all()
        parity.check_forward(res, batch, rho, 1003, True)


def test_ties_at_the_threshold_are_kept():
    rho = 0.25
    L = math.log(rho)
    z = np.full((2, 64), -20.0, dtype=np.float32)
    z[:, 0] = 4.0
    tau = np.float32(np.float64(4.0) + L)
    tau_up = tau if np.float64(tau) >= 4.0 + L else np.nextafter(tau, np.float32(np.inf))
    z[0, 1] = tau_up                                   # smallest float >= threshold: kept
    z[0, 2] = np.nextafter(tau_up, np.float32(-np.inf))   # next float below: pruned
    z[1, 3] = tau_up
    batch = _manual_batch(z, None, [1, 2])
    res = _forward(batch, rho, True)
    torch.cuda.synchronize()
    assert res.train.count.tolist() == [2, 2]
    assert res.flags.tolist()[0] & 1 and not (res.flags.tolist()[1] & 1)
    want = parity.run_oracle(batch.train, batch.infer, batch.ids, rho, batch.upstream, True)
    assert np.array_equal(parity.unpack_mask(res.train.mask, 64), want.train.mask)
    assert want.train.count.tolist() == [2, 2]


def test_all_equal_row_huge_logits_and_sampled_token_outside_the_set():
    z = np.zeros((4, 300), dtype=np.float32)
    z[0, :] = 1.25                                     # all equal: everything is safe
    z[1, :] = np.linspace(-3.0e4, 3.0e4, 300)          # huge magnitudes
    z[2, :] = np.linspace(0, 30, 300)
    z[3, :] = np.linspace(0, 30, 300)
    ids = [17, 299, 0, 299]                            # row 2: sampled token is pruned
    zi = z.copy()
    zi[3, 299] = -50.0                                 # pruned on the inference side only
    batch = _manual_batch(z, zi, ids, g=[1.0, -2.0, 3.0, 0.5])
    res = _forward(batch, 1e-3, True)
    torch.cuda.synchronize()
    report, want = parity.check_forward(res, batch, 1e-3, 300, True)
    assert res.train.count[0].item() == 300
    assert res.log_ratio[2].item() == -math.inf and res.log_ratio[3].item() == math.inf
    assert res.grad_train[2].abs().max().item() == 0.0


def test_missing_and_out_of_range_ids_set_flags_and_never_trap():
    w = W["c0_small_f32"]
    batch = inputs.make_rows(w, seed=4, device=DEV, T=8, V=2048)
    batch.ids[1] = -1
    batch.ids[2] = 2048
    batch.ids[3] = 10 ** 12
    res = _forward(batch, 1e-3, True)
    torch.cuda.synchronize()
    flags = res.flags.tolist()
    assert flags[1] & binding.DVP_FLAG_NO_ID and flags[2] & binding.DVP_FLAG_BAD_ID
    assert flags[3] & binding.DVP_FLAG_BAD_ID
    assert torch.isnan(res.train.logp_mp[1:4]).all() and torch.isnan(res.log_ratio[1:4]).all()
    assert res.grad_train[1:4].abs().max().item() == 0.0
    assert (res.train.count[1:4] >= 1).all()
    parity.check_forward(res, batch, 1e-3, 2048, True)
    # int32 ids give the same result
    b32 = dataclasses.replace(batch, ids=batch.ids.clamp(max=2 ** 31 - 1).to(torch.int32))
    res32 = _forward(b32, 1e-3, True)
    torch.cuda.synchronize()
    assert torch.equal(res32.grad_train, res.grad_train)
    assert torch.equal(res32.flags, res.flags)


def test_train_only_and_forward_only_calls():
    w = W["c1_bf16_fwd"]
    batch = inputs.make_rows(w, seed=6, device=DEV, T=16, V=20000)
    res = binding.dvp_forward(batch.train, batch.ids, 1e-3, want_mask=True)
    torch.cuda.synchronize()
    assert res.infer is None and res.grad_train is None
    want = parity.run_oracle(batch.train, None, batch.ids, 1e-3, want_mask=True)
    rep = {}
    parity.check_side(res.train, want.train, batch.train, 20000, "train", rep)
    res2 = _forward(batch, 1e-3, False)
    torch.cuda.synchronize()
    parity.check_forward(res2, batch, 1e-3, 20000, False)


def test_standalone_backward_matches_fused_sweep_and_oracle():
    for name, V in (("c0_small_f32", 4096), ("c2_bf16_fwdbwd", 151936)):
        w = W[name]
        batch = inputs.make_rows(w, seed=8, device=DEV, T=40, V=V)
        fwd = _forward(batch, 1e-3, True, want_mask=False)
        grad = binding.dvp_backward(batch.train, batch.ids, 1e-3, batch.upstream, fwd)
        torch.cuda.synchronize()
        want = parity.run_oracle(batch.train, batch.infer, batch.ids, 1e-3, batch.upstream)
        rep = {}
        parity.check_grad(grad, want.grad, rep, label="standalone")
        parity.check_grad(fwd.grad_train, want.grad, rep, label="fused")
        # without the saved complement the a-th entry comes from 1 - exp(.)
        grad2 = binding.dvp_backward(batch.train, batch.ids, 1e-3, batch.upstream, fwd, use_comp=False)
        torch.cuda.synchronize()
        parity.check_grad(grad2, want.grad, rep, label="standalone_nocomp")
    # unaligned rows take the scalar map
    w = W["c0_small_f32"]
    batch = inputs.make_rows(w, seed=9, device=DEV, T=5, V=1001, ld=1003)
    fwd = _forward(batch, 1e-2, True)
    grad = binding.dvp_backward(batch.train, batch.ids, 1e-2, batch.upstream, fwd)
    torch.cuda.synchronize()
    want = parity.run_oracle(batch.train, batch.infer, batch.ids, 1e-2, batch.upstream)
    parity.check_grad(grad, want.grad, {})


def test_results_do_not_depend_on_launch_shape_and_are_reproducible():
    w = W["c2_bf16_fwdbwd"]
    batch = inputs.make_rows(w, seed=10, device=DEV, T=20, V=50000)
    base = _forward(batch, 1e-4, True)
    again = _forward(batch, 1e-4, True)
    torch.cuda.synchronize()
    for name in ("lse", "lse_safe", "logp_mp", "count"):
        assert torch.equal(getattr(base.train, name), getattr(again.train, name)), name
    assert torch.equal(base.grad_train, again.grad_train)
    want = parity.run_oracle(batch.train, batch.infer, batch.ids, 1e-4, batch.upstream)
    for threads in (64, 128, 512):
        for unroll in (0, 2):
            res = _forward(batch, 1e-4, True, launch_hint=threads | (unroll << 16))
            torch.cuda.synchronize()
            assert torch.equal(res.train.count, base.train.count)
            assert torch.equal(res.train.mask, base.train.mask)
            parity.check_grad(res.grad_train, want.grad, {})
            d = torch.nan_to_num(res.train.logp_mp, neginf=-1e30) - torch.nan_to_num(base.train.logp_mp, neginf=-1e30)
            assert d.abs().max().item() < 1e-5


def test_host_side_argument_errors():
    w = W["c0_small_f32"]
    batch = inputs.make_rows(w, seed=12, device=DEV, T=4, V=512)
    with pytest.raises(binding.DvpError) as e:
        binding.dvp_forward(batch.train, batch.ids, 1.5)
    assert e.value.status == binding.DVP_ERR_INVALID_ARG
    with pytest.raises(binding.DvpError):
        binding.dvp_forward(batch.train, batch.ids, float("nan"))
    with pytest.raises(binding.DvpError):
        binding.dvp_forward(batch.train, batch.ids, 1e-3, launch_hint=100)
    empty = binding.dvp_forward(batch.train[:0], batch.ids[:0], 1e-3)
    assert empty.train.max.numel() == 0


def test_bf16_logits_with_float32_gradients_at_full_row_length():
    """bf16 logits, V = 151,936, gradients stored in float32: nothing of the storage type's
    rounding is left in the bound, so the kernel's own arithmetic is held to the plain 1e-3
    relative L2 per row; the same rows with bf16 gradients are reported beside it."""
    w = W["c2_bf16_fwdbwd"]
    batch = inputs.make_rows(w, seed=21, device=DEV, T=128)
    for rho in (1e-4, 1e-3):
        res = _forward(batch, rho, True, grad_dtype=torch.float32)
        torch.cuda.synchronize()
        assert res.grad_train.dtype == torch.float32
        report, want = parity.check_forward(res, batch, rho, w.V, True)
        assert report["grad_worst_row_rel_l2"] <= 1e-3
        res16 = _forward(batch, rho, True)
        torch.cuda.synchronize()
        rep16 = {}
        parity.check_grad(res16.grad_train, want.grad, rep16)
        print(f"rho={rho}: fp32 gradients worst row {report['grad_worst_row_rel_l2']:.2e}; bf16 gradients worst row "
              f"{rep16['grad_worst_row_rel_l2']:.2e}, {rep16['grad_frac_rows_above_1e-3']:.3f} of the rows above 1e-3")


@pytest.mark.parametrize("grad_dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("sigma,rho", [(1.28, 1e-4), (1.28, 1e-3), (2.2, 1e-4)])
def test_rows_whose_safe_set_is_most_of_the_vocabulary(sigma, rho, grad_dtype):
    """bf16 rows of V = 151,936 without a dominant token (the logits a linear head gives for random
    hidden states): the threshold lies inside the bulk, the safe set holds from a tenth to nearly
    all of the tokens, most 32-byte pieces of a row are revisited and a warp's list of them
    overflows, so sweeps 2 and 3 walk every piece instead."""
    w = W["c2_bf16_fwdbwd"]
    batch = inputs.make_rows(w, seed=31, device=DEV, T=24)
    g = torch.Generator(device=DEV)
    g.manual_seed(32)
    train = (sigma * torch.randn(24, w.V, device=DEV, generator=g)).to(torch.bfloat16)
    infer = (train.float() + 0.02 * torch.randn(24, w.V, device=DEV, generator=g)).to(torch.bfloat16)
    ids = torch.multinomial(torch.softmax(infer.float(), dim=1), 1, generator=g).squeeze(1)  # a ~ softmax(z')
    batch = dataclasses.replace(batch, train=train, infer=infer, ids=ids)
    res = _forward(batch, rho, True, grad_dtype=grad_dtype)
    torch.cuda.synchronize()
    report, want = parity.check_forward(res, batch, rho, w.V, True)
    assert report["mean_safe_set_size"] > 0.1 * w.V
    assert report["grad_zero_rows"] < 24   # sampled tokens below the threshold give zero rows; not all are


@pytest.mark.parametrize("name,rho_index", [("c2_bf16_fwdbwd", 0), ("c2_bf16_fwdbwd", 1), ("c3_f32_heavy", 0)])
def test_full_size_sampled_rows_and_size_free_properties(name, rho_index):
    """The benchmark's own launch at its full size: rows sampled across the
    batch are compared with the oracle one by one, and properties that hold at
    any size are checked on every row."""
    w = W[name]
    free, _ = torch.cuda.mem_get_info()
    need = 3 * w.T * w.V * (2 if w.dtype == "bf16" else 4) + (6 << 30)
    T = w.T if free > need else max(1024, int(w.T * (free - (8 << 30)) / need) // 256 * 256)
    batch = inputs.make_rows(w, seed=0, device=DEV, T=T)
    rho = w.rhos[rho_index]
    res = _forward(batch, rho, True, want_mask=False)
    torch.cuda.synchronize()
    # size-free properties
    assert (res.train.count >= 1).all() and (res.infer.count >= 1).all()
    member = (res.flags & 1).bool()
    assert (res.train.logp_mp[member] <= 1e-6).all()
    assert torch.isneginf(res.train.logp_mp[~member]).all()
    assert (res.train.lse_safe <= res.train.lse + 1e-4).all()
    assert (res.train.logp_mp[member] >= res.train.logp[member] - 1e-5).all()
    step = max(1, T // 16)
    for r0 in range(0, T, 4096):                       # row sums of the gradient vanish
        rows = slice(r0, min(T, r0 + 4096))
        sums = res.grad_train[rows].float().sum(dim=1)
        scale = res.grad_train[rows].float().abs().sum(dim=1)
        u = parity.UNIT_ROUNDOFF[res.grad_train.dtype]
        assert (sums.abs() <= (1e-3 + 4 * u) * scale + 1e-12).all()
    pick = torch.unique(torch.cat([torch.arange(0, T, step), torch.tensor([0, T - 1, T // 2 + 1])])).to(DEV)
    sub = inputs.RowBatch(batch.train[pick], batch.infer[pick], batch.ids[pick], batch.upstream[pick])
    sub_res = type(res)(train=_take(res.train, pick), infer=_take(res.infer, pick),
                        log_ratio=res.log_ratio[pick], flags=res.flags[pick],
                        grad_train=res.grad_train[pick])
    parity.check_forward(sub_res, sub, rho, w.V, True)


@pytest.mark.parametrize("rho", [1e-4, 1e-3])
def test_full_size_forward_only_configuration(rho):
    """T = 8192 x V = 151,936 bf16, forward only, both thresholds, as the benchmark
    launches it: size-free properties on every row, sampled rows against the oracle."""
    w = W["c1_bf16_fwd"]
    batch = inputs.make_rows(w, seed=0, device=DEV)
    T = batch.train.shape[0]
    res = _forward(batch, rho, False, want_mask=False)
    torch.cuda.synchronize()
    assert res.grad_train is None
    assert (res.train.count >= 1).all() and (res.infer.count >= 1).all()
    member = (res.flags & 1).bool()
    assert (res.train.logp_mp[member] <= 1e-6).all()
    assert torch.isneginf(res.train.logp_mp[~member]).all()
    assert (res.infer.lse_safe <= res.infer.lse + 1e-4).all()
    both = ((res.flags & 3) == 3)
    assert torch.isfinite(res.log_ratio[both]).all() and both.float().mean().item() > 0.8
    pick = torch.unique(torch.cat([torch.arange(0, T, T // 32), torch.tensor([0, T - 1])])).to(DEV)
    sub = inputs.RowBatch(batch.train[pick], batch.infer[pick], batch.ids[pick], batch.upstream[pick])
    sub_res = type(res)(train=_take(res.train, pick), infer=_take(res.infer, pick),
                        log_ratio=res.log_ratio[pick], flags=res.flags[pick], grad_train=None)
    parity.check_forward(sub_res, sub, rho, w.V, False)


def _take(side, pick):
    out = type(side)()
    for k, v in vars(side).items():
        setattr(out, k, v[pick] if isinstance(v, torch.Tensor) else v)
    return out
