"""Parity of the tensor-core contraction and of the fused LM-head entry point
with the fp64 oracle, through the C ABI.

Membership in the fused variant is decided on bf16 x bf16 products accumulated
in fp32 by the tensor cores (H/16 accumulation steps, each good to one unit in
the last place of the running sum), so it cannot be bit-exact against fp64
logits: a logit within (H/16 + 2) 2^-24 max|z| + 1e-6 of the threshold (the
rounding band) may fall on either side.  The device's packed safe set is
therefore read back: outside the band it must equal the set of Def. 5.1 on the
float64 logits bit for bit; inside the band either decision is accepted, and the
oracle then states what every other quantity must be for the set the device took
(dvp_oracle_side_given_set).  Against that, every token is compared exactly
like the row kernels: counts, flags and infinities exact, log-probabilities
within 1e-4.  How many logits sat in the band, and how many of them the device
decided the other way, is reported.
Gradients: per token row of d_hidden and per vocabulary row of d_w,
||X - X_oracle||_2 <= 1e-3 ||X_oracle||_2 + 1e-6 * (largest row norm), the second
term covering rows that are zero up to the float16 grid of the gradient panel.
d_w is compared on every vocabulary row in every test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_23087_b200 import binding, inputs

import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _bits(x):
    return x.detach().cpu().view(torch.int16).numpy().view(np.uint16)


@pytest.mark.parametrize("single", [False, True])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
@pytest.mark.parametrize("m,n,k", [(128, 256, 64), (128, 256, 512), (300, 520, 200), (1, 8, 8),
                                   (1000, 776, 1032), (257, 4096, 4104), (2048, 512, 8192)])
def test_gemm_tn_matches_float64_matmul(dtype, m, n, k, single):
    """Both kernels: 256 x 256 tiles on pairs of blocks (default) and 128 x 256 tiles on single blocks."""
    g = torch.Generator(device=DEV).manual_seed(m * 7 + n * 3 + k)
    a = torch.randn(m, k, generator=g, device=DEV).to(dtype)
    b = torch.randn(n, k, generator=g, device=DEV).to(dtype)
    ref = (a.double() @ b.double().t())
    out, status = binding.dvp_gemm_tn(a, b, alpha=0.5, single_block_tiles=single)
    torch.cuda.synchronize()
    assert status.item() == 0
    # fp32 accumulation in tensor memory: up to one unit in the last place per 16-wide step
    tol = (2.0 ** -24 * (k / 16) + 1e-6) * ref.abs().max().item()
    err = (out.double() - 0.5 * ref).abs().max().item()
    assert err <= tol, (err, tol)
    # accumulate on top, strided operands, misaligned-free views
    out2, status = binding.dvp_gemm_tn(a, b, alpha=0.25, out=out.clone(), accumulate=True,
                                       single_block_tiles=single)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert (out2.double() - 0.75 * ref).abs().max().item() <= 2 * tol


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
@pytest.mark.parametrize("m,n,k", [(256, 256, 64), (512, 256, 256), (304, 520, 200), (8, 8, 8), (1000, 776, 1032),
                                   (4104, 512, 4096), (2048, 264, 8200)])
def test_gemm_tn_transposed_a_operand(dtype, m, n, k):
    """A given as [k, m] with m contiguous: the tensor cores read it as an MN-major
    operand (this is how d_w = G^T hidden takes the gradient panel without a transpose)."""
    g = torch.Generator(device=DEV).manual_seed(m * 5 + n * 3 + k)
    at = torch.randn(k, m + 8, generator=g, device=DEV).to(dtype)[:, :m]      # padded row stride
    b = torch.randn(n, k, generator=g, device=DEV).to(dtype)
    ref = at.double().t() @ b.double().t()
    out, status = binding.dvp_gemm_tn(at, b, alpha=0.5, a_transposed=True)
    torch.cuda.synchronize()
    assert status.item() == 0
    tol = (2.0 ** -24 * (k / 16) + 1e-6) * ref.abs().max().item()
    assert (out.double() - 0.5 * ref).abs().max().item() <= tol
    plain, _ = binding.dvp_gemm_tn(at.t().contiguous(), b, alpha=0.5)
    torch.cuda.synchronize()
    assert (out - plain).abs().max().item() <= 2 * tol
    out2, status = binding.dvp_gemm_tn(at, b, alpha=0.25, out=out.clone(), accumulate=True, a_transposed=True)
    torch.cuda.synchronize()
    assert status.item() == 0 and (out2.double() - 0.75 * ref).abs().max().item() <= 2 * tol
    with pytest.raises(binding.DvpError):          # only the paired kernel reads a transposed A
        binding.dvp_gemm_tn(at, b, a_transposed=True, single_block_tiles=True)


@pytest.mark.parametrize("m,n,k,transposed", [(256, 256, 8192, False), (1000, 776, 4104, False), (512, 264, 20000, True),
                                              (300, 520, 200, False), (128, 256, 64, False)])
def test_gemm_tn_split_k(m, n, k, transposed):
    """Two halves of the k range per tile, met in C by atomic adds: same result as one
    pass (up to the order of two partial sums), reruns bit-identical, accumulate on top."""
    g = torch.Generator(device=DEV).manual_seed(m + n + k)
    a = torch.randn(m, k, generator=g, device=DEV).to(torch.float16)
    b = torch.randn(n, k, generator=g, device=DEV).to(torch.float16)
    ref = a.double() @ b.double().t()
    arg = a.t().contiguous() if transposed else a
    out, status = binding.dvp_gemm_tn(arg, b, alpha=0.5, split_k=True, a_transposed=transposed)
    out_b, _ = binding.dvp_gemm_tn(arg, b, alpha=0.5, split_k=True, a_transposed=transposed)
    torch.cuda.synchronize()
    assert status.item() == 0
    tol = (2.0 ** -24 * (k / 16) + 1e-6) * ref.abs().max().item()
    assert (out.double() - 0.5 * ref).abs().max().item() <= tol
    assert torch.equal(out, out_b)
    out2, status = binding.dvp_gemm_tn(arg, b, alpha=0.25, out=out.clone(), accumulate=True, split_k=True,
                                       a_transposed=transposed)
    torch.cuda.synchronize()
    assert status.item() == 0 and (out2.double() - 0.75 * ref).abs().max().item() <= 2 * tol


def test_gemm_tn_padded_strides_and_argument_errors():
    g = torch.Generator(device=DEV).manual_seed(5)
    a = torch.randn(200, 328, generator=g, device=DEV).to(torch.bfloat16)[:, :320]
    b = torch.randn(130, 336, generator=g, device=DEV).to(torch.bfloat16)[:, :320]
    out = torch.full((200, 136), 7.0, device=DEV)[:, :130]
    binding.dvp_gemm_tn(a, b, out=out)
    torch.cuda.synchronize()
    ref = a.double() @ b.double().t()
    assert (out.double() - ref).abs().max().item() < 1e-3
    with pytest.raises(binding.DvpError) as e:
        binding.dvp_gemm_tn(a[:, :317], b[:, :317].contiguous())      # lda = 328 ok, ldb = 317 not
    assert e.value.status == binding.DVP_ERR_UNSUPPORTED


def _oracle_with_the_devices_set(batch, rho, res, weight=None, rep=None):
    """The oracle's result for the safe set the device took.  The set of Def. 5.1 is computed
    on the float64 logits; logits within the rounding band of the threshold may fall on either
    side on the device, every other logit must agree exactly.  The oracle then states what all
    other quantities must be for the device's set (dvp_oracle_side_given_set)."""
    rep = {} if rep is None else rep
    H, V = batch.hidden.shape[1], batch.w_vocab.shape[0]
    z = oracle.fused_logits(_bits(batch.hidden), _bits(batch.w_vocab))
    ids = batch.ids.cpu().numpy()
    own = oracle.dvp_rows_f64(z, np.where((ids >= 0) & (ids < V), ids, -1), rho, want_mask=True).train
    width = (H / 16 + 2) * 2.0 ** -24 * np.abs(z).max(axis=1, keepdims=True) + 1e-6
    band = np.abs(z - own.tau[:, None]) <= width
    dev_set = parity.unpack_mask(res.train.mask, V)
    assert np.array_equal(dev_set[~band], own.mask[~band]), "membership differs outside the rounding band"
    rep["band_tokens"] = rep.get("band_tokens", 0) + int(band.sum())
    rep["band_rows"] = rep.get("band_rows", 0) + int(band.any(axis=1).sum())
    rep["band_tokens_decided_otherwise"] = rep.get("band_tokens_decided_otherwise", 0) + \
        int((dev_set[band] != own.mask[band]).sum())
    wkw = {} if weight is None else dict(weight_kind=weight[0], weight_lo=weight[1], weight_hi=weight[2])
    want = oracle.dvp_fused_lmhead(_bits(batch.hidden), _bits(batch.w_vocab), _bits(batch.infer), ids, rho,
                                   batch.upstream.cpu().numpy().astype(np.float64), logits=z,
                                   train_set=np.where(band, dev_set, own.mask).astype(np.uint8), **wkw)
    return want, rep


def _rows_close(got, ref, name, rep, rows=None):
    got = got.cpu().double().numpy() if isinstance(got, torch.Tensor) else got
    if rows is not None:
        got, ref = got[rows], ref[rows]
    num = np.sqrt(((got - ref) ** 2).sum(axis=1))
    den = np.sqrt((ref ** 2).sum(axis=1))
    bound = 1e-3 * den + 1e-6 * den.max()
    assert (num <= bound).all(), f"{name}: worst {np.max(num / np.maximum(den, 1e-300)):.3e}"
    rep[name] = float(np.max(num / np.maximum(den, 1e-6 * den.max())))


def _check_fused(batch, rho, res, want, V, weight=None, rerun=None, d_w_extra=0.0, check_dw=True, rep=None):
    """Every token against the oracle's result for the device's safe set: counts, flags and
    infinities exact, log-probabilities within 1e-4, gradient rows within 1e-3 relative L2.
    weight: (kind, lo, hi) of an importance-weighted call; tokens whose ratio sits within 5e-4
    relative of a masking bound (where the weight jumps) are left out of the gradient rows, and
    d_w is then compared on a second call (rerun(upstream)) with their upstream gradient zeroed.
    d_w_extra is what d_w held before an accumulating call."""
    rep = {} if rep is None else rep
    T = len(want.rows.train.count)
    for label, got, side in (("train", res.train, want.rows.train), ("infer", res.infer, want.rows.infer)):
        if got is None:
            continue
        assert np.array_equal(got.count.cpu().numpy().astype(np.int64), side.count), f"{label}.count"
        np.testing.assert_allclose(got.max.cpu().numpy(), side.max, atol=1e-4, rtol=0)
        np.testing.assert_allclose(got.lse.cpu().numpy(), side.lse, atol=1e-4, rtol=0)
        np.testing.assert_allclose(got.lse_safe.cpu().numpy(), side.lse_safe, atol=1e-4, rtol=0)
        np.testing.assert_allclose(got.log_cov.cpu().numpy(), side.log_cov, atol=1e-4, rtol=0)
        parity._close(got.logp.cpu(), side.logp, 1e-4, f"{label}.logp")
        parity._close(got.logp_mp.cpu(), side.logp_mp, 1e-4, f"{label}.logp_mp")
    flags = res.flags.cpu().numpy()
    assert np.array_equal(flags & 1, want.rows.train.member)
    if res.infer is not None:
        assert np.array_equal((flags >> 1) & 1, want.rows.infer.member)
        parity._close(res.log_ratio.cpu(), want.rows.log_ratio, 2e-4, "log_ratio")
    ok = np.ones(T, dtype=bool)
    if weight is not None:
        ratio = np.exp(want.rows.log_ratio)
        near = np.zeros(T, dtype=bool)
        if weight[0] == oracle.WEIGHT_MASK:
            with np.errstate(invalid="ignore"):
                near = (np.abs(ratio - weight[1]) <= 5e-4 * weight[1]) | (np.abs(ratio - weight[2]) <= 5e-4 * weight[2])
        rep["near_weight_bound_rows"] = int(near.sum())
        ok = ~near
        got_w = res.weight.cpu().numpy().astype(np.float64)
        assert np.array_equal(np.isnan(got_w), np.isnan(want.rows.weight))
        assert (np.abs(got_w - want.rows.weight)[ok] <= 2e-4 * np.abs(want.rows.weight[ok]) + 1e-12).all(), "weight"
        rep["zero_weight_rows"] = int((want.rows.weight[ok] == 0).sum())
    _rows_close(res.d_hidden, want.d_hidden, "d_hidden", rep, ok)
    rep["ok_rows"] = ok
    if not check_dw:
        return rep
    if ok.all():
        _rows_close(res.d_w, want.d_w + d_w_extra, "d_w", rep)
    else:
        # the tokens left out contribute G_t^T h_t each: zero their upstream on the device,
        # take their terms out of the oracle's sum
        up = batch.upstream.clone()
        up[torch.from_numpy(~ok).to(up.device)] = 0.0
        again = rerun(up)
        h = batch.hidden.detach().cpu().double().numpy()
        _rows_close(again.d_w, want.d_w - want.rows.grad[~ok].T @ h[~ok] + d_w_extra, "d_w", rep)
    return rep


def _run_fused(T, H, V, rho, seed, weight=None, **kw):
    w = inputs.WORKLOADS["c4_fused_lmhead"]
    batch = inputs.make_fused(w, seed=seed, device=DEV, T=T, H=H, V=V)
    wkw = {} if weight is None else dict(weight_kind=weight[0], weight_lo=weight[1], weight_hi=weight[2])

    def rerun(upstream):
        r = binding.dvp_fused_lmhead_forward_backward(batch.hidden, batch.w_vocab, batch.ids, rho, upstream,
                                                      infer_logits=batch.infer, want_mask=True, **wkw, **kw)
        torch.cuda.synchronize()
        assert r.workspace[:4].view(torch.int32).item() == 0, "a tensor-core kernel gave up waiting"
        return r
    res = rerun(batch.upstream)
    want, rep = _oracle_with_the_devices_set(batch, rho, res, weight)
    return batch, res, want, rerun


@pytest.mark.parametrize("T,H,V,rho", [(200, 256, 3000, 1e-3), (64, 128, 1000, 1e-2), (130, 512, 5008, 1e-4),
                                       (128, 4096, 4096, 1e-3),
                                       # vocabularies that end inside a 32-byte piece of the fp32 panel and
                                       # inside a 16-element block of the contractions' tiles
                                       (96, 128, 1003, 1e-2), (140, 256, 4099, 1e-3), (70, 64, 7, 1e-1)])
def test_fused_lmhead_small(T, H, V, rho):
    batch, res, want, rerun = _run_fused(T, H, V, rho, seed=T)
    _check_fused(batch, rho, res, want, V, rerun=rerun)


@pytest.mark.parametrize("weight", [(oracle.WEIGHT_TRUNCATE, 0.0, 1.004), (oracle.WEIGHT_MASK, 0.985, 1.01)],
                         ids=["truncate", "mask"])
@pytest.mark.parametrize("T,H,V,rho,panel", [(200, 256, 3000, 1e-3, 0), (300, 128, 2048, 1e-2, 128)])
def test_fused_lmhead_importance_weighted(T, H, V, rho, panel, weight):
    """Thm. 5.3 per token through the LM head: the inference rows are swept first, the
    training panels take the weight from them; one panel and several."""
    batch, res, want, rerun = _run_fused(T, H, V, rho, seed=T + 1, weight=weight, panel_rows=panel)
    rep = _check_fused(batch, rho, res, want, V, weight=weight, rerun=rerun)
    assert (want.rows.weight != np.exp(want.rows.log_ratio))[np.isfinite(want.rows.log_ratio)].any()   # the bounds do cut
    if weight[0] == oracle.WEIGHT_MASK:
        assert rep["zero_weight_rows"] >= 1
    plain = binding.dvp_fused_lmhead_forward_backward(batch.hidden, batch.w_vocab, batch.ids, rho, batch.upstream,
                                                      infer_logits=batch.infer, panel_rows=panel)
    torch.cuda.synchronize()
    assert torch.equal(plain.train.logp_mp, res.train.logp_mp) and torch.equal(plain.flags, res.flags)
    fin = torch.isfinite(plain.log_ratio)
    assert torch.equal(plain.log_ratio[fin], res.log_ratio[fin])


def test_fused_lmhead_several_panels_and_dw_accumulation():
    T, H, V, rho = 300, 256, 2048, 1e-3
    w = inputs.WORKLOADS["c4_fused_lmhead"]
    batch = inputs.make_fused(w, seed=9, device=DEV, T=T, H=H, V=V)
    d_w = torch.full((V, H), 0.5, device=DEV)
    res = binding.dvp_fused_lmhead_forward_backward(batch.hidden, batch.w_vocab, batch.ids, rho,
                                                    batch.upstream, infer_logits=batch.infer,
                                                    panel_rows=128, d_w=d_w, accumulate_dw=True, want_mask=True)
    torch.cuda.synchronize()
    assert res.workspace[:4].view(torch.int32).item() == 0
    want, rep = _oracle_with_the_devices_set(batch, rho, res)
    _check_fused(batch, rho, res, want, V, d_w_extra=0.5, rep=rep)
    one = binding.dvp_fused_lmhead_forward_backward(batch.hidden, batch.w_vocab, batch.ids, rho,
                                                    batch.upstream, infer_logits=batch.infer)
    torch.cuda.synchronize()
    assert (one.d_hidden - res.d_hidden).abs().max().item() <= 1e-5 * res.d_hidden.abs().max().item()
    assert torch.equal(one.train.count, res.train.count)


@pytest.mark.parametrize("panel", [0, 4224, 128])
def test_fused_lmhead_tokens_that_share_a_sampled_id(panel):
    """A small vocabulary: most sampled ids occur many times, so the 1[k = a] terms of many tokens
    meet in the same rows of d_w (they are added in token order: reruns are bit-identical).  A
    panel of 4224 tokens spans two chunks of that order-fixing step."""
    T, H, V, rho = 4224, 128, 512, 1e-2
    batch, res, want, rerun = _run_fused(T, H, V, rho, seed=21, panel_rows=panel)
    assert len(np.unique(batch.ids.cpu().numpy())) < T // 4
    _check_fused(batch, rho, res, want, V, rerun=rerun)
    again = rerun(batch.upstream)
    assert torch.equal(again.d_w, res.d_w) and torch.equal(again.d_hidden, res.d_hidden)


def test_fused_lmhead_full_vocabulary_rows():
    """V = 151,936 with the LM-head statistics of the benchmark configuration."""
    batch, res, want, rerun = _run_fused(256, 1024, 151936, 1e-3, seed=3)
    rep = _check_fused(batch, 1e-3, res, want, 151936, rerun=rerun)
    assert want.rows.train.count.mean() > 1000        # dense safe sets, as in the full configuration


def _rows_of(res, sl):
    """The per-token part of a fused result restricted to the rows `sl`."""
    from types import SimpleNamespace

    def side(s):
        if s is None:
            return None
        return SimpleNamespace(**{k: (v[sl] if isinstance(v, torch.Tensor) else v) for k, v in vars(s).items()})
    return SimpleNamespace(train=side(res.train), infer=side(res.infer), log_ratio=res.log_ratio[sl],
                           flags=res.flags[sl], d_hidden=res.d_hidden[sl], d_w=None,
                           weight=None if getattr(res, "weight", None) is None else res.weight[sl])


@pytest.mark.parametrize("rho", [1e-4, 1e-3])
def test_fused_lmhead_benchmark_shape_full_panel_and_ragged_panel(rho):
    """The benchmark configuration's own H = 4096 and V = 151,936 with its default panels: one
    full panel of 4096 tokens and a ragged one of 128, d_w accumulated across them, K = 4096
    accumulation steps per logit and K = V in the d_hidden contraction.  The oracle works through
    the tokens in slabs (float64 logits of a slab are 0.6 GB); per-token outputs and d_hidden are
    compared on every token, d_w on every vocabulary row, all for the safe sets the device took
    (which must be the oracle's outside the rounding band; the band's size is printed)."""
    T, H, V, slab = 4096 + 128, 4096, 151936, 512
    if _host_memory_available() < 40 << 30:
        pytest.skip("the float64 oracle of this shape needs about 25 GB of host memory")
    w = inputs.WORKLOADS["c4_fused_lmhead"]
    batch = inputs.make_fused(w, seed=11, device=DEV, T=T, H=H, V=V)
    res = binding.dvp_fused_lmhead_forward_backward(batch.hidden, batch.w_vocab, batch.ids, rho, batch.upstream,
                                                    infer_logits=batch.infer, want_mask=True)
    torch.cuda.synchronize()
    assert res.workspace[:4].view(torch.int32).item() == 0, "a tensor-core kernel gave up waiting"
    d_w = np.zeros((V, H))
    rep = {}
    for r0 in range(0, T, slab):
        sl = slice(r0, min(T, r0 + slab))
        sub = inputs.FusedBatch(batch.hidden[sl], batch.w_vocab, batch.infer[sl], batch.ids[sl], batch.upstream[sl])
        sub_res = _rows_of(res, sl)
        want, rep = _oracle_with_the_devices_set(sub, rho, sub_res, rep=rep)
        _check_fused(sub, rho, sub_res, want, V, check_dw=False, rep=rep)
        d_w += want.d_w
        del want
    print(f"rho={rho}: {rep['band_tokens']} logits of {rep['band_rows']} tokens (of {T}) lie within rounding "
          f"distance of the threshold; the device decided {rep['band_tokens_decided_otherwise']} of them the "
          f"other way; worst d_hidden row {rep['d_hidden']:.2e}")
    den = np.sqrt((d_w ** 2).sum(axis=1))
    num = np.empty(V)
    for k0 in range(0, V, 16384):                     # vocabulary rows in chunks: no second 5 GB copy
        ks = slice(k0, min(V, k0 + 16384))
        num[ks] = np.sqrt(((res.d_w[ks].cpu().double().numpy() - d_w[ks]) ** 2).sum(axis=1))
    assert (num <= 1e-3 * den + 1e-6 * den.max()).all(), f"d_w: worst {np.max(num / np.maximum(den, 1e-300)):.3e}"
    assert rep["band_tokens_decided_otherwise"] <= rep["band_tokens"]


def _host_memory_available() -> int:
    """Bytes of host memory this process may still take: the smaller of what the machine has
    free and what is left under the container's limit."""
    import psutil
    avail = psutil.virtual_memory().available
    try:
        limit = open("/sys/fs/cgroup/memory.max").read().strip()
        used = int(open("/sys/fs/cgroup/memory.current").read())
        if limit != "max":
            avail = min(avail, int(limit) - used)
    except OSError:
        pass
    return avail


def test_fused_argument_errors():
    w = inputs.WORKLOADS["c4_fused_lmhead"]
    batch = inputs.make_fused(w, seed=1, device=DEV, T=16, H=64, V=256)
    with pytest.raises(binding.DvpError) as e:
        binding.dvp_fused_lmhead_forward_backward(batch.hidden, batch.w_vocab, batch.ids, 1e-3,
                                                  batch.upstream, panel_rows=100)
    assert e.value.status == binding.DVP_ERR_INVALID_ARG
    with pytest.raises(binding.DvpError) as e:
        binding.dvp_fused_lmhead_forward_backward(batch.hidden, batch.w_vocab, batch.ids, 1e-3,
                                                  batch.upstream, workspace=torch.empty(512, dtype=torch.uint8, device=DEV))
    assert e.value.status == binding.DVP_ERR_WORKSPACE


def test_fused_missing_and_out_of_range_ids_and_empty_batch():
    w = inputs.WORKLOADS["c4_fused_lmhead"]
    batch = inputs.make_fused(w, seed=2, device=DEV, T=40, H=128, V=1024)
    batch.ids[3] = -1
    batch.ids[7] = 5000
    res = binding.dvp_fused_lmhead_forward_backward(batch.hidden, batch.w_vocab, batch.ids, 1e-2,
                                                    batch.upstream, infer_logits=batch.infer)
    torch.cuda.synchronize()
    flags = res.flags.tolist()
    assert flags[3] & binding.DVP_FLAG_NO_ID and flags[7] & binding.DVP_FLAG_BAD_ID
    assert torch.isnan(res.train.logp_mp[[3, 7]]).all() and torch.isnan(res.log_ratio[[3, 7]]).all()
    assert res.d_hidden[[3, 7]].abs().max().item() == 0.0
    ids = batch.ids.clone()
    ids[3] = 0
    ids[7] = 0
    want = oracle.dvp_fused_lmhead(_bits(batch.hidden), _bits(batch.w_vocab), _bits(batch.infer),
                                   batch.ids.cpu().numpy(), 1e-2, batch.upstream.cpu().numpy().astype(np.float64))
    keep = np.ones(40, dtype=bool)
    keep[[3, 7]] = False
    num = np.linalg.norm(res.d_hidden.cpu().double().numpy()[keep] - want.d_hidden[keep], axis=1)
    den = np.linalg.norm(want.d_hidden[keep], axis=1)
    assert (num <= 1e-3 * den + 1e-6 * den.max()).all()
    empty = binding.dvp_fused_lmhead_forward_backward(batch.hidden[:0], batch.w_vocab, batch.ids[:0], 1e-2,
                                                      batch.upstream[:0])
    assert empty.d_hidden.shape[0] == 0
