"""Pins for the fp64 oracle: it is checked against what the paper and the
mathematics fix, never against itself.

Each test names the passage of the paper it leans on.  A second implementation
inside a test is always written a different way (probability space instead of
logit space, a library log-softmax on -inf-masked logits, autograd, central
differences, exact rational arithmetic where it applies).
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(rng, T, V, scale=3.0):
    return rng.normal(size=(T, V)) * scale


def _safe_set(z: torch.Tensor, rho: float) -> torch.Tensor:
    """Def. 5.1 as printed, in probability space: k is safe iff pi(k) >= rho max_j pi(j).
    The inputs of these tests keep every logit away from the threshold, so that this and the
    logit-space form decide alike (checked)."""
    with torch.no_grad():
        pi = torch.softmax(z.detach().to(torch.float64), dim=-1)
        safe = pi >= rho * pi.max(dim=-1, keepdim=True).values
        if rho > 0:
            gap = (torch.log(pi) - torch.log(rho * pi.max(dim=-1, keepdim=True).values)).abs().min()
            assert gap > 1e-9, "a logit sits on the threshold: the two forms of Def. 5.1 may differ"
    return safe


def _log_pi_mp(z: torch.Tensor, rho: float) -> torch.Tensor:
    """ln pi^mp of Def. 5.2 by explicit renormalisation: pi^mp(k) = pi(k) / Z on the safe set,
    Z = sum of pi over the safe set; -inf off it.  Differentiable in z with the set held fixed."""
    safe = _safe_set(z, rho)
    pi = torch.softmax(z, dim=-1)
    cover = (pi * safe).sum(dim=-1, keepdim=True)
    inside = torch.log(torch.where(safe, pi, torch.ones_like(pi)) / cover)
    return torch.where(safe, inside, torch.full_like(inside, -math.inf))


# --------------------------------------------------------------------------
# Brute force in probability space (Def. 5.1 and Def. 5.2 as printed), tiny V,
# extended precision, every token a enumerated.
# --------------------------------------------------------------------------
@pytest.mark.parametrize("rho", [0.5, 0.1, 1e-2, 1e-4])
def test_bruteforce_probability_space_every_token(rho):
    rng = np.random.default_rng(7)
    ld = np.longdouble
    for V in (2, 3, 5, 8, 12):
        z = _rows(rng, 6, V, scale=2.5)
        # keep clear of the threshold so both spaces decide alike
        tau = z.max(1, keepdims=True) + math.log(rho)
        assert np.abs(z - tau).min() > 1e-9
        for a in range(V):
            ids = np.full(6, a)
            res = oracle.dvp_rows_f64(z, ids, rho, want_mask=True)
            for t in range(6):
                e = np.exp(z[t].astype(ld) - z[t].max().astype(ld))
                pi = e / e.sum()
                safe = pi >= ld(rho) * pi.max()                    # Def. 5.1
                Z = pi[safe].sum()                                 # Def. 5.2
                pi_mp = np.where(safe, pi / Z, ld(0))
                assert abs(float(pi_mp.sum()) - 1.0) < 1e-15
                assert np.array_equal(res.train.mask[t].astype(bool), safe)
                assert res.train.count[t] == safe.sum()
                assert res.train.member[t] == int(safe[a])
                assert res.train.logp[t] == pytest.approx(float(np.log(pi[a])), abs=1e-12)
                assert res.train.log_cov[t] == pytest.approx(float(np.log(Z)), abs=1e-12)
                if safe[a]:
                    assert res.train.logp_mp[t] == pytest.approx(float(np.log(pi_mp[a])), abs=1e-12)
                else:
                    assert res.train.logp_mp[t] == -np.inf
                assert res.train.max[t] == z[t].max()


def test_rho_zero_is_full_log_softmax():
    """Every token satisfies pi >= 0: the limit rho -> 0 of Def. 5.1."""
    rng = np.random.default_rng(1)
    z = _rows(rng, 5, 301, scale=4.0)
    ids = rng.integers(0, 301, size=5)
    res = oracle.dvp_rows_f64(z, ids, 0.0, want_mask=True)
    ref = torch.log_softmax(torch.from_numpy(z), dim=-1).numpy()
    want = ref[np.arange(5), ids]
    np.testing.assert_allclose(res.train.logp_mp, want, atol=1e-12, rtol=0)
    np.testing.assert_allclose(res.train.logp, want, atol=1e-12, rtol=0)
    assert (res.train.count == 301).all() and res.train.mask.all()
    np.testing.assert_allclose(res.train.log_cov, 0.0, atol=1e-14)
    lse = torch.logsumexp(torch.from_numpy(z), dim=-1).numpy()
    np.testing.assert_allclose(res.train.lse, lse, atol=1e-12, rtol=0)
    np.testing.assert_allclose(res.train.lse_safe, lse, atol=1e-12, rtol=0)


def test_rho_one_keeps_exactly_the_argmax_ties():
    z = np.array([[0.5, 2.0, -1.0, 2.0, 1.999999, 2.0],
                  [3.0, 1.0, 0.0, -2.0, 2.9, 1.0]])
    res = oracle.dvp_rows_f64(z, np.array([1, 0]), 1.0, want_mask=True)
    assert res.train.mask.tolist() == [[0, 1, 0, 1, 0, 1], [1, 0, 0, 0, 0, 0]]
    assert res.train.count.tolist() == [3, 1]
    assert res.train.logp_mp[0] == pytest.approx(-math.log(3.0), abs=1e-15)
    assert res.train.logp_mp[1] == pytest.approx(0.0, abs=1e-15)
    # a token just under the maximum is pruned at rho = 1
    res = oracle.dvp_rows_f64(z, np.array([4, 4]), 1.0)
    assert res.train.member.tolist() == [0, 0]
    assert np.isneginf(res.train.logp_mp).all()


def test_threshold_tie_is_kept():
    """Def. 5.1 uses >=, and the listing of App. A prunes with a strict <."""
    L = math.log(0.25)
    z = np.array([[4.0, 4.0 + L, np.nextafter(4.0 + L, -np.inf), 0.0]])
    res = oracle.dvp_rows_f64(z, np.array([1]), 0.25, want_mask=True)
    assert res.train.mask.tolist() == [[1, 1, 0, 0]]
    assert res.train.member[0] == 1


@pytest.mark.parametrize("rho", [1.0, 0.3, 1e-3, math.exp(-13), 1e-20, 0.0])
def test_invariants(rho):
    rng = np.random.default_rng(11)
    z = _rows(rng, 40, 257, scale=5.0)
    ids = rng.integers(0, 257, size=40)
    res = oracle.dvp_rows_f64(z, ids, rho, want_mask=True)
    s = res.train
    amax = z.argmax(1)
    assert s.mask[np.arange(40), amax].all()              # argmax is always safe
    assert (s.count >= 1).all() and (s.count == s.mask.sum(1)).all()
    assert (s.log_cov <= 1e-15).all()                     # Z <= 1
    member = s.member.astype(bool)
    assert (s.logp_mp[member] >= s.logp[member] - 1e-15).all()   # pi/Z >= pi
    np.testing.assert_allclose(s.logp_mp[member], (s.logp - s.log_cov)[member], atol=1e-12)
    assert np.isneginf(s.logp_mp[~member]).all()
    # renormalised probabilities over the safe set sum to one
    for t in range(40):
        p = np.exp(z[t][s.mask[t].astype(bool)] - s.lse_safe[t])
        assert math.fsum(p) == pytest.approx(1.0, abs=1e-13)
        assert s.lse_safe[t] <= s.lse[t] + 1e-15


@pytest.mark.parametrize("rho", [0.2, 1e-2, 1e-4])
def test_masked_logit_policy_equivalence(rho):
    """Prop. 5.6 part 1: the softmax of logits whose pruned entries are -inf is pi^mp.  The
    safe set comes from Def. 5.1 in probability space; a library log-softmax of the masked
    logits and the explicit renormalisation of Def. 5.2 must both give the oracle's value."""
    rng = np.random.default_rng(3)
    z = torch.from_numpy(_rows(rng, 16, 500, scale=3.0))
    safe = _safe_set(z, rho)
    ref = torch.log_softmax(z.masked_fill(~safe, -math.inf), dim=-1).numpy()
    ref2 = _log_pi_mp(z, rho).numpy()
    for a_kind in ("random", "argmax"):
        ids = rng.integers(0, 500, size=16) if a_kind == "random" else z.numpy().argmax(1)
        res = oracle.dvp_rows_f64(z.numpy(), ids, rho, want_mask=True)
        np.testing.assert_allclose(res.train.logp_mp, ref[np.arange(16), ids], atol=1e-12, rtol=0)
        np.testing.assert_allclose(res.train.logp_mp, ref2[np.arange(16), ids], atol=1e-12, rtol=0)
        assert np.array_equal(res.train.mask.astype(bool), safe.numpy())


@pytest.mark.parametrize("rho", [0.3, 1e-2, 1e-4])
def test_gradient_matches_autograd_of_the_renormalised_policy(rho):
    """Prop. 5.4 / Prop. 5.6 part 2 with the set fixed (App. A protocol 1): autograd through
    pi(a) / Z of Def. 5.2, the safe set entering as a constant."""
    rng = np.random.default_rng(5)
    T, V = 12, 200
    z = torch.from_numpy(_rows(rng, T, V, scale=3.0)).requires_grad_(True)
    g = torch.from_numpy(rng.normal(size=T))
    ids_np = rng.integers(0, V, size=T)
    ids_np[:4] = z.detach().numpy().argmax(1)[:4]
    logp = _log_pi_mp(z, rho)[torch.arange(T), torch.from_numpy(ids_np)]
    member = torch.isfinite(logp)
    (logp[member] * g[member]).sum().backward()
    res = oracle.dvp_rows_f64(z.detach().numpy(), ids_np, rho, upstream=g.numpy())
    np.testing.assert_allclose(res.grad, z.grad.numpy(), atol=1e-13, rtol=1e-12)
    assert (res.grad[~member.numpy()] == 0).all()          # pruned token: zero row
    assert member.numpy().sum() >= 4 and (~member.numpy()).sum() >= 1


def test_gradient_central_differences_and_structure():
    rng = np.random.default_rng(9)
    T, V, rho, h = 6, 40, 5e-2, 1e-5
    z = _rows(rng, T, V, scale=2.0)
    tau = z.max(1, keepdims=True) + math.log(rho)
    assert np.abs(z - tau).min() > 10 * h
    ids = z.argsort(1)[:, -2]                               # second largest: a member
    g = rng.normal(size=T)
    res = oracle.dvp_rows_f64(z, ids, rho, upstream=g, want_mask=True)
    mask = res.train.mask.astype(bool)

    def logp_mp_frozen(zz, t):
        zs = zz[mask[t]]
        m = zs.max()
        return zz[ids[t]] - (m + math.log(math.fsum(np.exp(zs - m))))

    for t in range(T):
        for k in range(V):
            zp, zm = z[t].copy(), z[t].copy()
            zp[k] += h
            zm[k] -= h
            fd = g[t] * (logp_mp_frozen(zp, t) - logp_mp_frozen(zm, t)) / (2 * h)
            assert res.grad[t, k] == pytest.approx(fd, abs=2e-9)
        assert (res.grad[t][~mask[t]] == 0).all()
        assert math.fsum(res.grad[t]) == pytest.approx(0.0, abs=1e-14)
        # the sampled entry is g (1 - pi^mp(a)), every other safe entry is -g pi^mp(k)
        assert res.grad[t, ids[t]] == pytest.approx(g[t] * (1 - math.exp(res.train.logp_mp[t])), abs=1e-14)


def test_single_element_safe_set_has_exactly_zero_gradient():
    z = np.array([[50.0, 1.0, 0.0, -3.0]])
    res = oracle.dvp_rows_f64(z, np.array([0]), 1e-3, upstream=np.array([2.0]))
    assert res.train.count[0] == 1 and res.train.logp_mp[0] == 0.0
    assert (res.grad == 0).all()


def test_total_variation_equals_one_minus_coverage():
    """Proof of Prop. 5.5: TV(pi^mp, pi) = 1 - Z, by the half-L1 definition."""
    rng = np.random.default_rng(13)
    z = _rows(rng, 20, 9, scale=2.0)
    res = oracle.dvp_rows_f64(z, np.zeros(20, dtype=np.int64), 0.2, want_mask=True)
    for t in range(20):
        pi = np.exp(z[t] - z[t].max())
        pi /= pi.sum()
        safe = res.train.mask[t].astype(bool)
        pi_mp = np.where(safe, pi / pi[safe].sum(), 0.0)
        tv = 0.5 * np.abs(pi_mp - pi).sum()
        assert tv == pytest.approx(1.0 - math.exp(res.train.log_cov[t]), abs=1e-14)


def test_coverage_statistics_of_sequences():
    """dvp_coverage: Z_min and mean Z per sequence.  Pinned through the identity of the proof
    of Prop. 5.5 (Z = 1 - TV(pi^mp, pi), computed here from the probabilities, not from the
    oracle's ln Z) and exact summation; empty sequences give +inf and NaN."""
    rng = np.random.default_rng(31)
    z = _rows(rng, 37, 11, scale=2.5)
    res = oracle.dvp_rows_f64(z, np.zeros(37, dtype=np.int64), 0.1, want_mask=True)
    cov = []
    for t in range(37):
        pi = np.exp(z[t] - z[t].max())
        pi /= pi.sum()
        safe = res.train.mask[t].astype(bool)
        pi_mp = np.where(safe, pi / pi[safe].sum(), 0.0)
        cov.append(1.0 - 0.5 * np.abs(pi_mp - pi).sum())
    off = np.array([0, 5, 5, 6, 37, 37], dtype=np.int64)
    lo, mean = oracle.dvp_coverage(res.train.log_cov, off)
    for s in range(5):
        seg = cov[off[s]:off[s + 1]]
        if not seg:
            assert math.isinf(lo[s]) and lo[s] > 0 and math.isnan(mean[s])
        else:
            assert lo[s] == pytest.approx(min(seg), abs=1e-13)
            assert mean[s] == pytest.approx(math.fsum(seg) / len(seg), abs=1e-13)
    assert lo[3] < mean[3] < 1.0
    # the bound of Prop. 5.5 for R_max = 1 is T (1 - Z_min): it grows with the sequence, and a
    # sequence whose every state keeps the whole vocabulary has bound zero
    full = oracle.dvp_rows_f64(z, np.zeros(37, dtype=np.int64), 0.0)
    lo0, mean0 = oracle.dvp_coverage(full.train.log_cov, np.array([0, 37], dtype=np.int64))
    assert lo0[0] == pytest.approx(1.0, abs=1e-14) and mean0[0] == pytest.approx(1.0, abs=1e-14)


@pytest.mark.parametrize("eps_max", [1e-3, 1e-2, 1e-1])
def test_asymmetric_vulnerability_bound(eps_max):
    """Prop. 4.2.  Its proof bounds |Delta_a| by 2 eps_max (1 - p_a(z_c)) at a
    point z_c of the segment; log p_a is concave along the segment, so the
    smallest p_a(z_c) sits at an end point and the testable form is
    |Delta_a| <= 2 eps_max (1 - min(p_a, p'_a))."""
    rng = np.random.default_rng(17)
    T, V = 64, 300
    z = _rows(rng, T, V, scale=3.0)
    zi = z + rng.uniform(-eps_max, eps_max, size=z.shape)
    for pick in ("argmax", "random"):
        ids = z.argmax(1) if pick == "argmax" else rng.integers(0, V, size=T)
        tr = oracle.dvp_rows_f64(z, ids, 0.0).train
        inf = oracle.dvp_rows_f64(zi, ids, 0.0).train
        delta = tr.logp - inf.logp
        p_min = np.minimum(np.exp(tr.logp), np.exp(inf.logp))
        assert (np.abs(delta) <= 2 * eps_max * (1 - p_min) + 1e-12).all()
        if pick == "argmax":
            # the bound contracts for high-probability tokens
            assert np.abs(delta).max() < 2 * eps_max


def test_log_ratio_sign_and_conventions():
    """Delta = train - infer (Thm. 4.1); ratio zero when a leaves the training
    set (remark after Thm. 5.3); +inf when only the inference set drops it."""
    z = np.array([[5.0, 4.0, 2.0, -1.0]] * 3, dtype=np.float32)
    zi = z.copy()
    zi[0, 1] = 4.5                      # token 1 more likely under infer
    zi[1, 2] = -4.0                     # row 1: token 2 pruned on the infer side only
    z[2, 2] = -4.0                      # row 2: token 2 pruned on the train side only
    ids = np.array([1, 2, 2])
    res = oracle.dvp_rows(z, ids, 0.02, infer=zi)          # ln(0.02) = -3.9: tau = 1.09
    assert res.log_ratio[0] < 0 and np.isfinite(res.log_ratio[0])
    assert res.log_ratio[0] == pytest.approx(res.train.logp_mp[0] - res.infer.logp_mp[0])
    assert res.train.member.tolist() == [1, 1, 0] and res.infer.member.tolist() == [1, 0, 1]
    assert res.log_ratio[1] == np.inf and res.log_ratio[2] == -np.inf


def test_printed_constants():
    with open(os.path.join(GOLDEN, "paper_constants.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 4
    for name, expr, printed, digits, *_ in rows:
        value = eval(expr, {"exp": math.exp})
        assert float(f"{value:.{int(digits) - 1}e}") == float(printed), name
    # the default threshold enters the oracle as log(rho) = -13
    z = np.array([[0.0, -12.999, -13.001]])
    res = oracle.dvp_rows_f64(z, np.array([0]), math.exp(-13), want_mask=True)
    assert res.train.mask.tolist() == [[1, 1, 0]]


def test_storage_types_widen_exactly_and_strides_are_honoured():
    rng = np.random.default_rng(21)
    x = torch.from_numpy(rng.normal(size=(5, 64)).astype(np.float32) * 4)
    ids = rng.integers(0, 48, size=5)
    for dt, code in ((torch.bfloat16, oracle.BF16), (torch.float16, oracle.F16)):
        xs = x.to(dt)
        bits = xs.view(torch.int16).numpy().view(np.uint16)
        got = oracle.dvp_rows(bits[:, :48], ids, 1e-2, dtype=code)       # row stride 64 > V 48
        want = oracle.dvp_rows_f64(xs[:, :48].to(torch.float64).numpy(), ids, 1e-2)
        for name in ("max", "lse", "lse_safe", "logp_mp", "count"):
            assert np.array_equal(getattr(got.train, name), getattr(want.train, name)), name
    sub = torch.tensor([1e-7, -3e-6, 6e-5, 0.0], dtype=torch.float16)   # subnormal halves
    got = oracle.dvp_rows(sub.view(torch.int16).numpy().view(np.uint16)[None, :], np.array([2]), 0.0,
                          dtype=oracle.F16)
    assert got.train.max[0] == float(sub.max())


def test_batch_driver_threads_agree_and_no_id_rows():
    rng = np.random.default_rng(23)
    z = (rng.normal(size=(37, 130)) * 3).astype(np.float32)
    zi = (z + rng.normal(size=z.shape) * 0.01).astype(np.float32)
    ids = rng.integers(0, 130, size=37)
    ids[5] = -1
    g = rng.normal(size=37)
    r1 = oracle.dvp_rows(z, ids, 1e-3, infer=zi, upstream=g, want_grad=True, want_mask=True, threads=1)
    r4 = oracle.dvp_rows(z, ids, 1e-3, infer=zi, upstream=g, want_grad=True, want_mask=True, threads=4)
    assert r4.threads == 4
    assert np.array_equal(r1.grad, r4.grad) and np.array_equal(r1.train.mask, r4.train.mask)
    np.testing.assert_array_equal(r1.log_ratio, r4.log_ratio)
    assert np.isnan(r1.train.logp_mp[5]) and (r1.grad[5] == 0).all() and r1.train.count[5] >= 1


def test_fused_lmhead_matches_autograd_through_the_head():
    """Chain rule of Prop. 5.6 part 2 through z = h W^T, by torch autograd."""
    rng = np.random.default_rng(29)
    T, H, V, rho = 5, 8, 23, 5e-2
    hb = torch.from_numpy(rng.normal(size=(T, H)).astype(np.float32)).to(torch.bfloat16)
    wb = torch.from_numpy((rng.normal(size=(V, H)) * 0.5).astype(np.float32)).to(torch.bfloat16)
    h = hb.to(torch.float64).requires_grad_(True)
    w = wb.to(torch.float64).requires_grad_(True)
    z = h @ w.t()
    zi = (z.detach() + torch.from_numpy(rng.normal(size=(T, V)) * 0.02)).to(torch.bfloat16)
    ids = rng.integers(0, V, size=T)
    ids[:3] = z.detach().numpy().argmax(1)[:3]
    g = torch.from_numpy(rng.normal(size=T))
    logp = _log_pi_mp(z, rho)[torch.arange(T), torch.from_numpy(ids)]
    member = torch.isfinite(logp)
    (logp[member] * g[member]).sum().backward()
    bits = lambda x: x.view(torch.int16).numpy().view(np.uint16)
    res = oracle.dvp_fused_lmhead(bits(hb), bits(wb), bits(zi), ids, rho, g.numpy())
    np.testing.assert_allclose(res.logits, z.detach().numpy(), atol=1e-13)
    np.testing.assert_allclose(res.d_hidden, h.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(res.d_w, w.grad.numpy(), atol=1e-12)
    want = logp.detach().numpy()
    np.testing.assert_allclose(res.rows.train.logp_mp[member.numpy()], want[member.numpy()], atol=1e-12)
    # infer side: an ordinary row pass on the stored bf16 logits
    ref_i = oracle.dvp_rows(bits(zi), ids, rho, dtype=oracle.BF16)
    assert np.array_equal(res.rows.infer.logp_mp, ref_i.train.logp_mp)


def test_fused_lmhead_with_a_supplied_safe_set():
    """dvp_oracle_side_given_set / _grad_given_set through dvp_fused_lmhead(train_set=...):
    (i) with the set Def. 5.1 derives, the very numbers of the threshold form; (ii) with an
    arbitrary set (the argmax plus random tokens), pi^mp by explicit renormalisation over that
    set in probability space (Def. 5.2) and its gradient by autograd through h W^T."""
    rng = np.random.default_rng(41)
    T, H, V, rho = 6, 8, 19, 5e-2
    hb = torch.from_numpy(rng.normal(size=(T, H)).astype(np.float32)).to(torch.bfloat16)
    wb = torch.from_numpy((rng.normal(size=(V, H)) * 0.5).astype(np.float32)).to(torch.bfloat16)
    bits = lambda x: x.view(torch.int16).numpy().view(np.uint16)
    z = oracle.fused_logits(bits(hb), bits(wb))
    np.testing.assert_allclose(z, hb.double().numpy() @ wb.double().numpy().T, atol=1e-13)
    zi = torch.from_numpy(z + rng.normal(size=z.shape) * 0.02).to(torch.bfloat16)
    ids = rng.integers(0, V, size=T)
    g = rng.normal(size=T)
    plain = oracle.dvp_fused_lmhead(bits(hb), bits(wb), bits(zi), ids, rho, g)
    own = (z >= plain.rows.train.tau[:, None]).astype(np.uint8)
    same = oracle.dvp_fused_lmhead(bits(hb), bits(wb), bits(zi), ids, rho, g, logits=z, train_set=own)
    for name in ("max", "lse", "lse_safe", "log_cov", "logp", "logp_mp", "sum_safe", "sum_safe_x", "count", "member"):
        assert np.array_equal(getattr(same.rows.train, name), getattr(plain.rows.train, name), equal_nan=True), name
    assert np.array_equal(same.d_hidden, plain.d_hidden) and np.array_equal(same.d_w, plain.d_w)
    assert np.array_equal(same.rows.log_ratio, plain.rows.log_ratio, equal_nan=True)
    # an arbitrary set
    chosen = rng.random(size=(T, V)) < 0.4
    chosen[np.arange(T), z.argmax(1)] = True
    ids[:4] = [np.flatnonzero(chosen[t])[0] for t in range(4)]     # sampled tokens inside the set
    ids[4] = np.flatnonzero(~chosen[4])[0]                         # and one outside: zero row
    res = oracle.dvp_fused_lmhead(bits(hb), bits(wb), bits(zi), ids, rho, g, train_set=chosen.astype(np.uint8))
    h = hb.to(torch.float64).requires_grad_(True)
    w = wb.to(torch.float64).requires_grad_(True)
    pi = torch.softmax(h @ w.t(), dim=-1)
    sel = torch.from_numpy(chosen)
    cover = (pi * sel).sum(dim=-1)                                 # Z of Def. 5.2 for the supplied set
    pi_mp = pi * sel / cover[:, None]
    picked = pi_mp[torch.arange(T), torch.from_numpy(ids)]
    inside = picked > 0
    (torch.log(picked[inside]) * torch.from_numpy(g)[inside]).sum().backward()
    np.testing.assert_allclose(res.rows.train.logp_mp[inside.numpy()], torch.log(picked[inside]).detach().numpy(),
                               atol=1e-12)
    assert np.isneginf(res.rows.train.logp_mp[~inside.numpy()]).all() and not inside[4]
    np.testing.assert_allclose(res.rows.train.log_cov, torch.log(cover).detach().numpy(), atol=1e-12)
    assert np.array_equal(res.rows.train.count, chosen.sum(1))
    np.testing.assert_allclose(res.d_hidden, h.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(res.d_w, w.grad.numpy(), atol=1e-12)
    assert (res.rows.grad[~chosen] == 0).all() and (res.d_hidden[4] == 0).all()


def test_sequence_level_ratio_is_the_product_of_token_ratios_and_veto_rule():
    """Sec. 4.4 (Delta_y = sum of token mismatches), Thm. 5.3 (trajectory ratio =
    product of token ratios), App. A protocol 5 (veto below 1e-4)."""
    rng = np.random.default_rng(31)
    T, V = 60, 50
    z = _rows(rng, T, V, scale=2.0)
    zi = z + rng.normal(size=z.shape) * 0.05
    ids = rng.integers(0, V, size=T)
    tr = oracle.dvp_rows_f64(z, ids, 1e-2).train
    inf = oracle.dvp_rows_f64(zi, ids, 1e-2).train
    with np.errstate(invalid="ignore"):
        lr = np.where(tr.member == 0, -np.inf, np.where(inf.member == 0, np.inf, tr.logp_mp - inf.logp_mp))
    off = np.array([0, 7, 7, 30, 60])                       # one empty sequence
    res = oracle.dvp_sequences(lr, off, 1e-4)
    with open(os.path.join(GOLDEN, "paper_constants.txt")) as f:
        veto_printed = [float(ln.split()[2]) for ln in f if ln.startswith("veto_threshold")][0]
    for s in range(4):
        seg = slice(off[s], off[s + 1])
        w = np.where(tr.member[seg] == 0, 0.0, np.exp(lr[seg]))       # token weights pi^mp_t / pi^mp_i
        prod = np.prod(w)
        if res.n_zero_weight[s] == 0 and np.isfinite(res.seq_log_ratio[s]):
            assert math.exp(res.seq_log_ratio[s]) == pytest.approx(prod, rel=1e-12)
            both = (tr.member[seg] == 1) & (inf.member[seg] == 1)
            direct = math.fsum(tr.logp_mp[seg][both]) - math.fsum(inf.logp_mp[seg][both])
            assert res.seq_log_ratio[s] == pytest.approx(direct, abs=1e-12)
        elif res.n_zero_weight[s] > 0:
            assert prod == 0.0 and res.seq_log_ratio[s] == -np.inf
        assert res.veto[s] == int((w < veto_printed).any())
        assert res.n_valid[s] == off[s + 1] - off[s]
        assert res.n_zero_weight[s] == int((tr.member[seg] == 0).sum())
    assert res.seq_log_ratio[1] == 0.0 and res.veto[1] == 0 and res.min_log_ratio[1] == np.inf
    # the veto threshold acts on the weight, not on its logarithm
    res = oracle.dvp_sequences(np.array([0.0, math.log(1.01e-4), 0.1, math.log(0.99e-4), np.nan]),
                               np.array([0, 3, 5]), 1e-4)
    assert res.veto.tolist() == [0, 1] and res.n_valid.tolist() == [3, 1]


@pytest.mark.parametrize("dt,code", [(torch.bfloat16, oracle.BF16), (torch.float32, oracle.F32)])
def test_listing_variant_against_its_closed_form(dt, code):
    """The finite-mask variant (App. A, Sec. 5.5 "-50.0 in BF16"): pruned tokens keep the
    probability mass of the mask value.  Stated here as a closed form, not as masked logits:
    with K the kept set and n the number of pruned tokens,
        p(a) = e^{z_a} / (sum_K e^{z_k} + n e^{mv}) for a in K,  e^{mv} / (same) otherwise.
    The threshold is formed in the logits' own type: ln(rho) rounded to it, added to the row
    maximum in float32, the sum rounded to the type again (an eager tensor expression of that
    type does exactly this, which the first assertion checks against torch itself)."""
    rng = np.random.default_rng(41)
    T, V, rho, mv = 10, 400, 1e-2, -50.0
    logits = torch.from_numpy((rng.normal(size=(T, V)) * 3).astype(np.float32)).to(dt)
    top = logits.max(dim=-1).values
    threshold = (top.to(torch.float32) + torch.tensor(math.log(rho)).to(dt).to(torch.float32)).to(dt)[:, None]
    assert torch.equal(threshold[:, 0], top + math.log(rho)) and threshold.dtype == dt
    kept = logits >= threshold
    pruned = ~kept
    z64 = logits.to(torch.float64).requires_grad_(True)
    mass_mv = math.exp(torch.tensor(mv, dtype=dt).to(torch.float64).item())
    ids = rng.integers(0, V, size=T)
    ids[:3] = logits.float().numpy().argmax(1)[:3]
    ids[3] = int(np.flatnonzero(pruned[3].numpy())[0])          # a pruned sampled token
    g = torch.from_numpy(rng.normal(size=T))
    shift = z64.detach().max(dim=-1, keepdim=True).values       # sums formed relative to the maximum
    total = (torch.exp(z64 - shift) * kept).sum(dim=-1) + pruned.sum(dim=-1) * mass_mv * torch.exp(-shift[:, 0])
    picked = z64[torch.arange(T), torch.from_numpy(ids)]
    own = torch.where(kept[torch.arange(T), torch.from_numpy(ids)], torch.exp(picked - shift[:, 0]),
                      mass_mv * torch.exp(-shift[:, 0]))
    logp = torch.log(own / total)
    (logp * g).sum().backward()
    out, grad, thr = oracle.dvp_rows_listing(z64.detach().numpy(), ids, rho, mv, dtype=code, upstream=g.numpy())
    np.testing.assert_array_equal(thr, threshold[:, 0].to(torch.float64).numpy())
    np.testing.assert_array_equal(out["count"], (~pruned).sum(1).numpy())
    np.testing.assert_allclose(out["logp_masked"], logp.detach().numpy(), atol=1e-12)
    np.testing.assert_allclose(grad, z64.grad.numpy(), atol=1e-13)
    assert out["member"][3] == 0 and np.isfinite(out["logp_masked"][3]) and np.abs(grad[3]).sum() > 0
    # with rho small enough that nothing is pruned it is the plain log-softmax
    out0, _, _ = oracle.dvp_rows_listing(z64.detach().numpy(), ids, 1e-30, mv, dtype=code)
    ref = torch.log_softmax(z64.detach(), dim=-1)[torch.arange(T), torch.from_numpy(ids)].numpy()
    np.testing.assert_allclose(out0["logp_masked"], ref, atol=1e-12)
    # and it differs from the exact -inf semantics by the mass of the masked tokens
    exact = oracle.dvp_rows_f64(z64.detach().numpy(), ids, rho)
    kept = out["member"] == 1
    extra = np.log1p((V - out["count"]) * np.exp(mv - exact.train.lse_safe))
    np.testing.assert_allclose((exact.train.logp_mp - out["logp_masked"])[kept], extra[kept], atol=1e-9)


def test_monitoring_quantities_against_library_routines_and_invariants():
    """Sec. 6 monitors the KL divergence between the inference and training
    policies; the oracle's values are pinned to torch's kl_div and Categorical
    entropy, to KL >= 0 with equality for equal rows, to shift invariance, and to
    the second-order value Var_pi(eps) / 2 for a small perturbation eps."""
    rng = np.random.default_rng(43)
    T, V = 9, 700
    z = _rows(rng, T, V, scale=3.0)
    zi = z + rng.normal(size=z.shape) * 0.3
    got = oracle.dvp_monitor(z, zi)
    lt, li = torch.log_softmax(torch.from_numpy(z), -1), torch.log_softmax(torch.from_numpy(zi), -1)
    kl_it = torch.nn.functional.kl_div(lt, li, log_target=True, reduction="none").sum(-1).numpy()
    kl_ti = torch.nn.functional.kl_div(li, lt, log_target=True, reduction="none").sum(-1).numpy()
    np.testing.assert_allclose(got[:, 0], kl_it, atol=1e-12)
    np.testing.assert_allclose(got[:, 1], kl_ti, atol=1e-12)
    np.testing.assert_allclose(got[:, 2], torch.distributions.Categorical(logits=torch.from_numpy(z)).entropy().numpy(), atol=1e-12)
    np.testing.assert_allclose(got[:, 3], torch.distributions.Categorical(logits=torch.from_numpy(zi)).entropy().numpy(), atol=1e-12)
    assert (got[:, :2] > 0).all() and (got[:, 2:] <= math.log(V) + 1e-12).all()
    same = oracle.dvp_monitor(z, z + 7.5)                      # softmax ignores a shift of the row
    np.testing.assert_allclose(same[:, :2], 0.0, atol=1e-12)
    np.testing.assert_allclose(same[:, 2], same[:, 3], atol=1e-12)
    eps = rng.normal(size=z.shape) * 1e-3
    small = oracle.dvp_monitor(z, z + eps)
    pi = torch.softmax(torch.from_numpy(z), -1).numpy()
    var = (pi * eps ** 2).sum(1) - (pi * eps).sum(1) ** 2
    np.testing.assert_allclose(small[:, 0], var / 2, rtol=5e-3)
    flat = oracle.dvp_monitor(np.zeros((1, 64)), np.zeros((1, 64)))
    assert flat[0, 2] == pytest.approx(math.log(64), abs=1e-14)


@pytest.mark.parametrize("kind,lo,hi", [(oracle.WEIGHT_RATIO, 0.0, math.inf), (oracle.WEIGHT_TRUNCATE, 0.0, 1.05),
                                        (oracle.WEIGHT_MASK, 0.9, 1.1)])
def test_importance_weighted_gradient_matches_autograd_with_a_detached_weight(kind, lo, hi):
    """Thm. 5.3's estimator per token: weight pi^mp_train(a) / pi^mp_infer(a), formed as the
    exponential of the difference of log-probabilities (App. A protocol 4) and held constant,
    times grad log pi^mp_train(a); truncated / masked as the comparison methods of Sec. 6 do.
    Checked against autograd of sum_t c_t * stopgrad(w_t) * log pi^mp_train(a_t)."""
    rng = np.random.default_rng(17)
    T, V, rho = 40, 300, 1e-3
    z_np = _rows(rng, T, V, scale=3.0)
    zi_np = z_np + rng.normal(size=z_np.shape) * 0.15
    z = torch.from_numpy(z_np).requires_grad_(True)
    zi = torch.from_numpy(zi_np)
    c = torch.from_numpy(rng.normal(size=T))
    ids_np = rng.integers(0, V, size=T)
    ids_np[:30] = z_np.argsort(1)[np.arange(30), -1 - rng.integers(0, 3, size=30)]     # mostly likely tokens
    ids = torch.from_numpy(ids_np)

    def masked_logp(x):
        return _log_pi_mp(x, rho)[torch.arange(T), ids]

    lt, li = masked_logp(z), masked_logp(zi)
    with torch.no_grad():
        ratio = torch.exp(lt - li)                       # +inf when only the inference side pruned a
        ratio = torch.where(torch.isfinite(lt), ratio, torch.zeros_like(ratio))   # ratio zero when train pruned a
        if kind == oracle.WEIGHT_TRUNCATE:
            w = torch.clamp(ratio, max=hi)
        elif kind == oracle.WEIGHT_MASK:
            w = torch.where((ratio >= lo) & (ratio <= hi), ratio, torch.zeros_like(ratio))
        else:
            w = ratio
    live = torch.isfinite(lt) & torch.isfinite(w) & (w != 0)
    (c[live] * w[live] * lt[live]).sum().backward()
    res = oracle.dvp_rows_f64(z_np, ids_np, rho, upstream=c.numpy(), infer=zi_np, weight_kind=kind,
                              weight_lo=lo, weight_hi=hi)
    fin = np.isfinite(w.numpy())
    np.testing.assert_allclose(res.weight[fin], w.numpy()[fin], rtol=1e-12, atol=0)
    assert np.array_equal(np.isinf(res.weight), np.isinf(w.numpy()))
    rows = live.numpy() | (w.numpy() == 0) | ~np.isfinite(lt.detach().numpy())
    np.testing.assert_allclose(res.grad[rows], z.grad.numpy()[rows], atol=1e-13, rtol=1e-11)
    assert (res.grad[w.numpy() == 0] == 0).all()
    # the three kinds really differ on this batch
    assert (ratio > 1.05).any() and (ratio < 0.9).any() and live.sum() >= 10


def test_importance_weight_closed_forms_and_pruned_tokens():
    W = oracle.token_weight
    assert W(0.0, oracle.WEIGHT_NONE) == 1.0 and W(-3.0, oracle.WEIGHT_NONE) == 1.0
    assert W(0.0, oracle.WEIGHT_RATIO) == 1.0
    assert W(math.log(2.0), oracle.WEIGHT_RATIO) == pytest.approx(2.0, rel=1e-15)
    assert W(math.log(2.0), oracle.WEIGHT_TRUNCATE, 0.0, 1.5) == 1.5
    assert W(math.log(0.5), oracle.WEIGHT_TRUNCATE, 0.0, 1.5) == pytest.approx(0.5, rel=1e-15)
    assert W(math.log(2.0), oracle.WEIGHT_MASK, 0.5, 1.5) == 0.0
    assert W(math.log(1.25), oracle.WEIGHT_MASK, 0.5, 1.5) == pytest.approx(1.25, rel=1e-15)
    assert W(math.log(0.25), oracle.WEIGHT_MASK, 0.5, 1.5) == 0.0
    # a outside the training safe set: ratio zero (remark after Thm. 5.3) in every kind
    for kind in (oracle.WEIGHT_RATIO, oracle.WEIGHT_TRUNCATE, oracle.WEIGHT_MASK):
        assert W(-math.inf, kind, 0.5, 1.5) == 0.0
    # a outside the inference safe set only: unbounded ratio
    assert W(math.inf, oracle.WEIGHT_RATIO) == math.inf
    assert W(math.inf, oracle.WEIGHT_TRUNCATE, 0.0, 1.5) == 1.5
    assert W(math.inf, oracle.WEIGHT_MASK, 0.5, 1.5) == 0.0
    # identical policies: every weight is one, the weighted gradient is the plain one
    rng = np.random.default_rng(3)
    z = _rows(rng, 6, 64)
    ids = z.argmax(1)
    g = rng.normal(size=6)
    plain = oracle.dvp_rows_f64(z, ids, 1e-2, upstream=g, infer=z.copy())
    weighted = oracle.dvp_rows_f64(z, ids, 1e-2, upstream=g, infer=z.copy(), weight_kind=oracle.WEIGHT_RATIO)
    assert (weighted.weight == 1.0).all() and np.array_equal(plain.grad, weighted.grad)
    off = oracle.dvp_rows_f64(z, ids, 1e-2, upstream=g, infer=z.copy(), weight_kind=oracle.WEIGHT_MASK,
                              weight_lo=1.5, weight_hi=2.0)
    assert (off.weight == 0.0).all() and (off.grad == 0.0).all()


@pytest.mark.parametrize("kind,lo,hi", [(oracle.WEIGHT_TRUNCATE, 0.0, 1.01), (oracle.WEIGHT_MASK, 0.98, 1.05)])
def test_weighted_fused_lmhead_matches_autograd_through_the_head(kind, lo, hi):
    """The per-token estimator of Thm. 5.3 through a linear LM head: autograd of
    sum_t c_t stopgrad(w_t) ln pi^mp_train(a_t) with z = h W^T gives dH and dW."""
    rng = np.random.default_rng(31)
    T, H, V, rho = 24, 8, 40, 2e-2
    hb = torch.from_numpy(rng.normal(size=(T, H)).astype(np.float32)).to(torch.bfloat16)
    wb = torch.from_numpy((rng.normal(size=(V, H)) * 0.5).astype(np.float32)).to(torch.bfloat16)
    h = hb.to(torch.float64).requires_grad_(True)
    w = wb.to(torch.float64).requires_grad_(True)
    z = h @ w.t()
    zi = (z.detach() + torch.from_numpy(rng.normal(size=(T, V)) * 0.05)).to(torch.bfloat16)
    order = z.detach().numpy().argsort(1)
    ids = order[np.arange(T), -1 - rng.integers(0, 2, size=T)]
    ids[-3:] = order[np.arange(T - 3, T), 0]                     # pruned tokens
    idt = torch.from_numpy(ids)
    c = torch.from_numpy(rng.normal(size=T))

    def masked_logp(x):
        return _log_pi_mp(x, rho)[torch.arange(T), idt]

    lt, li = masked_logp(z), masked_logp(zi.to(torch.float64))
    with torch.no_grad():
        ratio = torch.where(torch.isfinite(lt), torch.exp(lt - li), torch.zeros_like(lt))
        wgt = torch.clamp(ratio, max=hi) if kind == oracle.WEIGHT_TRUNCATE else \
            torch.where((ratio >= lo) & (ratio <= hi), ratio, torch.zeros_like(ratio))
    live = torch.isfinite(lt) & (wgt != 0)
    (c[live] * wgt[live] * lt[live]).sum().backward()
    bits = lambda x: x.view(torch.int16).numpy().view(np.uint16)
    res = oracle.dvp_fused_lmhead(bits(hb), bits(wb), bits(zi), ids, rho, c.numpy(), weight_kind=kind,
                                  weight_lo=lo, weight_hi=hi)
    np.testing.assert_allclose(res.rows.weight, wgt.numpy(), rtol=1e-11, atol=0)
    np.testing.assert_allclose(res.d_hidden, h.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(res.d_w, w.grad.numpy(), atol=1e-12)
    assert live.sum() >= 8 and (wgt == 0).sum() >= 3 and (ratio != wgt).any()
