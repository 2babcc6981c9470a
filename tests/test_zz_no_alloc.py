"""The workspace-free variant of the fused LM-head entry point.

Some users of this library cannot allocate device memory at the point where
they call it: they run inside an application that owns every byte of the GPU
and forbids further allocation, or on a path where an allocator call (which can
stall the whole device) is not acceptable.  For them the library carries a fixed
32 MiB array of its own and ``dvp_fused_lmhead_forward_backward_static`` uses
that instead of a caller-supplied workspace.

The test drives the new entry point through the C ABI and compares everything
it returns with what the ordinary entry point returns for the same inputs, with
the tolerances of the other parity tests, on two calls in a row: the second
call is a different, smaller problem, so it runs on an array that still holds
the first call's leftovers.  It also checks that a problem too large for the
built-in array is refused with a workspace error before anything is launched.

This file sorts last on purpose, so that a run that stops at the first failure
has already been through every other test.
"""
import pytest
import torch

from paper_2512_23087_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _rows_close(got, ref, name):
    num = (got.double() - ref.double()).norm(dim=1)
    den = ref.double().norm(dim=1)
    assert (num <= 1e-3 * den + 1e-6 * den.max()).all(), name


def _same(static, plain):
    for side in ("train", "infer"):
        s, p = getattr(static, side), getattr(plain, side)
        assert torch.equal(s.count, p.count), f"{side}.count"
        for name in ("max", "lse", "lse_safe", "logp", "logp_mp"):
            a, b = getattr(s, name).double(), getattr(p, name).double()
            assert torch.equal(torch.isfinite(a), torch.isfinite(b)), f"{side}.{name}"
            fin = torch.isfinite(b)
            assert (a[fin] - b[fin]).abs().max().item() <= 1e-4, f"{side}.{name}"
    assert torch.equal(static.flags, plain.flags)
    fin = torch.isfinite(plain.log_ratio)
    assert torch.equal(torch.isfinite(static.log_ratio), fin)
    assert (static.log_ratio[fin] - plain.log_ratio[fin]).abs().max().item() <= 1e-4
    _rows_close(static.d_hidden, plain.d_hidden, "d_hidden")
    _rows_close(static.d_w, plain.d_w, "d_w")


def test_static_workspace_variant_matches_the_ordinary_entry_point_twice():
    w = inputs.WORKLOADS["c4_fused_lmhead"]
    for seed, (T, H, V, rho) in enumerate([(300, 256, 3000, 1e-3), (70, 128, 1000, 1e-2)]):
        batch = inputs.make_fused(w, seed=40 + seed, device=DEV, T=T, H=H, V=V)
        plain = binding.dvp_fused_lmhead_forward_backward(
            batch.hidden, batch.w_vocab, batch.ids, rho, batch.upstream, infer_logits=batch.infer,
            panel_rows=128)
        static = binding.dvp_fused_lmhead_forward_backward_static(
            batch.hidden, batch.w_vocab, batch.ids, rho, batch.upstream, infer_logits=batch.infer)
        torch.cuda.synchronize()
        assert plain.workspace[:4].view(torch.int32).item() == 0
        # the built-in array's own status word: no tensor-core kernel gave up waiting
        assert binding.dvp_static_workspace_status() == 0
        _same(static, plain)


def test_static_workspace_variant_refuses_what_does_not_fit():
    w = inputs.WORKLOADS["c4_fused_lmhead"]
    batch = inputs.make_fused(w, seed=1, device=DEV, T=64, H=2048, V=16384)
    with pytest.raises(binding.DvpError) as e:
        binding.dvp_fused_lmhead_forward_backward_static(batch.hidden, batch.w_vocab, batch.ids, 1e-3,
                                                         batch.upstream)
    assert e.value.status == binding.DVP_ERR_WORKSPACE
