"""The bounds-checking build of the library (every shared-memory index of the row kernels'
on-chip tables and every global element offset compared with its extent, reported through a
status word, nothing traps) run over small parity cases: the results must be those of the
oracle, and no check may have failed.  It stands in for a memory checker."""
import dataclasses

import pytest
import torch

from paper_2512_23087_b200 import binding, inputs

import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
W = inputs.WORKLOADS


@pytest.fixture()
def checked():
    with binding.bounds_checking_library():
        assert binding.dvp_debug_bounds_status() == 0
        yield
        assert binding.dvp_debug_bounds_status() == 0, "an index was out of range"


def test_the_ordinary_build_says_it_has_no_checks():
    with pytest.raises(binding.DvpError) as e:
        binding.dvp_debug_bounds_status()
    assert e.value.status == binding.DVP_ERR_UNSUPPORTED


@pytest.mark.parametrize("hint", [0, 256 | (2 << 16) | (2 << 24), 256 | (2 << 16) | (4 << 24), 3 << 16, 4 << 16,
                                  0x11 << 16, 64, 512],
                         ids=["default", "cluster2", "cluster4", "store3", "store4", "resident", "64threads",
                              "512threads"])
@pytest.mark.parametrize("dtype,V,ld", [("bf16", 151936, 151936), ("bf16", 33000, 33008), ("f16", 4097, 4112),
                                        ("f32", 20000, 20000), ("bf16", 1003, 1008), ("f32", 7, 8)])
def test_row_kernels_under_the_checks(checked, dtype, V, ld, hint):
    w = dataclasses.replace(W["c2_bf16_fwdbwd"], dtype=dtype)
    batch = inputs.make_rows(w, seed=V, device=DEV, T=12, V=V, ld=ld)
    for rho in (1e-4, 1e-2, 0.0):
        res = binding.dvp_forward(batch.train, batch.ids, rho, infer_logits=batch.infer, upstream=batch.upstream,
                                  want_mask=True, launch_hint=hint)
        grad2 = binding.dvp_backward(batch.train, batch.ids, rho, batch.upstream, res)
        torch.cuda.synchronize()
        report, want = parity.check_forward(res, batch, rho, V, True)
        parity.check_grad(grad2, want.grad, report, label="standalone")
    binding.dvp_monitor(batch.train, batch.infer)


def test_weighted_and_finite_mask_calls_under_the_checks(checked):
    w = W["c2_bf16_fwdbwd"]
    batch = inputs.make_rows(w, seed=3, device=DEV, T=16, V=40000)
    for hint in (0, 3 << 16):
        binding.dvp_forward(batch.train, batch.ids, 1e-3, infer_logits=batch.infer, upstream=batch.upstream,
                            weight_kind=binding.DVP_WEIGHT_TRUNCATE, weight_hi=1.02, launch_hint=hint)
        binding.dvp_forward(batch.train, batch.ids, 1e-3, infer_logits=batch.infer, upstream=batch.upstream,
                            mask_value=-50.0, threshold_in_logits_dtype=True, launch_hint=hint)


def test_fused_entry_under_the_checks(checked):
    """The panel's row kernel (4-byte logits, row maxima handed over by the contraction)."""
    fw = W["c4_fused_lmhead"]
    fb = inputs.make_fused(fw, seed=0, device=DEV, T=200, H=256, V=3000)
    r = binding.dvp_fused_lmhead_forward_backward(fb.hidden, fb.w_vocab, fb.ids, 1e-2, fb.upstream,
                                                  infer_logits=fb.infer, panel_rows=128)
    torch.cuda.synchronize()
    assert r.workspace[:4].view(torch.int32).item() == 0
