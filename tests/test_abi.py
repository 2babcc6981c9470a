"""The C ABI without a GPU: the library builds, loads, exports every symbol the
header declares, its structs have the layout the binding assumes, and argument
errors are reported before any CUDA call."""
import ctypes
import os
import re
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "dvp.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2512_23087_b200 import build, binding
    build.build()
    return binding.load_library()


def _declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dvp_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2512_23087_b200 import binding
    names = _declared_functions()
    assert set(names) == set(binding.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_struct_layout_matches_the_header(tmp_path):
    from paper_2512_23087_b200 import binding
    structs = {"dvp_forward_args": binding.ForwardArgs, "dvp_backward_args": binding.BackwardArgs,
               "dvp_fused_args": binding.FusedArgs, "dvp_side_out": binding.SideOut,
               "dvp_sequence_args": binding.SequenceArgs, "dvp_monitor_args": binding.MonitorArgs}
    lines = []
    for cname, cls in structs.items():
        lines.append(f'printf("{cname} %zu\\n", sizeof({cname}));')
        for fname, _ in cls._fields_:
            lines.append(f'printf("{cname}.{fname} %zu\\n", offsetof({cname}, {fname}));')
    src = tmp_path / "layout.c"
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "dvp.h"\nint main(void){'
                   + "".join(lines) + "return 0;}\n")
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    out = dict(l.split() for l in subprocess.run([str(exe)], capture_output=True, text=True,
                                                  check=True).stdout.splitlines())
    for cname, cls in structs.items():
        assert int(out[cname]) == ctypes.sizeof(cls), cname
        for fname, _ in cls._fields_:
            assert int(out[f"{cname}.{fname}"]) == getattr(cls, fname).offset, f"{cname}.{fname}"


def test_status_strings_and_version(lib):
    from paper_2512_23087_b200 import binding
    assert binding.status_string(0) == "DVP_OK"
    assert binding.status_string(binding.DVP_ERR_WORKSPACE) == "DVP_ERR_WORKSPACE"
    assert binding.status_string(99) == "DVP_ERR_UNKNOWN"
    assert lib.dvp_version() >= 100


def test_argument_errors_are_reported_before_any_launch(lib):
    """None of these reaches a kernel launch, so they run without a GPU."""
    from paper_2512_23087_b200 import binding as b
    a = b.ForwardArgs()
    assert lib.dvp_forward(None) == b.DVP_ERR_INVALID_ARG
    assert lib.dvp_forward(ctypes.byref(a)) == b.DVP_ERR_INVALID_ARG          # struct_size 0
    a.struct_size = ctypes.sizeof(b.ForwardArgs)
    a.T, a.V, a.rho = 4, 16, 0.5
    a.ld_train = 16
    assert lib.dvp_forward(ctypes.byref(a)) == b.DVP_ERR_INVALID_ARG          # no logits
    a.train_logits = 0x1000
    for bad_rho in (-0.1, 1.0001, float("nan")):
        a.rho = bad_rho
        assert lib.dvp_forward(ctypes.byref(a)) == b.DVP_ERR_INVALID_ARG
    a.rho = 0.5
    a.logits_dtype = 7
    assert lib.dvp_forward(ctypes.byref(a)) == b.DVP_ERR_UNSUPPORTED
    a.logits_dtype = b.DVP_BF16
    a.ld_train = 15
    assert lib.dvp_forward(ctypes.byref(a)) == b.DVP_ERR_INVALID_ARG          # ld < V
    a.ld_train = 16
    a.upstream = 0x2000                                                       # upstream without grad
    assert lib.dvp_forward(ctypes.byref(a)) == b.DVP_ERR_INVALID_ARG
    a.upstream = None
    a.log_ratio = 0x3000                                                      # infer outputs without infer
    assert lib.dvp_forward(ctypes.byref(a)) == b.DVP_ERR_INVALID_ARG
    a.log_ratio = None
    a.launch_hint = 33
    assert lib.dvp_forward(ctypes.byref(a)) == b.DVP_ERR_INVALID_ARG
    a.launch_hint = 0
    a.T = 0
    assert lib.dvp_forward(ctypes.byref(a)) == b.DVP_OK                       # empty batch: no-op
    a.T = -1
    assert lib.dvp_forward(ctypes.byref(a)) == b.DVP_ERR_INVALID_ARG
    bw = b.BackwardArgs()
    bw.struct_size = ctypes.sizeof(b.BackwardArgs)
    bw.T, bw.V, bw.rho, bw.ld_train, bw.ld_grad = 2, 8, 0.1, 8, 8
    assert lib.dvp_backward(ctypes.byref(bw)) == b.DVP_ERR_INVALID_ARG        # missing pointers
    fa = b.FusedArgs()
    assert lib.dvp_fused_lmhead_forward_backward(ctypes.byref(fa)) == b.DVP_ERR_INVALID_ARG
    assert lib.dvp_fused_lmhead_forward_backward_static(ctypes.byref(fa)) == b.DVP_ERR_INVALID_ARG
    sa = b.SequenceArgs()
    sa.struct_size = ctypes.sizeof(b.SequenceArgs)
    sa.S, sa.T = 3, 10
    assert lib.dvp_sequence_aggregate(ctypes.byref(sa)) == b.DVP_ERR_INVALID_ARG   # null inputs
    sa.veto_threshold = -1.0
    sa.seq_offsets, sa.log_ratio = 0x1000, 0x2000
    assert lib.dvp_sequence_aggregate(ctypes.byref(sa)) == b.DVP_ERR_INVALID_ARG   # negative threshold
    sa.S = 0
    sa.veto_threshold = 1e-4
    assert lib.dvp_sequence_aggregate(ctypes.byref(sa)) == b.DVP_OK                # no sequences: no-op


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    from paper_2512_23087_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        binding.load_library()


def test_product_package_never_touches_the_oracle():
    pkg = os.path.join(ROOT, "paper_2512_23087_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(import|from)\s+oracle\b", text, flags=re.M), f
                assert "dvp_oracle" not in text, f"{f} reaches into the oracle"
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c", ".h")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2512_23087_b200" not in text and "binding" not in text
