"""ctypes binding of the C ABI in ``include/dvp.h``.

Argument marshalling only: tensors are turned into raw device pointers and
sizes, outputs are allocated with torch, and every step of the computation
runs in the CUDA library.  There is no fallback: if ``libdvp_b200.so`` has not
been built, the first call raises.
"""
from __future__ import annotations

import contextlib
import ctypes
import os
from types import SimpleNamespace

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdvp_b200.so")
BOUNDS_LIB_PATH = os.path.join(_HERE, "libdvp_b200_bounds.so")   # the bounds-checking build

DVP_OK, DVP_ERR_INVALID_ARG, DVP_ERR_UNSUPPORTED, DVP_ERR_WORKSPACE, DVP_ERR_CUDA = range(5)
DVP_F32, DVP_BF16, DVP_F16 = 0, 1, 2
DVP_ID_I64, DVP_ID_I32 = 0, 1
DVP_FLAG_IN_TRAIN, DVP_FLAG_IN_INFER, DVP_FLAG_NO_ID, DVP_FLAG_BAD_ID = 1, 2, 64, 128
DVP_ENTRY_FORWARD, DVP_ENTRY_BACKWARD, DVP_ENTRY_FUSED_LMHEAD = 0, 1, 2
DVP_STATIC_WORKSPACE_BYTES = 32 * 1024 * 1024
DVP_MODE_FINITE_MASK, DVP_MODE_THRESHOLD_IN_LOGITS_DTYPE = 1, 2
DVP_WEIGHT_NONE, DVP_WEIGHT_RATIO, DVP_WEIGHT_TRUNCATE, DVP_WEIGHT_MASK = 0, 1, 2, 3

EXPORTS = ("dvp_forward", "dvp_backward", "dvp_fused_lmhead_forward_backward",
           "dvp_fused_lmhead_forward_backward_static", "dvp_sequence_aggregate", "dvp_monitor", "dvp_gemm_tn",
           "dvp_workspace_bytes", "dvp_status_string", "dvp_version", "dvp_row_wait_status",
           "dvp_static_workspace_status", "dvp_debug_bounds_status")

_DTYPES = {torch.float32: DVP_F32, torch.bfloat16: DVP_BF16, torch.float16: DVP_F16}
_SIDE_FIELDS = ("max", "lse", "lse_safe", "logp", "logp_mp", "comp_mp", "count", "mask", "log_cov")


class DvpError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


class SideOut(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in _SIDE_FIELDS]


class ForwardArgs(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("logits_dtype", ctypes.c_int32),
        ("grad_dtype", ctypes.c_int32),
        ("id_dtype", ctypes.c_int32),
        ("T", ctypes.c_int64),
        ("V", ctypes.c_int64),
        ("ld_train", ctypes.c_int64),
        ("ld_infer", ctypes.c_int64),
        ("ld_grad", ctypes.c_int64),
        ("rho", ctypes.c_double),
        ("train_logits", ctypes.c_void_p),
        ("infer_logits", ctypes.c_void_p),
        ("ids", ctypes.c_void_p),
        ("upstream", ctypes.c_void_p),
        ("grad_train", ctypes.c_void_p),
        ("train", SideOut),
        ("infer", SideOut),
        ("log_ratio", ctypes.c_void_p),
        ("flags", ctypes.c_void_p),
        ("stream", ctypes.c_void_p),
        ("launch_hint", ctypes.c_uint32),
        ("mode", ctypes.c_uint32),
        ("mask_value", ctypes.c_float),
        ("weight_kind", ctypes.c_uint32),
        ("weight_lo", ctypes.c_float),
        ("weight_hi", ctypes.c_float),
        ("weight_out", ctypes.c_void_p),
    ]


class BackwardArgs(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("logits_dtype", ctypes.c_int32),
        ("grad_dtype", ctypes.c_int32),
        ("id_dtype", ctypes.c_int32),
        ("T", ctypes.c_int64),
        ("V", ctypes.c_int64),
        ("ld_train", ctypes.c_int64),
        ("ld_grad", ctypes.c_int64),
        ("rho", ctypes.c_double),
        ("train_logits", ctypes.c_void_p),
        ("ids", ctypes.c_void_p),
        ("upstream", ctypes.c_void_p),
        ("max_t", ctypes.c_void_p),
        ("lse_safe_t", ctypes.c_void_p),
        ("comp_mp_t", ctypes.c_void_p),
        ("flags", ctypes.c_void_p),
        ("grad_train", ctypes.c_void_p),
        ("stream", ctypes.c_void_p),
        ("launch_hint", ctypes.c_uint32),
        ("mode", ctypes.c_uint32),
        ("mask_value", ctypes.c_float),
        ("reserved_", ctypes.c_uint32),
    ]


class FusedArgs(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("id_dtype", ctypes.c_int32),
        ("T", ctypes.c_int64),
        ("H", ctypes.c_int64),
        ("V", ctypes.c_int64),
        ("ld_hidden", ctypes.c_int64),
        ("ld_w", ctypes.c_int64),
        ("ld_infer", ctypes.c_int64),
        ("ld_dh", ctypes.c_int64),
        ("ld_dw", ctypes.c_int64),
        ("rho", ctypes.c_double),
        ("hidden", ctypes.c_void_p),
        ("w_vocab", ctypes.c_void_p),
        ("infer_logits", ctypes.c_void_p),
        ("ids", ctypes.c_void_p),
        ("upstream", ctypes.c_void_p),
        ("d_hidden", ctypes.c_void_p),
        ("d_w", ctypes.c_void_p),
        ("accumulate_dw", ctypes.c_int32),
        ("panel_rows", ctypes.c_int32),
        ("train", SideOut),
        ("infer", SideOut),
        ("log_ratio", ctypes.c_void_p),
        ("flags", ctypes.c_void_p),
        ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_size_t),
        ("stream", ctypes.c_void_p),
        ("weight_kind", ctypes.c_uint32),
        ("weight_lo", ctypes.c_float),
        ("weight_hi", ctypes.c_float),
        ("weight_out", ctypes.c_void_p),
    ]


class SequenceArgs(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("reserved_", ctypes.c_uint32),
        ("T", ctypes.c_int64),
        ("S", ctypes.c_int64),
        ("seq_offsets", ctypes.c_void_p),
        ("log_ratio", ctypes.c_void_p),
        ("veto_threshold", ctypes.c_double),
        ("seq_log_ratio", ctypes.c_void_p),
        ("min_log_ratio", ctypes.c_void_p),
        ("n_valid", ctypes.c_void_p),
        ("n_zero_weight", ctypes.c_void_p),
        ("veto", ctypes.c_void_p),
        ("stream", ctypes.c_void_p),
        ("log_cov", ctypes.c_void_p),
        ("min_cov", ctypes.c_void_p),
        ("mean_cov", ctypes.c_void_p),
    ]


class MonitorArgs(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("logits_dtype", ctypes.c_int32),
        ("T", ctypes.c_int64),
        ("V", ctypes.c_int64),
        ("ld_train", ctypes.c_int64),
        ("ld_infer", ctypes.c_int64),
        ("train_logits", ctypes.c_void_p),
        ("infer_logits", ctypes.c_void_p),
        ("kl_infer_train", ctypes.c_void_p),
        ("kl_train_infer", ctypes.c_void_p),
        ("entropy_train", ctypes.c_void_p),
        ("entropy_infer", ctypes.c_void_p),
        ("stream", ctypes.c_void_p),
    ]


_lib = None


def load_library() -> ctypes.CDLL:
    """Load ``libdvp_b200.so``; raises if it is missing (there is no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2512_23087_b200.build`; "
                "this package has no CPU or PyTorch fallback")
        lib = ctypes.CDLL(LIB_PATH)
        lib.dvp_forward.argtypes = [ctypes.POINTER(ForwardArgs)]
        lib.dvp_forward.restype = ctypes.c_int
        lib.dvp_backward.argtypes = [ctypes.POINTER(BackwardArgs)]
        lib.dvp_backward.restype = ctypes.c_int
        lib.dvp_fused_lmhead_forward_backward.argtypes = [ctypes.POINTER(FusedArgs)]
        lib.dvp_fused_lmhead_forward_backward.restype = ctypes.c_int
        lib.dvp_fused_lmhead_forward_backward_static.argtypes = [ctypes.POINTER(FusedArgs)]
        lib.dvp_fused_lmhead_forward_backward_static.restype = ctypes.c_int
        lib.dvp_sequence_aggregate.argtypes = [ctypes.POINTER(SequenceArgs)]
        lib.dvp_sequence_aggregate.restype = ctypes.c_int
        lib.dvp_monitor.argtypes = [ctypes.POINTER(MonitorArgs)]
        lib.dvp_monitor.restype = ctypes.c_int
        lib.dvp_gemm_tn.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_int64,
                                    ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                                    ctypes.c_int64, ctypes.c_int32, ctypes.c_float, ctypes.c_int32,
                                    ctypes.c_void_p, ctypes.c_void_p]
        lib.dvp_gemm_tn.restype = ctypes.c_int
        lib.dvp_workspace_bytes.argtypes = [ctypes.c_int, ctypes.c_void_p]
        lib.dvp_workspace_bytes.restype = ctypes.c_size_t
        lib.dvp_status_string.argtypes = [ctypes.c_int]
        lib.dvp_status_string.restype = ctypes.c_char_p
        lib.dvp_version.restype = ctypes.c_int
        lib.dvp_row_wait_status.argtypes = [ctypes.POINTER(ctypes.c_uint32)]
        lib.dvp_row_wait_status.restype = ctypes.c_int
        lib.dvp_static_workspace_status.argtypes = [ctypes.POINTER(ctypes.c_uint32)]
        lib.dvp_static_workspace_status.restype = ctypes.c_int
        lib.dvp_debug_bounds_status.argtypes = [ctypes.POINTER(ctypes.c_uint32)]
        lib.dvp_debug_bounds_status.restype = ctypes.c_int
        _lib = lib
    return _lib


@contextlib.contextmanager
def bounds_checking_library():
    """Inside the block every call of this module goes to the bounds-checking build of the
    library (``python -m paper_2512_23087_b200.build --debug-bounds``), whose kernels compare
    every index of their on-chip tables and every global offset with its extent;
    ``dvp_debug_bounds_status()`` then tells whether any check failed."""
    global _lib, LIB_PATH
    if not os.path.exists(BOUNDS_LIB_PATH):
        raise RuntimeError(f"{BOUNDS_LIB_PATH} is missing: build it with "
                           "`python -m paper_2512_23087_b200.build --debug-bounds`")
    saved = (_lib, LIB_PATH)
    _lib, LIB_PATH = None, BOUNDS_LIB_PATH
    try:
        yield load_library()
    finally:
        _lib, LIB_PATH = saved


def dvp_debug_bounds_status() -> int:
    """Waits for the current device and returns (and clears) the word into which the
    bounds-checking build ORs a code for every index it found out of range; raises
    ``DvpError(DVP_ERR_UNSUPPORTED)`` on the ordinary build, which has no checks."""
    out = ctypes.c_uint32(0)
    st = load_library().dvp_debug_bounds_status(ctypes.byref(out))
    if st != DVP_OK:
        raise DvpError(st, "dvp_debug_bounds_status")
    return int(out.value)


def status_string(status: int) -> str:
    return load_library().dvp_status_string(int(status)).decode()


def _ptr(t: torch.Tensor | None):
    return None if t is None else t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def _check_matrix(name: str, x: torch.Tensor):
    if x.dim() != 2 or x.stride(1) != 1:
        raise ValueError(f"{name} must be 2-D with unit inner stride")
    if not x.is_cuda:
        raise ValueError(f"{name} must live on a CUDA device")


def _side(device, T: int, V: int, want_mask: bool):
    o = SimpleNamespace()
    for n in ("max", "lse", "lse_safe", "logp", "logp_mp", "comp_mp", "log_cov"):
        setattr(o, n, torch.empty(T, dtype=torch.float32, device=device))
    o.count = torch.empty(T, dtype=torch.int32, device=device)
    o.mask = torch.empty(T, (V + 31) // 32, dtype=torch.int32, device=device) if want_mask else None
    s = SideOut(*(_ptr(getattr(o, n)) for n in _SIDE_FIELDS))
    return o, s


def _id_dtype(ids: torch.Tensor) -> int:
    if ids.dtype == torch.int64:
        return DVP_ID_I64
    if ids.dtype == torch.int32:
        return DVP_ID_I32
    raise TypeError("ids must be int64 or int32")


def dvp_forward(train_logits: torch.Tensor, ids: torch.Tensor, rho: float, *,
                infer_logits: torch.Tensor | None = None, upstream: torch.Tensor | None = None,
                grad_train: torch.Tensor | None = None, grad_dtype: torch.dtype | None = None,
                want_mask: bool = False, stream=None, launch_hint: int = 0, out=None,
                mask_value: float | None = None, threshold_in_logits_dtype: bool = False,
                weight_kind: int = DVP_WEIGHT_NONE, weight_lo: float = 0.0, weight_hi: float = float("inf")):
    """Pruned log-probabilities of the sampled tokens for the training and the
    inference logits (Def. 5.1, Def. 5.2), their log-ratio, and, when
    ``upstream`` is given, dLoss/dlogits (Prop. 5.4) in the same launch.

    ``mask_value`` (finite) switches to the App. A listing's semantics: pruned
    logits are replaced by it instead of by -inf; ``threshold_in_logits_dtype``
    rounds the threshold the way an eager tensor expression would.
    ``weight_kind`` (``DVP_WEIGHT_*``) multiplies each token's upstream gradient
    inside the kernel by the token's importance weight e^{log_ratio}, plain,
    truncated at ``weight_hi`` or masked outside [``weight_lo``, ``weight_hi``]
    (Thm. 5.3 per token); the weights used come back as ``weight``.

    Returns a namespace with ``train`` / ``infer`` (per-token tensors),
    ``log_ratio``, ``flags`` and ``grad_train``.  Pass the namespace of an
    earlier call as ``out`` to reuse its buffers.
    """
    lib = load_library()
    _check_matrix("train_logits", train_logits)
    T, V = train_logits.shape
    dev = train_logits.device
    a = ForwardArgs()
    a.struct_size = ctypes.sizeof(ForwardArgs)
    a.logits_dtype = _DTYPES[train_logits.dtype]
    a.id_dtype = _id_dtype(ids)
    a.T, a.V, a.rho = T, V, float(rho)
    a.ld_train = train_logits.stride(0)
    a.train_logits = _ptr(train_logits)
    a.ids = _ptr(ids)
    res = out if out is not None else SimpleNamespace(train=None, infer=None, log_ratio=None,
                                                      flags=None, grad_train=None)
    if out is None:
        res.train, res._train_struct = _side(dev, T, V, want_mask)
        res.flags = torch.empty(T, dtype=torch.uint8, device=dev)
    a.train = res._train_struct
    a.flags = _ptr(res.flags)
    if infer_logits is not None:
        _check_matrix("infer_logits", infer_logits)
        if infer_logits.dtype != train_logits.dtype or infer_logits.shape != train_logits.shape:
            raise ValueError("infer_logits must match train_logits in dtype and shape")
        a.infer_logits = _ptr(infer_logits)
        a.ld_infer = infer_logits.stride(0)
        if out is None:
            res.infer, res._infer_struct = _side(dev, T, V, want_mask)
            res.log_ratio = torch.empty(T, dtype=torch.float32, device=dev)
        a.infer = res._infer_struct
        a.log_ratio = _ptr(res.log_ratio)
    if upstream is not None:
        if upstream.dtype != torch.float32:
            raise TypeError("upstream must be float32")
        if grad_train is None:
            grad_train = res.grad_train
        if grad_train is None:
            grad_train = torch.empty(T, V, dtype=grad_dtype or train_logits.dtype, device=dev)
        _check_matrix("grad_train", grad_train)
        res.grad_train = grad_train
        a.upstream = _ptr(upstream)
        a.grad_train = _ptr(grad_train)
        a.grad_dtype = _DTYPES[grad_train.dtype]
        a.ld_grad = grad_train.stride(0)
    a.stream = _stream(stream)
    a.launch_hint = launch_hint
    a.mode = (DVP_MODE_FINITE_MASK if mask_value is not None else 0) | \
        (DVP_MODE_THRESHOLD_IN_LOGITS_DTYPE if threshold_in_logits_dtype else 0)
    a.mask_value = float(mask_value) if mask_value is not None else 0.0
    a.weight_kind = int(weight_kind)
    a.weight_lo, a.weight_hi = float(weight_lo), float(weight_hi)
    if weight_kind != DVP_WEIGHT_NONE:
        if getattr(res, "weight", None) is None:
            res.weight = torch.empty(T, dtype=torch.float32, device=dev)
        a.weight_out = _ptr(res.weight)
    st = lib.dvp_forward(ctypes.byref(a))
    if st != DVP_OK:
        raise DvpError(st, "dvp_forward")
    return res


def dvp_backward(train_logits: torch.Tensor, ids: torch.Tensor, rho: float, upstream: torch.Tensor,
                 saved, *, grad_train: torch.Tensor | None = None,
                 grad_dtype: torch.dtype | None = None, use_comp: bool = True, stream=None,
                 launch_hint: int = 0, mask_value: float | None = None,
                 threshold_in_logits_dtype: bool = False) -> torch.Tensor:
    """dLoss/dlogits from the vectors an earlier ``dvp_forward`` saved
    (``saved`` = its result namespace) and a per-token upstream gradient."""
    lib = load_library()
    _check_matrix("train_logits", train_logits)
    T, V = train_logits.shape
    if grad_train is None:
        grad_train = torch.empty(T, V, dtype=grad_dtype or train_logits.dtype,
                                 device=train_logits.device)
    _check_matrix("grad_train", grad_train)
    a = BackwardArgs()
    a.struct_size = ctypes.sizeof(BackwardArgs)
    a.logits_dtype = _DTYPES[train_logits.dtype]
    a.grad_dtype = _DTYPES[grad_train.dtype]
    a.id_dtype = _id_dtype(ids)
    a.T, a.V, a.rho = T, V, float(rho)
    a.ld_train, a.ld_grad = train_logits.stride(0), grad_train.stride(0)
    a.train_logits, a.ids, a.upstream = _ptr(train_logits), _ptr(ids), _ptr(upstream)
    a.max_t, a.lse_safe_t = _ptr(saved.train.max), _ptr(saved.train.lse_safe)
    a.comp_mp_t = _ptr(saved.train.comp_mp) if use_comp else None
    a.flags = _ptr(saved.flags)
    a.grad_train = _ptr(grad_train)
    a.stream = _stream(stream)
    a.launch_hint = launch_hint
    a.mode = (DVP_MODE_FINITE_MASK if mask_value is not None else 0) | \
        (DVP_MODE_THRESHOLD_IN_LOGITS_DTYPE if threshold_in_logits_dtype else 0)
    a.mask_value = float(mask_value) if mask_value is not None else 0.0
    st = lib.dvp_backward(ctypes.byref(a))
    if st != DVP_OK:
        raise DvpError(st, "dvp_backward")
    return grad_train


def dvp_row_wait_status() -> int:
    """Synchronises the current device and returns (and clears) the status word of
    the resident-row kernel: 0 unless one of its bounded waits ran out."""
    out = ctypes.c_uint32(0)
    st = load_library().dvp_row_wait_status(ctypes.byref(out))
    if st != 0:
        raise DvpError(st, "dvp_row_wait_status")
    return int(out.value)


def dvp_gemm_tn(a: torch.Tensor, b: torch.Tensor, *, alpha: float = 1.0, out: torch.Tensor | None = None,
                accumulate: bool = False, single_block_tiles: bool = False, stream=None,
                a_transposed: bool = False, split_k: bool = False):
    """``out (+)= alpha * a @ b.T`` on the tensor cores; a [m, k] and b [n, k] are
    both bf16 or both f16 with k contiguous, out is float32.  With ``a_transposed``
    ``a`` is given as [k, m] with m contiguous (``out (+)= alpha * a.T @ b.T``).
    ``split_k`` computes every tile as two halves of the k range added into ``out``.
    Returns (out, status) where status is a device int32 that is non-zero if the
    kernel gave up waiting."""
    lib = load_library()
    _check_matrix("a", a)
    _check_matrix("b", b)
    if a.dtype != b.dtype or a.dtype not in (torch.bfloat16, torch.float16):
        raise TypeError("a and b must both be bfloat16 or both float16")
    m, k = (a.shape[1], a.shape[0]) if a_transposed else a.shape
    n = b.shape[0]
    if out is None:
        out = torch.empty(m, n, dtype=torch.float32, device=a.device)
    status = torch.zeros(1, dtype=torch.int32, device=a.device)
    mode = int(accumulate) | (2 if single_block_tiles else 0) | (4 if a_transposed else 0) | (8 if split_k else 0)
    st = lib.dvp_gemm_tn(_ptr(a), a.stride(0), _ptr(b), b.stride(0), _ptr(out), out.stride(0), m, n, k,
                         _DTYPES[a.dtype], float(alpha), mode, _ptr(status), _stream(stream))
    if st != DVP_OK:
        raise DvpError(st, "dvp_gemm_tn")
    return out, status


def dvp_workspace_bytes(entry_point: int, args: ctypes.Structure) -> int:
    return int(load_library().dvp_workspace_bytes(int(entry_point), ctypes.byref(args)))


def _fused_args(hidden, w_vocab, ids, rho, upstream, infer_logits, d_w, accumulate_dw, panel_rows, stream,
                want_mask=False):
    """Marshals the arguments both fused entry points share; creates the output tensors."""
    _check_matrix("hidden", hidden)
    _check_matrix("w_vocab", w_vocab)
    T, H = hidden.shape
    V = w_vocab.shape[0]
    dev = hidden.device
    if hidden.dtype != torch.bfloat16 or w_vocab.dtype != torch.bfloat16:
        raise TypeError("hidden and w_vocab must be bfloat16")
    a = FusedArgs()
    a.struct_size = ctypes.sizeof(FusedArgs)
    a.id_dtype = _id_dtype(ids)
    a.T, a.H, a.V, a.rho = T, H, V, float(rho)
    a.ld_hidden, a.ld_w = hidden.stride(0), w_vocab.stride(0)
    a.hidden, a.w_vocab, a.ids, a.upstream = _ptr(hidden), _ptr(w_vocab), _ptr(ids), _ptr(upstream)
    res = SimpleNamespace(infer=None, log_ratio=None)
    res.train, a.train = _side(dev, T, V, want_mask)
    res.flags = torch.empty(T, dtype=torch.uint8, device=dev)
    a.flags = _ptr(res.flags)
    if infer_logits is not None:
        _check_matrix("infer_logits", infer_logits)
        if infer_logits.dtype != torch.bfloat16:
            raise TypeError("infer_logits must be bfloat16")
        a.infer_logits, a.ld_infer = _ptr(infer_logits), infer_logits.stride(0)
        res.infer, a.infer = _side(dev, T, V, False)
        res.log_ratio = torch.empty(T, dtype=torch.float32, device=dev)
        a.log_ratio = _ptr(res.log_ratio)
    res.d_hidden = torch.empty(T, H, dtype=torch.float32, device=dev)
    res.d_w = d_w if d_w is not None else torch.empty(V, H, dtype=torch.float32, device=dev)
    a.d_hidden, a.ld_dh = _ptr(res.d_hidden), res.d_hidden.stride(0)
    a.d_w, a.ld_dw = _ptr(res.d_w), res.d_w.stride(0)
    a.accumulate_dw = int(accumulate_dw)
    a.panel_rows = int(panel_rows)
    a.stream = _stream(stream)
    return a, res


def dvp_fused_lmhead_forward_backward(hidden: torch.Tensor, w_vocab: torch.Tensor, ids: torch.Tensor,
                                      rho: float, upstream: torch.Tensor, *,
                                      infer_logits: torch.Tensor | None = None,
                                      d_w: torch.Tensor | None = None, accumulate_dw: bool = False,
                                      panel_rows: int = 0, workspace: torch.Tensor | None = None,
                                      stream=None, weight_kind: int = DVP_WEIGHT_NONE,
                                      weight_lo: float = 0.0, weight_hi: float = 1.0, want_mask: bool = False):
    """Pruned log-probabilities and gradients with respect to ``hidden`` and
    ``w_vocab`` with the training logits hidden x w_vocab^T produced panel by
    panel inside the library and never stored as a [T, V] matrix.  With
    ``weight_kind`` (truncate or mask, finite ``weight_hi``) each token's upstream
    gradient is multiplied by its importance weight; the weights come back as
    ``weight``.  ``want_mask`` asks for the packed training safe set."""
    lib = load_library()
    a, res = _fused_args(hidden, w_vocab, ids, rho, upstream, infer_logits, d_w, accumulate_dw, panel_rows,
                         stream, want_mask)
    need = dvp_workspace_bytes(DVP_ENTRY_FUSED_LMHEAD, a)
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=hidden.device)
    res.workspace = workspace
    a.workspace, a.workspace_bytes = _ptr(workspace), workspace.numel() * workspace.element_size()
    a.weight_kind = int(weight_kind)
    if weight_kind != DVP_WEIGHT_NONE:
        a.weight_lo, a.weight_hi = float(weight_lo), float(weight_hi)
        res.weight = torch.empty(hidden.shape[0], dtype=torch.float32, device=hidden.device)
        a.weight_out = _ptr(res.weight)
    st = lib.dvp_fused_lmhead_forward_backward(ctypes.byref(a))
    if st != DVP_OK:
        raise DvpError(st, "dvp_fused_lmhead_forward_backward")
    return res


def dvp_fused_lmhead_forward_backward_static(hidden: torch.Tensor, w_vocab: torch.Tensor,
                                             ids: torch.Tensor, rho: float, upstream: torch.Tensor, *,
                                             infer_logits: torch.Tensor | None = None,
                                             d_w: torch.Tensor | None = None,
                                             accumulate_dw: bool = False, panel_rows: int = 0,
                                             stream=None):
    """The fused LM-head computation for callers that have no device memory of
    their own to offer as a workspace: the library uses a fixed 32 MiB array that
    is part of its image instead, and the call allocates nothing (this wrapper
    only creates the output tensors a caller would normally already own).

    Problems whose workspace would not fit raise ``DvpError`` with
    ``DVP_ERR_WORKSPACE``.  All calls on a GPU share that one array, so calls
    that could overlap on the GPU (different streams) must be ordered by the
    caller.  Make the first call on each device outside any stream capture.
    ``dvp_static_workspace_status`` reads the status word of the last call."""
    lib = load_library()
    a, res = _fused_args(hidden, w_vocab, ids, rho, upstream, infer_logits, d_w, accumulate_dw, panel_rows,
                         stream)
    st = lib.dvp_fused_lmhead_forward_backward_static(ctypes.byref(a))
    if st != DVP_OK:
        raise DvpError(st, "dvp_fused_lmhead_forward_backward_static")
    return res


def dvp_static_workspace_status() -> int:
    """Waits for the current device and returns the status word that the tensor-core kernels of
    the last ``dvp_fused_lmhead_forward_backward_static`` call left in the built-in workspace:
    0 when every kernel finished, non-zero when one gave up waiting (results invalid)."""
    out = ctypes.c_uint32(0)
    st = load_library().dvp_static_workspace_status(ctypes.byref(out))
    if st != DVP_OK:
        raise DvpError(st, "dvp_static_workspace_status")
    return int(out.value)


def dvp_sequence_aggregate(log_ratio: torch.Tensor, seq_offsets: torch.Tensor,
                           veto_threshold: float = 1e-4, stream=None, log_cov: torch.Tensor | None = None):
    """Per-sequence sum and minimum of the token log-ratios, token counts and the
    veto flag (Sec. 4.4, Thm. 5.3, App. A protocol 5).  ``seq_offsets`` is an
    int64 device tensor of S + 1 non-decreasing token offsets.  With ``log_cov``
    (ln Z per token from ``dvp_forward``) also the minimum and the mean of the
    coverage Z over each sequence (Def. 5.2; the Z_min of Prop. 5.5)."""
    lib = load_library()
    if log_ratio.dtype != torch.float32 or seq_offsets.dtype != torch.int64:
        raise TypeError("log_ratio must be float32 and seq_offsets int64")
    S = seq_offsets.numel() - 1
    dev = log_ratio.device
    res = SimpleNamespace(
        seq_log_ratio=torch.empty(S, dtype=torch.float32, device=dev),
        min_log_ratio=torch.empty(S, dtype=torch.float32, device=dev),
        n_valid=torch.empty(S, dtype=torch.int32, device=dev),
        n_zero_weight=torch.empty(S, dtype=torch.int32, device=dev),
        veto=torch.empty(S, dtype=torch.uint8, device=dev))
    a = SequenceArgs()
    a.struct_size = ctypes.sizeof(SequenceArgs)
    a.T, a.S = log_ratio.numel(), S
    a.seq_offsets, a.log_ratio = _ptr(seq_offsets), _ptr(log_ratio)
    a.veto_threshold = float(veto_threshold)
    a.seq_log_ratio, a.min_log_ratio = _ptr(res.seq_log_ratio), _ptr(res.min_log_ratio)
    a.n_valid, a.n_zero_weight, a.veto = _ptr(res.n_valid), _ptr(res.n_zero_weight), _ptr(res.veto)
    a.stream = _stream(stream)
    if log_cov is not None:
        if log_cov.dtype != torch.float32 or log_cov.numel() != log_ratio.numel():
            raise TypeError("log_cov must be float32 with one entry per token")
        res.min_cov = torch.empty(S, dtype=torch.float32, device=dev)
        res.mean_cov = torch.empty(S, dtype=torch.float32, device=dev)
        a.log_cov, a.min_cov, a.mean_cov = _ptr(log_cov), _ptr(res.min_cov), _ptr(res.mean_cov)
    st = lib.dvp_sequence_aggregate(ctypes.byref(a))
    if st != DVP_OK:
        raise DvpError(st, "dvp_sequence_aggregate")
    return res


def dvp_monitor(train_logits: torch.Tensor, infer_logits: torch.Tensor, stream=None):
    """Per-token KL(infer || train), KL(train || infer) and the two entropies over
    the full vocabulary (Sec. 6's stability metric), in nats."""
    lib = load_library()
    _check_matrix("train_logits", train_logits)
    _check_matrix("infer_logits", infer_logits)
    if infer_logits.dtype != train_logits.dtype or infer_logits.shape != train_logits.shape:
        raise ValueError("infer_logits must match train_logits in dtype and shape")
    T, V = train_logits.shape
    dev = train_logits.device
    res = SimpleNamespace(**{n: torch.empty(T, dtype=torch.float32, device=dev)
                             for n in ("kl_infer_train", "kl_train_infer", "entropy_train", "entropy_infer")})
    a = MonitorArgs()
    a.struct_size = ctypes.sizeof(MonitorArgs)
    a.logits_dtype = _DTYPES[train_logits.dtype]
    a.T, a.V = T, V
    a.ld_train, a.ld_infer = train_logits.stride(0), infer_logits.stride(0)
    a.train_logits, a.infer_logits = _ptr(train_logits), _ptr(infer_logits)
    a.kl_infer_train, a.kl_train_infer = _ptr(res.kl_infer_train), _ptr(res.kl_train_infer)
    a.entropy_train, a.entropy_infer = _ptr(res.entropy_train), _ptr(res.entropy_infer)
    a.stream = _stream(stream)
    st = lib.dvp_monitor(ctypes.byref(a))
    if st != DVP_OK:
        raise DvpError(st, "dvp_monitor")
    return res
