"""fp64 CPU oracle for Dynamic Vocabulary Pruning -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It never imports the CUDA package and shares nothing with it.

The row arithmetic lives in ``dvp_oracle.c`` (plain C, fp64, one row at a time,
written from Def. 5.1, Def. 5.2, Prop. 5.4, Prop. 5.6 and App. A of the paper).
This module compiles that file with gcc, loads it through ctypes and adds the
LM-head composition of the fused variant, whose matrix products are numpy
float64 ``matmul`` calls (a library primitive used as one step).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dvp_oracle.c")
_LIB = os.path.join(_HERE, "libdvp_oracle.so")

F32, BF16, F16 = 0, 1, 2
# kinds of token-level importance weight (dvp_oracle_token_weight)
WEIGHT_NONE, WEIGHT_RATIO, WEIGHT_TRUNCATE, WEIGHT_MASK = 0, 1, 2, 3


def build(force: bool = False) -> str:
    """Compile the C oracle into a shared object beside its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.run(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-o", tmp, _SRC,
             "-lm", "-lpthread"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


class _Side(ctypes.Structure):
    _fields_ = [
        ("max", ctypes.c_double),
        ("lse", ctypes.c_double),
        ("lse_safe", ctypes.c_double),
        ("log_cov", ctypes.c_double),
        ("logp", ctypes.c_double),
        ("logp_mp", ctypes.c_double),
        ("sum_safe", ctypes.c_double),
        ("sum_safe_x", ctypes.c_double),
        ("tau", ctypes.c_double),
        ("count", ctypes.c_int64),
        ("member", ctypes.c_int32),
        ("pad_", ctypes.c_int32),
    ]


_SIDE_DTYPE = np.dtype(
    [("max", "f8"), ("lse", "f8"), ("lse_safe", "f8"), ("log_cov", "f8"), ("logp", "f8"),
     ("logp_mp", "f8"), ("sum_safe", "f8"), ("sum_safe_x", "f8"), ("tau", "f8"),
     ("count", "i8"), ("member", "i4"), ("pad_", "i4")]
)


class _Batch(ctypes.Structure):
    _fields_ = [
        ("train", ctypes.c_void_p),
        ("infer", ctypes.c_void_p),
        ("dtype", ctypes.c_int32),
        ("want_mask", ctypes.c_int32),
        ("T", ctypes.c_int64),
        ("V", ctypes.c_int64),
        ("ld_train", ctypes.c_int64),
        ("ld_infer", ctypes.c_int64),
        ("ids", ctypes.c_void_p),
        ("upstream", ctypes.c_void_p),
        ("rho", ctypes.c_double),
        ("side_t", ctypes.c_void_p),
        ("side_i", ctypes.c_void_p),
        ("log_ratio", ctypes.c_void_p),
        ("grad", ctypes.c_void_p),
        ("mask_t", ctypes.c_void_p),
        ("mask_i", ctypes.c_void_p),
        ("weight_kind", ctypes.c_int32),
        ("pad_", ctypes.c_int32),
        ("weight_lo", ctypes.c_double),
        ("weight_hi", ctypes.c_double),
        ("weight", ctypes.c_void_p),
    ]


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.dvp_oracle_batch.argtypes = [ctypes.POINTER(_Batch), ctypes.c_int]
        lib.dvp_oracle_batch.restype = ctypes.c_int
        lib.dvp_oracle_side.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                        ctypes.c_double, ctypes.c_void_p, ctypes.c_void_p]
        lib.dvp_oracle_side.restype = None
        lib.dvp_oracle_side_grad.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                             ctypes.c_double, ctypes.c_void_p, ctypes.c_void_p]
        lib.dvp_oracle_side_grad.restype = None
        lib.dvp_oracle_side_given_set.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                                  ctypes.c_void_p, ctypes.c_void_p]
        lib.dvp_oracle_side_given_set.restype = None
        lib.dvp_oracle_side_grad_given_set.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                                       ctypes.c_double, ctypes.c_void_p, ctypes.c_void_p,
                                                       ctypes.c_void_p]
        lib.dvp_oracle_side_grad_given_set.restype = None
        lib.dvp_oracle_log_ratio.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
        lib.dvp_oracle_log_ratio.restype = ctypes.c_double
        lib.dvp_oracle_token_weight.argtypes = [ctypes.c_double, ctypes.c_int, ctypes.c_double, ctypes.c_double]
        lib.dvp_oracle_token_weight.restype = ctypes.c_double
        assert lib.dvp_oracle_sizeof_side() == ctypes.sizeof(_Side) == _SIDE_DTYPE.itemsize
        assert lib.dvp_oracle_sizeof_batch() == ctypes.sizeof(_Batch)
        _lib = lib
    return _lib


@dataclass
class Side:
    """Per-row results for one policy (train or infer); every field is [T]."""
    max: np.ndarray
    lse: np.ndarray
    lse_safe: np.ndarray
    log_cov: np.ndarray
    logp: np.ndarray
    logp_mp: np.ndarray
    sum_safe: np.ndarray
    sum_safe_x: np.ndarray
    tau: np.ndarray
    count: np.ndarray
    member: np.ndarray
    mask: np.ndarray | None = None  # [T, V] uint8 when requested


@dataclass
class Result:
    train: Side
    infer: Side | None
    log_ratio: np.ndarray | None
    grad: np.ndarray | None  # [T, V] float64
    threads: int = 1
    weight: np.ndarray | None = None  # [T] token-level importance weights, when asked for


def _storage(x: np.ndarray, dtype: int) -> np.ndarray:
    """Stored logits as the C side reads them: float32, or the raw 16-bit patterns."""
    if dtype == F32:
        if x.dtype != np.float32:
            raise TypeError("F32 logits must be a float32 array")
    elif x.dtype != np.uint16:
        raise TypeError("BF16/F16 logits must be passed as their uint16 bit patterns")
    if x.ndim != 2 or x.strides[1] != x.itemsize or x.strides[0] % x.itemsize:
        raise ValueError("logits must be a 2-D array with unit inner stride")
    return x


def _side(arr: np.ndarray, mask) -> Side:
    return Side(*(np.ascontiguousarray(arr[name]) for name in _SIDE_DTYPE.names[:-1]), mask=mask)


def dvp_rows(train: np.ndarray, ids: np.ndarray | None, rho: float, *, dtype: int = F32,
             infer: np.ndarray | None = None, upstream: np.ndarray | None = None,
             want_grad: bool = False, want_mask: bool = False, threads: int = 1,
             weight_kind: int = WEIGHT_NONE, weight_lo: float = 0.0, weight_hi: float = float("inf")) -> Result:
    """Run the row oracle on ``[T, V]`` logits (row stride may exceed V).

    ``ids`` are the sampled tokens (int64, negative = none), ``upstream`` the
    per-token gradient g of the loss with respect to log pi^mp_train(a).  With a
    ``weight_kind`` the gradient row is that of ``g * w`` with ``w`` the token's
    importance weight (``dvp_oracle_token_weight``), held constant.
    """
    lib = _load()
    if not (0.0 <= rho <= 1.0):
        raise ValueError("rho must lie in [0, 1]")
    train = _storage(train, dtype)
    T, V = train.shape
    b = _Batch()
    b.train = train.ctypes.data
    b.ld_train = train.strides[0] // train.itemsize
    b.dtype = dtype
    b.T, b.V, b.rho = T, V, float(rho)
    keep = [train]
    if infer is not None:
        infer = _storage(infer, dtype)
        if infer.shape != train.shape:
            raise ValueError("infer logits must have the shape of the train logits")
        b.infer = infer.ctypes.data
        b.ld_infer = infer.strides[0] // infer.itemsize
        keep.append(infer)
    if ids is not None:
        ids = np.ascontiguousarray(ids, dtype=np.int64)
        assert ids.shape == (T,)
        b.ids = ids.ctypes.data
        keep.append(ids)
    if upstream is not None:
        upstream = np.ascontiguousarray(upstream, dtype=np.float64)
        assert upstream.shape == (T,)
        b.upstream = upstream.ctypes.data
        keep.append(upstream)
    side_t = np.zeros(T, dtype=_SIDE_DTYPE)
    b.side_t = side_t.ctypes.data
    side_i = log_ratio = grad = mask_t = mask_i = None
    if infer is not None:
        side_i = np.zeros(T, dtype=_SIDE_DTYPE)
        log_ratio = np.zeros(T, dtype=np.float64)
        b.side_i = side_i.ctypes.data
        b.log_ratio = log_ratio.ctypes.data
    if want_grad:
        grad = np.zeros((T, V), dtype=np.float64)
        b.grad = grad.ctypes.data
    weight = None
    if weight_kind != WEIGHT_NONE:
        if infer is None:
            raise ValueError("importance weights need the inference logits")
        b.weight_kind, b.weight_lo, b.weight_hi = int(weight_kind), float(weight_lo), float(weight_hi)
        weight = np.zeros(T, dtype=np.float64)
        b.weight = weight.ctypes.data
    if want_mask:
        b.want_mask = 1
        mask_t = np.zeros((T, V), dtype=np.uint8)
        b.mask_t = mask_t.ctypes.data
        if infer is not None:
            mask_i = np.zeros((T, V), dtype=np.uint8)
            b.mask_i = mask_i.ctypes.data
    used = lib.dvp_oracle_batch(ctypes.byref(b), int(threads)) if T > 0 else 0
    del keep
    return Result(
        train=_side(side_t, mask_t),
        infer=_side(side_i, mask_i) if side_i is not None else None,
        log_ratio=log_ratio,
        grad=grad,
        threads=used,
        weight=weight,
    )


def _bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns widened exactly to float64."""
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


@dataclass
class FusedResult:
    rows: Result          # per-token results; rows.grad is dL/dz [T, V]
    logits: np.ndarray    # z = h W^T, float64 [T, V]
    d_hidden: np.ndarray  # [T, H] float64
    d_w: np.ndarray       # [V, H] float64


def fused_logits(hidden_bf16: np.ndarray, w_bf16: np.ndarray) -> np.ndarray:
    """z = h W^T in float64 from bfloat16 bit patterns: the training logits of the LM-head
    composition, which never round."""
    return _bf16_bits_to_f64(hidden_bf16) @ _bf16_bits_to_f64(w_bf16).T


def dvp_fused_lmhead(hidden_bf16: np.ndarray, w_bf16: np.ndarray, infer_bf16: np.ndarray,
                     ids: np.ndarray, rho: float, upstream: np.ndarray, threads: int = 1,
                     weight_kind: int = WEIGHT_NONE, weight_lo: float = 0.0,
                     weight_hi: float = float("inf"), logits: np.ndarray | None = None,
                     train_set: np.ndarray | None = None) -> FusedResult:
    """LM-head composition: z = h W^T, then the row computation on z, then the
    chain rule of Prop. 5.6 part 2 through the linear head:
    dH = G W and dW = G^T h with G = dL/dz.

    hidden [T, H], w [V, H] and infer logits [T, V] are bfloat16 bit patterns
    (uint16).  Train logits are taken in float64, so they never round.  With a
    ``weight_kind`` each token's upstream gradient is multiplied by its importance
    weight (``dvp_oracle_token_weight``), held constant.  ``logits`` hands in a
    ``fused_logits`` result computed before.  ``train_set`` ([T, V] bytes) supplies
    the training safe set instead of deriving it (``dvp_oracle_side_given_set``):
    the set of Def. 5.1 is fixed only up to tokens within rounding distance of the
    threshold when the logits themselves come out of rounded arithmetic.
    """
    h = _bf16_bits_to_f64(hidden_bf16)
    w = _bf16_bits_to_f64(w_bf16)
    z = h @ w.T if logits is None else logits
    zi = _bf16_bits_to_f64(infer_bf16)
    if train_set is not None:
        train_set = np.ascontiguousarray(train_set, dtype=np.uint8)
        assert train_set.shape == z.shape
    T, V = z.shape
    # The C rows read float32 or 16-bit storage; float64 logits go through the
    # same per-row functions one row at a time.
    lib = _load()
    side_t = np.zeros(T, dtype=_SIDE_DTYPE)
    side_i = np.zeros(T, dtype=_SIDE_DTYPE)
    log_ratio = np.zeros(T)
    grad = np.zeros((T, V))
    log_rho = float(np.log(rho)) if rho > 0 else -np.inf
    ids = np.ascontiguousarray(ids, dtype=np.int64)
    up = np.ascontiguousarray(upstream, dtype=np.float64)
    step = _SIDE_DTYPE.itemsize
    weight = np.ones(T)
    for t in range(T):
        zt = np.ascontiguousarray(z[t])
        zit = np.ascontiguousarray(zi[t])
        pt = side_t.ctypes.data + t * step
        pi = side_i.ctypes.data + t * step
        if train_set is None:
            lib.dvp_oracle_side(zt.ctypes.data, V, int(ids[t]), log_rho, pt, None)
        else:
            lib.dvp_oracle_side_given_set(zt.ctypes.data, V, int(ids[t]), train_set[t].ctypes.data, pt)
        lib.dvp_oracle_side(zit.ctypes.data, V, int(ids[t]), log_rho, pi, None)
        log_ratio[t] = lib.dvp_oracle_log_ratio(pt, pi)
        g = float(up[t])
        if weight_kind != WEIGHT_NONE:
            weight[t] = lib.dvp_oracle_token_weight(float(log_ratio[t]), int(weight_kind), float(weight_lo),
                                                    float(weight_hi))
            if not np.isnan(weight[t]):
                g *= float(weight[t])
        if train_set is None:
            lib.dvp_oracle_side_grad(zt.ctypes.data, V, int(ids[t]), g, pt, grad.ctypes.data + t * V * 8)
        else:
            lib.dvp_oracle_side_grad_given_set(zt.ctypes.data, V, int(ids[t]), g, train_set[t].ctypes.data, pt,
                                               grad.ctypes.data + t * V * 8)
    rows = Result(train=_side(side_t, None), infer=_side(side_i, None), log_ratio=log_ratio,
                  grad=grad, threads=1, weight=weight if weight_kind != WEIGHT_NONE else None)
    return FusedResult(rows=rows, logits=z, d_hidden=grad @ w, d_w=grad.T @ h)


def token_weight(log_ratio: float, kind: int, lo: float = 0.0, hi: float = float("inf")) -> float:
    """The importance weight of one token from its log-ratio."""
    return float(_load().dvp_oracle_token_weight(float(log_ratio), int(kind), float(lo), float(hi)))


def dvp_rows_f64(z: np.ndarray, ids: np.ndarray, rho: float, upstream: np.ndarray | None = None,
                 want_mask: bool = False, infer: np.ndarray | None = None, weight_kind: int = WEIGHT_NONE,
                 weight_lo: float = 0.0, weight_hi: float = float("inf")) -> Result:
    """Row oracle on float64 logits given directly (tiny cases in the tests)."""
    lib = _load()
    z = np.ascontiguousarray(z, dtype=np.float64)
    T, V = z.shape
    side = np.zeros(T, dtype=_SIDE_DTYPE)
    mask = np.zeros((T, V), dtype=np.uint8) if want_mask else None
    grad = np.zeros((T, V)) if upstream is not None else None
    log_rho = float(np.log(rho)) if rho > 0 else -np.inf
    ids = np.ascontiguousarray(ids, dtype=np.int64)
    step = _SIDE_DTYPE.itemsize
    side_i = log_ratio = weight = None
    if infer is not None:
        infer = np.ascontiguousarray(infer, dtype=np.float64)
        side_i = np.zeros(T, dtype=_SIDE_DTYPE)
        log_ratio = np.zeros(T)
        weight = np.ones(T)
    elif weight_kind != WEIGHT_NONE:
        raise ValueError("importance weights need the inference logits")
    for t in range(T):
        p = side.ctypes.data + t * step
        lib.dvp_oracle_side(z.ctypes.data + t * V * 8, V, int(ids[t]), log_rho, p,
                            mask.ctypes.data + t * V if want_mask else None)
        g = float(upstream[t]) if upstream is not None else 0.0
        if infer is not None:
            q = side_i.ctypes.data + t * step
            lib.dvp_oracle_side(infer.ctypes.data + t * V * 8, V, int(ids[t]), log_rho, q, None)
            log_ratio[t] = lib.dvp_oracle_log_ratio(p, q)
            weight[t] = lib.dvp_oracle_token_weight(float(log_ratio[t]), int(weight_kind), float(weight_lo),
                                                    float(weight_hi))
            if weight_kind != WEIGHT_NONE and not np.isnan(weight[t]):
                g = g * float(weight[t])
        if grad is not None:
            lib.dvp_oracle_side_grad(z.ctypes.data + t * V * 8, V, int(ids[t]), g, p,
                                     grad.ctypes.data + t * V * 8)
    return Result(train=_side(side, mask), infer=_side(side_i, None) if side_i is not None else None,
                  log_ratio=log_ratio, grad=grad, weight=weight if weight_kind != WEIGHT_NONE else None)


@dataclass
class SequenceResult:
    seq_log_ratio: np.ndarray   # [S] Delta_y = sum of the token log-ratios
    min_log_ratio: np.ndarray   # [S]
    n_valid: np.ndarray         # [S] tokens with a sampled id
    n_zero_weight: np.ndarray   # [S] tokens outside the training safe set
    veto: np.ndarray            # [S] 1 when some token weight is below the threshold


def dvp_sequences(log_ratio: np.ndarray, seq_offsets: np.ndarray, veto_threshold: float = 1e-4
                  ) -> SequenceResult:
    """Sequence-level mismatch and token veto (Sec. 4.4, Thm. 5.3, App. A protocol 5)."""
    lib = _load()
    lr = np.ascontiguousarray(log_ratio, dtype=np.float64)
    off = np.ascontiguousarray(seq_offsets, dtype=np.int64)
    S = len(off) - 1
    assert S >= 0 and (S == 0 or (off[0] >= 0 and off[-1] <= len(lr) and (np.diff(off) >= 0).all()))
    out = SequenceResult(np.zeros(S), np.zeros(S), np.zeros(S, dtype=np.int64),
                         np.zeros(S, dtype=np.int64), np.zeros(S, dtype=np.uint8))
    lib.dvp_oracle_sequences.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_double,
                                         ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                         ctypes.c_void_p, ctypes.c_void_p]
    lib.dvp_oracle_sequences.restype = None
    if S > 0:
        lib.dvp_oracle_sequences(lr.ctypes.data, off.ctypes.data, S, float(veto_threshold),
                                 out.seq_log_ratio.ctypes.data, out.min_log_ratio.ctypes.data,
                                 out.n_valid.ctypes.data, out.n_zero_weight.ctypes.data,
                                 out.veto.ctypes.data)
    return out


def dvp_coverage(log_cov: np.ndarray, seq_offsets: np.ndarray):
    """Per sequence: min and mean over its states of the coverage Z = e^{ln Z}
    (Def. 5.2; the minimum is the Z_min of the bias bound of Prop. 5.5)."""
    lib = _load()
    lc = np.ascontiguousarray(log_cov, dtype=np.float64)
    off = np.ascontiguousarray(seq_offsets, dtype=np.int64)
    S = len(off) - 1
    assert S >= 0 and (S == 0 or (off[0] >= 0 and off[-1] <= len(lc) and (np.diff(off) >= 0).all()))
    lo, mean = np.zeros(S), np.zeros(S)
    lib.dvp_oracle_coverage.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
                                        ctypes.c_void_p]
    lib.dvp_oracle_coverage.restype = None
    if S > 0:
        lib.dvp_oracle_coverage(lc.ctypes.data, off.ctypes.data, S, lo.ctypes.data, mean.ctypes.data)
    return lo, mean


_LISTING_DTYPE = np.dtype([("max", "f8"), ("lse_full", "f8"), ("lse_masked", "f8"), ("logp_masked", "f8"),
                           ("comp", "f8"), ("count", "i8"), ("member", "i4"), ("pad_", "i4")])


def round_to_storage(x: np.ndarray, dtype: int) -> np.ndarray:
    """Round float32 values to the storage type (nearest, ties to even) and widen
    them back to float64: F32 is the identity, BF16 keeps the upper 16 bits."""
    x = np.asarray(x, dtype=np.float32)
    if dtype == F32:
        return x.astype(np.float64)
    if dtype == F16:
        return x.astype(np.float16).astype(np.float64)
    bits = x.view(np.uint32).astype(np.uint64)
    bits = (bits + 0x7FFF + ((bits >> 16) & 1)) & 0xFFFF0000        # nearest-even on the low half
    return bits.astype(np.uint32).view(np.float32).astype(np.float64)


def dvp_rows_listing(z: np.ndarray, ids: np.ndarray, rho: float, mask_value: float, *, dtype: int = F32,
                     upstream: np.ndarray | None = None, threshold_in_storage_type: bool = True):
    """The App. A listing taken literally (finite mask value kept in the partition
    sum).  ``z`` holds the stored logits widened to float64.  The threshold is
    max + log(rho), formed in float32 and rounded to the storage type when
    ``threshold_in_storage_type`` is set, otherwise the exact double sum."""
    lib = _load()
    assert lib.dvp_oracle_sizeof_listing() == _LISTING_DTYPE.itemsize
    lib.dvp_oracle_listing.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_double,
                                       ctypes.c_double, ctypes.c_double, ctypes.c_void_p, ctypes.c_void_p]
    lib.dvp_oracle_listing.restype = None
    z = np.ascontiguousarray(z, dtype=np.float64)
    T, V = z.shape
    log_rho = float(np.log(rho)) if rho > 0 else -np.inf
    m = z.max(axis=1)
    if threshold_in_storage_type:
        with np.errstate(over="ignore"):
            c = round_to_storage(np.array([log_rho], dtype=np.float32), dtype).astype(np.float32)[0]
            thr = round_to_storage(m.astype(np.float32) + c, dtype)
    else:
        thr = m + log_rho
    mv = float(round_to_storage(np.array([mask_value]), dtype)[0])
    out = np.zeros(T, dtype=_LISTING_DTYPE)
    grad = np.zeros((T, V)) if upstream is not None else None
    ids = np.ascontiguousarray(ids, dtype=np.int64)
    for t in range(T):
        lib.dvp_oracle_listing(z.ctypes.data + t * V * 8, V, int(ids[t]), float(thr[t]), mv,
                               float(upstream[t]) if upstream is not None else 0.0,
                               out.ctypes.data + t * _LISTING_DTYPE.itemsize,
                               grad.ctypes.data + t * V * 8 if grad is not None else None)
    return out, grad, thr


def dvp_monitor(z: np.ndarray, zi: np.ndarray) -> np.ndarray:
    """Per-token KL(infer || train), KL(train || infer), H(train), H(infer) in nats over
    the full vocabulary; ``z`` and ``zi`` are the stored logits widened to float64.
    Returns a [T, 4] array."""
    lib = _load()
    lib.dvp_oracle_monitor.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p]
    lib.dvp_oracle_monitor.restype = None
    z = np.ascontiguousarray(z, dtype=np.float64)
    zi = np.ascontiguousarray(zi, dtype=np.float64)
    assert z.shape == zi.shape and z.ndim == 2
    T, V = z.shape
    out = np.zeros((T, 4))
    for t in range(T):
        lib.dvp_oracle_monitor(z.ctypes.data + t * V * 8, zi.ctypes.data + t * V * 8, V,
                               out.ctypes.data + t * 32)
    return out
