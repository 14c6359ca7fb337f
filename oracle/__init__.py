"""fp64 CPU oracle for routed hybrid attention -- TEST INFRASTRUCTURE ONLY.

Thin ctypes loader around ``flux_oracle.c`` (plain C, fp64, explicit kept-index
lists).  Only ``tests/``, the smoke check and the benchmark's CPU-baseline legs
may import this package; the CUDA library never does, and nothing here imports
the CUDA package.

Tensors cross as numpy ``uint16`` arrays of bf16 bit patterns (``to_bits``
turns a torch bf16 CPU tensor into one).  Layouts: Q, O ``[rows][Hq][D]``; K, V
``[tokens][Hkv][D]``.  Mode encoding follows Sec. 3.1: 1 = FA, 0 = SA.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

FA = 1
SA = 0

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "flux_oracle.c")
_LIB = os.path.join(_HERE, "libflux_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP for the row loops)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB)
        i64, i32, dbl = ctypes.c_int64, ctypes.c_int32, ctypes.c_double
        vp = ctypes.c_void_p
        L.flux_oracle_kept.restype = i64
        L.flux_oracle_kept.argtypes = [ctypes.c_int, i64, i64, i64, vp]
        L.flux_oracle_attend.restype = None
        L.flux_oracle_attend.argtypes = [vp, vp, vp, i64, vp, i64, ctypes.c_int, dbl, vp, vp, vp, vp]
        L.flux_oracle_prefill.restype = None
        L.flux_oracle_prefill.argtypes = [ctypes.c_int, vp, vp, vp, i64, i64, i64, ctypes.c_int,
                                          ctypes.c_int, ctypes.c_int, i64, i64, dbl, vp]
        L.flux_oracle_prefill_rows.restype = None
        L.flux_oracle_prefill_rows.argtypes = [ctypes.c_int, vp, vp, vp, i64, i64, vp, vp, i64,
                                               ctypes.c_int, ctypes.c_int, ctypes.c_int, i64, i64,
                                               dbl, vp]
        L.flux_oracle_kept_blocks.restype = i64
        L.flux_oracle_kept_blocks.argtypes = [i64, i64, vp, i64, vp]
        L.flux_oracle_prefill_blocks.restype = None
        L.flux_oracle_prefill_blocks.argtypes = [vp, vp, vp, i64, i64, i64, vp, vp, i64, ctypes.c_int,
                                                 ctypes.c_int, ctypes.c_int, i64, vp, i64, dbl, vp]
        L.flux_oracle_decode.restype = None
        L.flux_oracle_decode.argtypes = [ctypes.c_int, vp, vp, vp, i64, i64, ctypes.c_int,
                                         ctypes.c_int, ctypes.c_int, i64, i64, dbl, vp,
                                         ctypes.c_int, vp]
        L.flux_oracle_route.restype = i64
        L.flux_oracle_route.argtypes = [vp, i64, i64, vp]
        L.flux_oracle_msr.restype = dbl
        L.flux_oracle_msr.argtypes = [vp, i64, i64]
        L.flux_oracle_retained.restype = i64
        L.flux_oracle_retained.argtypes = [i64, i64, i64, vp]
        L.flux_oracle_compact_slot.restype = i64
        L.flux_oracle_compact_slot.argtypes = [i64, i64, i64]
        L.flux_oracle_merge.restype = None
        L.flux_oracle_merge.argtypes = [ctypes.c_int, dbl, dbl, vp, dbl, dbl, vp, vp, vp, vp]
        _lib = L
    return _lib


def set_threads(n: int) -> None:
    """Thread count for the OpenMP row loops (read by libgomp at first use)."""
    os.environ["OMP_NUM_THREADS"] = str(int(n))


def to_bits(t) -> np.ndarray:
    """torch bf16 CPU tensor (or a uint16 numpy array) -> C-contiguous uint16 bits."""
    if isinstance(t, np.ndarray):
        assert t.dtype == np.uint16
        return np.ascontiguousarray(t)
    import torch

    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return np.ascontiguousarray(t.contiguous().view(torch.int16).numpy().view(np.uint16))


def bits_to_f64(b: np.ndarray) -> np.ndarray:
    """Exact upcast of bf16 bit patterns to float64 (for checks written in numpy)."""
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f64_to_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float -> bf16 bit patterns (input preparation for tests)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = ((u >> 16) & 1) + 0x7FFF
    return ((u + r) >> 16).astype(np.uint16)


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def kept(mode: int, i: int, S: int, W: int) -> np.ndarray:
    """Sorted key positions query position ``i`` attends to (Eq. 1 / Eq. 2)."""
    idx = np.empty(i + 1, dtype=np.int64)
    n = lib().flux_oracle_kept(mode, i, S, W, _p(idx))
    return idx[:n].copy()


def attend(q, K, V, idx, scale, want_p=False):
    """One output row over an explicit index list.

    q ``[D]``, K/V ``[tokens][D]`` (one KV head) uint16 bits.  Returns
    ``(o[D] fp64, p or None, m, l)``.
    """
    q = np.ascontiguousarray(q)
    assert K.dtype == np.uint16 and V.dtype == np.uint16 and K.ndim == 2
    assert K.strides[1] == 2 and V.strides == K.strides
    D = q.shape[0]
    idx = np.ascontiguousarray(idx, dtype=np.int64)
    o = np.empty(D, dtype=np.float64)
    p = np.empty(len(idx), dtype=np.float64) if want_p else None
    m = ctypes.c_double()
    l = ctypes.c_double()
    lib().flux_oracle_attend(_p(q), _p(K), _p(V), K.strides[0] // 2, _p(idx), len(idx), D,
                             float(scale), _p(o), _p(p), ctypes.byref(m), ctypes.byref(l))
    return o, p, m.value, l.value


def _kv_stride(K):
    assert K.dtype == np.uint16 and K.ndim == 3 and K.strides[2] == 2
    assert K.strides[1] == 2 * K.shape[2], "KV heads of one token must be contiguous"
    return K.strides[0] // 2


def prefill(mode, Q, K, V, q_start, S, W, scale):
    """Q ``[Nq][Hq][D]``, K/V ``[>= q_start+Nq][Hkv][D]`` bits -> O ``[Nq][Hq][D]`` fp64."""
    Q = np.ascontiguousarray(Q)
    Nq, Hq, D = Q.shape
    Hkv = K.shape[1]
    assert K.shape[0] >= q_start + Nq and V.shape == K.shape and V.strides == K.strides
    assert Hq % Hkv == 0
    O = np.empty((Nq, Hq, D), dtype=np.float64)
    lib().flux_oracle_prefill(mode, _p(Q), _p(K), _p(V), _kv_stride(K), q_start, Nq, Hq, Hkv, D,
                              S, W, float(scale), _p(O))
    return O


def prefill_rows(mode, Q, K, V, q_start, rows, heads, S, W, scale):
    """Selected (position, head) rows of a prefill -> ``[n_rows][D]`` fp64."""
    Q = np.ascontiguousarray(Q)
    Nq, Hq, D = Q.shape
    Hkv = K.shape[1]
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    heads = np.ascontiguousarray(heads, dtype=np.int32)
    assert len(rows) == len(heads)
    assert rows.min(initial=q_start) >= q_start and rows.max(initial=q_start) < q_start + Nq
    assert K.shape[0] > rows.max(initial=0) and V.shape == K.shape and V.strides == K.strides
    O = np.empty((len(rows), D), dtype=np.float64)
    lib().flux_oracle_prefill_rows(mode, _p(Q), _p(K), _p(V), _kv_stride(K), q_start, _p(rows),
                                   _p(heads), len(rows), Hq, Hkv, D, S, W, float(scale), _p(O))
    return O


def kept_blocks(i: int, B: int, bm: np.ndarray) -> np.ndarray:
    """Sorted key positions query position ``i`` attends to under the block mask ``bm[qb][kb]``
    (block size ``B``; causal inside kept blocks)."""
    bm = np.ascontiguousarray(bm, dtype=np.uint8)
    assert bm.ndim == 2 and i // B < bm.shape[0] and i // B < bm.shape[1]
    idx = np.empty(i + 1, dtype=np.int64)
    n = lib().flux_oracle_kept_blocks(int(i), int(B), _p(bm), bm.shape[1], _p(idx))
    return idx[:n].copy()


def streaming_block_mask(n_qb: int, n_kb: int, S: int, W: int, B: int) -> np.ndarray:
    """The streaming pattern (sink + local window, Table 3) at block granularity: query block qb
    keeps the key blocks that hold sink positions and the ceil(W / B) blocks ending with its own
    (so a row sees between W - B + 1 and W local positions when B divides W)."""
    qb = np.arange(n_qb)[:, None]
    kb = np.arange(n_kb)[None, :]
    n_sink = -(-S // B)
    n_local = -(-W // B)
    return ((kb <= qb) & ((kb < n_sink) | (kb > qb - n_local))).astype(np.uint8)


def prefill_blocks(Q, K, V, q_start, B, bm, scale, rows=None, heads=None):
    """Prefill under a block mask.  ``rows`` / ``heads`` (equal-length arrays of absolute query
    positions and query heads) select outputs -> ``[n][D]``; otherwise ``[Nq][Hq][D]``."""
    Q = np.ascontiguousarray(Q)
    Nq, Hq, D = Q.shape
    Hkv = K.shape[1]
    bm = np.ascontiguousarray(bm, dtype=np.uint8)
    assert K.shape[0] >= q_start + Nq and V.shape == K.shape and V.strides == K.strides
    assert bm.shape[0] * B >= q_start + Nq and bm.shape[1] * B >= q_start + Nq
    if rows is None:
        O = np.empty((Nq, Hq, D), dtype=np.float64)
        lib().flux_oracle_prefill_blocks(_p(Q), _p(K), _p(V), _kv_stride(K), q_start, Nq, None, None, 0, Hq,
                                         Hkv, D, int(B), _p(bm), bm.shape[1], float(scale), _p(O))
        return O
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    heads = np.ascontiguousarray(heads, dtype=np.int32)
    assert len(rows) == len(heads) and rows.min() >= q_start and rows.max() < q_start + Nq
    O = np.empty((len(rows), D), dtype=np.float64)
    lib().flux_oracle_prefill_blocks(_p(Q), _p(K), _p(V), _kv_stride(K), q_start, Nq, _p(rows), _p(heads),
                                     len(rows), Hq, Hkv, D, int(B), _p(bm), bm.shape[1], float(scale), _p(O))
    return O


def decode(mode, q, K, V, n, S, W, scale, heads=None):
    """One decode step: q ``[Hq][D]``, K/V ``[>= n][Hkv][D]`` (new token at n-1)."""
    q = np.ascontiguousarray(q)
    Hq, D = q.shape
    Hkv = K.shape[1]
    assert K.shape[0] >= n >= 1 and V.shape == K.shape and V.strides == K.strides
    if heads is not None:
        heads = np.ascontiguousarray(heads, dtype=np.int32)
        cnt = len(heads)
    else:
        cnt = Hq
    o = np.empty((cnt, D), dtype=np.float64)
    lib().flux_oracle_decode(mode, _p(q), _p(K), _p(V), _kv_stride(K), n, Hq, Hkv, D, S, W,
                             float(scale), _p(heads), 0 if heads is None else cnt, _p(o))
    return o


def route(logits) -> np.ndarray:
    """logits ``[B][L][2]`` fp32 (FA first) -> mask ``[B][L]`` uint8, 1 = FA, 0 = SA."""
    lg = np.ascontiguousarray(logits, dtype=np.float32)
    B, L, two = lg.shape
    assert two == 2
    mask = np.empty((B, L), dtype=np.uint8)
    bad = lib().flux_oracle_route(_p(lg), B, L, _p(mask))
    if bad:
        raise ValueError("NaN routing logit")
    return mask


def msr(mask_row, H: int) -> float:
    """Model Sparsity Ratio (Eq. 3) of one request's layer mask."""
    m = np.ascontiguousarray(mask_row, dtype=np.uint8)
    return lib().flux_oracle_msr(_p(m), len(m), H)


def retained(n: int, S: int, W: int) -> np.ndarray:
    idx = np.empty(n, dtype=np.int64)
    c = lib().flux_oracle_retained(n, S, W, _p(idx))
    return idx[:c].copy()


def compact_slot(j: int, S: int, W: int) -> int:
    return lib().flux_oracle_compact_slot(j, S, W)


def merge(m1, l1, o1, m2, l2, o2):
    o1 = np.ascontiguousarray(o1, dtype=np.float64)
    o2 = np.ascontiguousarray(o2, dtype=np.float64)
    o = np.empty_like(o1)
    m = ctypes.c_double()
    l = ctypes.c_double()
    lib().flux_oracle_merge(len(o1), m1, l1, _p(o1), m2, l2, _p(o2), ctypes.byref(m),
                            ctypes.byref(l), _p(o))
    return m.value, l.value, o
