"""ctypes binding of ``libflux_attn.so`` -- argument marshalling only.

Every function named ``flux_*`` forwards to the C entry point of the same name
(declared in ``include/flux_attn.h``).  :class:`Plan` wraps them for torch
tensors: it passes ``data_ptr()`` and the current CUDA stream, nothing else.
There is no fallback: if the library is missing or a call fails, an exception
is raised.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libflux_attn.so")

FLUX_OK = 0
FLUX_E_INVALID_ARG = -1
FLUX_E_UNSUPPORTED_SHAPE = -2
FLUX_E_CAPACITY = -3
FLUX_E_WORKSPACE = -4
FLUX_E_DEVICE_TIMEOUT = -5
FLUX_E_CUDA = -6
FLUX_E_DEVICE_FLAG = -7

FLUX_STATUS_BAD_MASK = 1
FLUX_STATUS_NAN_LOGIT = 2
FLUX_STATUS_BAD_LENGTH = 4
FLUX_STATUS_WAIT_EXPIRED = 8

FLUX_KERNEL_DECODE = 0
FLUX_KERNEL_PREFILL = 1

FLUX_DECODE_AUTO = 0
FLUX_DECODE_TWO_LAUNCH = 1
FLUX_DECODE_SINGLE_LAUNCH = 2

FLUX_KV_FULL = 0
FLUX_KV_COMPACT_SA = 1

EXPORTS = [
    "flux_plan_create", "flux_plan_destroy", "flux_workspace_size", "flux_plan_set_workspace",
    "flux_router_apply", "flux_router_forward", "flux_attn_prefill", "flux_attn_prefill_blocks", "flux_kv_retain", "flux_kv_append",
    "flux_attn_decode", "flux_attn_decode_heads", "flux_attn_decode_partial", "flux_attn_combine", "flux_attn_decode_partial_push", "flux_attn_combine_wait", "flux_attn_decode_step", "flux_attn_decode_noalloc", "flux_attn_decode_host", "flux_attn_prefill_host", "flux_plan_status",
    "flux_debug_dispatch", "flux_debug_touched", "flux_debug_decode_kernel", "flux_plan_set_launch_overlap", "flux_debug_wait_probe", "flux_profile_enable", "flux_profile_read", "flux_launch_count", "flux_last_error", "flux_version",
]


class FluxConfig(ctypes.Structure):
    _fields_ = [
        ("n_layers", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("sink", ctypes.c_int32), ("window", ctypes.c_int32),
        ("softmax_scale", ctypes.c_float), ("max_batch", ctypes.c_int32),
        ("max_context", ctypes.c_int32), ("kv_layout", ctypes.c_int32),
    ]


class FluxRouterWeights(ctypes.Structure):
    _fields_ = [
        ("enc_dim", ctypes.c_int32), ("head_hidden", ctypes.c_int32),
        ("w_enc1", ctypes.c_void_p), ("b_enc1", ctypes.c_void_p),
        ("w_enc2", ctypes.c_void_p), ("b_enc2", ctypes.c_void_p),
        ("w_head1", ctypes.c_void_p), ("b_head1", ctypes.c_void_p),
        ("w_head2", ctypes.c_void_p), ("b_head2", ctypes.c_void_p),
    ]


class PeerSet(ctypes.Structure):
    _fields_ = [
        ("world", ctypes.c_int32), ("rank", ctypes.c_int32),
        ("gather_o", ctypes.c_void_p * 8), ("gather_ml", ctypes.c_void_p * 8), ("flags", ctypes.c_void_p * 8),
    ]


class FluxError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__("flux_attn error %d: %s" % (code, msg))
        self.code = code


_lib = None


def load():
    """Load the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            LIB_PATH + " is missing: build it with `python -m paper_2604_07394_b200.build` "
            "(there is no CPU fallback)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
    cfgp = ctypes.POINTER(FluxConfig)
    L.flux_plan_create.argtypes = [cfgp, ctypes.POINTER(vp)]
    L.flux_plan_destroy.argtypes = [vp]
    L.flux_workspace_size.argtypes = [cfgp, ctypes.POINTER(sz)]
    L.flux_plan_set_workspace.argtypes = [vp, vp, sz]
    L.flux_router_apply.argtypes = [vp, vp, vp, i32, vp, vp]
    L.flux_router_forward.argtypes = [vp, ctypes.POINTER(FluxRouterWeights), vp, i32, vp, i32, vp, vp]
    L.flux_attn_prefill.argtypes = [vp, i32, i32, vp, vp, vp, i32, i32, vp, vp]
    L.flux_attn_prefill_blocks.argtypes = [vp, vp, vp, vp, i32, i32, vp, i32, vp, vp]
    L.flux_kv_retain.argtypes = [vp, i32, i32, vp, vp, i32, vp, vp, vp]
    L.flux_kv_append.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp]
    L.flux_attn_decode.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp]
    L.flux_attn_decode_partial.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    L.flux_attn_combine.argtypes = [vp, i32, i32, vp, vp, vp, vp]
    L.flux_attn_decode_partial_push.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, ctypes.c_uint32, vp]
    L.flux_attn_combine_wait.argtypes = [vp, i32, i32, vp, vp, vp, ctypes.c_uint32, ctypes.c_int64, vp, vp]
    L.flux_attn_decode_heads.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, vp]
    L.flux_attn_decode_step.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
    L.flux_attn_decode_noalloc.argtypes = [cfgp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
    L.flux_attn_decode_host.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    L.flux_attn_prefill_host.argtypes = [vp, i32, i32, vp, vp, vp, vp, i32, i32, vp, vp, vp]
    L.flux_plan_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32), vp]
    L.flux_debug_dispatch.argtypes = [vp, vp, i32, ctypes.POINTER(i32), vp]
    L.flux_debug_decode_kernel.argtypes = [vp, i32]
    L.flux_plan_set_launch_overlap.argtypes = [vp, i32]
    L.flux_debug_touched.argtypes = [vp, vp, i32]
    L.flux_debug_wait_probe.argtypes = [vp, ctypes.c_int64, vp]
    L.flux_profile_enable.argtypes = [vp, i32]
    L.flux_profile_read.argtypes = [vp, i32, ctypes.POINTER(ctypes.c_double),
                                    ctypes.POINTER(ctypes.c_int64), vp]
    L.flux_launch_count.argtypes = [vp]
    L.flux_launch_count.restype = ctypes.c_int64
    L.flux_last_error.restype = ctypes.c_char_p
    L.flux_version.restype = ctypes.c_char_p
    for name in EXPORTS:
        fn = getattr(L, name)
        if name not in ("flux_launch_count", "flux_last_error", "flux_version"):
            fn.restype = ctypes.c_int
    _lib = L
    return L


def last_error() -> str:
    return load().flux_last_error().decode()


def _check(rc: int) -> None:
    if rc != FLUX_OK:
        raise FluxError(rc, last_error())


def _ptr(t):
    """Address of a torch tensor / numpy array / int / None."""
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        return t.data_ptr()
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return int(t)


def _stream():
    return torch.cuda.current_stream().cuda_stream


def make_config(n_layers, n_q_heads, n_kv_heads, sink, window, max_batch, max_context,
                kv_layout=FLUX_KV_FULL, softmax_scale=0.0, head_dim=128) -> FluxConfig:
    return FluxConfig(n_layers, n_q_heads, n_kv_heads, head_dim, sink, window, softmax_scale,
                      max_batch, max_context, kv_layout)


def flux_workspace_size(cfg: FluxConfig) -> int:
    out = ctypes.c_size_t()
    _check(load().flux_workspace_size(ctypes.byref(cfg), ctypes.byref(out)))
    return out.value


class Plan:
    """Owns a ``flux_plan`` and the torch-allocated workspace it was given."""

    def __init__(self, cfg: FluxConfig, device="cuda:0"):
        L = load()
        self.cfg = cfg
        self.device = torch.device(device)
        self._h = ctypes.c_void_p()
        with torch.cuda.device(self.device):
            _check(L.flux_plan_create(ctypes.byref(cfg), ctypes.byref(self._h)))
            nbytes = flux_workspace_size(cfg)
            self.workspace = torch.zeros(nbytes, dtype=torch.uint8, device=self.device)
            _check(L.flux_plan_set_workspace(self._h, self.workspace.data_ptr(), nbytes))
        self.mask = None

    def close(self):
        if self._h:
            load().flux_plan_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- entry points, same names as the C ABI ------------------------------------------------
    def flux_router_apply(self, logits=None, mask=None, B=None, mask_out=None):
        """logits fp32 [B][L][2] or mask uint8 [B][L] (torch on device, or numpy on host)."""
        src = mask if mask is not None else logits
        if B is None:
            B = int(src.shape[0])
        if mask_out is None:
            mask_out = torch.empty((B, self.cfg.n_layers), dtype=torch.uint8, device=self.device)
        _check(load().flux_router_apply(self._h, _ptr(logits), _ptr(mask), B, _ptr(mask_out), _stream()))
        self.mask = mask_out          # keep the cached decision alive
        return mask_out

    def flux_router_forward(self, weights, q_first, q_last, logits_out=None):
        """weights: dict of device tensors (w_enc1, b_enc1, w_enc2, b_enc2, w_head1, b_head1, w_head2,
        b_head2); q_first / q_last: bf16 [tokens][Hq][D] device tensors; logits_out: fp32 [2] device."""
        if logits_out is None:
            logits_out = torch.empty(2, dtype=torch.float32, device=self.device)
        w = FluxRouterWeights(int(weights["w_enc1"].shape[0]), int(weights["w_head1"].shape[0]),
                              *[_ptr(weights[k]) for k in ("w_enc1", "b_enc1", "w_enc2", "b_enc2",
                                                           "w_head1", "b_head1", "w_head2", "b_head2")])
        _check(load().flux_router_forward(self._h, ctypes.byref(w), _ptr(q_first), int(q_first.shape[0]),
                                          _ptr(q_last), int(q_last.shape[0]), _ptr(logits_out), _stream()))
        return logits_out

    def flux_attn_prefill(self, layer, req, q, k, v, q_start, out=None):
        Nq = int(q.shape[0])
        if out is None:
            out = torch.empty_like(q)
        _check(load().flux_attn_prefill(self._h, layer, req, _ptr(q), _ptr(k), _ptr(v), q_start, Nq,
                                        _ptr(out), _stream()))
        return out

    def flux_attn_prefill_blocks(self, q, k, v, q_start, block_mask, out=None):
        """block_mask: uint8 device tensor [n_q_blocks][n_kv_blocks], rows = absolute query blocks."""
        Nq = int(q.shape[0])
        if out is None:
            out = torch.empty_like(q)
        _check(load().flux_attn_prefill_blocks(self._h, _ptr(q), _ptr(k), _ptr(v), q_start, Nq,
                                               _ptr(block_mask), int(block_mask.shape[1]), _ptr(out), _stream()))
        return out

    def flux_attn_prefill_host(self, layer, req, q_host, q_dev, k, v, q_start, out_dev, out_host):
        Nq = int(q_host.shape[0])
        _check(load().flux_attn_prefill_host(self._h, layer, req, _ptr(q_host), _ptr(q_dev), _ptr(k),
                                             _ptr(v), q_start, Nq, _ptr(out_dev), _ptr(out_host),
                                             _stream()))
        return out_host

    def flux_kv_retain(self, layer, req, k_src, v_src, n, k_cache, v_cache):
        _check(load().flux_kv_retain(self._h, layer, req, _ptr(k_src), _ptr(v_src), n, _ptr(k_cache),
                                     _ptr(v_cache), _stream()))

    def flux_kv_append(self, layer, B, k_new, v_new, k_caches, v_caches, pos):
        _check(load().flux_kv_append(self._h, layer, B, _ptr(k_new), _ptr(v_new), _ptr(k_caches),
                                     _ptr(v_caches), _ptr(pos), _stream()))

    def flux_attn_decode(self, layer, B, q, k_caches, v_caches, ctx_len, out=None):
        if out is None:
            out = torch.empty_like(q)
        _check(load().flux_attn_decode(self._h, layer, B, _ptr(q), _ptr(k_caches), _ptr(v_caches),
                                       _ptr(ctx_len), _ptr(out), _stream()))
        return out

    def flux_attn_decode_partial(self, layer, B, q, k_caches, v_caches, ctx_len, key_begin, key_end, part_o=None, part_ml=None):
        """One piece of a decode step over the key positions [key_begin[b], key_end[b]) -> (part_o fp32 [B][Hq][D],
        part_ml fp32 [B][Hq][2])."""
        if part_o is None:
            part_o = torch.empty((B, self.cfg.n_q_heads, 128), dtype=torch.float32, device=self.device)
        if part_ml is None:
            part_ml = torch.empty((B, self.cfg.n_q_heads, 2), dtype=torch.float32, device=self.device)
        _check(load().flux_attn_decode_partial(self._h, layer, B, _ptr(q), _ptr(k_caches), _ptr(v_caches), _ptr(ctx_len),
                                               _ptr(key_begin), _ptr(key_end), _ptr(part_o), _ptr(part_ml), _stream()))
        return part_o, part_ml

    def flux_attn_combine(self, B, part_o, part_ml, out=None):
        """part_o fp32 [n_sets][B][Hq][D], part_ml fp32 [n_sets][B][Hq][2] -> out bf16 [B][Hq][D]."""
        n_sets = int(part_o.shape[0])
        if out is None:
            out = torch.empty((B, self.cfg.n_q_heads, 128), dtype=torch.bfloat16, device=self.device)
        _check(load().flux_attn_combine(self._h, B, n_sets, _ptr(part_o), _ptr(part_ml), _ptr(out), _stream()))
        return out

    def flux_attn_decode_partial_push(self, layer, B, q, k_caches, v_caches, ctx_len, key_begin, key_end, rank, gather_o, gather_ml, flags, seq):
        """This rank's piece stored straight into slot `rank` of every rank's gather buffer; gather_o / gather_ml / flags:
        one tensor per rank (fp32 [world][B][Hq][D], fp32 [world][B][Hq][2], int32 or uint32 [world]), addressable from this GPU."""
        ps = PeerSet()
        ps.world, ps.rank = len(gather_o), rank
        for p in range(ps.world):
            ps.gather_o[p], ps.gather_ml[p], ps.flags[p] = _ptr(gather_o[p]), _ptr(gather_ml[p]), _ptr(flags[p])
        _check(load().flux_attn_decode_partial_push(self._h, layer, B, _ptr(q), _ptr(k_caches), _ptr(v_caches), _ptr(ctx_len),
                                                    _ptr(key_begin), _ptr(key_end), ctypes.byref(ps), seq, _stream()))

    def flux_attn_combine_wait(self, B, gather_o, gather_ml, flags, seq, out=None, wait_cycles=0):
        """Waits (bounded) until every rank's flag equals seq, then merges this rank's gather buffer -> out bf16 [B][Hq][D]."""
        if out is None:
            out = torch.empty((B, self.cfg.n_q_heads, 128), dtype=torch.bfloat16, device=self.device)
        _check(load().flux_attn_combine_wait(self._h, B, int(gather_o.shape[0]), _ptr(gather_o), _ptr(gather_ml), _ptr(flags), seq,
                                             wait_cycles, _ptr(out), _stream()))
        return out

    def flux_attn_decode_heads(self, B, q, k_caches, v_caches, ctx_len, head_mask, out=None):
        """head_mask: uint8 device tensor [B][Hkv], 1 = dense head group, 0 = sink + window."""
        if out is None:
            out = torch.empty_like(q)
        _check(load().flux_attn_decode_heads(self._h, B, _ptr(q), _ptr(k_caches), _ptr(v_caches),
                                             _ptr(ctx_len), _ptr(head_mask), _ptr(out), _stream()))
        return out

    def flux_attn_decode_step(self, layer, B, q, k_new, v_new, k_caches, v_caches, ctx_len, out=None):
        if out is None:
            out = torch.empty_like(q)
        _check(load().flux_attn_decode_step(self._h, layer, B, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_caches),
                                            _ptr(v_caches), _ptr(ctx_len), _ptr(out), _stream()))
        return out

    def flux_attn_decode_host(self, layer, B, q_host, k_new_host, v_new_host, k_caches, v_caches,
                              pos, ctx_len, out_host):
        _check(load().flux_attn_decode_host(self._h, layer, B, _ptr(q_host), _ptr(k_new_host),
                                            _ptr(v_new_host), _ptr(k_caches), _ptr(v_caches),
                                            _ptr(pos), _ptr(ctx_len), _ptr(out_host), _stream()))
        return out_host

    def flux_plan_status(self, raise_on_flag=True) -> int:
        bits = ctypes.c_uint32()
        rc = load().flux_plan_status(self._h, ctypes.byref(bits), _stream())
        if rc != FLUX_OK and (raise_on_flag or rc not in (FLUX_E_DEVICE_FLAG, FLUX_E_DEVICE_TIMEOUT)):
            _check(rc)
        return bits.value

    def flux_debug_dispatch(self, max_records=None) -> np.ndarray:
        """Records ``[n][8]``: mode, layer, request, n, a_begin, a_end, b_begin, b_end."""
        if max_records is None:
            max_records = self.cfg.max_batch
        rec = np.zeros((max_records, 8), dtype=np.int32)
        n = ctypes.c_int32()
        _check(load().flux_debug_dispatch(self._h, rec.ctypes.data, max_records, ctypes.byref(n), _stream()))
        return rec[: n.value].copy()

    def flux_debug_touched(self, bitmap=None) -> None:
        """bitmap: int32/uint32 device tensor [max_batch][words] (zeroed by the caller) or None (off)."""
        words = 0 if bitmap is None else int(bitmap.shape[1])
        _check(load().flux_debug_touched(self._h, _ptr(bitmap), words))
        self._touch = bitmap          # keep it alive while the plan points at it

    def flux_debug_wait_probe(self, limit_cycles: int) -> None:
        _check(load().flux_debug_wait_probe(self._h, limit_cycles, _stream()))

    def flux_plan_set_launch_overlap(self, on: bool) -> None:
        _check(load().flux_plan_set_launch_overlap(self._h, 1 if on else 0))

    def flux_debug_decode_kernel(self, which: int) -> None:
        _check(load().flux_debug_decode_kernel(self._h, which))

    def flux_profile_enable(self, max_records: int) -> None:
        _check(load().flux_profile_enable(self._h, max_records))

    def flux_profile_read(self, kind: int):
        """(total milliseconds, launches) of the recorded dominant-kernel launches of ``kind``."""
        ms = ctypes.c_double()
        n = ctypes.c_int64()
        _check(load().flux_profile_read(self._h, kind, ctypes.byref(ms), ctypes.byref(n), _stream()))
        return ms.value, n.value

    def flux_launch_count(self) -> int:
        return load().flux_launch_count(self._h)


def flux_attn_decode_noalloc(cfg: FluxConfig, layer, B, mask, q, k_caches, v_caches, ctx_len, out=None,
                             status_out=None):
    """Decode step for callers that cannot allocate device memory: needs no plan and no workspace.

    The split-K scratch is a fixed array inside the library (B <= 64, at most 8 query heads per KV
    head, at most 16 KV heads).  Calls on one device share that array, so calls that could overlap
    on the GPU must be serialised by the caller.  ``out`` is the caller's tensor (allocated here
    with torch only when omitted, as a convenience of this wrapper)."""
    if out is None:
        out = torch.empty_like(q)
    _check(load().flux_attn_decode_noalloc(ctypes.byref(cfg), layer, B, _ptr(mask), _ptr(q), _ptr(k_caches),
                                           _ptr(v_caches), _ptr(ctx_len), _ptr(out), _ptr(status_out),
                                           _stream()))
    return out


def pointer_table(tensors, device) -> torch.Tensor:
    """Device array of the tensors' addresses (the ``k_caches`` / ``v_caches`` argument)."""
    return torch.tensor([t.data_ptr() for t in tensors], dtype=torch.int64, device=device)
