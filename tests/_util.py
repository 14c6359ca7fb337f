"""Shared helpers for the GPU parity tests (comparison rule, cache builders)."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2604_07394_b200 import synth

ABS_TOL = 2e-2      # every element: |gpu - ref| <= ABS_TOL
REL_TOL = 1e-2      # every output row: ||gpu - ref||_2 <= REL_TOL * ||ref||_2, and every element
                    # |gpu - ref| <= REL_TOL * (|ref| + rms(ref row))
# The elementwise rule is a relative bound with an absolute floor tied to the row's own scale
# (outputs are averages of N(0,1) values, so many elements are near zero and a bare relative
# error is unbounded).  Where it comes from: the output is rounded to bf16, and the softmax
# weights are rounded to bf16 before the PV product, which adds independent errors whose sum has
# a standard deviation of about 1e-3 * rms(row) with extremes of 5..6 sigma over 10^6..10^8
# elements.  tests/test_tolerance_model.py evaluates that rounding scheme by itself in fp64 and
# shows where it sits under each of the three bounds.
# This is the one comparison rule: the smoke check and the benchmark's oracle leg call compare() too.

def compare(gpu, ref, what=""):
    """gpu: bf16/float tensor or array [..., D]; ref: fp64 array of the same shape."""
    if isinstance(gpu, torch.Tensor):
        gpu = gpu.detach().float().cpu().numpy().astype(np.float64)
    gpu = np.asarray(gpu, dtype=np.float64).reshape(-1, ref.shape[-1])
    ref = np.asarray(ref, dtype=np.float64).reshape(-1, ref.shape[-1])
    assert gpu.shape == ref.shape, (gpu.shape, ref.shape)
    assert np.isfinite(gpu).all(), what + ": non-finite output"
    err = np.abs(gpu - ref)
    max_abs = err.max()
    row_norm = np.linalg.norm(ref, axis=1)
    row_rel = np.linalg.norm(gpu - ref, axis=1) / np.maximum(row_norm, 1e-30)
    rms = row_norm / np.sqrt(ref.shape[1])
    el_rel = (err / (np.abs(ref) + rms[:, None])).max()
    msg = "%s: max_abs=%.3e row_rel_l2=%.3e el_rel=%.3e" % (what, max_abs, row_rel.max(), el_rel)
    assert max_abs <= ABS_TOL, msg
    assert row_rel.max() <= REL_TOL, msg
    assert el_rel <= REL_TOL, msg
    return max_abs, row_rel.max(), el_rel


def bits(t: torch.Tensor) -> np.ndarray:
    return oracle.to_bits(t.detach().cpu())


def expand_ranges(rec) -> list:
    """Dispatch record -> sorted list of cache rows read for the newest query."""
    _, _, _, _, a0, a1, b0, b1 = [int(x) for x in rec]
    return list(range(a0, a1)) + list(range(b0, b1))


def compact_rows_to_positions(rows, n, S, W):
    """Invert the compact-cache slot rule for a context of n tokens, using the oracle's rule."""
    held = {}
    for j in oracle.retained(n, S, W):
        held[oracle.compact_slot(int(j), S, W)] = int(j)
    return sorted(held[r] for r in rows)


def logical_view(cache: torch.Tensor, n: int, S: int, W: int, compact: bool) -> torch.Tensor:
    """Rows of a cache as a position-indexed [n][Hkv][D] CPU tensor (evicted rows are zero)."""
    c = cache.detach().cpu()
    if not compact:
        return c[:n]
    out = torch.zeros((n,) + tuple(c.shape[1:]), dtype=c.dtype)
    for j in oracle.retained(n, S, W):
        out[int(j)] = c[oracle.compact_slot(int(j), S, W)]
    return out
