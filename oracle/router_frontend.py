"""fp64 CPU oracle for the Layer Router's front end -- TEST INFRASTRUCTURE ONLY.

Sec. 3.1 ("Architecture and Feature Extraction") describes the router in words only: the layer's
query tensor x_Q [s][h][d'] goes through a Prefill-Suffix Pooling over the first and the last
prompt tokens (100 + 100, Appendix D.1), a Context Encoder (an MLP) and a Router Head (an MLP) that
ends in the two logits (pi_FA, pi_SA).  The pooling operator, the layer widths and the activation
are not given.  PARITY UNPINNED with respect to the paper for those choices; the reading taken
here, and by the CUDA path independently, is

    f   = concat( mean over the first-segment tokens of x_Q, mean over the last-segment tokens )
          -- a vector of 2*h*d' numbers, index = segment*h*d' + head*d' + channel
    h1  = silu(W_e1 f  + b_e1)        Context Encoder, hidden layer      [E]
    u   =      W_e2 h1 + b_e2         Context Encoder, output            [E]
    h2  = silu(W_r1 u  + b_r1)        Router Head, hidden layer          [R]
    pi  =      W_r2 h2 + b_r2         Router Head, output (pi_FA, pi_SA) [2]
    silu(x) = x / (1 + exp(-x))

Weights are bf16 (upcast exactly), biases fp32, everything evaluated in fp64 by plain numpy
matrix-vector products in the order written above.  What *is* fixed independently of those
choices -- the mean, the layer algebra, the activation's closed-form values, the segment
bounds -- is pinned by the CPU tests.
"""
from __future__ import annotations

import numpy as np

from . import bits_to_f64


def segments(n_tokens: int, n_pool: int):
    """Token ranges [a, b) of the two pooled segments of a prompt of n_tokens tokens: the first
    min(n_pool, n) tokens and the last min(n_pool, n) tokens (Appendix D.1: n_pool = 100).  For a
    prompt shorter than 2 * n_pool the two ranges overlap; nothing is dropped or double-weighted
    inside a segment."""
    m = min(n_pool, n_tokens)
    return (0, m), (n_tokens - m, n_tokens)


def pool(q_first_bits: np.ndarray, q_last_bits: np.ndarray) -> np.ndarray:
    """Prefill-Suffix Pooling (Sec. 3.1): per-segment token mean, concatenated.
    q_*_bits: uint16 bf16 bit patterns [tokens][Hq][D], at least one token each."""
    a = bits_to_f64(q_first_bits)
    b = bits_to_f64(q_last_bits)
    fa = a.reshape(a.shape[0], -1).sum(axis=0) / a.shape[0]
    fb = b.reshape(b.shape[0], -1).sum(axis=0) / b.shape[0]
    return np.concatenate([fa, fb])


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def mlp(f: np.ndarray, w: dict) -> np.ndarray:
    """Context Encoder + Router Head on a pooled descriptor f (fp64).  w: w_enc1 [E][F],
    w_enc2 [E][E], w_head1 [R][E], w_head2 [2][R] as uint16 bf16 bit patterns; b_* fp32 arrays.
    Returns (pi_FA, pi_SA) as fp64."""
    W1, W2 = bits_to_f64(w["w_enc1"]), bits_to_f64(w["w_enc2"])
    W3, W4 = bits_to_f64(w["w_head1"]), bits_to_f64(w["w_head2"])
    b1, b2 = np.asarray(w["b_enc1"], np.float64), np.asarray(w["b_enc2"], np.float64)
    b3, b4 = np.asarray(w["b_head1"], np.float64), np.asarray(w["b_head2"], np.float64)
    h1 = silu(W1 @ f + b1)
    u = W2 @ h1 + b2
    h2 = silu(W3 @ u + b3)
    return W4 @ h2 + b4


def logits(q_first_bits: np.ndarray, q_last_bits: np.ndarray, w: dict) -> np.ndarray:
    """x_Q segments -> (pi_FA, pi_SA), the whole front end of Sec. 3.1."""
    return mlp(pool(q_first_bits, q_last_bits), w)
