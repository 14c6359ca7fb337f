"""CPU pins for the oracle of the Layer Router's front end (Sec. 3.1, Appendix D.1).

The paper fixes neither the pooling operator, the widths nor the activation, so the oracle's
reading (token mean; Linear-SiLU-Linear encoder; Linear-SiLU-Linear head) cannot be pinned to the
paper.  What the reading implies mathematically is pinned here against hand-typed values, closed
forms and an independent library evaluation (torch fp64 `linear` / `silu`)."""
import numpy as np
import torch

import oracle
from oracle import router_frontend as rf
from paper_2604_07394_b200 import synth


def _bf16_bits(x):
    return oracle.to_bits(torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16))


def test_segments_first_and_last_100_tokens():
    # Appendix D.1: the first 100 and the last 100 tokens
    assert rf.segments(250, 100) == ((0, 100), (150, 250))
    assert rf.segments(200, 100) == ((0, 100), (100, 200))
    assert rf.segments(150, 100) == ((0, 100), (50, 150))      # overlapping middle
    assert rf.segments(60, 100) == ((0, 60), (0, 60))          # prompt shorter than one segment
    assert rf.segments(1, 100) == ((0, 1), (0, 1))


def test_pool_hand_values():
    # Hq = 1, D = 2 (values exact in bf16): first segment 3 tokens, last segment 2 tokens
    first = _bf16_bits([[[1.0, -2.0]], [[3.0, 4.0]], [[5.0, 0.5]]])
    last = _bf16_bits([[[8.0, 1.0]], [[-2.0, 1.5]]])
    f = rf.pool(first, last)
    assert f.tolist() == [3.0, 2.5 / 3.0, 3.0, 1.25]


def test_pool_layout_segment_head_channel():
    # one-hot probe: token mean of a tensor that is 1 only at (head 2, channel 5) lands at index h*D+d
    Hq, D = 4, 8
    a = np.zeros((3, Hq, D), np.float32)
    a[:, 2, 5] = 1.0
    b = np.zeros((2, Hq, D), np.float32)
    b[:, 1, 0] = 2.0
    f = rf.pool(_bf16_bits(a), _bf16_bits(b))
    want = np.zeros(2 * Hq * D)
    want[2 * D + 5] = 1.0
    want[Hq * D + 1 * D + 0] = 2.0
    assert np.array_equal(f, want)


def test_silu_closed_forms():
    x = np.array([0.0, 1.0, -1.0, 30.0, -30.0, 2.5])
    y = rf.silu(x)
    assert y[0] == 0.0
    assert abs(y[1] - 1.0 / (1.0 + np.e ** -1.0)) < 1e-15
    assert np.allclose(y - rf.silu(-x), x, atol=1e-15)          # silu(x) - silu(-x) = x
    assert abs(y[3] - 30.0) < 1e-11 and abs(y[4]) < 1e-11       # identity / zero in the tails
    # minimum of silu is about -0.27846 at x about -1.27846
    g = rf.silu(np.linspace(-3, 0, 30001))
    assert abs(g.min() + 0.2784645427610738) < 1e-9


def _weights(F, E, R, seed=5):
    w = synth.router_weights(seed, 0, F, E, R)
    return {k: (oracle.to_bits(v) if v.dtype == torch.bfloat16 else v.numpy()) for k, v in w.items()}, w


def test_mlp_zero_weights_gives_bias_path():
    wb, _ = _weights(16, 8, 8)
    for k in ("w_enc1", "w_enc2", "w_head1"):
        wb[k] = np.zeros_like(wb[k])
    # f is irrelevant; h1 = silu(b1) is multiplied by zero; u = b2; h2 = silu(b3); pi = W4 h2 + b4
    pi = rf.mlp(np.arange(16, dtype=np.float64), wb)
    b3 = wb["b_head1"].astype(np.float64)
    h2 = b3 / (1.0 + np.exp(-b3))
    want = oracle.bits_to_f64(wb["w_head2"]) @ h2 + wb["b_head2"].astype(np.float64)
    assert np.allclose(pi, want, rtol=0, atol=1e-15)


def test_mlp_hand_example_non_square():
    # F = 3, E = 2, R = 1: every number typed by hand, shapes all different (a transposed operand
    # or a swapped layer cannot go unnoticed)
    w = {"w_enc1": _bf16_bits([[1.0, 0.0, -1.0], [0.5, 2.0, 0.0]]), "b_enc1": np.array([0.0, -1.0], np.float32),
         "w_enc2": _bf16_bits([[1.0, 1.0], [0.0, -2.0]]), "b_enc2": np.array([0.5, 0.0], np.float32),
         "w_head1": _bf16_bits([[2.0, -1.0]]), "b_head1": np.array([0.25], np.float32),
         "w_head2": _bf16_bits([[3.0], [-1.0]]), "b_head2": np.array([0.0, 1.0], np.float32)}
    f = np.array([2.0, 1.0, -1.0])
    s = lambda x: x / (1.0 + np.exp(-x))
    a1 = [1 * 2 + 0 * 1 + (-1) * (-1) + 0.0, 0.5 * 2 + 2 * 1 + 0 - 1.0]          # 3, 2
    h1 = [s(a1[0]), s(a1[1])]
    u = [h1[0] + h1[1] + 0.5, -2 * h1[1]]
    a3 = 2 * u[0] - u[1] + 0.25
    h2 = s(a3)
    want = [3 * h2, -h2 + 1.0]
    assert a1 == [3.0, 2.0]
    assert np.allclose(rf.mlp(f, w), want, rtol=0, atol=1e-14)


def test_mlp_against_torch_fp64_library_ops():
    F, E, R = 64, 24, 16
    wb, wt = _weights(F, E, R, seed=11)
    f = np.random.default_rng(3).normal(size=F)
    x = torch.from_numpy(f)
    d = {k: v.double() for k, v in wt.items()}
    h1 = torch.nn.functional.silu(torch.nn.functional.linear(x, d["w_enc1"], d["b_enc1"]))
    u = torch.nn.functional.linear(h1, d["w_enc2"], d["b_enc2"])
    h2 = torch.nn.functional.silu(torch.nn.functional.linear(u, d["w_head1"], d["b_head1"]))
    pi = torch.nn.functional.linear(h2, d["w_head2"], d["b_head2"]).numpy()
    assert np.allclose(rf.mlp(f, wb), pi, rtol=1e-13, atol=1e-13)


def test_logits_feed_hard_routing():
    # the front end's output plugs into the hard decision of Sec. 3.1: 1 (FA) iff pi_FA >= pi_SA
    Hq, D, E, R = 2, 8, 8, 8
    wb, _ = _weights(2 * Hq * D, E, R, seed=2)
    q = synth.normal_bf16((40, Hq, D), 9, 1)
    (a0, a1), (b0, b1) = rf.segments(40, 10)
    pi = rf.logits(oracle.to_bits(q[a0:a1]), oracle.to_bits(q[b0:b1]), wb)
    mask = oracle.route(pi.astype(np.float32).reshape(1, 1, 2))
    assert int(mask[0, 0]) == int(pi.astype(np.float32)[0] >= pi.astype(np.float32)[1])
