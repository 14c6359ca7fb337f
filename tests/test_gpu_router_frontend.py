"""GPU parity of the Layer Router front end (Sec. 3.1) through the C ABI against the fp64 oracle.

Tolerance: the kernels accumulate in fp32 (pooling: 100-term sums; matrix-vector products: up to
8192-term dot products of O(1/sqrt(n))-sized terms, results O(1)).  A dot product of n terms summed
in fp32 has an error of about sqrt(n) * 2^-24 * |result scale| = 5e-6 at n = 8192, and the four layers
propagate it with gain O(1) (weights drawn with variance 1 / fan_in), so |gpu - oracle| <= 1e-4 *
(1 + |oracle|) leaves a factor of about 20.  The hard decision is taken on the fp32 logits the
kernel wrote, by the same rule on both sides; where the oracle's own margin exceeds the tolerance
it must agree with the oracle's decision too."""
import numpy as np
import pytest
import torch

import oracle
from oracle import router_frontend as rf
from paper_2604_07394_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def flux():
    from paper_2604_07394_b200 import build, flux as f
    build.build()
    f.load()
    return f


def _bits(w):
    return {k: (oracle.to_bits(v.cpu()) if v.dtype == torch.bfloat16 else v.cpu().numpy()) for k, v in w.items()}


@pytest.mark.parametrize("Hq,Hkv,E,R,N,P", [
    (32, 8, 512, 128, 4096, 100),     # Llama-3.1-8B attention shape, the paper's 100 + 100 tokens
    (28, 4, 1024, 256, 1000, 100),    # 28 / 4 heads
    (8, 2, 8, 8, 150, 100),           # smallest widths, overlapping segments
    (8, 2, 4096, 4096, 37, 100),      # largest widths, prompt shorter than one segment
    (8, 8, 64, 24, 300, 1),           # one token per segment
])
def test_router_forward_matches_oracle(flux, Hq, Hkv, E, R, N, P):
    plan = flux.Plan(flux.make_config(3, Hq, Hkv, 64, 256, 2, max(N, 1024)), DEV)
    q = synth.normal_bf16((N, Hq, 128), 77, synth.stream_id("q"), DEV)
    (a0, a1), (b0, b1) = rf.segments(N, P)
    logits = torch.zeros((2, 3, 2), dtype=torch.float32, device=DEV)
    ref = np.zeros((2, 3, 2))
    for layer in range(3):
        w = synth.router_weights(77, layer, 2 * Hq * 128, E, R, DEV)
        for req in range(2):
            # the two requests pool different parts of the same tensor
            s = 7 * req
            first, last = q[a0:a1 - s] if a1 - s > a0 else q[a0:a1], q[b0 + s:b1] if b0 + s < b1 else q[b0:b1]
            plan.flux_router_forward(w, first, last, logits[req, layer])
            ref[req, layer] = rf.logits(oracle.to_bits(first.cpu()), oracle.to_bits(last.cpu()), _bits(w))
    got = logits.cpu().numpy().astype(np.float64)
    err = np.abs(got - ref)
    assert np.all(err <= 1e-4 * (1.0 + np.abs(ref))), "max err %.3e (ref %s, got %s)" % (err.max(), ref.ravel(), got.ravel())
    # hard routing on the logits the kernels wrote
    mask = plan.flux_router_apply(logits=logits).cpu().numpy()
    assert np.array_equal(mask, oracle.route(logits.cpu().numpy()))
    margin = ref[..., 0] - ref[..., 1]
    clear = np.abs(margin) > 4e-4 * (1.0 + np.abs(ref).max(axis=-1))
    assert np.array_equal(mask[clear], (margin >= 0).astype(np.uint8)[clear])
    assert plan.flux_plan_status() == 0


def test_router_forward_rejects_bad_arguments(flux):
    plan = flux.Plan(flux.make_config(1, 8, 2, 64, 256, 1, 1024), DEV)
    q = synth.normal_bf16((16, 8, 128), 1, 1, DEV)
    w = synth.router_weights(1, 0, 2 * 8 * 128, 16, 16, DEV)
    out = torch.zeros(2, dtype=torch.float32, device=DEV)
    with pytest.raises(flux.FluxError) as e:
        plan.flux_router_forward(w, q[:0], q, out)
    assert e.value.code == flux.FLUX_E_INVALID_ARG
    w12 = synth.router_weights(1, 0, 2 * 8 * 128, 12, 16, DEV)
    with pytest.raises(flux.FluxError) as e:
        plan.flux_router_forward(w12, q, q, out)
    assert e.value.code == flux.FLUX_E_UNSUPPORTED_SHAPE
    big = dict(w)
    big["w_head1"] = torch.zeros((4104, 16), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(flux.FluxError) as e:
        plan.flux_router_forward(big, q, q, out)
    assert e.value.code == flux.FLUX_E_CAPACITY
    with pytest.raises(flux.FluxError) as e:
        plan.flux_router_forward(w, q, q, torch.zeros(2, dtype=torch.float32))     # host logits_out
    assert e.value.code == flux.FLUX_E_INVALID_ARG
    assert plan.flux_plan_status() == 0


def _router_case(Hq=32, Hkv=8, E=256, R=64, N=600, L=3):
    q = synth.normal_bf16((N, Hq, 128), 91, synth.stream_id("q"), DEV)
    ws = [synth.router_weights(91, layer, 2 * Hq * 128, E, R, DEV) for layer in range(L)]
    first, last = q[:100], q[-100:]
    ref = np.stack([rf.logits(oracle.to_bits(first.cpu()), oracle.to_bits(last.cpu()), _bits(w)) for w in ws])
    return ws, first, last, ref


def test_router_forward_in_a_replayed_graph(flux):
    """The kernel tells this launch's activations from an older launch's by a launch number kept on the
    device: a captured graph replays the same arguments, so every replay must still find fresh values.
    Logits after each of several replays equal the oracle's; a call issued outside the graph between
    replays (one more launch number) changes nothing."""
    ws, first, last, ref = _router_case()
    plan = flux.Plan(flux.make_config(3, 32, 8, 64, 256, 1, 1024), DEV)
    logits = torch.zeros((1, 3, 2), dtype=torch.float32, device=DEV)

    def one_pass():
        for layer, w in enumerate(ws):
            plan.flux_router_forward(w, first, last, logits[0, layer])

    one_pass()                                      # first use outside capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        one_pass()
    for rep in range(6):
        logits.fill_(float("nan"))
        graph.replay()
        if rep == 3:
            plan.flux_router_forward(ws[1], first, last, logits[0, 1])
        torch.cuda.synchronize()
        got = logits[0].cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - ref) <= 1e-4 * (1.0 + np.abs(ref))), (rep, got, ref)
    assert plan.flux_plan_status() == 0


def test_router_forward_after_a_cleared_timeout(flux):
    """Reading a status word that reports a timed-out wait puts the router's counters and its launch number
    back to zero (a kernel that gave up leaves them anywhere); the tagged activations are cleared with them,
    so the launches that follow start again from launch number one and are correct."""
    ws, first, last, ref = _router_case(L=2)
    plan = flux.Plan(flux.make_config(2, 32, 8, 64, 256, 1, 1024), DEV)
    logits = torch.zeros((1, 2, 2), dtype=torch.float32, device=DEV)
    for rounds in range(2):
        for _ in range(3):                          # launch numbers 1..6 leave their tags behind
            for layer, w in enumerate(ws):
                plan.flux_router_forward(w, first, last, logits[0, layer])
        plan.flux_debug_wait_probe(2_000_000)       # a bounded wait that runs out: the status bit, nothing else
        with pytest.raises(flux.FluxError) as e:
            plan.flux_plan_status()
        assert e.value.code == flux.FLUX_E_DEVICE_TIMEOUT
        logits.fill_(float("nan"))
        for layer, w in enumerate(ws):
            plan.flux_router_forward(w, first, last, logits[0, layer])
        got = logits[0].cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - ref) <= 1e-4 * (1.0 + np.abs(ref))), (rounds, got, ref)
        assert plan.flux_plan_status() == 0
