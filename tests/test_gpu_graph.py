"""The layer inside a CUDA graph: `bench.py` times replays of one captured step, so a replay has to
produce what the plain launches produce.  The library forks onto its own side streams inside a call
and keeps a few counters on the device between calls (the two sets of histogram counters and their
parity, the selection's ticket); both have to survive capture and replay."""
import numpy as np
import pytest
import torch

from paper_2501_17116_b200 import workloads as WL

pytestmark = pytest.mark.gpu


def _dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


@pytest.mark.parametrize("M,K,N1,N2,alpha", [(256, 384, 256, 128, 0.999), (1024, 256, 384, 640, 0.97)])
def test_replays_of_a_captured_step_equal_plain_launches(lib, M, K, N1, N2, alpha):
    """Two linears that share their activation (the second re-uses the first's quantised operand),
    forward and backward, captured once and replayed: outputs bit for bit those of plain launches,
    on the captured inputs, again on a second replay, and on new inputs written in place.  The second
    shape takes the forward's dense tail and the weight gradient's tensor-core class."""
    rng = np.random.default_rng(3)
    a_bits, w1_bits, g1_bits = WL.small_case(M, K, N1, seed=41, alpha_outliers=9)
    _, w2_bits, g2_bits = WL.small_case(M, K, N2, seed=42, alpha_outliers=9)
    A, W1, W2, G1, G2 = _dev(a_bits), _dev(w1_bits), _dev(w2_bits), _dev(g1_bits), _dev(g2_bits)
    ctx = lib.Context(0, int(lib.load_library().fp4_workspace_bytes(M, K, max(N1, N2))))
    out = {n: torch.empty(s, dtype=torch.bfloat16, device="cuda")
           for n, s in (("Y1", (M, N1)), ("Y2", (M, N2)), ("dA1", (M, K)), ("dA2", (M, K)), ("dW1", (K, N1)),
                        ("dW2", (K, N2)))}
    sa = lib.QTensor(M, K, 0, A.device, lib.tail_capacity(M, K, alpha))
    sw1, sw2 = lib.QTensor(K, N1, 1, A.device), lib.QTensor(K, N2, 1, A.device)

    def step():
        lib.fp4_linear_fwd(ctx, A, W1, alpha, sa, sw1, out=out["Y1"])
        lib.fp4_linear_bwd(ctx, G1, W1, sa, sw1, dA=out["dA1"], dW=out["dW1"])
        lib.fp4_linear_fwd(ctx, A, W2, alpha, sa, sw2, out=out["Y2"], reuse_a=True)
        lib.fp4_linear_bwd(ctx, G2, W2, sa, sw2, dA=out["dA2"], dW=out["dW2"])

    def plain():
        step()
        torch.cuda.synchronize()
        return {n: t.clone() for n, t in out.items()}

    def check(want, what):
        torch.cuda.synchronize()
        assert ctx.read_status() == 0
        for n, t in out.items():
            assert torch.equal(t.view(torch.int16), want[n].view(torch.int16)), (what, n)

    for _ in range(3):                                   # an odd number of calls before the capture
        step()
    want = plain()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            step()
    for rep in range(3):
        for t in out.values():
            t.zero_()
        graph.replay()
        check(want, f"replay {rep}")
    # new inputs in place: the graph holds the addresses, not the values
    a2, _, g1b = WL.small_case(M, K, N1, seed=43, alpha_outliers=9, dist="student_t3")
    A.copy_(_dev(a2))
    G1.copy_(_dev(g1b))
    graph.replay()
    torch.cuda.synchronize()
    got = {n: t.clone() for n, t in out.items()}
    want2 = plain()                                      # plain launches between replays
    for n in out:
        assert torch.equal(got[n].view(torch.int16), want2[n].view(torch.int16)), ("new inputs", n)
    graph.replay()
    check(want2, "replay after plain launches")
    ctx.close()
