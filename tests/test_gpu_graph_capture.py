"""The three calls (and the fused round) are plain asynchronous launches on the caller's stream with
no allocation and no host synchronisation, so a decoding round can be captured in a CUDA graph and
replayed (Section 4 runs its chain path that way).  The kernels are launched with programmatic
dependent launch; the capture must keep those edges, and every replay must give the eager result."""
import pytest
import torch

from paper_2608_20961_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cid,hint", [(2, 32), (1, 5)])
def test_round_captured_in_a_cuda_graph_replays_the_eager_result(cid, hint):
    from paper_2608_20961_b200 import binding as tw
    dev = torch.device("cuda:0")
    w = wl.make_workload(cid, B=6, H_v=4, seed=91)
    d = lambda t: t.to(dev)
    off, par, alpha, beta = d(w.node_offsets), d(w.parent), d(w.alpha), d(w.beta)
    q, k, v, acc = d(w.q), d(w.k), d(w.v), d(w.accepted)
    S_init = d(w.S0)

    def buffers():
        return dict(S=S_init.clone(), tree=tw.Tree.empty(off, par, w.H_v, hint),
                    O=torch.zeros((w.T, w.H_v, 128), dtype=torch.bfloat16, device=dev),
                    U=torch.zeros((w.T, w.H_v, 128), dtype=torch.float32, device=dev),
                    status=torch.zeros(w.B, dtype=torch.int32, device=dev))

    def round_(b):
        tw.treewy_tree_prepare(b["tree"], alpha, b["status"])
        tw.treewy_verify(b["S"], q, k, v, beta, b["tree"], w.H_qk, b["O"], b["U"], b["status"])
        tw.treewy_commit(b["S"], b["U"], k, b["tree"], w.H_qk, acc, None, b["status"])

    eager = buffers()
    round_(eager)
    round_(eager)                                   # two rounds: the state is carried from one to the next
    torch.cuda.synchronize()

    cap = buffers()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        round_(cap)                                 # warm-up outside the capture (module load, attributes)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    cap["S"].copy_(S_init)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        round_(cap)
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert not eager["status"].any() and not cap["status"].any()
    for name in ("S", "O", "U"):
        assert torch.equal(eager[name], cap[name]), name
