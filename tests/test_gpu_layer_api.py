"""The user-level step API: pipelined steps over three streams give exactly what the same steps
give on one stream, and the first step matches the oracle."""
import numpy as np
import pytest
import torch

from paper_2608_20961_b200 import workloads as wl
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def _host(w):
    names = ("q", "k", "v", "alpha", "beta", "parent", "node_offsets", "accepted")
    return {n: getattr(w, n).contiguous().clone().pin_memory() for n in names}


def test_pipelined_steps_equal_sequential_steps(oracle):
    from paper_2608_20961_b200 import binding as tw
    dev = torch.device("cuda:0")
    ws = [wl.make_workload(2, B=7, H_v=4, seed=100 + i) for i in range(5)]   # five decoding rounds
    hosts = [_host(w) for w in ws]
    T = ws[0].T

    def run(pipelined):
        layer = tw.VerifyCommitLayer(ws[0].S0.to(dev).clone(), ws[0].H_qk, T, 32)
        outs = [torch.empty((T, 4, 128), dtype=torch.bfloat16).pin_memory() for _ in ws]
        for h, o in zip(hosts, outs):
            (layer.step_async if pipelined else layer.step)(h, o)
        layer.synchronize()
        torch.cuda.synchronize(dev)
        assert not layer.status.any()
        return [o.clone() for o in outs], layer.S0.cpu()

    seq_O, seq_S = run(False)
    pipe_O, pipe_S = run(True)
    for a, b in zip(seq_O, pipe_O):
        assert torch.equal(a, b)
    assert torch.equal(seq_S, pipe_S)

    # round 0 against the oracle (bf16 outputs: Frobenius gate)
    _, ref = pu.run_oracle(oracle, ws[0])
    m, f = pu.worst_errors(seq_O[0].double().numpy(), ref.O, ws[0].node_offsets.numpy(), True)
    assert f <= pu.FROB_GATE
    # the state after five rounds against five rounds of the oracle, each fed the rounded state
    S = ws[0].S0.clone()
    for w in ws:
        w2 = w.select_sequences(range(w.B))
        w2.S0 = S
        _, r = pu.run_oracle(oracle, w2)
        S = torch.from_numpy(r.S_commit).to(torch.bfloat16)
    err = (seq_S.double() - S.double()).abs().max() / S.double().abs().max()
    assert float(err) < 2e-2     # a few bf16 roundings may fall the other way over five rounds
