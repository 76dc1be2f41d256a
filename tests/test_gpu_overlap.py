"""Launch overlap (programmatic stream serialization): chained rounds issued back to
back on one stream give the same bits with and without it, and match the oracle chain.

Section 4.1: pull requests do not depend on the local update, so the peer sampler may run
ahead; it must still not overwrite the table the preceding aggregation reads."""
import numpy as np
import pytest
import torch

import oracle
import paper_1908_07782_b200 as combo
from gpu_util import DEV

pytestmark = pytest.mark.gpu


def run_chain(x0, weights, seed, rounds, S, R, overlap, stream, bf16=False):
    N, P = x0.shape
    combo.combo_set_launch_overlap(overlap)
    try:
        bufs = [x0.clone(), torch.empty_like(x0)]
        idx = torch.empty((N, S, R), dtype=torch.int32, device=DEV)
        with torch.cuda.stream(stream):
            cur = 0
            for t in range(rounds):
                combo.combo_select_peers(seed, t, N, S, R, idx, stream=stream)
                if bf16:
                    combo.combo_segment_aggregate_bf16(bufs[cur], bufs[1 - cur], weights, idx, N, P, S, R,
                                                       stream=stream)
                else:
                    combo.combo_segment_aggregate(bufs[cur], bufs[1 - cur], weights, idx, N, P, S, R,
                                                  stream=stream)
                cur = 1 - cur
        stream.synchronize()
        combo.combo_device_status()
        return bufs[cur].clone(), idx.clone()
    finally:
        combo.combo_set_launch_overlap(True)


@pytest.mark.parametrize("N,P,S,R,rounds", [(8, 300_000, 4, 2, 7), (32, 70_001, 8, 3, 5), (16, 1_048_576, 32, 4, 4)])
def test_chained_rounds_same_bits_with_and_without_overlap(N, P, S, R, rounds):
    g = torch.Generator().manual_seed(5)
    x0 = (torch.randn(N, P, generator=g) * 0.05).to(DEV)
    w = torch.randint(500, 1501, (N,), generator=g).float().to(DEV)
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    a, idx_a = run_chain(x0, w, 11, rounds, S, R, True, st)
    b, idx_b = run_chain(x0, w, 11, rounds, S, R, False, st)
    assert torch.equal(idx_a, idx_b)
    assert torch.equal(a.view(torch.int32), b.view(torch.int32))
    # the oracle's fixed-order chain, round by round
    cur = x0.cpu().numpy()
    wn = w.cpu().numpy()
    for t in range(rounds):
        idx_t = oracle.select_peers(11, t, N, S, R)
        cur = oracle.segment_aggregate_ordered_f32(cur, idx_t, S, R, weights=wn)
    assert (idx_a.cpu().numpy() == idx_t).all()
    assert (a.cpu().numpy().view(np.uint32) == cur.view(np.uint32)).all()


def test_chained_rounds_bf16_unaligned_rows():
    N, P, S, R, rounds = 12, 50_002, 3, 4, 5          # pitch 4 mod 16 bytes: word mode
    g = torch.Generator().manual_seed(6)
    x0 = (torch.randn(N, P, generator=g) * 0.02).to(torch.bfloat16).to(DEV)
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    a, _ = run_chain(x0, None, 3, rounds, S, R, True, st, bf16=True)
    b, _ = run_chain(x0, None, 3, rounds, S, R, False, st, bf16=True)
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_graph_replay_of_overlapped_rounds():
    N, P, S, R, rounds = 8, 262_144, 4, 2, 6
    g = torch.Generator().manual_seed(7)
    x0 = (torch.randn(N, P, generator=g) * 0.05).to(DEV)
    bufs = [x0.clone(), torch.empty_like(x0)]
    idx = torch.empty((N, S, R), dtype=torch.int32, device=DEV)
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())

    def body():
        cur = 0
        for t in range(rounds):
            combo.combo_select_peers(9, t, N, S, R, idx, stream=st)
            combo.combo_segment_aggregate(bufs[cur], bufs[1 - cur], None, idx, N, P, S, R, stream=st)
            cur = 1 - cur
        return cur

    with torch.cuda.stream(st):
        body()                                   # first calls outside the capture (set-up)
        st.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=st):
            last = body()
        for _ in range(3):
            bufs[0].copy_(x0)
            graph.replay()
    st.synchronize()
    combo.combo_device_status()
    cur = x0.cpu().numpy()
    for t in range(rounds):
        cur = oracle.segment_aggregate_ordered_f32(cur, oracle.select_peers(9, t, N, S, R), S, R)
    assert (bufs[last].cpu().numpy().view(np.uint32) == cur.view(np.uint32)).all()
