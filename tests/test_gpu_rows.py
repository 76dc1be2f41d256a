"""Worker-sharded aggregation (Section 3 "Segmented Pulling" + Eq. 3): rows in separate
allocations, ranks emulated one after another on one GPU (each forms the models of the
workers it hosts); the union must be the oracle's round, bit for bit in the fixed order,
and identical to the dense kernel's result."""
import numpy as np
import pytest
import torch

import oracle
import paper_1908_07782_b200 as combo
from paper_1908_07782_b200 import sharding
from gpu_util import DEV, check_against_oracle, to_bits

pytestmark = pytest.mark.gpu


def make_rows(N, P, dtype, seed):
    """N rows, each its own allocation (16-byte aligned), plus the stacked copy."""
    g = torch.Generator().manual_seed(seed)
    dense = (torch.randn(N, P, generator=g) * 0.05).to(dtype).to(DEV)
    rows = [dense[j].clone() for j in range(N)]
    table = torch.tensor([r.data_ptr() for r in rows], dtype=torch.int64, device=DEV)
    assert combo.combo_check_rows(table, N) == 0
    return dense, rows, table


@pytest.mark.parametrize("N,P,S,R,world,dtype,weighted", [
    (8, 40_000, 4, 2, 1, torch.float32, False),
    (12, 70_001, 5, 3, 3, torch.float32, True),       # odd P: ragged last group, odd segment length
    (7, 33_333, 3, 2, 2, torch.float32, True),        # uneven shares
    (16, 50_002, 7, 4, 4, torch.bfloat16, False),
    (9, 1_003, 9, 8, 3, torch.bfloat16, True),        # R = N - 1: every worker pulls from all others
    (5, 300, 300, 1, 5, torch.float32, False),        # one-element segments
    (6, 4_096, 1, 0, 2, torch.float32, False),        # R = 0: identity
    (64, 120_008, 10, 4, 8, torch.float32, False),    # 8 hosted workers of 64: many shared pulls
    (128, 30_008, 16, 4, 4, torch.bfloat16, True),
    (30, 100_000, 10, 12, 3, torch.float32, True),    # the wide kernel (R > 8)
    (12, 70_000, 5, 6, 2, torch.float32, False),      # the unspecialised one
    # few hosted rows: tiles of several boxes (2, 4 and 8; bfloat16 up to 1024 columns)
    (16, 300_004, 5, 3, 1, torch.float32, True),
    (16, 300_004, 5, 3, 4, torch.float32, False),     # 4 hosted workers
    (6, 200_001, 3, 2, 1, torch.float32, False),      # 6 rows: 1024 columns per tile, ragged end
    (3, 150_000, 2, 1, 3, torch.float32, True),       # one hosted worker: 2048 columns
    (24, 260_010, 7, 4, 2, torch.bfloat16, False),
    (24, 260_010, 7, 4, 1, torch.bfloat16, True),
    # bfloat16 with unit weights: the mixed-precision sum, in each kernel instance
    (128, 30_010, 16, 4, 4, torch.bfloat16, False),
    (10, 9_999, 3, 1, 2, torch.bfloat16, False),
    (20, 40_003, 6, 6, 2, torch.bfloat16, False),
    (30, 60_000, 10, 12, 3, torch.bfloat16, False),
])
@pytest.mark.parametrize("path", [0, 3])
def test_rows_kernel_matches_oracle_and_dense_kernel(N, P, S, R, world, dtype, weighted, path):
    e = 4 if dtype == torch.float32 else 2
    dense, rows, table = make_rows(N, P, dtype, seed=N * 1000 + S)
    w = None
    if weighted:
        w = torch.randint(500, 1501, (N,), generator=torch.Generator().manual_seed(2)).float().to(DEV)
    idx = torch.empty((N, S, max(R, 1)), dtype=torch.int32, device=DEV)[:, :, :R].contiguous()
    combo.combo_select_peers(3, 1, N, S, R, idx)
    idx_np = oracle.select_peers(3, 1, N, S, R)
    vec = 16 // e
    pitch = -(-P // vec) * vec
    union = torch.empty(N, P, dtype=dtype, device=DEV)
    for rank in range(world):
        a, b = sharding.worker_range(rank, world, N)
        guard = 64
        buf = torch.full(((b - a) * pitch + 2 * guard,), 7.0, dtype=dtype, device=DEV)
        out = buf[guard:guard + (b - a) * pitch].view(b - a, pitch)
        combo.combo_set_kernel_path(path)          # 3: nothing staged; 0: staged where the tile's rows fit
        try:
            combo.combo_segment_aggregate_rows(table, out, pitch, e, w, idx, N, P, S, R, a, b - a)
        finally:
            combo.combo_set_kernel_path(0)
        torch.cuda.synchronize()
        staged_expected = path == 0 and (b - a) * P >= 65536
        assert combo.combo_last_kernel_path() == (4 if staged_expected else 3)
        assert (buf[:guard] == 7.0).all() and (buf[guard + (b - a) * pitch:] == 7.0).all()
        if pitch > P:
            assert (out[:, P:] == 7.0).all(), "write into the row padding"
        union[a:b] = out[:, :P]
    check_against_oracle(dense, union, idx_np, S, R, weights=w)
    # the dense kernels on the stacked rows give the same bits
    ref = torch.empty_like(dense)
    if dtype == torch.bfloat16:
        combo.combo_segment_aggregate_bf16(dense, ref, w, idx, N, P, S, R)
    else:
        combo.combo_segment_aggregate(dense, ref, w, idx, N, P, S, R)
    torch.cuda.synchronize()
    assert torch.equal(union.view(torch.int16 if e == 2 else torch.int32),
                       ref.view(torch.int16 if e == 2 else torch.int32))
    combo.combo_device_status()


@pytest.mark.parametrize("weighted", [True, False])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_rows_kernel_skips_pulls_that_found_no_peer(dtype, weighted):
    # a table from the online sampler holds -1 rows for offline workers and -1 pulls
    # (Section 4.2); the worker-sharded call must skip them like the dense kernels do
    N, P, S, R = 10, 20_003, 4, 3
    e = 4 if dtype == torch.float32 else 2
    dense, rows, table = make_rows(N, P, dtype, seed=5)
    w = torch.randint(500, 1501, (N,), generator=torch.Generator().manual_seed(3)).float().to(DEV) if weighted else None
    active = np.ones(N, np.uint8)
    active[[2, 7]] = 0
    idx_np = oracle.select_peers_active(4, 1, N, S, R, active)
    idx_np[0, 1, :] = -1                      # a segment left without any peer
    idx_np[5, 2, 1] = -1                      # one pull of three missing
    assert (idx_np[2] == -1).all()
    idx = torch.from_numpy(idx_np).to(DEV)
    vec = 16 // e
    pitch = -(-P // vec) * vec
    out = torch.empty(N, pitch, dtype=dtype, device=DEV)
    combo.combo_segment_aggregate_rows(table, out, pitch, e, w, idx, N, P, S, R, 0, N)
    torch.cuda.synchronize()
    got = out[:, :P].contiguous()
    want = oracle.segment_aggregate_members(to_bits(dense), idx_np, S, R, w.cpu().numpy() if weighted else None,
                                            np.zeros(N, np.uint8), ordered=True)
    assert (to_bits(got).view(np.uint8) == want.view(np.uint8)).all()
    # offline workers keep their values
    assert torch.equal(got[2], dense[2]) and torch.equal(got[7], dense[7])
    ref = torch.empty_like(dense)
    combo.combo_segment_aggregate_members(dense, ref, w, idx, None, N, P, S, R)
    torch.cuda.synchronize()
    assert torch.equal(got, ref)
    combo.combo_device_status()


def test_rows_argument_errors_and_pointer_check():
    N, P, S, R = 4, 1024, 2, 1
    dense, rows, table = make_rows(N, P, torch.float32, 1)
    idx = torch.zeros((N, S, R), dtype=torch.int32, device=DEV)
    out = torch.empty(2, P, device=DEV)
    lib = combo.load()

    def call(**kw):
        a = dict(rows=table.data_ptr(), out=out.data_ptr(), pitch=P, e=4, w=None, idx=idx.data_ptr(), N=N, P=P,
                 S=S, R=R, wb=0, nl=2)
        a.update(kw)
        return lib.combo_segment_aggregate_rows(a["rows"], a["out"], a["pitch"], a["e"], a["w"], a["idx"], a["N"],
                                                a["P"], a["S"], a["R"], a["wb"], a["nl"], None)
    assert call() == 0
    assert call(rows=None) == 1
    assert call(pitch=P - 4) == 1           # pitch below the vector length
    assert call(pitch=P + 1) == 1           # rows of the output would not start on 16 bytes
    assert call(wb=3, nl=2) == 1            # hosted range beyond N
    assert call(nl=0) == 1
    assert call(e=8) == 1
    assert call(R=N) == 1
    assert call(idx=None) == 1
    torch.cuda.synchronize()
    bad = table.clone()
    bad[2] += 4
    assert combo.combo_check_rows(bad, N) == 3
    bad[1] = 0
    assert combo.combo_check_rows(bad, N) == 2


_FEDERATION_SCRIPT = r"""
import os, sys
import numpy as np, torch, torch.distributed as dist
sys.path.insert(0, sys.argv[1])
import oracle
import paper_1908_07782_b200 as combo
from paper_1908_07782_b200.sharding import ShardedFederation
os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
os.environ.setdefault("MASTER_PORT", sys.argv[2])
torch.cuda.set_device(0)
dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
N, P, S, R = 6, 10_001, 4, 2
fed = ShardedFederation(N, P, S, R, torch.float32)
g = torch.Generator().manual_seed(4)
x0 = torch.randn(N, P, generator=g) * 0.05
fed.rows().copy_(x0.cuda())
cur = x0.numpy()
for t in range(3):
    got = fed.round(5, t)
    cur = oracle.segment_aggregate_ordered_f32(cur, oracle.select_peers(5, t, N, S, R), S, R)
torch.cuda.synchronize()
assert (got.cpu().numpy().view(np.uint32) == cur.view(np.uint32)).all()
combo.combo_device_status()
dist.destroy_process_group()
print("federation ok")
"""


def test_sharded_federation_single_rank(tmp_path):
    """The multi-GPU driver (symmetric memory, row tables, barriers) with a process group of
    one rank: three chained rounds equal the oracle's chain."""
    import os
    import socket
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    script = tmp_path / "fed.py"
    script.write_text(_FEDERATION_SCRIPT)
    r = subprocess.run([sys.executable, str(script), root, str(port)], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and "federation ok" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]
