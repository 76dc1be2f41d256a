"""Workers spread over the GPUs of one node (one process per GPU).

The paper's workers each hold their own model and pull segments from one another
(Section 3, "Segmented Pulling").  Here rank g hosts a contiguous range of the N workers;
their rows live in that GPU's memory, registered as symmetric memory so that the other
ranks can read them over NVLink.  One round on every rank:

  1. all ranks wait until every rank's rows are final (Section 4.1 step 3: a worker sends
     its segments once its local update has finished),
  2. the peer table of the round is computed locally (a pure function of the seed),
  3. ``combo_segment_aggregate_rows`` forms the hosted workers' new models, loading the
     pulled segments straight from the peers' memory (Eq. 2, Eq. 3),
  4. the new models go to the second symmetric buffer, which becomes the next round's rows.

The host-side arithmetic (who hosts whom, what crosses which link) is plain Python/numpy
and is tested on CPU; the device part needs the CUDA library.
"""
from __future__ import annotations

import numpy as np


def worker_range(rank: int, world: int, N: int) -> tuple[int, int]:
    """Workers [begin, end) hosted by ``rank``: contiguous, sizes differing by at most one."""
    if not (0 <= rank < world) or N < world:
        raise ValueError("need 0 <= rank < world <= N")
    base, extra = divmod(N, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def owner_of(w: int, world: int, N: int) -> int:
    """Rank that hosts worker ``w``."""
    base, extra = divmod(N, world)
    cut = extra * (base + 1)
    return w // (base + 1) if w < cut else extra + (w - cut) // base


def segment_lengths(P: int, S: int) -> np.ndarray:
    """Eq. 1 with L = ceil(P/S): the last segment is shorter, trailing ones may be empty."""
    L = -(-P // S)
    lo = np.minimum(np.arange(S, dtype=np.int64) * L, P)
    hi = np.minimum(lo + L, P)
    return hi - lo


def pull_traffic(idx: np.ndarray, world: int, P: int, elem_bytes: int) -> np.ndarray:
    """Bytes that rank a pulls from rank b in one round, as a [world][world] matrix (the
    diagonal is what stays inside a GPU).  idx: the round's peer table [N][S][R].  Each
    pulled segment crosses once, as in the paper (S*R segments per worker, Section 3)."""
    N, S, R = idx.shape
    seg = segment_lengths(P, S) * elem_bytes
    owners = np.array([owner_of(w, world, N) for w in range(N)])
    out = np.zeros((world, world), dtype=np.int64)
    for w in range(N):
        a = owners[w]
        for l in range(S):
            for r in range(R):
                k = int(idx[w, l, r])
                if k >= 0:
                    out[a, owners[k]] += seg[l]
    return out


def distinct_rows_read(idx: np.ndarray, world: int, rank: int, P: int) -> tuple[float, float]:
    """What the staged worker-sharded kernel reads on ``rank``, in units of whole rows (P
    elements): (local, remote).  Per segment it brings the hosted workers' own rows and every
    DISTINCT other row some hosted worker pulls -- a (peer, segment) that several hosted
    workers pull is fetched once -- so the figures are sums over segments of distinct counts
    weighted by the segment's share of the vector."""
    N, S, R = idx.shape
    a, b = worker_range(rank, world, N)
    seg = segment_lengths(P, S).astype(np.float64) / float(P)
    local = remote = 0.0
    for l in range(S):
        pulled = set(int(k) for k in idx[a:b, l, :].ravel() if k >= 0)
        others = [k for k in pulled if not (a <= k < b)]
        n_remote = sum(1 for k in others if owner_of(k, world, N) != rank)
        local += seg[l] * ((b - a) + len(others) - n_remote)
        remote += seg[l] * n_remote
    return local, remote


def row_addresses(bases, N: int, pitch_bytes: int) -> list[int]:
    """Address of every worker's row given each rank's buffer base (``bases[g]`` as rank g maps
    it): worker w lives on owner_of(w), at local row w - (first worker of that rank)."""
    world = len(bases)
    addr = []
    for w in range(N):
        o = owner_of(w, world, N)
        first, _ = worker_range(o, world, N)
        addr.append(int(bases[o]) + (w - first) * pitch_bytes)
    return addr


class ShardedFederation:
    """The hosted workers of this rank and the rounds over them.  Needs an initialised
    NCCL process group (one rank per GPU of the node) and the CUDA library."""

    def __init__(self, N: int, P: int, S: int, R: int, dtype, group=None, weights=None):
        import torch
        import torch.distributed as dist
        import torch.distributed._symmetric_memory as symm_mem

        self.torch = torch
        self.dist = dist
        self.group = group if group is not None else dist.group.WORLD
        self.rank = dist.get_rank(self.group)
        self.world = dist.get_world_size(self.group)
        self.N, self.P, self.S, self.R = N, P, S, R
        self.dtype = dtype
        self.elem_bytes = torch.empty((), dtype=dtype).element_size()
        self.w_begin, self.w_end = worker_range(self.rank, self.world, N)
        self.n_local = self.w_end - self.w_begin
        vec = 16 // self.elem_bytes
        self.pitch = -(-P // vec) * vec                      # rows start on 16-byte boundaries
        self.dev = torch.device("cuda", torch.cuda.current_device())
        # every rank allocates room for the largest share, so that the buffers are symmetric
        self.max_local = -(-N // self.world)
        self.bufs, self.handles, self.row_tables = [], [], []
        for _ in range(2):
            t = symm_mem.empty((self.max_local, self.pitch), dtype=dtype, device=self.dev)
            h = symm_mem.rendezvous(t, self.group)
            self.bufs.append(t)
            self.handles.append(h)
            addr = row_addresses([int(b) for b in h.buffer_ptrs], N, self.pitch * self.elem_bytes)
            self.row_tables.append(torch.tensor(addr, dtype=torch.int64, device=self.dev))
        self.weights = weights
        self.idx = torch.empty((N, S, max(R, 1)), dtype=torch.int32, device=self.dev)
        self.cur = 0

    def rows(self):
        """This rank's hosted models, [n_local][P] view of the current buffer."""
        return self.bufs[self.cur][: self.n_local, : self.P]

    def round(self, seed: int, rnd: int, stream=None):
        """One synchronization round; returns the view of the new hosted models."""
        from . import binding as combo
        torch = self.torch
        s = stream if stream is not None else torch.cuda.current_stream()
        # rows of every rank must be final before anybody pulls (Section 4.1 step 3), and the
        # buffer about to be overwritten must no longer be read by a peer's previous round
        s.synchronize()
        self.dist.barrier(self.group)
        combo.combo_select_peers(seed, rnd, self.N, self.S, self.R, self.idx, stream=s)
        nxt = 1 - self.cur
        combo.combo_segment_aggregate_rows(self.row_tables[self.cur], self.bufs[nxt], self.pitch,
                                           self.elem_bytes, self.weights, self.idx, self.N, self.P, self.S,
                                           self.R, self.w_begin, self.n_local, stream=s)
        self.cur = nxt
        return self.rows()
