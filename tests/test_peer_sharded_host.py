"""The peer form of the multi-process step (sharded.PeerShardedStep) on CPU: two gloo ranks, two workers each.

On GPUs the processes map each other's workspaces and exchange nothing but loads and stores.  Here the
"workspace" of a rank is a block of POSIX shared memory that holds its message buffers, a "device address"
is (rank + 1) << 40 plus a byte offset, and the stand-in for the library's phases dereferences such
addresses - so what is under test is exactly what PeerShardedStep computes: the row addresses in global
worker order, the chunk and word offsets of a rank's range, the destination addresses of the server range,
and the order of phases and barriers.  The arithmetic is the numpy stand-in of test_sharded_host.py; the
result must equal a single four-worker run of the C oracle."""
import os
import sys
from multiprocessing import shared_memory

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))

from test_sharded_host import CHUNK, D, N_TOTAL, OracleBackend, _free_port, _inputs, _reference

SHIFT = 40


class FakePeers:
    """Opens 'handles' (rank and shared-memory name) and resolves fake device addresses."""

    def __init__(self):
        self.blocks = {}                                          # owner rank -> (SharedMemory, numpy byte view)
        self.opened, self.closed = [], []

    def register(self, rank, shm):
        self.blocks[rank] = (shm, np.ndarray((shm.size,), dtype=np.uint8, buffer=shm.buf))

    def apms_ipc_open(self, handle: bytes) -> int:
        rank, name = handle.decode().split(":")
        self.register(int(rank), shared_memory.SharedMemory(name=name))
        self.opened.append(int(rank))
        return (int(rank) + 1) << SHIFT

    def apms_ipc_close(self, base: int):
        rank = (base >> SHIFT) - 1
        shm, _ = self.blocks.pop(rank)
        shm.close()
        self.closed.append(rank)

    def at(self, ptr: int, count: int, dtype):
        _, view = self.blocks[(ptr >> SHIFT) - 1]
        off = ptr & ((1 << SHIFT) - 1)
        return view[off:off + count * np.dtype(dtype).itemsize].view(dtype)


class PeerOracleBackend(OracleBackend):
    """OracleBackend whose messages live in shared memory and are reachable through fake addresses."""

    def __init__(self, rank, peers, d, n, chunk, x0, v, m):
        super().__init__(d, n, chunk, x0, v, m)
        self.rank, self.peers = rank, peers
        row = 256 * ((4 * self.W + 255) // 256) + 256 * ((4 * self.C + 255) // 256)
        self.shm = shared_memory.SharedMemory(create=True, size=row * (n + 1))
        peers.register(rank, self.shm)
        self._off = {}
        for k, i in enumerate(list(range(n)) + [-1]):
            self._off[i] = (k * row, k * row + 256 * ((4 * self.W + 255) // 256))
        base = (rank + 1) << SHIFT
        # the stand-in's message arrays become views onto the shared block (index n = the server's, as in the base class)
        for k, i in enumerate(list(range(n)) + [-1]):
            self.bits[k] = torch.from_numpy(peers.at(base + self._off[i][0], self.W, np.int32))
            self.scales[k] = torch.from_numpy(peers.at(base + self._off[i][1], self.C, np.float32))
            self.bits[k].zero_(); self.scales[k].zero_()

    def message_offsets(self, i):
        return self._off[i]

    def message_ptrs(self, i):
        base = (self.rank + 1) << SHIFT
        return base + self._off[i][0], base + self._off[i][1]

    def ipc_export(self) -> bytes:
        return f"{self.rank}:{self.shm.name}".encode()

    def synchronize(self):
        pass

    def server_phase_rows(self, bits_ptrs, scale_ptrs, cb, ce):
        lo, hi = cb * self.chunk, min(self.d, ce * self.chunk)
        nwords = (hi + 31) // 32 - lo // 32
        bits_rows = torch.stack([torch.from_numpy(self.peers.at(p, nwords, np.int32).copy()) for p in bits_ptrs])
        scale_rows = torch.stack([torch.from_numpy(self.peers.at(p, ce - cb, np.float32).copy()) for p in scale_ptrs])
        self.server_phase(bits_rows, scale_rows, cb, ce)

    def put_server_range(self, dst_bits, dst_scales, cb, ce):
        lo, hi = cb * self.chunk, min(self.d, ce * self.chunk)
        w0, w1 = lo // 32, (hi + 31) // 32
        self.peers.at(dst_bits + 4 * w0, w1 - w0, np.int32)[:] = self.bits[-1].numpy()[w0:w1]
        self.peers.at(dst_scales + 4 * cb, ce - cb, np.float32)[:] = self.scales[-1].numpy()[cb:ce]

    def release(self):
        self.bits, self.scales = [], []
        self.peers.blocks.pop(self.rank, None)
        self.shm.close()
        self.shm.unlink()


def _rank_main(rank, world, port, out):
    from paper_2008_11343_b200 import sharded

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    x0, v, m, grads = _inputs()
    n_local = N_TOTAL // world
    peers = FakePeers()
    backend = PeerOracleBackend(rank, peers, D, n_local, CHUNK, x0, v, m)
    step = sharded.PeerShardedStep(backend, peers=peers)
    bits_ptrs, scale_ptrs = step.row_pointers()
    order_ok = [(p >> SHIFT) - 1 for p in bits_ptrs] == [r for r in range(world) for _ in range(n_local)]
    for gs in grads:
        step.step([torch.from_numpy(g) for g in gs[rank * n_local:(rank + 1) * n_local]])
    ref = _reference()
    ok = bool(order_ok and np.array_equal(backend.x, ref.x) and np.array_equal(backend.m, ref.m)
              and np.array_equal(backend.bits[-1].numpy().view(np.uint32), ref.server_bits)
              and np.array_equal(backend.scales[-1].numpy(), ref.server_scales))
    for i in range(n_local):
        ok = ok and bool(np.array_equal(backend.err[i], ref.worker_err(rank * n_local + i)))
    # the worker phase ran range by range, starting after the rank's own range and ending with it
    own_last = [step.ranges[(rank + 1 + j) % world] for j in range(world)]
    ok = ok and backend.ranges_seen == own_last * len(grads) and own_last[-1] == step.ranges[rank]
    wire = step.wire_bytes_per_step()
    step.close()
    ok = ok and peers.opened == [r for r in range(world) if r != rank] and sorted(peers.closed) == peers.opened
    dist.barrier()
    backend.release()
    out[rank] = (ok, wire)
    dist.destroy_process_group()


def test_two_ranks_exchange_by_peer_addresses_and_equal_one_four_worker_run():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] and res[1][0]
    assert max(res[0][1], res[1][1]) < 0.1 * 4 * D * (N_TOTAL // world)


def _flags_main(rank, world, port, out):
    from paper_2008_11343_b200 import sharded

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    flags = sharded.HostFlags(dist, None, world, 2, timeout_s=0.5)
    flags.post(0, 1)
    flags.wait_all(0, 1)                                        # both ranks posted stage 0 of step 1
    seen = ""
    if rank == 0:
        flags.post(1, 1)
        try:
            flags.wait_all(1, 1)                                # rank 1 never reports stage 1
        except RuntimeError as exc:
            seen = str(exc)
    dist.barrier()
    flags.close(dist, None)
    out[rank] = seen
    dist.destroy_process_group()


def test_a_process_that_never_reports_is_an_error_on_the_host_not_a_hang():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_flags_main, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert "processes [1] did not reach stage 1 of step 1" in res[0] and res[1] == ""
