"""A compression-phase step across several processes, one GPU each.

The paper runs its workers on separate GPUs and moves the 1-bit messages with a Gather-Scatter
AllReduce (Figure 1; Section 3.3 steps 3 and 5): every worker sends the k-th part of its
compressed momentum to worker k, worker k averages and recompresses what it received, and sends
the result back to everybody.  `ShardedStep` does exactly that between the phases of the
library's phase-wise step (apms_worker_phase / apms_server_phase / apms_apply_phase): process r
holds `n_local` workers and serves a contiguous range of chunks; exchange 1 is a set of
point-to-point transfers of (sign words, scales) shards, exchange 2 an all-gather of the server
shards.  Only packed sign words and chunk scales cross the wire (d/8 + 4 C bytes per worker and
direction instead of 4 d).

The arithmetic stays in the library: this module only slices, sends and receives.  The rows a
server averages are ordered by global worker index (rank * n_local + i), so P processes with
n_local workers each give bit for bit the result of one context with P * n_local workers.

`backend` is anything with the attributes d, n, chunk, C, W and the methods worker_phase(grads),
message(i) -> (sign-word tensor, scale tensor) views (i = -1: the server's message),
server_phase(bits_rows, scale_rows, chunk_begin, chunk_end) and apply_phase(): a
`binding.Context` on a GPU, or a CPU stand-in in the tests of the exchange logic.

`PeerShardedStep` is the one-node form in which the GPUs move the messages themselves: every process
maps its peers' workspaces once (CUDA IPC), the server kernel then loads its rows straight from the
workers' message buffers wherever they lie (exchange 1 costs no copy and no staging buffer: the
transfer is the kernel's own loads over NVLink), and each process stores its range of the server
message into every peer's buffer (exchange 2).  `torch.distributed` carries only the handles and
two host barriers per step.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple


def chunk_ranges(n_chunks: int, world: int) -> List[Tuple[int, int]]:
    """Contiguous, near-equal ranges of chunks, one per process (the paper's 'k-th chunk to worker k')."""
    return [(r * n_chunks // world, (r + 1) * n_chunks // world) for r in range(world)]


def chunk_for_servers(d: int, servers: int) -> int:
    """The paper's own layout has one chunk per worker-as-server (Section 3.3: the vector is cut into n
    chunks).  This is that chunk length: d / servers rounded up to the next multiple of 32 elements (a
    chunk holds whole sign words); the last chunk is shorter when d is not a multiple of it."""
    per = -(-d // servers)
    return -(-per // 32) * 32


def word_range(chunk_begin: int, chunk_end: int, chunk: int, d: int) -> Tuple[int, int]:
    """Sign words [w0, w1) that hold the elements of chunks [chunk_begin, chunk_end)."""
    first = chunk_begin * chunk
    last = min(chunk_end * chunk, d)
    return first // 32, (last + 31) // 32


def _round4(words: int) -> int:
    return (words + 3) // 4 * 4


class ShardedStep:
    def __init__(self, backend, group=None):
        import torch.distributed as dist

        self.b = backend
        self.dist = dist
        self.group = group
        self.rank = dist.get_rank(group)
        self.world = dist.get_world_size(group)
        if backend.C < self.world:
            raise ValueError(f"{backend.C} chunks cannot be served by {self.world} processes")
        self.ranges = chunk_ranges(backend.C, self.world)
        self.words = [word_range(cb, ce, backend.chunk, backend.d) for cb, ce in self.ranges]
        self.row_words = [_round4(w1 - w0) for w0, w1 in self.words]
        # what accompanies the sign words: one scale per chunk - or, with the top-k compressor, where the words are
        # a selection mask, the chunk's kept values (`per` = ceil(fraction * chunk) floats per chunk)
        self.topk = bool(getattr(backend, "topk", False))
        self.per = backend.topk_values_per_chunk() if self.topk else 1
        self.row_scales = [(ce - cb) * self.per for cb, ce in self.ranges]
        self._buffers = None
        self._sends = []
        self._packed = None

    # ------------------------------------------------------------------ buffers (made once)
    def _make_buffers(self, like_bits, like_scales):
        import torch

        n, me = self.b.n, self.rank
        dev = like_bits.device
        mk = lambda shape, dt: torch.zeros(shape, dtype=dt, device=dev)
        self._buffers = {
            "recv_bits": mk((self.world * n, self.row_words[me]), like_bits.dtype),
            "recv_scales": mk((self.world * n, self.row_scales[me]), like_scales.dtype),
            "gather_bits": mk((self.world, max(self.row_words)), like_bits.dtype),
            "gather_scales": mk((self.world, max(self.row_scales)), like_scales.dtype),
            "mine_bits": mk((max(self.row_words),), like_bits.dtype),
            "mine_scales": mk((max(self.row_scales),), like_scales.dtype),
        }

    def global_rank(self, k: int) -> int:
        return k if self.group is None else self.dist.get_global_rank(self.group, k)

    # ------------------------------------------------------------------ the step
    def step(self, grads: Sequence) -> None:
        """Section 3.3 steps 1-6 for this process's workers; `grads`: its n_local gradients.

        The worker phase runs range by range, in the order of the serving processes (the same order on every
        process, so that the grouped transfers of a range pair up like one gather and cannot deadlock): as soon
        as the kernels of range k are enqueued, this process's rows of that range are handed - straight from
        the message buffers, no packing - to the transfer to process k, which runs while the later ranges are
        still being compressed.  Transfers are
        stream-ordered after the kernels (NCCL) - nothing waits on the host until the server phase needs the
        received rows."""
        b, dist, n, me = self.b, self.dist, self.b.n, self.rank
        for req in self._sends:                                                 # the previous step's transfers have read the messages
            req.wait()
        self._sends = []
        ranged = hasattr(b, "worker_phase_range") and not self.topk
        if not ranged:
            b.worker_phase(grads)                                               # steps 1-2, whole vector
        msgs = [b.message(i) for i in range(n)]
        if self.topk:                                                           # the kept values, packed chunk by chunk
            import torch

            if self._packed is None:
                self._packed = [torch.zeros(b.C * self.per, dtype=torch.float32, device=msgs[0][0].device) for _ in range(n + 1)]
            for i in range(n):
                b.topk_pack_values(i, 0, b.C, self._packed[i])
            msgs = [(msgs[i][0], self._packed[i]) for i in range(n)]
        if self._buffers is None:
            self._make_buffers(msgs[0][0], msgs[0][1])
        buf = self._buffers
        per = self.per
        recvs = []
        for k in range(self.world):
            (w0, w1), (cb, ce) = self.words[k], self.ranges[k]
            if ranged:
                b.worker_phase_range(grads, cb, ce)                             # steps 1-2 for the chunks process k serves
            # step 3 (exchange 1): the part of every local message that process k serves goes to process k,
            # straight from the message buffers (a contiguous piece of each) into the receiver's rows
            ops = []
            if k == me:
                for q in range(self.world):
                    for i in range(n):
                        row = q * n + i
                        if q == me:
                            buf["recv_bits"][row, :w1 - w0].copy_(msgs[i][0][w0:w1])
                            buf["recv_scales"][row, :(ce - cb) * per].copy_(msgs[i][1][cb * per:ce * per])
                            continue
                        peer = self.global_rank(q)
                        ops.append(dist.P2POp(dist.irecv, buf["recv_bits"][row, :w1 - w0], peer, self.group))
                        ops.append(dist.P2POp(dist.irecv, buf["recv_scales"][row, :(ce - cb) * per], peer, self.group))
            else:
                peer = self.global_rank(k)
                for bits, scales in msgs:
                    ops.append(dist.P2POp(dist.isend, bits[w0:w1], peer, self.group))
                    ops.append(dist.P2POp(dist.isend, scales[cb * per:ce * per], peer, self.group))
            if ops:
                (recvs if k == me else self._sends).extend(dist.batch_isend_irecv(ops))
        for req in recvs:
            req.wait()

        # step 4: average and recompress the chunks this process serves
        cb, ce = self.ranges[me]
        if self.topk:
            b.topk_server_phase(buf["recv_bits"], buf["recv_scales"], cb, ce)   # and steps 5-6 for the elements it keeps
        else:
            b.server_phase(buf["recv_bits"], buf["recv_scales"], cb, ce)

        # step 5 (exchange 2): every process's range of the server message goes to everybody
        sbits, sscales = b.message(-1)
        w0, w1 = self.words[me]
        buf["mine_bits"][:w1 - w0].copy_(sbits[w0:w1])
        if self.topk:
            b.topk_pack_values(-1, cb, ce, self._packed[n])
            buf["mine_scales"][:(ce - cb) * per].copy_(self._packed[n][:(ce - cb) * per])
        else:
            buf["mine_scales"][:ce - cb].copy_(sscales[cb:ce])
        if self.world > 1:
            dist.all_gather_into_tensor(buf["gather_bits"].view(-1), buf["mine_bits"], group=self.group)
            dist.all_gather_into_tensor(buf["gather_scales"].view(-1), buf["mine_scales"], group=self.group)
            for k in range(self.world):
                if k == me:
                    continue
                (v0, v1), (kb, ke) = self.words[k], self.ranges[k]
                if self.topk:                                                   # mask, kept values to their places, steps 5-6 for them
                    b.topk_put_server_range(buf["gather_bits"][k], buf["gather_scales"][k], kb, ke)
                else:
                    sbits[v0:v1].copy_(buf["gather_bits"][k, :v1 - v0])
                    sscales[kb:ke].copy_(buf["gather_scales"][k, :ke - kb])

        b.apply_phase()                                                         # steps 5-6

    def wire_bytes_per_step(self) -> int:
        """Bytes this process sends per step (both exchanges), for comparison with 4 d per worker."""
        n, me = self.b.n, self.rank
        ex1 = sum(4 * n * ((self.words[k][1] - self.words[k][0]) + self.row_scales[k]) for k in range(self.world) if k != me)
        ex2 = (self.world - 1) * 4 * (self.row_words[me] + self.row_scales[me])
        return ex1 + ex2


class HostFlags:
    """Step counters shared by the processes of one node (POSIX shared memory): flag [r, k] is the number of
    the last step in which process r finished its part of stage k.  Processes tell each other on the host
    how far they are - no kernel ever waits for another process.  A wait that lasts longer than `timeout_s`
    raises: a peer that died or never joined shows up as an error on the host, with every GPU still usable."""

    def __init__(self, dist, group, world: int, stages: int, timeout_s: float = 120.0):
        import numpy as np
        from multiprocessing import shared_memory

        self.rank, self.world, self.timeout_s = dist.get_rank(group), world, timeout_s
        name = [None]
        if self.rank == 0:
            self._shm = shared_memory.SharedMemory(create=True, size=8 * world * stages)
            name[0] = self._shm.name
        dist.broadcast_object_list(name, src=0 if group is None else dist.get_global_rank(group, 0), group=group)
        if self.rank != 0:
            self._shm = shared_memory.SharedMemory(name=name[0])
        self.flags = np.ndarray((world, stages), dtype=np.int64, buffer=self._shm.buf)
        if self.rank == 0:
            self.flags[:] = 0
        dist.barrier(group=group)

    def post(self, stage: int, step: int) -> None:
        self.flags[self.rank, stage] = step

    def wait_all(self, stage: int, step: int) -> None:
        import time

        t0 = time.monotonic()
        while True:
            if (self.flags[:, stage] >= step).all():
                return
            if time.monotonic() - t0 > self.timeout_s:
                late = [r for r in range(self.world) if self.flags[r, stage] < step]
                raise RuntimeError(f"processes {late} did not reach stage {stage} of step {step} within {self.timeout_s} s")
            time.sleep(0)

    def close(self, dist, group) -> None:
        self.flags = None
        dist.barrier(group=group)
        self._shm.close()
        if self.rank == 0:
            self._shm.unlink()


class PeerShardedStep:
    """Section 3.3 steps 1-6 across processes of one node, the exchanges done by peer loads and stores.

    `backend`: a `binding.Context` made with library_workspace=True (its workspace must be exportable);
    `peers`: what opens and closes a handle - by default the binding's apms_ipc_open / apms_ipc_close.
    No kernel waits on another GPU: the processes tell each other on the host (`HostFlags`) which part of
    their messages is complete.  The worker phase runs range by range, every process starting with the range
    after its own, so the range a process serves is finished everywhere one range before the end of the
    worker phase: its server phase does not wait for the slowest process's last kernel.

    With the top-k compressor (a backend with a torch workspace and set_compressor(TOPK) done) the messages are
    stored, not loaded: see _init_topk.
    """

    def __init__(self, backend, group=None, peers=None, timeout_s: float = 120.0, share=None):
        import torch.distributed as dist

        self.b, self.dist, self.group = backend, dist, group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)
        if backend.C < self.world:
            raise ValueError(f"{backend.C} chunks cannot be served by {self.world} processes")
        if peers is None:
            from . import binding as peers
        self._peers = peers
        self.ranges = chunk_ranges(backend.C, self.world)
        self.steps = 0
        self.base = []
        self.topk = bool(getattr(backend, "topk", False))
        if self.topk:
            self._init_topk(share, timeout_s)
            return
        n = backend.n
        self.off = {i: backend.message_offsets(i) for i in range(-1, n)}
        mine = (backend.ipc_export(), (backend.d, n, backend.chunk), tuple(sorted(self.off.items())))
        everyone = [None] * self.world
        dist.all_gather_object(everyone, mine, group=group)
        for r, (_, shape, off) in enumerate(everyone):
            if shape != mine[1] or off != mine[2]:
                raise ValueError(f"process {r} holds a context of another shape: {shape} against {mine[1]}")
        own_base = backend.message_ptrs(0)[0] - self.off[0][0]
        self.base = [own_base if r == self.rank else peers.apms_ipc_open(h) for r, (h, _, _) in enumerate(everyone)]
        # stages 0 .. world-1: "my workers' messages for range k are complete"; stage world: "my server range is stored everywhere"
        self.flags = HostFlags(dist, group, self.world, self.world + 1, timeout_s)
        self.order = [(self.rank + 1 + j) % self.world for j in range(self.world)]      # own range last
        dist.barrier(group=group)

    # ------------------------------------------------------------------ the top-k compressor
    def _init_topk(self, share, timeout_s):
        """With the top-k compressor a message is a selection mask plus the kept values, packed (Section 5.1);
        packing is a kernel of its own, so it writes straight into the serving process's receive rows: device
        buffers that every process makes for its own range and shares with its peers (`share`: a pair of
        functions (export(tensor) -> picklable, open(picklable) -> tensor); by default torch's CUDA IPC
        reductions).  The backend needs a torch workspace here (the masks are read through its message views)."""
        import torch

        b, dist, n, me = self.b, self.dist, self.b.n, self.rank
        if share is None:
            from torch.multiprocessing.reductions import reduce_tensor

            share = (reduce_tensor, lambda handle: handle[0](*handle[1]))
        export, open_ = share
        self.per = b.topk_values_per_chunk()
        self.words = [word_range(cb, ce, b.chunk, b.d) for cb, ce in self.ranges]
        self.row_words = [_round4(w1 - w0) for w0, w1 in self.words]
        self.row_vals = [(ce - cb) * self.per for cb, ce in self.ranges]
        bits0 = b.message(0)[0]
        mk = lambda shape, dt: torch.zeros(shape, dtype=dt, device=bits0.device)
        self.own = {"recv_bits": mk((self.world * n, self.row_words[me]), bits0.dtype),
                    "recv_vals": mk((self.world * n, self.row_vals[me]), torch.float32),
                    "gather_bits": mk((self.world, max(self.row_words)), bits0.dtype),
                    "gather_vals": mk((self.world, max(self.row_vals)), torch.float32)}
        mine = ({k: export(t) for k, t in self.own.items()}, (b.d, n, b.chunk, self.per))
        everyone = [None] * self.world
        dist.all_gather_object(everyone, mine, group=self.group)
        for r, (_, shape) in enumerate(everyone):
            if shape != mine[1]:
                raise ValueError(f"process {r} holds a context of another shape: {shape} against {mine[1]}")
        self.bufs = [self.own if r == me else {k: open_(h) for k, h in handles.items()} for r, (handles, _) in enumerate(everyone)]
        # stage 0: "my workers' rows are stored in every serving process"; stage 1: "my server range is stored everywhere"
        self.flags = HostFlags(dist, self.group, self.world, 2, timeout_s)
        dist.barrier(group=self.group)

    def _step_topk(self, grads: Sequence) -> None:
        b, n, me, flags, per = self.b, self.b.n, self.rank, self.flags, self.per
        self.steps += 1
        b.worker_phase(grads)                                                   # steps 1-2 (top-k: the whole vector)
        for k in range(self.world):                                             # step 3: masks and packed values into process k's rows
            (w0, w1), (cb, ce) = self.words[k], self.ranges[k]
            dst = self.bufs[k]
            for i in range(n):
                row = me * n + i
                dst["recv_bits"][row, :w1 - w0].copy_(b.message(i)[0][w0:w1])
                b.topk_pack_values(i, cb, ce, dst["recv_vals"][row, :(ce - cb) * per])
        b.synchronize()
        flags.post(0, self.steps)
        flags.wait_all(0, self.steps)                                           # every process's rows of my range have arrived
        cb, ce = self.ranges[me]
        w0, w1 = self.words[me]
        b.topk_server_phase(self.own["recv_bits"], self.own["recv_vals"], cb, ce)   # step 4, and steps 5-6 for the elements it keeps
        mine_vals = self.own["gather_vals"][me, :(ce - cb) * per]
        b.topk_pack_values(-1, cb, ce, mine_vals)
        sbits = b.message(-1)[0]
        for r in range(self.world):                                             # step 5: my range of the server's message to every peer
            if r != me:
                self.bufs[r]["gather_bits"][me, :w1 - w0].copy_(sbits[w0:w1])
                self.bufs[r]["gather_vals"][me, :(ce - cb) * per].copy_(mine_vals)
        b.synchronize()
        flags.post(1, self.steps)
        flags.wait_all(1, self.steps)                                           # every range is stored everywhere
        for k in range(self.world):
            if k != me:
                kb, ke = self.ranges[k]
                b.topk_put_server_range(self.own["gather_bits"][k], self.own["gather_vals"][k], kb, ke)
        b.apply_phase()

    def row_pointers(self):
        """(sign-word addresses, scale addresses) of all world * n senders' rows for this process's chunk range,
        in global worker order."""
        cb, ce = self.ranges[self.rank]
        w0, _ = word_range(cb, ce, self.b.chunk, self.b.d)
        bits = [self.base[r] + self.off[i][0] + 4 * w0 for r in range(self.world) for i in range(self.b.n)]
        scales = [self.base[r] + self.off[i][1] + 4 * cb for r in range(self.world) for i in range(self.b.n)]
        return bits, scales

    def step(self, grads: Sequence) -> None:
        if self.topk:
            return self._step_topk(grads)
        b, me, flags = self.b, self.rank, self.flags
        self.steps += 1
        events = []
        for k in self.order:                                                    # steps 1-2, range by range
            b.worker_phase_range(grads, *self.ranges[k])
            events.append((k, b.record_event()))
        for k, ev in events:
            ev.synchronize()
            flags.post(k, self.steps)                                           # my rows of range k may be read
        flags.wait_all(me, self.steps)                                          # every process's rows of my range are complete
        cb, ce = self.ranges[me]
        bits, scales = self.row_pointers()
        b.server_phase_rows(bits, scales, cb, ce)                               # steps 3-4: the kernel loads the rows
        for r in range(self.world):                                             # step 5: my range to every peer
            if r != me:
                b.put_server_range(self.base[r] + self.off[-1][0], self.base[r] + self.off[-1][1], cb, ce)
        b.synchronize()
        flags.post(self.world, self.steps)
        flags.wait_all(self.world, self.steps)                                  # every range is stored everywhere
        b.apply_phase()                                                         # steps 5-6

    def close(self):
        """Unmaps the peers' workspaces.  Collective: returns when every process has unmapped, so that each may
        then free its own workspace."""
        self.dist.barrier(group=self.group)                                     # nobody reads a mapping that goes away
        if self.topk:
            self.b.synchronize()
            self.bufs = []                                                      # the peers' buffers are unmapped with their last reference
        for r, base in enumerate(self.base):
            if r != self.rank and base is not None:
                self._peers.apms_ipc_close(base)
        self.base = []
        self.flags.close(self.dist, self.group)
        self.dist.barrier(group=self.group)                                     # nobody frees memory that is still mapped

    def wire_bytes_per_step(self) -> int:
        """Bytes that cross between GPUs per step because of this process: the rows it loads from peers and the
        range it stores to them."""
        cb, ce = self.ranges[self.rank]
        w0, w1 = word_range(cb, ce, self.b.chunk, self.b.d)
        if self.topk:                                                           # what it stores into peers: its workers' rows, its server range
            ex1 = sum(4 * self.b.n * ((self.words[k][1] - self.words[k][0]) + self.row_vals[k]) for k in range(self.world) if k != self.rank)
            return ex1 + (self.world - 1) * 4 * ((w1 - w0) + self.row_vals[self.rank])
        per_row = 4 * (w1 - w0) + 4 * (ce - cb)
        return (self.world - 1) * self.b.n * per_row + (self.world - 1) * per_row
