"""The multi-process step (paper_2008_11343_b200/sharded.py) on CPU: two gloo ranks, two workers each, exchange
the 1-bit messages as in Figure 1 and must end where a single four-worker run of the C oracle ends.

The arithmetic of the ranks is a numpy stand-in built on the oracle's compressor (this file only; the product's
arithmetic lives in the CUDA library and cannot run here) - what is under test is the slicing, the point-to-point
exchange, the row order of the average and the all-gather of the server shards."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

D, CHUNK, N_TOTAL = 7 * 256 + 100, 256, 4
BETA1, LR, EPS = 0.9, 1e-3, 1e-8


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _fma32(a, b, c):
    """float32 fma through float64 (the product is exact there)."""
    return (np.float64(a) * b.astype(np.float64) + c.astype(np.float64)).astype(np.float32)


class OracleBackend:
    """Phase-wise step of `n` local workers in numpy + the oracle's compressor."""

    def __init__(self, d, n, chunk, x0, v, m):
        from oracle import apms_oracle as ao

        self.ao = ao
        self.d, self.n, self.chunk = d, n, chunk
        self.C, self.W = (d + chunk - 1) // chunk, (d + 31) // 32
        self.x, self.v, self.m = x0.copy(), v.copy(), m.copy()
        self.err = [np.zeros(d, np.float32) for _ in range(n)]
        self.server_err = np.zeros(d, np.float32)
        self.bits = [torch.zeros(self.W, dtype=torch.int32) for _ in range(n + 1)]       # last = server
        self.scales = [torch.zeros(self.C, dtype=torch.float32) for _ in range(n + 1)]
        self.ranges_seen = []

    def _chunks(self, cb, ce):
        for c in range(cb, ce):
            yield c, c * self.chunk, min(self.d, (c + 1) * self.chunk)

    def message(self, i):
        return self.bits[i], self.scales[i]

    def worker_phase(self, grads):
        self.worker_phase_range(grads, 0, self.C)

    def record_event(self):
        class Done:                                                # the stand-in works synchronously
            def synchronize(self):
                pass
        return Done()

    def worker_phase_range(self, grads, cb, ce):
        self.ranges_seen.append((cb, ce))
        omb1 = np.float32(1.0) - np.float32(BETA1)
        for i, g in enumerate(grads):
            g = g.numpy()
            for c, lo, hi in self._chunks(cb, ce):
                z = _fma32(np.float32(BETA1), self.m[lo:hi], omb1 * g[lo:hi]) + self.err[i][lo:hi]
                bits, s = self.ao.compress_1bit(z)
                self.err[i][lo:hi] = z - self.ao.decompress_1bit(bits, s, hi - lo)
                self.bits[i].numpy().view(np.uint32)[lo // 32:lo // 32 + bits.size] = bits
                self.scales[i][c] = float(s)

    def server_phase(self, bits_rows, scale_rows, cb, ce):
        rows = bits_rows.shape[0]
        w_first = cb * self.chunk // 32
        for c, lo, hi in self._chunks(cb, ce):
            acc = np.zeros(hi - lo, np.float32)
            for j in range(rows):                                   # row order = global worker order
                words = bits_rows[j].numpy().view(np.uint32)[lo // 32 - w_first:(hi + 31) // 32 - w_first]
                acc = acc + self.ao.decompress_1bit(words, scale_rows[j, c - cb].item(), hi - lo)
            z = acc / np.float32(rows) + self.server_err[lo:hi]
            bits, s = self.ao.compress_1bit(z)
            self.server_err[lo:hi] = z - self.ao.decompress_1bit(bits, s, hi - lo)
            self.bits[-1].numpy().view(np.uint32)[lo // 32:lo // 32 + bits.size] = bits
            self.scales[-1][c] = float(s)

    def apply_phase(self):
        for c, lo, hi in self._chunks(0, self.C):
            words = self.bits[-1].numpy().view(np.uint32)[lo // 32:(hi + 31) // 32]
            q = self.ao.decompress_1bit(words, self.scales[-1][c].item(), hi - lo)
            self.m[lo:hi] = q
            self.x[lo:hi] = self.x[lo:hi] - (np.float32(LR) * q) / (np.sqrt(self.v[lo:hi]) + np.float32(EPS))


FRAC = 0.05


def _pack_mask(sel):
    pad = (-sel.size) % 32
    return np.packbits(np.concatenate([sel, np.zeros(pad, np.uint8)]), bitorder="little").view(np.uint32)


def _unpack_mask(words, length):
    return np.unpackbits(np.ascontiguousarray(words).view(np.uint8), bitorder="little")[:length].astype(bool)


class TopkOracleBackend(OracleBackend):
    """The same stand-in with the top-k compressor (Section 5.1): a message is the selection mask plus the kept
    values in index order, `per` slots per chunk."""

    topk = True

    def __init__(self, *args):
        super().__init__(*args)
        self.q = [np.zeros(self.d, np.float32) for _ in range(self.n + 1)]      # C[z] of every worker, last = server

    def topk_values_per_chunk(self):
        return self.ao.topk_count(FRAC, self.chunk)

    def worker_phase(self, grads):
        omb1 = np.float32(1.0) - np.float32(BETA1)
        for i, g in enumerate(grads):
            g = g.numpy()
            for c, lo, hi in self._chunks(0, self.C):
                z = _fma32(np.float32(BETA1), self.m[lo:hi], omb1 * g[lo:hi]) + self.err[i][lo:hi]
                q, sel = self.ao.compress_topk(z, self.ao.topk_count(FRAC, hi - lo))
                self.err[i][lo:hi] = z - q
                self.q[i][lo:hi] = q
                words = _pack_mask(sel)
                self.bits[i].numpy().view(np.uint32)[lo // 32:lo // 32 + words.size] = words

    def topk_pack_values(self, worker, cb, ce, out):
        per = self.topk_values_per_chunk()
        for c, lo, hi in self._chunks(cb, ce):
            sel = _unpack_mask(self.bits[worker].numpy().view(np.uint32)[lo // 32:(hi + 31) // 32], hi - lo)
            vals = self.q[worker][lo:hi][sel]
            out[(c - cb) * per:(c - cb) * per + vals.size] = torch.from_numpy(vals)

    def _take_over(self, c, lo, hi, q, sel):
        self.q[-1][lo:hi] = q
        words = _pack_mask(sel.astype(np.uint8))
        self.bits[-1].numpy().view(np.uint32)[lo // 32:lo // 32 + words.size] = words
        self.m[lo:hi] = q
        self.x[lo:hi] = self.x[lo:hi] - (np.float32(LR) * q) / (np.sqrt(self.v[lo:hi]) + np.float32(EPS))

    def topk_server_phase(self, mask_rows, val_rows, cb, ce):
        per, rows, w_first = self.topk_values_per_chunk(), mask_rows.shape[0], cb * self.chunk // 32
        for c, lo, hi in self._chunks(cb, ce):
            acc = np.zeros(hi - lo, np.float32)
            for j in range(rows):                                   # row order = global worker order
                sel = _unpack_mask(mask_rows[j].numpy().view(np.uint32)[lo // 32 - w_first:(hi + 31) // 32 - w_first], hi - lo)
                qj = np.zeros(hi - lo, np.float32)
                qj[sel] = val_rows[j, (c - cb) * per:(c - cb) * per + int(sel.sum())].numpy()
                acc = acc + qj
            z = acc / np.float32(rows) + self.server_err[lo:hi]
            q, sel = self.ao.compress_topk(z, self.ao.topk_count(FRAC, hi - lo))
            self.server_err[lo:hi] = z - q
            self._take_over(c, lo, hi, q, sel)

    def topk_put_server_range(self, mask_words, vals, kb, ke):
        per, w_first = self.topk_values_per_chunk(), kb * self.chunk // 32
        for c, lo, hi in self._chunks(kb, ke):
            sel = _unpack_mask(mask_words.numpy().view(np.uint32)[lo // 32 - w_first:(hi + 31) // 32 - w_first], hi - lo)
            q = np.zeros(hi - lo, np.float32)
            q[sel] = vals[(c - kb) * per:(c - kb) * per + int(sel.sum())].numpy()
            self._take_over(c, lo, hi, q, sel)

    def apply_phase(self):                                          # the kept elements were updated where their range was served or taken over
        pass


def _inputs():
    rng = np.random.default_rng(77)
    x0 = (rng.standard_normal(D) * 0.02).astype(np.float32)
    v = ((rng.standard_normal(D) * 1e-2) ** 2 + 1e-10).astype(np.float32)
    m = (rng.standard_normal(D) * 1e-3).astype(np.float32)
    grads = [[(rng.standard_normal(D) * 0.01).astype(np.float32) for _ in range(N_TOTAL)] for _ in range(4)]
    return x0, v, m, grads


def _reference():
    from oracle import apms_oracle as ao

    x0, v, m, grads = _inputs()
    o = ao.Oracle(D, N_TOTAL, BETA1, 0.999, EPS, LR, CHUNK)
    o.set_params(x0)
    o.freeze_v()
    o.v[:], o.m[:] = v, m
    for gs in grads:
        o.compressed_step(gs)
    return o


def _rank_main(rank, world, port, out):
    from paper_2008_11343_b200 import sharded

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    x0, v, m, grads = _inputs()
    n_local = N_TOTAL // world
    backend = OracleBackend(D, n_local, CHUNK, x0, v, m)
    step = sharded.ShardedStep(backend)
    for gs in grads:
        step.step([torch.from_numpy(g) for g in gs[rank * n_local:(rank + 1) * n_local]])
    ref = _reference()
    ok = bool(np.array_equal(backend.x, ref.x) and np.array_equal(backend.m, ref.m)
              and np.array_equal(backend.bits[-1].numpy().view(np.uint32), ref.server_bits)
              and np.array_equal(backend.scales[-1].numpy(), ref.server_scales))
    for i in range(n_local):
        ok = ok and bool(np.array_equal(backend.err[i], ref.worker_err(rank * n_local + i)))
    cb, ce = step.ranges[rank]
    lo, hi = cb * CHUNK, min(D, ce * CHUNK)
    ok = ok and bool(np.array_equal(backend.server_err[lo:hi], ref.server_err[lo:hi]))      # a rank owns only its range
    # the worker phase ran range by range, in the order of the serving processes, on every rank alike
    ok = ok and backend.ranges_seen == list(step.ranges) * len(grads)
    out[rank] = (ok, step.wire_bytes_per_step())
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_two_workers_each_equal_one_four_worker_run():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] and res[1][0]
    # the wire carries packed sign words and scales only: far below 4 d bytes per worker
    assert max(res[0][1], res[1][1]) < 0.1 * 4 * D * (N_TOTAL // world)


def _rank_main_topk(rank, world, port, out):
    from oracle import apms_oracle as ao
    from paper_2008_11343_b200 import sharded

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    x0, v, m, grads = _inputs()
    n_local = N_TOTAL // world
    backend = TopkOracleBackend(D, n_local, CHUNK, x0, v, m)
    step = sharded.ShardedStep(backend)
    for gs in grads:
        step.step([torch.from_numpy(g) for g in gs[rank * n_local:(rank + 1) * n_local]])
    ref = ao.Oracle(D, N_TOTAL, BETA1, 0.999, EPS, LR, CHUNK)
    ref.set_compressor(ao.TOPK); ref.set_topk_fraction(FRAC)
    ref.set_params(x0)
    ref.freeze_v()
    ref.v[:], ref.m[:] = v, m
    for gs in grads:
        ref.compressed_step(gs)
    ok = bool(np.array_equal(backend.x, ref.x) and np.array_equal(backend.m, ref.m)
              and np.array_equal(_unpack_mask(backend.bits[-1].numpy().view(np.uint32), D), ref.server_selected.astype(bool)))
    for i in range(n_local):
        ok = ok and bool(np.array_equal(backend.err[i], ref.worker_err(rank * n_local + i)))
    cb, ce = step.ranges[rank]
    lo, hi = cb * CHUNK, min(D, ce * CHUNK)
    ok = ok and bool(np.array_equal(backend.server_err[lo:hi], ref.server_err[lo:hi]))
    out[rank] = (ok, step.wire_bytes_per_step())
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_carry_the_topk_compressor():
    """ShardedStep with the top-k compressor over two gloo ranks: masks and packed kept values cross the wire, the
    result equals one four-worker run of the C oracle with the same compressor."""
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main_topk, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] and res[1][0]
    assert max(res[0][1], res[1][1]) < (0.1 + 2 * FRAC) * 4 * D * (N_TOTAL // world)


def test_chunk_and_word_ranges_tile_the_vector():
    from paper_2008_11343_b200 import sharded

    for C, world in [(7, 2), (8, 8), (10228, 8), (5, 5), (100, 3)]:
        r = sharded.chunk_ranges(C, world)
        assert r[0][0] == 0 and r[-1][1] == C and all(a[1] == b[0] for a, b in zip(r, r[1:]))
        assert max(e - b for b, e in r) - min(e - b for b, e in r) <= 1
    d, chunk = 335_141_888, 32768
    r = sharded.chunk_ranges(-(-d // chunk), 8)
    words = [sharded.word_range(b, e, chunk, d) for b, e in r]
    assert words[0][0] == 0 and words[-1][1] == -(-d // 32) and all(a[1] == b[0] for a, b in zip(words, words[1:]))


def test_chunk_for_servers_gives_one_chunk_per_server():
    from paper_2008_11343_b200 import sharded

    for d, n in [(335_141_888, 16), (109_482_240, 8), (2049, 2), (4096, 2), (1, 1)]:
        chunk = sharded.chunk_for_servers(d, n)
        assert chunk % 32 == 0 and -(-d // chunk) <= n and chunk * n >= d
        assert chunk - 32 < -(-d // n)                           # not rounded further than whole sign words need
    assert sharded.chunk_for_servers(335_141_888, 16) == 335_141_888 // 16     # the headline set: exactly d / 16
    assert -(-335_141_888 // sharded.chunk_for_servers(335_141_888, 16)) == 16
