"""The peer form of the multi-process step on the GPU.

(1) One process, two emulated ranks: two contexts of two workers each on one GPU, run phase by phase in one
    stream; the server kernels read the rows through per-row pointers into both contexts' message buffers and
    each context stores its range of the server message into the other's.  Equal, bit for bit, to one context
    with all four workers and to the oracle.
(2) Two processes sharing the one GPU: each maps the other's workspace through CUDA IPC and runs
    sharded.PeerShardedStep (host barriers over gloo; no kernel waits on another process).  This is the code
    path of a one-process-per-GPU run, with the peer's memory on the same device instead of across NVLink."""
import os
import socket
import sys

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import gpu_harness as H
from oracle import apms_oracle as ao
from paper_2008_11343_b200 import binding as B
from paper_2008_11343_b200 import sharded
from paper_2008_11343_b200 import workloads as wl
from test_gpu_parity import tiny

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("d,chunk", [(11 * 2048 + 77, 2048), (9 * 96 + 5, 96), (3 * 32768 + 23552, 32768)])
def test_rows_from_two_emulated_ranks_equal_the_whole_step(d, chunk):
    w = tiny(d, 4, chunk, cfg_id=142)
    whole = B.Context(w.d, 4, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    ranks = [B.Context(w.d, 2, w.beta1, w.beta2, w.eps, w.lr, w.chunk, library_workspace=(r == 1)) for r in range(2)]
    orc = ao.Oracle(w.d, 4, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    x0 = wl.initial_params(w)
    orc.set_params(x0); orc.freeze_v()
    for c in [whole] + ranks:
        c.set_params(x0)
        c.freeze_v()
    ranges = sharded.chunk_ranges(whole.C, 2)
    for k in range(3):
        host = wl.host_gradients(w, k)
        gs = H.upload(host)
        whole.compressed_step(gs)
        orc.compressed_step(host)
        for r in range(2):
            ranks[r].worker_phase(gs[2 * r:2 * r + 2])
        for r in range(2):
            cb, ce = ranges[r]
            w0 = cb * chunk // 32
            bits = [ranks[q].message_ptrs(i)[0] + 4 * w0 for q in range(2) for i in range(2)]
            scales = [ranks[q].message_ptrs(i)[1] + 4 * cb for q in range(2) for i in range(2)]
            ranks[r].server_phase_rows(bits, scales, cb, ce)
            ranks[r].put_server_range(*ranks[1 - r].message_ptrs(-1), cb, ce)
        for r in range(2):
            ranks[r].apply_phase()
        for r in range(2):
            for which in (B.STATE_X, B.STATE_M, B.STATE_SERVER_BITS, B.STATE_SERVER_SCALES):
                assert np.array_equal(ranks[r].get_state(which).view(np.uint32), whole.get_state(which).view(np.uint32)), (k, r, which)
            lo, hi = ranges[r][0] * chunk, min(d, ranges[r][1] * chunk)
            assert np.array_equal(ranks[r].get_state(B.STATE_SERVER_ERR)[lo:hi].view(np.uint32),
                                  whole.get_state(B.STATE_SERVER_ERR)[lo:hi].view(np.uint32))
            for i in range(2):
                assert np.array_equal(ranks[r].get_state(B.STATE_WORKER_ERR, i).view(np.uint32),
                                      whole.get_state(B.STATE_WORKER_ERR, 2 * r + i).view(np.uint32))
        assert np.array_equal(whole.get_state(B.STATE_SERVER_BITS), orc.server_bits)
        np.testing.assert_allclose(whole.get_state(B.STATE_X), orc.x, rtol=H.REL, atol=1e-12)


def test_rows_argument_errors_are_status_codes():
    w = tiny(4 * 2048, 2, 2048, cfg_id=143)
    ctx = B.Context(w.d, 2, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    ctx.set_params(wl.initial_params(w)); ctx.freeze_v()
    gs = H.upload(wl.host_gradients(w, 0))
    bits = [ctx.message_ptrs(i)[0] for i in range(2)]
    scales = [ctx.message_ptrs(i)[1] for i in range(2)]
    with pytest.raises(B.ApmsError) as e:
        ctx.server_phase_rows(bits, scales, 0, ctx.C)               # no worker phase yet
    assert e.value.status == B.ERR_BAD_STATE
    ctx.worker_phase(gs)
    with pytest.raises(B.ApmsError) as e:
        ctx.server_phase_rows([bits[0], bits[1] + 2], scales, 0, ctx.C)     # not a word address
    assert e.value.status == B.ERR_INVALID_ARG
    with pytest.raises(B.ApmsError) as e:
        ctx.server_phase_rows(bits, scales, 0, ctx.C + 1)
    assert e.value.status == B.ERR_INVALID_ARG
    with pytest.raises(B.ApmsError) as e:
        ctx.put_server_range(*ctx.message_ptrs(-1), 0, ctx.C)       # before the server phase
    assert e.value.status == B.ERR_BAD_STATE
    with pytest.raises(B.ApmsError) as e:
        ctx.ipc_export()                                            # the workspace is a torch tensor
    assert e.value.status == B.ERR_BAD_STATE
    ctx.server_phase_rows(bits, scales, 0, ctx.C)
    ctx.apply_phase()
    assert ctx.message_offsets(0)[0] % 256 == 0 and ctx.message_offsets(-1)[1] % 256 == 0


def _report(outdir, rank, result):
    import json

    with open(os.path.join(outdir, f"rank{rank}.json"), "w") as f:
        json.dump(result, f)


def _rank_main(rank, world, port, d, chunk, n_local, steps, outdir):
    import torch
    import torch.distributed as dist

    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    try:
        torch.cuda.set_device(0)
        dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
        w = tiny(d, world * n_local, chunk, cfg_id=144)
        ctx = B.Context(w.d, n_local, w.beta1, w.beta2, w.eps, w.lr, w.chunk, library_workspace=True)
        x0 = wl.initial_params(w)
        ctx.set_params(x0); ctx.freeze_v()
        step = sharded.PeerShardedStep(ctx)
        orc = ao.Oracle(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
        orc.set_params(x0); orc.freeze_v()
        for k in range(steps):
            host = wl.host_gradients(w, k)
            step.step(H.upload(host[rank * n_local:(rank + 1) * n_local]))
            orc.compressed_step(host)
        ok = bool(np.array_equal(ctx.get_state(B.STATE_SERVER_BITS), orc.server_bits))
        ok = ok and bool(np.array_equal(ctx.get_state(B.STATE_SERVER_SCALES).view(np.uint32), orc.server_scales.view(np.uint32)))
        ok = ok and bool(np.array_equal(ctx.get_state(B.STATE_X).view(np.uint32), orc.x.view(np.uint32)))
        for i in range(n_local):
            ok = ok and bool(np.array_equal(ctx.get_state(B.STATE_WORKER_ERR, i).view(np.uint32),
                                            orc.worker_err(rank * n_local + i).view(np.uint32)))
        wire = step.wire_bytes_per_step()
        step.close()
        ctx.close()
        _report(outdir, rank, [ok, wire, ""])
        dist.destroy_process_group()
    except Exception as exc:                                        # reported to the parent, which fails the test
        _report(outdir, rank, [False, 0, repr(exc)])
        raise


def test_two_processes_on_one_gpu_exchange_through_mapped_workspaces(tmp_path):
    import json

    import torch.multiprocessing as mp

    d, chunk, n_local, world = 9 * 2048 + 300, 2048, 2, 2
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    # results come back through files: nothing is forked from this process, which holds a CUDA context
    mp.spawn(_rank_main, args=(world, port, d, chunk, n_local, 3, str(tmp_path)), nprocs=world, join=True)
    res = {r: json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)}
    assert res[0][0] and res[1][0], res
    assert max(res[0][1], res[1][1]) < 0.1 * 4 * d * n_local


def _rank_main_topk(rank, world, port, d, chunk, n_local, steps, frac, outdir):
    import torch
    import torch.distributed as dist

    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    try:
        torch.cuda.set_device(0)
        dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
        w = tiny(d, world * n_local, chunk, cfg_id=145)
        ctx = B.Context(w.d, n_local, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
        ctx.set_compressor(B.COMPRESSOR_TOPK, frac)
        orc = ao.Oracle(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
        orc.set_compressor(ao.TOPK); orc.set_topk_fraction(frac)
        x0 = wl.initial_params(w)
        ctx.set_params(x0); orc.set_params(x0)
        ctx.freeze_v(); orc.freeze_v()
        step = sharded.PeerShardedStep(ctx)
        for k in range(1, steps + 1):
            host = wl.host_gradients(w, k)
            step.step(H.upload(host[rank * n_local:(rank + 1) * n_local]))
            orc.compressed_step(host)
        idx = np.arange(w.d)
        mask = (ctx.get_state(B.STATE_SERVER_BITS)[idx // 32] >> (idx % 32).astype(np.uint32)) & 1
        bad = []
        if not np.array_equal(mask.astype(np.uint8), orc.server_selected):
            bad.append("server mask")
        for name, which, ref in (("x", B.STATE_X, orc.x), ("m", B.STATE_M, orc.m)):
            if not np.array_equal(ctx.get_state(which).view(np.uint32), ref.view(np.uint32)):
                bad.append(name)
        cb, ce = step.ranges[rank]                                  # a range's server error lives where the range is served
        e0, e1 = cb * w.chunk, min(ce * w.chunk, w.d)
        if not np.array_equal(ctx.get_state(B.STATE_SERVER_ERR)[e0:e1].view(np.uint32), orc.server_err[e0:e1].view(np.uint32)):
            bad.append("server error")
        for i in range(n_local):
            if not np.array_equal(ctx.get_state(B.STATE_WORKER_ERR, i).view(np.uint32), orc.worker_err(rank * n_local + i).view(np.uint32)):
                bad.append(f"error of worker {rank * n_local + i}")
        wire = step.wire_bytes_per_step()
        step.close()
        ctx.close()
        _report(outdir, rank, [not bad, wire, ", ".join(bad)])
        dist.destroy_process_group()
    except Exception as exc:                                        # reported to the parent, which fails the test
        _report(outdir, rank, [False, 0, repr(exc)])
        raise


@pytest.mark.parametrize("d,chunk,frac", [(9 * 2048 + 300, 2048, 0.03), (5 * 4096 + 77, 4096, 0.25)])
def test_two_processes_on_one_gpu_carry_the_topk_compressor(d, chunk, frac, tmp_path):
    """The peer form with the top-k compressor: every process packs its workers' kept values straight into the
    serving process's receive rows (device buffers shared through CUDA IPC), the server ranges go back the same
    way; state equal, bit for bit, to the oracle holding all workers."""
    import json

    import torch.multiprocessing as mp

    n_local, world = 2, 2
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    mp.spawn(_rank_main_topk, args=(world, port, d, chunk, n_local, 4, frac, str(tmp_path)), nprocs=world, join=True)
    res = {r: json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)}
    assert res[0][0] and res[1][0], res
    assert max(res[0][1], res[1][1]) < (0.1 + 2 * frac) * 4 * d * n_local


@pytest.mark.parametrize("path,nproc,extra", [("peer", 2, ()), ("sharded", 1, ()), ("peer", 1, ()),
                                              ("peer", 2, ("--compressor", "topk", "--topk-fraction", "0.01"))])
def test_bench_runs_the_split_layouts(path, nproc, extra, tmp_path):
    """bench.py --path peer under a two-process launch with both processes on the one GPU (what a
    one-process-per-GPU run executes, the peer's memory on the same device), and both split paths with a single
    process: one JSON line, strong scaling, the workload's workers divided over the processes."""
    import json
    import subprocess

    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={nproc}",
           "--master-addr", "127.0.0.1", "--master-port", str(port),
           os.path.join(ROOT, "bench.py"), "--gpus", str(nproc), "--path", path, "--config", "1",
           "--steps", "3", "--warmup", "3", "--no-cpu-baseline", *extra]
    if nproc > 1:
        cmd.append("--one-gpu")
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, res.stdout
    line = json.loads(lines[0])
    assert line["scaling"] == "strong" and line["n_gpus"] == nproc and line["value"] > 0
    assert line["config"]["n_workers"] == 8 and f"{nproc} processes x {8 // nproc} workers" in line["config"]["parallelism"]
    assert line["gpu_launches"] >= 3 * 3 and "worker" in line["roofline"]["kernel_ms"]
