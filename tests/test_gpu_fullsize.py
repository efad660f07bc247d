"""Parity at the benchmark's full size, in the launch configuration the benchmark times:
BERT-Large-shaped parameter set, n = 16 workers, chunk = 32768, device-resident gradients.

The oracle cannot run 335M x 16 elements in a test, but chunks are independent problems
(Supplement A: the algorithm equals a parameter-server step per chunk), so a sample of chunks -
the first, the ragged last one and random ones - is run by the oracle as a small problem of its own,
on the same gradients, and compared with the same chunks of the device state step by step."""
import gc

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import gpu_harness as H
from oracle import apms_oracle as ao
from paper_2008_11343_b200 import binding as B
from paper_2008_11343_b200 import workloads as wl


def _slices(w, chunks):
    return [(c * w.chunk, min(w.d, (c + 1) * w.chunk) - c * w.chunk) for c in chunks]


def _gather(ctx, which, sl, worker=0):
    return np.concatenate([ctx.get_state_slice(which, lo, cnt, worker=worker) for lo, cnt in sl])


def _gather_words(ctx, which, sl, worker=0):
    return np.concatenate([ctx.get_state_slice(which, lo // 32, (cnt + 31) // 32, worker=worker) for lo, cnt in sl])


# (configuration, sampled chunks, worker-count override, chunk override, compressed steps)
FULL = [(3, 10, None, None, 12), (2, 6, None, None, 12),
        (3, 6, 32, 1024, 4), (3, 5, 32, 65536, 4), (3, 3, 16, 20946368, 3)]


@pytest.mark.parametrize("cfg,samples,n,chunk,steps", FULL,
                         ids=["bert-large-n16-32768", "bert-base-n16-16384", "sweep-n32-1024", "sweep-n32-65536",
                              "one-chunk-per-server-n16"])
def test_sampled_chunks_free_running_at_full_size(cfg, samples, n, chunk, steps):
    """The oracle's copy of the sampled chunks is seeded ONCE (parameters before the first step) and then runs
    freely beside the device for the warmup steps, the phase switch and `steps` compression-phase steps: no
    state is copied from the device afterwards, so a drift on either side would show.  Sign words must be equal
    at every step; scales, errors, momentum and model within the tolerance; at most 2 scales may round
    differently over the whole run."""
    import torch

    w = wl.config(cfg)
    if n is not None:
        w = w.with_(n=n)
    if chunk is not None:
        w = w.with_(chunk=chunk)
    gc.collect()
    torch.cuda.empty_cache()                                 # memory cached for earlier tests counts as free
    free, _ = torch.cuda.mem_get_info()
    need = B.apms_workspace_bytes(w.d, w.n, w.chunk) + 4 * w.d * w.n + (2 << 30)
    if free < need:
        pytest.skip(f"needs {need / 2**30:.0f} GiB of device memory, {free / 2**30:.0f} GiB free")
    chunks = list(wl.sample_chunks(w, samples))
    assert chunks[-1] == w.n_chunks - 1                      # the ragged chunk is part of the sample
    sl = _slices(w, chunks)
    # the sampled chunks keep their lengths in the oracle's small problem only if all but the last are whole
    assert all(cnt == w.chunk for _, cnt in sl[:-1])
    dsub = sum(cnt for _, cnt in sl)

    ctx = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    x0 = torch.empty(w.d, dtype=torch.float32, device="cuda").normal_(0.0, w.x0_std)
    ctx.set_params(x0)
    del x0
    grads = [torch.empty(w.d, dtype=torch.float32, device="cuda") for _ in range(w.n)]

    def draw(step):
        for i in range(w.n):
            wl.device_gradient(w, step, i, grads[i])
        return [np.concatenate([g[lo:lo + cnt].cpu().numpy() for lo, cnt in sl]) for g in grads]

    orc = ao.Oracle(dsub, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    orc.set_threads(orc.max_threads())
    orc.set_params(_gather(ctx, B.STATE_X, sl))              # the only state the oracle ever takes from the device

    # warmup steps: element-wise, so the sampled elements can simply be replayed
    for step in range(2):
        gsub = draw(step)
        ctx.warmup_step(grads)
        orc.warmup_step(gsub)
    for which, ref in ((B.STATE_X, orc.x), (B.STATE_M, orc.m), (B.STATE_V, orc.v)):
        got = _gather(ctx, which, sl)
        assert np.array_equal(got.view(np.uint32), ref.view(np.uint32)), f"warmup state {which}"
    ctx.freeze_v()
    orc.freeze_v()

    mismatched_scales = 0
    idx = np.asarray(chunks)
    cidx = H.chunk_of(w.chunk, dsub)
    for step in range(2, 2 + steps):
        gsub = draw(step)
        ctx.compressed_step(grads)
        orc.compressed_step(gsub)
        # sign words: bit-exact
        assert np.array_equal(_gather_words(ctx, B.STATE_SERVER_BITS, sl), orc.server_bits), f"step {step}: server sign words differ"
        for i in range(w.n):
            assert np.array_equal(_gather_words(ctx, B.STATE_WORKER_BITS, sl, worker=i), orc.worker_bits(i)), \
                f"step {step}: worker {i} sign words differ"
        # scales
        Sg = np.array([ctx.get_state_slice(B.STATE_SERVER_SCALES, int(c), 1)[0] for c in idx])
        np.testing.assert_allclose(Sg, orc.server_scales, rtol=H.REL)
        mismatched_scales += int((Sg != orc.server_scales).sum())
        last = step == 1 + steps
        for i in range(w.n):
            sg = np.array([ctx.get_state_slice(B.STATE_WORKER_SCALES, int(c), 1, worker=i)[0] for c in idx])
            np.testing.assert_allclose(sg, orc.worker_scales(i), rtol=H.REL)
            mismatched_scales += int((sg != orc.worker_scales(i)).sum())
            if last or i == step % w.n:                      # every worker's errors at the end, one worker's per step
                e_ref = orc.worker_err(i)
                tol = H.REL * np.maximum(np.abs(e_ref), orc.worker_scales(i)[cidx])
                assert (np.abs(_gather(ctx, B.STATE_WORKER_ERR, sl, worker=i) - e_ref) <= tol).all()
        e_ref = orc.server_err
        tol = H.REL * np.maximum(np.abs(e_ref), orc.server_scales[cidx])
        assert (np.abs(_gather(ctx, B.STATE_SERVER_ERR, sl) - e_ref) <= tol).all()
        np.testing.assert_allclose(_gather(ctx, B.STATE_M, sl), orc.m, rtol=H.REL)
        stepsize = w.lr * orc.server_scales[cidx] / (np.sqrt(orc.v.astype(np.float64)) + w.eps)
        assert (np.abs(_gather(ctx, B.STATE_X, sl) - orc.x) <= H.REL * (np.abs(orc.x) + stepsize)).all()
    # the binary64 sums make a differently rounded scale a rare event, not the rule
    assert mismatched_scales <= 2

    # properties that hold at any size, on the whole vector: payload and padding
    W = (w.d + 31) // 32
    last = ctx.get_state_slice(B.STATE_SERVER_BITS, W - 1, 1)[0]
    if w.d % 32:
        assert int(last) >> (w.d % 32) == 0
    assert np.isfinite(ctx.get_state_slice(B.STATE_SERVER_SCALES, 0, w.n_chunks)).all()


@pytest.mark.parametrize("frac", [0.01, 0.05])
def test_topk_sampled_chunks_at_full_size(frac):
    """The top-k compressor at the benchmark's size and launch shape: sampled chunks replayed by the oracle from
    the device state, over steps that take the kernels' first-step route and then their predicted-threshold
    routes; masks, errors, momentum and model bit-identical."""
    import torch

    w = wl.config(3)
    gc.collect()
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    need = B.apms_workspace_bytes(w.d, w.n, w.chunk) + 4 * w.d * w.n + (2 << 30)
    if free < need:
        pytest.skip(f"needs {need / 2**30:.0f} GiB of device memory, {free / 2**30:.0f} GiB free")
    chunks = list(wl.sample_chunks(w, 6, seed_key=7))
    assert chunks[-1] == w.n_chunks - 1
    sl = _slices(w, chunks)
    dsub = sum(cnt for _, cnt in sl)
    # the sampled chunks keep their lengths in the oracle's small problem only if all but the last are whole
    assert all(cnt == w.chunk for _, cnt in sl[:-1])

    ctx = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    ctx.set_compressor(B.COMPRESSOR_TOPK, frac)
    x0 = torch.empty(w.d, dtype=torch.float32, device="cuda").normal_(0.0, w.x0_std)
    ctx.set_params(x0)
    grads = [torch.empty(w.d, dtype=torch.float32, device="cuda") for _ in range(w.n)]

    def draw(step):
        for i in range(w.n):
            wl.device_gradient(w, step, i, grads[i])
        return [np.concatenate([g[lo:lo + cnt].cpu().numpy() for lo, cnt in sl]) for g in grads]

    orc = ao.Oracle(dsub, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    orc.set_threads(orc.max_threads())
    orc.set_compressor(ao.TOPK); orc.set_topk_fraction(frac)
    orc.set_params(_gather(ctx, B.STATE_X, sl))
    gsub = draw(0)
    ctx.warmup_step(grads); orc.warmup_step(gsub)
    ctx.freeze_v(); orc.freeze_v()
    idx = np.arange(dsub)
    for step in range(1, 5):
        orc.x[:] = _gather(ctx, B.STATE_X, sl)
        orc.m[:] = _gather(ctx, B.STATE_M, sl)
        orc.server_err[:] = _gather(ctx, B.STATE_SERVER_ERR, sl)
        for i in range(w.n):
            orc.worker_err(i)[:] = _gather(ctx, B.STATE_WORKER_ERR, sl, worker=i)
        gsub = draw(step)
        ctx.compressed_step(grads)
        orc.compressed_step(gsub)
        for which, ref in ((B.STATE_X, orc.x), (B.STATE_M, orc.m), (B.STATE_SERVER_ERR, orc.server_err)):
            assert np.array_equal(_gather(ctx, which, sl).view(np.uint32), ref.view(np.uint32)), (step, which)
        words = _gather_words(ctx, B.STATE_SERVER_BITS, sl)
        assert np.array_equal(((words[idx // 32] >> (idx % 32).astype(np.uint32)) & 1).astype(np.uint8), orc.server_selected), step
        for i in range(w.n):
            assert np.array_equal(_gather(ctx, B.STATE_WORKER_ERR, sl, worker=i).view(np.uint32),
                                  orc.worker_err(i).view(np.uint32)), (step, i)
            words = _gather_words(ctx, B.STATE_WORKER_BITS, sl, worker=i)
            assert np.array_equal(((words[idx // 32] >> (idx % 32).astype(np.uint32)) & 1).astype(np.uint8),
                                  orc.worker_selected(i)), (step, i, "mask")


@pytest.mark.parametrize("chunk,topk", [(None, None), ("d/16", None), (1024, None), (128, None), (None, 0.01), (None, 0.03)],
                         ids=["chunk-32768", "one-chunk-per-server", "chunk-1024", "chunk-128", "topk-1%", "topk-3%"])
def test_two_runs_at_full_size_leave_the_same_state(chunk, topk):
    """Thousands of CTAs of the step's kernels overlap in time at full size and in changing order; the state they
    leave must not depend on it: two runs from the same inputs, the whole server message and the whole model
    compared bit for bit after every compressed step (checksums on the host)."""
    import zlib

    import torch

    w = wl.config(3)
    if chunk is not None:
        w = w.with_(chunk=w.d // 16 if chunk == "d/16" else chunk)
    gc.collect(); torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < B.apms_workspace_bytes(w.d, w.n, w.chunk) + (w.n + 2) * 4 * w.d + (4 << 30):
        pytest.skip("not enough device memory for the full-size workload")
    grads = [torch.empty(w.d, dtype=torch.float32, device="cuda") for _ in range(w.n)]
    x0 = torch.from_numpy(wl.initial_params(w)).cuda()
    crc = lambda a: zlib.crc32(np.ascontiguousarray(a).tobytes())
    runs = []
    for rep in range(2):
        ctx = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
        if topk is not None:
            ctx.set_compressor(B.COMPRESSOR_TOPK, topk)
        ctx.set_params(x0)
        rec = []
        for step in range(5 if topk is None else 8):       # top-k: the predicted-threshold routes need a few steps of history
            for i in range(w.n):
                wl.device_gradient(w, step, i, grads[i])
            if step < 2:
                ctx.warmup_step(grads)
                if step == 1:
                    ctx.freeze_v()
                continue
            ctx.compressed_step(grads)
            rec.append((crc(ctx.get_state(B.STATE_SERVER_SCALES)), crc(ctx.get_state(B.STATE_SERVER_BITS)),
                        crc(ctx.get_state(B.STATE_SERVER_ERR)), crc(ctx.get_state(B.STATE_X)),
                        crc(ctx.get_state(B.STATE_WORKER_SCALES, w.n - 1)), crc(ctx.get_state(B.STATE_WORKER_BITS, w.n - 1))))
        runs.append(rec)
        ctx.close()
        del ctx
        gc.collect(); torch.cuda.empty_cache()
    assert runs[0] == runs[1]
