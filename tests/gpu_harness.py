"""Shared helpers of the GPU parity tests: run the CUDA library and the CPU oracle on the
same seeded inputs and compare their state element by element."""
from __future__ import annotations

import numpy as np

from oracle import apms_oracle as ao
from paper_2008_11343_b200 import binding as B
from paper_2008_11343_b200 import workloads as wl

REL = 1e-5          # tolerance for scales, errors and parameters (floating-point outputs)
TIE = 1e-7          # a sign may differ only where |z| < TIE * scale


def upload(grads):
    import torch

    return [torch.from_numpy(np.ascontiguousarray(g)).cuda() for g in grads]


def make_pair(w: wl.Workload, x0=None, team_mode=None):
    """A CUDA context and an oracle with the same shape, hyper-parameters and x0."""
    x0 = wl.initial_params(w) if x0 is None else x0
    ctx = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    if team_mode is not None:
        ctx.set_team_mode(team_mode)
    ctx.set_params(x0)
    orc = ao.Oracle(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    orc.set_threads(orc.max_threads())
    orc.set_params(x0)
    return ctx, orc


def chunk_of(w_or_chunk, d):
    chunk = w_or_chunk if isinstance(w_or_chunk, int) else w_or_chunk.chunk
    return np.arange(d) // chunk


def compare_bits(gpu_bits, ref_bits, z_ref_abs=None, scale_per_elem=None, what="bits"):
    """Sign words must be equal; a differing bit is tolerated only at a tie (|z| < TIE*scale).
    Returns the element indices whose bits differ (empty when bit-exact)."""
    diff = np.nonzero(gpu_bits != ref_bits)[0]
    if diff.size == 0:
        return np.zeros(0, dtype=np.int64)
    elems = []
    for wi in diff:
        x = int(gpu_bits[wi]) ^ int(ref_bits[wi])
        elems += [32 * int(wi) + b for b in range(32) if (x >> b) & 1]
    elems = np.asarray(elems, dtype=np.int64)
    assert z_ref_abs is not None, f"{what}: {elems.size} sign bits differ (no tie information given)"
    bad = z_ref_abs[elems] >= TIE * scale_per_elem[elems]
    assert not bad.any(), f"{what}: {int(bad.sum())} sign bits differ away from ties, first at {elems[bad][:5]}"
    return elems


def compare_state(ctx, orc, w, phase_compressed=True, exact=False, tainted=None):
    """Element-by-element comparison of every state array.  With exact=True everything must be
    bit-identical; otherwise bits exact (ties aside) and values within REL as below."""
    d, n, C = w.d, w.n, (w.d + w.chunk - 1) // w.chunk
    cidx = chunk_of(w, d)
    report = {}

    def close(name, got, ref, atol_vec):
        if exact:
            assert np.array_equal(got.view(np.uint32), ref.view(np.uint32)), \
                f"{name}: {int((got.view(np.uint32) != ref.view(np.uint32)).sum())} elements not bit-identical"
            report[name] = 0.0
            return
        err = np.abs(got.astype(np.float64) - ref.astype(np.float64))
        if tainted is not None and tainted.size and got.size == d:
            err[tainted] = 0.0
        worst = float((err / np.maximum(atol_vec, 1e-300)).max()) if err.size else 0.0
        assert worst <= 1.0, f"{name}: error {worst:.3g} x tolerance"
        report[name] = float((got != ref).mean())

    x, v = ctx.get_state(B.STATE_X), ctx.get_state(B.STATE_V)
    close("v", v, orc.v, REL * np.abs(orc.v) + 1e-38)
    if not phase_compressed:
        m = ctx.get_state(B.STATE_M)
        close("m", m, orc.m, REL * np.abs(orc.m) + 1e-30)
        close("x", x, orc.x, REL * np.abs(orc.x) + 1e-30)
        return report

    Sbar = ctx.get_state(B.STATE_SERVER_SCALES)
    close("server_scales", Sbar, orc.server_scales, REL * np.abs(orc.server_scales))
    S_elem = orc.server_scales[cidx]
    ebar_ref = orc.server_err
    zbar_abs = np.abs(orc.m.astype(np.float64) + ebar_ref)          # |zbar| = |C[zbar] + dbar_new|
    t2 = compare_bits(ctx.get_state(B.STATE_SERVER_BITS), orc.server_bits, zbar_abs, S_elem, "server bits")
    close("server_err", ctx.get_state(B.STATE_SERVER_ERR), ebar_ref,
          REL * np.maximum(np.abs(ebar_ref), S_elem))
    close("m", ctx.get_state(B.STATE_M), orc.m, REL * np.abs(orc.m))
    # one step moves x by lr*S/(sqrt(v)+eps); allow REL of that on top of REL of |x|
    step = np.float64(w.lr) * S_elem / (np.sqrt(orc.v.astype(np.float64)) + w.eps)
    close("x", x, orc.x, REL * (np.abs(orc.x) + step))
    for i in range(n):
        s_ref = orc.worker_scales(i)
        close(f"worker_scales[{i}]", ctx.get_state(B.STATE_WORKER_SCALES, i), s_ref, REL * np.abs(s_ref))
        s_elem = s_ref[cidx]
        e_ref = orc.worker_err(i)
        sent = np.where(((orc.worker_bits(i)[np.arange(d) // 32] >> (np.arange(d) % 32).astype(np.uint32)) & 1) == 1,
                        s_elem, -s_elem).astype(np.float64)
        z_abs = np.abs(sent + e_ref)
        compare_bits(ctx.get_state(B.STATE_WORKER_BITS, i), orc.worker_bits(i), z_abs, s_elem, f"worker {i} bits")
        close(f"worker_err[{i}]", ctx.get_state(B.STATE_WORKER_ERR, i), e_ref,
              REL * np.maximum(np.abs(e_ref), s_elem))
    report["server_tie_elems"] = int(t2.size)
    return report


def teacher_force(ctx, orc, w):
    """Overwrite the CUDA context's state with the oracle's (before a step)."""
    ctx.set_state(B.STATE_X, orc.x)
    ctx.set_state(B.STATE_V, orc.v)
    ctx.set_state(B.STATE_M, orc.m)
    ctx.set_state(B.STATE_SERVER_ERR, orc.server_err)
    for i in range(w.n):
        ctx.set_state(B.STATE_WORKER_ERR, orc.worker_err(i), worker=i)


def run_both(w: wl.Workload, warmup=None, compressed=None, check_every_step=True, exact=False,
             grads_fn=None, team_mode=None, upload_fn=None):
    """Free-running: both sides step from the same x0 on the same gradients."""
    warmup = w.warmup_steps if warmup is None else warmup
    compressed = w.compressed_steps if compressed is None else compressed
    grads_fn = grads_fn or (lambda step: wl.host_gradients(w, step))
    upload = upload_fn or globals()["upload"]
    ctx, orc = make_pair(w, team_mode=team_mode)
    reports = []
    step = 0
    for _ in range(warmup):
        gs = grads_fn(step)
        ctx.warmup_step(upload(gs))
        orc.warmup_step(gs)
        step += 1
        if check_every_step:
            reports.append(compare_state(ctx, orc, w, phase_compressed=False, exact=exact))
    ctx.freeze_v()
    orc.freeze_v()
    for k in range(compressed):
        gs = grads_fn(step)
        ctx.compressed_step(upload(gs))
        orc.compressed_step(gs)
        step += 1
        if check_every_step or k == compressed - 1:
            reports.append(compare_state(ctx, orc, w, exact=exact))
    return ctx, orc, reports
