"""Guard bytes around every array of the workspace, in place of a memory checker.

With apms_set_guard_bytes(4096) a context lays out its workspace with at least 4 KiB that belong to no array
behind every row of every array (and before the first).  The kernels then run the edge shapes of the parity
tests - every launch shape, both compressors, the phase-wise calls, 16-bit and host gradients, the monitor -
and afterwards every guard byte must still hold its pattern: no kernel wrote outside the extent of an array.
The results are compared with the oracle as well, so the guard layout itself (other strides) is covered."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import gpu_harness as H
from oracle import apms_oracle as ao
from paper_2008_11343_b200 import binding as B
from paper_2008_11343_b200 import workloads as wl
from test_gpu_parity import EDGE, STAGED, tiny

GUARD = 4096


@pytest.fixture(autouse=True)
def guard_layout():
    B.apms_set_guard_bytes(GUARD)
    try:
        yield
    finally:
        B.apms_set_guard_bytes(0)


@pytest.mark.parametrize("team", [B.TEAM_AUTO, B.TEAM_CTA, B.TEAM_WARP, B.TEAM_STAGED],
                         ids=["auto", "cta-per-tile", "warp-per-tile", "staged"])
@pytest.mark.parametrize("d,n,chunk", EDGE + STAGED)
def test_onebit_steps_leave_the_guard_bytes_alone(d, n, chunk, team):
    w = tiny(d, n, chunk, warmup_steps=2, compressed_steps=3)
    B.apms_set_guard_bytes(0)
    plain = B.apms_workspace_bytes(d, n, chunk)
    B.apms_set_guard_bytes(GUARD)
    assert B.apms_workspace_bytes(d, n, chunk) >= plain + (3 * n + 10) * GUARD     # the guard layout is in force
    ctx, orc, _ = H.run_both(w, exact=True, team_mode=team, check_every_step=False)
    ctx.check_guards()
    ctx.error_norms()
    ctx.check_guards()


@pytest.mark.parametrize("d,n,chunk,frac", [(5 * 4096 + 1234, 3, 4096, 0.01), (3 * 1024 + 5, 4, 96, 0.1), (2 * 32768 + 23552, 4, 32768, 0.01),
                                            (70000, 16, 160, 0.05), (3 * 65536 + 7, 2, 65536, 0.001), (131072 + 5000, 2, 131072, 0.01),
                                            (2 * 32768 + 100, 3, 32768, 0.1), (1, 1, 32, 0.3)])
def test_topk_steps_leave_the_guard_bytes_alone(d, n, chunk, frac):
    import torch

    w = tiny(d, n, chunk, cfg_id=190)
    ctx, orc = H.make_pair(w)
    ctx.set_compressor(B.COMPRESSOR_TOPK, frac)
    orc.set_compressor(ao.TOPK); orc.set_topk_fraction(frac)
    gs = wl.host_gradients(w, 0)
    ctx.warmup_step(H.upload(gs)); orc.warmup_step(gs)
    ctx.freeze_v(); orc.freeze_v()
    for step in range(1, 6):
        gs = wl.host_gradients(w, step)
        if step == 4:
            ctx.compressed_step_host([torch.from_numpy(g).pin_memory() for g in gs])
        else:
            ctx.compressed_step(H.upload(gs))
        orc.compressed_step(gs)
    assert np.array_equal(ctx.get_state(B.STATE_X).view(np.uint32), orc.x.view(np.uint32))
    ctx.error_norms()
    ctx.check_guards()
    # one more step through the phase-wise calls: messages packed, unpacked, served in two ranges
    from test_gpu_parity import _topk_rows

    gs = wl.host_gradients(w, 6)
    ctx.worker_phase(H.upload(gs)); orc.compressed_step(gs)
    mid = ctx.C // 2
    for cb, ce in ((0, mid), (mid, ctx.C)):
        if cb == ce:
            continue
        masks, vals = _topk_rows([ctx], cb, ce)
        ctx.topk_server_phase(masks, vals, cb, ce)
    ctx.apply_phase()
    assert np.array_equal(ctx.get_state(B.STATE_X).view(np.uint32), orc.x.view(np.uint32))
    ctx.check_guards()


@pytest.mark.parametrize("d,n,chunk,cuts", [(9 * 2048 + 300, 4, 2048, (0, 3, 10)), (7 * 96 + 5, 5, 96, (0, 4, 8)), (3 * 70016, 2, 70016, (0, 2, 3)),
                                            (5 * 2080 + 100, 3, 2080, (0, 2, 6)), (23 * 512 + 9, 2, 512, (0, 5, 6, 24))])
def test_phase_wise_steps_variants_and_16_bit_gradients_leave_the_guard_bytes_alone(d, n, chunk, cuts):
    import torch

    w = tiny(d, n, chunk, cfg_id=191)
    for variant in (B.VARIANT_MOMENTUM, B.VARIANT_GRADIENT):
        ctx = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
        ctx.set_variant(variant)
        ctx.set_params(wl.initial_params(w))
        ctx.warmup_step([torch.from_numpy(g).to(torch.bfloat16).cuda() for g in wl.host_gradients(w, 0)])
        ctx.freeze_v()
        for step in range(1, 4):
            gs = H.upload(wl.host_gradients(w, step))
            for cb, ce in zip(cuts, cuts[1:]):
                ctx.worker_phase_range(gs, cb, ce)
            bits = [ctx.message_ptrs(i)[0] for i in range(n)]
            scales = [ctx.message_ptrs(i)[1] for i in range(n)]
            for cb, ce in zip(cuts, cuts[1:]):
                w0 = cb * chunk // 32
                ctx.server_phase_rows([p + 4 * w0 for p in bits], [p + 4 * cb for p in scales], cb, ce)
            ctx.apply_phase()
            ctx.compressed_step([torch.from_numpy(g).to(torch.float16).cuda() for g in wl.host_gradients(w, 10 + step)])
        ctx.uncompressed_step(H.upload(wl.host_gradients(w, 20)))
        ctx.check_guards()


def test_a_changed_guard_byte_is_found_and_named():
    """The detector itself: one guard byte changed from the host side (through the torch view of the workspace)
    is reported with its offset and the array it follows."""
    w = tiny(3 * 1024 + 5, 2, 1024, cfg_id=192)
    ctx = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    ctx.set_params(wl.initial_params(w))
    ctx.freeze_v()
    ctx.check_guards()
    bits_ptr, _ = ctx.message_ptrs(1)                                    # worker 1's sign words; W words are its own
    off = bits_ptr - ctx.workspace.data_ptr() + 4 * ctx.W + 17          # a byte behind them
    assert int(ctx.workspace[off]) == 0xA5
    ctx.workspace[off] = 0
    with pytest.raises(B.ApmsError) as e:
        ctx.check_guards()
    assert e.value.status == B.ERR_BOUNDS and e.value.bad_offset == off and "B_i" in str(e.value)
    ctx.workspace[off] = 0xA5
    ctx.check_guards()
    B.apms_set_guard_bytes(0)
    plain = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    plain.set_params(wl.initial_params(w))
    with pytest.raises(B.ApmsError) as e:
        plain.check_guards()                                            # the ordinary layout has no guard bytes
    assert e.value.status == B.ERR_BAD_STATE
    with pytest.raises(B.ApmsError):
        B.apms_set_guard_bytes(100)


def test_checked_accessors_refuse_a_store_into_guard_bytes():
    """Only in the checked build of the library (the same tests are run against it by test_gpu_checked_build.py):
    a checked store aimed at the guard bytes behind x is skipped and reported, the guard bytes stay untouched,
    and the context goes on working."""
    if not B.apms_build_is_checked():
        w = tiny(100, 2, 32, cfg_id=193)
        ctx = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
        ctx.set_params(wl.initial_params(w))
        with pytest.raises(B.ApmsError) as e:
            B.apms_selftest_bounds(ctx._h)                       # the ordinary build has no checked accessors
        assert e.value.status == B.ERR_BAD_STATE
        return
    w = tiny(3 * 1024 + 5, 2, 1024, cfg_id=193)
    ctx, orc = H.make_pair(w)
    B.apms_selftest_bounds(ctx._h)
    gs = wl.host_gradients(w, 0)
    ctx.warmup_step(H.upload(gs)); orc.warmup_step(gs)
    ctx.freeze_v(); orc.freeze_v()
    for step in range(1, 4):
        gs = wl.host_gradients(w, step)
        ctx.compressed_step(H.upload(gs)); orc.compressed_step(gs)
    H.compare_state(ctx, orc, w, exact=True)
    ctx.check_guards()
