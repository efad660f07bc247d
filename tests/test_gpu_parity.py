"""CUDA library vs CPU oracle, element by element, through the C ABI (needs a B200)."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import gpu_harness as H
from oracle import apms_oracle as ao
from paper_2008_11343_b200 import binding as B
from paper_2008_11343_b200 import workloads as wl


def tiny(d, n, chunk, cfg_id=100, **kw):
    return wl.Workload(f"tiny-{d}-{n}-{chunk}", cfg_id, n=n, chunk=chunk, tensor_sizes=(d,), dist="gauss",
                       scale_lo=1e-3, scale_hi=1e-1, **kw)


# ------------------------------------------------------------------ edge sizes, bit-identical

EDGE = [(1, 1, 32), (31, 2, 32), (32, 2, 32), (33, 3, 32), (127, 4, 128), (128, 4, 128), (129, 4, 128),
        (4095, 2, 4096), (4096, 2, 4096), (4097, 2, 4096), (1000, 5, 96), (12345, 3, 1024),
        (5 * 8192 + 77, 2, 8192), (3 * 65536 + 1, 2, 65536), (70000, 16, 160), (2050, 64, 2048),
        (300000, 2, 131104), (4 * 70016, 4, 70016), (5000, 3, 1024), (40000, 2, 4096),
        (3000, 32, 96), (9000, 12, 1024), (7 * 1056 + 31, 8, 1056)]


# shapes for the staged forms (chunk a multiple of 2048): one slab, many slabs, ragged last slab and chunk,
# split chunks, n not a power of two (IEEE division instead of the exact multiplication by 1/n), n = 64
STAGED = [(2048, 1, 2048), (10 * 2048 + 1, 5, 2048), (6144 * 3 + 33, 7, 6144), (3 * 131072 + 4099, 3, 131072),
          (8 * 32768 + 23552, 16, 32768), (2 * 4096 + 2047, 64, 4096), (65536 + 2049, 2, 65536),
          (3 * 512 + 100, 3, 512), (7 * 1536 + 511, 2, 1536), (9 * 4096 + 513, 4, 1024),
          (5 * 4096 + 100, 32, 4096), (3 * 2048 + 7, 12, 2048), (2 * 32768 + 1000, 32, 32768), (6 * 8192 + 5, 8, 8192),
          (65536 + 4097, 32, 65536), (11 * 1024 + 9, 32, 1024),
          # chunks that are not multiples of a slab, a tile or 512: sign-word rows off the 16-byte boundary, a chunk
          # boundary inside a warp's 512 elements; short chunks packed several to a slab, any worker count
          (5 * 2080 + 100, 3, 2080), (3 * 4128 + 33, 16, 4128), (2 * 20960 + 7000, 4, 20960), (3 * 66592 + 5, 2, 66592),
          (7 * 2048 * 3 + 2016 * 5, 5, 2016 * 3), (3 * 2048 + 700, 5, 256), (9 * 2048 + 1500, 7, 512), (40 * 2048 + 130, 16, 128),
          (6 * 1056 + 1000, 4, 1056), (5 * 544 + 17, 2, 544)]


@pytest.mark.parametrize("team", [B.TEAM_CTA, B.TEAM_WARP, B.TEAM_AUTO, B.TEAM_STAGED],
                         ids=["cta-per-tile", "warp-per-tile", "auto", "staged"])
@pytest.mark.parametrize("d,n,chunk", EDGE + STAGED)
def test_free_running_edge_sizes_bit_identical(d, n, chunk, team):
    """Ragged tails, d below / at / above a word, a vector and a chunk; several tiles.  On these
    sizes every scale is expected to round identically on both sides, so the whole state must be
    bit-identical (the binary64 sums differ only in the order of additions)."""
    w = tiny(d, n, chunk, warmup_steps=3, compressed_steps=4)
    H.run_both(w, exact=True, team_mode=team)


@pytest.mark.parametrize("n", [32, 16, 12, 8])
def test_many_short_chunks_per_cta_bit_identical(n):
    """Enough chunks that every CTA of the fused server kernel walks several of them (1200 chunks of 4096 on
    148 SMs), at the worker counts the benchmark's sweep uses (each its own unrolled instantiation) and at one
    count that takes the generic loop: the whole state bit-identical after free-running steps."""
    w = tiny(1200 * 4096 + 777, n, 4096, cfg_id=111, warmup_steps=1, compressed_steps=3)
    H.run_both(w, exact=True, check_every_step=False)


def test_teacher_forced_steps_bits_exact():
    """The oracle's state is uploaded before every step; after the step the packed sign words
    must equal the oracle's exactly and every value must be bit-identical."""
    w = tiny(6 * 1024 + 333, 4, 1024, cfg_id=101, lr=1e-3)
    ctx, orc = H.make_pair(w)
    for step in range(2):
        gs = wl.host_gradients(w, step)
        ctx.warmup_step(H.upload(gs))
        orc.warmup_step(gs)
    ctx.freeze_v()
    orc.freeze_v()
    rng = np.random.default_rng(3)
    for step in range(2, 7):
        # disturb the oracle's state so that each step starts from a state the CUDA side never produced
        orc.server_err[:] += (rng.standard_normal(w.d) * 1e-4).astype(np.float32)
        for i in range(w.n):
            orc.worker_err(i)[:] += (rng.standard_normal(w.d) * 1e-4).astype(np.float32)
        orc.m[:] = (rng.standard_normal(w.d) * 1e-3).astype(np.float32)
        H.teacher_force(ctx, orc, w)
        gs = wl.host_gradients(w, step)
        ctx.compressed_step(H.upload(gs))
        orc.compressed_step(gs)
        H.compare_state(ctx, orc, w, exact=True)


# ------------------------------------------------------------------ 16-bit gradients

@pytest.mark.parametrize("team", [B.TEAM_AUTO, B.TEAM_WARP], ids=["auto", "warp-per-tile"])
@pytest.mark.parametrize("kind", ["bfloat16", "float16"])
@pytest.mark.parametrize("d,n,chunk", [(5 * 4096 + 1234, 3, 4096), (3 * 1024 + 5, 2, 96), (70000, 16, 160),
                                       (2 * 32768 + 23552, 4, 32768), (1 * 512 + 3, 2, 512)])
def test_sixteen_bit_gradients_bit_identical(d, n, chunk, kind, team):
    """Gradients given as bfloat16 / binary16 arrays: the library widens them exactly, so the state must be
    bit-identical to the oracle's run on the same values held in binary32 (warmup and compressed steps)."""
    import torch

    dt = getattr(torch, kind)
    w = tiny(d, n, chunk, cfg_id=120, warmup_steps=2, compressed_steps=3)

    def grads(step):          # the values the 16-bit arrays hold, as binary32, for the oracle
        return [torch.from_numpy(g).to(dt).to(torch.float32).numpy() for g in wl.host_gradients(w, step)]

    def upload16(gs):
        return [torch.from_numpy(g).to(dt).cuda() for g in gs]

    H.run_both(w, exact=True, grads_fn=grads, upload_fn=upload16, team_mode=team)


def test_sixteen_bit_host_gradients_and_alignment():
    import torch

    w = tiny(3 * 2048 + 77, 2, 2048, cfg_id=121)
    ref = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    ctx = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    for c in (ref, ctx):
        c.set_params(wl.initial_params(w))
        c.freeze_v()
    for step in range(3):
        g16 = [torch.from_numpy(g).to(torch.bfloat16) for g in wl.host_gradients(w, step)]
        ref.compressed_step([g.cuda() for g in g16])
        ctx.compressed_step_host([g.pin_memory() for g in g16])
    for k in (B.STATE_X, B.STATE_SERVER_BITS, B.STATE_SERVER_SCALES, B.STATE_SERVER_ERR):
        assert np.array_equal(ref.get_state(k).view(np.uint32), ctx.get_state(k).view(np.uint32))
    g = torch.zeros(w.d + 8, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.ApmsError) as e:                       # 2-byte offset: not 8-byte aligned
        B.apms_compressed_step_typed(ctx._h, [g.data_ptr() + 2, g.data_ptr()], B.GRAD_BF16)
    assert e.value.status == B.ERR_INVALID_ARG
    with pytest.raises(B.ApmsError) as e:
        B.apms_compressed_step_typed(ctx._h, [g.data_ptr(), g.data_ptr()], 7)
    assert e.value.status == B.ERR_INVALID_ARG


# ------------------------------------------------------------------ the other reading of the scale

@pytest.mark.parametrize("team", [B.TEAM_AUTO, B.TEAM_CTA, B.TEAM_WARP], ids=["auto", "cta-per-tile", "warp-per-tile"])
@pytest.mark.parametrize("d,n,chunk", [(5 * 4096 + 1234, 3, 4096), (3 * 1024 + 5, 4, 96), (3 * 70016, 2, 70016),
                                       (2 * 32768 + 23552, 16, 32768), (9 * 512 + 3, 2, 512)])
def test_mean_absolute_scale_matches_the_oracle_switch(d, n, chunk, team):
    """scale = mean |z| on both sides (the oracle's switch, the library's apms_set_scale_kind): bit-identical state."""
    w = tiny(d, n, chunk, cfg_id=150, warmup_steps=1, compressed_steps=4)
    ctx, orc = H.make_pair(w, team_mode=team)
    ctx.set_scale_kind(B.SCALE_L1_MEAN)
    orc.set_scale_kind(ao.SCALE_L1_MEAN)
    gs = wl.host_gradients(w, 0)
    ctx.warmup_step(H.upload(gs)); orc.warmup_step(gs)
    ctx.freeze_v(); orc.freeze_v()
    for step in range(1, 5):
        gs = wl.host_gradients(w, step)
        ctx.compressed_step(H.upload(gs)); orc.compressed_step(gs)
        H.compare_state(ctx, orc, w, exact=True)
    z = np.abs(orc.m[:min(chunk, d)].astype(np.float64) + orc.server_err[:min(chunk, d)])    # |zbar| of chunk 0
    assert abs(float(ctx.get_state(B.STATE_SERVER_SCALES)[0]) - z.mean()) <= 1e-6 * z.mean()


# ------------------------------------------------------------------ the comparison variants of Section 5.3

@pytest.mark.parametrize("team", [B.TEAM_AUTO, B.TEAM_CTA, B.TEAM_WARP], ids=["auto", "cta-per-tile", "warp-per-tile"])
@pytest.mark.parametrize("d,n,chunk", [(5 * 4096 + 1234, 3, 4096), (3 * 1024 + 5, 4, 96), (3 * 70016, 2, 70016),
                                       (2 * 32768 + 23552, 16, 32768), (9 * 512 + 3, 2, 512), (1, 1, 32)])
def test_gradient_variant_bit_identical(d, n, chunk, team):
    """Error-compensated compression of the gradient instead of the momentum: every state array bit-identical
    to the oracle's variant, step by step (the momentum stays binary32 and is updated from the received gradient)."""
    w = tiny(d, n, chunk, cfg_id=160, warmup_steps=2, compressed_steps=4)
    ctx, orc = H.make_pair(w, team_mode=team)
    ctx.set_variant(B.VARIANT_GRADIENT)
    orc.set_variant(ao.VARIANT_GRADIENT)
    for step in range(2):
        gs = wl.host_gradients(w, step)
        ctx.warmup_step(H.upload(gs)); orc.warmup_step(gs)
    ctx.freeze_v(); orc.freeze_v()
    for step in range(2, 6):
        gs = wl.host_gradients(w, step)
        if step == 4:
            import torch
            ctx.compressed_step_host([torch.from_numpy(g).pin_memory() for g in gs])      # the host-gradient path too
        else:
            ctx.compressed_step(H.upload(gs))
        orc.compressed_step(gs)
        for which, ref in ((B.STATE_X, orc.x), (B.STATE_M, orc.m), (B.STATE_V, orc.v), (B.STATE_SERVER_ERR, orc.server_err),
                           (B.STATE_SERVER_BITS, orc.server_bits), (B.STATE_SERVER_SCALES, orc.server_scales)):
            assert np.array_equal(ctx.get_state(which).view(np.uint32), ref.view(np.uint32)), (step, which)
        for i in range(n):
            assert np.array_equal(ctx.get_state(B.STATE_WORKER_ERR, i).view(np.uint32), orc.worker_err(i).view(np.uint32))
            assert np.array_equal(ctx.get_state(B.STATE_WORKER_BITS, i), orc.worker_bits(i))
    with pytest.raises(B.ApmsError) as e:
        ctx.set_variant(B.VARIANT_MOMENTUM)                    # fixed once a compression-phase step has run
    assert e.value.status == B.ERR_BAD_STATE


@pytest.mark.parametrize("d,n,chunk", [(4 * 1024 + 3, 4, 1024), (70001, 3, 4096), (2, 2, 32)])
def test_uncompressed_step_equals_the_identity_compressor(d, n, chunk):
    """v frozen, nothing compressed: the oracle with the identity compressor, bit for bit; then a compressed
    step after it still agrees (the momentum was handed over in binary32)."""
    w = tiny(d, n, chunk, cfg_id=161)
    ctx, orc = H.make_pair(w)
    for step in range(2):
        gs = wl.host_gradients(w, step)
        ctx.warmup_step(H.upload(gs)); orc.warmup_step(gs)
    ctx.freeze_v(); orc.freeze_v()
    orc.set_compressor(ao.IDENTITY)
    for step in range(2, 6):
        gs = wl.host_gradients(w, step)
        ctx.uncompressed_step(H.upload(gs)); orc.compressed_step(gs)
        for which, ref in ((B.STATE_X, orc.x), (B.STATE_M, orc.m)):
            assert np.array_equal(ctx.get_state(which).view(np.uint32), ref.view(np.uint32)), (step, which)
    orc.set_compressor(ao.ONEBIT)
    for step in range(6, 9):
        gs = wl.host_gradients(w, step)
        ctx.compressed_step(H.upload(gs)); orc.compressed_step(gs)
        if step == 7:                                          # and back: the momentum is spelled out from the message
            gs = wl.host_gradients(w, 100)
            orc.set_compressor(ao.IDENTITY)
            saved = [orc.worker_err(i).copy() for i in range(n)], orc.server_err.copy()
            for i in range(n):
                orc.worker_err(i)[:] = 0                       # the library's uncompressed step leaves the errors alone
            orc.server_err[:] = 0
            ctx.uncompressed_step(H.upload(gs)); orc.compressed_step(gs)
            for i in range(n):
                orc.worker_err(i)[:] = saved[0][i]
            orc.server_err[:] = saved[1]
            orc.set_compressor(ao.ONEBIT)
    H.compare_state(ctx, orc, w, exact=True)


# ------------------------------------------------------------------ the top-k compressor

def _topk_compare(ctx, orc, w, step):
    d, n = w.d, w.n
    idx = np.arange(d)
    for which, ref in ((B.STATE_X, orc.x), (B.STATE_M, orc.m), (B.STATE_SERVER_ERR, orc.server_err)):
        assert np.array_equal(ctx.get_state(which).view(np.uint32), ref.view(np.uint32)), (step, which)
    mask = (ctx.get_state(B.STATE_SERVER_BITS)[idx // 32] >> (idx % 32).astype(np.uint32)) & 1
    assert np.array_equal(mask.astype(np.uint8), orc.server_selected), (step, "server mask")
    for i in range(n):
        assert np.array_equal(ctx.get_state(B.STATE_WORKER_ERR, i).view(np.uint32), orc.worker_err(i).view(np.uint32)), (step, i)
        mask = (ctx.get_state(B.STATE_WORKER_BITS, i)[idx // 32] >> (idx % 32).astype(np.uint32)) & 1
        assert np.array_equal(mask.astype(np.uint8), orc.worker_selected(i)), (step, i, "mask")


@pytest.mark.parametrize("d,n,chunk,frac", [(5 * 4096 + 1234, 3, 4096, 0.01), (3 * 1024 + 5, 4, 96, 0.1), (2 * 32768 + 23552, 4, 32768, 0.01),
                                            (70000, 16, 160, 0.05), (9 * 512 + 3, 2, 512, 0.5), (300, 2, 64, 1.0), (1, 1, 32, 0.3),
                                            (3 * 65536 + 7, 2, 65536, 0.001),
                                            (131072 + 5000, 2, 131072, 0.01), (2 * 32768 + 100, 3, 32768, 0.1)])
def test_topk_compressor_bit_identical(d, n, chunk, frac):
    """Top-k compression of the momentum: selection masks, errors, momentum and model bit-identical to the oracle,
    through warmup, device-gradient steps, a host-gradient step and a bfloat16-gradient step."""
    import torch

    w = tiny(d, n, chunk, cfg_id=180)
    ctx, orc = H.make_pair(w)
    ctx.set_compressor(B.COMPRESSOR_TOPK, frac)
    orc.set_compressor(ao.TOPK); orc.set_topk_fraction(frac)
    for step in range(2):
        gs = wl.host_gradients(w, step)
        ctx.warmup_step(H.upload(gs)); orc.warmup_step(gs)
    ctx.freeze_v(); orc.freeze_v()
    for step in range(2, 8):
        gs = wl.host_gradients(w, step)
        if step == 5:
            ctx.compressed_step_host([torch.from_numpy(g).pin_memory() for g in gs])
        elif step == 6:
            g16 = [torch.from_numpy(g).to(torch.bfloat16) for g in gs]
            gs = [g.to(torch.float32).numpy() for g in g16]
            ctx.compressed_step([g.cuda() for g in g16])
        else:
            ctx.compressed_step(H.upload(gs))
        orc.compressed_step(gs)
        _topk_compare(ctx, orc, w, step)
    with pytest.raises(B.ApmsError) as e:
        ctx.set_compressor(B.COMPRESSOR_ONEBIT)               # fixed once a compression-phase step has run
    assert e.value.status == B.ERR_BAD_STATE


def test_topk_ties_and_teacher_forced_errors():
    """Many equal magnitudes (gradients drawn from three values) and errors forced from the oracle: the tie rule
    (lower index first) and apms_set_state in top-k mode."""
    w = tiny(4 * 256 + 40, 2, 256, cfg_id=181)
    ctx, orc = H.make_pair(w, x0=np.zeros(w.d, np.float32))
    ctx.set_compressor(B.COMPRESSOR_TOPK, 0.07)
    orc.set_compressor(ao.TOPK); orc.set_topk_fraction(0.07)
    ctx.freeze_v(); orc.freeze_v()
    rng = np.random.default_rng(5)
    for step in range(5):
        gs = [rng.choice(np.array([-0.5, 0.25, 0.5], np.float32), size=w.d) for _ in range(w.n)]
        if step == 3:
            orc.server_err[:] = rng.choice(np.array([-0.125, 0.0, 0.125], np.float32), size=w.d)
            for i in range(w.n):
                orc.worker_err(i)[:] = rng.choice(np.array([-0.125, 0.0, 0.125], np.float32), size=w.d)
            H.teacher_force(ctx, orc, w)
        ctx.compressed_step(H.upload(gs)); orc.compressed_step(gs)
        _topk_compare(ctx, orc, w, step)


def test_topk_threshold_jumps():
    """The kernels guess each chunk's threshold from the previous step's.  Gradients that grow and shrink by
    large factors between steps make the guess useless in both directions (no key reaches the window; the
    K-th key lies far above it): the selection must stay exact."""
    w = tiny(3 * 8192 + 700, 3, 8192, cfg_id=182)
    ctx, orc = H.make_pair(w)
    ctx.set_compressor(B.COMPRESSOR_TOPK, 0.02)
    orc.set_compressor(ao.TOPK); orc.set_topk_fraction(0.02)
    gs = wl.host_gradients(w, 0)
    ctx.warmup_step(H.upload(gs)); orc.warmup_step(gs)
    ctx.freeze_v(); orc.freeze_v()
    for step, factor in enumerate([1.0, 1.0, 4096.0, 1.0, 1.0 / 4096.0, 1.0 / 4096.0, 64.0, 1.0], start=1):
        gs = [(g * np.float32(factor)).astype(np.float32) for g in wl.host_gradients(w, step)]
        ctx.compressed_step(H.upload(gs)); orc.compressed_step(gs)
        _topk_compare(ctx, orc, w, step)


@pytest.mark.parametrize("lr,eps", [(-1e-3, 1e-8), (1e-3, 0.0)])
def test_topk_updates_every_element_when_skipping_is_not_exact(lr, eps):
    """With a negative learning rate or eps = 0 an element that is not kept need not come out of the update
    unchanged, so the server must not skip it: same bit-identical comparison, on the route that updates all."""
    w = tiny(5 * 4096 + 321, 3, 4096, cfg_id=184, lr=lr, eps=eps)
    ctx, orc = H.make_pair(w)
    ctx.set_compressor(B.COMPRESSOR_TOPK, 0.02)
    orc.set_compressor(ao.TOPK); orc.set_topk_fraction(0.02)
    for step in range(2):
        gs = wl.host_gradients(w, step)
        ctx.warmup_step(H.upload(gs)); orc.warmup_step(gs)
    ctx.freeze_v(); orc.freeze_v()
    for step in range(2, 8):
        gs = wl.host_gradients(w, step)
        ctx.compressed_step(H.upload(gs)); orc.compressed_step(gs)
        _topk_compare(ctx, orc, w, step)


@pytest.mark.parametrize("frac,chunk", [(0.01, 8192), (0.1, 8192), (0.03, 32768), (0.1, 32768), (0.25, 4096)])
def test_topk_long_free_run(frac, chunk):
    """60 free-running top-k steps: the predicted-threshold routes (one-sided window, two-sided band) run on
    thresholds that drift as the errors build up; masks, errors, momentum and model stay bit-identical."""
    w = tiny((6 if chunk < 32768 else 2) * chunk + 500, 3, chunk, cfg_id=183)
    ctx, orc = H.make_pair(w)
    ctx.set_compressor(B.COMPRESSOR_TOPK, frac)
    orc.set_compressor(ao.TOPK); orc.set_topk_fraction(frac)
    gs = wl.host_gradients(w, 0)
    ctx.warmup_step(H.upload(gs)); orc.warmup_step(gs)
    ctx.freeze_v(); orc.freeze_v()
    for step in range(1, 61):
        gs = wl.host_gradients(w, step)
        ctx.compressed_step(H.upload(gs)); orc.compressed_step(gs)
        if step % 10 == 0:
            _topk_compare(ctx, orc, w, step)


def test_topk_route_counts_add_up():
    """Every (worker, chunk) and every server chunk is settled on exactly one of the three routes each step, and
    with enough history the predicted list settles some of them (K = 984 of 32768: the two-sided band)."""
    w = tiny(4 * 32768 + 999, 3, 32768, cfg_id=189)
    ctx, orc = H.make_pair(w)
    ctx.set_compressor(B.COMPRESSOR_TOPK, 0.03)
    orc.set_compressor(ao.TOPK); orc.set_topk_fraction(0.03)
    gs = wl.host_gradients(w, 0)
    ctx.warmup_step(H.upload(gs)); orc.warmup_step(gs)
    ctx.freeze_v(); orc.freeze_v()
    ctx.topk_route_counts()
    predicted = 0
    for step in range(1, 25):
        gs = wl.host_gradients(w, step)
        ctx.compressed_step(H.upload(gs)); orc.compressed_step(gs)
        wr, sr = ctx.topk_route_counts()
        assert sum(wr[:3]) == w.n * w.n_chunks and sum(sr[:3]) == w.n_chunks, (step, wr, sr)
        assert sum(wr[3:]) <= w.n * w.n_chunks and min(wr) >= 0 and min(sr) >= 0
        predicted += wr[0]
    assert ctx.topk_route_counts() == ([0] * 6, [0] * 6)            # reset by the call
    assert predicted > 0
    _topk_compare(ctx, orc, w, 24)


def _topk_rows(ctxs, cb, ce):
    """The messages of all workers of `ctxs` for chunks [cb, ce) as a receiver holds them: mask rows (word 0 = first
    word of chunk cb) and rows of packed values, in worker order."""
    import torch

    c0 = ctxs[0]
    per = c0.topk_values_per_chunk()
    w0, w1 = cb * c0.chunk // 32, (min(c0.d, ce * c0.chunk) + 31) // 32
    masks, vals = [], []
    for ctx in ctxs:
        for i in range(ctx.n):
            masks.append(ctx.message(i)[0][w0:w1].clone())
            v = torch.full(((ce - cb) * per,), float("nan"), dtype=torch.float32, device="cuda")
            ctx.topk_pack_values(i, cb, ce, v)
            vals.append(v)
    return torch.stack(masks).contiguous(), torch.stack(vals).contiguous()


@pytest.mark.parametrize("d,n,chunk,frac,cuts", [(5 * 4096 + 1234, 3, 4096, 0.01, (0, 2, 6)), (7 * 96 + 5, 4, 96, 0.1, (0, 1, 5, 8)),
                                                 (2 * 32768 + 23552, 4, 32768, 0.05, (0, 1, 3)), (131072 + 5000, 2, 131072, 0.01, (0, 1, 2)),
                                                 (9 * 512 + 3, 2, 512, 0.5, (0, 4, 10)), (3 * 2080 + 64, 2, 2080, 1.0, (0, 3, 4))])
def test_topk_phase_wise_step_equals_the_whole_step(d, n, chunk, frac, cuts):
    """Top-k through the phase-wise calls: worker phase, the server phase range by range from packed messages
    (masks + the kept values, as they would arrive from other processes), apply phase - bit-identical to
    apms_compressed_step and to the oracle, over steps that take the kernels' different routes."""
    w = tiny(d, n, chunk, cfg_id=185)
    a, orc = H.make_pair(w)
    b = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    b.set_params(wl.initial_params(w))
    for c in (a, b):
        c.set_compressor(B.COMPRESSOR_TOPK, frac)
    orc.set_compressor(ao.TOPK); orc.set_topk_fraction(frac)
    gs = wl.host_gradients(w, 0)
    for c in (a, b):
        c.warmup_step(H.upload(gs))
        c.freeze_v()
    orc.warmup_step(gs); orc.freeze_v()
    assert cuts[-1] == a.C
    for step in range(1, 6):
        host = wl.host_gradients(w, step)
        gs = H.upload(host)
        a.compressed_step(gs)
        orc.compressed_step(host)
        b.worker_phase(gs)
        with pytest.raises(B.ApmsError) as e:
            b.server_phase_rows([b.message_ptrs(i)[0] for i in range(n)], [b.message_ptrs(i)[1] for i in range(n)], 0, b.C)
        assert e.value.status == B.ERR_BAD_STATE                    # top-k messages have their own server call
        for cb, ce in zip(cuts, cuts[1:]):
            masks, vals = _topk_rows([b], cb, ce)
            b.topk_server_phase(masks, vals, cb, ce)
        b.apply_phase()
        _topk_compare(a, orc, w, step)
        for k in (B.STATE_X, B.STATE_M, B.STATE_SERVER_ERR, B.STATE_SERVER_BITS):
            assert np.array_equal(a.get_state(k).view(np.uint32), b.get_state(k).view(np.uint32)), (step, k)
        for i in range(n):
            for k in (B.STATE_WORKER_ERR, B.STATE_WORKER_BITS):
                assert np.array_equal(a.get_state(k, i).view(np.uint32), b.get_state(k, i).view(np.uint32)), (step, k, i)
    with pytest.raises(B.ApmsError) as e:
        b.worker_phase_range(H.upload(wl.host_gradients(w, 9)), 0, 1)       # top-k compresses the whole vector at once
    assert e.value.status in (B.ERR_INVALID_ARG, B.ERR_BAD_STATE)


@pytest.mark.parametrize("d,chunk,frac", [(11 * 2048 + 77, 2048, 0.02), (3 * 32768 + 23552, 32768, 0.01), (9 * 96 + 5, 96, 0.25)])
def test_topk_two_emulated_ranks_equal_one_four_worker_run(d, chunk, frac):
    """Two contexts of two workers each stand for two processes: each serves half of the chunks from all four workers'
    packed messages and hands its range of the server's message (mask + kept values) to the other, which takes it over.
    Equal, bit for bit, to one context with all four workers and to the oracle."""
    import torch

    w = tiny(d, 4, chunk, cfg_id=186)
    whole, orc = H.make_pair(w)
    ranks = [B.Context(w.d, 2, w.beta1, w.beta2, w.eps, w.lr, w.chunk) for _ in range(2)]
    for c in [whole] + ranks:
        c.set_compressor(B.COMPRESSOR_TOPK, frac)
    orc.set_compressor(ao.TOPK); orc.set_topk_fraction(frac)
    x0 = wl.initial_params(w)
    for c in ranks:
        c.set_params(x0)
    host = wl.host_gradients(w, 0)
    gs = H.upload(host)
    whole.warmup_step(gs); orc.warmup_step(host)
    for r in range(2):                                   # the warmup phase averages all four workers' gradients everywhere
        ranks[r].restore(0, B.PHASE_WARMUP)
    whole.freeze_v(); orc.freeze_v()
    for r in range(2):
        for k in (B.STATE_X, B.STATE_V, B.STATE_M):
            ranks[r].set_state(k, whole.get_state(k))
        ranks[r].restore(1, B.PHASE_COMPRESSED)
    from paper_2008_11343_b200 import sharded
    ranges = sharded.chunk_ranges(whole.C, 2)
    per = whole.topk_values_per_chunk()
    for step in range(1, 5):
        host = wl.host_gradients(w, step)
        gs = H.upload(host)
        whole.compressed_step(gs)
        orc.compressed_step(host)
        for r in range(2):
            ranks[r].worker_phase(gs[2 * r:2 * r + 2])
        for r in range(2):
            cb, ce = ranges[r]
            masks, vals = _topk_rows(ranks, cb, ce)
            ranks[r].topk_server_phase(masks, vals, cb, ce)
        for r in range(2):                               # exchange 2: my range of the server's message to the other rank
            cb, ce = ranges[r]
            w0, w1 = cb * chunk // 32, (min(d, ce * chunk) + 31) // 32
            mask = ranks[r].message(-1)[0][w0:w1].clone()
            vals = torch.zeros((ce - cb) * per, dtype=torch.float32, device="cuda")
            ranks[r].topk_pack_values(-1, cb, ce, vals)
            ranks[1 - r].topk_put_server_range(mask, vals, cb, ce)
        for r in range(2):
            ranks[r].apply_phase()
        _topk_compare(whole, orc, w, step)
        for r in range(2):
            for which in (B.STATE_X, B.STATE_M, B.STATE_SERVER_BITS):
                assert np.array_equal(ranks[r].get_state(which).view(np.uint32), whole.get_state(which).view(np.uint32)), (step, r, which)
            lo, hi = ranges[r][0] * chunk, min(d, ranges[r][1] * chunk)
            assert np.array_equal(ranks[r].get_state(B.STATE_SERVER_ERR)[lo:hi].view(np.uint32),
                                  whole.get_state(B.STATE_SERVER_ERR)[lo:hi].view(np.uint32))
            for i in range(2):
                assert np.array_equal(ranks[r].get_state(B.STATE_WORKER_ERR, i).view(np.uint32),
                                      whole.get_state(B.STATE_WORKER_ERR, 2 * r + i).view(np.uint32))


def test_sharded_step_with_the_topk_compressor_equals_the_whole_step():
    import socket

    import torch.distributed as dist

    from paper_2008_11343_b200 import sharded

    w = tiny(11 * 2048 + 77, 4, 2048, cfg_id=187)
    a = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    b = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    for c in (a, b):
        c.set_compressor(B.COMPRESSOR_TOPK, 0.03)
        c.set_params(wl.initial_params(w))
        c.warmup_step(H.upload(wl.host_gradients(w, 0)))
        c.freeze_v()
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1)
    try:
        step = sharded.ShardedStep(b)
        for k in range(1, 5):
            gs = H.upload(wl.host_gradients(w, k))
            a.compressed_step(gs)
            step.step(gs)
        for k in (B.STATE_X, B.STATE_M, B.STATE_SERVER_ERR, B.STATE_SERVER_BITS):
            assert np.array_equal(a.get_state(k).view(np.uint32), b.get_state(k).view(np.uint32))
        for i in range(w.n):
            assert np.array_equal(a.get_state(B.STATE_WORKER_ERR, i).view(np.uint32), b.get_state(B.STATE_WORKER_ERR, i).view(np.uint32))
    finally:
        dist.destroy_process_group()


# ------------------------------------------------------------------ phase driver and error monitor

def test_scheduled_steps_follow_algorithm_1():
    """apms_step under a schedule = T_w Adam steps, the phase switch, then compression-phase steps, each with
    the schedule's learning rate; compared with the oracle driven by hand, bit for bit."""
    w = tiny(4 * 2048 + 300, 3, 2048, cfg_id=130)
    sc = B.Schedule(3, 2e-3, 4, 0.5, 2)                      # T_w = 3; ramp over 4 steps; halve every 2 steps
    ctx, orc = H.make_pair(w)
    ctx.set_schedule(sc)
    for k in range(9):
        gs = wl.host_gradients(w, k)
        lr = B.apms_schedule_lr(sc, k)
        orc.set_lr(lr)
        if k == 3:
            orc.freeze_v()
        (orc.warmup_step if k < 3 else orc.compressed_step)(gs)
        ctx.step(H.upload(gs))
        assert ctx.steps_taken == k + 1 and ctx.phase == (B.PHASE_WARMUP if k < 3 else B.PHASE_COMPRESSED)
        H.compare_state(ctx, orc, w, phase_compressed=k >= 3, exact=True)
    assert ctx.t == 3
    ctx.set_schedule(None)
    with pytest.raises(B.ApmsError) as e:
        ctx.step(H.upload(wl.host_gradients(w, 9)))
    assert e.value.status == B.ERR_BAD_STATE


def test_error_norms_match_the_oracle_state():
    """The monitor's squared norms of the worker and server errors against binary64 sums over the oracle's errors."""
    w = tiny(9 * 4096 + 777, 5, 4096, cfg_id=131)
    ctx, orc, _ = H.run_both(w, warmup=2, compressed=4, check_every_step=False)
    workers, server = ctx.error_norms()
    for i in range(w.n):
        ref = float(np.sum(orc.worker_err(i).astype(np.float64) ** 2))
        assert abs(workers[i] - ref) <= 1e-12 * ref
    ref = float(np.sum(orc.server_err.astype(np.float64) ** 2))
    assert abs(server - ref) <= 1e-12 * ref
    fresh = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    fresh.set_params(wl.initial_params(w))
    with pytest.raises(B.ApmsError) as e:
        fresh.error_norms()                                  # no errors exist before the phase switch
    assert e.value.status == B.ERR_BAD_STATE
    fresh.freeze_v()
    assert fresh.error_norms() == ([0.0] * w.n, 0.0)


# ------------------------------------------------------------------ phase-wise step (the multi-process form)

@pytest.mark.parametrize("d,n,chunk,cuts", [(9 * 2048 + 300, 4, 2048, (0, 3, 10)), (5 * 4096 + 1, 3, 4096, (0, 1, 5, 6)),
                                            (7 * 96 + 5, 5, 96, (0, 4, 8)), (3 * 70016, 2, 70016, (0, 2, 3)),
                                            (6 * 32768, 16, 32768, (0, 6)), (9 * 4096 + 100, 4, 4096, (0, 2, 3, 7, 10)),
                                            (5 * 2080 + 100, 3, 2080, (0, 2, 6)), (23 * 512 + 9, 2, 512, (0, 5, 6, 24)),
                                            (9 * 1056 + 700, 4, 1056, (0, 1, 2, 5, 9, 10)), (4 * 70016 + 33, 2, 70016, (0, 1, 3, 5))])
def test_phase_wise_step_equals_the_whole_step(d, n, chunk, cuts):
    """worker phase, the server phase range by range from COPIES of the messages laid out as a receiver would
    hold them (rows = senders, word 0 = first word of the range), apply phase: bit-identical to apms_compressed_step."""
    import torch

    w = tiny(d, n, chunk, cfg_id=140)
    a = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    b = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    for c in (a, b):
        c.set_params(wl.initial_params(w))
        c.warmup_step(H.upload(wl.host_gradients(w, 0)))
        c.freeze_v()
    assert cuts[-1] == a.C
    for step in range(1, 5):
        gs = H.upload(wl.host_gradients(w, step))
        a.compressed_step(gs)
        if step == 1:
            b.worker_phase(gs)
        else:                                                  # range by range, in another order every step
            pieces = list(zip(cuts, cuts[1:]))
            pieces = pieces[::-1] if step % 2 else pieces[1:] + pieces[:1]
            for cb, ce in pieces[:-1]:
                b.worker_phase_range(gs, cb, ce)
            with pytest.raises(B.ApmsError) as e:              # the worker phase does not cover every chunk yet
                b.server_phase_rows([b.message_ptrs(i)[0] for i in range(n)], [b.message_ptrs(i)[1] for i in range(n)], 0, b.C)
            assert e.value.status == B.ERR_BAD_STATE
            b.worker_phase_range(gs, *pieces[-1])
            with pytest.raises(B.ApmsError) as e:
                b.worker_phase_range(gs, 0, 1)                 # every chunk has been covered
            assert e.value.status == B.ERR_BAD_STATE
        msgs = [b.message(i) for i in range(n)]
        for cb, ce in zip(cuts, cuts[1:]):
            w0, w1 = cb * chunk // 32, (min(d, ce * chunk) + 31) // 32
            row_words = (w1 - w0 + 3) // 4 * 4
            bits_rows = torch.zeros((n, row_words), dtype=torch.int32, device="cuda")
            scale_rows = torch.zeros((n, ce - cb), dtype=torch.float32, device="cuda")
            for i, (bits, scales) in enumerate(msgs):
                bits_rows[i, :w1 - w0] = bits[w0:w1]
                scale_rows[i] = scales[cb:ce]
            b.server_phase(bits_rows, scale_rows, cb, ce)
        with pytest.raises(B.ApmsError) as e:
            b.compressed_step(gs)                              # a phase-wise step is in progress
        assert e.value.status == B.ERR_BAD_STATE
        b.apply_phase()
        for k in range(9):
            for i in (range(n) if k in (3, 4, 5) else [0]):
                assert np.array_equal(a.get_state(k, i).view(np.uint32), b.get_state(k, i).view(np.uint32)), (step, k, i)
    with pytest.raises(B.ApmsError) as e:
        b.apply_phase()                                        # nothing to apply
    assert e.value.status == B.ERR_BAD_STATE


def test_sharded_step_with_one_process_equals_the_whole_step():
    import socket

    import torch.distributed as dist

    from paper_2008_11343_b200 import sharded

    w = tiny(11 * 2048 + 77, 4, 2048, cfg_id=141)
    a = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    b = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    for c in (a, b):
        c.set_params(wl.initial_params(w))
        c.freeze_v()
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1)
    try:
        step = sharded.ShardedStep(b)
        for k in range(3):
            gs = H.upload(wl.host_gradients(w, k))
            a.compressed_step(gs)
            step.step(gs)
        for k in (B.STATE_X, B.STATE_M, B.STATE_SERVER_ERR, B.STATE_SERVER_BITS, B.STATE_SERVER_SCALES):
            assert np.array_equal(a.get_state(k).view(np.uint32), b.get_state(k).view(np.uint32))
    finally:
        dist.destroy_process_group()


def test_a_step_can_be_captured_in_a_cuda_graph_and_replayed():
    """apms_compressed_step only enqueues kernels on the context's stream, so it can be captured once and
    replayed (gradients refreshed in place between replays): the replayed steps equal eager steps bit for bit."""
    import torch

    w = tiny(6 * 4096 + 77, 3, 4096, cfg_id=151)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        a = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk, stream=s)
        b = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk, stream=s)
        gs = [g.to("cuda") for g in map(torch.from_numpy, wl.host_gradients(w, 0))]
        for c in (a, b):
            c.set_params(wl.initial_params(w))
            c.warmup_step(gs)
            c.freeze_v()
            c.compressed_step(gs)              # the first step of the phase differs (binary32 momentum): not the one to capture
        s.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=s):
            b.compressed_step(gs)              # recorded, not run
        for step in range(1, 6):
            for g, h in zip(gs, wl.host_gradients(w, step)):
                g.copy_(torch.from_numpy(h), non_blocking=False)
            a.compressed_step(gs)
            graph.replay()
        s.synchronize()
        for which in (B.STATE_X, B.STATE_SERVER_BITS, B.STATE_SERVER_SCALES, B.STATE_SERVER_ERR):
            assert np.array_equal(a.get_state(which).view(np.uint32), b.get_state(which).view(np.uint32)), which
        for i in range(w.n):
            assert np.array_equal(a.get_state(B.STATE_WORKER_ERR, i).view(np.uint32), b.get_state(B.STATE_WORKER_ERR, i).view(np.uint32))


# ------------------------------------------------------------------ the benchmark's small configurations

def test_config0_free_running_10_steps():
    """d = 2^20, n = 4, chunk = 4096: 5 warmup + 10 compressed steps, free-running.  Sign words
    bit-exact (ties aside), scales / errors / parameters within 1e-5 after 10 steps."""
    w = wl.config(0)
    _, _, reports = H.run_both(w, check_every_step=False)
    assert reports[-1]["server_tie_elems"] == 0


def test_long_free_run_does_not_drift():
    """150 compression-phase steps without any correction from the oracle, on a set that spans several chunk
    shapes' kernels (fine worker + fused staged server): the state stays bit-identical, i.e. nothing in the
    stored-z form, the 1-bit momentum or the error feedback accumulates a difference."""
    w = tiny(24 * 4096 + 1000, 4, 4096, cfg_id=150)
    ctx, orc, reports = H.run_both(w, warmup=3, compressed=150, check_every_step=False, exact=True)
    assert reports[-1]["server_tie_elems"] == 0


def test_config1_mixed_tensors_zero_gradients():
    """d = 2^24 in 64 tensors with per-tensor scales over three decades and 20 % zero gradient
    entries, n = 8, chunk = 8192, free-running for the configuration's own 10 warmup + 50 compressed steps;
    compared after the warmup phase, after the 10th compressed step and at the end."""
    w = wl.config(1)
    assert (w.warmup_steps, w.compressed_steps) == (10, 50)
    ctx, orc = H.make_pair(w)
    for step in range(w.warmup_steps):
        gs = wl.host_gradients(w, step)
        ctx.warmup_step(H.upload(gs)); orc.warmup_step(gs)
    H.compare_state(ctx, orc, w, phase_compressed=False)
    ctx.freeze_v(); orc.freeze_v()
    for k in range(w.compressed_steps):
        gs = wl.host_gradients(w, w.warmup_steps + k)
        ctx.compressed_step(H.upload(gs)); orc.compressed_step(gs)
        if k + 1 in (10, w.compressed_steps):
            report = H.compare_state(ctx, orc, w)
            assert report["server_tie_elems"] == 0


def test_structural_zero_gradients_stay_finite():
    """Elements whose gradient is always zero have v = 0; the update divides by eps alone and must
    stay finite and equal to the oracle's."""
    w = tiny(4096 + 40, 2, 1024, cfg_id=102, eps=1e-8)
    mask = np.ones(w.d, dtype=np.float32)
    mask[::7] = 0.0

    def grads(step):
        return [g * mask for g in wl.host_gradients(w, step)]

    ctx, orc, _ = H.run_both(w, warmup=2, compressed=3, exact=True, grads_fn=grads)
    assert np.isfinite(ctx.get_params()).all()


def test_all_zero_chunk_and_constant_magnitude():
    """Degenerate chunks: an all-zero chunk gives scale 0, all bits 1 and zero error; a chunk whose
    compensated entries all have one magnitude compresses without error."""
    d, n, chunk = 256, 2, 64
    w = tiny(d, n, chunk, cfg_id=103)
    ctx, orc = H.make_pair(w, x0=np.zeros(d, np.float32))
    ctx.freeze_v()
    orc.freeze_v()
    g = np.zeros(d, np.float32)
    g[64:128] = 0.5 * np.where(np.arange(64) % 3 == 0, -1.0, 1.0)
    g[128:192] = np.linspace(-1, 1, 64, dtype=np.float32)
    ctx.compressed_step(H.upload([g, g]))
    orc.compressed_step([g, g])
    H.compare_state(ctx, orc, w, exact=True)
    s0 = ctx.get_state(B.STATE_WORKER_SCALES, 0)
    bits = ctx.get_state(B.STATE_WORKER_BITS, 0)
    err = ctx.get_state(B.STATE_WORKER_ERR, 0)
    assert s0[0] == 0.0 and bits[0] == 0xFFFFFFFF and bits[1] == 0xFFFFFFFF and not err[:64].any()
    assert not err[64:128].any()                      # constant magnitude: C[z] = z


def test_nonfinite_gradient_propagates_like_the_oracle():
    w = tiny(300, 2, 64, cfg_id=104)
    ctx, orc = H.make_pair(w)
    ctx.freeze_v()
    orc.freeze_v()
    gs = wl.host_gradients(w, 0)
    gs[1][17] = np.nan
    ctx.compressed_step(H.upload(gs))
    orc.compressed_step(gs)
    for i in range(2):
        assert np.array_equal(ctx.get_state(B.STATE_WORKER_BITS, i), orc.worker_bits(i))
        a, b = ctx.get_state(B.STATE_WORKER_SCALES, i), orc.worker_scales(i)
        assert np.array_equal(np.isnan(a), np.isnan(b)) and np.array_equal(a[~np.isnan(a)], b[~np.isnan(b)])


# ------------------------------------------------------------------ properties of the CUDA path alone

def test_run_twice_is_bitwise_deterministic():
    w = tiny(9 * 4096 + 5, 4, 4096, cfg_id=105)

    def run():
        ctx = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
        ctx.set_params(wl.initial_params(w))
        for s in range(2):
            ctx.warmup_step(H.upload(wl.host_gradients(w, s)))
        ctx.freeze_v()
        for s in range(2, 6):
            ctx.compressed_step(H.upload(wl.host_gradients(w, s)))
        return [ctx.get_state(k, i) for k in range(9) for i in (range(w.n) if k in (3, 4, 5) else [0])]

    for a, b in zip(run(), run()):
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


def test_host_gradient_entry_point_matches_device_entry_point():
    import torch

    w = tiny(5 * 2048 + 100, 3, 2048, cfg_id=106)
    outs = []
    for host in (False, True):
        ctx = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
        ctx.set_params(wl.initial_params(w))
        ctx.warmup_step(H.upload(wl.host_gradients(w, 0)))
        ctx.freeze_v()
        x_host = torch.empty(w.d, dtype=torch.float32).pin_memory()
        for s in range(1, 4):
            gs = wl.host_gradients(w, s)
            if host:
                pinned = [torch.from_numpy(g).pin_memory() for g in gs]
                ctx.compressed_step_host(pinned, x_host)
                assert np.array_equal(x_host.numpy(), ctx.get_params())
            else:
                ctx.compressed_step(H.upload(gs))
        outs.append([ctx.get_state(k, i) for k in range(9) for i in (range(w.n) if k in (3, 4, 5) else [0])])
    for a, b in zip(*outs):
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


def test_checkpoint_restore_continues_bit_identically():
    w = tiny(3 * 1024 + 17, 2, 1024, cfg_id=107)
    a = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    a.set_params(wl.initial_params(w))
    a.warmup_step(H.upload(wl.host_gradients(w, 0)))
    a.freeze_v()
    for s in range(1, 4):
        a.compressed_step(H.upload(wl.host_gradients(w, s)))
    saved = {k: a.get_state(k) for k in (B.STATE_X, B.STATE_V, B.STATE_M, B.STATE_SERVER_ERR)}
    werr = [a.get_state(B.STATE_WORKER_ERR, i) for i in range(w.n)]
    b = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    b.set_params(np.zeros(w.d, np.float32))
    b.restore(a.t, B.PHASE_COMPRESSED)
    for k, val in saved.items():
        b.set_state(k, val)
    for i in range(w.n):
        b.set_state(B.STATE_WORKER_ERR, werr[i], worker=i)
    for s in range(4, 7):
        gs = H.upload(wl.host_gradients(w, s))
        a.compressed_step(gs)
        b.compressed_step(gs)
    for k in (B.STATE_X, B.STATE_M, B.STATE_SERVER_ERR, B.STATE_SERVER_BITS, B.STATE_SERVER_SCALES):
        assert np.array_equal(a.get_state(k).view(np.uint32), b.get_state(k).view(np.uint32))
    for i in range(w.n):
        assert np.array_equal(a.get_state(B.STATE_WORKER_ERR, i), b.get_state(B.STATE_WORKER_ERR, i))


@pytest.mark.parametrize("stop_at", [2, 5])
def test_checkpoint_under_a_schedule_resumes_the_learning_rate_and_the_warmup_count(stop_at):
    """A run driven by apms_step is checkpointed in the middle of the learning-rate ramp - once still in the
    warmup phase, once in the compression phase - and resumed in a fresh context: the resumed run must be
    bit-identical to the uninterrupted one (same learning rates, same number of Adam steps, same phase switch)."""
    w = tiny(4 * 1024 + 17, 3, 1024, cfg_id=112)
    sc = B.Schedule(3, 2e-3, 8, 0.5, 2)                      # T_w = 3; ramp over 8 steps; then halve every 2 steps
    a = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    a.set_params(wl.initial_params(w))
    a.set_schedule(sc)
    for k in range(stop_at):
        a.step(H.upload(wl.host_gradients(w, k)))
    compressed = a.phase == B.PHASE_COMPRESSED
    assert compressed == (stop_at > 3)
    saved = {k: a.get_state(k) for k in (B.STATE_X, B.STATE_V, B.STATE_M)}
    if compressed:
        saved[B.STATE_SERVER_ERR] = a.get_state(B.STATE_SERVER_ERR)
        werr = [a.get_state(B.STATE_WORKER_ERR, i) for i in range(w.n)]
    b = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    b.set_params(np.zeros(w.d, np.float32))
    b.set_schedule(sc)
    b.restore(a.t, a.phase, steps=a.steps_taken)
    for k, val in saved.items():
        b.set_state(k, val)
    if compressed:
        for i in range(w.n):
            b.set_state(B.STATE_WORKER_ERR, werr[i], worker=i)
    assert (b.t, b.phase, b.steps_taken) == (a.t, a.phase, a.steps_taken)
    for k in range(stop_at, 12):
        gs = H.upload(wl.host_gradients(w, k))
        a.step(gs)
        b.step(gs)
    assert (b.t, b.phase, b.steps_taken) == (a.t, a.phase, a.steps_taken) == (3, B.PHASE_COMPRESSED, 12)
    for k in (B.STATE_X, B.STATE_M, B.STATE_V, B.STATE_SERVER_ERR, B.STATE_SERVER_BITS, B.STATE_SERVER_SCALES):
        assert np.array_equal(a.get_state(k).view(np.uint32), b.get_state(k).view(np.uint32)), k
    for i in range(w.n):
        assert np.array_equal(a.get_state(B.STATE_WORKER_ERR, i).view(np.uint32), b.get_state(B.STATE_WORKER_ERR, i).view(np.uint32))
    if compressed:
        with pytest.raises(B.ApmsError) as e:
            b.set_variant(B.VARIANT_GRADIENT)                  # compression-phase steps count as taken after the restore
        assert e.value.status == B.ERR_BAD_STATE


def test_restore_to_warmup_spells_out_a_momentum_held_as_a_message():
    """After compression-phase steps the momentum lives in the server's message.  Going back to the WARMUP phase
    must hand Adam that momentum in binary32: the next Adam step equals the oracle's from the same state."""
    w = tiny(3 * 2048 + 40, 2, 2048, cfg_id=113)
    ctx, orc, _ = H.run_both(w, warmup=2, compressed=3, check_every_step=False, exact=True)
    ctx.restore(2, B.PHASE_WARMUP)
    fresh = ao.Oracle(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    fresh.set_params(orc.x.copy())
    gs = wl.host_gradients(w, 0)
    fresh.warmup_step(gs); fresh.warmup_step(gs)               # brings its t to 2; its state is replaced next
    fresh.x[:] = orc.x; fresh.m[:] = orc.m; fresh.v[:] = orc.v
    gs = wl.host_gradients(w, 9)
    ctx.warmup_step(H.upload(gs)); fresh.warmup_step(gs)
    assert ctx.t == 3
    for which, ref in ((B.STATE_X, fresh.x), (B.STATE_M, fresh.m), (B.STATE_V, fresh.v)):
        assert np.array_equal(ctx.get_state(which).view(np.uint32), ref.view(np.uint32)), which


def test_error_norms_with_the_topk_compressor():
    """Top-k mode keeps masks where the 1-bit mode keeps scales: the monitor must use delta = z where not sent."""
    w = tiny(5 * 4096 + 300, 3, 4096, cfg_id=114)
    ctx, orc = H.make_pair(w)
    ctx.set_compressor(B.COMPRESSOR_TOPK, 0.03)
    orc.set_compressor(ao.TOPK); orc.set_topk_fraction(0.03)
    gs = wl.host_gradients(w, 0)
    ctx.warmup_step(H.upload(gs)); orc.warmup_step(gs)
    ctx.freeze_v(); orc.freeze_v()
    for step in range(1, 4):
        gs = wl.host_gradients(w, step)
        ctx.compressed_step(H.upload(gs)); orc.compressed_step(gs)
    workers, server = ctx.error_norms()
    for i in range(w.n):
        ref = float(np.sum(orc.worker_err(i).astype(np.float64) ** 2))
        assert ref > 0 and abs(workers[i] - ref) <= 1e-12 * ref
    ref = float(np.sum(orc.server_err.astype(np.float64) ** 2))
    assert ref > 0 and abs(server - ref) <= 1e-12 * ref


def test_state_slices_agree_with_full_arrays():
    w = tiny(4 * 512 + 9, 2, 512, cfg_id=108)
    ctx, _, _ = H.run_both(w, warmup=1, compressed=2, check_every_step=False)
    for which in range(9):
        full = ctx.get_state(which, 1)
        lo, cnt = (3, 5) if full.size < 100 else (500, 777)
        lo, cnt = min(lo, full.size - 1), min(cnt, full.size - min(lo, full.size - 1))
        part = ctx.get_state_slice(which, lo, cnt, worker=1)
        assert np.array_equal(part.view(np.uint32), full[lo:lo + cnt].view(np.uint32))


# ------------------------------------------------------------------ boundary behaviour (error codes, no faults)

def test_phase_and_argument_errors_are_status_codes():
    import torch

    w = tiny(100, 2, 32, cfg_id=109)
    ctx = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    g = [torch.zeros(w.d, device="cuda") for _ in range(2)]
    with pytest.raises(B.ApmsError) as e:
        ctx.warmup_step(g)                      # no parameters yet
    assert e.value.status == B.ERR_BAD_STATE
    ctx.set_params(np.zeros(w.d, np.float32))
    with pytest.raises(B.ApmsError) as e:
        ctx.compressed_step(g)                  # before the phase switch
    assert e.value.status == B.ERR_BAD_STATE
    with pytest.raises(B.ApmsError) as e:
        B.apms_warmup_step(ctx._h, [g[0].data_ptr(), 0])
    assert e.value.status == B.ERR_INVALID_ARG
    with pytest.raises(B.ApmsError) as e:
        B.apms_warmup_step(ctx._h, [g[0].data_ptr(), g[1].data_ptr() + 4])     # misaligned
    assert e.value.status == B.ERR_INVALID_ARG
    ctx.warmup_step(g)
    ctx.freeze_v()
    with pytest.raises(B.ApmsError) as e:
        ctx.warmup_step(g)                      # after the phase switch
    assert e.value.status == B.ERR_BAD_STATE
    with pytest.raises(B.ApmsError) as e:
        ctx.freeze_v()
    assert e.value.status == B.ERR_BAD_STATE
    with pytest.raises(B.ApmsError) as e:
        ctx.get_state(B.STATE_WORKER_ERR, 5)
    assert e.value.status == B.ERR_INVALID_ARG
    for bad in [(0, 1, 32), (10, 0, 32), (10, 65, 32), (10, 1, 48), (10, 1, 0)]:
        with pytest.raises(B.ApmsError):
            B.apms_create(bad[0], bad[1], 0.9, 0.999, 1e-8, 1e-3, bad[2])
        assert B.apms_workspace_bytes(*bad) == 0
    ctx.compressed_step(g)                      # the context is still usable after all of the above
    assert ctx.launch_count == 1 + 3 + 1            # the warmup step; worker, server, update; sqrt(v) + eps formed once


def test_a_wait_that_gives_up_is_reported_and_the_context_survives():
    """A bounded wait that runs out (a barrier nothing completes, bound of a millisecond) sets the status word;
    the next synchronising call returns APMS_ERR_TIMEOUT; after apms_set_params the context works again."""
    w = tiny(3 * 2048 + 5, 2, 2048, cfg_id=170)
    ctx = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    x0 = wl.initial_params(w)
    ctx.set_params(x0)
    B.apms_selftest_wait_report(ctx._h)                       # reported and cleared
    assert np.array_equal(ctx.get_params(), x0)
    B.apms_selftest_wait_report(ctx._h, leave_reported=True)
    with pytest.raises(B.ApmsError) as e:
        ctx.get_params()
    assert e.value.status == B.ERR_TIMEOUT
    ctx.set_params(x0)                                        # clears the word
    ctx.freeze_v()
    ctx.compressed_step(H.upload(wl.host_gradients(w, 0)))
    assert np.isfinite(ctx.get_params()).all()


def test_library_owned_workspace_and_default_stream():
    """apms_create without apms_bind: the library allocates its own workspace."""
    import torch

    w = tiny(1000, 2, 128, cfg_id=110)
    h = B.apms_create(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    x0 = wl.initial_params(w)
    B.apms_set_params(h, x0.ctypes.data, False)
    orc = ao.Oracle(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    orc.set_params(x0)
    gs = wl.host_gradients(w, 0)
    dev = H.upload(gs)
    torch.cuda.synchronize()
    B.apms_warmup_step(h, [t.data_ptr() for t in dev])
    orc.warmup_step(gs)
    B.apms_freeze_v(h)
    orc.freeze_v()
    B.apms_compressed_step(h, [t.data_ptr() for t in dev])
    orc.compressed_step(gs)
    out = np.empty(w.d, np.float32)
    B.apms_get_params(h, out.ctypes.data, False)
    assert np.array_equal(out, orc.x)
    B.apms_destroy(h)
