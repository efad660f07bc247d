"""Checks that pin the CPU oracle to things other than itself.

Every check takes the oracle's shared library as an argument, so the same
checks run against the real oracle (they must pass) and against oracles with a
planted mistake (at least one must fail; see test_oracle_mutants.py).
Each check raises AssertionError on failure.
"""
from __future__ import annotations

import os
from fractions import Fraction

import numpy as np

from oracle import apms_oracle as ao
from oracle import ps_reference as ps

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_fixture(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = [float(v) for v in vals]
    return out


def _rand_state(o, rng, err_scale=1e-3):
    """Put a frozen oracle into a generic mid-run state (nonzero m, v, errors)."""
    d, n = o.d, o.n
    o.x[:] = rng.standard_normal(d).astype(np.float32) * 0.02
    o.m[:] = rng.standard_normal(d).astype(np.float32) * 1e-3
    o.v[:] = (rng.standard_normal(d).astype(np.float32) * 1e-3) ** 2 + 1e-12
    o.server_err[:] = rng.standard_normal(d).astype(np.float32) * err_scale
    for i in range(n):
        o.worker_err(i)[:] = rng.standard_normal(d).astype(np.float32) * err_scale


def _frozen(lib, d, n, chunk, beta1=0.9, beta2=0.999, eps=1e-8, lr=1e-4):
    o = ao.Oracle(d, n, beta1, beta2, eps, lr, chunk, library=lib)
    o.set_params(np.zeros(d, dtype=np.float32))
    o.freeze_v()
    return o


def _unpack(bits, length):
    idx = np.arange(length)
    return ((bits[idx // 32] >> (idx % 32).astype(np.uint32)) & 1).astype(bool)


# ------------------------------------------------------------------ worked examples (golden text)

def check_worked_onebit_step(lib):
    """Hand-derived step with exact dyadic numbers (Section 3.3 + Section 5.1)."""
    f = read_fixture("onebit_step_worked_example.txt")
    o = ao.Oracle(4, 2, f["beta1"][0], 0.999, f["eps"][0], f["lr"][0], 32, library=lib)
    o.set_params(np.zeros(4, dtype=np.float32))
    o.freeze_v()
    o.m[:], o.v[:], o.x[:] = f["m"], f["v"], f["x"]
    o.worker_err(0)[:], o.worker_err(1)[:], o.server_err[:] = f["e0"], f["e1"], f["ebar"]
    o.compressed_step([np.array(f["g0"], np.float32), np.array(f["g1"], np.float32)])
    assert o.worker_scales(0)[0] == f["expect_scale0"][0]
    assert o.worker_scales(1)[0] == f["expect_scale1"][0]
    assert int(o.worker_bits(0)[0]) == int(f["expect_bits0"][0])
    assert int(o.worker_bits(1)[0]) == int(f["expect_bits1"][0])
    assert np.array_equal(o.worker_err(0), np.array(f["expect_e0"], np.float32))
    assert np.array_equal(o.worker_err(1), np.array(f["expect_e1"], np.float32))
    assert o.server_scales[0] == f["expect_Sbar"][0]
    assert int(o.server_bits[0]) == int(f["expect_Bbar"][0])
    assert np.array_equal(o.server_err, np.array(f["expect_ebar"], np.float32))
    assert np.array_equal(o.m, np.array(f["expect_m"], np.float32))
    assert np.array_equal(o.x, np.array(f["expect_x"], np.float32))


def check_worked_adam(lib):
    """Hand-derived first two Adam steps (Section 3.2)."""
    f = read_fixture("adam_first_steps_worked_example.txt")
    o = ao.Oracle(2, 2, f["beta1"][0], f["beta2"][0], f["eps"][0], f["lr"][0], 32, library=lib)
    o.set_params(np.array(f["x0"], np.float32))
    o.warmup_step([np.array(f["step1_g0"], np.float32), np.array(f["step1_g1"], np.float32)])
    assert np.array_equal(o.m, np.array(f["expect1_m"], np.float32))
    assert np.array_equal(o.v, np.array(f["expect1_v"], np.float32))
    assert np.array_equal(o.x, np.array(f["expect1_x"], np.float32))
    o.warmup_step([np.array(f["step2_g0"], np.float32), np.array(f["step2_g1"], np.float32)])
    assert np.array_equal(o.m, np.array(f["expect2_m"], np.float32))
    assert np.array_equal(o.v, np.array(f["expect2_v"], np.float32))
    np.testing.assert_allclose(o.x, f["expect2_x"], rtol=2e-7, atol=0)


# ------------------------------------------------------------------ library routine: Adam

def check_adam_matches_torch(lib):
    """Warmup phase == torch.optim.Adam (float64) on the worker-averaged gradient."""
    import torch

    rng = np.random.default_rng(11)
    d, n, steps = 257, 3, 12
    # the hyper-parameters are binary32 values at the oracle's interface; give torch the same reals
    b1, b2, eps, lr = (float(np.float32(h)) for h in (0.9, 0.999, 1e-8, 1e-3))
    x0 = rng.standard_normal(d) * 0.02
    o = ao.Oracle(d, n, b1, b2, eps, lr, 64, library=lib)
    o.set_params(x0.astype(np.float32))
    p = torch.nn.Parameter(torch.tensor(x0.astype(np.float32).astype(np.float64)))
    opt = torch.optim.Adam([p], lr=lr, betas=(b1, b2), eps=eps)
    for t in range(steps):
        if t == 6:
            lr = float(np.float32(5e-4))                # the schedule gamma_t may change per step
            o.set_lr(lr)
            opt.param_groups[0]["lr"] = lr
        gs = [(rng.standard_normal(d) * 0.01).astype(np.float32) for _ in range(n)]
        o.warmup_step(gs)
        p.grad = torch.tensor(np.mean(np.stack(gs).astype(np.float64), axis=0))
        opt.step()
    ref = p.detach().numpy()
    moved = np.abs(ref - x0).max()
    assert np.abs(o.x - ref).max() <= 2e-5 * moved + 1e-9, np.abs(o.x - ref).max() / moved
    st = opt.state[p]
    mm, vv = st["exp_avg"].numpy(), st["exp_avg_sq"].numpy()
    np.testing.assert_allclose(o.m, mm, rtol=0, atol=1e-6 * np.abs(mm).max())
    np.testing.assert_allclose(o.v, vv, rtol=0, atol=1e-6 * np.abs(vv).max())
    assert o.t == steps


# ------------------------------------------------------------------ compressor alone

def check_compressor_magnitude_and_signs(lib):
    """||scale * sign(z)||_2 = ||z||_2 (Section 5.1) and bit j <-> (z_j >= 0), LSB first."""
    rng = np.random.default_rng(5)
    for L in (1, 2, 31, 32, 33, 100, 4096):
        z = (rng.standard_normal(L) * 10.0 ** rng.uniform(-6, 2)).astype(np.float32)
        bits, s = ao.compress_1bit(z, library=lib)
        zz = z.astype(np.float64)
        np.testing.assert_allclose(float(s) * np.sqrt(L), np.sqrt((zz * zz).sum()), rtol=2e-7)
        assert np.array_equal(_unpack(bits, L), z >= 0)
        if L % 32:
            assert int(bits[-1]) >> (L % 32) == 0          # padding bits are zero
        q = ao.decompress_1bit(bits, s, L, library=lib)
        assert np.array_equal(q, np.where(z >= 0, s, -s).astype(np.float32))
        # payload: L/8 bytes of signs (rounded up to words) + one 4-byte scale
        assert bits.nbytes == 4 * ((L + 31) // 32)


def check_compressor_special_cases(lib):
    a = np.float32(0.375)
    signs = np.array([1, -1, -1, 1, 1, 1, -1, 1, -1], dtype=np.float32)
    bits, s = ao.compress_1bit(a * signs, library=lib)            # |z_j| = a  =>  scale = a, C[z] = z
    assert s == a and np.array_equal(ao.decompress_1bit(bits, s, 9, library=lib), a * signs)
    bits, s = ao.compress_1bit(np.zeros(40, np.float32), library=lib)   # zero chunk: scale 0, all bits 1
    assert s == 0.0 and int(bits[0]) == 0xFFFFFFFF and int(bits[1]) == 0xFF
    bits, s = ao.compress_1bit(np.array([-2.5], np.float32), library=lib)   # L = 1: scale = |z|
    assert s == np.float32(2.5) and int(bits[0]) == 0
    bits, s = ao.compress_1bit(np.array([-0.0, 0.0, -1.0, np.nan], np.float32), library=lib)
    assert int(bits[0]) == 0b0011                                  # -0.0 counts as >= 0; NaN gives 0
    z = np.array([3.0, -4.0], np.float32)                          # l1-mean switch: mean |z|
    _, s1 = ao.compress_1bit(z, ao.SCALE_L1_MEAN, library=lib)
    _, s2 = ao.compress_1bit(z, ao.SCALE_L2, library=lib)
    assert s1 == np.float32(3.5) and s2 == np.float32(np.sqrt(12.5))
    # idempotence: compressing an already compressed vector changes nothing
    zc = ao.decompress_1bit(*ao.compress_1bit(np.array([1, -7, -1, 7], np.float32), library=lib), 4,
                            library=lib)
    b2, s2 = ao.compress_1bit(zc, library=lib)
    assert np.array_equal(ao.decompress_1bit(b2, s2, 4, library=lib), zc)


# ------------------------------------------------------------------ invariants of one step

def check_error_compensation_identity(lib):
    """C[z] + delta_new = z (Section 3.1; Supplement A), worker and server side, plus
    magnitude preservation per chunk, on a ragged multi-chunk problem."""
    rng = np.random.default_rng(7)
    d, n, chunk = 5 * 96 + 41, 3, 96
    o = _frozen(lib, d, n, chunk, beta1=0.9)
    _rand_state(o, rng)
    m_old, e_old, eb_old = o.m.copy(), [o.worker_err(i).copy() for i in range(n)], o.server_err.copy()
    gs = [(rng.standard_normal(d) * 3e-3).astype(np.float32) for _ in range(n)]
    o.compressed_step(gs)
    b1 = np.float32(0.9)
    avg = np.zeros(d, np.float64)
    for i in range(n):
        z = (np.float64(b1) * m_old + np.float64(np.float32(1) - b1) * gs[i]) + e_old[i]   # binary64
        sent = np.empty(d, np.float32)
        for c in range(o.C):
            sl = slice(c * chunk, min(d, (c + 1) * chunk))
            L = sl.stop - sl.start
            sent[sl] = ao.decompress_1bit(o.worker_bits(i)[sl.start // 32:], o.worker_scales(i)[c], L,
                                          library=lib)
            np.testing.assert_allclose(float(o.worker_scales(i)[c]) * np.sqrt(L),
                                       np.sqrt((z[sl] ** 2).sum()), rtol=1e-5)
        assert np.array_equal(sent >= 0, z >= 0) or np.abs(z[(sent >= 0) != (z >= 0)]).max() < 1e-9
        np.testing.assert_allclose(sent.astype(np.float64) + o.worker_err(i), z, rtol=0,
                                   atol=4e-7 * np.abs(z).max())
        avg += sent
    zbar = avg / n + eb_old
    for c in range(o.C):
        sl = slice(c * chunk, min(d, (c + 1) * chunk))
        L = sl.stop - sl.start
        np.testing.assert_allclose(float(o.server_scales[c]) * np.sqrt(L),
                                   np.sqrt((zbar[sl] ** 2).sum()), rtol=1e-5)
    np.testing.assert_allclose(o.m.astype(np.float64) + o.server_err, zbar, rtol=0,
                               atol=4e-7 * np.abs(zbar).max())
    # the broadcast momentum is the decompressed server message
    for c in range(o.C):
        sl = slice(c * chunk, min(d, (c + 1) * chunk))
        q = ao.decompress_1bit(o.server_bits[sl.start // 32:], o.server_scales[c], sl.stop - sl.start,
                               library=lib)
        assert np.array_equal(o.m[sl], q)


def check_two_formulations(lib):
    """Chunked binary32 oracle == per-chunk parameter-server form in binary64 (Supplement A)."""
    rng = np.random.default_rng(13)
    d, n, chunk, steps = 4 * 64 + 17, 4, 64, 6
    beta, lr, eps = 0.9, 1e-3, 1e-8
    o = _frozen(lib, d, n, chunk, beta1=beta, lr=lr, eps=eps)
    _rand_state(o, rng)
    m, x, v = o.m.astype(np.float64), o.x.astype(np.float64), o.v.astype(np.float64)
    we = [o.worker_err(i).astype(np.float64) for i in range(n)]
    se = o.server_err.astype(np.float64)
    beta64 = float(np.float32(beta))
    for _ in range(steps):
        gs = [(rng.standard_normal(d) * 2e-3).astype(np.float32) for _ in range(n)]
        # teacher-force the binary64 side from the oracle's state so ties cannot accumulate
        m, x = o.m.astype(np.float64), o.x.astype(np.float64)
        we = [o.worker_err(i).astype(np.float64) for i in range(n)]
        se = o.server_err.astype(np.float64)
        m, x, we, se = ps.chunked_step(m, x, v, we, se, [g.astype(np.float64) for g in gs],
                                       beta64, float(np.float32(lr)), float(np.float32(eps)), chunk)
        o.compressed_step(gs)
        scale = np.abs(m).max()
        np.testing.assert_allclose(o.m, m, rtol=2e-6, atol=0)              # same signs, same scales
        np.testing.assert_allclose(o.server_err, se, rtol=0, atol=3e-6 * scale)
        for i in range(n):
            np.testing.assert_allclose(o.worker_err(i), we[i], rtol=0, atol=3e-6 * np.abs(we[i]).max())
        np.testing.assert_allclose(o.x, x, rtol=0, atol=1e-6 * np.abs(x).max())


def check_telescoping_and_virtual_sequence(lib):
    """m_t + dbar_t = beta m_{t-1} + (1-beta) gbar_t + dbar_{t-1}   (Supplement A, last display)
    and the shadow sequence y = x - lr/(1-beta) (beta m + dbar)/(sqrt v + eps) moves by
    -lr gbar/(sqrt v + eps) per step (Lemma 2's auxiliary sequence, indices aligned to the
    state between two steps), so the compressed run tracks uncompressed preconditioned SGD."""
    rng = np.random.default_rng(17)
    d, n, chunk, steps = 3 * 128 + 50, 4, 128, 25
    beta, lr, eps = 0.9, 2e-3, 1e-6
    b = float(np.float32(beta))
    omb = float(np.float32(1) - np.float32(beta))
    o = _frozen(lib, d, n, chunk, beta1=beta, lr=lr, eps=eps)
    o.x[:] = rng.standard_normal(d).astype(np.float32) * 0.02
    o.m[:] = rng.standard_normal(d).astype(np.float32) * 1e-3
    o.v[:] = (rng.standard_normal(d).astype(np.float32) * 1e-3) ** 2 + 1e-10
    pre = 1.0 / (np.sqrt(o.v.astype(np.float64)) + float(np.float32(eps)))
    lr64 = float(np.float32(lr))

    def dbar():
        return sum(o.worker_err(i).astype(np.float64) for i in range(n)) / n + o.server_err

    def y():
        return o.x - lr64 / (1.0 - b) * (b * o.m.astype(np.float64) + dbar()) * pre

    y0, gsum = y(), np.zeros(d)
    for _ in range(steps):
        m_prev, dbar_prev = o.m.astype(np.float64), dbar()
        gs = [(rng.standard_normal(d) * 2e-3).astype(np.float32) for _ in range(n)]
        gbar = np.mean(np.stack(gs).astype(np.float64), axis=0)
        o.compressed_step(gs)
        lhs = o.m.astype(np.float64) + dbar()
        rhs = b * m_prev + omb * gbar + dbar_prev
        np.testing.assert_allclose(lhs, rhs, rtol=0, atol=1e-6 * np.abs(rhs).max())
        gsum += gbar
    # 1 - b is not exactly omb in binary32/64 mix; tolerance covers that and the fp32 steps
    drift = y() - y0
    expect = -lr64 * gsum * pre
    np.testing.assert_allclose(drift, expect, rtol=0, atol=2e-5 * np.abs(expect).max())


def check_identity_compressor_closed_form(lib):
    """With C = identity (the paper's "uncompressed" variant, Section 5.3) errors stay 0 and
    m_T = beta^T m_0 + (1-beta) sum_k beta^(T-k) gbar_k ;  x_T = x_0 - lr sum_t m_t/(sqrt v + eps)."""
    rng = np.random.default_rng(19)
    d, n, chunk, steps = 200, 4, 64, 9
    beta, lr, eps = 0.9, 1e-2, 1e-8
    o = _frozen(lib, d, n, chunk, beta1=beta, lr=lr, eps=eps)
    o.set_compressor(ao.IDENTITY)
    _rand_state(o, rng, err_scale=0.0)
    b = float(np.float32(beta))
    omb = float(np.float32(1) - np.float32(beta))
    m = o.m.astype(np.float64)
    x = o.x.astype(np.float64)
    pre = float(np.float32(lr)) / (np.sqrt(o.v.astype(np.float64)) + float(np.float32(eps)))
    for _ in range(steps):
        gs = [(rng.standard_normal(d) * 1e-2).astype(np.float32) for _ in range(n)]
        o.compressed_step(gs)
        m = b * m + omb * np.mean(np.stack(gs).astype(np.float64), axis=0)
        x = x - pre * m
        assert not o.server_err.any() and not any(o.worker_err(i).any() for i in range(n))
    np.testing.assert_allclose(o.m, m, rtol=0, atol=2e-6 * np.abs(m).max())
    np.testing.assert_allclose(o.x, x, rtol=0, atol=1e-6 * np.abs(x).max())


# ------------------------------------------------------------------ the gradient-compressing variant

def check_gradient_variant_worked_example(lib):
    """Hand-derived step of the gradient-compressing variant (Section 5.3, item 4) in exact dyadic numbers."""
    f = read_fixture("gradient_variant_worked_example.txt")
    o = ao.Oracle(4, 2, f["beta1"][0], 0.999, f["eps"][0], f["lr"][0], 32, library=lib)
    o.set_params(np.zeros(4, dtype=np.float32))
    o.freeze_v()
    o.set_variant(ao.VARIANT_GRADIENT)
    o.m[:], o.v[:], o.x[:] = f["m"], f["v"], f["x"]
    o.worker_err(0)[:], o.worker_err(1)[:], o.server_err[:] = f["e0"], f["e1"], f["ebar"]
    o.compressed_step([np.array(f["g0"], np.float32), np.array(f["g1"], np.float32)])
    assert o.worker_scales(0)[0] == f["expect_scale0"][0] and o.worker_scales(1)[0] == f["expect_scale1"][0]
    assert int(o.worker_bits(0)[0]) == int(f["expect_bits0"][0]) and int(o.worker_bits(1)[0]) == int(f["expect_bits1"][0])
    assert np.array_equal(o.worker_err(0), np.array(f["expect_e0"], np.float32))
    assert np.array_equal(o.worker_err(1), np.array(f["expect_e1"], np.float32))
    assert o.server_scales[0] == f["expect_Sbar"][0] and int(o.server_bits[0]) == int(f["expect_Bbar"][0])
    assert np.array_equal(o.server_err, np.array(f["expect_ebar"], np.float32))
    assert np.array_equal(o.m, np.array(f["expect_m"], np.float32))
    assert np.array_equal(o.x, np.array(f["expect_x"], np.float32))


def check_gradient_variant_identity_is_momentum_sgd(lib):
    """Gradient variant with C = identity: nothing is lost, so the run is momentum SGD on the averaged
    gradient with the frozen preconditioner - checked against torch.optim.SGD (momentum = dampening =
    beta1, binary64) fed with the preconditioned gradient gbar/(sqrt v + eps)."""
    import torch

    rng = np.random.default_rng(23)
    d, n, chunk, steps = 150, 3, 64, 10
    beta, lr, eps = (float(np.float32(h)) for h in (0.9, 1e-2, 1e-8))
    o = _frozen(lib, d, n, chunk, beta1=beta, lr=lr, eps=eps)
    o.set_compressor(ao.IDENTITY)
    o.set_variant(ao.VARIANT_GRADIENT)
    _rand_state(o, rng, err_scale=0.0)
    pre = 1.0 / (np.sqrt(o.v.astype(np.float64)) + eps)
    p = torch.nn.Parameter(torch.tensor(o.x.astype(np.float64)))
    opt = torch.optim.SGD([p], lr=lr, momentum=beta, dampening=float(np.float32(beta)))
    # dampening must be beta1 as binary32 rounds 1 - beta1: use the oracle's own (1 - beta1)
    opt.param_groups[0]["dampening"] = 1.0 - float(np.float32(1) - np.float32(beta))
    opt.state[p]["momentum_buffer"] = torch.tensor(o.m.astype(np.float64) * pre)     # m/(sqrt v + eps) evolves linearly
    x0 = o.x.astype(np.float64).copy()
    for _ in range(steps):
        gs = [(rng.standard_normal(d) * 1e-2).astype(np.float32) for _ in range(n)]
        o.compressed_step(gs)
        p.grad = torch.tensor(np.mean(np.stack(gs).astype(np.float64), axis=0) * pre)
        opt.step()
        assert not o.server_err.any() and not any(o.worker_err(i).any() for i in range(n))
    ref = p.detach().numpy()
    assert np.abs(o.x - ref).max() <= 2e-6 * np.abs(ref - x0).max() + 1e-7 * np.abs(ref).max()
    np.testing.assert_allclose(o.m * pre, opt.state[p]["momentum_buffer"].numpy(), rtol=0,
                               atol=2e-6 * np.abs(o.m * pre).max())


def check_gradient_variant_invariants(lib):
    """Gradient variant, 1-bit compressor: ghat_t + dbar_t = gbar_t + dbar_{t-1} (the telescoping of
    Supplement A written for the gradient), m_t = beta m_{t-1} + (1-beta) ghat_t with ghat_t the
    decompressed server message, and x moves by -lr m_t/(sqrt v + eps) with the NEW momentum."""
    rng = np.random.default_rng(29)
    d, n, chunk, steps = 3 * 96 + 20, 4, 96, 8
    beta, lr, eps = 0.9, 2e-3, 1e-6
    b, omb = float(np.float32(beta)), float(np.float32(1) - np.float32(beta))
    o = _frozen(lib, d, n, chunk, beta1=beta, lr=lr, eps=eps)
    o.set_variant(ao.VARIANT_GRADIENT)
    _rand_state(o, rng)
    pre = float(np.float32(lr)) / (np.sqrt(o.v.astype(np.float64)) + float(np.float32(eps)))

    def dbar():
        return sum(o.worker_err(i).astype(np.float64) for i in range(n)) / n + o.server_err

    for _ in range(steps):
        m_prev, x_prev, dbar_prev = o.m.astype(np.float64), o.x.astype(np.float64), dbar()
        gs = [(rng.standard_normal(d) * 2e-3).astype(np.float32) for _ in range(n)]
        gbar = np.mean(np.stack(gs).astype(np.float64), axis=0)
        o.compressed_step(gs)
        ghat = np.concatenate([ao.decompress_1bit(o.server_bits[c * chunk // 32:], o.server_scales[c],
                                                  min(d, (c + 1) * chunk) - c * chunk, library=lib)
                               for c in range(o.C)]).astype(np.float64)
        rhs = gbar + dbar_prev
        np.testing.assert_allclose(ghat + dbar(), rhs, rtol=0, atol=1e-6 * np.abs(rhs).max())
        np.testing.assert_allclose(o.m, b * m_prev + omb * ghat, rtol=0, atol=2e-7 * np.abs(ghat).max())
        step = pre * o.m.astype(np.float64)
        np.testing.assert_allclose(x_prev - o.x, step, rtol=0, atol=1e-6 * np.abs(step).max() + 2e-7 * np.abs(x_prev).max())


# ------------------------------------------------------------------ the top-k compressor

def check_topk_compressor_against_a_library_sort(lib):
    """Kept set = the first K of a stable sort by descending |z| (numpy), ties to the lower index."""
    rng = np.random.default_rng(31)
    for L, K in [(1, 1), (8, 2), (33, 5), (100, 100), (257, 1), (1000, 10), (4096, 41)]:
        z = (rng.standard_normal(L) * 10.0 ** rng.uniform(-3, 1)).astype(np.float32)
        z[rng.random(L) < 0.2] = 0.0
        if L >= 8:
            z[3], z[5], z[6] = z[1], -z[1], z[1]                  # equal magnitudes of both signs
            z[7] = -0.0
        q, sel = ao.compress_topk(z, K, library=lib)
        order = np.argsort(-np.abs(z.astype(np.float64)), kind="stable")      # stable: lower index first among equals
        expect = np.zeros(L, bool)
        expect[order[:K]] = True
        assert np.array_equal(sel.astype(bool), expect), (L, K)
        assert np.array_equal(q[expect], z[expect]) and not q[~expect].any()
        assert int(sel.sum()) == K
    assert ao.topk_count(0.01, 32768, library=lib) == 328 and ao.topk_count(0.5, 7, library=lib) == 4
    assert ao.topk_count(1e-9, 100, library=lib) == 1 and ao.topk_count(1.0, 100, library=lib) == 100


def check_topk_worked_step(lib):
    """Hand-derived step with the top-k compressor (Section 5.1 + Section 3.3), exact dyadic numbers."""
    f = read_fixture("topk_step_worked_example.txt")
    o = ao.Oracle(8, 2, f["beta1"][0], 0.999, f["eps"][0], f["lr"][0], 32, library=lib)
    o.set_params(np.zeros(8, dtype=np.float32))
    o.freeze_v()
    o.set_compressor(ao.TOPK)
    o.set_topk_fraction(f["frac"][0])
    o.m[:], o.v[:], o.x[:] = f["m"], f["v"], f["x"]
    o.worker_err(0)[:], o.worker_err(1)[:], o.server_err[:] = f["e0"], f["e1"], f["ebar"]
    o.compressed_step([np.array(f["g0"], np.float32), np.array(f["g1"], np.float32)])
    assert np.array_equal(o.worker_selected(0), np.array(f["expect_sel0"], np.uint8))
    assert np.array_equal(o.worker_selected(1), np.array(f["expect_sel1"], np.uint8))
    assert np.array_equal(o.worker_err(0), np.array(f["expect_e0"], np.float32))
    assert np.array_equal(o.worker_err(1), np.array(f["expect_e1"], np.float32))
    assert np.array_equal(o.server_selected, np.array(f["expect_selbar"], np.uint8))
    assert np.array_equal(o.server_err, np.array(f["expect_ebar"], np.float32))
    assert np.array_equal(o.m, np.array(f["expect_m"], np.float32))
    assert np.array_equal(o.x, np.array(f["expect_x"], np.float32))


def check_topk_invariants_and_full_fraction(lib):
    """Top-k steps on a ragged multi-chunk problem: K elements kept per chunk and message, the error is
    zero on them and the whole compensated value elsewhere, no dropped magnitude exceeds a kept one, the
    telescoping identity of Supplement A holds (it needs nothing of the compressor), the momentum is the
    server's sparse message.  With k = 100 % the compressor is the identity: same run, bit for bit."""
    rng = np.random.default_rng(37)
    d, n, chunk, frac = 4 * 96 + 37, 3, 96, 0.1
    b, omb = float(np.float32(0.9)), float(np.float32(1) - np.float32(0.9))
    o = _frozen(lib, d, n, chunk, beta1=0.9, lr=1e-3)
    o.set_compressor(ao.TOPK)
    o.set_topk_fraction(frac)
    _rand_state(o, rng)

    def dbar():
        return sum(o.worker_err(i).astype(np.float64) for i in range(n)) / n + o.server_err

    for _ in range(5):
        m_prev, dbar_prev, x_prev = o.m.astype(np.float64), dbar(), o.x.copy()
        e_prev = [o.worker_err(i).copy() for i in range(n)]
        gs = [(rng.standard_normal(d) * 3e-3).astype(np.float32) for _ in range(n)]
        o.compressed_step(gs)
        for c in range(o.C):
            sl = slice(c * chunk, min(d, (c + 1) * chunk))
            K = ao.topk_count(frac, sl.stop - sl.start, library=lib)
            for i in range(n):
                sel = o.worker_selected(i)[sl].astype(bool)
                z = (b * m_prev[sl] + omb * gs[i][sl].astype(np.float64)) + e_prev[i][sl]       # binary64 view of z
                assert int(sel.sum()) == K and not o.worker_err(i)[sl][sel].any()
                np.testing.assert_allclose(o.worker_err(i)[sl][~sel], z[~sel], rtol=0, atol=4e-7 * np.abs(z).max())
                assert np.abs(z[sel]).min() >= np.abs(z[~sel]).max() - 4e-7 * np.abs(z).max()
            sel = o.server_selected[sl].astype(bool)
            assert int(sel.sum()) == K and not o.server_err[sl][sel].any() and not o.m[sl][~sel].any()
            assert np.array_equal(o.x[sl][~sel], x_prev[sl][~sel])          # nothing received, nothing moves
        rhs = b * m_prev + omb * np.mean(np.stack(gs).astype(np.float64), axis=0) + dbar_prev
        np.testing.assert_allclose(o.m.astype(np.float64) + dbar(), rhs, rtol=0, atol=1e-6 * np.abs(rhs).max())

    a1 = _frozen(lib, d, n, chunk, beta1=0.9, lr=1e-3)
    a2 = _frozen(lib, d, n, chunk, beta1=0.9, lr=1e-3)
    a1.set_compressor(ao.TOPK); a1.set_topk_fraction(1.0)
    a2.set_compressor(ao.IDENTITY)
    rng2 = np.random.default_rng(41)
    _rand_state(a1, rng2, err_scale=0.0)
    a2.x[:], a2.m[:], a2.v[:] = a1.x, a1.m, a1.v
    for _ in range(4):
        gs = [(rng2.standard_normal(d) * 3e-3).astype(np.float32) for _ in range(n)]
        a1.compressed_step(gs); a2.compressed_step(gs)
        assert np.array_equal(a1.x.view(np.uint32), a2.x.view(np.uint32)) and np.array_equal(a1.m.view(np.uint32), a2.m.view(np.uint32))


def check_phase_switch(lib):
    """After warmup: v stays fixed, raw m carries over, all errors start at zero (Algorithm 1
    initialisation; Section 3.3 first paragraph)."""
    rng = np.random.default_rng(23)
    d, n = 96, 2
    o = ao.Oracle(d, n, 0.9, 0.999, 1e-8, 1e-3, 32, library=lib)
    o.set_params(rng.standard_normal(d).astype(np.float32))
    for _ in range(3):
        o.warmup_step([rng.standard_normal(d).astype(np.float32) for _ in range(n)])
    m_w, v_w = o.m.copy(), o.v.copy()
    try:
        o.compressed_step([np.zeros(d, np.float32)] * n)
        raise AssertionError("compressed step accepted before the phase switch")
    except RuntimeError:
        pass
    o.freeze_v()
    assert np.array_equal(o.m, m_w) and np.array_equal(o.v, v_w)
    assert not o.server_err.any() and not o.worker_err(0).any() and not o.worker_err(1).any()
    gs = [rng.standard_normal(d).astype(np.float32) for _ in range(n)]
    x_before = o.x.copy()
    o.compressed_step(gs)
    assert np.array_equal(o.v, v_w)                     # v no longer updated
    # first compressed step uses Adam's raw momentum: z_i = 0.9 m_w + 0.1 g_i exactly (errors 0)
    z0 = np.float32(0.9) * m_w.astype(np.float64) + np.float64(np.float32(1) - np.float32(0.9)) * gs[0]
    assert np.array_equal(_unpack(o.worker_bits(0), d), z0 >= 0)
    # model update uses sqrt(v) + eps of the frozen, not bias-corrected, v
    expect = x_before - np.float64(np.float32(1e-3)) * o.m / (np.sqrt(v_w.astype(np.float64)) + 1e-8)
    np.testing.assert_allclose(o.x, expect, rtol=3e-7)
    try:
        o.warmup_step(gs)
        raise AssertionError("warmup step accepted after the phase switch")
    except RuntimeError:
        pass


# ------------------------------------------------------------------ metamorphic

def check_metamorphic(lib):
    rng = np.random.default_rng(29)
    d, n, chunk = 3 * 64 + 7, 2, 64

    def run(scale=1.0, flip=1.0, perm=(0, 1)):
        o = _frozen(lib, d, n, chunk, beta1=0.9, lr=1e-3)
        r = np.random.default_rng(31)
        _rand_state(o, r)
        f = np.float32(scale * flip)
        o.m[:] *= f
        o.server_err[:] *= f
        errs = [o.worker_err(i).copy() * f for i in range(n)]
        for i in range(n):
            o.worker_err(i)[:] = errs[perm[i]]
        out = []
        for _ in range(3):
            gs = [(r.standard_normal(d) * 1e-3).astype(np.float32) * f for _ in range(n)]
            o.compressed_step([gs[perm[i]] for i in range(n)])
            out.append((o.server_bits.copy(), o.server_scales.copy(), o.m.copy(),
                        [o.worker_bits(i).copy() for i in range(n)],
                        [o.worker_err(i).copy() for i in range(n)]))
        return out

    base = run()
    for k, (a, b) in enumerate(zip(base, run(scale=2.0 ** -7))):       # power-of-two scaling is exact
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1] * np.float32(2.0 ** -7), b[1]), k
        assert all(np.array_equal(x * np.float32(2.0 ** -7), y) for x, y in zip(a[4], b[4]))
    pad = np.uint32((1 << (d % 32)) - 1)
    for a, b in zip(base, run(flip=-1.0)):                             # global sign flip
        assert np.array_equal(a[1], b[1]) and np.array_equal(a[2], -b[2])
        full = (~a[0]).astype(np.uint32)
        full[-1] &= pad
        assert np.array_equal(full, b[0])                              # no exact zeros in this draw
    for a, b in zip(base, run(perm=(1, 0))):                           # worker order: n = 2 sums commute
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
        assert np.array_equal(a[3][0], b[3][1]) and np.array_equal(a[4][1], b[4][0])


# ------------------------------------------------------------------ exact-rational brute force

def check_bruteforce_exact(lib):
    """Tiny problems on a dyadic grid where every binary32 operation is exact, replayed in exact
    rational arithmetic; scales are compared through their squares (scale^2 * L = sum z^2 needs
    a perfect square, so inputs are drawn until the rational scale is exact)."""
    rng = np.random.default_rng(37)
    half = Fraction(1, 2)
    done = 0
    for trial in range(4000):
        L, n = int(rng.integers(1, 5)), int(rng.integers(1, 4))
        m = [Fraction(int(v), 4) for v in rng.integers(-8, 9, L)]
        eb = [Fraction(int(v), 4) for v in rng.integers(-8, 9, L)]
        es = [[Fraction(int(v), 4) for v in rng.integers(-8, 9, L)] for _ in range(n)]
        gs = [[Fraction(int(v), 2) for v in rng.integers(-16, 17, L)] for _ in range(n)]

        def csqrt(fr):                       # exact rational square root or None
            import math
            a, b = math.isqrt(fr.numerator), math.isqrt(fr.denominator)
            return Fraction(a, b) if a * a == fr.numerator and b * b == fr.denominator else None

        ok, sent, new_es, scales, bitsw = True, [], [], [], []
        for i in range(n):
            z = [half * m[j] + half * gs[i][j] + es[i][j] for j in range(L)]
            s = csqrt(sum(v * v for v in z) / L)
            if s is None:
                ok = False
                break
            q = [s if v >= 0 else -s for v in z]
            sent.append(q)
            new_es.append([z[j] - q[j] for j in range(L)])
            scales.append(s)
            bitsw.append(sum(1 << j for j in range(L) if z[j] >= 0))
        if not ok:
            continue
        if n == 3:                           # division by 3 is not exact in binary32
            continue
        zb = [sum(sent[i][j] for i in range(n)) / n + eb[j] for j in range(L)]
        S = csqrt(sum(v * v for v in zb) / L)
        if S is None:
            continue
        qb = [S if v >= 0 else -S for v in zb]
        o = ao.Oracle(L, n, 0.5, 0.999, 0.0, 0.5, 32, library=lib)
        o.set_params(np.zeros(L, np.float32))
        o.freeze_v()
        o.m[:] = [float(v) for v in m]
        o.v[:] = 4.0                                           # sqrt(v) = 2: division stays exact
        o.x[:] = 1.0
        o.server_err[:] = [float(v) for v in eb]
        for i in range(n):
            o.worker_err(i)[:] = [float(v) for v in es[i]]
        o.compressed_step([np.array([float(v) for v in g], np.float32) for g in gs])
        for i in range(n):
            assert Fraction(float(o.worker_scales(i)[0])) == scales[i]
            assert int(o.worker_bits(i)[0]) == bitsw[i]
            assert [Fraction(float(v)) for v in o.worker_err(i)] == new_es[i]
        assert Fraction(float(o.server_scales[0])) == S
        assert int(o.server_bits[0]) == sum(1 << j for j in range(L) if zb[j] >= 0)
        assert [Fraction(float(v)) for v in o.server_err] == [zb[j] - qb[j] for j in range(L)]
        assert [Fraction(float(v)) for v in o.m] == qb
        assert [Fraction(float(v)) for v in o.x] == [1 - half * qb[j] / 2 for j in range(L)]
        done += 1
        if done >= 60:
            break
    assert done >= 20, f"only {done} exact cases found"


ALL_CHECKS = [
    check_worked_onebit_step,
    check_worked_adam,
    check_adam_matches_torch,
    check_compressor_magnitude_and_signs,
    check_compressor_special_cases,
    check_error_compensation_identity,
    check_two_formulations,
    check_telescoping_and_virtual_sequence,
    check_identity_compressor_closed_form,
    check_phase_switch,
    check_metamorphic,
    check_bruteforce_exact,
    check_gradient_variant_worked_example,
    check_gradient_variant_identity_is_momentum_sgd,
    check_gradient_variant_invariants,
    check_topk_compressor_against_a_library_sort,
    check_topk_worked_step,
    check_topk_invariants_and_full_fraction,
]
