"""The allocation-free entry point, apms_compress_noalloc, against the ordinary path and the CPU oracle.

Some callers of this library cannot allocate device memory: a step function running inside a
framework region where allocator calls are forbidden, a plugin that owns nothing but the buffers
and the stream it was handed, a loop that cannot tolerate the device-wide synchronisation a
cudaMalloc implies.  For them the library compresses a vector using only a fixed scratch array
that is part of the library itself.  This test drives that entry point through the C ABI and
requires the same sign words and scales as the context-based step produces for the same vector -
and as the CPU oracle's compressor (Section 5.1) gives chunk by chunk -
on two calls issued back to back (the second must not be disturbed by what the first left in
the shared scratch array), and requires that oversize shapes are refused with a message.

Collected last on purpose (file name), so that a run stopping at the first failure has already
run every other test.  It builds all of its own inputs and passes in a fresh process as well.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import apms_oracle as ao
from paper_2008_11343_b200 import binding as B

REL = 1e-5      # the scale tolerance of the parity tests; sign words must be equal


def _reference(z: np.ndarray, chunk: int):
    """Sign words and scales of z from the existing entry point: with one worker, beta1 = 0,
    zero momentum and zero errors, the compensated vector of a compression-phase step is the
    gradient itself, so the worker's message is C[z]."""
    import torch

    ctx = B.Context(z.size, 1, 0.0, 0.999, 1e-8, 1e-4, chunk)
    ctx.set_params(np.zeros(z.size, np.float32))
    ctx.freeze_v()
    ctx.compressed_step([torch.from_numpy(z).cuda()])
    bits, scales = ctx.get_state(B.STATE_WORKER_BITS, 0), ctx.get_state(B.STATE_WORKER_SCALES, 0)
    ctx.close()
    return bits, scales


def _oracle(z: np.ndarray, chunk: int):
    """Sign words and scales of z from the CPU oracle's 1-bit compressor, one chunk at a time."""
    bits = np.zeros((z.size + 31) // 32, np.uint32)
    scales = []
    for lo in range(0, z.size, chunk):
        b, s = ao.compress_1bit(z[lo:lo + chunk])
        bits[lo // 32:lo // 32 + b.size] = b          # chunks are multiples of 32 elements: whole words
        scales.append(s)
    return bits, np.asarray(scales, np.float32)


def _vector(d: int, seed: int) -> np.ndarray:
    rng = np.random.default_rng(seed)
    z = (rng.standard_normal(d) * 10.0 ** rng.uniform(-4, 0, size=d)).astype(np.float32)
    z[rng.random(d) < 0.05] = 0.0                 # exact zeros count as non-negative
    return z


def test_two_calls_in_a_row_match_the_context_path():
    import torch

    # call 1: chunks longer than a tile (several scratch slots per chunk) and a ragged last chunk;
    # call 2: a different, smaller shape, so that slots written by call 1 are stale when it runs
    cases = [(300_000, 131_104, 1), (5 * 8192 + 77, 8192, 2)]
    inputs = [_vector(d, seed) for d, _, seed in cases]
    expected = [_reference(z, chunk) for z, (_, chunk, _) in zip(inputs, cases)]

    dev_in = [torch.from_numpy(z).cuda() for z in inputs]
    outs = []
    for (d, chunk, _) in cases:                  # every buffer the calls need exists before them
        bits = torch.full(((d + 31) // 32,), -1, dtype=torch.int32, device="cuda")
        scales = torch.full(((d + chunk - 1) // chunk,), float("nan"), dtype=torch.float32, device="cuda")
        outs.append((bits, scales))
    stream = torch.cuda.current_stream().cuda_stream
    # the first call on a device also looks up the scratch array's address: do it once up front
    B.apms_compress_noalloc(dev_in[1].data_ptr(), cases[1][0], cases[1][1],
                            outs[1][0].data_ptr(), outs[1][1].data_ptr(), stream)
    torch.cuda.synchronize()
    outs[1][0].fill_(-1)
    outs[1][1].fill_(float("nan"))
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for z, (d, chunk, _), (bits, scales) in zip(dev_in, cases, outs):      # back to back, one stream
        B.apms_compress_noalloc(z.data_ptr(), d, chunk, bits.data_ptr(), scales.data_ptr(), stream)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after >= free_before, "device memory was allocated during the calls"

    for z, zdev, (d, chunk, _), (bits, scales), (ref_bits, ref_scales) in zip(inputs, dev_in, cases, outs, expected):
        got_bits = bits.cpu().numpy().view(np.uint32)
        assert np.array_equal(got_bits, ref_bits), f"d={d} chunk={chunk}: sign words differ"
        np.testing.assert_allclose(scales.cpu().numpy(), ref_scales, rtol=REL, atol=0)
        orc_bits, orc_scales = _oracle(z, chunk)
        assert np.array_equal(got_bits, orc_bits), f"d={d} chunk={chunk}: sign words differ from the oracle's"
        np.testing.assert_allclose(scales.cpu().numpy(), orc_scales, rtol=REL, atol=0)
        assert np.array_equal(zdev.cpu().numpy(), z)                       # the input is not modified


def test_shapes_beyond_the_fixed_scratch_are_refused_with_a_message():
    import torch

    z = torch.zeros(64, dtype=torch.float32, device="cuda")
    bits = torch.zeros(2, dtype=torch.int32, device="cuda")
    scales = torch.zeros(2, dtype=torch.float32, device="cuda")
    too_many_chunks = (B.NOALLOC_MAX_TILES + 1) * 32          # chunk = 32 -> one tile per chunk
    for d, chunk in [(too_many_chunks, 32), (2 ** 40, 2 ** 20), (0, 32), (64, 48)]:
        with pytest.raises(B.ApmsError) as e:                 # refused before any launch
            B.apms_compress_noalloc(z.data_ptr(), d, chunk, bits.data_ptr(), scales.data_ptr())
        assert e.value.status == B.ERR_INVALID_ARG and "apms_compress_noalloc" in str(e.value)
    with pytest.raises(B.ApmsError):
        B.apms_compress_noalloc(z.data_ptr() + 4, 32, 32, bits.data_ptr(), scales.data_ptr())   # misaligned
    B.apms_compress_noalloc(z.data_ptr(), 64, 32, bits.data_ptr(), scales.data_ptr())           # still usable
    torch.cuda.synchronize()
    assert bits.cpu().numpy().view(np.uint32).tolist() == [0xFFFFFFFF, 0xFFFFFFFF]
    assert scales.cpu().numpy().tolist() == [0.0, 0.0]
