"""Launch ONE kernel of the library a few times on a small case, for a profiler to capture.

    python -m paper_2008_11343_b200.profile_kernels --kernel k_apply [--d 33554432] [--n 8] [--launches 3]

Every kernel of the library can be reached by name; the case (d = 2^25 elements of the BERT-Large-shaped
set, n = 8 workers unless the kernel needs otherwise) is larger than L2 and holds a few GB on the device,
so that a capture of a handful of counters ends by itself in seconds.  The module only calls the public
binding; it computes nothing itself.  Prints one line per kernel with the CUDA-event time per launch and
the bytes the launch has to move, so that the same command is useful without a profiler too.
"""
from __future__ import annotations

import argparse
import json
import sys


def _setup(d, n, chunk, compressor=None, variant=None, team=None, first_step=False, grad_dtype="float32", steps=1):
    import torch

    from . import binding as B
    from . import workloads as wl

    w = wl.sliced(wl.config(3), d).with_(n=n, chunk=chunk)
    ctx = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk)
    if compressor is not None:
        ctx.set_compressor(B.COMPRESSOR_TOPK, compressor)
    if variant is not None:
        ctx.set_variant(variant)
    if team is not None:
        ctx.set_team_mode(team)
    x0 = torch.empty(w.d, dtype=torch.float32, device="cuda").normal_(0.0, w.x0_std)
    ctx.set_params(x0)
    dt = getattr(torch, grad_dtype)
    grads = []
    for i in range(n):
        g = torch.empty(w.d, dtype=torch.float32, device="cuda")
        wl.device_gradient(w, 0, i, g)
        grads.append(g if dt == torch.float32 else g.to(dt))
    ctx.warmup_step(grads)
    ctx.warmup_step(grads)
    ctx.freeze_v()
    if not first_step:
        for _ in range(steps):              # the first step of the phase reads the binary32 momentum: not the steady state
            ctx.compressed_step(grads)      # (top-k: the predicted-threshold routes need a few steps of history)
    torch.cuda.synchronize()
    return ctx, w, grads


# kernel name -> (what to set up, what to call per launch, which timer of the library sees it)
def _cases(args):
    from . import binding as B

    d, n = args.d, args.n
    return {
        "k_warmup_adam": dict(setup=dict(chunk=32768), phase="warmup", timer=B.KERNEL_WARMUP_ADAM,
                              bytes=lambda w: (4 * w.n + 24) * w.d),
        "k_worker_fine": dict(setup=dict(chunk=32768), call="worker_phase", timer=B.KERNEL_WORKER,
                              bytes=lambda w: w.n * (12 * w.d + w.d // 8) + w.d // 8),
        "k_worker_fine_split": dict(setup=dict(chunk=32768 + 32), call="worker_phase", timer=B.KERNEL_WORKER,
                                    bytes=lambda w: w.n * (12 * w.d + w.d // 8) + w.d // 8),
        "k_worker_fine_bf16": dict(setup=dict(chunk=32768, grad_dtype="bfloat16"), call="worker_phase", timer=B.KERNEL_WORKER,
                                   bytes=lambda w: w.n * (10 * w.d + w.d // 8) + w.d // 8),
        "k_worker_fine_words": dict(setup=dict(chunk=128), call="worker_phase", timer=B.KERNEL_WORKER,
                                    bytes=lambda w: w.n * (12 * w.d + w.d // 8) + w.d // 8),
        "k_finalize_words": dict(setup=dict(chunk=128), call="worker_phase", timer=B.KERNEL_WORKER,
                                 bytes=lambda w: w.n * (8 * (w.d // 32) + 4 * w.n_chunks)),
        "k_worker": dict(setup=dict(chunk=160, team=B.TEAM_WARP), call="worker_phase", timer=B.KERNEL_WORKER,
                         bytes=lambda w: w.n * (12 * w.d + w.d // 8) + w.d // 8),
        "k_worker_m32": dict(setup=dict(chunk=32768, first_step=True), call="first_worker_phase", timer=B.KERNEL_WORKER,
                             bytes=lambda w: w.n * (12 * w.d + w.d // 8) + 4 * w.d),
        "k_finalize_fine": dict(setup=dict(chunk=32768), call="worker_phase", timer=B.KERNEL_WORKER,
                                bytes=lambda w: w.n * (8 * (w.d // 512) + 4 * w.n_chunks)),
        "k_server_staged": dict(setup=dict(chunk=32768), call="step", timer=B.KERNEL_SERVER,
                                bytes=lambda w: w.n * w.d // 8 + 8 * w.d + w.d // 8 + 12 * w.d),
        "k_server_staged_unfused": dict(setup=dict(chunk=4 * 65536), call="worker_phase", timer=B.KERNEL_SERVER,
                                        bytes=lambda w: w.n * w.d // 8 + 8 * w.d + w.d // 8),
        "k_server_staged_lagged": dict(setup=dict(chunk=4 * 65536), call="step", timer=B.KERNEL_SERVER,
                                       bytes=lambda w: w.n * w.d // 8 + 8 * w.d + w.d // 4 + 12 * w.d),
        "k_server_packed": dict(setup=dict(chunk=1024), call="step", timer=B.KERNEL_SERVER,
                                bytes=lambda w: w.n * w.d // 8 + 8 * w.d + w.d // 8 + 12 * w.d),
        "k_server": dict(setup=dict(chunk=160), call="step", timer=B.KERNEL_SERVER,
                         bytes=lambda w: w.n * w.d // 8 + 8 * w.d + w.d // 8),
        "k_apply": dict(setup=dict(chunk=160), call="step", timer=B.KERNEL_APPLY,
                        bytes=lambda w: 12 * w.d + w.d // 8),
        "k_make_den": dict(setup=dict(chunk=32768, first_step=True), call="make_den", timer=None,
                           bytes=lambda w: 8 * w.d),
        "k_apply_gradient": dict(setup=dict(chunk=32768, variant=B.VARIANT_GRADIENT), call="step", timer=B.KERNEL_APPLY,
                                 bytes=lambda w: 20 * w.d + w.d // 8),
        "k_uncompressed": dict(setup=dict(chunk=32768), call="uncompressed", timer=B.KERNEL_WARMUP_ADAM,
                               bytes=lambda w: (4 * w.n + 20) * w.d),
        "k_noalloc_compress": dict(setup=None, call="noalloc", timer=None, bytes=lambda w: 4 * w.d + w.d // 8),
        "k_topk_worker": dict(setup=dict(chunk=32768, compressor=0.01), call="step", timer=B.KERNEL_WORKER,
                              bytes=lambda w: w.n * (12 * w.d + w.d // 4) + 4 * w.d),
        "k_topk_server": dict(setup=dict(chunk=32768, compressor=0.01), call="step", timer=B.KERNEL_SERVER,
                              bytes=lambda w: w.n * (w.d // 8 + int(0.04 * w.d)) + 24 * w.d + w.d // 8),
        "k_topk_worker_band": dict(setup=dict(chunk=32768, compressor=0.03, steps=8), call="step", timer=B.KERNEL_WORKER,
                                   bytes=lambda w: w.n * (12 * w.d + w.d // 4) + 4 * w.d),
        "k_topk_worker_two_pass": dict(setup=dict(chunk=32768, compressor=0.1, steps=1), call="step", timer=B.KERNEL_WORKER,
                                       bytes=lambda w: w.n * (12 * w.d + w.d // 4) + 4 * w.d),
        "k_topk_server_dense": dict(setup=dict(chunk=32768, compressor=0.03, steps=8), call="step", timer=B.KERNEL_SERVER,
                                    bytes=lambda w: w.n * (w.d // 8 + int(0.12 * w.d)) + 24 * w.d + w.d // 8),
        "k_error_norm_tiles": dict(setup=dict(chunk=32768), call="error_norms", timer=None,
                                   bytes=lambda w: 4 * (w.n + 1) * w.d),
    }


def main(argv=None) -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--kernel", required=True)
    ap.add_argument("--d", type=int, default=1 << 25)
    ap.add_argument("--n", type=int, default=8)
    ap.add_argument("--launches", type=int, default=3)
    args = ap.parse_args(argv)

    import torch

    from . import binding as B
    from . import workloads as wl

    cases = _cases(args)
    if args.kernel not in cases:
        print("unknown kernel; one of: " + " ".join(sorted(cases)), file=sys.stderr)
        return 2
    case = cases[args.kernel]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if case["setup"] is None:                                   # the entry point without a context
        w = wl.sliced(wl.config(3), args.d).with_(n=1, chunk=32768)
        z = torch.empty(w.d, dtype=torch.float32, device="cuda").normal_()
        bits = torch.empty((w.d + 31) // 32, dtype=torch.int32, device="cuda")
        scales = torch.empty(w.n_chunks, dtype=torch.float32, device="cuda")
        stream = torch.cuda.current_stream().cuda_stream
        call = lambda: B.apms_compress_noalloc(z.data_ptr(), w.d, w.chunk, bits.data_ptr(), scales.data_ptr(), stream)
        call()
        ctx = None
    else:
        ctx, w, grads = _setup(args.d, args.n, **case["setup"])
        kind = case.get("call")
        if case.get("phase") == "warmup":
            ctx.restore(2, B.PHASE_WARMUP)
            call = lambda: ctx.warmup_step(grads)
        elif kind == "step":
            call = lambda: ctx.compressed_step(grads)
        elif kind == "worker_phase":
            def call():
                ctx.worker_phase(grads)
                ctx.server_phase_rows([ctx.message_ptrs(i)[0] for i in range(w.n)],
                                      [ctx.message_ptrs(i)[1] for i in range(w.n)], 0, ctx.C)
                ctx.apply_phase()
        elif kind == "first_worker_phase":
            def call():                                          # the binary32 momentum is authoritative again after set_state(M)
                ctx.set_state(B.STATE_M, ctx.get_state(B.STATE_M))
                ctx.compressed_step(grads)
        elif kind == "make_den":
            def call():                                          # a new v invalidates the stored sqrt(v) + eps
                ctx.set_state(B.STATE_V, ctx.get_state(B.STATE_V))
                ctx.compressed_step(grads)
        elif kind == "uncompressed":
            call = lambda: ctx.uncompressed_step(grads)
        elif kind == "error_norms":
            call = lambda: ctx.error_norms()
        else:
            raise AssertionError(kind)
        call()
    torch.cuda.synchronize()
    if ctx is not None and case["timer"] is not None:
        ctx.set_timing(True)
        ctx.kernel_time(case["timer"])
    e0.record()
    for _ in range(args.launches):
        call()
    e1.record()
    torch.cuda.synchronize()
    out = {"kernel": args.kernel, "d": w.d, "n": w.n, "chunk": w.chunk, "launches": args.launches,
           "algorithmic_bytes_per_launch": int(case["bytes"](w))}
    if ctx is not None and case["timer"] is not None:
        ms, cnt = ctx.kernel_time(case["timer"])
        out["ms_per_launch"] = ms / max(cnt, 1)
        out["timed"] = "library events around the kernel (and, for the worker, its finalize kernel)"
    else:
        out["ms_per_launch"] = e0.elapsed_time(e1) / args.launches
        out["timed"] = "events around the whole call"
    out["algorithmic_gbs"] = out["algorithmic_bytes_per_launch"] / (out["ms_per_launch"] * 1e-3) / 1e9
    print(json.dumps(out))
    return 0


if __name__ == "__main__":
    sys.exit(main())
