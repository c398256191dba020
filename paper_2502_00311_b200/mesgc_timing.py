"""Step time of memory-efficient SGC (Section 4.4) on one flat gradient, timed on the device.

    python -m paper_2502_00311_b200.mesgc_timing [--d 16777216] [--steps 20] [--warmup 3] [--configs c:k:s,c:k:s,...]
    python -m paper_2502_00311_b200.mesgc_timing --cesgc m:n:r:c:k:s_c [--streams N]   (CESGC: the projections around the same core)

One JSON line per configuration (c chunks, k_c rows of A and s_c kept entries per chunk).  Gradients are synthetic
(Student-t noise plus c * s_c planted entries), four buffers used in rotation so that no step finds its input in L2;
CUDA events on the launching stream bracket the timed steps.  "launches" is what one step enqueued.
"""
import argparse
import json

import numpy as np
import torch

from . import binding, inputs

# the paper's settings: c = 256, s_c = 1, kappa = 8 (its reported runs) and the corners of its chunk-count study
# (s = 4096 entries in all, kappa = 7)
DEFAULT = "256:8:1,256:112:16,1024:28:4,4096:7:1"


def time_config(d, c, k, s_c, steps, warmup):
    hp = inputs.ADAM
    m = binding.Mesgc(d, c, k, s_c, 1, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], alpha=2.0)
    grads = []
    for i in range(4):
        supp, sign = inputs.planted_support(d, c * s_c, 100 + i)
        grads.append(torch.from_numpy(inputs.gradient(d, "student", supp, sign, 200 + i)).cuda())
    w = torch.from_numpy(inputs.weights(d, 5)).cuda()
    stream = torch.cuda.current_stream()
    for i in range(warmup):
        m.step(grads[i % 4], w)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    start.record(stream)
    for i in range(steps):
        m.step(grads[(warmup + i) % 4], w)
    stop.record(stream)
    torch.cuda.synchronize()
    ms = start.elapsed_time(stop) / steps
    out = dict(metric="mesgc_step_ms", d=d, c=c, k_c=k, s_c=s_c, value=ms, unit="ms", steps=steps, warmup=warmup,
               launches=m.chunks[0].last_launches(),
               status=int(np.bitwise_or.reduce([int(st.get("status")) for st in m.chunks[:: max(1, c // 16)]])),
               gradient_GBps=4.0 * d / ms / 1e6, data="synthetic", l2="4 rotating gradients of %d MiB" % (4 * d >> 20))
    m.close()
    return out


def time_cesgc(m, n, r, c, k, s_c, steps, warmup, n_streams=1):
    """CESGC (Section 4.4): the same core on the projected gradient B G (r x n), plus the two projections.

    n_streams > 1: that many matrices of this shape, each with its own states, stepped side by side on streams of their
    own (the small kernels of one matrix leave most of the GPU idle); the value is then the time per matrix."""
    hp = inputs.ADAM
    gen = torch.Generator(device="cuda").manual_seed(3)
    grads = [torch.randn(m, n, device="cuda", generator=gen) * 1e-3 for _ in range(4)]
    q, _ = torch.linalg.qr(torch.randn(m, r, device="cuda", generator=gen))       # any orthonormal B serves the timing
    B = q.t().contiguous()
    mats = []
    for _ in range(n_streams):
        ce = binding.Cesgc(m, n, r, c, k, s_c, 1, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], alpha=2.0)
        ce.set_projection(B)
        mats.append((ce, torch.zeros(m, n, device="cuda"), torch.cuda.Stream() if n_streams > 1 else torch.cuda.current_stream()))
    main_stream = torch.cuda.current_stream()

    def one_step(i):
        for ce, w, st in mats:
            if n_streams > 1:
                st.wait_stream(main_stream)
            ce.step(grads[i % 4], w, stream=st)
        if n_streams > 1:
            for _, _, st in mats:
                main_stream.wait_stream(st)

    for i in range(warmup):
        one_step(i)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    start.record(main_stream)
    for i in range(steps):
        one_step(warmup + i)
    stop.record(main_stream)
    torch.cuda.synchronize()
    ms = start.elapsed_time(stop) / steps / n_streams
    out = dict(metric="cesgc_step_ms_per_matrix", m=m, n=n, r=r, c=c, k_c=k, s_c=s_c, matrices_side_by_side=n_streams, value=ms,
               unit="ms", steps=steps, warmup=warmup, gradient_GBps=4.0 * m * n / ms / 1e6, data="synthetic",
               l2="4 rotating gradients of %d MiB" % (4 * m * n >> 20))
    for ce, _, _ in mats:
        ce.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--d", type=int, default=4096 * 4096)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--configs", default=DEFAULT)
    ap.add_argument("--cesgc", default="", help="m:n:r:c:k:s_c, e.g. 4096:4096:32:64:217:31 (the paper's CESGC setting)")
    ap.add_argument("--streams", type=int, default=1, help="with --cesgc: matrices stepped side by side, one stream each")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("a CUDA device is required")
    binding.lib()
    if args.cesgc:
        m, n, r, c, k, s_c = (int(v) for v in args.cesgc.split(":"))
        print(json.dumps(time_cesgc(m, n, r, c, k, s_c, args.steps, max(args.warmup, 3), args.streams)), flush=True)
        return
    for item in args.configs.split(","):
        c, k, s_c = (int(v) for v in item.split(":"))
        print(json.dumps(time_config(args.d, c, k, s_c, args.steps, max(args.warmup, 3))), flush=True)


if __name__ == "__main__":
    main()
