"""Seeded synthetic inputs for the SGC step (gradients, weights, planted supports).

This module serves both the CUDA path and the CPU oracle and therefore contains none of the
method's arithmetic: it only draws numbers.  Everything is generated with numpy's PCG64 so that a
(config, matrix, step) triple names the same buffer on every machine.

Workloads (shapes follow LLaMA-2-7B projection matrices; gradients follow the premise of
Section 3.2 that fine-tuning gradients are quasi-sparse: a few dominant entries over small noise):

  kind "gauss"    : N(0, 0.1^2) noise, planted magnitudes U(1, 2)         (small 64x64 case)
  kind "student"  : 1e-3 * Student-t(nu=3) noise, planted magnitudes U(0.5, 1)

Planted entries REPLACE the noise at s uniformly drawn distinct positions with a random sign.  The
planted support and signs are fixed for a whole run (the paper assumes the support of the
sparsified gradient drifts little over time, Section 3.3); magnitudes and noise are fresh each step.
"""
import numpy as np

# name -> (matrices [(rows, cols)], k, s, kind, seed_A, steps)
CONFIGS = {
    "c1_64x64": dict(shapes=[(64, 64)], k=256, s=16, kind="gauss", seed=0, steps=10),
    "c2_4096x4096": dict(shapes=[(4096, 4096)], k=2048, s=64, kind="student", seed=1, steps=100),
    "c3_llama7b_layer": dict(shapes=[(4096, 4096)] * 4 + [(11008, 4096)] * 2 + [(4096, 11008)], k=2048, s=128,
                             kind="student", seed=1, steps=50),
    "c4_llama7b_32layers": dict(shapes=([(4096, 4096)] * 4 + [(11008, 4096)] * 2 + [(4096, 11008)]) * 32, k=1024,
                                s=64, kind="student", seed=1, steps=20),
}
C5_SHAPE = (4096, 11008)
C5_PAIRS = [(256, 16), (1024, 16), (1024, 64), (4096, 16), (4096, 64), (4096, 256), (16384, 16), (16384, 64),
            (16384, 256)]

ADAM = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8)


def planted_support(d, s, seed):
    """s distinct positions in [0, d) (ascending) and a +-1 sign for each."""
    rng = np.random.Generator(np.random.PCG64(int(seed)))
    if d <= 1 << 20:
        idx = rng.choice(d, size=s, replace=False)
    else:
        idx = np.unique(rng.integers(0, d, size=4 * s + 16))
        rng.shuffle(idx)
        idx = idx[:s]
    idx = np.sort(idx).astype(np.uint32)
    sign = np.where(rng.random(s) < 0.5, -1.0, 1.0).astype(np.float32)
    return idx, sign


def gradient(d, kind, support, sign, seed):
    """One float32 gradient of length d for the given planted support; seed names the step."""
    rng = np.random.Generator(np.random.PCG64(int(seed)))
    if kind == "gauss":
        g = rng.standard_normal(d, dtype=np.float32) * np.float32(0.1)
        mag = rng.uniform(1.0, 2.0, size=support.size)
    elif kind == "student":
        g = (rng.standard_t(3.0, size=d) * 1e-3).astype(np.float32)
        mag = rng.uniform(0.5, 1.0, size=support.size)
    elif kind == "zero":
        g = np.zeros(d, dtype=np.float32)
        mag = rng.uniform(0.5, 1.0, size=support.size)
    else:
        raise ValueError(kind)
    g[support] = (sign * mag).astype(np.float32)
    return g


def weights(d, seed):
    """Random-init weights N(0, 0.02^2), float32."""
    rng = np.random.Generator(np.random.PCG64(int(seed)))
    return rng.standard_normal(d, dtype=np.float32) * np.float32(0.02)


def support_seed(cfg_id, matrix_id):
    return 1000 * cfg_id + matrix_id


def step_seed(cfg_id, matrix_id, step):
    return 1_000_000 * cfg_id + 1000 * matrix_id + step


def gradient_on_device(out, support, sign, seed, chunk=1 << 24):
    """Fills the float32 CUDA tensor `out` with a "student" gradient drawn on the device (torch's generator): the same law
    as gradient(kind="student") -- 1e-3 * Student-t(3) noise, planted entries sign * U(0.5, 1) at `support` (CUDA int64
    tensor) -- but not the same numbers.  For workloads too large to draw on the host (the whole-model configurations);
    nothing that is compared with the oracle uses it."""
    import torch
    gen = torch.Generator(device=out.device)
    gen.manual_seed(int(seed))
    d = out.numel()
    for lo in range(0, d, chunk):
        n = min(chunk, d - lo)
        z = torch.randn(4, n, device=out.device, generator=gen)
        chi = (z[1] * z[1] + z[2] * z[2] + z[3] * z[3]) * (1.0 / 3.0)          # chi^2_3 / 3
        out[lo:lo + n] = z[0] * torch.rsqrt(chi) * 1e-3
    mag = torch.rand(support.numel(), device=out.device, generator=gen) * 0.5 + 0.5
    out[support] = sign * mag
    return out
