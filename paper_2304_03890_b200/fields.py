"""Seeded synthetic inputs shaped like the paper's workloads (Table IV: RTM, Hurricane, CESM-ATM fields;
message sizes of tens to hundreds of MB) and like a ResNet-50 gradient vector (Sec. I).

This module only makes input data.  It contains none of the compressor's or the collectives' arithmetic,
so both the CUDA library and the test oracle may be fed from it.  Everything is built with torch ops so the
same recipe runs on the CPU (small test sizes) and on the GPU (full benchmark sizes); a given (seed, device
type) always yields the same bytes.
"""
import math

import torch

BASE_SEED = 230403890
BLOCK_LEN = 128


def seed_for(config: int, rank: int = 0) -> int:
    return BASE_SEED + 1000 * config + rank


def _gen(seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def sines_1d(n, seed, device="cpu"):
    """Smooth 1-D signal: four unit-amplitude sines, frequencies U[1,50] cycles over the buffer, phases
    U[0,2pi), plus N(0, 1e-3) noise; built in fp64 and rounded to fp32."""
    g = _gen(seed, device)
    f = 1.0 + 49.0 * torch.rand(4, generator=g, device=device, dtype=torch.float64)
    ph = 2.0 * math.pi * torch.rand(4, generator=g, device=device, dtype=torch.float64)
    t = torch.arange(n, device=device, dtype=torch.float64) / max(n, 1)
    x = torch.zeros(n, device=device, dtype=torch.float64)
    for k in range(4):
        x += torch.sin(2.0 * math.pi * f[k] * t + ph[k])
    x += 1e-3 * torch.randn(n, generator=g, device=device, dtype=torch.float64)
    return x.to(torch.float32)


def smooth_field(shape, sigma, lo, hi, seed, device="cpu"):
    """Gaussian random field: white N(0,1) noise blurred by a periodic Gaussian of `sigma` cells per axis
    (applied in Fourier space), then scaled affinely so that its extremes are exactly lo and hi.
    Returned flattened, C order (last axis fastest): the compressor sees fields as 1-D."""
    g = _gen(seed, device)
    w = torch.randn(*shape, generator=g, device=device, dtype=torch.float32)
    spec = torch.fft.rfftn(w)
    del w
    nd = len(shape)
    for ax, size in enumerate(shape):
        fr = torch.fft.rfftfreq(size, device=device) if ax == nd - 1 else torch.fft.fftfreq(size, device=device)
        tf = torch.exp(-2.0 * (math.pi * sigma) ** 2 * fr.to(torch.float32) ** 2)
        view = [1] * nd
        view[ax] = tf.numel()
        spec *= tf.view(view)
    x = torch.fft.irfftn(spec, s=shape)
    del spec
    mn, mx = x.min(), x.max()
    x = (x - mn) / (mx - mn)
    x = torch.clamp(lo + x * (hi - lo), min=lo, max=hi)
    return x.reshape(-1).contiguous()


def force_constant_blocks(x, frac, seed, block_len=BLOCK_LEN):
    """Overwrites each whole block, independently with probability `frac`, by the block's first value."""
    n = x.numel()
    nb = n // block_len
    if nb == 0:
        return x
    g = _gen(seed, x.device)
    pick = torch.rand(nb, generator=g, device=x.device) < frac
    v = x[: nb * block_len].view(nb, block_len)
    v[pick] = v[pick][:, :1].expand(-1, block_len).clone()
    return x


def laplace_gradients(n, scale, zero_frac, seed, device="cpu"):
    """Gradient-like vector: Laplace(0, scale) by inverse CDF, each entry set to exactly 0 with
    probability zero_frac."""
    g = _gen(seed, device)
    u = torch.rand(n, generator=g, device=device, dtype=torch.float32) - 0.5
    x = -scale * torch.sign(u) * torch.log1p(-2.0 * u.abs().clamp(max=0.4999999))
    z = torch.rand(n, generator=g, device=device, dtype=torch.float32) < zero_frac
    x[z] = 0.0
    return x.contiguous()


def eb_from_range(x, rel):
    """Absolute bound from a relative one: fp32( rel * (max - min) ), the difference taken in fp64."""
    rng = float(x.max().double() - x.min().double())
    return float(torch.tensor(rel * rng, dtype=torch.float64).to(torch.float32))


# ---------------------------------------------------------------------------------------------------------
# The five benchmark configurations.  `shrink` divides every axis (or the length) so that the CPU tests can
# run the same recipes at a size the oracle finishes in seconds.
# ---------------------------------------------------------------------------------------------------------

def config1(device="cpu", n=1 << 20):
    x = sines_1d(n, seed_for(1), device)
    return {"x": x, "eb": eb_from_range(x, 1e-3), "block_len": BLOCK_LEN}


def config2(device="cpu", shape=(512, 512, 256), sigma=8.0):
    x = smooth_field(shape, sigma, -100.0, 100.0, seed_for(2), device)
    x = force_constant_blocks(x, 0.2, seed_for(2, 1))
    return {"x": x, "eb": eb_from_range(x, 1e-4), "block_len": BLOCK_LEN}


def config3(device="cpu", P=8, shape=(256, 256, 256), sigma=4.0):
    xs = torch.stack([smooth_field(shape, sigma, -1.0, 1.0, seed_for(3, r), device) for r in range(P)])
    return {"x": xs, "eb": 1e-4, "block_len": BLOCK_LEN, "P": P}


def config4(device="cpu", P=32, shape=(1024, 512, 512), sigma=6.0):
    x = smooth_field(shape, sigma, 0.0, 1000.0, seed_for(4), device)
    return {"x": x, "eb": eb_from_range(x, 1e-3), "block_len": BLOCK_LEN, "P": P}


def config5(device="cpu", P=16, n=25557032):
    xs = torch.stack([laplace_gradients(n, 1e-3, 0.05, seed_for(5, r), device) for r in range(P)])
    return {"x": xs, "eb": 1e-5, "block_len": BLOCK_LEN, "P": P}
