"""Seeded synthetic inputs for the tests and the benchmark.

This module only draws random tensors and lists tensor shapes.  It contains none of the
optimizer's or the quantizer's arithmetic, so that the CUDA path and the CPU checker can
both be fed the same bytes from here without sharing any code of the method.

The paper trains ResNet / DF-ResNet speaker-embedding extractors on a speech corpus
(Section V) that is not available; the shapes below follow its layer tables (3x3 / 1x1
convolutions of 32-256 channels, batch-norm vectors, a 256-d embedding layer and a
5,994-speaker classifier) and the value distributions are stand-ins for trained weights
and real gradients.
"""
from __future__ import annotations

import math
from typing import List, Sequence, Tuple

import torch

Shape = Tuple[int, ...]


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def normal(n, std: float, seed: int, device="cpu", dtype=torch.float32) -> torch.Tensor:
    """N(0, std) of n elements, drawn in fp32 then cast."""
    x = torch.randn(n, generator=_gen(seed, device), device=device, dtype=torch.float32) * std
    return x.to(dtype)


def student_t(n, nu: int, scale: float, seed: int, device="cpu") -> torch.Tensor:
    """scale * Student-t(nu): a normal over the root of a scaled chi-square (heavy tails)."""
    g = _gen(seed, device)
    z = torch.randn(n, generator=g, device=device, dtype=torch.float32)
    chi2 = torch.zeros(n, device=device, dtype=torch.float32)
    for _ in range(nu):
        chi2 += torch.randn(n, generator=g, device=device, dtype=torch.float32) ** 2
    return z / torch.sqrt(chi2 / nu) * scale


def laplace_outliers(n, seed: int, frac: float = 1e-3, gain: float = 100.0, device="cpu") -> torch.Tensor:
    """Laplace(0,1) samples with a random `frac` of them multiplied by `gain`."""
    g = _gen(seed, device)
    u = torch.rand(n, generator=g, device=device, dtype=torch.float32) - 0.5
    x = -torch.sign(u) * torch.log1p(-2.0 * u.abs().clamp(max=0.4999999))
    pick = torch.rand(n, generator=g, device=device, dtype=torch.float32) < frac
    return torch.where(pick, x * gain, x)


# ---------------------------------------------------------------------------------------
# Shape manifests
# ---------------------------------------------------------------------------------------
def conv3x3_shapes() -> List[Shape]:
    """37 conv3x3 weight tensors of 32/64/128/256 channels, 6,561,792 elements in total."""
    out: List[Shape] = []
    for ch, count in ((32, 8), (64, 8), (128, 14), (256, 7)):
        out += [(ch, ch, 3, 3)] * count
    return out


def resnet_speaker_manifest() -> List[Tuple[str, Shape, str]]:
    """(name, shape, kind) for ~200 tensors of a deep bottleneck ResNet speaker extractor.

    kind is one of 'conv', 'fc', 'bn_weight', 'bias' and selects the initialisation.
    Stem conv + BN, 20 bottleneck blocks over widths 32/64/128/256 (3/4/10/3 blocks; each
    1x1, 3x3, 1x1 conv with a BN after every conv), a 1x1 shortcut conv + BN where the
    width changes, a 256-d embedding layer with bias and BN, and a 5,994-way classifier.
    """
    m: List[Tuple[str, Shape, str]] = []

    def bn(prefix: str, c: int):
        m.append((prefix + ".bn.weight", (c,), "bn_weight"))
        m.append((prefix + ".bn.bias", (c,), "bias"))

    m.append(("stem.conv", (32, 1, 3, 3), "conv"))
    bn("stem", 32)
    prev = 32
    for stage, (width, blocks) in enumerate(((32, 3), (64, 4), (128, 10), (256, 3))):
        for b in range(blocks):
            cin = prev if b == 0 else width
            p = f"stage{stage}.block{b}"
            m.append((p + ".conv1", (width, cin, 1, 1), "conv"))
            bn(p + ".conv1", width)
            m.append((p + ".conv2", (width, width, 3, 3), "conv"))
            bn(p + ".conv2", width)
            m.append((p + ".conv3", (width, width, 1, 1), "conv"))
            bn(p + ".conv3", width)
            if b == 0 and cin != width:
                m.append((p + ".shortcut", (width, cin, 1, 1), "conv"))
                bn(p + ".shortcut", width)
        prev = width
    m.append(("embed.fc.weight", (256, 5120), "fc"))
    m.append(("embed.fc.bias", (256,), "bias"))
    bn("embed", 256)
    m.append(("classifier.weight", (5994, 256), "fc"))
    return m


def numel(shape: Sequence[int]) -> int:
    return int(math.prod(shape))


def init_param(shape: Shape, kind: str, seed: int, device="cpu") -> torch.Tensor:
    """He-normal for conv / fc weights, ones for BN weights, zeros for biases (flat fp32)."""
    n = numel(shape)
    if kind == "bn_weight":
        return torch.ones(n, device=device, dtype=torch.float32)
    if kind == "bias":
        return torch.zeros(n, device=device, dtype=torch.float32)
    fan_in = numel(shape[1:])
    return normal(n, math.sqrt(2.0 / fan_in), seed, device)


# ---------------------------------------------------------------------------------------
# Workloads (one function per configuration)
# ---------------------------------------------------------------------------------------
ADAM_FLAT_SMALL = dict(n=1 << 20, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0,
                       block_size=2048, seed=0)
SGD_CONV = dict(lr=0.1, momentum=0.9, weight_decay=1e-4, block_size=2048, steps=100, seed=1)
ADAM_RESNET = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.05, block_size=2048,
                   steps=100, seed=2)
QUANT_SWEEP = dict(sizes=(1 << 20, 1 << 24, 1 << 27), block_sizes=(256, 2048, 4096), seed=3)
ADAM_FLAT_LARGE = dict(n=1 << 28, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01,
                       block_size=2048, prewarm_steps=10, seed=4)


def flat_adam_inputs(n: int, seed: int, device="cpu"):
    """w ~ N(0, 0.02), g ~ N(0, 1e-3), both fp32 and flat."""
    return normal(n, 0.02, seed * 1000 + 1, device), normal(n, 1e-3, seed * 1000 + 2, device)


def fresh_grad(n: int, seed: int, step: int, device="cpu", dtype=torch.float32) -> torch.Tensor:
    """g ~ N(0, 1e-3) for a given step of a multi-step run."""
    return normal(n, 1e-3, seed * 1000 + 100 + step, device, dtype)


def conv_sgd_params(seed: int, device="cpu") -> List[torch.Tensor]:
    return [init_param(s, "conv", seed * 1000 + i, device) for i, s in enumerate(conv3x3_shapes())]


def conv_sgd_grads(seed: int, step: int, device="cpu") -> List[torch.Tensor]:
    """1e-3 * Student-t(3) gradients, one flat fp32 tensor per conv weight."""
    return [student_t(numel(s), 3, 1e-3, seed * 100000 + step * 100 + i, device)
            for i, s in enumerate(conv3x3_shapes())]


def resnet_adam_params(seed: int, device="cpu") -> List[torch.Tensor]:
    return [init_param(s, kind, seed * 1000 + i, device)
            for i, (_, s, kind) in enumerate(resnet_speaker_manifest())]


def resnet_adam_grads(seed: int, step: int, device="cpu") -> List[torch.Tensor]:
    """N(0, 1e-3) gradients rounded to bf16, one flat tensor per manifest entry."""
    return [normal(numel(s), 1e-3, seed * 1000000 + step * 1000 + i, device, torch.bfloat16)
            for i, (_, s, _) in enumerate(resnet_speaker_manifest())]
