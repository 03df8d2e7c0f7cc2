"""Seeded synthetic gradients shaped like the paper's workloads.

This module only draws random numbers and lists tensor shapes.  It holds none
of the compression arithmetic, so both the CPU oracle's tests and the CUDA
path's tests may import it without sharing any part of the method.

The paper trains on MNIST, CIFAR10, ImageNet, BN50 and Shakespeare (Table 1);
none of those gradients can be had offline, so every workload here is a
stand-in: the layer *shapes* follow the networks the paper lists (Section
"Methodology" and Table 1) and the values are seeded noise.

Recipe (all indices 0-based)::

    rng   = default_rng(SeedSequence([1712, 2679, cfg, learner, tensor, step]))
    sigma = 10 ** default_rng(SeedSequence([1712, 2679, cfg, 999, tensor])).uniform(-4, -2)
    gaussian:     dW = rng.normal(0, sigma, n).astype(float32)
    heavy-tailed: g = rng.normal(0, sigma, n); mask = rng.random(n) < 0.01
                  lap = rng.laplace(0, 10*sigma, n); dW = where(mask, lap, g).astype(float32)
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List

import numpy as np

_SEED_PREFIX = (1712, 2679)


@dataclass(frozen=True)
class TensorSpec:
    """One layer's gradient: a flat fp32 vector with its own bin length."""

    name: str
    n: int
    L_T: int
    kind: str  # "conv", "bn", "fc"


def rng_for(cfg: int, learner: int, tensor: int, step: int) -> np.random.Generator:
    return np.random.default_rng(
        np.random.SeedSequence([*_SEED_PREFIX, cfg, learner, tensor, step]))


def sigma_for(cfg: int, tensor: int) -> float:
    """Per-tensor standard deviation, log-uniform in [1e-4, 1e-2]."""
    r = np.random.default_rng(np.random.SeedSequence([*_SEED_PREFIX, cfg, 999, tensor]))
    return float(10.0 ** r.uniform(-4.0, -2.0))


def gaussian_dw(n: int, sigma: float, rng: np.random.Generator) -> np.ndarray:
    return rng.normal(0.0, sigma, n).astype(np.float32)


def heavy_dw(n: int, sigma: float, rng: np.random.Generator) -> np.ndarray:
    """Gaussian body with 1 % of the entries replaced by Laplace(0, 10*sigma)."""
    g = rng.normal(0.0, sigma, n)
    mask = rng.random(n) < 0.01
    lap = rng.laplace(0.0, 10.0 * sigma, n)
    return np.where(mask, lap, g).astype(np.float32)


# ----------------------------------------------------------------------------
# Workload shape lists
# ----------------------------------------------------------------------------

def config1_tensors() -> List[TensorSpec]:
    """One 784x128 fully connected layer, bin length 50 (ragged tail of 2)."""
    return [TensorSpec("fc_784x128", 784 * 128, 50, "fc")]


def config2_tensors() -> List[TensorSpec]:
    """Small conv net: six 3x3 conv weights and two FC weights."""
    conv = [(32, 3), (32, 32), (64, 32), (64, 64), (128, 64), (128, 128)]
    out = [TensorSpec(f"conv{i}_{o}x{c}x3x3", o * c * 9, 500, "conv")
           for i, (o, c) in enumerate(conv)]
    out.append(TensorSpec("fc_2048x512", 2048 * 512, 50, "fc"))
    out.append(TensorSpec("fc_512x10", 512 * 10, 50, "fc"))
    return out


def resnet50_tensors(lt_conv: int = 500, lt_fc: int = 50) -> List[TensorSpec]:
    """The 161 weight and bias tensors of a ResNet-50 in definition order.

    Stem conv 64x3x7x7; four stages of widths 64/128/256/512 with 3/4/6/3
    bottleneck blocks of [1x1 w<-in, 3x3 w<-w, 1x1 4w<-w]; a 1x1 projection
    4w<-in in each stage's first block; every conv is followed by a batch-norm
    weight and bias; a final 1000x2048 FC with bias.  Batch-norm tensors take
    the conv bin length, the FC bias takes the FC one.
    """
    out: List[TensorSpec] = []

    def conv_bn(tag: str, o: int, c: int, k: int) -> None:
        out.append(TensorSpec(f"{tag}.conv_{o}x{c}x{k}x{k}", o * c * k * k, lt_conv, "conv"))
        out.append(TensorSpec(f"{tag}.bn_w_{o}", o, lt_conv, "bn"))
        out.append(TensorSpec(f"{tag}.bn_b_{o}", o, lt_conv, "bn"))

    conv_bn("stem", 64, 3, 7)
    inp = 64
    for s, (w, blocks) in enumerate(zip((64, 128, 256, 512), (3, 4, 6, 3))):
        for b in range(blocks):
            tag = f"s{s}b{b}"
            conv_bn(tag + ".a", w, inp, 1)
            conv_bn(tag + ".b", w, w, 3)
            conv_bn(tag + ".c", 4 * w, w, 1)
            if b == 0:
                conv_bn(tag + ".proj", 4 * w, inp, 1)
            inp = 4 * w
    out.append(TensorSpec("fc_w_1000x2048", 1000 * 2048, lt_fc, "fc"))
    out.append(TensorSpec("fc_b_1000", 1000, lt_fc, "fc"))
    return out


def config4_tensors(hidden: int = 2048) -> List[TensorSpec]:
    """Speech-style FC DNN: 440 -> 6 hidden layers -> 9300 outputs, weights only."""
    dims = [440] + [hidden] * 6 + [9300]
    return [TensorSpec(f"fc{i}_{dims[i]}x{dims[i + 1]}", dims[i] * dims[i + 1], 50, "fc")
            for i in range(len(dims) - 1)]


def lstm_tensors(vocab: int = 67, hidden: int = 512) -> List[TensorSpec]:
    """Character-level LSTM of the paper's model list: two LSTM layers (67 -> 512, 512 -> 512) and a fully
    connected layer (512 -> 67).  The paper names the layers by their input and output widths; the tensors
    here are the gate-stacked matrices a framework keeps for them (input-to-hidden and hidden-to-hidden
    weights of four gates, their biases) and the output layer with its bias, all with the bin length the
    paper uses for LSTM and fully connected layers."""
    out = []
    for i, width in enumerate((vocab, hidden)):
        out += [TensorSpec(f"lstm{i}_w_ih_{4 * hidden}x{width}", 4 * hidden * width, 500, "lstm"),
                TensorSpec(f"lstm{i}_w_hh_{4 * hidden}x{hidden}", 4 * hidden * hidden, 500, "lstm"),
                TensorSpec(f"lstm{i}_b_ih", 4 * hidden, 500, "lstm"),
                TensorSpec(f"lstm{i}_b_hh", 4 * hidden, 500, "lstm")]
    out += [TensorSpec(f"fc_{vocab}x{hidden}", vocab * hidden, 500, "fc"), TensorSpec("fc_bias", vocab, 500, "fc")]
    return out


def config5_sizes() -> List[int]:
    """Flat gradient sizes of the bandwidth sweep: 2^20 ... 2^30 in 4x steps."""
    return [1 << (20 + 2 * j) for j in range(6)]


def make_dw(cfg: int, learner: int, tensor: int, step: int, n: int,
            heavy: bool, sigma: float | None = None) -> np.ndarray:
    """dW of one tensor at one step for one learner, per the recipe above."""
    if sigma is None:
        sigma = sigma_for(cfg, tensor)
    rng = rng_for(cfg, learner, tensor, step)
    return heavy_dw(n, sigma, rng) if heavy else gaussian_dw(n, sigma, rng)
