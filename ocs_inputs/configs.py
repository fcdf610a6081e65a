"""The five synthetic workloads (shapes, value distributions, seeds).

They stand in for the paper's ImageNet CNNs (Section 5) and WikiText-2 LSTM (Section 6),
whose data and trained weights are not available: only shapes, sizes and value
distributions are reproduced.  This module builds input arrays and layer lists; it
performs no splitting, clipping or quantization.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import prng


# --------------------------------------------------------------------------- config 1
def config1(seed: int = 0):
    """One fully-connected layer: W [256, 512] Laplace(0, 0.02) + 8 outliers at +-(10..20) std;
    activations [64, 512] half-normal."""
    O, C, M = 256, 512, 64
    b = 0.02
    W = prng.laplace(seed, 0, (O, C), b)
    std = b * np.sqrt(2.0)
    pos = prng.distinct_positions(seed, 1, O * C, 8)
    mag = 10.0 + 10.0 * prng.Stream(seed, 4).uniform(0, 8)
    sg = prng.signs(seed, 3, 8)
    W.reshape(-1)[pos] = (sg * mag * std).astype(np.float32)
    A = prng.normal(seed, 4, (M, C), absolute=True)
    return dict(name="fc_256x512", W=W, A=A, ratio=0.05, w_bits=8, a_bits=8, a_signed=0,
                clip="none", seed=seed)


# --------------------------------------------------------------------------- config 2
def config2(seed: int = 1, batch: int = 32):
    """One 3x3 stride-1 pad-1 conv, 256 -> 256 channels on 14x14 maps; heavy-tailed weights."""
    O, C, k, H = 256, 256, 3, 14
    fan_in = C * k * k
    # Student-t(3) has variance 3; rescale to the Kaiming std sqrt(2 / fan_in)
    W = prng.student_t3(seed, 0, (O, C, k, k), np.sqrt(2.0 / fan_in) / np.sqrt(3.0))
    X = prng.normal(seed, 8, (batch, C, H, H), absolute=True)   # NCHW
    return dict(name="conv3x3_256_14", W=W, X=X, stride=1, pad=1, ratio=0.02, w_bits=6,
                a_bits=8, a_signed=0, clip="mse", n_candidates=128, seed=seed)


# --------------------------------------------------------------------------- config 3
CONFIG3_RATIOS = (0.0, 0.01, 0.02, 0.05, 0.1)
CONFIG3_BITS = (4, 5, 6, 8)


def config3(seed: int = 2, O: int = 4096, C: int = 25088, M: int = 128):
    """fc6-shaped layer: W [4096, 25088] Laplace(0, 0.005), 0.01 % of entries set to +-15 std
    (one common magnitude, random sign); activations [128, 25088] half-normal.  O, C, M can be
    reduced to get a same-recipe case the CPU checker finishes quickly."""
    b = 0.005
    W = prng.laplace(seed, 0, (O, C), b)
    n_out = int(round(1e-4 * O * C))
    pos = prng.distinct_positions(seed, 1, O * C, n_out)
    sg = prng.signs(seed, 2, n_out)
    W.reshape(-1)[pos] = (sg * (15.0 * b * np.sqrt(2.0))).astype(np.float32)
    A = prng.normal(seed, 4, (M, C), absolute=True)
    return dict(name=f"fc6_{O}x{C}", W=W, A=A, ratios=CONFIG3_RATIOS, bits=CONFIG3_BITS,
                a_bits=8, a_signed=0, clip="mse", n_candidates=128, seed=seed)


# --------------------------------------------------------------------------- config 4
@dataclass
class ConvSpec:
    name: str
    C: int          # input channels
    O: int          # output channels
    k: int          # square kernel
    stride: int
    pad: int
    H_in: int       # square input map
    relu: bool = True
    residual_from: str | None = None   # name of the tensor added before the ReLU
    input_from: str | None = None      # name of the tensor this layer reads (None: previous)

    @property
    def H_out(self) -> int:
        return (self.H_in + 2 * self.pad - self.k) // self.stride + 1


def resnet50_layers(image: int = 224):
    """The 53 convolutions + 1 fully-connected layer of ResNet-50 (bottleneck blocks 3-4-6-3,
    stride carried by each stage's first 3x3), as (ConvSpec list, fc spec)."""
    layers: list[ConvSpec] = []
    H = image
    layers.append(ConvSpec("conv1", 3, 64, 7, 2, 3, H))
    H = layers[-1].H_out
    H = (H + 2 - 3) // 2 + 1          # 3x3 stride-2 pad-1 max pool
    c_in = 64
    prev_out = "pool"
    for stage, (width, blocks) in enumerate(zip((64, 128, 256, 512), (3, 4, 6, 3)), start=1):
        for blk in range(blocks):
            stride = 2 if (blk == 0 and stage > 1) else 1
            p = f"s{stage}b{blk}"
            block_in = prev_out
            layers.append(ConvSpec(p + ".c1", c_in, width, 1, 1, 0, H, input_from=block_in))
            layers.append(ConvSpec(p + ".c2", width, width, 3, stride, 1, H))
            H2 = layers[-1].H_out
            if blk == 0:
                layers.append(ConvSpec(p + ".ds", c_in, width * 4, 1, stride, 0, H, relu=False,
                                       input_from=block_in))
                res = p + ".ds"
            else:
                res = block_in
            layers.append(ConvSpec(p + ".c3", width, width * 4, 1, 1, 0, H2, relu=True,
                                   residual_from=res, input_from=p + ".c2"))
            H = H2
            c_in = width * 4
            prev_out = p + ".out"
    fc = ConvSpec("fc", 2048, 1000, 1, 1, 0, 1, relu=False)
    return layers, fc


def config4(seed: int = 3, batch: int = 128, image: int = 224):
    """ResNet-50 stack at random init: Kaiming-normal weights, batch norm folded with
    gamma ~ U(0.5, 1.5), beta ~ N(0, 0.1), running mean 0 / variance 1 / eps 1e-5."""
    layers, fc = resnet50_layers(image)
    params = {}
    inv = np.float32(1.0 / np.sqrt(1.0 + 1e-5))
    for i, L in enumerate(layers):
        fan_in = L.C * L.k * L.k
        W = prng.normal(seed, 10 + 4 * i, (L.O, L.C, L.k, L.k), std=np.sqrt(2.0 / fan_in))
        gamma = prng.uniform(seed, 11 + 4 * i, (L.O,), 0.5, 1.5)
        beta = prng.normal(seed, 12 + 4 * i, (L.O,), std=0.1)
        factor = (gamma * inv).astype(np.float32)
        params[L.name] = ((W * factor[:, None, None, None]).astype(np.float32), beta)
    Wfc = prng.normal(seed, 1000, (fc.O, fc.C), std=np.sqrt(2.0 / fc.C))
    params["fc"] = (Wfc.reshape(fc.O, fc.C, 1, 1), np.zeros(fc.O, dtype=np.float32))
    X = prng.normal(seed, 2000, (batch, 3, image, image))
    return dict(name="resnet50", layers=layers, fc=fc, params=params, X=X, ratio=0.01,
                w_bits=8, a_bits=8, clip="none", seed=seed)


# --------------------------------------------------------------------------- config 5
def _with_outliers(seed, stream, W, frac, magnitude):
    n = int(round(frac * W.size))
    pos = prng.distinct_positions(seed, stream, W.size, n)
    sg = prng.signs(seed, stream + 1, n)
    W.reshape(-1)[pos] = (sg * magnitude).astype(np.float32)
    return W


def config5(seed: int = 4, hidden: int = 650, vocab: int = 33278, batch: int = 20, seq: int = 35):
    """Two-layer LSTM language model at random init U(-0.05, 0.05) with 0.05 % weight outliers
    at 10 std; Zipf(1.1) token ids."""
    a = 0.05
    mag = 10.0 * a / np.sqrt(3.0)
    p = {}
    p["emb"] = prng.uniform(seed, 0, (vocab, hidden), -a, a)
    s = 10
    for layer in range(2):
        for nm in ("W_ih", "W_hh"):
            W = prng.uniform(seed, s, (4 * hidden, hidden), -a, a)
            p[f"{nm}{layer}"] = _with_outliers(seed, s + 1, W, 5e-4, mag)
            s += 4
        for nm in ("b_ih", "b_hh"):
            p[f"{nm}{layer}"] = prng.uniform(seed, s, (4 * hidden,), -a, a)
            s += 4
    W = prng.uniform(seed, s, (vocab, hidden), -a, a)
    p["W_dec"] = _with_outliers(seed, s + 1, W, 5e-4, mag)
    p["b_dec"] = prng.uniform(seed, s + 4, (vocab,), -a, a)
    tokens = prng.zipf_tokens(seed, 500, (seq, batch), vocab, 1.1)
    return dict(name="lstm650", params=p, tokens=tokens, hidden=hidden, vocab=vocab,
                ratio=0.02, w_bits=6, a_bits=8, a_signed=1, clip="none", seed=seed)


# --------------------------------------------------------------------------- small generic cases
def random_fc(seed: int, O: int, C: int, M: int, n_outliers: int = 4, scale: float = 0.02):
    """A generic fc-shaped case with a few distinct outliers, for odd-sized parity cases."""
    W = prng.laplace(seed, 0, (O, C), scale)
    n_outliers = min(n_outliers, O * C)
    if n_outliers:
        pos = prng.distinct_positions(seed, 1, O * C, n_outliers)
        mag = 8.0 + 8.0 * prng.Stream(seed, 4).uniform(0, n_outliers)
        W.reshape(-1)[pos] = (prng.signs(seed, 3, n_outliers) * mag * scale).astype(np.float32)
    A = prng.normal(seed, 4, (M, C), absolute=True)
    return W, A


def random_codes(seed: int, stream_id: int, shape, lo: int, hi: int, dtype) -> np.ndarray:
    """Uniform integer codes in [lo, hi]."""
    n = int(np.prod(shape))
    v = prng.Stream(seed, 2 * stream_id).bits(0, n) % np.uint64(hi - lo + 1)
    return (v.astype(np.int64) + lo).astype(dtype).reshape(shape)
