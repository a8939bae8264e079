"""Seeded synthetic activation sets (input generators only: none of the method's arithmetic).

The paper evaluates on activations of ResNet-20 (CIFAR), ResNet-18 / ResNet-50 /
MobileNetV2 (ImageNet) produced from generator-synthesised images (Section 5.1).
Neither the datasets, the trained networks nor the image generator are available,
so these tensors stand in for them: same NCHW shapes, same value structure
(post-ReLU half-normal, ReLU6 saturation, dead channels, outlier channels, heavy
tails), per-channel spread drawn from a log-normal law.  Everything is a pure
function of (config, tensor index, batch block), so any slice of the batch can be
regenerated independently and the same bytes feed the CPU oracle and the GPU.

Random streams are numpy Philox generators keyed by SeedSequence([seed, stream, block]).
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, replace
from typing import List, Tuple

import numpy as np

_STREAM_SIGMA, _STREAM_FLAGS, _STREAM_X, _STREAM_GY = 1, 2, 3, 4
_BLOCK = 8  # samples generated per random stream


@dataclass(frozen=True)
class TensorSpec:
    config: int                 # 1..5, the workload family
    index: int                  # position inside the family
    shape: Tuple[int, int, int, int]   # N, C, H, W
    dist: str                   # "relu" | "relu6" | "student_t3"
    sigma_log_std: float        # per-channel sigma ~ LogNormal(0, sigma_log_std)
    dead_frac: float = 0.0      # fraction of channels that are all-zero
    outlier_frac: float = 0.0   # fraction of channels whose sigma is multiplied by 20
    bits: Tuple[int, ...] = (4,)
    dtypes: Tuple[str, ...] = ("f32",)

    @property
    def seed(self) -> int:
        return 0 if self.config == 1 else 1000 * self.config + self.index

    @property
    def numel(self) -> int:
        n, c, h, w = self.shape
        return n * c * h * w

    def with_batch(self, n: int) -> "TensorSpec":
        """Same tensor law at another batch size (small cases for the slow CPU oracle)."""
        return replace(self, shape=(n,) + tuple(self.shape[1:]))

    @property
    def name(self) -> str:
        return f"cfg{self.config}.{self.index}[{','.join(map(str, self.shape))}]"


def config_tensors(config: int) -> List[TensorSpec]:
    """The tensor list of one of the five workload families."""
    if config == 1:   # ResNet-20 first-layer activation
        return [TensorSpec(1, 0, (16, 16, 32, 32), "relu", 0.5, bits=(3,))]
    if config == 2:   # ResNet-20 CIFAR activation set: stem + 3 stages x 3 blocks x 2 convs
        shapes = [(256, 16, 32, 32)] * 7 + [(256, 32, 16, 16)] * 6 + [(256, 64, 8, 8)] * 6
        return [TensorSpec(2, i, s, "relu", 0.7, dead_frac=0.05, bits=(3, 4)) for i, s in enumerate(shapes)]
    if config == 3:   # ResNet-18 ImageNet-shaped
        shapes = [(128, 64, 112, 112), (128, 64, 56, 56), (128, 128, 28, 28), (128, 256, 14, 14), (128, 512, 7, 7)]
        return [TensorSpec(3, i, s, "relu", 1.0, bits=(4, 5)) for i, s in enumerate(shapes)]
    if config == 4:   # MobileNetV2 ImageNet-shaped
        shapes = [(128, 32, 112, 112), (128, 96, 112, 112), (128, 144, 56, 56), (128, 192, 28, 28),
                  (128, 384, 14, 14), (128, 960, 7, 7), (128, 1280, 7, 7)]
        return [TensorSpec(4, i, s, "relu6", 1.0, outlier_frac=0.02, bits=(4, 5)) for i, s in enumerate(shapes)]
    if config == 5:   # bandwidth sweep, ResNet-50-shaped
        shapes = [(256, 256, 56, 56), (256, 512, 28, 28), (256, 1024, 14, 14), (256, 2048, 7, 7)]
        return [TensorSpec(5, i, s, "student_t3", 1.0, bits=(2, 3, 4, 5, 6, 7, 8), dtypes=("f32", "bf16"))
                for i, s in enumerate(shapes)]
    raise ValueError("config must be 1..5")


def _rng(seed: int, stream: int, block: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(np.random.SeedSequence([seed, stream, block])))


def channel_sigma(spec: TensorSpec) -> np.ndarray:
    """Per-channel spread (float32 [C]); dead channels get 0, outlier channels x20."""
    c = spec.shape[1]
    sigma = np.exp(spec.sigma_log_std * _rng(spec.seed, _STREAM_SIGMA).standard_normal(c)).astype(np.float32)
    u = _rng(spec.seed, _STREAM_FLAGS).random(c)
    if spec.outlier_frac > 0:
        sigma = np.where(u < spec.outlier_frac, sigma * np.float32(20), sigma).astype(np.float32)
    if spec.dead_frac > 0:
        sigma = np.where(u > 1.0 - spec.dead_frac, np.float32(0), sigma).astype(np.float32)
    return sigma


def _fill_block(spec: TensorSpec, sigma: np.ndarray, out: np.ndarray, b: int, block_offset: int = 0) -> None:
    n0 = b * _BLOCK
    n1 = min(n0 + _BLOCK, spec.shape[0])
    shp = (n1 - n0,) + tuple(spec.shape[1:])
    g = _rng(spec.seed, _STREAM_X, b + block_offset)
    v = g.standard_normal(shp, dtype=np.float32)
    if spec.dist == "student_t3":
        q = np.square(g.standard_normal(shp, dtype=np.float32))
        q += np.square(g.standard_normal(shp, dtype=np.float32))
        q += np.square(g.standard_normal(shp, dtype=np.float32))
        np.maximum(q, np.float32(1e-12), out=q)
        v /= np.sqrt(q * np.float32(1.0 / 3.0))
    v *= sigma.reshape(1, -1, 1, 1)
    if spec.dist in ("relu", "relu6"):
        np.maximum(v, np.float32(0), out=v)
    if spec.dist == "relu6":
        np.minimum(v, np.float32(6), out=v)
    v += np.float32(0)          # no negative zeros
    out[n0:n1] = v


def _parallel_blocks(n: int, fn, threads: int) -> None:
    nb = (n + _BLOCK - 1) // _BLOCK
    if threads <= 1 or nb == 1:
        for b in range(nb):
            fn(b)
    else:
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(fn, range(nb)))


def make_activation(spec: TensorSpec, out: np.ndarray | None = None, threads: int = 8,
                    block_offset: int = 0) -> np.ndarray:
    """float32 NCHW activation tensor of the spec (finite, no -0).  `block_offset` shifts the
    random streams, giving another batch of the same law (one per data-parallel replica)."""
    if out is None:
        out = np.empty(spec.shape, np.float32)
    sigma = channel_sigma(spec)
    _parallel_blocks(spec.shape[0], lambda b: _fill_block(spec, sigma, out, b, block_offset), threads)
    return out


def make_upstream_grad(spec: TensorSpec, out: np.ndarray | None = None, threads: int = 8,
                       block_offset: int = 0) -> np.ndarray:
    """float32 upstream gradient ~ N(0, 1) of the same shape."""
    if out is None:
        out = np.empty(spec.shape, np.float32)

    def fill(b):
        n0 = b * _BLOCK
        n1 = min(n0 + _BLOCK, spec.shape[0])
        out[n0:n1] = _rng(spec.seed, _STREAM_GY, b + block_offset).standard_normal((n1 - n0,) + tuple(spec.shape[1:]),
                                                                    dtype=np.float32)
    _parallel_blocks(spec.shape[0], fill, threads)
    return out


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round-to-nearest-even; input preparation only."""
    u = np.ascontiguousarray(a, np.float32).view(np.uint32)
    r = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float32, exact."""
    return (np.ascontiguousarray(h, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# ---------------------------------------------------------------------------------------
# Weight tensors (Section 5.1: channel-wise quantization of all weights).  Shapes of the
# convolution and classifier weights of ResNet-20 (CIFAR) and ResNet-18 (ImageNet); values
# He-normal with a per-output-channel log-normal spread (trained weights are not available).
# ---------------------------------------------------------------------------------------
_STREAM_W, _STREAM_GW = 5, 6


def weight_shapes(net: str) -> List[Tuple[int, ...]]:
    """[C_out, C_in, k, k] (or [C_out, C_in]) of every quantized weight tensor of the network."""
    if net == "resnet20":
        shapes = [(16, 3, 3, 3)]
        cin = 16
        for cout in (16, 32, 64):
            for blk in range(3):
                shapes += [(cout, cin, 3, 3), (cout, cout, 3, 3)]
                if blk == 0 and cin != cout:
                    shapes.append((cout, cin, 1, 1))
                cin = cout
        return shapes + [(100, 64)]
    if net == "resnet18":
        shapes = [(64, 3, 7, 7)]
        cin = 64
        for cout in (64, 128, 256, 512):
            for blk in range(2):
                shapes += [(cout, cin, 3, 3), (cout, cout, 3, 3)]
                if blk == 0 and cin != cout:
                    shapes.append((cout, cin, 1, 1))
                cin = cout
        return shapes + [(1000, 512)]
    raise ValueError(net)


def make_weights(net: str, seed: int = 7000, grads: bool = False) -> List[np.ndarray]:
    """fp32 weight tensors (or their upstream gradients ~ N(0, 1e-2)) of `net`, seeded per tensor."""
    out = []
    for i, shape in enumerate(weight_shapes(net)):
        fan_in = int(np.prod(shape[1:]))
        if grads:
            w = _rng(seed, _STREAM_GW, i).standard_normal(shape) * 0.1
        else:
            spread = np.exp(0.5 * _rng(seed, _STREAM_SIGMA, i).standard_normal((shape[0],) + (1,) * (len(shape) - 1)))
            w = _rng(seed, _STREAM_W, i).standard_normal(shape) * np.sqrt(2.0 / fan_in) * spread
        out.append((w.astype(np.float32) + np.float32(0)))
    return out
