"""Seeded synthetic inputs: parameter layouts and counter-based value generators.

This module holds no update arithmetic.  It only produces the *inputs* both the
CUDA path and the CPU oracle are fed with: the tensor lists of the models the
paper trains (ResNet-20 / ResNet-50 in Section 4.1; ResNet-56 and VGG-16 are
the same families at other depths) and reproducible values for weights and
per-iteration, per-worker gradients.

Every value is a pure function of (seed, stream, iteration, worker, element
index), built from 64-bit integer mixing only, followed by one exact
int -> float32 conversion and one IEEE float32 multiply.  The same torch code
therefore yields the same bytes on a CPU tensor and on a CUDA tensor, and any
single element can be produced without generating its neighbours (used by the
full-size sampled parity tests).

Integer mixer: the SplitMix64 output function (Steele, Lea, Flood, "Fast
splittable pseudorandom number generators", OOPSLA 2014).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Sequence

import torch

SEED = 20201205          # base seed for every workload in this repository
ALIGN_ELEMS = 4          # tensors start on 16-byte boundaries of an fp32 arena

# stream ids: one per kind of buffer
STREAM_WEIGHT = 1
STREAM_GRAD = 2
STREAM_MOM = 3
STREAM_PRE = 4
STREAM_WLOC = 5

_MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB


def _s64(x: int) -> int:
    """Python int (mod 2^64) -> the int64 with the same bit pattern."""
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


def _mix_int(x: int) -> int:
    x &= _MASK64
    x ^= x >> 30
    x = (x * _M1) & _MASK64
    x ^= x >> 27
    x = (x * _M2) & _MASK64
    x ^= x >> 31
    return x


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor (torch's >> is arithmetic)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix_tensor(x: torch.Tensor) -> torch.Tensor:
    x = x ^ _lsr(x, 30)
    x = x * _s64(_M1)
    x = x ^ _lsr(x, 27)
    x = x * _s64(_M2)
    x = x ^ _lsr(x, 31)
    return x


def stream_key(seed: int, stream: int, iteration: int = 0, worker: int = 0) -> int:
    """Scalar key of one buffer: nested mixes of the four identifiers."""
    k = _mix_int(seed)
    k = _mix_int(k + stream * _GOLDEN)
    k = _mix_int(k + iteration * _GOLDEN + 1)
    k = _mix_int(k + worker * _GOLDEN + 2)
    return k


def _hash_at(key: int, idx: torch.Tensor, lane: int, lanes: int) -> torch.Tensor:
    """64 random bits for element index idx (int64 tensor), sub-draw `lane`."""
    ctr = idx * lanes + lane
    return _mix_tensor(ctr * _s64(_GOLDEN) + _s64(key))


def normal_at(key: int, idx: torch.Tensor, sigma: float) -> torch.Tensor:
    """Approximately N(0, sigma^2) float32 deviates at the given element indices.

    Irwin-Hall with 12 terms: the sum of twelve 16-bit uniform integers, centred,
    is converted to float32 exactly (|sum| < 2^24) and scaled by
    float32(sigma) * 2^-16 (one rounding, identical everywhere).
    """
    total = torch.zeros_like(idx)
    for lane in range(3):
        h = _hash_at(key, idx, lane, 3)
        total = total + (h & 0xFFFF) + (_lsr(h, 16) & 0xFFFF) \
            + (_lsr(h, 32) & 0xFFFF) + _lsr(h, 48)
    centred = (total - 6 * 65535).to(torch.float32)
    scale = torch.tensor(float(sigma), dtype=torch.float32, device=idx.device) \
        * torch.tensor(2.0 ** -16, dtype=torch.float32, device=idx.device)
    return centred * scale


def uniform_at(key: int, idx: torch.Tensor) -> torch.Tensor:
    """Uniform float32 on [-1, 1): a 24-bit integer, centred, times 2^-23 (exact)."""
    h = _hash_at(key, idx, 0, 1)
    u = _lsr(h, 40) - (1 << 23)
    return u.to(torch.float32) * (2.0 ** -23)


_CHUNK = 1 << 24


def _fill(fn, n: int, device) -> torch.Tensor:
    out = torch.empty(n, dtype=torch.float32, device=device)
    for lo in range(0, n, _CHUNK):
        hi = min(n, lo + _CHUNK)
        idx = torch.arange(lo, hi, dtype=torch.int64, device=device)
        out[lo:hi] = fn(idx)
    return out


def normal(key: int, n: int, sigma: float, device="cpu") -> torch.Tensor:
    return _fill(lambda idx: normal_at(key, idx, sigma), n, device)


def uniform(key: int, n: int, device="cpu") -> torch.Tensor:
    return _fill(lambda idx: uniform_at(key, idx), n, device)


# --------------------------------------------------------------------------
# parameter layouts
# --------------------------------------------------------------------------

@dataclass
class Layout:
    """Ordered list of trainable tensors packed into one arena.

    `offsets[t]` is the element offset of tensor t; every tensor starts on a
    multiple of ALIGN_ELEMS elements; `padded_numel` is the arena length.
    kinds: "he" (He-normal, sigma = sqrt(2 / fan_in)), "one" (BN gamma),
    "zero" (BN beta, biases).
    """
    name: str
    names: List[str] = field(default_factory=list)
    numels: List[int] = field(default_factory=list)
    kinds: List[str] = field(default_factory=list)
    fan_ins: List[int] = field(default_factory=list)

    def add(self, name: str, numel: int, kind: str, fan_in: int = 0) -> None:
        self.names.append(name)
        self.numels.append(int(numel))
        self.kinds.append(kind)
        self.fan_ins.append(int(fan_in))

    @property
    def num_tensors(self) -> int:
        return len(self.numels)

    @property
    def numel(self) -> int:
        return sum(self.numels)

    @property
    def offsets(self) -> List[int]:
        offs, pos = [], 0
        for n in self.numels:
            offs.append(pos)
            pos += -(-n // ALIGN_ELEMS) * ALIGN_ELEMS
        return offs

    @property
    def padded_numel(self) -> int:
        return sum(-(-n // ALIGN_ELEMS) * ALIGN_ELEMS for n in self.numels)


def _conv_bn(lay: Layout, name: str, cin: int, cout: int, k: int, bias: bool = False,
             bn: bool = True) -> None:
    lay.add(f"{name}.weight", cout * cin * k * k, "he", cin * k * k)
    if bias:
        lay.add(f"{name}.bias", cout, "zero")
    if bn:
        lay.add(f"{name}.bn.gamma", cout, "one")
        lay.add(f"{name}.bn.beta", cout, "zero")


def resnet_cifar(depth: int) -> Layout:
    """ResNet-(6n+2) for CIFAR-10: 3x3 convs at 16/32/64 channels, parameter-free
    shortcuts, BN after every conv, FC 64x10 with bias."""
    assert (depth - 2) % 6 == 0
    n = (depth - 2) // 6
    lay = Layout(f"resnet{depth}_cifar10")
    _conv_bn(lay, "stem", 3, 16, 3)
    cin = 16
    for s, width in enumerate((16, 32, 64)):
        for b in range(n):
            _conv_bn(lay, f"s{s}.b{b}.conv1", cin, width, 3)
            _conv_bn(lay, f"s{s}.b{b}.conv2", width, width, 3)
            cin = width
    lay.add("fc.weight", 64 * 10, "he", 64)
    lay.add("fc.bias", 10, "zero")
    return lay


def resnet50_imagenet() -> Layout:
    """ResNet-50: 7x7 stem, bottleneck stages (3,4,6,3), projection shortcut on the
    first block of each stage, BN after every conv, FC 2048x1000 with bias."""
    lay = Layout("resnet50_imagenet")
    _conv_bn(lay, "stem", 3, 64, 7)
    cin = 64
    for s, (blocks, planes) in enumerate(zip((3, 4, 6, 3), (64, 128, 256, 512))):
        for b in range(blocks):
            p = f"s{s}.b{b}"
            _conv_bn(lay, f"{p}.conv1", cin, planes, 1)
            _conv_bn(lay, f"{p}.conv2", planes, planes, 3)
            _conv_bn(lay, f"{p}.conv3", planes, planes * 4, 1)
            if b == 0:
                _conv_bn(lay, f"{p}.proj", cin, planes * 4, 1)
            cin = planes * 4
    lay.add("fc.weight", 2048 * 1000, "he", 2048)
    lay.add("fc.bias", 1000, "zero")
    return lay


def vgg16_imagenet() -> Layout:
    """VGG-16: thirteen 3x3 convs with biases, FC 25088x4096, 4096x4096, 4096x1000."""
    lay = Layout("vgg16_imagenet")
    cin = 3
    for i, cout in enumerate((64, 64, 128, 128, 256, 256, 256, 512, 512, 512, 512, 512, 512)):
        _conv_bn(lay, f"conv{i}", cin, cout, 3, bias=True, bn=False)
        cin = cout
    for i, (fin, fout) in enumerate(((25088, 4096), (4096, 4096), (4096, 1000))):
        lay.add(f"fc{i}.weight", fin * fout, "he", fin)
        lay.add(f"fc{i}.bias", fout, "zero")
    return lay


def flat(n: int) -> Layout:
    """A single tensor of n elements (the bandwidth-sweep layout)."""
    lay = Layout(f"flat{n}")
    lay.add("flat", n, "he", 1)
    return lay


def get_layout(name: str) -> Layout:
    if name == "resnet20":
        return resnet_cifar(20)
    if name == "resnet56":
        return resnet_cifar(56)
    if name == "resnet50":
        return resnet50_imagenet()
    if name == "vgg16":
        return vgg16_imagenet()
    if name.startswith("flat"):
        return flat(int(name[4:]))
    raise KeyError(name)


def valid_mask(lay: Layout, device="cpu") -> torch.Tensor:
    """float32 arena of 1.0 on real elements and 0.0 on alignment padding."""
    m = torch.zeros(lay.padded_numel, dtype=torch.float32, device=device)
    for off, n in zip(lay.offsets, lay.numels):
        m[off:off + n] = 1.0
    return m


def init_weights(lay: Layout, seed: int = SEED, device="cpu") -> torch.Tensor:
    """Arena of initial weights: He-normal conv/FC weights, gamma = 1, beta = bias = 0."""
    w = torch.zeros(lay.padded_numel, dtype=torch.float32, device=device)
    for t, (off, n, kind, fan) in enumerate(zip(lay.offsets, lay.numels, lay.kinds, lay.fan_ins)):
        if kind == "he":
            key = stream_key(seed, STREAM_WEIGHT, 0, t)
            w[off:off + n] = normal(key, n, math.sqrt(2.0 / fan), device)
        elif kind == "one":
            w[off:off + n] = 1.0
    return w


def gradient(lay: Layout, iteration: int, worker: int, sigma: float, seed: int = SEED,
             device="cpu", mask: torch.Tensor | None = None) -> torch.Tensor:
    """Arena of one worker's gradient for one iteration, N(0, sigma^2), zero on padding."""
    key = stream_key(seed, STREAM_GRAD, iteration, worker)
    g = normal(key, lay.padded_numel, sigma, device)
    if lay.padded_numel != lay.numel:
        g *= mask if mask is not None else valid_mask(lay, device)
    return g


def gradient_at(lay: Layout, iteration: int, worker: int, sigma: float, idx: torch.Tensor,
                seed: int = SEED) -> torch.Tensor:
    """The same gradient values as `gradient`, only at arena indices `idx` (int64)."""
    key = stream_key(seed, STREAM_GRAD, iteration, worker)
    g = normal_at(key, idx, sigma)
    if lay.padded_numel != lay.numel:
        g = g * valid_mask(lay, idx.device)[idx]
    return g


def uniform_buffer(stream: int, n: int, iteration: int = 0, worker: int = 0,
                   seed: int = SEED, device="cpu") -> torch.Tensor:
    """uniform[-1, 1) buffer of the bandwidth-sweep workload."""
    return uniform(stream_key(seed, stream, iteration, worker), n, device)


def to_bf16(x: torch.Tensor) -> torch.Tensor:
    """Round-to-nearest-even float32 -> bfloat16 (input preparation only)."""
    return x.to(torch.bfloat16)


def bf16_bits(x: torch.Tensor):
    """bfloat16 tensor -> numpy uint16 array of its bit patterns (CPU)."""
    return x.detach().cpu().view(torch.int16).numpy().view("uint16")
