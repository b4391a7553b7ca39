"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random numbers and lays them out; it contains none of
the method's arithmetic (no scoring, no sampling rule, no loss).  Both the CUDA
library's callers and the CPU oracle's callers take their inputs from here, so
that the two sides see identical data.

The inputs stand in for the datasets the paper trained on (Sec. "Image classification": MNIST,
FashionMNIST, EMNIST, CIFAR10; Sec. "Machine Translation": Multi30k, WMT14 En-De): the shapes,
sizes and value ranges follow them (pixel vectors in [0, 1), 3*32*32 = 3072
features, 10..1000 classes, sentence lengths 8..128, vocabularies of tens of
thousands of tokens) and no dataset item is used.  "N(0, s)" below always means
standard deviation s.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def normal(shape, std: float, seed: int, dtype=torch.float32, device="cpu") -> torch.Tensor:
    t = torch.randn(shape, generator=_gen(seed, device), device=device, dtype=torch.float32) * std
    return t.to(dtype)


def uniform01(shape, seed: int, dtype=torch.float32, device="cpu") -> torch.Tensor:
    t = torch.rand(shape, generator=_gen(seed, device), device=device, dtype=torch.float32)
    t = t.to(dtype)
    if dtype == torch.bfloat16:
        # rounding to bf16 can reach 1.0; keep the pixel range half-open
        t = torch.clamp(t, max=0.99609375)
    return t


def randint(lo: int, hi: int, shape, seed: int, device="cpu") -> torch.Tensor:
    return torch.randint(lo, hi, shape, generator=_gen(seed, device), device=device, dtype=torch.int32)


def to_oracle(t: torch.Tensor) -> np.ndarray:
    """Host NumPy view for the oracle: bf16 becomes its uint16 bit pattern."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


# --------------------------------------------------------------------------
# Assistant parameters
# --------------------------------------------------------------------------

def linear_assistant(d: int, seed: int, device="cpu", std: float = 0.01):
    """w ~ N(0, std), b = 0 (fp32)."""
    return normal((d,), std, seed, torch.float32, device), torch.zeros(1, dtype=torch.float32, device=device)


def mlp_assistant(d: int, hidden: int, seed: int, device="cpu"):
    """W1 [hidden, d] ~ N(0, 1/sqrt(d)) fp32 master, w2 ~ N(0, 1/sqrt(hidden)), biases 0."""
    W1 = normal((hidden, d), 1.0 / float(np.sqrt(d)), seed, torch.float32, device)
    w2 = normal((hidden,), 1.0 / float(np.sqrt(hidden)), seed + 1, torch.float32, device)
    b1 = torch.zeros(hidden, dtype=torch.float32, device=device)
    b2 = torch.zeros(1, dtype=torch.float32, device=device)
    return W1, b1, w2, b2


# --------------------------------------------------------------------------
# Workloads
# --------------------------------------------------------------------------

@dataclass
class TinyRef:
    """Small reference case: fp32 features ~ N(0,1), 10-class fp32 logits ~ N(0,2)."""
    n: int = 4096
    d: int = 64
    classes: int = 10
    gamma: float = 0.1
    lr: float = 0.1
    philox_seed: int = 0
    step: int = 0

    def make(self, device="cpu"):
        w, b = linear_assistant(self.d, 2, device)
        return {
            "x": normal((self.n, self.d), 1.0, 1, torch.float32, device),
            "w": w, "b": b,
            "logits": normal((self.n, self.classes), 2.0, 3, torch.float32, device),
            "labels": randint(0, self.classes, (self.n,), 4, device),
        }


@dataclass
class ImageShape:
    """Image-classification shape: bf16 pixel vectors U[0,1), d = 3*32*32, 100-class fp32 logits ~ N(0,3)."""
    n: int = 65536
    d: int = 3072
    classes: int = 100
    gamma: float = 0.1
    lr: float = 0.05
    philox_seed: int = 0

    def pool(self, pool_id: int, device="cpu") -> torch.Tensor:
        return uniform01((self.n, self.d), 100 + pool_id, torch.bfloat16, device)

    def assistant(self, device="cpu"):
        return linear_assistant(self.d, 2, device)

    def logits(self, pool_id: int, device="cpu") -> torch.Tensor:
        return normal((self.n, self.classes), 3.0, 200 + pool_id, torch.float32, device)

    def labels(self, pool_id: int, device="cpu") -> torch.Tensor:
        return randint(0, self.classes, (self.n,), 300 + pool_id, device)


@dataclass
class TranslationShape:
    """Translation shape: hashed bag-of-words CSR features, bf16 token logits ~ N(0,4) over a 32,000 vocabulary."""
    n: int = 16384
    buckets: int = 1 << 18
    len_lo: int = 8
    len_hi: int = 128
    vocab: int = 32000
    token_budget: int = 25000
    gamma: float = 0.2
    lr: float = 0.05
    philox_seed: int = 0

    def csr(self, device="cpu"):
        lengths = randint(self.len_lo, self.len_hi + 1, (self.n,), 5, "cpu").to(torch.int64)
        indptr = torch.zeros(self.n + 1, dtype=torch.int64)
        indptr[1:] = torch.cumsum(lengths, 0)
        nnz = int(indptr[-1])
        col = randint(0, self.buckets, (nnz,), 6, "cpu")
        val = torch.ones(nnz, dtype=torch.float32)
        return (indptr.to(torch.int32).to(device), col.to(device), val.to(device),
                lengths.to(torch.int32).to(device))

    def assistant(self, device="cpu"):
        return linear_assistant(self.buckets, 2, device)

    def token_logits(self, rows: int, device="cpu") -> torch.Tensor:
        return normal((rows, self.vocab), 4.0, 7, torch.bfloat16, device)

    def token_ids(self, rows: int, device="cpu") -> torch.Tensor:
        return randint(0, self.vocab, (rows,), 8, device)


def token_budget_offsets(lengths_of_batch: np.ndarray, budget: int) -> np.ndarray:
    """Offsets [S+1] of the longest prefix of sentences whose token total stays within the budget."""
    csum = np.cumsum(lengths_of_batch.astype(np.int64))
    s = int(np.searchsorted(csum, budget, side="right"))
    off = np.zeros(s + 1, dtype=np.int32)
    off[1:] = csum[:s]
    return off


@dataclass
class MlpShape:
    """Two-layer Assistant case: bf16 features ~ N(0,1), d -> hidden (ReLU) -> 1, 1000-class fp32 logits ~ N(0,3)."""
    n: int = 262144
    d: int = 3072
    hidden: int = 256
    classes: int = 1000
    gamma: float = 0.1
    lr: float = 0.01
    philox_seed: int = 0

    def pool(self, device="cpu") -> torch.Tensor:
        return normal((self.n, self.d), 1.0, 9, torch.bfloat16, device)

    def assistant(self, device="cpu"):
        return mlp_assistant(self.d, self.hidden, 10, device)

    def logits(self, rows: int, device="cpu") -> torch.Tensor:
        return normal((rows, self.classes), 3.0, 12, torch.float32, device)

    def labels(self, rows: int, device="cpu") -> torch.Tensor:
        return randint(0, self.classes, (rows,), 13, device)


@dataclass
class ConvShape:
    """Convolutional Assistant case: the image shape's bf16 pixel pools read as 3 x 32 x 32 images, a first ResNet-style
    convolution (16 channels of 3 x 3 taps ~ N(0, sqrt(2 / 27)), standing in for the Boss's) and 4 x 4 average pooling:
    1024 features per instance for the linear layer."""
    n: int = 65536
    c_in: int = 3
    height: int = 32
    width: int = 32
    c_out: int = 16
    ksize: int = 3
    pool: int = 4
    gamma: float = 0.1
    lr: float = 0.05
    philox_seed: int = 0

    @property
    def d(self) -> int:
        return self.c_in * self.height * self.width

    @property
    def features(self) -> int:
        return self.c_out * (self.height // self.pool) * (self.width // self.pool)

    def pool_images(self, pool_id: int, device="cpu") -> torch.Tensor:
        return uniform01((self.n, self.d), 100 + pool_id, torch.bfloat16, device)

    def conv(self, device="cpu"):
        fan_in = self.c_in * self.ksize * self.ksize
        weight = normal((self.c_out, self.c_in, self.ksize, self.ksize), float(np.sqrt(2.0 / fan_in)), 20, torch.float32, device)
        bias = torch.zeros(self.c_out, dtype=torch.float32, device=device)
        return weight, bias

    def assistant(self, device="cpu"):
        return linear_assistant(self.features, 21, device)


@dataclass
class SweepShape:
    """Scaling sweep: fp32 features ~ N(0,1), d = 512, pools of 2^20 .. 2^24 instances."""
    n: int = 1 << 20
    d: int = 512
    gamma: float = 0.05
    philox_seed: int = 0

    def pool(self, device="cpu") -> torch.Tensor:
        return normal((self.n, self.d), 1.0, 14, torch.float32, device)

    def assistant(self, device="cpu"):
        return linear_assistant(self.d, 2, device)


def sweep_logits(rows: int, vocab: int, device="cpu", seed: int = 15) -> torch.Tensor:
    """bf16 token logits ~ N(0,4) for the instance-loss sweep."""
    return normal((rows, vocab), 4.0, seed, torch.bfloat16, device)


def ragged_offsets(rows: int, len_lo: int, len_hi: int, seed: int) -> np.ndarray:
    """Offsets of consecutive segments with lengths U{len_lo..len_hi} covering exactly `rows` rows."""
    rng = np.random.default_rng(seed)
    off = [0]
    while off[-1] < rows:
        off.append(min(rows, off[-1] + int(rng.integers(len_lo, len_hi + 1))))
    return np.asarray(off, dtype=np.int32)
