"""Seeded synthetic gradient tensors.

Input synthesis only: this module holds none of the compression method's
arithmetic, so both the CUDA library's tests and the CPU oracle's tests draw
their inputs from it.

The tensors stand in for the neural gradients (gradients with respect to layer
outputs) of ImageNet CNN backward passes: each nonzero magnitude is
exp(N(mu, sigma^2)) with a random sign, and a Bernoulli mask sets a fraction of
the entries to exactly zero (the zeros a ReLU leaves in its input gradient).
Shapes are the conv-output shapes of the standard ResNet-18 / ResNet-50
topologies at a given batch size.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

_CHUNK = 1 << 24


def lognormal_tensor(n: int, mu: float, sigma: float, zero_frac: float, seed: int,
                     dtype: torch.dtype = torch.float32, device: str = "cpu",
                     clip: Optional[float] = None,
                     mixture: Optional[Sequence[Tuple[float, float]]] = None) -> torch.Tensor:
    """Flat tensor of n elements: sign * exp(mu + sigma*z), z ~ N(0,1), zeroed
    with probability ``zero_frac``; magnitudes optionally clipped at ``clip``.
    ``mixture`` = [(mu, sigma), ...] draws each element's parameters uniformly
    from the list instead.  Magnitudes are formed in fp64 and rounded once to
    ``dtype`` (bf16: round-to-nearest-even), so values may land in the fp32
    subnormal range."""
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    out = torch.empty(n, dtype=dtype, device=device)
    for lo in range(0, n, _CHUNK):
        m = min(_CHUNK, n - lo)
        z = torch.randn(m, generator=gen, device=device, dtype=torch.float64)
        u_sign = torch.rand(m, generator=gen, device=device)
        u_zero = torch.rand(m, generator=gen, device=device)
        if mixture is None:
            y = mu + sigma * z
        else:
            comp = torch.randint(0, len(mixture), (m,), generator=gen, device=device)
            mus = torch.tensor([c[0] for c in mixture], dtype=torch.float64, device=device)[comp]
            sgs = torch.tensor([c[1] for c in mixture], dtype=torch.float64, device=device)[comp]
            y = mus + sgs * z
        mag = torch.exp(y)
        if clip is not None:
            mag = torch.clamp(mag, max=float(clip))
        val = torch.where(u_sign < 0.5, -mag, mag)
        val = torch.where(u_zero < zero_frac, torch.zeros_like(val), val)
        out[lo:lo + m] = val.to(torch.float32).to(dtype)
    return out


def bimodal_tensor(n: int, mu_right: float, sigma_right: float, mu_left: float, sigma_left: float,
                   left_frac: float, seed: int, dtype: torch.dtype = torch.float32, device: str = "cpu"):
    """A gradient before batch-norm and the mask that tells its two modes apart
    (the entries where the gradient after batch-norm is non-zero): returns
    (g, right_mode).  right_mode is a uint8 tensor, 1 with probability
    1 - left_frac; g is dense, sign * exp(N(mu_right, sigma_right^2)) where the
    mask is 1 and sign * exp(N(mu_left, sigma_left^2)) elsewhere."""
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    g = torch.empty(n, dtype=dtype, device=device)
    mask = torch.empty(n, dtype=torch.uint8, device=device)
    for lo in range(0, n, _CHUNK):
        m = min(_CHUNK, n - lo)
        z = torch.randn(m, generator=gen, device=device, dtype=torch.float64)
        u_sign = torch.rand(m, generator=gen, device=device)
        right = torch.rand(m, generator=gen, device=device) >= left_frac
        y = torch.where(right, mu_right + sigma_right * z, mu_left + sigma_left * z)
        mag = torch.exp(y)
        g[lo:lo + m] = torch.where(u_sign < 0.5, -mag, mag).to(torch.float32).to(dtype)
        mask[lo:lo + m] = right.to(torch.uint8)
    return g, mask


def as_numpy_bits(t: torch.Tensor) -> np.ndarray:
    """Host numpy view of a tensor: float32 stays float32, bfloat16 becomes its
    raw uint16 bit patterns (numpy has no bfloat16)."""
    t = t.detach().contiguous().cpu()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    if t.dtype == torch.float32:
        return t.numpy()
    raise TypeError(t.dtype)


def from_numpy_bits(a: np.ndarray, device: str = "cpu") -> torch.Tensor:
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).to(device)
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device)


# --------------------------------------------------------------------------- shapes
@dataclass
class LayerShape:
    name: str
    shape: Tuple[int, int, int, int]
    kernel: int            # spatial size of the conv that produced this output

    @property
    def numel(self) -> int:
        return int(np.prod(self.shape))


def resnet18_conv_outputs(batch: int = 256) -> List[LayerShape]:
    """The 20 conv outputs of ImageNet ResNet-18: stem, 16 block convs,
    3 downsample convs."""
    L = [LayerShape("conv1", (batch, 64, 112, 112), 7)]
    res = {64: 56, 128: 28, 256: 14, 512: 7}
    for si, ch in enumerate((64, 128, 256, 512)):
        hw = res[ch]
        for b in range(2):
            for c in range(2):
                L.append(LayerShape(f"layer{si+1}.{b}.conv{c+1}", (batch, ch, hw, hw), 3))
        if si > 0:
            L.append(LayerShape(f"layer{si+1}.0.downsample", (batch, ch, hw, hw), 1))
    return L


def resnet50_conv_outputs(batch: int = 256) -> List[LayerShape]:
    """The 53 conv outputs of ImageNet ResNet-50 (stride on the 3x3 conv)."""
    L = [LayerShape("conv1", (batch, 64, 112, 112), 7)]
    blocks = (3, 4, 6, 3)
    hw_in = 56
    for si, (width, nb) in enumerate(zip((64, 128, 256, 512), blocks)):
        hw_out = hw_in if si == 0 else hw_in // 2
        for b in range(nb):
            first = (b == 0)
            hw1 = hw_in if first else hw_out
            L.append(LayerShape(f"layer{si+1}.{b}.conv1", (batch, width, hw1, hw1), 1))
            L.append(LayerShape(f"layer{si+1}.{b}.conv2", (batch, width, hw_out, hw_out), 3))
            L.append(LayerShape(f"layer{si+1}.{b}.conv3", (batch, 4 * width, hw_out, hw_out), 1))
            if first:
                L.append(LayerShape(f"layer{si+1}.0.downsample", (batch, 4 * width, hw_out, hw_out), 1))
        hw_in = hw_out
    return L


@dataclass
class LayerSpec:
    name: str
    numel: int
    mu: float
    sigma: float
    zero_frac: float
    sparsity: float        # requested S for pruning
    data_seed: int


def resnet18_prune_workload(batch: int = 256, seed: int = 0) -> List[LayerSpec]:
    """Per layer: zero fraction U[0.3,0.6], mu U[-16,-9], sigma U[1.5,3.0],
    requested sparsity drawn from {0.5, 0.7, 0.85, 0.9}."""
    rs = np.random.RandomState(seed)
    specs = []
    for k, ls in enumerate(resnet18_conv_outputs(batch)):
        specs.append(LayerSpec(ls.name, ls.numel,
                               mu=float(rs.uniform(-16, -9)), sigma=float(rs.uniform(1.5, 3.0)),
                               zero_frac=float(rs.uniform(0.3, 0.6)),
                               sparsity=float(rs.choice([0.5, 0.7, 0.85, 0.9])),
                               data_seed=seed * 1000 + k))
    return specs


def resnet50_quant_workload(batch: int = 256, seed: int = 0) -> List[LayerSpec]:
    """Per layer: mu U[-16,-9], sigma U[1.5,3.0]; outputs of 1x1 convs have no
    exact zeros, every other output has 50 % zeros (after a ReLU)."""
    rs = np.random.RandomState(seed)
    specs = []
    for k, ls in enumerate(resnet50_conv_outputs(batch)):
        specs.append(LayerSpec(ls.name, ls.numel,
                               mu=float(rs.uniform(-16, -9)), sigma=float(rs.uniform(1.5, 3.0)),
                               zero_frac=0.0 if ls.kernel == 1 else 0.5,
                               sparsity=0.0, data_seed=seed * 1000 + k))
    return specs


def make_layers(specs: Sequence[LayerSpec], dtype: torch.dtype, device: str) -> List[torch.Tensor]:
    return [lognormal_tensor(s.numel, s.mu, s.sigma, s.zero_frac, s.data_seed, dtype, device)
            for s in specs]
