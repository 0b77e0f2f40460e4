"""Seeded synthetic inputs and layer shapes for the variance-based gradient compression path.

This module serves both the CUDA path and the CPU oracle: it produces bytes, never results.
It holds no arithmetic of the method (no squared-gradient sum, no send test, no quantiser,
no decoder).  Every tensor is generated ONCE, on whichever device is asked for, and then
copied to whoever needs it, so both sides always consume identical bits.

The paper trains a VGG-like net on CIFAR-10 and ResNet-50 on ImageNet (Sec. 6); neither the
data nor trained weights are available, so the tensors below take those networks' layer
shapes, the paper's per-worker batch sizes and its hyper-parameters, and stand in for them.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence, Tuple

import numpy as np
import torch

_MASK64 = (1 << 64) - 1


# ----------------------------------------------------------------------------------------
# layer shapes (architecture facts)
# ----------------------------------------------------------------------------------------
@dataclass(frozen=True)
class LayerSpec:
    """One weight tensor.  kind 'fc': weight [cout, cin]; 'conv': weight [cout, cin, k, k]."""
    name: str
    kind: str
    cin: int
    cout: int
    k: int = 1
    stride: int = 1
    pad: int = 0
    hin: int = 1

    @property
    def hout(self) -> int:
        return (self.hin + 2 * self.pad - self.k) // self.stride + 1

    @property
    def n_params(self) -> int:
        return self.cout * self.cin * self.k * self.k

    def gemm_mnk(self, batch: int) -> Tuple[int, int, int]:
        """(M, N, K) of the squared-operand contraction: M=cout, N=cin*k*k, K=batch*positions."""
        pos = self.hout * self.hout if self.kind == "conv" else 1
        return self.cout, self.cin * self.k * self.k, batch * pos

    def x_shape(self, batch: int):
        return (batch, self.cin, self.hin, self.hin) if self.kind == "conv" else (batch, self.cin)

    def delta_shape(self, batch: int):
        return (batch, self.cout, self.hout, self.hout) if self.kind == "conv" else (batch, self.cout)


def dense_layers() -> List[LayerSpec]:
    """Single dense layer 256 -> 128 (32,768 weights)."""
    return [LayerSpec("fc", "fc", 256, 128)]


def mlp_layers() -> List[LayerSpec]:
    """MLP 784-1024-1024-10 (1,861,632 weights)."""
    return [LayerSpec("fc1", "fc", 784, 1024), LayerSpec("fc2", "fc", 1024, 1024),
            LayerSpec("fc3", "fc", 1024, 10)]


def resnet50_layers(h: int = 224) -> List[LayerSpec]:
    """53 conv + 1 fc weight tensors of ResNet-50 (stride on the 3x3 conv of each bottleneck)."""
    layers = [LayerSpec("conv1", "conv", 3, 64, 7, 2, 3, h)]
    hh = (h + 2 * 3 - 7) // 2 + 1          # conv1
    hh = (hh + 2 * 1 - 3) // 2 + 1         # 3x3 max pool, stride 2, pad 1
    inp = 64
    for si, (w, nblocks, s) in enumerate([(64, 3, 1), (128, 4, 2), (256, 6, 2), (512, 3, 2)], 1):
        for b in range(nblocks):
            st = s if b == 0 else 1
            ho = (hh + 2 - 3) // st + 1
            layers.append(LayerSpec(f"l{si}.{b}.c1", "conv", inp, w, 1, 1, 0, hh))
            layers.append(LayerSpec(f"l{si}.{b}.c2", "conv", w, w, 3, st, 1, hh))
            layers.append(LayerSpec(f"l{si}.{b}.c3", "conv", w, 4 * w, 1, 1, 0, ho))
            if b == 0:
                layers.append(LayerSpec(f"l{si}.{b}.ds", "conv", inp, 4 * w, 1, st, 0, hh))
            inp, hh = 4 * w, ho
    layers.append(LayerSpec("fc", "fc", 2048, 1000))
    return layers


def vgg16_layers(h: int = 224) -> List[LayerSpec]:
    """13 conv (3x3, stride 1, pad 1) + 3 fc weight tensors of VGG-16 (138,344,128 weights)."""
    cfg = [64, 64, "M", 128, 128, "M", 256, 256, 256, "M", 512, 512, 512, "M", 512, 512, 512, "M"]
    layers, c, hh, i = [], 3, h, 0
    for item in cfg:
        if item == "M":
            hh //= 2
        else:
            layers.append(LayerSpec(f"conv{i}", "conv", c, item, 3, 1, 1, hh))
            c, i = item, i + 1
    layers += [LayerSpec("fc6", "fc", 512 * 7 * 7, 4096), LayerSpec("fc7", "fc", 4096, 4096),
               LayerSpec("fc8", "fc", 4096, 1000)]
    return layers


def group_offsets(layers: Sequence[LayerSpec]) -> np.ndarray:
    """Offsets [K+1] (uint32) of each weight tensor in the flat parameter buffer."""
    offs = np.zeros(len(layers) + 1, np.int64)
    offs[1:] = np.cumsum([l.n_params for l in layers])
    assert offs[-1] < 2 ** 32
    return offs.astype(np.uint32)


# ----------------------------------------------------------------------------------------
# seeding
# ----------------------------------------------------------------------------------------
def _splitmix64(z: int) -> int:
    z = (z + 0x9E3779B97F4A7C15) & _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return z ^ (z >> 31)


def seed_for(config: int, worker: int = 0, step: int = 0, layer: int = 0, tensor: int = 0) -> int:
    """One 63-bit seed per (config, worker, step, layer, tensor); tensor 0: x, 1: delta, 2..: other."""
    key = 0x1802060580000000 + (config << 32) + (worker << 24) + (step << 12) + (layer << 2) + tensor
    return _splitmix64(key & _MASK64) >> 1


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def normal(shape, std: float, seed: int, device="cpu") -> torch.Tensor:
    """fp32 N(0, std^2) tensor (std is the standard deviation)."""
    out = torch.empty(shape, dtype=torch.float32, device=device)
    out.normal_(0.0, 1.0, generator=_gen(seed, device))
    return out.mul_(std)


def half_normal(shape, std: float, seed: int, device="cpu") -> torch.Tensor:
    """|N(0, std^2)|: the stand-in for post-ReLU conv activations."""
    return normal(shape, std, seed, device).abs_()


def relu_normal(shape, std: float, seed: int, device="cpu") -> torch.Tensor:
    """max(0, N(0, std^2)): about half the entries are exact zeros."""
    return normal(shape, std, seed, device).clamp_(min=0.0)


def layer_inputs(spec: LayerSpec, batch: int, config: int, worker: int, step: int, layer: int,
                 x_kind: str, delta_std: float, device="cpu"):
    """Layer input x and back-propagated error delta for one step of one worker."""
    make_x = {"normal": normal, "half_normal": half_normal, "relu_normal": relu_normal}[x_kind]
    x = make_x(spec.x_shape(batch), 1.0, seed_for(config, worker, step, layer, 0), device)
    delta = normal(spec.delta_shape(batch), delta_std, seed_for(config, worker, step, layer, 1), device)
    return x, delta


# ----------------------------------------------------------------------------------------
# the ordinary mini-batch gradient g: an INPUT of the compressor, made by the harness
# ----------------------------------------------------------------------------------------
def mean_gradient(spec: LayerSpec, x: torch.Tensor, delta: torch.Tensor) -> torch.Tensor:
    """sum_z grad_z / B of the layer's weight, flat in weight layout (library GEMM / conv)."""
    batch = x.shape[0]
    if spec.kind == "fc":
        return (delta.t() @ x).div_(batch).reshape(-1)
    gw = torch.nn.grad.conv2d_weight(x, (spec.cout, spec.cin, spec.k, spec.k), delta,
                                     stride=spec.stride, padding=spec.pad)
    return gw.div_(batch).reshape(-1)


def per_parameter_gs(n: int, batch: int, delta_std: float, seed: int, device="cpu",
                     chunk: int = 1 << 22):
    """g_i = sum_z a_z / B and s_i = sum_z a_z^2 / B^2 with a_z = delta*x drawn per parameter
    (x ~ |N(0,1)|, delta ~ N(0, delta_std^2)): the stand-in for a flat buffer whose layers'
    activations are too large to materialise (VGG-16 at batch 64)."""
    g = torch.empty(n, dtype=torch.float32, device=device)
    s = torch.empty(n, dtype=torch.float32, device=device)
    gen = _gen(seed, device)
    for lo in range(0, n, chunk):
        m = min(chunk, n - lo)
        a = torch.empty((m, batch), dtype=torch.float32, device=device).normal_(generator=gen).abs_()
        d = torch.empty((m, batch), dtype=torch.float32, device=device).normal_(generator=gen)
        a.mul_(d).mul_(delta_std)
        g[lo:lo + m] = a.sum(1) / batch
        s[lo:lo + m] = a.square_().sum(1) / float(batch * batch)
    return g, s


def planted_density_gs(n: int, alpha: float, q: float, seed: int, device="cpu"):
    """g ~ N(0,1) and s chosen so that a fraction ~q of the parameters sits clearly on the
    send side of r^2 > alpha*v at the first step and the rest clearly on the other side."""
    gen = _gen(seed, device)
    g = torch.empty(n, dtype=torch.float32, device=device).normal_(generator=gen)
    pick = torch.empty(n, dtype=torch.float32, device=device).uniform_(generator=gen) < q
    factor = torch.where(pick, torch.tensor(1.0 / (2.0 * alpha), device=device),
                         torch.tensor(2.0 / alpha, device=device))
    return g, g * g * factor


# ----------------------------------------------------------------------------------------
# generated messages for the decoder sweep
# ----------------------------------------------------------------------------------------
def random_message(n: int, offsets: np.ndarray, density: float, seed: int, device="cpu",
                   exp_lo: int = -20, exp_hi: int = -8, index_mask: torch.Tensor = None,
                   exp_seed: int = None, exp_jitter: int = 1):
    """A packed message with ~density*n sorted distinct uniform indices, uniform sign, uniform
    3-bit code, and per-group exponents uniform on [exp_lo, exp_hi].

    exp_seed: the workers of one job see the same parameters and mini-batches of the same distribution, so the
    largest residual of a weight tensor (whose exponent is the group exponent, Sec. 4.2) is of the same magnitude
    on every worker.  With exp_seed the per-group exponents are drawn once from that seed (shared by all messages
    built with it) and each message moves every group by a draw from [-exp_jitter, exp_jitter]; without it every
    message draws its own exponents over the whole range (workers that have nothing in common).

    Word layout: index << 4 | sign << 3 | code.  Returns (words, group_exp): words is an int32
    tensor holding the 32-bit patterns (view it as uint32), group_exp an int32 tensor."""
    gen = _gen(seed, device)
    if index_mask is None:
        index_mask = torch.empty(n, dtype=torch.float32, device=device).uniform_(generator=gen) < density
    idx = index_mask.nonzero().reshape(-1)
    low = torch.randint(0, 16, (idx.numel(),), generator=gen, device=device, dtype=torch.int64)
    w64 = (idx << 4) | low
    words = torch.where(w64 >= 2 ** 31, w64 - 2 ** 32, w64).to(torch.int32)   # same 32 bits
    k = len(offsets) - 1
    if exp_seed is None:
        gexp = torch.randint(exp_lo, exp_hi + 1, (k,), generator=gen, device=device, dtype=torch.int32)
    else:
        base = torch.randint(exp_lo, exp_hi + 1, (k,), generator=_gen(exp_seed, device), device=device, dtype=torch.int32)
        gexp = base + torch.randint(-exp_jitter, exp_jitter + 1, (k,), generator=gen, device=device, dtype=torch.int32)
    return words, gexp
