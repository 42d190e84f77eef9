"""Seeded synthetic workloads for the grouped aggregate + update path.

This module only MAKES INPUTS: parameter and gradient tensors with the sizes,
dtypes and value distributions of the five workloads, and the per-step mode
decisions (which worker goes into which group) drawn from a small counter-based
integer generator.  It holds none of the method's arithmetic: it neither
encodes schedules into CSR form nor touches the update rule, so both the CUDA
library and the CPU oracle can be fed from it.

The paper (Section III, set-up) trains ten small vision / language models on
CIFAR-10 and WikiText-2 under a cluster trace.  The cost of the PS-side update
depends only on the number of parameters n, the number of workers W, the
gradient dtype and the grouping, so seeded tensors of ResNet-50 / BERT-large /
VGG-16 / GPT-2-medium size stand in for those training runs.

Generation recipe (the same on any device, values differ between devices
because torch's CPU and CUDA generators differ; every consumer reads the
generated buffers, never regenerates them on another device):
  params     : N(0, param_std) fp32 from ``torch.Generator`` seeded
               ``stream_seed(seed, STREAM_PARAMS, tensor_index, 0)``
  momentum   : zeros
  grads[w]   : N(0, grad_std) fp32 from a generator seeded
               ``stream_seed(seed, STREAM_GRADS, step, w)`` (one generator per
               (step, worker), drawing the tensors of a list in list order),
               then, if outlier_prob > 0, multiplied by outlier_scale where a
               uniform draw from the same generator is < outlier_prob, then
               rounded to the gradient dtype (bf16: round to nearest even).
  decisions  : SplitMix64 seeded ``seed * 1000 + step``; Fisher-Yates shuffle.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional, Sequence, Tuple

import torch

STREAM_PARAMS = 1
STREAM_GRADS = 2

_MASK64 = (1 << 64) - 1


class SplitMix64:
    """SplitMix64 (Steele, Lea, Flood 2014): a 64-bit counter-based generator."""

    def __init__(self, seed: int):
        self.state = seed & _MASK64

    def next_u64(self) -> int:
        self.state = (self.state + 0x9E3779B97F4A7C15) & _MASK64
        z = self.state
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
        return z ^ (z >> 31)

    def below(self, bound: int) -> int:
        """Uniform integer in [0, bound) by rejection (no modulo bias)."""
        limit = (1 << 64) - ((1 << 64) % bound)
        while True:
            r = self.next_u64()
            if r < limit:
                return r % bound

    def permutation(self, n: int) -> List[int]:
        perm = list(range(n))
        for i in range(n - 1, 0, -1):
            j = self.below(i + 1)
            perm[i], perm[j] = perm[j], perm[i]
        return perm


def stream_seed(seed: int, stream: int, a: int, b: int) -> int:
    """A distinct 63-bit torch seed for every (seed, stream, a, b)."""
    g = SplitMix64((seed << 40) ^ (stream << 36) ^ (a << 12) ^ b)
    return g.next_u64() >> 1


@dataclasses.dataclass(frozen=True)
class ModeDecision:
    """What the mode-determination layer hands to the schedule encoder.

    kind = "labels"    : ``labels[w]`` = group of worker w (-1 = absent); groups
                         are taken in ascending label order.
    kind = "static_x"  : ``arrival_order`` and ``x``.
    kind = "dynamic_x" : ``iter_time[w]`` and ``labels[w]`` (cluster ids).
    """
    kind: str
    W: int
    labels: Optional[Tuple[int, ...]] = None
    arrival_order: Optional[Tuple[int, ...]] = None
    x: int = 0
    sort_members: bool = True
    iter_time: Optional[Tuple[float, ...]] = None


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    model: str
    shapes: Tuple[Tuple[str, Tuple[int, ...]], ...]   # per-tensor (name, shape)
    multi_tensor: bool
    W: int
    grad_dtype: str            # "f32" | "bf16"
    param_std: float
    grad_std: float
    outlier_prob: float
    outlier_scale: float
    lr: float
    mu: float
    wd: float
    steps: int
    seed: int
    schedule: str              # "fixed" | "shuffle4x4" | "asgd" | "random_2_8"
    fixed_labels: Optional[Tuple[int, ...]] = None

    @property
    def sizes(self) -> List[int]:
        out = []
        for _, shape in self.shapes:
            m = 1
            for d in shape:
                m *= d
            out.append(m)
        return out

    @property
    def n(self) -> int:
        return sum(self.sizes)

    @property
    def grad_bytes(self) -> int:
        return 2 if self.grad_dtype == "bf16" else 4

    def torch_grad_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.grad_dtype == "bf16" else torch.float32

    def decision(self, step: int) -> ModeDecision:
        """The grouping of the W workers for round ``step`` (0-based)."""
        W = self.W
        if self.schedule == "fixed":
            return ModeDecision("labels", W, labels=self.fixed_labels)
        if self.schedule == "asgd":
            return ModeDecision("static_x", W, arrival_order=tuple(range(W)), x=1)
        rng = SplitMix64(self.seed * 1000 + step)
        if self.schedule == "shuffle4x4":
            perm = rng.permutation(W)
            labels = [0] * W
            for pos, w in enumerate(perm):
                labels[w] = pos // (W // 4)
            return ModeDecision("labels", W, labels=tuple(labels))
        if self.schedule == "random_2_8":
            K = 2 + rng.below(7)
            perm = rng.permutation(W)
            gaps = rng.permutation(W - 1)[: K - 1]       # cut after position gap
            cuts = sorted(g + 1 for g in gaps)
            labels = [0] * W
            for pos, w in enumerate(perm):
                labels[w] = sum(1 for c in cuts if c <= pos)
            return ModeDecision("labels", W, labels=tuple(labels))
        raise ValueError(self.schedule)

    def algorithmic_bytes(self, scheduled_workers: int) -> int:
        """Bytes one fused round must move: every scheduled gradient element read
        once, p and v read once and written once."""
        return self.n * (scheduled_workers * self.grad_bytes + 16)


def gpt2_medium_shapes(layers: int = 24, vocab: int = 50257) -> Tuple[Tuple[str, Tuple[int, ...]], ...]:
    """The 292 parameter tensors of a GPT-2-medium-shaped model: d=1024, 24
    layers, vocabulary 50257, 1024 positions, tied output head.  Fewer layers
    or a smaller vocabulary give a shorter list of the same kinds of tensors."""
    d, positions = 1024, 1024
    shapes: List[Tuple[str, Tuple[int, ...]]] = [("wte", (vocab, d)), ("wpe", (positions, d))]
    for l in range(layers):
        pre = "h%d." % l
        shapes += [
            (pre + "ln_1.weight", (d,)), (pre + "ln_1.bias", (d,)),
            (pre + "attn.c_attn.weight", (d, 3 * d)), (pre + "attn.c_attn.bias", (3 * d,)),
            (pre + "attn.c_proj.weight", (d, d)), (pre + "attn.c_proj.bias", (d,)),
            (pre + "ln_2.weight", (d,)), (pre + "ln_2.bias", (d,)),
            (pre + "mlp.c_fc.weight", (d, 4 * d)), (pre + "mlp.c_fc.bias", (4 * d,)),
            (pre + "mlp.c_proj.weight", (4 * d, d)), (pre + "mlp.c_proj.bias", (d,)),
        ]
    shapes += [("ln_f.weight", (d,)), ("ln_f.bias", (d,))]
    return tuple(shapes)


def _flat(name: str, n: int) -> Tuple[Tuple[str, Tuple[int, ...]], ...]:
    return ((name, (n,)),)


WORKLOADS: Tuple[Workload, ...] = (
    Workload("cfg0_small_f32", "flat-1M", _flat("flat", 1_048_576), False, 4, "f32",
             0.05, 0.01, 0.0, 1.0, 0.1, 0.9, 1e-4, 1, 0, "fixed", (0, 0, 1, 1)),
    Workload("cfg1_resnet50", "ResNet-50-sized", _flat("flat", 25_557_032), False, 8, "bf16",
             0.05, 0.01, 0.0, 1.0, 0.1, 0.9, 1e-4, 10, 1, "fixed", (0, 0, 0, 1, 1, 1, 2, 2)),
    Workload("cfg2_bert_large", "BERT-large-sized", _flat("flat", 340_000_000), False, 16,
             "bf16", 0.02, 1e-3, 0.01, 100.0, 1e-3, 0.9, 0.01, 5, 2, "shuffle4x4"),
    Workload("cfg3_vgg16_asgd", "VGG-16-sized", _flat("flat", 138_357_544), False, 32, "bf16",
             0.05, 0.01, 0.0, 1.0, 0.01, 0.9, 5e-4, 3, 3, "asgd"),
    Workload("cfg4_gpt2_medium", "GPT-2-medium per-layer list", gpt2_medium_shapes(), True, 16,
             "bf16", 0.02, 1e-3, 0.0, 1.0, 3e-4, 0.9, 0.1, 5, 4, "random_2_8"),
)

BY_NAME: Dict[str, Workload] = {w.name: w for w in WORKLOADS}


def scaled(workload: Workload, n: int) -> Workload:
    """The same workload on a flat tensor of ``n`` elements (for small parity
    cases and bounded CPU samples)."""
    return dataclasses.replace(workload, shapes=_flat("flat", n), multi_tensor=False)


def reduced_list(workload: Workload, layers: int, vocab: int) -> Workload:
    """A tensor-list workload with the same tensor kinds but fewer layers and a
    smaller vocabulary (small cases for profiler captures)."""
    return dataclasses.replace(workload, shapes=gpt2_medium_shapes(layers, vocab))


def _generator(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def make_params(workload: Workload, device="cpu") -> List[torch.Tensor]:
    """One fp32 tensor per entry of ``workload.shapes`` (flat, 1-D)."""
    out = []
    for t, size in enumerate(workload.sizes):
        g = _generator(device, stream_seed(workload.seed, STREAM_PARAMS, t, 0))
        p = torch.empty(size, dtype=torch.float32, device=device)
        p.normal_(0.0, workload.param_std, generator=g)
        out.append(p)
    return out


def make_momentum(workload: Workload, device="cpu") -> List[torch.Tensor]:
    return [torch.zeros(size, dtype=torch.float32, device=device) for size in workload.sizes]


def fill_grads(workload: Workload, step: int, worker: int, out: Sequence[torch.Tensor]) -> None:
    """Write worker ``worker``'s gradient for round ``step`` into ``out`` (one
    tensor per parameter tensor, of the workload's gradient dtype)."""
    device = out[0].device
    g = _generator(device, stream_seed(workload.seed, STREAM_GRADS, step, worker))
    # Chunked so that the fp32 staging never exceeds 64 Mi elements.
    chunk = 1 << 26
    for dst in out:
        for start in range(0, dst.numel(), chunk):
            stop = min(dst.numel(), start + chunk)
            x = torch.empty(stop - start, dtype=torch.float32, device=device)
            x.normal_(0.0, workload.grad_std, generator=g)
            if workload.outlier_prob > 0.0:
                u = torch.empty(stop - start, dtype=torch.float32, device=device)
                u.uniform_(0.0, 1.0, generator=g)
                x = torch.where(u < workload.outlier_prob, x * workload.outlier_scale, x)
            dst[start:stop].copy_(x)       # rounds to bf16 (nearest even) if needed


def make_grads(workload: Workload, step: int, device="cpu") -> List[List[torch.Tensor]]:
    """``grads[w][t]``: gradient of worker w for parameter tensor t at ``step``."""
    dt = workload.torch_grad_dtype()
    grads = []
    for w in range(workload.W):
        bufs = [torch.empty(size, dtype=dt, device=device) for size in workload.sizes]
        fill_grads(workload, step, w, bufs)
        grads.append(bufs)
    return grads
