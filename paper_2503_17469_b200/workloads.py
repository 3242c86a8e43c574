"""Seeded synthetic workloads: tensor shapes, bucket layout, throughput draws, buffers.

This module holds no arithmetic of the method (no weighting, update or controller rule).  It only
decides WHAT the inputs are, so that the CUDA library and its CPU checker can be fed the same bits:
model tensor shapes (the models contribute shapes only; gradients are random), the packing of
tensors into contiguous buckets, heterogeneous worker throughputs, and the random buffers.
All randomness comes from a ``torch.Generator`` seeded by the caller.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import torch

BUCKET_BYTES = 25 * 1024 * 1024   # gradient bytes per bucket
TENSOR_ALIGN_BYTES = 16           # every tensor starts on a 16-byte boundary inside its bucket
BUCKET_ALIGN_BYTES = 256          # every bucket starts on a 256-byte boundary inside the flat buffer
BASE_SEED = 0x0517


# ------------------------------------------------------------------------------------------------
# Model tensor shapes (architecture rules of ResNet and VGG; totals asserted)
# ------------------------------------------------------------------------------------------------

def _bn(c: int) -> List[Tuple[int, ...]]:
    return [(c,), (c,)]


def resnet18_shapes() -> List[Tuple[int, ...]]:
    s: List[Tuple[int, ...]] = [(64, 3, 7, 7)] + _bn(64)
    cin = 64
    for stage, w in enumerate((64, 128, 256, 512)):
        for blk in range(2):
            s += [(w, cin, 3, 3)] + _bn(w) + [(w, w, 3, 3)] + _bn(w)
            if blk == 0 and stage > 0:
                s += [(w, cin, 1, 1)] + _bn(w)
            cin = w
    s += [(1000, 512), (1000,)]
    assert len(s) == 62 and sum(math.prod(t) for t in s) == 11_689_512
    return s


def resnet50_shapes() -> List[Tuple[int, ...]]:
    s: List[Tuple[int, ...]] = [(64, 3, 7, 7)] + _bn(64)
    cin = 64
    for w, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for blk in range(blocks):
            s += [(w, cin, 1, 1)] + _bn(w) + [(w, w, 3, 3)] + _bn(w) + [(4 * w, w, 1, 1)] + _bn(4 * w)
            if blk == 0:
                s += [(4 * w, cin, 1, 1)] + _bn(4 * w)
            cin = 4 * w
    s += [(1000, 2048), (1000,)]
    assert len(s) == 161 and sum(math.prod(t) for t in s) == 25_557_032
    return s


def vgg16_shapes() -> List[Tuple[int, ...]]:
    s: List[Tuple[int, ...]] = []
    cin = 3
    for w in (64, 64, 128, 128, 256, 256, 256, 512, 512, 512, 512, 512, 512):
        s += [(w, cin, 3, 3), (w,)]
        cin = w
    for fin, fout in ((25088, 4096), (4096, 4096), (4096, 1000)):
        s += [(fout, fin), (fout,)]
    assert len(s) == 32 and sum(math.prod(t) for t in s) == 138_357_544
    return s


# ------------------------------------------------------------------------------------------------
# Bucket layout
# ------------------------------------------------------------------------------------------------

@dataclass
class Bucket:
    start: int                 # element offset of the bucket in the flat buffer
    n: int                     # elements in the bucket, padding included
    tensors: List[Tuple[int, int, int]] = field(default_factory=list)  # (tensor index, offset in bucket, numel)


@dataclass
class Layout:
    buckets: List[Bucket]
    total: int                 # elements of the flat buffer, padding included
    numel: int                 # real parameters

    def tensor_slices(self):
        """(tensor index, flat start, numel) for every tensor."""
        for bk in self.buckets:
            for ti, off, ne in bk.tensors:
                yield ti, bk.start + off, ne


def _round_up(x: int, m: int) -> int:
    return (x + m - 1) // m * m


def pack_buckets(numels: Sequence[int], grad_elem_bytes: int, bucket_bytes: Optional[int] = BUCKET_BYTES) -> Layout:
    """Whole tensors in declaration order; a bucket closes when the next tensor would push its
    gradient bytes past ``bucket_bytes`` (an oversize tensor is a bucket of its own).
    ``bucket_bytes=None`` gives one flat bucket.  Offsets are in elements and keep every tensor
    16-byte aligned for the narrowest buffer (the gradient) and every bucket 256-byte aligned."""
    t_align = TENSOR_ALIGN_BYTES // grad_elem_bytes
    b_align = BUCKET_ALIGN_BYTES // grad_elem_bytes
    cap = None if bucket_bytes is None else bucket_bytes // grad_elem_bytes
    buckets: List[Bucket] = []
    cur = Bucket(start=0, n=0)
    for ti, ne in enumerate(numels):
        off = _round_up(cur.n, t_align)
        if cap is not None and cur.tensors and off + ne > cap:
            buckets.append(cur)
            cur = Bucket(start=_round_up(cur.start + cur.n, b_align), n=0)
            off = 0
        cur.tensors.append((ti, off, ne))
        cur.n = off + ne
    buckets.append(cur)
    total = _round_up(buckets[-1].start + buckets[-1].n, b_align)
    return Layout(buckets=buckets, total=total, numel=int(sum(numels)))


# ------------------------------------------------------------------------------------------------
# Workload configurations
# ------------------------------------------------------------------------------------------------

@dataclass
class Config:
    name: str
    index: int
    K: int
    shapes: List[Tuple[int, ...]]
    global_batch: int
    grad_dtype: str            # "f32" | "bf16"
    mode: str                  # "bsp" | "asp"
    steps: int
    rebatch_every: int         # 0 = once before the first step only
    lr: float = 0.1
    momentum: float = 0.9
    weight_decay: float = 0.0
    deadband: float = 0.10
    ewma_alpha: float = 1.0
    grad_std: Optional[float] = None     # None = per-tensor log-uniform in [1e-5, 1e-2]
    param_std: float = 0.05
    bucketed: bool = True
    throughputs: Optional[Tuple[float, ...]] = None   # fixed list, else drawn with an 8x ratio
    ratio: float = 8.0

    @property
    def numels(self) -> List[int]:
        return [math.prod(t) for t in self.shapes]

    @property
    def P(self) -> int:
        return sum(self.numels)

    @property
    def b_min(self) -> int:
        return max(1, (self.global_batch // self.K) // 8)

    @property
    def b_max(self) -> int:
        return 3 * self.global_batch // self.K

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index

    def layout(self) -> Layout:
        eb = 2 if self.grad_dtype == "bf16" else 4
        return pack_buckets(self.numels, eb, BUCKET_BYTES if self.bucketed else None)

    def bytes_per_param(self, with_lp: bool = False) -> int:
        """Bytes the method must move per parameter per step (reads + writes)."""
        gb = 2 if self.grad_dtype == "bf16" else 4
        if self.mode == "asp":
            return gb + 8 + (8 if self.momentum != 0 else 0) + (2 if with_lp else 0)
        return gb * self.K + 16 + (2 if with_lp else 0)


def config(name: str) -> Config:
    """The five synthetic configurations plus the fp32 twin of the mixed-precision one."""
    if name == "tiny":
        return Config("tiny", 0, 4, [(1 << 20,)], 64, "f32", "bsp", steps=10, rebatch_every=0,
                      grad_std=1e-3, bucketed=False, throughputs=(1.0, 2.0, 4.0, 8.0))
    if name == "resnet18":
        return Config("resnet18", 1, 8, resnet18_shapes(), 256, "f32", "bsp", steps=100, rebatch_every=10)
    if name == "resnet50_bf16":
        return Config("resnet50_bf16", 2, 16, resnet50_shapes(), 512, "bf16", "bsp", steps=20, rebatch_every=10)
    if name == "resnet50_f32":
        return Config("resnet50_f32", 2, 16, resnet50_shapes(), 512, "f32", "bsp", steps=20, rebatch_every=10)
    if name == "resnet50_asp":
        return Config("resnet50_asp", 3, 16, resnet50_shapes(), 512, "f32", "asp", steps=1000, rebatch_every=1,
                      momentum=0.0, grad_std=1e-3)
    if name == "vgg16":
        return Config("vgg16", 4, 32, vgg16_shapes(), 1024, "f32", "bsp", steps=50, rebatch_every=1,
                      grad_std=1e-4)
    raise KeyError(name)


CONFIG_NAMES = ("tiny", "resnet18", "resnet50_bf16", "resnet50_f32", "resnet50_asp", "vgg16")


def scaled(cfg: Config, numel_cap: int) -> Config:
    """The same configuration with every tensor shrunk so that no tensor exceeds ``numel_cap``
    elements (shape structure, tensor count and ragged sizes are kept).  For checks on the CPU."""
    shapes = []
    for t in cfg.shapes:
        ne = math.prod(t)
        shapes.append((min(ne, numel_cap + (ne % 7)),))
    c = Config(**{**cfg.__dict__, "shapes": shapes})
    return c


# ------------------------------------------------------------------------------------------------
# Throughputs
# ------------------------------------------------------------------------------------------------

def draw_throughputs(K: int, gen: torch.Generator, ratio: float = 8.0) -> List[float]:
    """Log-uniform worker throughputs rescaled so that the slowest is 1 and the fastest ``ratio``."""
    if K == 1:
        return [1.0]
    u = torch.rand(K, generator=gen, dtype=torch.float64)
    u = (u - u.min()) / (u.max() - u.min())
    return [float(ratio ** x) for x in u.tolist()]


def jitter_throughputs(base: Sequence[float], gen: torch.Generator, amp: float = 0.2) -> List[float]:
    """Multiplicative noise of +-amp around the base throughputs."""
    u = torch.rand(len(base), generator=gen, dtype=torch.float64).tolist()
    return [float(t * (1.0 + amp * (2.0 * x - 1.0))) for t, x in zip(base, u)]


def interference(base: Sequence[float], step: int, first: int = 15, last: int = 34, n_hit: int = 4) -> List[float]:
    """Dynamic-interference phase: the ``n_hit`` fastest workers run at half speed in [first, last]."""
    t = list(base)
    if first <= step <= last:
        order = sorted(range(len(t)), key=lambda k: (-base[k], k))[:n_hit]
        for k in order:
            t[k] = base[k] * 0.5
    return t


def pick_worker(u: float, rates: Sequence[float]) -> int:
    """Inverse-CDF draw of the next arriving worker from its iteration rates and a uniform u."""
    total = float(sum(rates))
    acc = 0.0
    for k, r in enumerate(rates):
        acc += r / total
        if u < acc:
            return k
    return len(rates) - 1


# ------------------------------------------------------------------------------------------------
# Buffers
# ------------------------------------------------------------------------------------------------

@dataclass
class Buffers:
    layout: Layout
    theta: torch.Tensor                    # float32, layout.total
    v: Optional[torch.Tensor]              # float32, layout.total, zeros
    grads: List[torch.Tensor]              # K tensors, float32 or bfloat16, layout.total
    grad_std: List[float]                  # per tensor


def make_buffers(cfg: Config, device, gen: Optional[torch.Generator] = None, n_grads: Optional[int] = None) -> Buffers:
    """Random parameters, zero momentum and K gradient buffers in the bucket layout.  Padding
    elements are zero in every buffer.  Gradients of the bf16 configuration are drawn in float32
    and rounded once to bfloat16 by torch; both sides consume the rounded values."""
    device = torch.device(device)
    if gen is None:
        gen = torch.Generator(device=device)
        gen.manual_seed(cfg.seed)
    lay = cfg.layout()
    K = cfg.K if n_grads is None else n_grads
    gdt = torch.bfloat16 if cfg.grad_dtype == "bf16" else torch.float32
    n_t = len(cfg.shapes)
    if cfg.grad_std is None:
        e = torch.rand(n_t, generator=gen, dtype=torch.float64, device=device).cpu()
        stds = [float(10.0 ** (-5.0 + 3.0 * x)) for x in e.tolist()]
    else:
        stds = [cfg.grad_std] * n_t
    # per-element standard deviation of the gradient; zero on padding
    std_vec = torch.zeros(lay.total, dtype=torch.float32, device=device)
    for ti, start, ne in lay.tensor_slices():
        std_vec[start:start + ne] = stds[ti]
    pad = std_vec == 0          # padding stays exactly +0 in every buffer
    theta = torch.empty(lay.total, dtype=torch.float32, device=device).normal_(0.0, cfg.param_std, generator=gen)
    theta.masked_fill_(pad, 0.0)
    v = torch.zeros(lay.total, dtype=torch.float32, device=device)
    grads = []
    for _ in range(K):
        g = torch.empty(lay.total, dtype=torch.float32, device=device).normal_(0.0, 1.0, generator=gen)
        g.mul_(std_vec).masked_fill_(pad, 0.0)
        grads.append(g if gdt == torch.float32 else g.to(gdt))
    del std_vec, pad
    return Buffers(layout=lay, theta=theta, v=v, grads=grads, grad_std=stds)
