"""Seeded synthetic parameter sets shaped like the paper's models.

Only shapes, layouts and random value recipes live here: nothing of the
optimizer's arithmetic.  Both the CUDA path and the CPU oracle are fed from
these generators (the oracle receives copies of the very same tensors).

The five workloads (index 0..4) follow the paper's evaluation models
(Section 9: ResNet-50 25.6 M and VGG-16 138 M parameters; ViT is named in the
abstract) plus a single flat tensor and a 1 B-parameter stress set.  Only the
*parameter-tensor shapes* of those public architectures are used; values are
random: "N(0, s)" means standard deviation s.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import torch

MASTER_SEED = 20260107


@dataclass
class Workload:
    name: str
    index: int
    shapes: list                    # tensor shapes, in model order
    hyper: dict                     # keyword arguments of NovakOptimizer / oracle Config
    steps: int
    grad_dtype: torch.dtype = torch.float32
    misalign: bool = False          # every third tensor starts 1..3 elements off a 16-B boundary
    init: str = "normal"            # how parameters are drawn, see init_params
    grad_zero_frac: float = 0.0
    notes: str = ""
    numel: list = field(init=False)

    def __post_init__(self):
        self.numel = [int(math.prod(s)) for s in self.shapes]

    @property
    def total(self) -> int:
        return sum(self.numel)


_HYPER = dict(lr=1e-3, betas=(0.9, 0.999), eps=1e-8, weight_decay=1e-2,
              nesterov="approximation", lookahead_k=5, lookahead_alpha=0.5)


def resnet50_shapes():
    """conv / BN / fc parameter tensors of ResNet-50 (161 tensors, 25,557,032)."""
    shapes = [(64, 3, 7, 7), (64,), (64,)]
    inplanes = 64
    for planes, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for b in range(blocks):
            shapes += [(planes, inplanes, 1, 1), (planes,), (planes,),
                       (planes, planes, 3, 3), (planes,), (planes,),
                       (planes * 4, planes, 1, 1), (planes * 4,), (planes * 4,)]
            if b == 0:
                shapes += [(planes * 4, inplanes, 1, 1), (planes * 4,), (planes * 4,)]
            inplanes = planes * 4
    shapes += [(1000, 2048), (1000,)]
    return shapes


def vgg16_shapes():
    """13 conv 3x3 (+bias) and 3 fc (+bias) of VGG-16 (32 tensors, 138,357,544)."""
    shapes, cin = [], 3
    for cout in (64, 64, 128, 128, 256, 256, 256, 512, 512, 512, 512, 512, 512):
        shapes += [(cout, cin, 3, 3), (cout,)]
        cin = cout
    for fin, fout in ((25088, 4096), (4096, 4096), (4096, 1000)):
        shapes += [(fout, fin), (fout,)]
    return shapes


def vit_b16_shapes():
    """ViT-B/16 parameter tensors (152 tensors, 86,567,656)."""
    d, mlp = 768, 3072
    shapes = [(1, 1, d), (1, 197, d), (d, 3, 16, 16), (d,)]
    for _ in range(12):
        shapes += [(d,), (d,), (3 * d, d), (3 * d,), (d, d), (d,),
                   (d,), (d,), (mlp, d), (mlp,), (d, mlp), (d,)]
    shapes += [(d,), (d,), (1000, d), (1000,)]
    return shapes


def loguniform_sizes(n=1000, total=1_000_000_000, lo=1024, hi=16 * 2 ** 20, seed=MASTER_SEED):
    """n sizes, log-uniform in [lo, hi], rescaled so that they sum to `total`
    exactly (the residual goes to the largest tensor).  Sizes are not rounded
    to multiples of 4: ragged tails are part of the workload."""
    g = torch.Generator().manual_seed(seed + 5)
    u = torch.rand(n, generator=g, dtype=torch.float64)
    raw = torch.exp(math.log(lo) + u * (math.log(hi) - math.log(lo)))
    sizes = raw
    for _ in range(8):  # rescale + clamp until the clamps stop moving the sum
        sizes = (sizes * (total / sizes.sum())).clamp(lo, hi)
    sizes = sizes.floor().to(torch.int64)
    sizes[sizes.argmax()] += total - int(sizes.sum())
    assert int(sizes.sum()) == total and int(sizes.min()) >= lo
    return [(int(s),) for s in sizes]


def get_workload(index: int, scale: float = 1.0) -> Workload:
    """index 0..4 = the five benchmark configurations.  `scale` < 1 shrinks
    workload 4 (the 1 B set) for tests that cannot hold 20 GB."""
    if index == 0:
        return Workload("flat-1M", 0, [(1_048_576,)], dict(_HYPER), 20, init="normal",
                        notes="one flat tensor; N(0,0.05) params, N(0,1e-2) grads")
    if index == 1:
        return Workload("resnet50", 1, resnet50_shapes(), dict(_HYPER), 100, init="kaiming",
                        notes="Kaiming-normal weights, gamma=1, beta/bias=0; per-tensor grad scale")
    if index == 2:
        return Workload("vgg16", 2, vgg16_shapes(), dict(_HYPER), 50, init="kaiming",
                        notes="He-normal weights, zero biases; N(0,1e-3) grads")
    if index == 3:
        h = dict(_HYPER, lookahead_k=6)
        return Workload("vit-b16", 3, vit_b16_shapes(), h, 100, grad_dtype=torch.bfloat16,
                        init="vit", notes="N(0,0.02) weights; bf16 grads N(0,1e-3)")
    if index == 4:
        total = int(round(1_000_000_000 * scale))
        n = 1000 if scale == 1.0 else max(8, int(1000 * scale))
        hi = 16 * 2 ** 20 if scale == 1.0 else max(4096, int(16 * 2 ** 20 * scale * 4))
        return Workload("loguniform-1B" if scale == 1.0 else f"loguniform-{total}", 4,
                        loguniform_sizes(n, total, hi=hi), dict(_HYPER), 20,
                        misalign=True, grad_zero_frac=0.01,
                        notes="log-uniform sizes, ragged, every third tensor misaligned; 1% zero grads")
    raise ValueError(f"no workload {index}")


# ---------------------------------------------------------------------------
# Layout: every tensor is a view into one flat buffer, so that a whole set is
# one allocation (and one host<->device copy).
# ---------------------------------------------------------------------------
def element_offsets(wl: Workload):
    """Start of each tensor in the flat buffer, in elements.  Tensors start on
    256-byte boundaries of an fp32 buffer (64 elements); with `misalign`, every
    third tensor is pushed 1..3 elements further."""
    offs, cur = [], 0
    for i, n in enumerate(wl.numel):
        cur = (cur + 63) // 64 * 64
        if wl.misalign and i % 3 == 2:
            cur += 1 + (i // 3) % 3
        offs.append(cur)
        cur += n
    return offs, (cur + 63) // 64 * 64


def views(flat: torch.Tensor, wl: Workload):
    offs, _ = element_offsets(wl)
    return [flat[o:o + n] for o, n in zip(offs, wl.numel)]


def alloc_flat(wl: Workload, dtype, device, pin=False):
    _, total = element_offsets(wl)
    if pin:
        return torch.zeros(total, dtype=dtype, pin_memory=True)
    return torch.zeros(total, dtype=dtype, device=device)


def _gen(device, seed):
    return torch.Generator(device=device).manual_seed(seed)


def init_params(wl: Workload, flat: torch.Tensor):
    """Fills the flat fp32 parameter buffer in place (seeded)."""
    g = _gen(flat.device, MASTER_SEED + 1000 * wl.index)
    for shape, v in zip(wl.shapes, views(flat, wl)):
        if wl.init == "normal":
            v.normal_(0.0, 0.05, generator=g)
        elif wl.init == "kaiming":
            if len(shape) >= 2:
                fan_in = math.prod(shape[1:])
                v.normal_(0.0, math.sqrt(2.0 / fan_in), generator=g)
            else:
                v.zero_()
        elif wl.init == "vit":
            if len(shape) >= 2:
                v.normal_(0.0, 0.02, generator=g)
            else:
                v.zero_()
    if wl.init == "kaiming" and wl.name == "resnet50":
        # BN gamma = 1: the first 1-d tensor after every conv weight
        vs = views(flat, wl)
        for i, shape in enumerate(wl.shapes[:-2]):
            if len(shape) == 4:
                vs[i + 1].fill_(1.0)
    if wl.init == "vit":
        vs = views(flat, wl)
        for i in range(12):
            base = 4 + 12 * i
            vs[base].fill_(1.0)       # LN1 gamma
            vs[base + 6].fill_(1.0)   # LN2 gamma
        vs[4 + 144].fill_(1.0)        # final LN gamma


def grad_scales(wl: Workload):
    """Per-tensor gradient standard deviation."""
    if wl.name == "resnet50":
        g = torch.Generator().manual_seed(MASTER_SEED + 77)
        z = torch.randn(len(wl.shapes), generator=g, dtype=torch.float64).abs() * 1e-3
        return [max(float(x), 1e-6) for x in z]
    if wl.name in ("vgg16", "vit-b16"):
        return [1e-3] * len(wl.shapes)
    return [1e-2] * len(wl.shapes)


class GradSource:
    """Seeded gradient stream: fill(flat_fp32_scratch, out_flat) draws step after
    step from one generator, so a run is reproducible from (workload, seed)."""

    def __init__(self, wl: Workload, device, seed_offset=0):
        self.wl = wl
        self.gen = _gen(device, MASTER_SEED + 1000 * wl.index + 500 + seed_offset)
        self.scales = grad_scales(wl)
        self.uniform = len(set(self.scales)) == 1

    def fill(self, out_flat: torch.Tensor, scratch: torch.Tensor | None = None):
        """Writes one step's gradients into out_flat (fp32 or bf16 flat buffer)."""
        wl = self.wl
        tgt = out_flat if out_flat.dtype == torch.float32 else scratch
        if tgt is None:
            tgt = torch.empty(out_flat.shape, dtype=torch.float32, device=out_flat.device)
        if self.uniform:
            tgt.normal_(0.0, self.scales[0], generator=self.gen)
        else:
            for s, v in zip(self.scales, views(tgt, wl)):
                v.normal_(0.0, s, generator=self.gen)
        if wl.grad_zero_frac > 0:
            blk = 1 << 26
            for lo in range(0, tgt.numel(), blk):
                part = tgt[lo:lo + blk]
                mask = torch.rand(part.shape, generator=self.gen, device=part.device,
                                  dtype=torch.float32) < wl.grad_zero_frac
                part.masked_fill_(mask, 0.0)
        if tgt is not out_flat:
            out_flat.copy_(tgt)


def sample_indices(wl: Workload, small=65536, edge=4096, stride=997):
    """Flat-buffer element indices of a fixed sample: tensors up to `small`
    elements whole, the first and last `edge` elements of every other tensor
    and every `stride`-th element in between.  Also returns, per sampled
    element, its tensor and its offset inside the tensor."""
    offs, _ = element_offsets(wl)
    idx, tid, local = [], [], []
    for i, (o, n) in enumerate(zip(offs, wl.numel)):
        if n <= small:
            loc = torch.arange(n, dtype=torch.int64)
        else:
            loc = torch.cat([torch.arange(edge, dtype=torch.int64),
                             torch.arange(edge, n - edge, stride, dtype=torch.int64),
                             torch.arange(n - edge, n, dtype=torch.int64)])
        idx.append(loc + o)
        local.append(loc)
        tid.append(torch.full_like(loc, i))
    return torch.cat(idx), torch.cat(tid), torch.cat(local)
