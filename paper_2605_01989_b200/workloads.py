"""Seeded synthetic inputs: tensor shapes, gradient values and loss-model parameters.

This module holds none of the method's arithmetic.  It only states *what goes in*: the parameter-tensor
shapes of the architectures the workloads are named after (written from the architectures' own rules),
Gaussian gradient values from a seeded generator, and the conversion of loss rates into the integer
thresholds that both the CUDA library and the CPU checker consume unchanged.
"""
import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import torch

TWO32 = 1 << 32


# ----------------------------------------------------------------------------------------------------------
# Tensor shapes
# ----------------------------------------------------------------------------------------------------------
def resnet50_numel() -> List[int]:
    """ResNet-50 with a 1000-way classifier: 161 parameter tensors, 25,557,032 parameters."""
    out = [64 * 3 * 7 * 7, 64, 64]                      # stem convolution + batch norm (weight, bias)
    cin = 64
    for planes, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for b in range(blocks):
            out += [cin * planes, planes, planes]               # 1x1 reduce + BN
            out += [planes * planes * 9, planes, planes]        # 3x3 + BN
            out += [planes * planes * 4, planes * 4, planes * 4]  # 1x1 expand + BN
            if b == 0:
                out += [cin * planes * 4, planes * 4, planes * 4]  # projection shortcut + BN
            cin = planes * 4
    out += [2048 * 1000, 1000]
    return out


def bert_large_numel() -> List[int]:
    """BERT-large encoder with pooler: 391 tensors, 335,141,888 parameters."""
    h, ff = 1024, 4096
    out = [30522 * h, 512 * h, 2 * h, h, h]
    for _ in range(24):
        out += [h * h, h] * 4          # query, key, value, attention output (weight, bias)
        out += [h, h]                  # layer norm
        out += [h * ff, ff, ff * h, h]  # feed-forward
        out += [h, h]                  # layer norm
    out += [h * h, h]
    return out


def gpt2_xl_numel() -> List[int]:
    """GPT-2 XL (48 layers, width 1600): 580 tensors, 1,557,611,200 parameters."""
    h = 1600
    out = [50257 * h, 1024 * h]
    for _ in range(48):
        out += [h, h, h * 3 * h, 3 * h, h * h, h, h, h, h * 4 * h, 4 * h, 4 * h * h, h]
    out += [h, h]
    return out


# ----------------------------------------------------------------------------------------------------------
# Loss-model parameters -> integer thresholds (a draw u in [0, 2^32) drops iff u < threshold)
# ----------------------------------------------------------------------------------------------------------
def threshold(prob: float) -> int:
    return min(TWO32, max(0, int(math.floor(prob * TWO32))))


@dataclass
class LossSpec:
    kind: str                       # "none" | "iid" | "ge" | "microburst"
    mean_loss: float = 0.0          # iid rate, or the burst chain's stationary loss
    mean_burst: float = 20.0        # ge: mean length of a run of drops, in packets
    window_frac: float = 0.05       # microburst: share of a worker's packets inside the window
    p_in: float = 0.30
    p_out: float = 0.001

    def thresholds(self, C: int) -> Dict[str, int]:
        """Field values of the loss-model struct, for a worker stream of C packets."""
        if self.kind == "none":
            return {}
        if self.kind == "iid":
            return {"t_drop": threshold(self.mean_loss)}
        if self.kind == "ge":
            # Simple Gilbert chain: every packet sent in the Bad state is dropped, none in Good.
            p_bg = 1.0 / self.mean_burst
            pi = self.mean_loss
            p_gb = p_bg * pi / (1.0 - pi) if pi < 1.0 else 1.0
            if p_gb > 1.0:
                raise ValueError("a mean loss of %g cannot be reached with bursts of mean length %g" % (pi, self.mean_burst))
            return {"t_gb": threshold(p_gb), "t_bg": threshold(p_bg), "t_init_bad": threshold(pi),
                    "t_drop_good": 0, "t_drop_bad": TWO32}
        if self.kind == "microburst":
            return {"window_len": min(C, int(math.ceil(self.window_frac * C))),
                    "t_drop_in": threshold(self.p_in), "t_drop_out": threshold(self.p_out)}
        raise ValueError(self.kind)


# ----------------------------------------------------------------------------------------------------------
# Workloads
# ----------------------------------------------------------------------------------------------------------
@dataclass
class Workload:
    name: str
    W: int
    dtype: str                      # "f32" | "bf16"
    payload_bytes: int
    numel: List[int]
    sigma: float
    loss: LossSpec
    seed: int
    bounds_ppm: Tuple[int, ...] = (8000,)
    round: int = 1
    note: str = ""

    @property
    def elem_size(self) -> int:
        return 4 if self.dtype == "f32" else 2

    @property
    def E(self) -> int:
        return self.payload_bytes // self.elem_size

    @property
    def N(self) -> int:
        return sum(self.numel)

    @property
    def C(self) -> int:
        return sum((n + self.E - 1) // self.E for n in self.numel)

    @property
    def M(self) -> int:
        return self.W * self.C

    def device_bytes(self) -> int:
        """Gradients + payload ring + fp32 aggregate + per-packet metadata and scratch."""
        return self.W * self.N * self.elem_size + self.M * self.payload_bytes + self.N * 4 + self.M * (32 + 4 + 8 + 8 + 8)


def config(i: int) -> Workload:
    """The five workloads: 0 flat 4 MiB fp32, 1 ResNet-50-shaped, 2 BERT-large-shaped bf16, 3 GPT-2-XL-shaped,
    4 one representative point of the size sweep."""
    if i == 0:
        return Workload("flat-1M-f32", 4, "f32", 1024, [1 << 20], 1e-3, LossSpec("iid", 0.01), 0)
    if i == 1:
        return Workload("resnet50-f32", 8, "f32", 1408, resnet50_numel(), 1e-3, LossSpec("ge", 0.01, 20.0), 1,
                        bounds_ppm=(24000,))
    if i == 2:
        return Workload("bert-large-bf16", 16, "bf16", 4096, bert_large_numel(), 1e-3,
                        LossSpec("microburst", window_frac=0.05, p_in=0.30, p_out=0.001), 2)
    if i == 3:
        return Workload("gpt2-xl-f32", 8, "f32", 4096, gpt2_xl_numel(), 1e-4, LossSpec("ge", 0.02, 20.0), 3,
                        bounds_ppm=(0, 10000, 50000, 100000))
    if i == 4:
        return sweep_point(1 << 24, 8, 4096, 0.05, "ge", 10)
    raise ValueError(i)


def sweep_point(buffer_bytes: int, W: int, payload_bytes: int, loss: float, kind: str, seed: int) -> Workload:
    spec = LossSpec("none") if loss == 0 else LossSpec(kind, loss, 20.0)
    return Workload("sweep-%dMB-W%d-P%d-%s%g-s%d" % (buffer_bytes >> 20, W, payload_bytes, kind, loss * 100, seed),
                    W, "f32", payload_bytes, [buffer_bytes // 4], 1e-3, spec, seed)


def sweep(max_device_bytes: Optional[int] = None) -> List[Workload]:
    """The cartesian sweep: buffer 1 MiB * 4^k (k = 0..5), W in {2, 8, 32}, payload {1024, 4096}, loss
    {0, 1, 5, 20} % iid and bursty, seeds 10..14.  Points above max_device_bytes are left out."""
    pts = []
    for k in range(6):
        for W in (2, 8, 32):
            for P in (1024, 4096):
                for loss in (0.0, 0.01, 0.05, 0.20):
                    for kind in (("iid",) if loss == 0 else ("iid", "ge")):
                        for seed in range(10, 15):
                            w = sweep_point((1 << 20) * 4 ** k, W, P, loss, kind, seed)
                            if max_device_bytes is None or w.device_bytes() <= max_device_bytes:
                                pts.append(w)
    return pts


def make_grads(wl: Workload, device="cpu", workers=None, elem_range: Optional[Tuple[int, int]] = None,
               out: Optional[torch.Tensor] = None) -> List[torch.Tensor]:
    """Worker w's flat gradient: N values N(0, sigma^2) from generator seed*1000 + w, cast to the workload's dtype.
    elem_range = (first, last): only that range of each worker's vector is kept (the whole vector is still drawn, so
    the values are those of the unsplit workload).  out: one tensor of len(workers) * (kept length) elements of the
    workload's dtype that receives the gradients back to back; the returned list then holds views into it."""
    ws = list(range(wl.W) if workers is None else workers)
    lo, hi = (0, wl.N) if elem_range is None else elem_range
    n = hi - lo
    res = []
    for k, w in enumerate(ws):
        g = torch.Generator(device=device)
        g.manual_seed(wl.seed * 1000 + w)
        x = torch.randn(wl.N, generator=g, device=device, dtype=torch.float32)
        x.mul_(wl.sigma)
        if elem_range is not None:
            x = x[lo:hi]
        if out is not None:
            view = out[k * n:(k + 1) * n]
            view.copy_(x)                      # casts to bf16 where the workload asks for it
            res.append(view)
        else:
            if wl.dtype == "bf16":
                x = x.to(torch.bfloat16)
            elif elem_range is not None:
                x = x.clone()                  # let go of the whole vector
            res.append(x)
        del x
    return res
