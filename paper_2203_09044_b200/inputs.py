"""Seeded synthetic gradient generators shared by the tests, the smoke check and the benchmark.

Nothing here belongs to the CO3 method: these functions only draw the inputs (fp32 gradients
with the shapes and value distributions of the benchmark configurations) that both the CUDA
library and the CPU oracle are then given.  The paper measures on CIFAR-10 training gradients,
which it models as i.i.d. generalized normal per layer; these draws stand in for them.

A zero-location generalized normal sample with shape beta and scale alpha is
x = alpha * sgn * G**(1/beta) with G ~ Gamma(1/beta, 1) and sgn a fair sign.
"""
import math
from dataclasses import dataclass, field
from typing import List, Optional

import torch


def gennorm(n: int, beta: float, alpha, gen: torch.Generator, device="cpu") -> torch.Tensor:
    """n fp32 samples; alpha is a float or a length-n tensor of per-element scales."""
    conc = torch.full((n,), 1.0 / beta, dtype=torch.float32, device=device)
    g = torch._standard_gamma(conc, generator=gen)
    x = g.pow_(1.0 / beta)
    sgn = torch.randint(0, 2, (n,), generator=gen, device=device, dtype=torch.int8)
    x = torch.where(sgn.bool(), x, -x)
    return (x * alpha).to(torch.float32)


def aligned_ld(d: int) -> int:
    """Row stride in elements that puts every row on a 16 KiB boundary."""
    return (d + 4095) // 4096 * 4096


def resnet18_cifar_tensor_sizes(num_classes: int = 10) -> List[int]:
    """Element counts of the parameter tensors of a CIFAR-style ResNet-18, in definition order."""
    sizes = [64 * 3 * 3 * 3, 64, 64]                       # stem conv + BN weight/bias
    for _ in range(2):                                     # stage 1: two basic blocks, 64 ch
        sizes += [64 * 64 * 9, 64, 64, 64 * 64 * 9, 64, 64]
    for c in (128, 256, 512):                              # stages 2-4
        h = c // 2
        sizes += [c * h * 9, c, c, c * c * 9, c, c, c * h, c, c]   # block 1 with 1x1 shortcut
        sizes += [c * c * 9, c, c, c * c * 9, c, c]                # block 2
    sizes += [num_classes * 512, num_classes]
    return sizes


@dataclass
class Workload:
    """One benchmark configuration: sizes, format, and a gradient(t) draw per iteration."""
    name: str
    index: int
    n_users: int
    d: int
    seg_offsets: List[int]
    exp_bits: int
    mant_bits: int
    beta: float
    iters: int
    gamma: float = 0.9
    seg_alpha: Optional[List[float]] = None     # per-segment GenNorm scale
    outlier_prob: float = 0.0
    outlier_gain: float = 1.0
    row_stride: Optional[int] = None            # elements between user rows; None = d rounded up to 4
    _alpha_vec: dict = field(default_factory=dict, repr=False)

    @property
    def ld(self) -> int:
        return self.row_stride if self.row_stride is not None else (self.d + 3) // 4 * 4

    def align_rows(self) -> "Workload":
        """Start every user's row on a 16 KiB boundary (what the benchmark uses: with rows that start
        in the middle of a 128-byte line every 512-byte warp access touches five lines, not four)."""
        self.row_stride = aligned_ld(self.d)
        return self

    @property
    def n_segments(self) -> int:
        return len(self.seg_offsets) - 1

    def _alpha(self, device):
        key = str(device)
        if key not in self._alpha_vec:
            a = torch.tensor(self.seg_alpha, dtype=torch.float32, device=device)
            if len(self.seg_alpha) == 1:
                self._alpha_vec[key] = float(self.seg_alpha[0])
            else:
                sizes = torch.tensor([self.seg_offsets[i + 1] - self.seg_offsets[i]
                                      for i in range(self.n_segments)], device=device)
                self._alpha_vec[key] = torch.repeat_interleave(a, sizes)
        return self._alpha_vec[key]

    def gradient(self, t: int, device="cpu", users=None) -> torch.Tensor:
        """[n_users][ld] fp32 gradients of iteration t (row padding is zero)."""
        users = range(self.n_users) if users is None else users
        out = torch.zeros((len(users), self.ld), dtype=torch.float32, device=device)
        for r, u in enumerate(users):
            gen = torch.Generator(device=device)
            gen.manual_seed(1_000_003 * self.index + 1009 * t + u)
            x = gennorm(self.d, self.beta, self._alpha(device), gen, device)
            if self.outlier_prob > 0.0:
                mask = torch.rand(self.d, generator=gen, device=device) < self.outlier_prob
                x = torch.where(mask, x * self.outlier_gain, x)
            out[r, :self.d] = x
        return out


def _equal_segments(d: int, s: int) -> List[int]:
    base, extra = divmod(d, s)
    off = [0]
    for i in range(s):
        off.append(off[-1] + base + (1 if i < extra else 0))
    return off


def workload(index: int, d: Optional[int] = None, n_users: Optional[int] = None) -> Workload:
    """The benchmark configurations 0-3; d / n_users override the size for scaled-down tests."""
    if index == 0:
        dd = d or 1 << 20
        return Workload("c0_flat_2p20_e4m3", 0, n_users or 1, dd, [0, dd], 4, 3, 1.0, 4,
                        seg_alpha=[1e-3])
    if index == 1:
        sizes = resnet18_cifar_tensor_sizes()
        if d is not None:                     # scaled-down: keep the tensor-size mix
            f = d / sum(sizes)
            sizes = [max(1, int(round(s * f))) for s in sizes]
        off = [0]
        for s in sizes:
            off.append(off[-1] + s)
        gen = torch.Generator().manual_seed(1_000_003)
        expo = torch.rand(len(sizes), generator=gen, dtype=torch.float64) * 2.0 - 4.0
        alphas = [float(10.0 ** e) for e in expo]
        return Workload("c1_resnet18_e4m3", 1, n_users or 8, off[-1], off, 4, 3, 0.8, 20,
                        seg_alpha=alphas)
    if index == 2:
        dd = d or 14_728_266
        return Workload("c2_16seg_e3m2", 2, n_users or 16, dd, _equal_segments(dd, 16), 3, 2, 1.2,
                        20, seg_alpha=[5e-4])
    if index == 3:
        dd = d or 124_439_808
        return Workload("c3_gpt2s_heavytail_e4m3", 3, n_users or 4, dd, [0, dd], 4, 3, 0.6, 10,
                        seg_alpha=[2e-4], outlier_prob=1e-3, outlier_gain=100.0)
    raise ValueError("workload index must be 0..3")


def sweep_cell(d: int, n_users: int, beta: float, exp_bits: int, mant_bits: int) -> Workload:
    """One cell of the size/users/shape/format sweep (single segment, alpha = 1e-3)."""
    idx = 4000 + int(math.log2(d)) * 100 + n_users + int(beta * 10) * 7 + exp_bits
    return Workload(f"sweep_d{d}_u{n_users}_b{beta}_e{exp_bits}m{mant_bits}", idx, n_users, d,
                    [0, d], exp_bits, mant_bits, beta, 5, seg_alpha=[1e-3])
