"""Seeded synthetic workloads shaped like the paper's training runs.

Holds only input generation (configs, x0 and per-step gradients) and none of
the optimizer's arithmetic, so the CUDA library's tests, the benchmark and the
CPU oracle's tests can all draw the same inputs from here.  The paper trains
WRN-40-8 on CIFAR-100 and ResNet-50 on ImageNet with 8 workers and momentum 0.9
(Section 5.1); those datasets are stood in for by random vectors with the same
parameter counts, worker counts, momentum and compression ratios.  Gradients
are exogenous draws, not gradients of a loss at x.

Values are drawn with torch's generator of the device they are produced on, so
a parity test must generate once and hand the same numbers to both sides.
"""
from dataclasses import dataclass, replace
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    d: int
    n_workers: int
    block_size: int
    R1: int            # ratio of the per-step compressor of the update
    R2: int            # ratio of the error-reset compressor
    H: int
    eta: float
    beta: float
    steps: int
    grad_kind: str     # "shared+noise" | "iid" | "student_t3"
    grad_shared_std: float = 0.0
    grad_noise_std: float = 0.0
    seed: int = 0

    @property
    def n_blocks(self):
        return (self.d + self.block_size - 1) // self.block_size

    @property
    def overall_ratio(self):
        """Overall compression ratio R_C = 1 / (1/R1 + 1/(R2 H)) (Section 5.1; R1 = 0 means no per-step part)."""
        inv = (1.0 / self.R1 if self.R1 else 0.0) + 1.0 / (self.R2 * self.H)
        return 1.0 / inv

    @property
    def comm_bytes_per_worker_step(self):
        """fp32 bytes a worker would put on the wire per step in a real deployment (average over H steps)."""
        return 4.0 * self.d / self.overall_ratio

    def scaled(self, d, steps=None):
        """Same hyper-parameters on a shorter vector (for quick tests)."""
        return replace(self, d=int(d), steps=self.steps if steps is None else int(steps),
                       name=f"{self.name}@d={int(d)}")


# N(0, v) in the workload descriptions is read as mean 0, variance v.
CONFIGS = {
    1: Workload("cfg1_d1M_n8_R4_H4_nomom", 1_048_576, 8, 256, 4, 4, 4, 0.1, 0.0, 20,
                "shared+noise", 1.0, 0.5),
    2: Workload("cfg2_wrn40x8_n8_R32_H8", 35_748_708, 8, 512, 32, 32, 8, 0.1, 0.9, 100,
                "shared+noise", 0.1, 0.05),
    3: Workload("cfg3_resnet50_n16_R256_16_H4", 25_557_032, 16, 1024, 256, 16, 4, 0.1, 0.9, 100,
                "iid", 0.0, 0.1),
    4: Workload("cfg4_resnet50_n8_R1024_H1", 25_557_032, 8, 256, 1024, 1024, 1, 0.05, 0.9, 100,
                "student_t3", 0.0, 0.01),
    5: Workload("cfg5_bertlarge_n8_R64_H8", 335_141_888, 8, 2048, 64, 64, 8, 1e-3, 0.9, 50,
                "iid", 0.0, 1e-3 ** 0.5),
}

# The paper's own tuned settings for WRN-40-8 (Appendix C, CSER rows), on the WRN-40-8-sized vector:
# overall ratio -> (R1 = its R_C2, R2 = its R_C1, H).
PAPER_TUNED = {
    rc: replace(CONFIGS[2], name=f"wrn40x8_paper_tuned_RC{rc}_R{r1}_{r2}_H{h}", R1=r1, R2=r2, H=h)
    for rc, (r1, r2, h) in {32: (64, 8, 8), 256: (512, 16, 32), 1024: (2048, 32, 64)}.items()
}


def _gen(device, *words):
    g = torch.Generator(device=device)
    s = 0x9E3779B97F4A7C15
    for w in words:
        s = (s * 6364136223846793005 + int(w) + 1442695040888963407) & 0x7FFFFFFFFFFFFFFF
    g.manual_seed(s)
    return g


def x0(w: Workload, device="cpu"):
    """Initial model x-hat_0 ~ N(0, 1), one [d] fp32 vector shared by all workers."""
    return torch.randn(w.d, generator=_gen(device, w.seed, 0xA0), device=device, dtype=torch.float32)


def gradients(w: Workload, t: int, device="cpu", out=None):
    """g_t as an [n, d] fp32 tensor, redrawn for every step t (1-based)."""
    n, d = w.n_workers, w.d
    if out is None:
        out = torch.empty((n, d), device=device, dtype=torch.float32)
    gen = _gen(device, w.seed, 0xB0, t)
    if w.grad_kind == "shared+noise":
        a = torch.randn(d, generator=gen, device=device, dtype=torch.float32) * w.grad_shared_std
        for i in range(n):
            out[i].normal_(0.0, w.grad_noise_std, generator=gen).add_(a)
    elif w.grad_kind == "iid":
        for i in range(n):
            out[i].normal_(0.0, w.grad_noise_std, generator=gen)
    elif w.grad_kind == "student_t3":
        for i in range(n):
            z = torch.randn((4, d), generator=gen, device=device, dtype=torch.float32)
            den = (z[1:].square().sum(0) / 3.0).sqrt_()
            out[i] = z[0].div_(den).mul_(w.grad_noise_std)
    else:
        raise ValueError(w.grad_kind)
    return out
