"""Seeded synthetic gradients shaped like the paper's workloads.

This module only draws random inputs; it holds none of the method's
arithmetic, so both the CUDA path and the CPU oracle may be fed from it.
The paper trains ResNet-18 on CIFAR-10 (Section 5.1: a 44 MB model, k = 300000
for top-k); without the dataset, gradients are replaced by random vectors of
the same sizes with heavy-tailed or layer-structured magnitudes.

Every draw is a pure function of (workload id, step, worker) through
``torch.Generator.manual_seed`` on the requested device.  CPU and CUDA
generators give different streams, so a comparison always draws once and
copies the bits to the other side.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch

BASE_SEED = 190505957

# ResNet-18 (CIFAR-10 head excluded: the 1000-way layer is kept so d = 11,689,512)
# parameter tensors in order; used as contiguous "layer slices" of workload 2.
RESNET18_SLICES = (
    9408, 64, 64,
    36864, 64, 64, 36864, 64, 64,
    36864, 64, 64, 36864, 64, 64,
    73728, 128, 128, 147456, 128, 128, 8192, 128, 128,
    147456, 128, 128, 147456, 128, 128,
    294912, 256, 256, 589824, 256, 256, 32768, 256, 256,
    589824, 256, 256, 589824, 256, 256,
    1179648, 512, 512, 2359296, 512, 512, 131072, 512, 512,
    2359296, 512, 512, 2359296, 512, 512,
    512000, 1000,
)
assert len(RESNET18_SLICES) == 62 and sum(RESNET18_SLICES) == 11_689_512


@dataclass(frozen=True)
class Q:
    op: str = "identity"     # identity | sign1 | topk | qsgd | clip | rsparse | ternary
    chunk: int = 0           # sign1 / qsgd / rsparse: entries per chunk; sign1 with 0: one factor for the whole vector
    k: int = 0
    levels: int = 0
    norm: int = 1            # sign1: scale from l1 (1) or l2 (2) magnitudes
    keep_one_in: int = 0     # rsparse: S, an entry survives with probability 1/S
    scaled: int = 0          # rsparse: 1 = survivors are multiplied by S (unbiased, no contraction)
    bits: int = 0            # clip: low bits of every number set to zero (16 or 24)


@dataclass(frozen=True)
class Workload:
    wid: int                 # 1..5 = the listed configurations; 6.. = added ones
    name: str
    n: int
    d: int
    steps: int
    dist: str                # normal | layered | laplace | student_t | hetero
    worker_q: Q
    server_q: Q
    gamma: float = 0.1
    seed: int = BASE_SEED    # Philox seed handed to the randomised Q
    compensate: bool = True  # False: the compressed methods of Section 5.1 that keep no error

    def scaled(self, d: int, n: int | None = None, steps: int | None = None) -> "Workload":
        """Same recipe at another size; top-k keeps its fraction of d."""
        def rq(q: Q) -> Q:
            if q.op != "topk":
                return q
            return replace(q, k=(q.k * d) // self.d)
        return replace(self, d=d, n=n or self.n, steps=steps or self.steps,
                       worker_q=rq(self.worker_q), server_q=rq(self.server_q))


def _wl() -> dict[int, Workload]:
    d3, d5 = 25_557_032, 60_000_000
    s4096, q2048 = Q("sign1", chunk=4096), Q("qsgd", chunk=2048, levels=255)
    return {
        1: Workload(1, "sign1_n4_d64k", 4, 65_536, 10, "normal", s4096, s4096),
        2: Workload(2, "sign1_n8_resnet18", 8, 11_689_512, 20, "layered", s4096, s4096),
        3: Workload(3, "topk1pct_n16_resnet50", 16, d3, 20, "laplace",
                    Q("topk", k=d3 // 100), Q("topk", k=d3 // 100)),
        4: Workload(4, "qsgd255_n8_gpt2small", 8, 124_439_808, 10, "student_t", q2048, q2048),
        5: Workload(5, "sign1_topk_n32_d60m", 32, d5, 50, "hetero", s4096, Q("topk", k=d5 // 200)),
        # beyond the five listed configurations: the shape of workload 2 with the 1-bit scale taken
        # from l2 magnitudes (the norm Section 3.2 prints)
        6: Workload(6, "sign1l2_n8_resnet18", 8, 11_689_512, 20, "layered",
                    Q("sign1", chunk=4096, norm=2), Q("sign1", chunk=4096, norm=2)),
        # ... and with clipping of the low 16 bits (Section 3.2) on both passes
        7: Workload(7, "clip16_n8_resnet18", 8, 11_689_512, 20, "layered", Q("clip", bits=16), Q("clip", bits=16)),
        # ... and with randomised sparsification (one entry in 32 survives, unscaled) on both passes
        8: Workload(8, "rsparse32_n8_resnet18", 8, 11_689_512, 20, "layered",
                    Q("rsparse", chunk=4096, keep_one_in=32), Q("rsparse", chunk=4096, keep_one_in=32)),
        # ... with the ternary quantiser of Section 5.1 (item 2) on both passes, error-compensated
        9: Workload(9, "ternary_n8_resnet18", 8, 11_689_512, 20, "layered", Q("ternary"), Q("ternary")),
        # ... with the 1-bit operator carrying ONE factor per vector, as Section 3.2 / 5.1 state it
        10: Workload(10, "sign1whole_n8_resnet18", 8, 11_689_512, 20, "layered", Q("sign1", chunk=0), Q("sign1", chunk=0)),
        # the two compressed methods of Section 5.1 that keep no error: "QSGD" (item 2: ternary workers, the
        # server sends the plain mean) and "Top-k SGD" (item 5), here with the paper's k = 300000
        11: Workload(11, "qsgd_baseline_n8_resnet18", 8, 11_689_512, 20, "layered", Q("ternary"), Q("identity"),
                     compensate=False),
        12: Workload(12, "topk_sgd_n8_resnet18", 8, 11_689_512, 20, "layered", Q("topk", k=300_000), Q("identity"),
                     compensate=False),
    }


WORKLOADS = _wl()


def _gen(device, *key: int) -> torch.Generator:
    seed = BASE_SEED
    for part in key:
        seed = (seed * 1_000_003 + int(part) + 1) % (2**63 - 1)
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def layer_sigmas(wl: Workload) -> torch.Tensor:
    """Per-slice standard deviations of the layered workload: log10 sigma ~ U[-4, -1]."""
    gen = _gen("cpu", wl.wid, 7777)
    return 10.0 ** (-4.0 + 3.0 * torch.rand(len(RESNET18_SLICES), generator=gen, dtype=torch.float64))


def _layer_scale_vector(wl: Workload, device) -> torch.Tensor:
    """sigma per element for the layered workload (slices rescaled when d is scaled down)."""
    sig = layer_sigmas(wl).to(torch.float32)
    full = sum(RESNET18_SLICES)
    if wl.d == full:
        sizes = torch.tensor(RESNET18_SLICES, dtype=torch.int64)
    else:
        edges = torch.tensor([0] + list(torch.cumsum(torch.tensor(RESNET18_SLICES), 0).tolist()),
                             dtype=torch.float64)
        edges = torch.round(edges * (wl.d / full)).to(torch.int64)
        sizes = edges[1:] - edges[:-1]
    return torch.repeat_interleave(sig.to(device), sizes.to(device))


def make_worker_gradient(wl: Workload, step: int, worker: int, device="cpu", out=None,
                         _scale_cache: dict | None = None) -> torch.Tensor:
    """g_t^{(i)}: the stochastic gradient of worker ``worker`` at iteration ``step`` ([d] fp32)."""
    d = wl.d
    gen = _gen(device, wl.wid, step, worker)
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=device)
    if wl.dist == "normal":
        out.normal_(0.0, 1.0, generator=gen)
    elif wl.dist == "layered":
        cache = _scale_cache if _scale_cache is not None else {}
        if "sigma" not in cache:
            cache["sigma"] = _layer_scale_vector(wl, device)
        out.normal_(0.0, 1.0, generator=gen)
        out.mul_(cache["sigma"])
    elif wl.dist == "laplace":
        # inverse CDF of Laplace(0, b), b = 1e-2
        out.uniform_(-0.5, 0.5, generator=gen)
        sgn = torch.sign(out)
        out.abs_().mul_(-2.0).add_(1.0).clamp_(min=1e-30).log_().mul_(sgn).mul_(-1e-2)
    elif wl.dist == "student_t":
        # t_3 = Z / sqrt(chi2_3 / 3), scaled by 1e-3
        out.normal_(0.0, 1.0, generator=gen)
        chi = torch.zeros_like(out)
        tmp = torch.empty_like(out)
        for _ in range(3):
            tmp.normal_(0.0, 1.0, generator=gen)
            chi.addcmul_(tmp, tmp)
        chi.div_(3.0).sqrt_().clamp_(min=1e-20)
        out.div_(chi).mul_(1e-3)
    elif wl.dist == "hetero":
        # g_i = mu_i + N(0, 1e-2); mu_i ~ N(0, 1e-3) drawn from (workload, worker) only
        out.normal_(0.0, 0.1, generator=gen)
        mu_gen = _gen(device, wl.wid, 424242, worker)
        mu = torch.empty_like(out).normal_(0.0, 1e-3 ** 0.5, generator=mu_gen)
        out.add_(mu)
    else:
        raise ValueError(wl.dist)
    return out


def make_gradients(wl: Workload, step: int, device="cpu", out=None) -> torch.Tensor:
    """g_t as an [n, d] fp32 tensor, row i = worker i."""
    if out is None:
        out = torch.empty(wl.n, wl.d, dtype=torch.float32, device=device)
    cache: dict = {}
    for i in range(wl.n):
        make_worker_gradient(wl, step, i, device=device, out=out[i], _scale_cache=cache)
    return out
