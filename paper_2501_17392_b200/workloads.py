"""Seeded synthetic inputs shaped like the five benchmark workloads.

This module only draws random numbers and lays them out in memory.  It holds
none of the aggregation method's arithmetic (no sign, no ring, no consensus,
no attack formula): it produces the honest update matrix every client would
send, plus the raw standard-normal / uniform draws an attack may consume.
Both the CUDA library and the CPU checker are fed the very same buffers, so
it does not matter that a CPU and a CUDA torch generator give different
streams for one seed: a buffer is generated once and shared.

The paper evaluates on gradients of a small CNN (Fashion-MNIST) and ResNet-20
(CIFAR-10) with n = 100 clients of which 20% are malicious and lambda = 5
(Section 5.1).  Neither datasets nor models are available offline, so these
synthetic draws stand in for them: same n / f / d scales, honest updates
Gaussian around a shared direction, heavy tails and client heterogeneity in
some workloads.
"""

from __future__ import annotations

from dataclasses import dataclass

import torch

BASE_SEED = 2501017392

# attack kinds (numbering of the C header)
ATTACK_SCALE_OWN = 1
ATTACK_GAUSSIAN = 2
ATTACK_SCALED_MEAN = 3
ATTACK_MEAN_SHIFT = 4
ATTACK_SPARSE_NOISE = 5


@dataclass(frozen=True)
class Workload:
    name: str
    n: int
    f: int
    d: int
    rounds: int
    honest: str          # recipe id, see honest_updates()
    attack: int
    scale: float = 1.0
    sigma: float = 1.0
    kappa: float = 3.0
    prob: float = 0.1

    @property
    def lam(self) -> float:
        # the paper uses lambda = 5 with n = 100 (Section 5.1): keep lambda / n
        return float((5 * self.n) // 100)

    @property
    def ld(self) -> int:
        return round_up(self.d, 128)


WORKLOADS = {
    "cfg1": Workload("cfg1", 8, 1, 100_000, 1, "gauss_offset", ATTACK_SCALE_OWN, scale=-10.0),
    "cfg2": Workload("cfg2", 20, 4, 1_663_370, 1, "shared_mean", ATTACK_GAUSSIAN, sigma=200.0),
    "cfg3": Workload("cfg3", 50, 10, 11_689_512, 1, "hetero_scale", ATTACK_SCALED_MEAN, scale=-5.0),
    "cfg4": Workload("cfg4", 100, 20, 25_557_032, 1, "gauss", ATTACK_MEAN_SHIFT, kappa=3.0),
    "cfg5": Workload("cfg5", 16, 3, 124_439_808, 5, "heavy_tail", ATTACK_SPARSE_NOISE, sigma=1.0, prob=0.1),
}


def round_up(x: int, m: int) -> int:
    return (x + m - 1) // m * m


def scaled(w: Workload, d: int, name: str | None = None) -> Workload:
    """Same recipe on a shorter (or longer) vector: used for parity cases and
    bounded CPU samples."""
    return Workload(name or f"{w.name}_d{d}", w.n, w.f, d, w.rounds, w.honest, w.attack,
                    w.scale, w.sigma, w.kappa, w.prob)


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed & 0x7FFFFFFFFFFFFFFF)
    return g


def _seed(w: Workload, round_idx: int, stream: int) -> int:
    cfg = sum(ord(ch) for ch in w.name.split("_")[0])
    return BASE_SEED + 1_000_003 * cfg + 7919 * round_idx + 104_729 * stream


def honest_updates(w: Workload, round_idx: int = 0, device="cpu", ld: int | None = None,
                   out: torch.Tensor | None = None) -> torch.Tensor:
    """float32 [n, ld] matrix (row i = client i's honest update, columns >= d
    are zero padding).  Every client, Byzantine ones included, gets an honest
    draw; an attack later overwrites the Byzantine rows."""
    ld = w.ld if ld is None else ld
    dev = torch.device(device)
    if out is None:
        out = torch.zeros((w.n, ld), dtype=torch.float32, device=dev)
    else:
        assert out.shape == (w.n, ld) and out.dtype == torch.float32
        out[:, w.d:].zero_()
    g = _gen(dev, _seed(w, round_idx, 1))
    d = w.d
    if w.honest == "gauss_offset":        # N(0.01, 0.1^2) iid
        for i in range(w.n):
            out[i, :d].normal_(0.01, 0.1, generator=g)
    elif w.honest == "shared_mean":       # mu ~ N(0, 0.05^2) shared + N(0, 0.02^2) per client
        mu = torch.empty(d, dtype=torch.float32, device=dev).normal_(0.0, 0.05, generator=g)
        for i in range(w.n):
            out[i, :d].normal_(0.0, 0.02, generator=g)
            out[i, :d] += mu
    elif w.honest == "hetero_scale":      # N(0, (0.01 s_i)^2), s_i ~ U(0.5, 2)
        s = torch.empty(w.n, dtype=torch.float32, device="cpu").uniform_(
            0.5, 2.0, generator=_gen("cpu", _seed(w, round_idx, 2)))
        for i in range(w.n):
            out[i, :d].normal_(0.0, 0.01 * float(s[i]), generator=g)
    elif w.honest == "gauss":             # N(0, 0.01^2)
        for i in range(w.n):
            out[i, :d].normal_(0.0, 0.01, generator=g)
    elif w.honest == "heavy_tail":        # 0.001 z; z ~ N(0,1), 1% of entries Student-t(3)
        step = 1 << 24
        for i in range(w.n):
            for b in range(0, d, step):
                e = min(d, b + step)
                z = torch.empty(e - b, dtype=torch.float32, device=dev).normal_(generator=g)
                pick = torch.empty(e - b, dtype=torch.float32, device=dev).uniform_(generator=g) < 0.01
                k = int(pick.sum())
                if k:
                    num = torch.empty(k, dtype=torch.float32, device=dev).normal_(generator=g)
                    den = torch.empty((3, k), dtype=torch.float32, device=dev).normal_(generator=g)
                    z[pick] = num / torch.sqrt((den * den).sum(0) / 3.0)
                out[i, b:e] = 0.001 * z
    else:
        raise ValueError(w.honest)
    return out


def attack_draws(w: Workload, round_idx: int = 0, device="cpu", ld: int | None = None):
    """(noise, uniform): float32 [f, ld] standard-normal and uniform[0,1) draws
    for the attacks that consume randomness, else (None, None)."""
    ld = w.ld if ld is None else ld
    dev = torch.device(device)
    noise = uniform = None
    if w.f == 0:
        return None, None
    if w.attack in (ATTACK_GAUSSIAN, ATTACK_SPARSE_NOISE):
        noise = torch.zeros((w.f, ld), dtype=torch.float32, device=dev)
        g = _gen(dev, _seed(w, round_idx, 3))
        for b in range(w.f):
            noise[b, :w.d].normal_(generator=g)
    if w.attack == ATTACK_SPARSE_NOISE:
        uniform = torch.ones((w.f, ld), dtype=torch.float32, device=dev)
        g = _gen(dev, _seed(w, round_idx, 4))
        for b in range(w.f):
            uniform[b, :w.d].uniform_(generator=g)
    return noise, uniform


def edge_value_updates(n: int, d: int, seed: int = 0, device="cpu", ld: int | None = None) -> torch.Tensor:
    """Matrix sprinkled with the float values a sign function must classify:
    +-0, denormals, +-Inf, NaN, +-FLT_MAX, among ordinary normals."""
    ld = d if ld is None else ld
    g = _gen("cpu", BASE_SEED + 31 * seed + 5)
    x = torch.zeros((n, ld), dtype=torch.float32)
    x[:, :d].normal_(generator=g)
    specials = torch.tensor([0.0, -0.0, 1e-45, -1e-45, float("inf"), float("-inf"), float("nan"),
                             3.4028234663852886e38, -3.4028234663852886e38, 1.17549435e-38], dtype=torch.float32)
    idx = torch.randint(0, specials.numel() * 3, (n, d), generator=g)
    mask = idx < specials.numel()
    x[:, :d][mask] = specials[idx[mask]]
    return x.to(device)


def small_integer_updates(n: int, d: int, seed: int = 0, device="cpu", ld: int | None = None,
                          lo: int = -3, hi: int = 3) -> torch.Tensor:
    """Small integer-valued float32 entries (many exact zeros and ties)."""
    ld = d if ld is None else ld
    g = _gen("cpu", BASE_SEED + 17 * seed + 3)
    x = torch.zeros((n, ld), dtype=torch.float32)
    x[:, :d] = torch.randint(lo, hi + 1, (n, d), generator=g).to(torch.float32)
    return x.to(device)
