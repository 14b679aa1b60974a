"""Seeded synthetic logits for the five benchmark workloads.

The draft and target model forwards are outside this library, so their logits
are generated: target logits z_p = 3*N(0,1) + bias(v) with a Zipf-shaped bias
(bias(v) = -zeta * ln(1 + rank(v)), rank an affine permutation of the token
ids), draft logits z_q = c * z_p + sigma * N(0,1), both rounded to the
workload's dtype.  Rows are i.i.d. over positions and rounds.

This module holds input generation only: none of the method's arithmetic, no
dependency on the CUDA library or on the CPU oracle.  Both consume what it
returns (the oracle through `to_numpy_bits`).  torch is used for its seeded
generators, on whichever device the caller names; CPU and CUDA generators give
different streams, so a comparison always generates once and copies.
"""
from dataclasses import dataclass, replace
import math

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    n_seq: int
    vocab: int
    dtype: str            # "bf16" | "fp32"
    k_max: int
    rounds: int
    n_arms: int
    policy: str           # "ucb1" | "ts"
    level: str            # "seq" | "token"
    seed: int
    zipf: float = 1.1
    c: float = 1.0
    sigma: str = "fixed:0.5"   # "fixed:x" | "per_seq:lo:hi" | "per_round:lo:hi" | "cycle:a,b,c:period"
    zipf_cycle: str = ""       # "" | "a,b:period"
    temp_draft: float = 1.0
    temp_target: float = 1.0

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    @property
    def elem_bytes(self):
        return 2 if self.dtype == "bf16" else 4

    @property
    def row_bytes(self):
        return self.vocab * self.elem_bytes


WORKLOADS = {
    "tiny": Workload("tiny", 1, 32000, "fp32", 8, 256, 3, "ucb1", "seq", seed=0,
                     sigma="per_round:0.2:2.0"),
    "batch64": Workload("batch64", 64, 128256, "bf16", 16, 1024, 5, "ucb1", "seq", seed=1,
                        sigma="per_seq:0.1:1.5"),
    "batch256_ts": Workload("batch256_ts", 256, 151936, "bf16", 12, 1024, 5, "ts", "token", seed=2,
                            c=0.8, sigma="fixed:1.0", temp_target=0.7),
    "throughput": Workload("throughput", 1024, 128256, "bf16", 8, 512, 5, "ucb1", "seq", seed=3,
                           sigma="fixed:0.5"),
    "shift": Workload("shift", 128, 256000, "bf16", 16, 4096, 5, "ucb1", "seq", seed=4,
                      sigma="cycle:0.1,0.8,2.0:512", zipf_cycle="1.0,1.4:512"),
}
WORKLOADS["shift_ts"] = replace(WORKLOADS["shift"], name="shift_ts", policy="ts")


def scaled(w: Workload, **kw) -> Workload:
    """A smaller or altered copy of a workload (parity tests at reduced size)."""
    return replace(w, **kw)


def _cpu_gen(*keys):
    g = torch.Generator(device="cpu")
    s = 0x9E3779B97F4A7C15
    for k in keys:
        s = (s * 6364136223846793005 + int(k) + 1442695040888963407) & 0x7FFFFFFFFFFFFFFF
    g.manual_seed(s)
    return g


def sigma_for(w: Workload, rnd: int) -> torch.Tensor:
    """Per-sequence draft-noise scale for one round (float32, CPU, [n_seq])."""
    kind, *args = w.sigma.split(":")
    S = w.n_seq
    if kind == "fixed":
        return torch.full((S,), float(args[0]))
    if kind == "per_seq":
        lo, hi = float(args[0]), float(args[1])
        return lo + (hi - lo) * torch.rand(S, generator=_cpu_gen(w.seed, 101))
    if kind == "per_round":
        lo, hi = float(args[0]), float(args[1])
        u = torch.rand(1, generator=_cpu_gen(w.seed, 102, rnd))
        return (lo + (hi - lo) * u).expand(S).clone()
    if kind == "cycle":
        vals = torch.tensor([float(x) for x in args[0].split(",")])
        period = int(args[1])
        phase = torch.randint(0, len(vals), (S,), generator=_cpu_gen(w.seed, 103))
        return vals[(phase + rnd // period) % len(vals)]
    raise ValueError(w.sigma)


def zipf_for(w: Workload, rnd: int) -> float:
    if not w.zipf_cycle:
        return w.zipf
    vals, period = w.zipf_cycle.split(":")
    vals = [float(x) for x in vals.split(",")]
    return vals[(rnd // int(period)) % len(vals)]


def _rank_permutation(w: Workload, device) -> torch.Tensor:
    """rank(v) = (A*v + B) mod V with gcd(A, V) = 1, A and B fixed by the seed."""
    V = w.vocab
    g = _cpu_gen(w.seed, 104)
    A = int(torch.randint(1, V, (1,), generator=g)) | 1
    while math.gcd(A, V) != 1:
        A += 2
    B = int(torch.randint(0, V, (1,), generator=g))
    v = torch.arange(V, dtype=torch.int64, device=device)
    return (A * v + B) % V


def round_logits(w: Workload, rnd: int, device="cpu"):
    """Logits of one speculation round.

    Returns (draft [n_seq, k_max, vocab], target [n_seq, k_max + 1, vocab]) in
    the workload's dtype on `device`, C-contiguous.
    """
    S, K, V = w.n_seq, w.k_max, w.vocab
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed((w.seed * 1_000_003 + rnd * 7919 + 17) & 0x7FFFFFFFFFFFFFFF)
    rank = _rank_permutation(w, dev)
    bias = (-zipf_for(w, rnd)) * torch.log1p(rank.to(torch.float32))
    sig = sigma_for(w, rnd).to(dev).view(S, 1)
    draft = torch.empty((S, K, V), dtype=w.torch_dtype, device=dev)
    target = torch.empty((S, K + 1, V), dtype=w.torch_dtype, device=dev)
    for i in range(K + 1):
        zp = torch.randn((S, V), generator=g, device=dev, dtype=torch.float32).mul_(3.0).add_(bias)
        target[:, i, :] = zp.to(w.torch_dtype)
        if i < K:
            g2 = torch.randn((S, V), generator=g, device=dev, dtype=torch.float32)
            draft[:, i, :] = (zp.mul_(w.c).add_(g2.mul_(sig))).to(w.torch_dtype)
    return draft, target


def peaked_round_logits(w: Workload, rnd: int, device="cpu"):
    """round_logits with one token per row lifted by U[6, 16] (the draft's by 0.9 of that): the rows of the
    configs are flat (top-1 probability about 1e-3), these have top-1 probabilities spread over (0, 1), so that
    every stop rule fires on some rows and drafts of every length occur.  Same shapes, dtype and seeding."""
    d, t = round_logits(w, rnd, device)
    g = torch.Generator(device="cpu")
    g.manual_seed(1234 + rnd)
    S, K, V = w.n_seq, w.k_max, w.vocab
    idx = torch.randint(0, V, (S, K + 1), generator=g).to(device)
    lift = (6 + 10 * torch.rand((S, K + 1), generator=g)).to(device)
    tt = t.float()
    tt.scatter_add_(2, idx.unsqueeze(-1), lift.unsqueeze(-1))
    dd = d.float()
    dd.scatter_add_(2, idx[:, :K].unsqueeze(-1), (lift[:, :K] * 0.9).unsqueeze(-1))
    return dd.to(d.dtype), tt.to(t.dtype)


def to_numpy_bits(t: torch.Tensor) -> np.ndarray:
    """Host copy as the arrays the oracle reads: float32, or uint16 holding bf16 bits."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def bf16_bits_from_float(x: np.ndarray) -> np.ndarray:
    """float array -> bf16 bit patterns (round to nearest even), as uint16."""
    return to_numpy_bits(torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16))
