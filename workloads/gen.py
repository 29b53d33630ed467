"""Seeded generators for DETOX parameter-server inputs.

What is produced follows the paper's problem statement (Section 2 and Section 3): p compute nodes
(called n here), a random partition into node groups of size r that all receive the same batch and
therefore send bitwise-identical honest gradients g_j, q Byzantine nodes whose rows are replaced by
an attack vector, and a random partition of the p/r votes into vote groups ("sets").

Attack models (Section 5.2, "Byzantine attack models"):
  reverse  : the node sends -c * g with c = 100
  alie     : all colluding nodes send mu + z * sigma per coordinate (z = -1), mu and sigma being the
             mean and the population standard deviation over the honest nodes' rows
  constant : every element equals -1

Nothing here computes a vote, a mean over sets, a median, a distance or a score.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional

import numpy as np
import torch

REVERSE_C = 100.0
ALIE_Z = -1.0


def padded_ld(d: int, multiple: int = 32) -> int:
    """Row stride (elements): d rounded up so that every row starts on a 128-byte boundary."""
    return (d + multiple - 1) // multiple * multiple


@dataclasses.dataclass(frozen=True)
class WorkloadSpec:
    name: str
    n: int
    r: int
    d: int
    sigma: float
    q: int
    attack: str = "none"          # none | reverse | alie | constant
    placement: str = "random"     # random | distinct | worst
    coord_scales: bool = False    # per-coordinate scale, log-uniform in [1e-4, 1e-1]
    group_jitter: float = 0.0     # g_j <- (1 + group_jitter * u_j) * g_j, u_j ~ U[-1, 1]
    set_size: Optional[int] = None  # votes per set; None = a single set holding every vote
    distinct_rows: bool = False   # every node draws its own gradient (no redundancy; r only groups)
    seed: int = 0


@dataclasses.dataclass
class Workload:
    spec: WorkloadSpec
    X: torch.Tensor              # [n, ld] float32; columns d..ld-1 are zero padding
    ld: int
    members: np.ndarray          # int32 [G*r]; group j owns members[j*r:(j+1)*r]
    set_offsets: np.ndarray      # int32 [S+1]
    set_members: np.ndarray      # int32 [G]; set s owns votes set_members[set_offsets[s]:set_offsets[s+1]]
    byzantine: np.ndarray        # bool [n]
    group_of: np.ndarray         # int32 [n]
    honest_member: np.ndarray    # int32 [G]; lowest honest worker id of the group, -1 if none
    q_hat: int                   # groups in which Byzantine members outnumber honest ones

    @property
    def G(self) -> int:
        return self.spec.n // self.spec.r

    @property
    def S(self) -> int:
        return len(self.set_offsets) - 1

    def data(self) -> torch.Tensor:
        return self.X[:, : self.spec.d]


def make_groups(n: int, r: int, rng: np.random.Generator) -> np.ndarray:
    """Random partition of the n nodes into n/r node groups of size r (Algorithm 1, step 1)."""
    if r < 1 or n % r != 0:
        raise ValueError("r must divide n")
    perm = rng.permutation(n).astype(np.int32)
    groups = perm.reshape(n // r, r)
    groups.sort(axis=1)
    return groups.reshape(-1).copy()


def make_sets(G: int, set_size: Optional[int], rng: np.random.Generator):
    """Random partition of the G votes into vote groups (Algorithm 2, step 2).

    With set_size None every vote goes into one set.  A remainder (G not a multiple of set_size) is
    spread one vote at a time over the first sets, giving uneven sets such as 7 and 8 out of 15.
    """
    perm = rng.permutation(G).astype(np.int32)
    if set_size is None or set_size >= G:
        return np.array([0, G], dtype=np.int32), perm
    S = max(G // set_size, 1)
    base, extra = divmod(G, S)
    sizes = [base + (1 if s >= S - extra else 0) for s in range(S)]
    offsets = np.zeros(S + 1, dtype=np.int32)
    offsets[1:] = np.cumsum(sizes)
    return offsets, perm


def place_byzantine(n: int, r: int, q: int, members: np.ndarray, placement: str,
                    rng: np.random.Generator) -> np.ndarray:
    """Choose which q nodes are Byzantine.

    random   : a uniformly random q-subset of the nodes
    distinct : q nodes in q different groups (no vote is lost)
    worst    : (r+1)/2 nodes in one group, so that they win its vote, the others in distinct groups
    """
    byz = np.zeros(n, dtype=bool)
    G = n // r
    groups = members.reshape(G, r)
    if q == 0:
        return byz
    if placement == "random":
        byz[rng.choice(n, size=q, replace=False)] = True
    elif placement == "distinct":
        if q > G:
            raise ValueError("distinct placement needs q <= n/r")
        for j in rng.choice(G, size=q, replace=False):
            byz[groups[j, rng.integers(r)]] = True
    elif placement == "worst":
        maj = (r + 1) // 2
        if q < maj or 1 + (q - maj) > G:
            raise ValueError("worst placement needs (r+1)/2 <= q <= (r+1)/2 + n/r - 1")
        order = rng.permutation(G)
        byz[rng.choice(groups[order[0]], size=maj, replace=False)] = True
        for j in order[1 : 1 + q - maj]:
            byz[groups[j, rng.integers(r)]] = True
    else:
        raise ValueError(f"unknown placement {placement!r}")
    return byz


def expected_byzantine_votes(p: int, q: int, r: int) -> float:
    """E[q_hat] for a uniformly random placement: the hypergeometric expression in the proof of Theorem 1,
    (p/r) * sum_{i=0}^{(r-1)/2} C(q, r-i) C(p-q, i) / C(p, r)."""
    tot = 0
    for i in range((r - 1) // 2 + 1):
        tot += math.comb(q, r - i) * math.comb(p - q, i)
    return (p / r) * tot / math.comb(p, r)


def _honest_stats(X: torch.Tensor, d: int, honest_rows: List[int], chunk: int = 1 << 20):
    """Per-coordinate mean and population standard deviation (fp64) over the honest rows."""
    idx = torch.as_tensor(honest_rows, device=X.device, dtype=torch.long)
    mu = torch.empty(d, dtype=torch.float64, device=X.device)
    sd = torch.empty(d, dtype=torch.float64, device=X.device)
    for c0 in range(0, d, chunk):
        c1 = min(d, c0 + chunk)
        blk = X[:, c0:c1].index_select(0, idx).to(torch.float64)
        m = blk.mean(dim=0)
        mu[c0:c1] = m
        sd[c0:c1] = ((blk - m) ** 2).mean(dim=0).sqrt()
    return mu, sd


def make_workload(spec: WorkloadSpec, device: str = "cpu") -> Workload:
    n, r, d = spec.n, spec.r, spec.d
    G = n // r
    rng = np.random.default_rng(spec.seed)
    members = make_groups(n, r, rng)
    set_offsets, set_members = make_sets(G, spec.set_size, rng)
    byz = place_byzantine(n, r, spec.q, members, spec.placement, rng)
    group_of = np.empty(n, dtype=np.int32)
    group_of[members] = np.repeat(np.arange(G, dtype=np.int32), r)

    tg = torch.Generator(device=device)
    tg.manual_seed(spec.seed)
    ld = padded_ld(d)
    X = torch.zeros((n, ld), dtype=torch.float32, device=device)

    scales = None
    if spec.coord_scales:
        e = torch.rand(d, generator=tg, device=device, dtype=torch.float32) * 3.0 - 4.0
        scales = torch.pow(torch.tensor(10.0, device=device), e)
    jit = rng.uniform(-1.0, 1.0, size=n if spec.distinct_rows else G)

    def draw(k: int) -> torch.Tensor:
        g = torch.randn(d, generator=tg, device=device, dtype=torch.float32) * spec.sigma
        if scales is not None:
            g = g * scales
        if spec.group_jitter:
            g = g * float(1.0 + spec.group_jitter * jit[k])
        return g

    groups = members.reshape(G, r)
    if spec.distinct_rows:
        for i in range(n):
            X[i, :d] = draw(i)
    else:
        for j in range(G):
            g = draw(j)
            for i in groups[j]:
                X[int(i), :d] = g           # bitwise copies of the group's honest gradient

    honest_rows = [i for i in range(n) if not byz[i]]
    byz_rows = [i for i in range(n) if byz[i]]
    if byz_rows:
        if spec.attack == "reverse":
            for i in byz_rows:
                X[i, :d] = X[i, :d] * (-REVERSE_C)
        elif spec.attack == "alie":
            mu, sd = _honest_stats(X, d, honest_rows)
            v = (mu + ALIE_Z * sd).to(torch.float32)
            for i in byz_rows:
                X[i, :d] = v
        elif spec.attack == "constant":
            for i in byz_rows:
                X[i, :d] = -1.0
        else:
            raise ValueError(f"q > 0 needs an attack, got {spec.attack!r}")

    honest_member = np.full(G, -1, dtype=np.int32)
    q_hat = 0
    for j in range(G):
        hon = [int(i) for i in groups[j] if not byz[i]]
        if hon:
            honest_member[j] = min(hon)
        if r - len(hon) > len(hon):
            q_hat += 1
    return Workload(spec=spec, X=X, ld=ld, members=members, set_offsets=set_offsets,
                    set_members=set_members, byzantine=byz, group_of=group_of,
                    honest_member=honest_member, q_hat=q_hat)


RESNET18_D = 11_173_962
VGG_D = 28_000_000
RESNET50_D = 25_557_032

# The four fixed configurations (the sweep is produced by sweep_specs()).
CONFIGS = {
    "cfg1": WorkloadSpec("cfg1", n=15, r=3, d=100_000, sigma=0.01, q=2, attack="reverse",
                         placement="distinct", set_size=None, seed=0),
    "cfg2": WorkloadSpec("cfg2", n=45, r=3, d=RESNET18_D, sigma=1e-3, q=5, attack="alie",
                         placement="worst", set_size=5, seed=0),
    "cfg3": WorkloadSpec("cfg3", n=45, r=3, d=RESNET18_D, sigma=1e-3, q=9, attack="reverse",
                         placement="random", set_size=None, group_jitter=0.02, seed=0),
    "cfg4": WorkloadSpec("cfg4", n=105, r=3, d=VGG_D, sigma=1e-3, q=15, attack="alie",
                         placement="random", coord_scales=True, set_size=5, seed=0),
}


def sweep_specs(ns=(15, 45, 105, 225), ds=(1_000_000, RESNET18_D, RESNET50_D),
                attacks=("reverse", "alie"), seed: int = 0) -> List[WorkloadSpec]:
    out = []
    for n in ns:
        for d in ds:
            for a in attacks:
                out.append(WorkloadSpec(f"sweep_n{n}_d{d}_{a}", n=n, r=3, d=d, sigma=1e-3, q=n // 10,
                                        attack=a, placement="random", set_size=5,
                                        group_jitter=0.02, seed=seed))
    return out


def sweep_legs(spec: WorkloadSpec, G: int, S: int) -> dict:
    """Which aggregations a sweep point runs (configuration only: names and parameters, no arithmetic).

    DETOX legs: the median of the set means (of the votes when there are fewer than three sets), and
    Multi-Krum / Bulyan over the G votes with a tolerance f_votes for the few Byzantine votes that survive the
    filter.  Direct legs: the same aggregators over all n rows with f = q.  Bulyan only where rows >= 4 f + 3."""
    fv = min(2, max((G - 3) // 4, 0))
    n, q = spec.n, spec.q
    legs = {
        "detox_median": dict(a0="mean" if S >= 3 else "none", a1="coord_median", f=0, m_sel=1),
        "detox_multikrum": dict(a0="none", a1="multikrum", f=fv, m_sel=G - fv),
        "detox_bulyan": dict(a0="none", a1="bulyan", f=fv, m_sel=1),
        "direct_median": dict(a1="coord_median"),
        "direct_multikrum": dict(a1="multikrum", f=q, m_sel=n - q),
    }
    if n >= 4 * q + 3:
        legs["direct_bulyan"] = dict(a1="bulyan", f=q)
    return legs


@dataclasses.dataclass
class MeanEstimation:
    """Inputs of the synthetic mean-estimation experiment (Section 5.3, "Mean estimation on synthetic data")."""
    X: torch.Tensor             # [p, d] float32
    members: np.ndarray         # int32 [p]; group j owns members[j*r:(j+1)*r]
    set_offsets: np.ndarray     # int32 [S+1], in groups: set s owns the groups set_offsets[s] .. set_offsets[s+1]-1
    byzantine: np.ndarray       # bool [p]
    p: int
    r: int
    q: int
    d: int
    q_hat: int                  # groups in which Byzantine members outnumber honest ones


def make_mean_estimation(d: int, p: int = 220_000, r: int = 11, samples: int = 20, n_sets: int = 25, seed: int = 0,
                         q: Optional[int] = None, device: str = "cpu") -> MeanEstimation:
    """p nodes in p / r groups; q = floor(e^r / 3) of them Byzantine, placed uniformly at random.

    The paper says that 20 samples are drawn iid from N(0, I_d); the reading taken here is that every group's batch
    holds `samples` such draws and the group's honest vector is their mean (an estimate of the true mean, zero),
    copied bitwise to its r members.  Byzantine nodes send the constant vector of l2 norm 100.  The votes are
    grouped into `n_sets` runs of consecutive groups (the group table is a random partition already)."""
    if p % r != 0:
        raise ValueError("r must divide p")
    G = p // r
    q = int(math.floor(math.exp(r) / 3.0)) if q is None else q
    rng = np.random.default_rng(seed)
    members = rng.permutation(p).astype(np.int32)
    byz = np.zeros(p, dtype=bool)
    byz[rng.choice(p, size=q, replace=False)] = True
    tg = torch.Generator(device=device)
    tg.manual_seed(seed)
    g = torch.empty((G, d), dtype=torch.float32, device=device)
    chunk = max(1, (1 << 24) // (samples * d))
    for j0 in range(0, G, chunk):
        j1 = min(G, j0 + chunk)
        draws = torch.randn((j1 - j0, samples, d), generator=tg, device=device, dtype=torch.float32)
        g[j0:j1] = draws.mean(dim=1)
    X = torch.empty((p, d), dtype=torch.float32, device=device)
    group_of = torch.empty(p, dtype=torch.long, device=device)
    group_of[torch.as_tensor(members, dtype=torch.long, device=device)] = torch.arange(G, device=device).repeat_interleave(r)
    X.copy_(g.index_select(0, group_of))
    X[torch.as_tensor(byz, device=device)] = 100.0 / math.sqrt(d)
    byz_in_group = byz[members].reshape(G, r).sum(axis=1)
    base, extra = divmod(G, n_sets)
    sizes = [base + (1 if s >= n_sets - extra else 0) for s in range(n_sets)]
    offsets = np.zeros(n_sets + 1, dtype=np.int32)
    offsets[1:] = np.cumsum(sizes)
    return MeanEstimation(X=X, members=members, set_offsets=offsets, byzantine=byz, p=p, r=r, q=q, d=d,
                          q_hat=int((2 * byz_in_group > r).sum()))
