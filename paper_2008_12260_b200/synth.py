"""Seeded synthetic inputs for the PolluxSched optimizer core.

This module only *draws inputs*: job parameter sets (theta_sys, phi, M0 of Eq. 12),
clusters, batch-size grids, current allocations, pre-computed speedup tables and
populations of allocation matrices.  It contains none of the method's arithmetic
(no goodput, fitness, repair or RNG-driven operator lives here), so both the CUDA
path and the CPU oracle can be fed from it without sharing any computation.

The paper's workload (Sec. 5.1: a 160-job, 8-hour sample of a production trace and six
profiled models) is not available; the generators below reproduce its *shape*: many
small jobs and few large ones, node-level synchronisation 2-5x costlier than local
(the jump beyond one node in Fig. 3), gamma in [1, 10] (Sec. 4.1), and a gradient noise
scale that grows about tenfold over a job's life (Sec. 3.1 / Fig. 2).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

F32 = np.float32

JOB_F32_FIELDS = (
    "alpha_grad", "beta_grad", "alpha_local", "beta_local", "alpha_node", "beta_node",
    "gamma", "phi", "m0", "m_max_total",
)


@dataclass
class Cluster:
    """A cluster is just the GPU count of every node (the length-N vector behind `a`)."""

    node_capacity: np.ndarray  # int16 [num_nodes]

    @property
    def num_nodes(self) -> int:
        return int(self.node_capacity.shape[0])

    @property
    def total_gpus(self) -> int:
        return int(self.node_capacity.astype(np.int64).sum())

    @property
    def k_max(self) -> int:
        return min(self.total_gpus, 64)

    @property
    def n_max(self) -> int:
        return min(self.num_nodes, 64)


def uniform_cluster(num_nodes: int, gpus_per_node: int) -> Cluster:
    return Cluster(np.full(num_nodes, gpus_per_node, dtype=np.int16))


@dataclass
class Jobs:
    """Host-side SoA of per-job inputs (all float fields fp32, as both sides consume them)."""

    alpha_grad: np.ndarray
    beta_grad: np.ndarray
    alpha_local: np.ndarray
    beta_local: np.ndarray
    alpha_node: np.ndarray
    beta_node: np.ndarray
    gamma: np.ndarray
    phi: np.ndarray
    m0: np.ndarray            # M0 as float (exact integer)
    m_max_total: np.ndarray   # M_max as float (exact integer)
    m_max_gpu: np.ndarray     # int32, per-GPU batch limit (grid upper end)
    m_grid: np.ndarray        # int32 [J][Gm]
    k_cap: np.ndarray         # int32
    age_sec: np.ndarray       # fp32, T_j
    num_restarts: np.ndarray  # int32, R_j
    active: np.ndarray        # uint8
    fair_k: np.ndarray = field(default=None)  # int32, filled by the caller
    fair_n: np.ndarray = field(default=None)
    alpha_rack: np.ndarray = field(default=None)  # fp32, third synchronisation pair (rack-level locality), optional
    beta_rack: np.ndarray = field(default=None)

    @property
    def num_jobs(self) -> int:
        return int(self.alpha_grad.shape[0])

    def take(self, idx) -> "Jobs":
        kw = {}
        for name, val in self.__dict__.items():
            kw[name] = None if val is None else np.ascontiguousarray(val[idx])
        return Jobs(**kw)


def make_m_grid(m_max_gpu: np.ndarray, grid_m: int) -> np.ndarray:
    """Log-spaced per-GPU batch sizes 1..m_max, `grid_m` points per job, ascending.

    Point i is round(exp(i * ln(m_max) / (grid_m - 1))), at least 1; duplicates may occur
    for small m_max.  Built once here, in Python floats, and handed as integers to every
    consumer so no two implementations can round it differently.
    """
    J = int(m_max_gpu.shape[0])
    out = np.empty((J, grid_m), dtype=np.int32)
    for j in range(J):
        lm = math.log(float(m_max_gpu[j]))
        for i in range(grid_m):
            v = 1.0 if grid_m == 1 else math.exp(i * lm / (grid_m - 1))
            out[j, i] = max(1, int(math.floor(v + 0.5)))
    return out


def make_m_samples(m0: np.ndarray, m_max_total: np.ndarray, num_samples: int) -> np.ndarray:
    """Candidate total batch sizes per job: `num_samples` integers log-spaced from M0 to M_max
    (inputs of the total-batch sampling search; built once on the host)."""
    J = int(m0.shape[0])
    out = np.empty((J, num_samples), dtype=np.int32)
    for j in range(J):
        lo, hi = math.log(float(m0[j])), math.log(float(m_max_total[j]))
        for i in range(num_samples):
            v = math.exp(lo + (hi - lo) * (i / (num_samples - 1) if num_samples > 1 else 0.0))
            out[j, i] = min(max(int(math.floor(v + 0.5)), int(m0[j])), int(m_max_total[j]))
    return out


def draw_jobs(num_jobs: int, seed: int, grid_m: int, grid_s: int, k_max: int,
              phi_hi: float = 1e5, with_history: bool = False) -> Jobs:
    """Draw job parameters in a fixed order from PCG64(seed).

    alpha_grad ~ U[0.01, 0.2] s, beta_grad ~ U[1e-4, 5e-3] s/sample,
    alpha_local ~ U[0.005, 0.05], beta_local ~ U[1e-4, 5e-3], node variants = local times
    independent U[2, 5] factors, gamma ~ U[1, 10], phi log-uniform [1e2, phi_hi],
    M0 in {64, 128, 256}, M_max = 32 M0, m_max ~ U{32..512}.  With `with_history`,
    T_j ~ U[60, 7200] s and R_j ~ U{0..floor(T_j / 420)}; otherwise T_j = 600, R_j = 0.
    """
    g = np.random.Generator(np.random.PCG64(seed))
    J = num_jobs
    alpha_grad = g.uniform(0.01, 0.2, J)
    beta_grad = g.uniform(1e-4, 5e-3, J)
    alpha_local = g.uniform(0.005, 0.05, J)
    beta_local = g.uniform(1e-4, 5e-3, J)
    alpha_node = alpha_local * g.uniform(2.0, 5.0, J)
    beta_node = beta_local * g.uniform(2.0, 5.0, J)
    gamma = g.uniform(1.0, 10.0, J)
    phi = np.exp(g.uniform(math.log(1e2), math.log(phi_hi), J))
    m0 = g.choice(np.array([64, 128, 256]), J).astype(np.float64)
    m_max_gpu = g.integers(32, 513, J).astype(np.int32)
    if with_history:
        age = g.uniform(60.0, 7200.0, J)
        restarts = np.floor(g.uniform(0.0, 1.0, J) * (np.floor(age / 420.0) + 1.0)).astype(np.int32)
    else:
        age = np.full(J, 600.0)
        restarts = np.zeros(J, dtype=np.int32)
    # the 1-GPU configuration must always have a feasible grid point (M0 <= m_max * Gs)
    assert np.all(m_max_gpu.astype(np.float64) * grid_s >= m0), "grid cannot reach M0 on one GPU"
    return Jobs(
        alpha_grad=alpha_grad.astype(F32), beta_grad=beta_grad.astype(F32),
        alpha_local=alpha_local.astype(F32), beta_local=beta_local.astype(F32),
        alpha_node=alpha_node.astype(F32), beta_node=beta_node.astype(F32),
        gamma=gamma.astype(F32), phi=phi.astype(F32), m0=m0.astype(F32),
        m_max_total=(32.0 * m0).astype(F32), m_max_gpu=m_max_gpu,
        m_grid=make_m_grid(m_max_gpu, grid_m),
        k_cap=np.full(J, k_max, dtype=np.int32),
        age_sec=age.astype(F32), num_restarts=restarts,
        active=np.ones(J, dtype=np.uint8),
    )


def draw_observations(jobs: "Jobs", per_job, seed: int, gpus_per_node: int = 4, noise: float = 0.02):
    """Profiled iteration times for fitting: per job a list of (K, N, m, s, T_iter) tuples at
    random allocations and batch sizes.  The times are passed in by the caller-supplied
    function of the test or benchmark (this module holds no model arithmetic): here only the
    configurations are drawn.  Returns (offset [J+1], K, N, m, s, noise factors)."""
    g = np.random.Generator(np.random.PCG64(seed))
    J = jobs.num_jobs
    counts = np.full(J, per_job, dtype=np.int64) if np.isscalar(per_job) else np.asarray(per_job, dtype=np.int64)
    offset = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    total = int(offset[-1])
    K = g.integers(1, 17, total).astype(np.int32)
    spread = g.integers(1, 5, total)
    N = np.where(K == 1, 1, np.minimum(np.maximum(spread, -(-K // gpus_per_node)), K)).astype(np.int32)
    job_of = np.repeat(np.arange(J), counts)
    m = (1 + g.integers(0, 1 << 30, total) % np.maximum(jobs.m_max_gpu[job_of], 1)).astype(np.int32)
    s = g.integers(0, 4, total).astype(np.int32)
    factor = np.exp(g.normal(0.0, noise, total))
    return offset, K, N, m, s, factor


def random_feasible_allocation(cluster: Cluster, num_jobs: int, seed: int,
                               k_hi: int = 8, active: np.ndarray | None = None) -> np.ndarray:
    """A random allocation matrix that satisfies node capacity and interference avoidance.

    Jobs are visited in a random order; each asks for K ~ U{0..k_hi} GPUs.  A request that
    fits one node is placed on a random node with enough free GPUs; a larger one takes
    whole free nodes that host no other multi-node job.  Requests that cannot be placed
    get nothing.  Purely constructive: no repair operator is involved.
    """
    g = np.random.Generator(np.random.PCG64(seed))
    N = cluster.num_nodes
    free = cluster.node_capacity.astype(np.int64).copy()
    has_dist = np.zeros(N, dtype=bool)
    A = np.zeros((num_jobs, N), dtype=np.int16)
    for j in g.permutation(num_jobs):
        K = int(g.integers(0, k_hi + 1))
        if K == 0 or (active is not None and not active[j]):
            continue
        fits = np.nonzero(free >= K)[0]
        if fits.size:
            n = int(fits[g.integers(0, fits.size)])
            A[j, n] = K
            free[n] -= K
            continue
        cand = np.nonzero((free > 0) & ~has_dist)[0]
        g.shuffle(cand)
        got, picked = 0, []
        for n in cand:
            take = int(min(free[n], K - got))
            picked.append((int(n), take))
            got += take
            if got == K:
                break
        if got == K and len(picked) >= 2:
            for n, take in picked:
                A[j, n] = take
                free[n] -= take
                has_dist[n] = True
    return A


def random_raw_population(population: int, num_jobs: int, cluster: Cluster, seed: int,
                          density: float = 0.15, v_hi: int = 6) -> np.ndarray:
    """Unconstrained random matrices (most entries zero): raw material for repair tests."""
    g = np.random.Generator(np.random.PCG64(seed))
    shape = (population, num_jobs, cluster.num_nodes)
    vals = g.integers(1, v_hi + 1, shape, dtype=np.int16)
    mask = g.uniform(0.0, 1.0, shape) < density
    return np.where(mask, vals, 0).astype(np.int16)


def stress_speedup_table(num_jobs: int, k_max: int, n_max: int, gpus_per_node: int,
                         seed: int) -> np.ndarray:
    """Pre-computed tables fp32 [J][k_max+1][n_max+1] for the fitness stress workload.

    For a valid (K, N) (1 <= N <= K, K <= N * gpus_per_node): K**u_j, times v_j when N >= 2,
    normalised to 1 at (K, N) = (2, 1); u_j ~ U[0.3, 1], v_j ~ U[0.5, 1].  Invalid entries 0.
    """
    g = np.random.Generator(np.random.PCG64(seed))
    u = g.uniform(0.3, 1.0, num_jobs)
    v = g.uniform(0.5, 1.0, num_jobs)
    K = np.arange(k_max + 1, dtype=np.float64)[None, :, None]
    N = np.arange(n_max + 1, dtype=np.float64)[None, None, :]
    val = np.power(np.maximum(K, 1.0), u[:, None, None]) * np.where(N >= 2, v[:, None, None], 1.0)
    val = val / np.power(2.0, u)[:, None, None]
    valid = (N >= 1) & (K >= N) & (K <= N * gpus_per_node) & (K >= 1)
    return np.where(valid, val, 0.0).astype(F32)


def stress_population(population: int, num_jobs: int, num_nodes: int, gpus_per_node: int,
                      seed: int, device="cpu", first_candidate: int = 0):
    """Dense int16 [P][J][num_nodes] matrices with mostly-empty rows (torch tensor on `device`).

    Per row: K = 0 with probability 0.5, else 1 + floor(64 u^3) capped at 64; with
    probability 0.7 packed on ceil(K / gpus_per_node) consecutive nodes from a random
    start (wrapping), else spread one GPU per node over K nodes starting at a random node
    with a random odd stride.  `first_candidate` offsets the seed so chunks of one large
    population can be generated independently.
    """
    import torch

    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed) * 1_000_003 + int(first_candidate))
    P, J, N, G = population, num_jobs, num_nodes, gpus_per_node
    u = torch.rand((P, J, 5), generator=gen, device=device)
    K = torch.where(u[..., 0] < 0.5, torch.zeros((), device=device),
                    torch.clamp(1.0 + torch.floor(64.0 * u[..., 1] ** 3), max=64.0)).to(torch.int64)
    packed = u[..., 2] < 0.7
    start = torch.clamp((u[..., 3] * N).to(torch.int64), max=N - 1)
    pow2 = N >= 8 and (N & (N - 1)) == 0
    if pow2:   # any odd stride visits distinct nodes when N is a power of two
        odd = 1 + 2 * torch.clamp((u[..., 4] * (N // 4)).to(torch.int64), max=N // 4 - 1)
    else:
        odd = torch.ones_like(start)
    stride = torch.where(packed, torch.ones_like(start), odd)
    S = min(64, N)
    slots = torch.arange(S, device=device, dtype=torch.int64)             # [S]
    node = (start[..., None] + slots * stride[..., None]) % N             # [P,J,S], distinct per row
    per_packed = torch.clamp(K[..., None] - slots * G, min=0, max=G)      # GPUs on the i-th packed node
    per_spread = (slots < K[..., None]).to(torch.int64)
    val = torch.where(packed[..., None], per_packed, per_spread).to(torch.int16)
    A = torch.zeros((P, J, N), dtype=torch.int16, device=device)
    A.scatter_(2, node, val)
    return A


# --------------------------------------------------------------------------------------
# Named configurations (the five workloads the throughput figures are quoted on)
# --------------------------------------------------------------------------------------
@dataclass
class Config:
    name: str
    num_nodes: int
    gpus_per_node: int
    num_jobs: int
    seed: int
    grid_m: int
    grid_s: int
    population: int
    generations: int
    p: float = -1.0
    phi_hi: float = 1e5
    delta_sec: float = 30.0
    speedup_floor: float = 1e-3
    mutate_prob: float = 0.05
    init_prob: float = 0.25
    num_elite: int = 2
    with_history: bool = False
    random_cur: bool = False

    def cluster(self) -> Cluster:
        return uniform_cluster(self.num_nodes, self.gpus_per_node)

    def jobs(self) -> Jobs:
        c = self.cluster()
        return draw_jobs(self.num_jobs, self.seed, self.grid_m, self.grid_s, c.k_max,
                         phi_hi=self.phi_hi, with_history=self.with_history)

    def cur(self, jobs: Jobs | None = None) -> np.ndarray:
        if not self.random_cur:
            return np.zeros((self.num_jobs, self.num_nodes), dtype=np.int16)
        return random_feasible_allocation(self.cluster(), self.num_jobs, self.seed + 1000,
                                          active=None if jobs is None else jobs.active)


def prob_to_threshold(prob: float) -> int:
    """A probability as the integer threshold floor(prob * 2**32), saturated to 2**32 - 1."""
    return int(min(max(math.floor(prob * 4294967296.0), 0), 4294967295))


TINY = Config("tiny", 4, 4, 8, 0, 32, 8, 32, 10, num_elite=2, mutate_prob=0.2)
TESTBED = Config("testbed", 16, 4, 48, 1, 64, 16, 100, 100, num_elite=4, mutate_prob=0.08,
                 with_history=True, random_cur=True)
LARGE = Config("large", 256, 8, 1024, 2, 128, 32, 512, 200, phi_hi=1e6, num_elite=16,
               mutate_prob=0.01, init_prob=0.02, with_history=True, random_cur=True)
CONFIGS = {c.name: c for c in (TINY, TESTBED, LARGE)}

STRESS = dict(name="stress", num_nodes=2048, gpus_per_node=8, num_jobs=8192, seed=3,
              population=4096, k_max=64, n_max=64, p_values=(-1.0, 0.5, 1.0))


@dataclass
class TraceJob:
    arrive_sec: float
    life_sec: float
    category: str


def trace_arrivals(num_jobs: int = 160, seed: int = 4, horizon_sec: float = 8 * 3600.0,
                   mean_gap_sec: float = 180.0) -> list[TraceJob]:
    """Poisson arrivals over the horizon with the size mix of the paper's Table 1.

    Categories Small / Medium / Large / XLarge with probabilities 72 / 20 / 6 / 2 % and
    lifetimes log-uniform in [5,30] / [30,120] / [120,360] / [360,480] minutes; lifetimes
    do not depend on the allocations, so every round's inputs can be generated up front.
    """
    g = np.random.Generator(np.random.PCG64(seed))
    gaps = g.exponential(mean_gap_sec, num_jobs)
    arrive = np.minimum(np.cumsum(gaps), horizon_sec - 60.0)
    cats = g.choice(4, num_jobs, p=[0.72, 0.20, 0.06, 0.02])
    lo = np.array([5, 30, 120, 360], dtype=np.float64) * 60.0
    hi = np.array([30, 120, 360, 480], dtype=np.float64) * 60.0
    life = np.exp(g.uniform(np.log(lo[cats]), np.log(hi[cats])))
    names = ["S", "M", "L", "XL"]
    return [TraceJob(float(arrive[i]), float(life[i]), names[int(cats[i])]) for i in range(num_jobs)]


def rack_of_nodes(num_nodes: int, nodes_per_rack: int) -> np.ndarray:
    """Rack id of every node: consecutive nodes share a rack (int16 [num_nodes])."""
    return (np.arange(num_nodes) // max(int(nodes_per_rack), 1)).astype(np.int16)


def draw_rack_pair(jobs: Jobs, seed: int, lo: float = 1.5, hi: float = 3.0):
    """Third synchronisation pair for allocations that span racks: the node pair times an
    independent factor U[lo, hi] each (crossing racks is slower than crossing nodes, as crossing
    nodes is slower than staying on one).  Returns (alpha_rack, beta_rack), fp32 [J]."""
    g = np.random.Generator(np.random.PCG64(seed))
    fa = g.uniform(lo, hi, jobs.num_jobs)
    fb = g.uniform(lo, hi, jobs.num_jobs)
    return (jobs.alpha_node * fa).astype(np.float32), (jobs.beta_node * fb).astype(np.float32)
