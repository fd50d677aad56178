"""Exhaustive parity on clusters small enough to enumerate: every allocation matrix of
  * 3 jobs on 2 nodes x 2 GPUs   (entries 0..2, 3^6 = 729 matrices),
  * 2 jobs on 2 nodes x 4 GPUs   (entries 0..4, 5^4 = 625),
  * 3 jobs on 3 nodes x 2 GPUs   (entries 0..2, 3^9 = 19 683),
feasible or not, goes through eval_fitness (Eq. 14 with the re-allocation penalty and the
floor; 1e-5 against the oracle) and through repair_population (Sec. 4.2: node capacity and
interference avoidance; bit for bit against the oracle).  Each set also runs embedded in an
8-node cluster whose extra nodes have no GPUs, which sends it through the batched kernels
(rows of whole 16-byte vectors) instead of the general ones."""
import itertools

import numpy as np
import pytest

from helpers import assert_close, feasible
from paper_2008_12260_b200 import synth

pytestmark = pytest.mark.gpu

SETS = {
    "2x2_3jobs": (3, 2, 2),     # jobs, nodes, GPUs per node
    "2x4_2jobs": (2, 2, 4),
    "3x2_3jobs": (3, 3, 2),
}


def _matrices(J, nodes, gpn, pad_to=None):
    mats = np.array(list(itertools.product(range(gpn + 1), repeat=J * nodes)), np.int16).reshape(-1, J, nodes)
    cap = np.full(nodes, gpn, np.int16)
    if pad_to:
        wide = np.zeros((mats.shape[0], J, pad_to), np.int16)
        wide[:, :, :nodes] = mats
        mats = wide
        cap = np.concatenate([cap, np.zeros(pad_to - nodes, np.int16)])
    return np.ascontiguousarray(mats), cap


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2008_12260_b200 import api
    assert torch.cuda.is_available()
    return torch, api


class _J:
    def __init__(self, k_cap=None, active=None):
        self.k_cap = k_cap
        self.active = active


@pytest.mark.parametrize("pad", [None, 8], ids=["plain", "padded8"])
@pytest.mark.parametrize("name", list(SETS))
def test_fitness_of_every_matrix(gpu, oracle, name, pad):
    torch, api = gpu
    J, nodes, gpn = SETS[name]
    mats, cap = _matrices(J, nodes, gpn, pad)
    k_max, n_max = nodes * gpn, nodes
    assert mats.shape[0] == (gpn + 1) ** (J * nodes)
    rng = np.random.default_rng(11)
    table = rng.uniform(0.2, 2.5, (J, k_max + 1, n_max + 1)).astype(np.float32)
    table[:, 0, :] = 0.0
    table[:, :, 0] = 0.0
    cur = mats[rng.integers(1, mats.shape[0])].copy()
    cur[J - 1] = 0                                  # one pending job: never penalised
    rf = rng.uniform(0.3, 0.95, J).astype(np.float32)
    rf[0] = 0.0                                     # a factor of zero: the floor decides
    s = api.Scheduler(node_capacity=cap, num_jobs=J, grid_m=1, grid_s=1, population=1, speedup_floor=1e-3,
                      k_max=k_max, n_max=n_max, stream=torch.cuda.current_stream().cuda_stream)
    d_pop = torch.from_numpy(mats).cuda()
    d_table, d_cur, d_rf = (torch.from_numpy(a).cuda() for a in (table, cur, rf))
    for p in (-1.0, 0.5, 1.0):
        out = torch.full((mats.shape[0],), -1.0, dtype=torch.float32, device="cuda")
        s.eval_fitness(d_pop, d_table, out, p=p, cur=d_cur, realloc_factor=d_rf)
        s.sync_status()
        ref = oracle.eval_fitness(mats, table.astype(np.float64), k_max, n_max, p, 1e-3, cur=cur,
                                  realloc=rf.astype(np.float64))
        assert_close(out.cpu().numpy(), ref, what="%s p=%g" % (name, p))
    s.close()


@pytest.mark.parametrize("pad", [None, 8], ids=["plain", "padded8"])
@pytest.mark.parametrize("name,k_cap,n_max", [
    ("2x2_3jobs", (4, 1, 2), 2), ("2x2_3jobs", (4, 4, 4), 1), ("2x4_2jobs", (8, 3), 2), ("2x4_2jobs", (5, 8), 1),
    ("3x2_3jobs", (6, 2, 3), 3), ("3x2_3jobs", (6, 6, 6), 2)])
def test_repair_of_every_matrix(gpu, oracle, name, k_cap, n_max, pad):
    torch, api = gpu
    J, nodes, gpn = SETS[name]
    mats, cap = _matrices(J, nodes, gpn, pad)
    k_max = nodes * gpn
    k_cap = np.array(k_cap, np.int32)
    seed, rnd, gen = 0x5EED0000 + nodes, 4, 9
    s = api.Scheduler(node_capacity=cap, num_jobs=J, grid_m=1, grid_s=1, population=1, k_max=k_max, n_max=n_max,
                      seed=seed, stream=torch.cuda.current_stream().cuda_stream)
    dj = api.DeviceJobs(_J(k_cap, None), "cuda:0", torch)
    d = torch.from_numpy(mats).cuda()
    s.repair_population(dj, d, round=rnd, generation=gen, first_candidate=0)
    s.sync_status()
    out = d.cpu().numpy()
    changed = 0
    for c in range(mats.shape[0]):
        want = oracle.repair(mats[c], cap, k_cap, k_max, n_max, seed, rnd, c, gen)
        assert np.array_equal(out[c], want), (name, c, mats[c].tolist(), out[c].tolist(), want.tolist())
        changed += int(not np.array_equal(want, mats[c]))
        if c % 97 == 0:
            assert feasible(out[c], cap, np.minimum(k_cap, k_max), n_max)
    assert 0 < changed < mats.shape[0]            # both feasible and infeasible inputs occurred
    s.close()
