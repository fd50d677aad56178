"""Pins of the oracle's Philox4x32-10 against an independent library implementation."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest

_TRITON_SCRIPT = r"""
import os, sys, json
os.environ["TRITON_INTERPRET"] = "1"
import numpy as np, torch, triton, triton.language as tl
n = int(sys.argv[1])
@triton.jit
def k(out, inp, N: tl.constexpr):
    o = tl.arange(0, N)
    c0 = tl.load(inp + o); c1 = tl.load(inp + N + o); c2 = tl.load(inp + 2 * N + o); c3 = tl.load(inp + 3 * N + o)
    k0 = tl.load(inp + 4 * N + o); k1 = tl.load(inp + 5 * N + o)
    a, b, c, d = tl.philox_impl(c0, c1, c2, c3, k0, k1)
    tl.store(out + o, a); tl.store(out + N + o, b); tl.store(out + 2 * N + o, c); tl.store(out + 3 * N + o, d)
rng = np.random.default_rng(12345)
inp = rng.integers(0, 2**32, (6, n), dtype=np.uint64).astype(np.uint32)
inp[:, 0] = 0
inp[:, 1] = 0xFFFFFFFF
t_in = torch.from_numpy(inp.view(np.int32).copy()).view(torch.uint32).reshape(-1)
t_out = torch.zeros(4 * n, dtype=torch.uint32)
k[(1,)](t_out, t_in, N=n)
print(json.dumps({"inp": inp.tolist(), "out": t_out.view(torch.int32).numpy().view(np.uint32).reshape(4, n).tolist()}))
"""


def test_against_library_philox(oracle):
    """Triton ships its own Philox4x32-10 (`tl.philox_impl`); its CPU interpreter runs it
    here, in a child process, on random counters and keys plus the all-zero and all-one
    blocks.  Used purely as an independent implementation of the published generator."""
    try:
        res = subprocess.run([sys.executable, "-c", _TRITON_SCRIPT, "256"], capture_output=True,
                             text=True, timeout=600, env={**os.environ, "TRITON_INTERPRET": "1"})
    except Exception as e:  # pragma: no cover
        pytest.skip("triton interpreter unavailable: %r" % (e,))
    if res.returncode != 0:
        pytest.skip("triton interpreter unavailable: " + res.stderr[-300:])
    data = json.loads(res.stdout.strip().splitlines()[-1])
    inp = np.array(data["inp"], dtype=np.uint32)
    out = np.array(data["out"], dtype=np.uint32)
    for i in range(inp.shape[1]):
        got = oracle.philox4x32_10(inp[0:4, i], inp[4:6, i])
        assert got.tolist() == out[:, i].tolist(), i


M0, M1 = 0xD2511F53, 0xCD9E8D57
W0, W1 = 0x9E3779B9, 0xBB67AE85
MASK = 0xFFFFFFFF


def _inverse(out, key):
    """Philox is a bijection of the counter for a fixed key: undo the ten rounds using the
    modular inverses of the two (odd) multipliers."""
    i0, i1 = pow(M0, -1, 1 << 32), pow(M1, -1, 1 << 32)
    c = [int(x) for x in out]
    for r in reversed(range(10)):
        k0 = (int(key[0]) + r * W0) & MASK
        k1 = (int(key[1]) + r * W1) & MASK
        p0 = (c[3] * i0) & MASK          # previous c0
        p2 = (c[1] * i1) & MASK          # previous c2
        p1 = c[0] ^ ((M1 * p2) >> 32) ^ k0
        p3 = c[2] ^ ((M0 * p0) >> 32) ^ k1
        c = [p0, p1, p2, p3]
    return c


def test_bijection(oracle):
    rng = np.random.default_rng(7)
    for _ in range(300):
        ctr = rng.integers(0, 2**32, 4, dtype=np.uint64).astype(np.uint32)
        key = rng.integers(0, 2**32, 2, dtype=np.uint64).astype(np.uint32)
        out = oracle.philox4x32_10(ctr, key)
        assert _inverse(out, key) == [int(x) for x in ctr]


def test_uniformity_and_stream_layout(oracle):
    # operator stream: key = (seed_lo ^ seed_hi, round), counter = (idx, cand, gen, slot)
    seed = 0x0123456789ABCDEF
    w = oracle.draw(seed, 9, 3, 4, 5, 2)
    assert w.tolist() == oracle.philox4x32_10([3, 4, 5, 2], [(seed & MASK) ^ (seed >> 32), 9]).tolist()
    words = np.concatenate([oracle.draw(1, 0, i, 0, 0, 0) for i in range(4096)])
    hist = np.bincount(words >> 24, minlength=256)
    expect = words.size / 256
    chi2 = ((hist - expect) ** 2 / expect).sum()
    assert chi2 < 350.0            # 255 dof: mean 255, sd ~22.6
    assert abs(words.astype(np.float64).mean() / 2**32 - 0.5) < 0.01
