"""The schedule builder's integer tables (closed forms) against the oracle's (Algorithm-1 recursion,
message walk).  Host-only: no GPU needed."""
import numpy as np
import pytest

import oracle
from paper_2602_17254_b200 import binding, build

LAT, BW = binding.LATENCY_OPTIMAL, binding.BANDWIDTH_OPTIMAL
TOPOS = [(3,), (9,), (27,), (81,), (243,), (3, 3), (9, 9), (3, 3, 3), (9, 9, 9), (3, 9), (27, 3), (3, 3, 9)]


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


@pytest.mark.parametrize("dims", TOPOS)
def test_steps_and_peers_match_oracle(dims):
    for variant in (LAT, BW):
        p = binding.Plan(dims, variant)
        n, S = oracle.num_steps(dims)
        assert (p.n, p.ndims, p.rows) == (n, len(dims), S if variant == LAT else 2 * S)
        for c in range(len(dims)):
            want = oracle.step_list(dims, c)
            for row in range(p.rows):
                t = row if row < S else 2 * S - 1 - row
                assert p.step(c, row) == want[t]
                if n <= 243 or row in (0, p.rows - 1):
                    assert np.array_equal(p.peers(c, row), oracle.peers(dims, t, c))


@pytest.mark.parametrize("dims", [(9,), (27,), (81,), (9, 9), (3, 3, 3), (3, 9), (27, 3), (3, 3, 9)])
def test_closed_form_send_sets_match_algorithm1(dims):
    p = binding.Plan(dims, BW)
    n, S = oracle.num_steps(dims)
    for c in range(len(dims)):
        for t in range(S):
            for dst in range(n):
                assert np.array_equal(p.send_set(c, t, dst), oracle.send_set(dims, dst, t, c)), (c, t, dst)


def test_send_sets_9x9x9_sampled():
    dims = (9, 9, 9)
    p = binding.Plan(dims, BW)
    rng = np.random.default_rng(0)
    for c in range(3):
        for t in range(6):
            for dst in rng.integers(0, 729, 6):
                assert np.array_equal(p.send_set(c, t, int(dst)), oracle.send_set(dims, int(dst), t, c))


@pytest.mark.parametrize("algo", [binding.ALGO_BRUCK, binding.ALGO_RECDOUB])
def test_comparator_tables(algo):
    dims = (27,) if algo == binding.ALGO_BRUCK else (16,)
    p = binding.Plan(dims, BW, algo)
    n, S = oracle.num_steps(dims, algo)
    assert (p.n, p.rows) == (n, 2 * S)
    for t in range(S):
        assert p.step(0, t) == oracle.step_list(dims, 0, algo)[t]
        assert np.array_equal(p.peers(0, t), oracle.peers(dims, t, 0, algo))
        for dst in range(n):
            assert np.array_equal(p.send_set(0, t, dst), oracle.send_set(dims, dst, t, 0, algo))


@pytest.mark.parametrize("dims,count", [((9,), 1024), ((81,), 2 ** 21), ((9, 9, 9), 2 ** 23), ((243,), 8192), ((3, 9), 5),
                                         ((9, 9), 1000)])
def test_block_bounds_match_oracle(dims, count):
    p = binding.Plan(dims, BW)
    for c in range(len(dims)):
        assert np.array_equal(p.block_bounds(count, c), oracle.block_bounds(count, len(dims), p.n, c))


@pytest.mark.parametrize("dims,count", [((9,), 1024), ((27,), 1000), ((9, 9), 1000), ((3, 3, 3), 77), ((3, 9), 500)])
def test_message_bytes_match_oracle_link_walk(dims, count):
    """Per-message bytes (closed-form sets x real block lengths) must reproduce the oracle's per-link
    byte tallies: on a dist-1 row every + link carries exactly one message, the one to node+1."""
    for variant in (LAT, BW):
        p = binding.Plan(dims, variant)
        ll = oracle.link_loads(dims, variant, count, 4)
        n, S = oracle.num_steps(dims)
        for c in range(len(dims)):
            for row in range(p.rows):
                d, dist = p.step(c, row)
                if dist != 1:
                    continue
                mb = p.message_bytes(count, 4, c, row)
                peers = p.peers(c, row)
                for r in range(n):
                    right = peers[r, 1]
                    want = ll["bytes"][row, r, d, 0]      # + link leaving r: the message r -> right
                    got = mb[right] if row < S or variant == LAT else mb[r]
                    assert got == want


def test_config1_message_bytes_by_hand():
    """Ring 9, 1024 int32 elements, bandwidth form: blocks of 113/114 elements."""
    p = binding.Plan((9,), BW)
    b = p.block_bounds(1024, 0)
    assert b.tolist() == [(j * 1024) // 9 for j in range(10)]
    ln = np.diff(b)
    for dst in range(9):
        assert p.message_bytes(1024, 4, 0, 0)[dst] == 4 * sum(ln[j] for j in range(9) if j % 3 == dst % 3)
        assert p.message_bytes(1024, 4, 0, 1)[dst] == 4 * ln[dst]
    lat = binding.Plan((9,), LAT)
    assert np.all(lat.message_bytes(1024, 4, 0, 1) == 4096)
