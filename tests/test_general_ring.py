"""Rings whose size is no power of three (Sec. 4.4): pins of the oracle against what the paper and
the arithmetic fix, and the library's host-side schedule against the oracle.  No GPU needed."""
import math
import os

import numpy as np
import pytest

import oracle
from paper_2602_17254_b200 import binding

SIZES = [2, 4, 5, 6, 7, 8, 10, 11, 13, 20, 26, 28, 32, 40, 53, 80, 82, 100]


def _pow3(n):
    while n % 3 == 0:
        n //= 3
    return n == 1


def _ceil_log3(n):
    s, p = 0, 1
    while p < n:
        p *= 3
        s += 1
    return s


@pytest.mark.parametrize("n", list(range(2, 260)))
def test_steps_and_distances(n):
    """ceil(log3 n) steps; distances 3^k for k < floor(log3 n), then ceil((n - 3^floor(log3 n)) / 2) (Sec. 4.4)."""
    S, dist = oracle.gen_num_steps(n)
    assert S == _ceil_log3(n)
    s = int(math.floor(math.log(n, 3) + 1e-9))
    assert dist[:s] == [3 ** k for k in range(s)]
    if not _pow3(n):
        assert len(dist) == s + 1 and dist[s] == -((3 ** s - n) // 2)


def test_example_32_distance():
    """Sec. 4.4: 32 nodes: 27 covered by the regular steps, 5 left, final distance 3."""
    S, dist = oracle.gen_num_steps(32)
    assert S == 4 and dist == [1, 3, 9, 3]


def test_figure_seven_nodes():
    """Sec. 4.4, figure for 7 nodes: two steps; in the first a node sends two blocks per direction to
    its neighbours, in the final one a single block at distance two (congestion two)."""
    k = 5
    ll = oracle.gen_link_loads(7, 7 * k, 4)
    S, dist = oracle.gen_num_steps(7)
    assert (S, dist) == (2, [1, 2])
    blk = 4 * k
    assert (ll["msgs"][0] == 1).all() and (ll["bytes"][0] == 2 * blk).all()
    assert (ll["msgs"][1] == 2).all() and (ll["bytes"][1] == 2 * blk).all()      # two messages of one block each
    # the AllGather mirrors it
    assert np.array_equal(ll["bytes"][2], ll["bytes"][1]) and np.array_equal(ll["bytes"][3], ll["bytes"][0])


def _golden_trees():
    path = os.path.join(os.path.dirname(__file__), "golden", "general_ring_trees.txt")
    trees = {}
    with open(path) as f:
        for line in f:
            line = line.split("#")[0].split()
            if line:
                n, v, q, t = map(int, line)
                trees.setdefault(n, {})[v] = (q, t)
    return trees


@pytest.mark.parametrize("n", [5, 7, 8, 10])
def test_tree_equals_the_hand_worked_one(n):
    """tests/golden/general_ring_trees.txt: parent and step of every node for block 0, worked by hand from the
    stated rule (Sec. 4.4 fixes steps and distances; holder order and left-before-right are the reading).  Every
    other block's tree is that one rotated."""
    gold = _golden_trees()[n]
    assert sorted(gold) == list(range(n))
    par, stp = oracle.gen_tree(n)
    for b in range(n):
        for v in range(n):
            q, t = gold[(v - b) % n]
            assert stp[b, v] == t, (b, v)
            assert par[b, v] == (-1 if q < 0 else (q + b) % n), (b, v)


@pytest.mark.parametrize("n", SIZES)
def test_tree_is_spanning_and_ordered(n):
    """Every node but the owner gets a block exactly once, from a node at that step's distance that got
    it in an earlier AllGather step (a later Reduce-Scatter step)."""
    S, dist = oracle.gen_num_steps(n)
    par, stp = oracle.gen_tree(n)
    for b in range(n):
        assert par[b, b] == -1 and stp[b, b] == -1
        for v in range(n):
            if v == b:
                continue
            q, t = par[b, v], stp[b, v]
            assert 0 <= t < S and (v - q) % n in (dist[t] % n, (-dist[t]) % n)
            assert q == b or stp[b, q] > t
        # the tree of block b is the tree of block 0 rotated by b
        assert np.array_equal(stp[b], np.roll(stp[0], b))


@pytest.mark.parametrize("n", SIZES)
def test_int32_sum_and_volume(n):
    """The result is the sum; per phase a node sends every block but one exactly once: m (n-1)/n bytes,
    inside the paper's bound of 2m for the whole AllReduce (Sec. 4.4)."""
    k = 3
    rng = np.random.default_rng(n)
    x = rng.integers(-2 ** 31, 2 ** 31 - 1, size=(n, n * k), dtype=np.int64).astype(np.int32)
    y, ctr = oracle.gen_allreduce(x, counters=True)
    want = x.astype(np.int64).sum(0).astype(np.int32)       # wraps modulo 2^32
    assert (y == want[None]).all()
    m = 4 * n * k
    assert (ctr["sent_rs"] == m * (n - 1) // n).all() and (ctr["sent_ag"] == m * (n - 1) // n).all()
    ll = oracle.gen_link_loads(n, n * k, 4)
    assert np.array_equal(ll["sent"], ctr["sent_rs"] + ctr["sent_ag"]) and (ll["sent"] <= 2 * m).all()


@pytest.mark.parametrize("n", [5, 7, 10, 32, 100])
@pytest.mark.parametrize("E", [0, 1, 3, 101])
def test_ragged_lengths(n, E):
    x = np.random.default_rng(E + n).integers(-1000, 1000, size=(n, E), dtype=np.int32)
    assert (oracle.gen_allreduce(x) == x.sum(0, dtype=np.int32)[None]).all()
    # a window of a longer vector gives the same values as the full run
    if E > 2:
        full = oracle.gen_allreduce(x)
        part = oracle.gen_allreduce(np.ascontiguousarray(x[:, 1:E - 1]), E=E, e0=1)
        assert np.array_equal(part, full[:, 1:E - 1])


@pytest.mark.parametrize("n", [n for n in SIZES if n > 2])
def test_final_step_congestion_is_its_distance(n):
    """Sec. 4.4: in the final step every link carries as many messages as the step's distance."""
    S, dist = oracle.gen_num_steps(n)
    ll = oracle.gen_link_loads(n, 4 * n, 4)
    assert (ll["msgs"][S - 1] == dist[S - 1]).all()
    assert (ll["msgs"][S] == dist[S - 1]).all()
    # regular steps: at most their distance
    for t in range(S - 1):
        assert ll["max_msgs"][t] <= dist[t]


@pytest.mark.parametrize("n", [3, 9, 27, 81])
def test_power_of_three_gives_the_regular_schedule(n):
    """With nothing to skip the rule is the regular schedule: same bits, same link loads."""
    rng = np.random.default_rng(n)
    x = rng.standard_normal((n, 2 * n + 1)).astype(np.float32)
    a = oracle.gen_allreduce(x)
    b = oracle.allreduce([n], oracle.VARIANT_BANDWIDTH, x)
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))
    la = oracle.gen_link_loads(n, 2 * n + 1, 4)
    lb = oracle.link_loads([n], oracle.VARIANT_BANDWIDTH, 2 * n + 1, 4)
    for key in ("msgs", "bytes", "max_msgs", "max_bytes"):
        assert np.array_equal(la[key], lb[key])


def _tree_value(x, b, v, par, stp, dist, col):
    """binary32 value node v forwards for block b: (from_left + own) + from_right, step by step."""
    n = x.shape[0]
    acc = np.float32(x[v, col])
    for t in range(len(dist)):
        if v != b and t >= stp[b, v]:
            break
        ql, qr = (v - dist[t]) % n, (v + dist[t]) % n
        if par[b, ql] == v and stp[b, ql] == t:
            acc = np.float32(_tree_value(x, b, ql, par, stp, dist, col) + acc)
        if qr != ql and par[b, qr] == v and stp[b, qr] == t:
            acc = np.float32(acc + _tree_value(x, b, qr, par, stp, dist, col))
    return acc


@pytest.mark.parametrize("n", [2, 4, 7, 10, 32])
def test_float32_order_against_tree_evaluator(n):
    """The binary32 result of every block is its tree evaluated node by node in the stated order, and it
    stays within the usual bound of the exact sum."""
    S, dist = oracle.gen_num_steps(n)
    par, stp = oracle.gen_tree(n)
    rng = np.random.default_rng(100 + n)
    x = (rng.standard_normal((n, n)) * 10.0 ** rng.integers(-3, 4, size=(n, n))).astype(np.float32)
    y = oracle.gen_allreduce(x)                 # E = n: block b is column b
    for b in range(n):
        want = _tree_value(x, b, b, par, stp, dist, b)
        assert (y[:, b].view(np.uint32) == np.float32(want).view(np.uint32)).all()
    exact = x.astype(np.float64).sum(0)
    bound = 2e-6 * np.abs(x.astype(np.float64)).sum(0)
    assert (np.abs(y.astype(np.float64) - exact[None]) <= bound[None]).all()


# ------------------------------------------------------------------ the library's host side

@pytest.mark.parametrize("n", SIZES + [244, 1000])
def test_plan_matches_oracle(n):
    S, dist = oracle.gen_num_steps(n)
    plan = binding.Plan([n], binding.BANDWIDTH_OPTIMAL)
    assert plan.n == n and plan.rows == 2 * S
    for row in range(2 * S):
        t = row if row < S else 2 * S - 1 - row
        assert plan.step(0, row) == (0, dist[t])
    par, stp = oracle.gen_tree(n)
    for t in range(S):
        for dst in sorted({0, 1, n // 2, n - 1}):
            want = np.zeros(n, np.uint8)
            for j in range(n):
                ql, qr = (dst - dist[t]) % n, (dst + dist[t]) % n
                if par[j, ql] == dst and stp[j, ql] == t:
                    want[j] |= 1
                if qr != ql and par[j, qr] == dst and stp[j, qr] == t:
                    want[j] |= 2
            assert np.array_equal(plan.send_mask(0, t, dst), want)
    # bytes sent by every node, summed over rows and both directions
    E = 3 * n + 5
    sent = np.zeros(n, np.int64)
    for row in range(2 * S):
        for side in (0, 1):
            sent += plan.message_bytes_side(E, 4, 0, row, side)
    assert np.array_equal(sent, oracle.gen_link_loads(n, E, 4)["sent"])
    plan.destroy()


def test_message_bytes_side_regular_plans():
    """For the regular schedules the per-side bytes are the per-row message sizes of the closed form."""
    for dims, variant in (([27], binding.BANDWIDTH_OPTIMAL), ([9, 3], binding.BANDWIDTH_OPTIMAL), ([9], binding.LATENCY_OPTIMAL)):
        plan = binding.Plan(dims, variant)
        E = 1000
        sent = np.zeros(plan.n, np.int64)
        for c in range(len(dims)):
            for row in range(plan.rows):
                for side in (0, 1):
                    sent += plan.message_bytes_side(E, 4, c, row, side)
        assert np.array_equal(sent, oracle.bytes_sent(dims, variant, E, 4))
        plan.destroy()


def test_unsupported_forms():
    for dims, variant in (([7], binding.LATENCY_OPTIMAL), ([7, 3], binding.LATENCY_OPTIMAL), ([33, 32], binding.BANDWIDTH_OPTIMAL),
                          ([2, 2, 2, 2, 2], binding.BANDWIDTH_OPTIMAL), ([1025], binding.BANDWIDTH_OPTIMAL)):
        with pytest.raises(binding.TrivanceError) as e:
            binding.Plan(dims, variant)
        assert e.value.status == binding.ERR_UNSUPPORTED
    plan = binding.Plan([10], binding.BANDWIDTH_OPTIMAL)
    assert plan.kernel_supported(binding.KERNEL_FUSED) and plan.kernel_supported(binding.KERNEL_STEP)
    with pytest.raises(binding.TrivanceError) as e:
        plan.message_bytes(100, 4, 0, 0)
    assert e.value.status == binding.ERR_UNSUPPORTED
    plan.destroy()
