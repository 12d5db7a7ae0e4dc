"""Tori with sides that are no powers of three (Sec. 4.4 composed with Sec. 5, bandwidth-optimal form): pins of the
oracle against what the paper and the arithmetic fix, against the (separately pinned) ring oracle, and against the
regular schedule where the sides are powers of three.  No GPU needed."""
import numpy as np
import pytest

import oracle
from paper_2602_17254_b200 import binding

TORI = [(4, 4), (8, 8), (7, 3), (3, 10), (2, 5), (5, 5), (2, 2), (4, 4, 4), (2, 3, 4), (6, 9), (16, 8)]
BW = oracle.VARIANT_BANDWIDTH


def _ceil_log3(n):
    s, p = 0, 1
    while p < n:
        p *= 3
        s += 1
    return s


def _coords(r, dims):
    out = []
    for a in dims:
        out.append(r % a)
        r //= a
    return out


def _rank(x, dims):
    r, st = 0, 1
    for v, a in zip(x, dims):
        r += (v % a) * st
        st *= a
    return r


@pytest.mark.parametrize("dims", TORI + [(32, 32), (8, 64), (16, 16, 4)])
def test_steps_are_the_ring_steps_of_every_dimension_in_round_robin_order(dims):
    """S = sum over dimensions of ceil(log3 side) (Sec. 4.4 per ring, one collective per dimension, Sec. 5); collective
    c starts on dimension c and moves on every step; a dimension's distances come in its ring's order."""
    n, S = oracle.gent_num_steps(dims)
    assert n == int(np.prod(dims)) and S == sum(_ceil_log3(a) for a in dims)
    ring = [oracle.gen_num_steps(a)[1] for a in dims]
    D = len(dims)
    for c in range(D):
        steps = oracle.gent_step_list(dims, c)
        assert len(steps) == S and steps[0][0] == c
        for d in range(D):
            assert [x for dd, x in steps if dd == d] == ring[d]
        left = [len(ring[d]) for d in range(D)]
        cur = c
        for dd, _ in steps:                     # round robin, skipping exhausted dimensions
            while left[cur] == 0:
                cur = (cur + 1) % D
            assert dd == cur
            left[cur] -= 1
            cur = (cur + 1) % D


def test_example_32x32():
    """32 x 32 (a torus the paper evaluates): four steps per dimension, distances 1, 3, 9 and the final 3 (Sec. 4.4)."""
    assert oracle.gent_step_list((32, 32), 0) == [(0, 1), (1, 1), (0, 3), (1, 3), (0, 9), (1, 9), (0, 3), (1, 3)]
    assert oracle.gent_step_list((32, 32), 1) == [(1, 1), (0, 1), (1, 3), (0, 3), (1, 9), (0, 9), (1, 3), (0, 3)]


@pytest.mark.parametrize("n", [2, 5, 7, 10, 32])
def test_one_dimension_is_the_ring(n):
    x = np.random.default_rng(n).standard_normal((n, 3 * n + 1)).astype(np.float32)
    assert np.array_equal(oracle.gent_allreduce((n,), x).view(np.uint32), oracle.gen_allreduce(x).view(np.uint32))
    pa, sa = oracle.gent_tree((n,))
    pb, sb = oracle.gen_tree(n)
    assert np.array_equal(pa, pb) and np.array_equal(sa, sb)
    la, lb = oracle.gent_link_loads((n,), 2 * n + 1), oracle.gen_link_loads(n, 2 * n + 1)
    for key in ("msgs", "bytes", "max_msgs", "max_bytes", "sent"):
        assert np.array_equal(la[key], lb[key])


@pytest.mark.parametrize("dims", [(3, 9), (9, 9), (3, 3, 3), (27, 3), (3, 3, 9)])
def test_power_of_three_sides_give_the_regular_schedule(dims):
    """Nothing is ever skipped: same bits and same link loads as the schedule of Sec. 5."""
    n = int(np.prod(dims))
    x = np.random.default_rng(n).standard_normal((n, 2 * n + 7)).astype(np.float32)
    a = oracle.gent_allreduce(dims, x)
    b = oracle.allreduce(dims, BW, x)
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))
    la, lb = oracle.gent_link_loads(dims, 5 * n + 3), oracle.link_loads(dims, BW, 5 * n + 3)
    for key in ("msgs", "bytes", "max_msgs", "max_bytes"):
        assert np.array_equal(la[key], lb[key])
    for c in range(len(dims)):
        assert oracle.gent_step_list(dims, c) == oracle.step_list(dims, c)


@pytest.mark.parametrize("dims", TORI)
def test_tree_is_the_product_of_the_ring_trees(dims):
    """A node gets block 0 when the LAST of its coordinates is reached, along that dimension, from the parent its
    ring tree names: the tree of a torus is the per-dimension ring trees (pinned on their own by hand-worked
    tables) composed in the collective's step order.  Every other block's tree is that one translated."""
    n, S = oracle.gent_num_steps(dims)
    D = len(dims)
    ring = [oracle.gen_tree(a) for a in dims]
    for c in range(D):
        steps = oracle.gent_step_list(dims, c)
        where = {}                                  # (dim, k-th visit) -> position in the step list
        seen = [0] * D
        for t, (d, _) in enumerate(steps):
            where[(d, seen[d])] = t
            seen[d] += 1
        par, stp = oracle.gent_tree(dims, c)
        for v in range(n):
            o = _coords(v, dims)
            if v == 0:
                assert par[0, 0] == -1 and stp[0, 0] == -1
                continue
            t_of = {d: where[(d, int(ring[d][1][0, o[d]]))] for d in range(D) if o[d]}
            d_star = min(t_of, key=t_of.get)        # AllGather runs the steps backwards: the smallest step comes last
            assert stp[0, v] == t_of[d_star]
            q = list(o)
            q[d_star] = int(ring[d_star][0][0, o[d_star]])
            assert par[0, v] == _rank(q, dims)
        for b in sorted({1, n // 2, n - 1}):
            bc = _coords(b, dims)
            for v in range(n):
                v0 = _rank([x - y for x, y in zip(_coords(v, dims), bc)], dims)
                assert stp[b, v] == stp[0, v0]
                if v != b:
                    p0 = _coords(int(par[0, v0]), dims)
                    assert par[b, v] == _rank([x + y for x, y in zip(p0, bc)], dims)


@pytest.mark.parametrize("dims", TORI)
def test_tree_is_spanning_and_ordered(dims):
    n, S = oracle.gent_num_steps(dims)
    for c in range(len(dims)):
        steps = oracle.gent_step_list(dims, c)
        par, stp = oracle.gent_tree(dims, c)
        for b in (0, n - 1):
            for v in range(n):
                if v == b:
                    continue
                q, t = int(par[b, v]), int(stp[b, v])
                d, dist = steps[t]
                cv, cq = _coords(v, dims), _coords(q, dims)
                assert all(cv[k] == cq[k] for k in range(len(dims)) if k != d)
                assert (cv[d] - cq[d]) % dims[d] in (dist % dims[d], (-dist) % dims[d])
                assert q == b or stp[b, q] > t


@pytest.mark.parametrize("dims", TORI + [(32, 32)])
def test_int32_sum_volume_and_windows(dims):
    """Every rank ends with the column sums (wrapping); per phase a node sends every block of every collective but
    its own exactly once: m (n - 1) / n bytes, within the paper's bound (Sec. 4.4); a window gives the full run's columns."""
    n, S = oracle.gent_num_steps(dims)
    D = len(dims)
    k = 2 if n < 200 else 1
    E = n * D * k
    rng = np.random.default_rng(n)
    x = rng.integers(-2 ** 31, 2 ** 31 - 1, size=(n, E), dtype=np.int64).astype(np.int32)
    y, ctr = oracle.gent_allreduce(dims, x, counters=True)
    want = x.astype(np.int64).sum(0).astype(np.int32)
    assert (y == want[None]).all()
    m = 4 * E
    assert (ctr["sent_rs"] == m * (n - 1) // n).all() and (ctr["sent_ag"] == m * (n - 1) // n).all()
    ll = oracle.gent_link_loads(dims, E, 4)
    assert np.array_equal(ll["sent"], ctr["sent_rs"] + ctr["sent_ag"]) and (ll["sent"] <= 2 * m).all()
    w0, w1 = E // 3 + 1, E - 2
    part = oracle.gent_allreduce(dims, np.ascontiguousarray(x[:, w0:w1]), E=E, e0=w0)
    assert np.array_equal(part, y[:, w0:w1])


@pytest.mark.parametrize("dims", [(4, 4), (7, 3), (2, 3, 4)])
@pytest.mark.parametrize("E", [0, 1, 5, 101])
def test_ragged_lengths(dims, E):
    n = int(np.prod(dims))
    x = np.random.default_rng(E + n).integers(-1000, 1000, size=(n, E), dtype=np.int32)
    assert (oracle.gent_allreduce(dims, x) == x.sum(0, dtype=np.int32)[None]).all()
    assert (oracle.allreduce(dims, BW, x) == x.sum(0, dtype=np.int32)[None]).all()      # the front end routes here


@pytest.mark.parametrize("dims", [(4, 4), (8, 8), (5, 5), (4, 4, 4), (32, 32)])
def test_final_step_congestion_is_its_distance(dims):
    """Equal sides: in every row each dimension carries one collective; in the last step of a dimension every one of
    its links carries as many messages as the step's distance (Sec. 4.4), in the regular steps at most the distance."""
    n, S = oracle.gent_num_steps(dims)
    D = len(dims)
    ll = oracle.gent_link_loads(dims, 4 * n * D, 4)
    for c in range(D):
        steps = oracle.gent_step_list(dims, c)
        last = {d: max(t for t, (dd, _) in enumerate(steps) if dd == d) for d in range(D)}
        for t, (d, dist) in enumerate(steps):
            for row in (t, 2 * S - 1 - t):
                if t == last[d]:
                    assert (ll["msgs"][row][:, d, :] == dist).all()
                else:
                    assert (ll["msgs"][row][:, d, :] <= dist).all()


def _tree_value(x, dims, steps, b, v, par, stp, col):
    """binary32 value node v forwards for block b: (from_left + own) + from_right, step by step."""
    acc = np.float32(x[v, col])
    for t, (d, dist) in enumerate(steps):
        if v != b and t >= stp[b, v]:
            break
        cv = _coords(v, dims)
        ql = _rank([cv[k] - (dist if k == d else 0) for k in range(len(dims))], dims)
        qr = _rank([cv[k] + (dist if k == d else 0) for k in range(len(dims))], dims)
        if par[b, ql] == v and stp[b, ql] == t:
            acc = np.float32(_tree_value(x, dims, steps, b, ql, par, stp, col) + acc)
        if qr != ql and par[b, qr] == v and stp[b, qr] == t:
            acc = np.float32(acc + _tree_value(x, dims, steps, b, qr, par, stp, col))
    return acc


@pytest.mark.parametrize("dims", [(4, 4), (7, 3), (2, 5), (2, 3, 4), (8, 8)])
def test_float32_order_against_tree_evaluator(dims):
    """The binary32 result of every block of every collective is its tree evaluated node by node in the stated order;
    all ranks end with the same bits; the result stays within the usual bound of the exact sum."""
    n, S = oracle.gent_num_steps(dims)
    D = len(dims)
    rng = np.random.default_rng(100 + n)
    E = n * D                                       # collective c = columns [c n, (c + 1) n), block b = column c n + b
    x = (rng.standard_normal((n, E)) * 10.0 ** rng.integers(-3, 4, size=(n, E))).astype(np.float32)
    y = oracle.gent_allreduce(dims, x)
    for c in range(D):
        steps = oracle.gent_step_list(dims, c)
        par, stp = oracle.gent_tree(dims, c)
        for b in range(n):
            want = _tree_value(x, dims, steps, b, b, par, stp, c * n + b)
            assert (y[:, c * n + b].view(np.uint32) == np.float32(want).view(np.uint32)).all()
    exact = x.astype(np.float64).sum(0)
    bound = 2e-6 * np.abs(x.astype(np.float64)).sum(0)
    assert (np.abs(y.astype(np.float64) - exact[None]) <= bound[None]).all()


# ------------------------------------------------------------------ the library's host side

@pytest.mark.parametrize("dims", TORI + [(32, 32), (8, 64), (16, 16, 4)])
def test_plan_matches_oracle(dims):
    """The library derives the tree as the product of per-dimension ring trees (no holder list); the oracle grows it
    with the holder list.  Step lists, receive masks and bytes sent must agree."""
    n, S = oracle.gent_num_steps(dims)
    D = len(dims)
    plan = binding.Plan(dims, binding.BANDWIDTH_OPTIMAL)
    assert plan.n == n and plan.rows == 2 * S and plan.nslices == D
    assert plan.kernel_supported(binding.KERNEL_FUSED) and plan.kernel_supported(binding.KERNEL_STEP)
    E = 3 * n * D + 5
    sent = np.zeros(n, np.int64)
    for c in range(D):
        steps = oracle.gent_step_list(dims, c)
        for row in range(2 * S):
            t = row if row < S else 2 * S - 1 - row
            assert plan.step(c, row) == steps[t]
            for side in (0, 1):
                sent += plan.message_bytes_side(E, 4, c, row, side)
        par, stp = oracle.gent_tree(dims, c)
        for t, (d, dist) in enumerate(steps):
            for dst in sorted({0, 1, n // 2, n - 1}):
                cd = _coords(dst, dims)
                ql = _rank([cd[k] - (dist if k == d else 0) for k in range(D)], dims)
                qr = _rank([cd[k] + (dist if k == d else 0) for k in range(D)], dims)
                want = np.zeros(n, np.uint8)
                want[(par[:, ql] == dst) & (stp[:, ql] == t)] |= 1
                if qr != ql:
                    want[(par[:, qr] == dst) & (stp[:, qr] == t)] |= 2
                assert np.array_equal(plan.send_mask(c, t, dst), want), (c, t, dst)
    assert np.array_equal(sent, oracle.gent_link_loads(dims, E, 4)["sent"])
    plan.destroy()


def test_latency_form_is_refused_for_such_sides():
    for dims in ((4, 4), (7, 3), (3, 10)):
        with pytest.raises(binding.TrivanceError) as e:
            binding.Plan(dims, binding.LATENCY_OPTIMAL)
        assert e.value.status == binding.ERR_UNSUPPORTED
