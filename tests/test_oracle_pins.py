"""Pins the CPU oracle to what the paper and plain mathematics fix.

Nothing here touches the CUDA library.  Each test states which passage of the
paper (or which definition) it checks.  The independent pieces written here are
deliberately of a different shape from the oracle's step-by-step message
passing: column sums, closed forms, a recursive ternary-tree evaluator, and a
set-based reachability enumeration.
"""
import itertools
import os

import numpy as np
import pytest

import oracle
from paper_2602_17254_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")
LAT, BW = oracle.VARIANT_LATENCY, oracle.VARIANT_BANDWIDTH

TOPOS = [(3,), (9,), (27,), (81,), (3, 3), (9, 9), (3, 3, 3), (3, 9), (9, 3), (3, 3, 9)]


def _n(dims):
    return int(np.prod(dims))


def _golden_rows(name):
    rows = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


# ------------------------------------------------------------------ result (Sec. 2.2)

@pytest.mark.parametrize("dims", TOPOS)
@pytest.mark.parametrize("variant", [LAT, BW])
@pytest.mark.parametrize("E", [1, 2, 5, 26, 27, 100, 731])
def test_int32_every_rank_holds_the_column_sum(dims, variant, E):
    """Sec. 2.2: every rank ends with the reduction over all n vectors (exact for integers)."""
    n = _n(dims)
    x = np.random.default_rng(E * 131 + n).integers(-1000, 1001, size=(n, E), dtype=np.int32)
    out = oracle.allreduce(dims, variant, x)
    want = x.sum(axis=0, dtype=np.int64).astype(np.int32)
    assert out.dtype == np.int32
    assert np.array_equal(out, np.broadcast_to(want, (n, E)))


def test_int32_wraps_modulo_2_32():
    x = np.full((9, 4), 2**30, np.int32)
    want = np.int32(np.int64(9 * 2**30 + 2**31) % 2**32 - 2**31)
    for variant in (LAT, BW):
        assert np.all(oracle.allreduce((9,), variant, x) == want)


@pytest.mark.parametrize("name", ["ring9_lat_int32"])
def test_config1_geometry_int32(name):
    w = synth.CONFIGS[name]
    x = synth.workload_inputs(w)
    assert x.shape == (9, 1024) and x.min() >= -1000 and x.max() <= 1000
    out = oracle.allreduce(w.dims, w.variant, x)
    assert np.array_equal(out, np.broadcast_to(x.sum(0, dtype=np.int64).astype(np.int32), x.shape))


# ------------------------------------------------------------------ step count (Theorem 1, Sec. 4.2; Sec. 3.2)

@pytest.mark.parametrize("dims,steps", [((3,), 1), ((9,), 2), ((27,), 3), ((81,), 4), ((243,), 5), ((729,), 6),
                                        ((9, 9), 4), ((9, 9, 9), 6), ((27, 27), 6), ((3, 9), 3)])
def test_step_count_is_log3_n(dims, steps):
    n, s = oracle.num_steps(dims)
    assert n == _n(dims) and s == steps and 3 ** s == n
    for variant, rows in ((LAT, steps), (BW, 2 * steps)):
        assert oracle.link_loads(dims, variant, 3 * n)["max_msgs"].shape == (rows,)


def test_non_power_of_three_is_refused():
    for dims in [(7,), (32,), (6, 3), (9, 8)]:
        with pytest.raises(oracle.OracleError):
            oracle.num_steps(dims)


# ------------------------------------------------------------------ peers (Sec. 4.1)

@pytest.mark.parametrize("n", [3, 9, 27, 81, 243])
def test_ring_peers_are_r_minus_and_plus_3k(n):
    s = oracle.num_steps((n,))[1]
    r = np.arange(n)
    for k in range(s):
        p = oracle.peers((n,), k)
        assert np.array_equal(p[:, 0], (r - 3 ** k) % n)
        assert np.array_equal(p[:, 1], (r + 3 ** k) % n)


def test_torus_collectives_use_distinct_dimensions_and_swap_each_step():
    """Sec. 5: collective 0 starts horizontal, collective 1 vertical; they swap in step 1 and
    return in step 2; every collective is on a different dimension in every step."""
    assert oracle.step_list((9, 9), 0) == [(0, 1), (1, 1), (0, 3), (1, 3)]
    assert oracle.step_list((9, 9), 1) == [(1, 1), (0, 1), (1, 3), (0, 3)]
    for dims in [(9, 9), (9, 9, 9), (27, 27), (3, 3, 3)]:
        D = len(dims)
        lists = [oracle.step_list(dims, c) for c in range(D)]
        for t in range(len(lists[0])):
            assert sorted(lst[t][0] for lst in lists) == list(range(D))
        for lst in lists:        # each dimension sees distances 1, 3, 9, ... in order
            for d in range(D):
                assert [x for (dd, x) in lst if dd == d] == [3 ** k for k in range(oracle.num_steps((dims[d],))[1])]


def test_torus_peers_move_along_one_dimension_only():
    dims = (3, 9)
    for c in range(2):
        for t, (d, dist) in enumerate(oracle.step_list(dims, c)):
            p = oracle.peers(dims, t, c)
            for r in range(27):
                x = [r % 3, r // 3]
                for side, sgn in ((0, -1), (1, +1)):
                    y = list(x)
                    y[d] = (y[d] + sgn * dist) % dims[d]
                    assert p[r, side] == y[0] + 3 * y[1]


# ------------------------------------------------------------------ coverage (Lemma 2, Fig. "received blocks")

def _contributors(dims, steps):
    """Row r = how often each node's data is contained in r's partial after `steps` steps
    (one-hot inputs, integer multiplicities)."""
    n = _n(dims)
    return oracle.allreduce(dims, LAT, np.eye(n, dtype=np.int32), max_steps=steps)


@pytest.mark.parametrize("n", [3, 9, 27, 81, 243])
def test_coverage_radius_after_each_step(n):
    """Lemma 2: after step k a node holds exactly the data within ring distance (3^(k+1)-1)/2, once each."""
    s = oracle.num_steps((n,))[1]
    idx = np.arange(n)
    ring_dist = np.minimum((idx[:, None] - idx[None, :]) % n, (idx[None, :] - idx[:, None]) % n)
    assert np.array_equal(_contributors((n,), 0), np.eye(n, dtype=np.int32))
    for k in range(s):
        R = (3 ** (k + 1) - 1) // 2
        assert np.array_equal(_contributors((n,), k + 1), (ring_dist <= R).astype(np.int32))


def test_ring9_worked_example():
    rows = _golden_rows("ring9_received_blocks.txt")
    assert rows
    for row in rows:
        assert row[0] == "after_step" and row[2] == "node" and row[4] == ":"
        k, r, nodes = int(row[1]), int(row[3]), sorted(int(v) for v in row[5:])
        got = _contributors((9,), k + 1)[r]
        assert sorted(np.nonzero(got)[0].tolist()) == nodes
        assert got.max() == 1
    after0 = _contributors((9,), 1)
    assert np.array_equal(after0.sum(1), np.full(9, 3))       # self + two neighbours only
    assert np.array_equal(_contributors((9,), 2), np.ones((9, 9), np.int32))


@pytest.mark.parametrize("dims", [(3, 3), (9, 9), (3, 3, 3), (3, 9)])
def test_torus_every_contribution_exactly_once(dims):
    n = _n(dims)
    x = np.tile(np.eye(n, dtype=np.int32), (1, len(dims)))      # every slice sees the one-hot pattern
    out = oracle.allreduce(dims, LAT, x)
    assert np.array_equal(out, np.ones_like(out))


# ------------------------------------------------------------------ block sets (Algorithm 1 vs closed form Pi)

def _closed_form_pi(n, p, k):
    """Sec. 4.3: Pi(n,r,p,k) = { p + sum_{i=k+1}^{s-1} eps_i 3^i mod n : eps_i in {-1,0,1} }."""
    s = round(np.log(n) / np.log(3))
    out = set()
    for eps in itertools.product((-1, 0, 1), repeat=max(s - 1 - k, 0)):
        out.add((p + sum(e * 3 ** (k + 1 + i) for i, e in enumerate(eps))) % n)
    return out


@pytest.mark.parametrize("n", [3, 9, 27, 81, 243])
def test_algorithm1_equals_closed_form(n):
    s = oracle.num_steps((n,))[1]
    for k in range(s):
        for p in range(n) if n <= 81 else range(0, n, 7):
            got = set(np.nonzero(oracle.send_set((n,), p, k))[0].tolist())
            assert got == _closed_form_pi(n, p, k)
            assert len(got) == 3 ** (s - 1 - k)               # Sec. 4.3: 3^(s-1-k) blocks


def test_block_propagation_from_step0_reaches_everyone_else():
    for n in (9, 27):
        for r in (0, 4):
            m = oracle.block_propagation((n,), r, 0)
            assert m.sum() >= n - 1 and all(m[q] for q in range(n) if q != r)


@pytest.mark.parametrize("dims", [(9,), (27,), (3, 3), (9, 3), (3, 3, 3)])
def test_block_propagation_is_every_increasing_path(dims):
    """Algorithm 1 (Sec. 4.3) reaches exactly the ranks at the end of a non-empty path whose hops are taken in
    steps of strictly increasing number >= step, each hop to one of the two peers of its step.  Brute force over
    all subsets of steps and all left/right choices."""
    n, S = oracle.num_steps(dims)
    for c in range(len(dims)):
        peers = [oracle.peers(dims, t, c) for t in range(S)]
        for step in range(S + 1):
            for r in range(0, n, 2):
                want = set()
                for mask in range(1, 1 << (S - step)):
                    used = [step + i for i in range(S - step) if mask >> i & 1]
                    for choice in itertools.product((0, 1), repeat=len(used)):
                        q = r
                        for t, side in zip(used, choice):
                            q = int(peers[t][q, side])
                        want.add(q)
                got = set(np.nonzero(oracle.block_propagation(dims, r, step, c))[0].tolist())
                assert got == want, (dims, c, step, r)


def test_ring9_send_sets_worked_by_hand():
    """n = 9: in step 0 rank 0 sends {1,4,7} to rank 1 and {8,2,5} to rank 8; in step 1 one block each."""
    f = lambda p, k: sorted(np.nonzero(oracle.send_set((9,), p, k))[0].tolist())
    assert f(1, 0) == [1, 4, 7] and f(8, 0) == [2, 5, 8]
    assert f(3, 1) == [3] and f(6, 1) == [6]


@pytest.mark.parametrize("dims", [(3, 3), (9, 9), (3, 3, 3), (3, 9)])
def test_torus_send_sets_partition_the_blocks(dims):
    """Each block is forwarded at most once per phase and reaches its owner: in every step the
    send sets towards the three nodes {left, self(kept), right} split the sender's active blocks."""
    n = _n(dims)
    for c in range(len(dims)):
        steps = oracle.step_list(dims, c)
        active = [np.ones(n, bool) for _ in range(n)]
        for t in range(len(steps)):
            p = oracle.peers(dims, t, c)
            new_active = []
            for r in range(n):
                to_l, to_r = oracle.send_set(dims, p[r, 0], t, c), oracle.send_set(dims, p[r, 1], t, c)
                keep = oracle.send_set(dims, r, t, c)
                assert not (to_l & to_r).any() and not (to_l & keep).any() and not (to_r & keep).any()
                assert np.array_equal(to_l | to_r | keep, active[r])
                new_active.append(keep)
            active = new_active
        for r in range(n):
            assert np.nonzero(active[r])[0].tolist() == [r]


# ------------------------------------------------------------------ volumes (Lemma 1, Sec. 4.2/4.3, Discussion)

@pytest.mark.parametrize("dims", [(9,), (27,), (81,), (9, 9), (3, 3, 3)])
def test_bytes_sent_and_reduced(dims):
    n, S = oracle.num_steps(dims)
    D = len(dims)
    E = n * D * 4
    m = 4 * E
    x = np.zeros((n, E), np.float32)
    _, c = oracle.allreduce(dims, BW, x, counters=True)
    assert np.all(c["sent_rs"] == m - m // n)                 # Lemma 1: m (1 - 1/n) per phase
    assert np.all(c["sent_ag"] == m - m // n)
    assert np.all(2 * c["reduced"] == 3 * (m - m // n))       # Discussion: 1.5 m (1 - 1/n)
    _, c = oracle.allreduce(dims, LAT, x, counters=True)
    # Table 1: the latency form moves log3 n times the optimum 2m (whole vector of every collective,
    # two ports, each of its log3 n steps)
    assert np.all(c["sent_rs"] == 2 * m * S)
    assert np.all(c["sent_ag"] == 0)


@pytest.mark.parametrize("n", [9, 27, 81])
def test_ring_message_sizes_shrink_by_three(n):
    """Sec. 4.1: the step-k message is m / 3^(k+1); the AllGather mirrors it."""
    s = oracle.num_steps((n,))[1]
    E = n * 5
    ll = oracle.link_loads((n,), BW, E, elem_size=4)
    for row in range(2 * s):
        k = row if row < s else 2 * s - 1 - row
        per_msg = ll["bytes"][row] // np.maximum(ll["msgs"][row], 1)
        assert np.all(per_msg == 4 * E // 3 ** (k + 1))


# ------------------------------------------------------------------ congestion (Sec. 2.1, Fig. 1, Sec. 4.1, App. B)

def test_fig1_congestion_values():
    rows = _golden_rows("fig1_max_link_congestion.txt")
    algo = {"trivance": oracle.ALGO_TRIVANCE, "bruck": oracle.ALGO_BRUCK, "recursive_doubling": oracle.ALGO_RECDOUB}
    assert len(rows) == 3
    for name, n, *want in rows:
        ll = oracle.link_loads((int(n),), LAT, 64, algo=algo[name])
        assert ll["max_msgs"].tolist() == [int(v) for v in want]


@pytest.mark.parametrize("n", [9, 27, 81, 243])
def test_trivance_congestion_is_uniform_3k(n):
    """Sec. 4.1: the congestion on all links is uniform and equals 3^k (both variants)."""
    s = oracle.num_steps((n,))[1]
    for variant in (LAT, BW):
        ll = oracle.link_loads((n,), variant, n * 2)
        for row in range(ll["msgs"].shape[0]):
            k = row if row < s else 2 * s - 1 - row
            assert np.all(ll["msgs"][row] == 3 ** k)


def test_bruck_uses_one_direction_only_and_is_three_times_trivance():
    """Sec. 3.1 / App. B: Bruck routes everything one way; its congestion is 3 * 3^k."""
    for n in (9, 27, 243):
        for variant in (LAT, BW):
            tv = oracle.link_loads((n,), variant, 3 * n)
            br = oracle.link_loads((n,), variant, 3 * n, algo=oracle.ALGO_BRUCK)
            assert np.all(br["msgs"][..., 1] == 0)
            assert np.array_equal(br["max_msgs"], 3 * tv["max_msgs"])
            assert np.array_equal(br["max_bytes"], 3 * tv["max_bytes"])


def test_recursive_doubling_congestion_2k_and_undefined_for_243():
    for q in (2, 3, 4, 5):
        ll = oracle.link_loads((2 ** q,), LAT, 64, algo=oracle.ALGO_RECDOUB)
        assert ll["max_msgs"].tolist() == [2 ** k for k in range(q)]      # App. B
    with pytest.raises(oracle.OracleError) as e:
        oracle.link_loads((243,), LAT, 64, algo=oracle.ALGO_RECDOUB)
    assert e.value.code == 2


def test_ring_tx_delay_factors():
    """Table 1: sum_k m_k c_k / m = (2/3) log3 n (bandwidth form), (n-1)/2 -> n/2 (latency form)."""
    for n in (9, 27, 81, 243):
        s = oracle.num_steps((n,))[1]
        E = 3 * n
        m = 4 * E
        assert 3 * int(oracle.link_loads((n,), BW, E)["max_bytes"].sum()) == 2 * s * m
        assert 2 * int(oracle.link_loads((n,), LAT, E)["max_bytes"].sum()) == (n - 1) * m


@pytest.mark.parametrize("dims", [(9, 9), (9, 9, 9), (27, 27), (3, 3, 3, 3)])
def test_torus_tx_delay_follows_appendix_b(dims):
    """App. B: 2 * sum_d sum_k 3^k / 3^(1+d+Dk), relative to m/D; Table 2: latency form D/2 * side."""
    D, a = len(dims), dims[0]
    n, S = oracle.num_steps(dims)
    E = n * D
    m_over_d = 4 * E // D
    from fractions import Fraction
    want = 2 * sum(Fraction(3 ** k, 3 ** (1 + d + D * k)) for d in range(D) for k in range(S // D))
    ll = oracle.link_loads(dims, BW, E)
    assert Fraction(int(ll["max_bytes"].sum()), m_over_d) == want
    assert np.all(ll["bytes"] == ll["max_bytes"][:, None, None, None])    # uniform over all links
    ll = oracle.link_loads(dims, LAT, E)
    assert int(ll["max_bytes"].sum()) == m_over_d * D * (a - 1) // 2


def test_torus_tx_delay_tends_to_table2():
    for D, want in [(int(r[1]), float(r[2])) for r in _golden_rows("tx_delay_factors.txt")]:
        closed = (3 ** D - 1) / (3 ** D - 3)
        assert abs(closed - want) < 0.006
        # finite-size value from the oracle approaches the limit from below as the side grows
        vals = []
        for a in (3, 9) if D >= 3 else (3, 9, 27):
            dims = (a,) * D
            n = a ** D
            ll = oracle.link_loads(dims, BW, n * D)
            vals.append(int(ll["max_bytes"].sum()) / (4 * n))
        assert all(v < closed for v in vals) and vals == sorted(vals)
        assert closed - vals[-1] < 0.06 * closed


# ------------------------------------------------------------------ floating point

def _tree(x, dims, steps, t, r, e):
    """Value rank r holds for column e after steps 0..t-1, straight from the definition of a joint
    reduction, (left + own) + right, with left = the peer at -dist.  Exponential, tiny n only."""
    if t == 0:
        return x[r, e]
    d, dist = steps[t - 1]
    stride = int(np.prod(dims[:d], dtype=np.int64))
    xd = (r // stride) % dims[d]
    rl = r + (((xd - dist) % dims[d]) - xd) * stride
    rr = r + (((xd + dist) % dims[d]) - xd) * stride
    a = _tree(x, dims, steps, t - 1, rl, e)
    b = _tree(x, dims, steps, t - 1, r, e)
    c = _tree(x, dims, steps, t - 1, rr, e)
    return np.float32(np.float32(a + b) + c)


@pytest.mark.parametrize("dims", [(3,), (9,), (27,), (3, 3), (3, 3, 3), (9, 3)])
def test_fp32_latency_form_is_the_ternary_tree_of_each_rank(dims):
    n, D = _n(dims), len(dims)
    E = 2 * D + 1
    x = np.random.default_rng(n).standard_normal((n, E)).astype(np.float32)
    out = oracle.allreduce(dims, LAT, x)
    for e in range(E):
        c = next(c for c in range(D) if (c * E) // D <= e < ((c + 1) * E) // D)
        steps = oracle.step_list(dims, c)
        for r in range(n):
            assert out[r, e] == _tree(x, dims, steps, len(steps), r, e)
    if n > 3:
        assert any(not np.array_equal(out[0], out[r]) for r in range(1, n))    # rows differ in rounding


@pytest.mark.parametrize("dims", [(9,), (27,), (81,), (9, 9), (3, 3, 3), (3, 9)])
@pytest.mark.parametrize("E", [7, 100, 1000])
def test_fp32_bandwidth_form_is_the_owners_latency_row(dims, E):
    """Reduce-Scatter follows the same pattern as the latency form (Sec. 4.2), so block j ends as
    rank j's latency-form value; the AllGather then copies it to everyone."""
    n, D = _n(dims), len(dims)
    x = np.random.default_rng(E + n).standard_normal((n, E)).astype(np.float32)
    lat = oracle.allreduce(dims, LAT, x)
    bw = oracle.allreduce(dims, BW, x)
    for c in range(D):
        b = oracle.block_bounds(E, D, n, c)
        for j in range(n):
            for r in range(n):
                assert np.array_equal(bw[r, b[j]:b[j + 1]], lat[j, b[j]:b[j + 1]])


@pytest.mark.parametrize("dims", [(27,), (9, 9), (3, 3, 3)])
def test_fp_paths_agree_with_int_path_on_small_integers(dims):
    n = _n(dims)
    xi = np.random.default_rng(3).integers(-1000, 1001, size=(n, 50), dtype=np.int32)
    for variant in (LAT, BW):
        want = oracle.allreduce(dims, variant, xi)
        assert np.array_equal(oracle.allreduce(dims, variant, xi.astype(np.float32)), want.astype(np.float32))
        assert np.array_equal(oracle.allreduce(dims, variant, xi.astype(np.float64)), want.astype(np.float64))


@pytest.mark.parametrize("dims,dist", [((27,), "normal"), ((81,), "normal"), ((9, 9, 9), "uniform"), ((243,), "normal")])
def test_fp32_error_bounds(dims, dist):
    """|fp32 - exact| <= 2 S 2^-24 sum|x| (each value passes through 2S roundings), and the stated
    tolerance 2e-6 sum|x| against the naive sequential binary32 sum."""
    n, S = oracle.num_steps(dims)
    E = 96
    x = synth.rank_matrix(dist, 11, n, E)
    exact = x.astype(np.float64).sum(0)
    sabs = np.abs(x.astype(np.float64)).sum(0)
    naive = oracle.naive_sum_f32(x).astype(np.float64)
    for variant in (LAT, BW):
        out = oracle.allreduce(dims, variant, x).astype(np.float64)
        assert np.all(np.abs(out - exact) <= 2 * S * 2.0 ** -24 * sabs * (1 + 1e-6))
        assert np.all(np.abs(out - naive) <= 2e-6 * sabs)
        o64 = oracle.allreduce(dims, variant, x.astype(np.float64))
        assert np.all(np.abs(o64 - exact) <= 2 * S * 2.0 ** -53 * sabs * (1 + 1e-6))


def test_naive_sum_is_sequential_fp32():
    x = np.random.default_rng(5).standard_normal((30, 17)).astype(np.float32)
    acc = x[0].copy()
    for u in range(1, 30):
        acc = (acc + x[u]).astype(np.float32)
    assert np.array_equal(oracle.naive_sum_f32(x), acc)


# ------------------------------------------------------------------ windows, slices, blocks

@pytest.mark.parametrize("dims", [(9,), (9, 9), (3, 3, 3)])
@pytest.mark.parametrize("variant", [LAT, BW])
def test_window_equals_columns_of_the_full_run(dims, variant):
    n = _n(dims)
    E = 1000
    x = np.random.default_rng(9).standard_normal((n, E)).astype(np.float32)
    full = oracle.allreduce(dims, variant, x)
    for e0, e1 in [(0, 1), (3, 400), (330, 340), (333, 334), (660, 1000), (999, 1000), (500, 500)]:
        part = oracle.allreduce(dims, variant, x[:, e0:e1], E=E, e0=e0)
        assert np.array_equal(part, full[:, e0:e1])


def test_block_and_slice_bounds():
    """Blocks of m/n (Sec. 4.1) and slices of 1/D (Sec. 5) with floor rounding; they tile the vector."""
    assert oracle.block_bounds(1024, 1, 9).tolist() == [(j * 1024) // 9 for j in range(10)]
    E, D, n = 2 ** 23, 3, 729
    prev_hi = 0
    for c in range(D):
        b = oracle.block_bounds(E, D, n, c)
        assert b[0] == prev_hi == (c * E) // D and np.all(np.diff(b) >= 0)
        L = ((c + 1) * E) // D - (c * E) // D
        assert set(np.diff(b).tolist()) <= {L // n, L // n + 1}
        prev_hi = b[-1]
    assert prev_hi == E
    assert np.diff(oracle.block_bounds(5, 1, 9)).tolist().count(0) == 4      # fewer elements than blocks


def test_slices_follow_different_step_orders():
    """Steps in different dimensions do not commute under rounding: the slices of a torus run must
    differ from a run that used slice 0's order everywhere."""
    dims = (9, 9)
    x = np.random.default_rng(2).standard_normal((81, 64)).astype(np.float32)
    out = oracle.allreduce(dims, LAT, x)
    swapped = oracle.allreduce(dims, LAT, np.concatenate([x[:, 32:], x[:, :32]], axis=1))
    assert not np.array_equal(out[:, :32], swapped[:, 32:])
    assert np.allclose(out[:, :32], swapped[:, 32:], rtol=1e-4, atol=1e-4)


# ------------------------------------------------------------------ cost model and optimality factors (Sec. 2.1, Tables 1 and 2)

@pytest.mark.parametrize("n", [9, 27, 81, 243])
def test_table1_factors_on_rings(n):
    """Table 1: Trivance (B) = (2, 1, 2/3 log3 n), Trivance (L) = (1, log3 n, n/2),
    Bruck (B) = (2, 1, 2 log3 n), Bruck (L) = (1, log3 n, 3n/2); 1 stands for 1 - 1/n and n/2 for (n-1)/2."""
    s = round(np.log(n) / np.log(3))
    E = 3 * n
    tb = oracle.cost_model((n,), BW, E, 4, 0.0, 1.0)
    tl = oracle.cost_model((n,), LAT, E, 4, 0.0, 1.0)
    bb = oracle.cost_model((n,), BW, E, 4, 0.0, 1.0, algo=oracle.ALGO_BRUCK)
    bl = oracle.cost_model((n,), LAT, E, 4, 0.0, 1.0, algo=oracle.ALGO_BRUCK)
    assert np.isclose(tb["lambda"], 2) and np.isclose(tb["delta"], 1 - 1 / n) and np.isclose(tb["theta"], 2 * s / 3)
    assert np.isclose(tl["lambda"], 1) and np.isclose(tl["delta"], s) and np.isclose(tl["theta"], (n - 1) / 2)
    assert np.isclose(bb["lambda"], 2) and np.isclose(bb["delta"], 1 - 1 / n) and np.isclose(bb["theta"], 2 * s)
    assert np.isclose(bl["lambda"], 1) and np.isclose(bl["delta"], s) and np.isclose(bl["theta"], 3 * (n - 1) / 2)


@pytest.mark.parametrize("q", [3, 4, 6])
def test_table1_recursive_doubling_latency_row(q):
    """Table 1: Rec.Doub. (L) = (log2 3, log2 n / 2, n); n stands for n - 1 (App. B: sum of 2^k)."""
    n = 2 ** q
    c = oracle.cost_model((n,), LAT, 4 * n, 4, 0.0, 1.0, algo=oracle.ALGO_RECDOUB)
    assert np.isclose(c["lambda"], np.log2(3)) and np.isclose(c["delta"], q / 2) and np.isclose(c["theta"], n - 1)


def test_cost_is_steps_alpha_plus_beta_times_weighted_bytes():
    """Sec. 2.1: C(m, A) = steps * alpha + sum_k beta * m_k * c_k, written out for the 9-ring:
    latency form m_k = m, c_k = 1, 3; bandwidth form m_k = m/3, m/9 (and the mirror), c_k = 1, 3."""
    m = 4 * 9 * 5
    alpha, beta = 1.5e-6, 1.0 / 100e9
    lat = oracle.cost_model((9,), LAT, 45, 4, alpha, beta)
    bw = oracle.cost_model((9,), BW, 45, 4, alpha, beta)
    assert np.isclose(lat["total"], 2 * alpha + beta * (m * 1 + m * 3))
    assert np.isclose(bw["total"], 4 * alpha + beta * 2 * (m / 3 * 1 + m / 9 * 3))
    assert lat["steps"] == 2 and bw["steps"] == 4


def test_table2_latency_form_on_tori():
    """Table 2: Trivance (L) = D/2 * n^(1/D) (exactly D (a-1)/2), Bruck (L) three times that."""
    for dims in [(9, 9), (9, 9, 9), (27, 27)]:
        D, a, n = len(dims), dims[0], int(np.prod(dims))
        t = oracle.cost_model(dims, LAT, n * D, 4, 0.0, 1.0)
        b = oracle.cost_model(dims, LAT, n * D, 4, 0.0, 1.0, algo=oracle.ALGO_BRUCK)
        assert np.isclose(t["theta"], D * (a - 1) / 2) and np.isclose(b["theta"], 3 * D * (a - 1) / 2)
