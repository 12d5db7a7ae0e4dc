"""Comparator schedules of Sec. 2.4 as link-load models: Swing, Bucket (ring), and the mirrored
sub-collectives.  Pins of the oracle against Sec. 2.4, Table 1 and App. B; the library's host-side
tables against the oracle.  No GPU needed."""
import math

import numpy as np
import pytest

import oracle
from paper_2602_17254_b200 import binding

LAT, BW = oracle.VARIANT_LATENCY, oracle.VARIANT_BANDWIDTH
M = oracle.ALGO_MIRROR


def rho(k):
    return (1 - (-2) ** (k + 1)) // 3


def test_golden_per_step_congestion():
    """tests/golden/table1_ring_comparators.txt: the per-step congestion App. B derives for each comparator."""
    import os
    algo = {"swing_latency": (oracle.ALGO_SWING, LAT), "swing_bandwidth_mirrored": (oracle.ALGO_SWING | M, BW),
            "recursive_doubling_latency": (oracle.ALGO_RECDOUB, LAT)}
    path = os.path.join(os.path.dirname(__file__), "golden", "table1_ring_comparators.txt")
    rows = [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 6
    for name, n, *want in rows:
        a, variant = algo[name]
        ll = oracle.link_loads([int(n)], variant, 64 * int(n), 4, algo=a)
        assert ll["max_msgs"][:len(want)].tolist() == [int(v) for v in want]


def test_swing_distances_and_pairs():
    """rho(k) = sum_{i<=k} (-2)^i = 1, -1, 3, -5, 11, ...; even ranks go to r + rho, odd ones to r - rho; the
    exchange is pairwise (Sec. 2.4)."""
    assert [rho(k) for k in range(6)] == [1, -1, 3, -5, 11, -21]
    for n in (2, 8, 64, 256):
        q = int(math.log2(n))
        assert oracle.step_list([n], 0, oracle.ALGO_SWING) == [(0, rho(k)) for k in range(q)]
        for k in range(q):
            pe = oracle.peers([n], k, 0, oracle.ALGO_SWING)[:, 0]
            for r in range(n):
                assert pe[r] == (r + rho(k) if r % 2 == 0 else r - rho(k)) % n
                assert pe[pe[r]] == r


@pytest.mark.parametrize("n", [8, 16, 64, 256, 1024])
def test_swing_congestion_matches_appendix_b(n):
    """App. B: latency-optimal Swing has congestion ceil(|rho(k)| / 2) in step k; with the mirrored collective
    the bandwidth-optimal one has |rho(k)| at message size m / 2^(k+2) per collective."""
    q = int(math.log2(n))
    ll = oracle.link_loads([n], LAT, 1024, 4, algo=oracle.ALGO_SWING)
    assert ll["max_msgs"].tolist() == [math.ceil(abs(rho(k)) / 2) for k in range(q)]
    E = 64 * n
    ll = oracle.link_loads([n], BW, E, 4, algo=oracle.ALGO_SWING | M)
    want = [abs(rho(k)) for k in range(q)]
    assert ll["max_msgs"].tolist() == want + want[::-1]
    m = 4 * E
    assert ll["max_bytes"].tolist() == [abs(rho(k)) * (m // 2) // 2 ** (k + 1) for k in range(q)] + \
        [abs(rho(k)) * (m // 2) // 2 ** (k + 1) for k in reversed(range(q))]
    cm = oracle.cost_model([n], BW, E, 4, 0.0, 1.0, algo=oracle.ALGO_SWING | M)
    theta = sum(abs(rho(k)) / 2 ** (k + 1) for k in range(q))
    assert np.isclose(cm["theta"], theta, rtol=1e-12)
    assert abs(theta - q / 3) < 0.45                      # Table 1: (1/3) log2 n, up to the constant the sum converges with
    assert np.isclose(cm["delta"], (n - 1) / n) and np.isclose(cm["lambda"], 2 * q / (math.log(n) / math.log(3)))


@pytest.mark.parametrize("n", [8, 64])
def test_swing_block_sets_partition(n):
    """Algorithm 1 on Swing's peers: n / 2^(k+1) blocks go out in step k and what a rank sends over all
    steps plus its own block is everything, each block once (bandwidth optimality, Sec. 2.3)."""
    q = int(math.log2(n))
    for r in (0, 1, n // 2 + 1):
        seen = np.zeros(n, int)
        seen[r] += 1
        for k in range(q):
            p = oracle.peers([n], k, 0, oracle.ALGO_SWING)[r, 0]
            s = oracle.send_set([n], p, k, 0, oracle.ALGO_SWING)
            assert s.sum() == n // 2 ** (k + 1)
            seen += s
        assert (seen == 1).all()


@pytest.mark.parametrize("n", [2, 7, 9, 32, 100])
def test_bucket_ring_matches_table_1(n):
    """The ring algorithm with both ports (Table 1, App. B): 2(n-1) steps, no two messages share a link,
    every message one block of one half: Delta = Theta = (n-1)/n -> 1, Lambda = 2(n-1)/log3 n."""
    E = 6 * n
    ll = oracle.link_loads([n], BW, E, 4, algo=oracle.ALGO_BUCKET | M)
    assert ll["msgs"].shape == (2 * (n - 1), n, 1, 2)
    assert (ll["msgs"] == 1).all() and (ll["bytes"] == 4 * 3).all()
    cm = oracle.cost_model([n], BW, E, 4, 0.0, 1.0, algo=oracle.ALGO_BUCKET | M)
    assert cm["steps"] == 2 * (n - 1)
    assert np.isclose(cm["theta"], (n - 1) / n) and np.isclose(cm["delta"], (n - 1) / n)
    assert np.isclose(cm["lambda"], 2 * (n - 1) / (math.log(n) / math.log(3)))
    one = oracle.link_loads([n], BW, E, 4, algo=oracle.ALGO_BUCKET)      # one port only: + links carry it all
    assert (one["msgs"][..., 0] == 1).all() and (one["msgs"][..., 1] == 0).all()
    with pytest.raises(oracle.OracleError):
        oracle.link_loads([n], LAT, E, 4, algo=oracle.ALGO_BUCKET)


@pytest.mark.parametrize("dims", [(3, 3), (4, 4), (8, 8), (5, 5, 5), (4, 4, 4, 4)])
def test_bucket_on_tori_matches_table_2(dims):
    """Bucket on an a^D torus with all 2D ports (Sec. 2.4, Table 2): 2D concurrent collectives on 1/(2D) of the vector
    each, every one in a different direction in every step, so no link ever carries two messages; 2 D (a - 1) steps;
    phase p of a collective moves messages of m / (2D a^(p+1)) bytes; Theta = Delta = (n - 1)/n -> Table 2's 1
    against the ideal m beta / D, Lambda = 2 D (a - 1) / log3 n (the table's 2 D n^(1/D) / log3 n counts a for a - 1)."""
    D, a = len(dims), dims[0]
    n = a ** D
    E = 2 * D * n * 3                   # every collective's slice splits into n blocks of 3 elements
    ll = oracle.link_loads(dims, BW, E, 4, algo=oracle.ALGO_BUCKET | M)
    S = D * (a - 1)
    assert ll["msgs"].shape == (2 * S, n, D, 2)
    assert (ll["msgs"] == 1).all()                              # every link, both directions, exactly one message
    per_row = [3 * 4 * n // a ** (p + 1) for p in range(D) for _ in range(a - 1)]
    assert ll["max_bytes"].tolist() == per_row + per_row[::-1]  # the AllGather takes the phases in reverse order
    assert (ll["bytes"].max(axis=(1, 2, 3)) == ll["bytes"].min(axis=(1, 2, 3))).all()      # all links alike in a row
    cm = oracle.cost_model(dims, BW, E, 4, 0.0, 1.0, algo=oracle.ALGO_BUCKET | M)
    assert cm["steps"] == 2 * S
    assert np.isclose(cm["theta"], (n - 1) / n) and np.isclose(cm["delta"], (n - 1) / n)
    assert np.isclose(cm["lambda"], 2 * S / (math.log(n) / math.log(3)))
    # one port per collective only (no mirrored sub-collectives): the + links carry everything
    one = oracle.link_loads(dims, BW, E, 4, algo=oracle.ALGO_BUCKET)
    assert (one["msgs"][..., 0] == 1).all() and (one["msgs"][..., 1] == 0).all()


def test_bucket_on_a_torus_worked_by_hand():
    """3 x 2 torus (rank = x0 + 3 x1), collective 0 (dimension 0 first): rows 0, 1 ring Reduce-Scatter along
    dimension 0 on super-blocks {j : j0 = x0 - s - 1}, row 2 along dimension 1 on the one block with j0 = x0,
    j1 = x1 - 1; then the AllGather: dimension 1 first, dimension 0 last.  Node 0 = (0, 0)."""
    E = 2 * 6 * 5
    ll = oracle.link_loads((3, 2), BW, E, 4, algo=oracle.ALGO_BUCKET)
    b = ll["bytes"]                     # [row][node][dimension][direction]
    # collective 0 uses, in row order, dimensions 0 0 1 | 1 0 0 with 2, 2, 1 | 1, 2, 2 blocks of 20 bytes per message;
    # collective 1 dimensions 1 0 0 | 0 0 1 with 3, 1, 1 | 1, 1, 3 blocks: with unequal sides they meet on a link (rows 1, 4)
    assert b[:, 0, 0, 0].tolist() == [40, 60, 20, 20, 60, 40] and b[:, 0, 1, 0].tolist() == [60, 0, 20, 20, 0, 60]
    assert ll["msgs"][:, 0, 0, 0].tolist() == [1, 2, 1, 1, 2, 1] and (ll["msgs"][..., 1] == 0).all()
    x = np.zeros((6, E), np.int32)
    for r in range(6):
        x[r] = 10 ** r
    y, ctr = oracle.allreduce_algo((3, 2), BW, x, oracle.ALGO_BUCKET, counters=True)
    assert (y == 111111).all()
    # per collective a node sends 2 x (2 blocks) + 1 block in the Reduce-Scatter: 5 of 6 blocks
    assert (ctr["sent_rs"] == 2 * 5 * 20).all() and (ctr["sent_ag"] == 2 * 5 * 20).all()


@pytest.mark.parametrize("n", [8, 64, 256])
def test_recursive_doubling_mirrored(n):
    """Both ports through a mirrored collective (Sec. 2.4): the bytes per node halve per collective
    (Delta = (n-1)/n).  On the links the two collectives overlap: the literal tally finds 2^(k+1) - 1
    half-size messages on the worst link of step k, where Table 1 / App. B count one collective's 2^k
    (the table's (1/2) log2 n) -- recorded here as it is tallied."""
    q = int(math.log2(n))
    E = 64 * n
    ll = oracle.link_loads([n], BW, E, 4, algo=oracle.ALGO_RECDOUB | M)
    want = [2 ** (k + 1) - 1 for k in range(q)]
    assert ll["max_msgs"].tolist() == want + want[::-1]
    cm = oracle.cost_model([n], BW, E, 4, 0.0, 1.0, algo=oracle.ALGO_RECDOUB | M)
    assert np.isclose(cm["delta"], (n - 1) / n)
    single = oracle.cost_model([n], BW, E, 4, 0.0, 1.0, algo=oracle.ALGO_RECDOUB)
    assert np.isclose(single["theta"], q)                 # one collective on the whole vector: 2 * q * 2^k / 2^(k+1)
    assert q / 2 < cm["theta"] < q


# ------------------------------------------------------------------ the library's host-side tables

CASES = [((8,), oracle.ALGO_SWING), ((64,), oracle.ALGO_SWING), ((64,), oracle.ALGO_SWING | M), ((16,), oracle.ALGO_RECDOUB | M),
         ((27,), oracle.ALGO_BRUCK | M), ((9,), oracle.ALGO_BUCKET), ((10,), oracle.ALGO_BUCKET | M),
         ((4, 4), oracle.ALGO_BUCKET | M), ((3, 5), oracle.ALGO_BUCKET), ((2, 3, 4), oracle.ALGO_BUCKET | M)]


@pytest.mark.parametrize("dims,algo", CASES)
@pytest.mark.parametrize("variant", [LAT, BW])
def test_plan_tables_match_oracle(dims, algo, variant):
    base = algo & ~M
    if base == oracle.ALGO_BUCKET and variant == LAT:
        with pytest.raises(binding.TrivanceError) as e:
            binding.Plan(dims, variant, algo)
        assert e.value.status == binding.ERR_UNSUPPORTED
        return
    plan = binding.Plan(dims, variant, algo)
    n = plan.n
    assert plan.nslices == len(dims) * (2 if algo & M else 1)
    E = 37 * n + 5
    sent = np.zeros(n, np.int64)
    for c in range(plan.nslices):
        for row in range(plan.rows):
            for side in (0, 1):
                sent += plan.message_bytes_side(E, 4, c, row, side)
    assert np.array_equal(sent, oracle.bytes_sent(dims, variant, E, 4, algo=algo))
    if base != oracle.ALGO_BUCKET:
        _, S = oracle.num_steps(dims, algo)
        for c in range(plan.nslices):
            steps = oracle.step_list(dims, c, algo)
            for t in range(S):
                assert plan.step(c, t) == steps[t]
                assert np.array_equal(plan.peers(c, t), oracle.peers(dims, t, c, algo))
                if variant == BW:
                    for dst in (0, 1, n - 1):
                        assert np.array_equal(plan.send_set(c, t, dst), oracle.send_set(dims, dst, t, c, algo))
    plan.destroy()


def test_mirror_flag_is_for_ring_comparators_only():
    for dims, algo in (((9,), oracle.ALGO_TRIVANCE | M), ((9, 9), oracle.ALGO_BRUCK | M)):
        with pytest.raises(binding.TrivanceError) as e:
            binding.Plan(dims, BW, algo)
        assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.TrivanceError) as e:
        binding.Plan((12,), BW, oracle.ALGO_SWING)
    assert e.value.status == binding.ERR_UNDEFINED_SCHEDULE


# ------------------------------------------------------------------ the comparators as data paths (Sec. 2.4, 3.1)

DATA_ALGOS = [(oracle.ALGO_BRUCK, [3, 9, 27]), (oracle.ALGO_RECDOUB, [2, 4, 8, 16]), (oracle.ALGO_SWING, [2, 4, 8, 16, 32]),
              (oracle.ALGO_BUCKET, [2, 3, 5, 8, 12])]


@pytest.mark.parametrize("algo,sizes", DATA_ALGOS)
@pytest.mark.parametrize("mirror", [0, oracle.ALGO_MIRROR])
def test_comparator_paths_give_the_column_sums_and_the_modelled_bytes(algo, sizes, mirror):
    """Every rank ends with the sum of all inputs (int32, wrapping); the bytes each node put on the wire are the ones
    the link-load model counts for the same schedule."""
    for n in sizes:
        for variant in (0, 1):
            if algo == oracle.ALGO_BUCKET and variant == 0:
                with pytest.raises(oracle.OracleError):
                    oracle.allreduce_algo((n,), 0, np.zeros((n, 4), np.int32), algo)
                continue
            E = 3 * n + 5
            x = np.random.default_rng(n).integers(-2 ** 31, 2 ** 31 - 1, size=(n, E), dtype=np.int64).astype(np.int32)
            y, ctr = oracle.allreduce_algo((n,), variant, x, algo | mirror, counters=True)
            assert (y == x.astype(np.int64).sum(0).astype(np.int32)[None]).all()
            assert np.array_equal(ctr["sent_rs"] + ctr["sent_ag"], oracle.bytes_sent((n,), variant, E, 4, algo | mirror))
            part = oracle.allreduce_algo((n,), variant, np.ascontiguousarray(x[:, 2:E - 3]), algo | mirror, E=E, e0=2)
            assert np.array_equal(part, y[:, 2:E - 3])          # a window gives the full run's columns


@pytest.mark.parametrize("dims", [(3, 3), (4, 4), (3, 5), (2, 3, 4), (5, 5, 5)])
@pytest.mark.parametrize("mirror", [0, oracle.ALGO_MIRROR])
def test_bucket_path_on_tori(dims, mirror):
    """Bucket dimension after dimension (Sec. 2.4): every rank ends with the column sums, the bytes on the wire are the
    modelled ones -- (n - 1)/n of a collective's slice per node and phase direction -- and a window of the vector gives
    the full run's columns."""
    n = int(np.prod(dims))
    E = 7 * n + 3
    x = np.random.default_rng(n).integers(-2 ** 31, 2 ** 31 - 1, size=(n, E), dtype=np.int64).astype(np.int32)
    y, ctr = oracle.allreduce_algo(dims, 1, x, oracle.ALGO_BUCKET | mirror, counters=True)
    assert (y == x.astype(np.int64).sum(0).astype(np.int32)[None]).all()
    assert np.array_equal(ctr["sent_rs"] + ctr["sent_ag"], oracle.bytes_sent(dims, 1, E, 4, oracle.ALGO_BUCKET | mirror))
    if E % (n * len(dims) * (2 if mirror else 1)) == 0:
        assert (ctr["sent_rs"] == 4 * E * (n - 1) // n).all()
    part = oracle.allreduce_algo(dims, 1, np.ascontiguousarray(x[:, 2:E - 3]), oracle.ALGO_BUCKET | mirror, E=E, e0=2)
    assert np.array_equal(part, y[:, 2:E - 3])
    xf = np.random.default_rng(n + 1).standard_normal((n, E)).astype(np.float32)
    yf = oracle.allreduce_algo(dims, 1, xf, oracle.ALGO_BUCKET | mirror)
    assert (yf == yf[0][None]).all()                            # one reduction order per block: every rank gets the same bits
    assert np.abs(yf[0].astype(np.float64) - xf.astype(np.float64).sum(0)).max() <= 2e-6 * np.abs(xf).sum(0).max()


@pytest.mark.parametrize("dims", [(9,), (27,), (3, 3), (9, 9), (3, 9), (3, 3, 3)])
@pytest.mark.parametrize("variant", [0, 1])
def test_generic_path_with_trivance_peers_is_the_trivance_path(dims, variant):
    """The message-by-message executor of the comparators, given Trivance's own peers, reproduces the dedicated
    Trivance oracle bit for bit: its association rule (m1 + own) + m0 is (from_left + own) + from_right there."""
    n = int(np.prod(dims))
    x = np.random.default_rng(n).standard_normal((n, 5 * n + 3)).astype(np.float32)
    a = oracle.allreduce_algo(dims, variant, x, oracle.ALGO_TRIVANCE)
    b = oracle.allreduce(dims, variant, x)
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


def _swing_peer(p, k, n):
    rho = sum((-2) ** i for i in range(k + 1))
    return (p + rho) % n if p % 2 == 0 else (p - rho) % n


@pytest.mark.parametrize("algo,n", [(oracle.ALGO_RECDOUB, 8), (oracle.ALGO_RECDOUB, 32), (oracle.ALGO_SWING, 8), (oracle.ALGO_SWING, 32),
                                    (oracle.ALGO_BRUCK, 9), (oracle.ALGO_BRUCK, 27)])
def test_latency_forms_against_their_step_formulas(algo, n):
    """Sec. 2.4 / 3.1: Recursive Doubling v[p] += v[p XOR 2^k]; Swing v[p] += v[pi(p, k)]; Bruck with joint reductions
    v[p] = (v[p - 2 3^k] + v[p]) + v[p - 3^k] (the reading of the association order), step by step in binary32."""
    x = (np.random.default_rng(n).standard_normal((n, 64)) * 100).astype(np.float32)
    v = x.copy()
    if algo == oracle.ALGO_BRUCK:
        d = 1
        while d < n:
            v = (np.roll(v, 2 * d, axis=0) + v) + np.roll(v, d, axis=0)
            d *= 3
    else:
        k = 0
        while (1 << k) < n:
            perm = [p ^ (1 << k) for p in range(n)] if algo == oracle.ALGO_RECDOUB else [_swing_peer(p, k, n) for p in range(n)]
            v = v + v[perm]
            k += 1
    got = oracle.allreduce_algo((n,), 0, x, algo)
    assert np.array_equal(got.view(np.uint32), v.view(np.uint32))
    exact = x.astype(np.float64).sum(0)
    assert (np.abs(got.astype(np.float64) - exact[None]) <= 2e-6 * np.abs(x.astype(np.float64)).sum(0)[None]).all()


@pytest.mark.parametrize("algo,n", [(oracle.ALGO_RECDOUB, 16), (oracle.ALGO_SWING, 16), (oracle.ALGO_BRUCK, 27), (oracle.ALGO_BUCKET, 7)])
def test_bandwidth_forms_all_rows_equal_and_blocks_are_the_owners_latency_rows(algo, n):
    E = 4 * n + 3
    rng = np.random.default_rng(n)
    x = (rng.standard_normal((n, E)) * 10.0 ** rng.integers(-3, 4, size=(n, E))).astype(np.float32)
    bw = oracle.allreduce_algo((n,), 1, x, algo)
    assert all(np.array_equal(bw[0].view(np.uint32), bw[r].view(np.uint32)) for r in range(n))
    if algo != oracle.ALGO_BUCKET:      # Reduce-Scatter is the latency pattern restricted to the blocks on their way to the owner
        lat = oracle.allreduce_algo((n,), 0, x, algo)
        bb = oracle.block_bounds(E, 1, n)
        for j in range(n):
            assert np.array_equal(bw[j, bb[j]:bb[j + 1]].view(np.uint32), lat[j, bb[j]:bb[j + 1]].view(np.uint32))
    xi = rng.integers(-100, 100, size=(n, E)).astype(np.float32)      # small integers: exact, equals the int path
    assert np.array_equal(oracle.allreduce_algo((n,), 1, xi, algo), oracle.allreduce_algo((n,), 1, xi.astype(np.int32), algo).astype(np.float32))


# ------------------------------------------------------------------ Table 2 / App. B: Recursive Doubling and Swing on tori

def _rho_abs(k):
    return abs(sum((-2) ** i for i in range(k + 1)))


POW2_TORI = [(4, 4), (8, 8), (16, 16), (4, 4, 4), (8, 8, 8), (4, 4, 4, 4)]


@pytest.mark.parametrize("dims", POW2_TORI)
def test_table2_swing_and_recursive_doubling_bandwidth_forms_on_tori(dims):
    """App. B: Theta of the bandwidth-optimal forms on a D-dimensional torus, relative to m beta / D, is
    sum_d sum_k c_k / 2^(1 + d + D k) with c_k = |rho(k)| (Swing, with its mirrored sub-collectives) resp. 2^k
    (Recursive Doubling).  The tally of Swing's 2 D superposed collectives gives that number exactly.  For Recursive
    Doubling the appendix counts ONE collective's congestion with the half-size messages of the mirrored set-up (as on
    rings): that is half the tally of the D unmirrored collectives; the mirrored tally lies between the two."""
    D, a = len(dims), dims[0]
    q = a.bit_length() - 1
    n = a ** D
    E = n * 2 * D * 4
    swing = sum(_rho_abs(k) / 2 ** (1 + d + D * k) for d in range(D) for k in range(q))
    rd = sum(2 ** k / 2 ** (1 + d + D * k) for d in range(D) for k in range(q))
    c = oracle.cost_model(dims, 1, E, 4, 0.0, 1.0, oracle.ALGO_SWING | oracle.ALGO_MIRROR)
    assert c["theta"] == pytest.approx(swing, rel=1e-12) and c["steps"] == 2 * D * q and c["delta"] == pytest.approx(1 - 1 / n)
    c = oracle.cost_model(dims, 1, E, 4, 0.0, 1.0, oracle.ALGO_RECDOUB)
    assert c["theta"] == pytest.approx(2 * rd, rel=1e-12)
    m = oracle.cost_model(dims, 1, E, 4, 0.0, 1.0, oracle.ALGO_RECDOUB | oracle.ALGO_MIRROR)
    assert rd <= m["theta"] <= 2 * rd and m["delta"] == pytest.approx(1 - 1 / n)


@pytest.mark.parametrize("dims", POW2_TORI)
def test_table2_latency_forms_use_a_single_collective(dims):
    """App. B: the latency-optimal Recursive Doubling and Swing run ONE collective on the whole vector ("only a single port
    per node"); per dimension the congestions 2^k resp. ceil(|rho(k)| / 2) add up, times D dimensions, times D again
    relative to m beta / D: D^2 (a - 1) and D^2 sum_k ceil(|rho(k)| / 2) (Table 2: D^2 n^(1/D) and D^2 / 3 n^(1/D))."""
    D, a = len(dims), dims[0]
    q = a.bit_length() - 1
    E = 1024
    c = oracle.cost_model(dims, 0, E, 4, 0.0, 1.0, oracle.ALGO_RECDOUB | oracle.ALGO_SINGLE)
    assert c["steps"] == D * q and c["theta"] == pytest.approx(D * D * (a - 1))
    c = oracle.cost_model(dims, 0, E, 4, 0.0, 1.0, oracle.ALGO_SWING | oracle.ALGO_SINGLE)
    assert c["theta"] == pytest.approx(D * D * sum(-(-_rho_abs(k) // 2) for k in range(q)))
    x = np.random.default_rng(a).integers(-1000, 1000, size=(a ** D, 40), dtype=np.int32)
    for algo in (oracle.ALGO_RECDOUB, oracle.ALGO_SWING):
        assert (oracle.allreduce_algo(dims, 0, x, algo | oracle.ALGO_SINGLE) == x.sum(0, dtype=np.int32)[None]).all()


def test_appendix_b_sums_tend_to_table2_closed_forms():
    """The sums of App. B converge to Table 2's closed forms: Swing (B) 2^D (2^D - 1) / ((2^D - 2)(2^D + 1)) = 1.2, 1.04, 1.01;
    Recursive Doubling (B) (2^D - 1) / (2^D - 2) = 1.5, 1.17, 1.07 for D = 2, 3, 4 (arithmetic on the paper's formulas only)."""
    for D, sw, rd in ((2, 1.2, 1.5), (3, 1.04, 1.17), (4, 1.01, 1.07)):
        q = 40
        s = sum(_rho_abs(k) / 2 ** (1 + d + D * k) for d in range(D) for k in range(q))
        r = sum(2 ** k / 2 ** (1 + d + D * k) for d in range(D) for k in range(q))
        assert s == pytest.approx(2 ** D * (2 ** D - 1) / ((2 ** D - 2) * (2 ** D + 1)), rel=1e-9) and round(s, 2) == sw
        assert r == pytest.approx((2 ** D - 1) / (2 ** D - 2), rel=1e-9) and round(r, 2) == rd


@pytest.mark.parametrize("algo", [oracle.ALGO_RECDOUB, oracle.ALGO_SWING])
@pytest.mark.parametrize("dims", [(4, 4), (2, 8), (4, 4, 4)])
def test_torus_comparator_paths_give_the_column_sums(algo, dims):
    n = int(np.prod(dims))
    for variant in (0, 1):
        for flag in (0, oracle.ALGO_MIRROR):
            E = 5 * n + 3
            x = np.random.default_rng(n).integers(-2 ** 31, 2 ** 31 - 1, size=(n, E), dtype=np.int64).astype(np.int32)
            y, ctr = oracle.allreduce_algo(dims, variant, x, algo | flag, counters=True)
            assert (y == x.astype(np.int64).sum(0).astype(np.int32)[None]).all()
            assert np.array_equal(ctr["sent_rs"] + ctr["sent_ag"], oracle.bytes_sent(dims, variant, E, 4, algo | flag))
