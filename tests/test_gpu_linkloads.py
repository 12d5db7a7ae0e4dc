"""GPU link-load tally (trv_link_loads) vs the oracle's hop-by-hop walk: integer tables, bit-exact."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2602_17254_b200 import binding, build

pytestmark = pytest.mark.gpu
LAT, BW = binding.LATENCY_OPTIMAL, binding.BANDWIDTH_OPTIMAL
GOLD = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available()


def _same(a, b):
    for k in ("msgs", "bytes", "max_msgs", "max_bytes"):
        assert a[k].dtype == b[k].dtype and np.array_equal(a[k], b[k]), k


@pytest.mark.parametrize("dims", [(3,), (9,), (27,), (81,), (243,), (729,), (3, 3), (9, 9), (3, 3, 3), (9, 9, 9), (3, 9),
                                  (27, 3), (3, 3, 9)])
@pytest.mark.parametrize("variant", [LAT, BW])
@pytest.mark.parametrize("count", [1024, 7, 100003])
def test_trivance_link_loads(dims, variant, count):
    got = binding.Plan(dims, variant).link_loads(count, 4)
    _same(got, oracle.link_loads(dims, variant, count, 4))


@pytest.mark.parametrize("dims", [(9,), (27,), (243,), (9, 9), (3, 9)])
@pytest.mark.parametrize("variant", [LAT, BW])
def test_bruck_link_loads(dims, variant):
    got = binding.Plan(dims, variant, binding.ALGO_BRUCK).link_loads(100003, 4)
    _same(got, oracle.link_loads(dims, variant, 100003, 4, algo=oracle.ALGO_BRUCK))


@pytest.mark.parametrize("n", [2, 8, 64, 1024])
@pytest.mark.parametrize("variant", [LAT, BW])
def test_recursive_doubling_link_loads(n, variant):
    got = binding.Plan((n,), variant, binding.ALGO_RECDOUB).link_loads(100003, 2)
    _same(got, oracle.link_loads((n,), variant, 100003, 2, algo=oracle.ALGO_RECDOUB))


def test_fig1_values_on_the_gpu():
    algo = {"trivance": binding.ALGO_TRIVANCE, "bruck": binding.ALGO_BRUCK, "recursive_doubling": binding.ALGO_RECDOUB}
    with open(os.path.join(GOLD, "fig1_max_link_congestion.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    for name, n, *want in rows:
        ll = binding.Plan((int(n),), LAT, algo[name]).link_loads(1024, 4)
        assert ll["max_msgs"].tolist() == [int(v) for v in want]


def test_config1_and_config5_tables():
    ll = binding.Plan((9,), LAT).link_loads(1024, 4)
    assert np.all(ll["msgs"][0] == 1) and np.all(ll["msgs"][1] == 3)
    assert np.all(ll["bytes"][0] == 4096) and np.all(ll["bytes"][1] == 12288)
    for count in (8192, 131072, 2097152, 8388608):
        for variant in (LAT, BW):
            tv = binding.Plan((243,), variant).link_loads(count, 4)
            br = binding.Plan((243,), variant, binding.ALGO_BRUCK).link_loads(count, 4)
            _same(tv, oracle.link_loads((243,), variant, count, 4))
            _same(br, oracle.link_loads((243,), variant, count, 4, algo=oracle.ALGO_BRUCK))
            k = [r if r < 5 else 9 - r for r in range(tv["max_msgs"].size)]
            assert tv["max_msgs"].tolist() == [3 ** v for v in k]
            assert br["max_msgs"].tolist() == [3 * 3 ** v for v in k]
    with pytest.raises(binding.TrivanceError) as e:
        binding.Plan((243,), LAT, binding.ALGO_RECDOUB)
    assert e.value.status == binding.ERR_UNDEFINED_SCHEDULE


@pytest.mark.parametrize("dims,algo", [((9,), binding.ALGO_TRIVANCE), ((243,), binding.ALGO_TRIVANCE), ((9, 9, 9), binding.ALGO_TRIVANCE),
                                       ((3, 9), binding.ALGO_TRIVANCE), ((27,), binding.ALGO_BRUCK), ((64,), binding.ALGO_RECDOUB)])
@pytest.mark.parametrize("variant", [LAT, BW])
def test_cost_model_matches_oracle(dims, algo, variant):
    """trv_cost_model (Sec. 2.1 cost, Table 1/2 factors) vs the oracle's: integers exact, doubles to rounding."""
    alpha, beta = 1.5e-6, 1.0 / 100e9
    for count in (100003, 8192):
        got = binding.Plan(dims, variant, algo).cost_model(count, 4, alpha, beta)
        want = oracle.cost_model(dims, variant, count, 4, alpha, beta, algo=algo)
        assert got.steps == want["steps"] and got.bytes_sent_per_node == want["bytes_sent_per_node"]
        assert got.tx_bytes == want["tx_bytes"]
        for name, key in [("latency_term", "latency_term"), ("tx_term", "tx_term"), ("total", "total"), ("lambda_", "lambda"),
                          ("delta", "delta"), ("theta", "theta")]:
            assert np.isclose(getattr(got, name), want[key], rtol=1e-12, atol=0), name


M = binding.ALGO_MIRRORED
NEW = [((8,), binding.ALGO_SWING), ((64,), binding.ALGO_SWING), ((1024,), binding.ALGO_SWING), ((64,), binding.ALGO_SWING | M),
       ((256,), binding.ALGO_SWING | M), ((16,), binding.ALGO_RECDOUB | M), ((512,), binding.ALGO_RECDOUB | M),
       ((27,), binding.ALGO_BRUCK | M), ((9,), binding.ALGO_BUCKET), ((10,), binding.ALGO_BUCKET | M),
       ((100,), binding.ALGO_BUCKET | M), ((2,), binding.ALGO_BUCKET | M),
       ((4, 4), binding.ALGO_BUCKET | M), ((3, 5), binding.ALGO_BUCKET), ((2, 3, 4), binding.ALGO_BUCKET | M), ((8, 8, 8), binding.ALGO_BUCKET | M)]


@pytest.mark.parametrize("dims,algo", NEW)
@pytest.mark.parametrize("variant", [LAT, BW])
def test_swing_bucket_and_mirrored_link_loads(dims, algo, variant):
    """Swing, the ring algorithm and the mirrored sub-collectives (Sec. 2.4): tally vs the oracle's walk."""
    if (algo & ~M) == binding.ALGO_BUCKET and variant == LAT:     # the ring algorithm has no latency-optimal form
        with pytest.raises(binding.TrivanceError) as e:
            binding.Plan(dims, variant, algo)
        assert e.value.status == binding.ERR_UNSUPPORTED
        return
    for count in (100003, 7):
        got = binding.Plan(dims, variant, algo).link_loads(count, 4)
        _same(got, oracle.link_loads(dims, variant, count, 4, algo=algo))
    alpha, beta = 1.5e-6, 1.0 / 100e9
    got = binding.Plan(dims, variant, algo).cost_model(100003, 4, alpha, beta)
    want = oracle.cost_model(dims, variant, 100003, 4, alpha, beta, algo=algo)
    assert got.steps == want["steps"] and got.bytes_sent_per_node == want["bytes_sent_per_node"] and got.tx_bytes == want["tx_bytes"]
    for name, key in [("total", "total"), ("lambda_", "lambda"), ("delta", "delta"), ("theta", "theta")]:
        assert np.isclose(getattr(got, name), want[key], rtol=1e-12, atol=0), name


def test_table_generator_reproduces_the_papers_entries():
    """paper_2602_17254_b200.tables: Table 1 on the ring of 27 and Table 2 on 9 x 9 and 4 x 4 x 4, from the GPU tally."""
    from paper_2602_17254_b200 import tables
    ring = {r["algorithm"]: r for r in tables.table((27,))}
    assert ring["Trivance (L)"]["steps"] == 3 and np.isclose(ring["Trivance (L)"]["lambda"], 1.0)
    assert np.isclose(ring["Trivance (L)"]["theta"], 13.0)                 # sum of 3^k: 1 + 3 + 9
    assert np.isclose(ring["Trivance (B)"]["delta"], 26 / 27) and np.isclose(ring["Bruck (L)"]["theta"], 39.0)
    assert np.isclose(ring["Bucket"]["theta"], 26 / 27) and ring["Bucket"]["steps"] == 52
    t2 = {r["algorithm"]: r for r in tables.table((9, 9))}
    assert np.isclose(t2["Trivance (L)"]["theta"], t2["Trivance (L)"]["paper_closed_form"])    # (D / 2)(a - 1) -> (D / 2) n^(1/D)
    assert np.isclose(t2["Bucket"]["theta"], 80 / 81)
    t3 = {r["algorithm"]: r for r in tables.table((4, 4, 4))}
    assert np.isclose(t3["Rec.Doub. (L)"]["theta"], 9 * 3) and np.isclose(t3["Bucket"]["theta"], 63 / 64)   # D^2 (a - 1)
