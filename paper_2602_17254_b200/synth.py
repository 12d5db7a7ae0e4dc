"""Seeded synthetic inputs for the Trivance AllReduce workloads.

This module only draws random numbers and names the workload shapes.  It holds
none of the method's arithmetic, so both the CUDA tests and the CPU oracle's
tests can use it without sharing any of the method's code.

The paper evaluates AllReduce sizes of 32 B - 128 MiB per node on rings and
tori (Sec. 6) and uses no dataset: payload values never matter to its network
simulator.  The vectors below stand in for those sizes.

Recipe: rank r's vector is drawn by ``numpy.random.Generator(PCG64(SeedSequence(
[seed, r])))`` -- one independent stream per rank, so any rank's vector (or a
prefix of it) can be regenerated on its own:
  * ``int32``  : integers uniform in [-1000, 1000]
  * ``normal`` : float32 standard normal
  * ``uniform``: float32 uniform in [-1, 1)
"""
from dataclasses import dataclass
from typing import Tuple

import numpy as np

LATENCY, BANDWIDTH = 0, 1


@dataclass(frozen=True)
class Workload:
    name: str
    dims: Tuple[int, ...]
    variant: int            # LATENCY or BANDWIDTH
    count: int              # elements per rank
    dist: str               # "int32", "normal", "uniform"
    seed: int

    @property
    def n(self):
        n = 1
        for a in self.dims:
            n *= a
        return n

    @property
    def dtype(self):
        return np.int32 if self.dist == "int32" else np.float32

    @property
    def bytes_per_rank(self):
        return 4 * self.count


KiB, MiB = 1024, 1024 * 1024

# The five benchmark configurations (per-rank sizes in bytes / 4 = elements).
CONFIGS = {
    "ring9_lat_int32": Workload("ring9_lat_int32", (9,), LATENCY, 1024, "int32", 0),
    "ring27_lat_2MiB": Workload("ring27_lat_2MiB", (27,), LATENCY, 2 * MiB // 4, "normal", 1),
    "ring81_bw_8MiB": Workload("ring81_bw_8MiB", (81,), BANDWIDTH, 8 * MiB // 4, "normal", 2),
    "torus9x9x9_lat_32MiB": Workload("torus9x9x9_lat_32MiB", (9, 9, 9), LATENCY, 32 * MiB // 4, "uniform", 3),
    "torus9x9x9_bw_32MiB": Workload("torus9x9x9_bw_32MiB", (9, 9, 9), BANDWIDTH, 32 * MiB // 4, "uniform", 3),
}
for _v, _vn in ((LATENCY, "lat"), (BANDWIDTH, "bw")):
    for _sz, _sn in ((32 * KiB, "32KiB"), (512 * KiB, "512KiB"), (8 * MiB, "8MiB"), (32 * MiB, "32MiB")):
        _name = "ring243_%s_%s" % (_vn, _sn)
        CONFIGS[_name] = Workload(_name, (243,), _v, _sz // 4, "normal", 4)


def rank_vector(dist, seed, r, count, start=0):
    """Elements [start, start+count) of rank r's vector."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(seed), int(r)])))
    total = start + count
    if dist == "int32":
        v = rng.integers(-1000, 1001, size=total, dtype=np.int32)
    elif dist == "normal":
        v = rng.standard_normal(size=total, dtype=np.float32)
    elif dist == "uniform":
        v = rng.random(size=total, dtype=np.float32) * np.float32(2.0) - np.float32(1.0)
    else:
        raise ValueError("unknown distribution %r" % (dist,))
    return v[start:]


def rank_matrix(dist, seed, n, count):
    """[n][count] array: all ranks' vectors."""
    out = np.empty((n, count), np.int32 if dist == "int32" else np.float32)
    for r in range(n):
        out[r] = rank_vector(dist, seed, r, count)
    return out


def workload_inputs(w: Workload, count=None):
    """All ranks' vectors of a workload (optionally only the first `count` elements)."""
    return rank_matrix(w.dist, w.seed, w.n, w.count if count is None else count)
# Rings whose size is no power of three (Sec. 4.4; 32 is the paper's worked example), bandwidth form.
for _n in (32, 100):
    _name = "ring%d_bw_8MiB" % _n
    CONFIGS[_name] = Workload(_name, (_n,), BANDWIDTH, 8 * MiB // 4, "normal", 5)
# Tori with sides that are no powers of three (Sec. 4.4 per dimension; 32 x 32, 8 x 64 and 16 x 16 x 16 are tori the
# paper evaluates -- 16 x 16 x 4 stands in for the last, which has more ranks than the engine takes), bandwidth form.
for _dims in ((32, 32), (8, 64), (16, 16, 4)):
    _name = "torus%s_bw_8MiB" % "x".join(map(str, _dims))
    CONFIGS[_name] = Workload(_name, _dims, BANDWIDTH, 8 * MiB // 4, "normal", 6)
# The other 729-rank shapes in the latency form (27 x 27 is a torus the paper evaluates), 8 MiB per rank.
for _dims in ((27, 27), (9, 81), (729,)):
    _name = ("torus%s_lat_8MiB" % "x".join(map(str, _dims))) if len(_dims) > 1 else "ring729_lat_8MiB"
    CONFIGS[_name] = Workload(_name, _dims, LATENCY, 8 * MiB // 4, "normal", 7)
