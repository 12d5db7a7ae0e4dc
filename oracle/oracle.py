"""numpy front end of the plain-C Trivance oracle (``trivance_oracle.c``).

TEST INFRASTRUCTURE ONLY: see the header of the C file.  This module compiles
the C file with gcc on first use (``-O2 -ffp-contract=off -fno-fast-math``) and
calls it through ctypes.  Nothing here knows about the CUDA library.
"""
import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "trivance_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lock = threading.Lock()
_lib = None

ALGO_TRIVANCE, ALGO_BRUCK, ALGO_RECDOUB, ALGO_SWING, ALGO_BUCKET = 0, 1, 2, 3, 4
ALGO_MIRROR = 16     # flag: add the mirrored sub-collective on the other half of the vector (comparators)
ALGO_SINGLE = 32     # flag: Recursive Doubling / Swing on a torus as ONE collective walking through the dimensions
VARIANT_LATENCY, VARIANT_BANDWIDTH = 0, 1
_DTYPES = {np.dtype(np.int32): 0, np.dtype(np.uint32): 0, np.dtype(np.float32): 1, np.dtype(np.float64): 2}
_ERR = {1: "bad argument", 2: "schedule undefined for these dimensions", 3: "out of memory", 4: "internal check failed"}


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__("oracle: " + _ERR.get(code, "error %d" % code))
        self.code = code


def build(force=False):
    """Compile the oracle's C file into ``liboracle.so`` next to it."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".%d.tmp" % os.getpid()
            subprocess.check_call(["gcc", "-O2", "-std=c99", "-ffp-contract=off", "-fno-fast-math", "-fPIC",
                                   "-shared", "-o", tmp, _SRC])
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        with _lock:
            if _lib is None:
                _lib = ctypes.CDLL(_LIB)
    return _lib


def _check(rc):
    if rc != 0:
        raise OracleError(rc)


def _dims(dims):
    a = np.ascontiguousarray(np.asarray(dims, dtype=np.int32).reshape(-1))
    return a, a.ctypes.data_as(ctypes.c_void_p), ctypes.c_int(a.size)


def _general_ring(dims, algo=ALGO_TRIVANCE):
    """n if dims is a ring whose size is no power of three (Trivance, Sec. 4.4), else 0."""
    a = np.atleast_1d(np.asarray(dims)).reshape(-1)
    if algo != ALGO_TRIVANCE or a.size != 1 or a[0] < 2:
        return 0
    n = int(a[0])
    while n % 3 == 0:
        n //= 3
    return int(a[0]) if n != 1 else 0


def _general_torus(dims, algo=ALGO_TRIVANCE):
    """True if dims is a torus of two or more dimensions with a side that is no power of three (Sec. 4.4 + Sec. 5)."""
    a = np.atleast_1d(np.asarray(dims)).reshape(-1)
    if algo != ALGO_TRIVANCE or a.size < 2:
        return False

    def pow3(v):
        v = int(v)
        while v > 1 and v % 3 == 0:
            v //= 3
        return v == 1 and int(v) >= 1

    return any(int(v) < 3 or not pow3(v) for v in a)


def num_steps(dims, algo=ALGO_TRIVANCE):
    """(n, steps per phase) of the schedule on a torus with these dimensions."""
    _, p, nd = _dims(dims)
    n, s = ctypes.c_int(), ctypes.c_int()
    _check(_load().orc_num_steps(p, nd, ctypes.c_int(algo), ctypes.byref(n), ctypes.byref(s)))
    return n.value, s.value


def step_list(dims, c=0, algo=ALGO_TRIVANCE):
    """[(dim, dist), ...] of collective (slice) c."""
    _, p, nd = _dims(dims)
    _, s = num_steps(dims, algo)
    d = np.zeros(s, np.int32)
    x = np.zeros(s, np.int32)
    _check(_load().orc_step_list(p, nd, ctypes.c_int(algo), ctypes.c_int(c), d.ctypes.data_as(ctypes.c_void_p),
                                 x.ctypes.data_as(ctypes.c_void_p)))
    return [(int(a), int(b)) for a, b in zip(d, x)]


def peers(dims, step, c=0, algo=ALGO_TRIVANCE):
    """[n][2] array: the peers each rank sends to in that step (Trivance: left, right)."""
    _, p, nd = _dims(dims)
    n, _ = num_steps(dims, algo)
    out = np.zeros((n, 2), np.int32)
    _check(_load().orc_peers(p, nd, ctypes.c_int(algo), ctypes.c_int(c), ctypes.c_int(step),
                             out.ctypes.data_as(ctypes.c_void_p)))
    return out


def block_propagation(dims, r, step, c=0, algo=ALGO_TRIVANCE):
    """Algorithm 1: boolean mask of the ranks reachable from r in steps step..S-1."""
    _, p, nd = _dims(dims)
    n, _ = num_steps(dims, algo)
    out = np.zeros(n, np.uint8)
    _check(_load().orc_block_propagation(p, nd, ctypes.c_int(algo), ctypes.c_int(c), ctypes.c_int(r),
                                         ctypes.c_int(step), out.ctypes.data_as(ctypes.c_void_p)))
    return out.astype(bool)


def send_set(dims, p_dst, k, c=0, algo=ALGO_TRIVANCE):
    """Boolean mask of the blocks sent to peer p_dst in Reduce-Scatter step k."""
    _, p, nd = _dims(dims)
    n, _ = num_steps(dims, algo)
    out = np.zeros(n, np.uint8)
    _check(_load().orc_send_set(p, nd, ctypes.c_int(algo), ctypes.c_int(c), ctypes.c_int(p_dst), ctypes.c_int(k),
                                out.ctypes.data_as(ctypes.c_void_p)))
    return out.astype(bool)


def block_bounds(E, D, n, c=0):
    """n+1 global element indices: where the blocks of slice c start."""
    out = np.zeros(n + 1, np.int64)
    _check(_load().orc_block_bounds(ctypes.c_int64(E), ctypes.c_int(D), ctypes.c_int(n), ctypes.c_int(c),
                                    out.ctypes.data_as(ctypes.c_void_p)))
    return out


def naive_sum_f32(x):
    """Sequential binary32 sum over ranks 0..n-1 of an [n][w] float32 array."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape[1], np.float32)
    _load().orc_naive_sum_f32(ctypes.c_int(x.shape[0]), ctypes.c_int64(x.shape[1]),
                              x.ctypes.data_as(ctypes.c_void_p), out.ctypes.data_as(ctypes.c_void_p))
    return out


def allreduce(dims, variant, x, E=None, e0=0, max_steps=-1, counters=False):
    """Trivance AllReduce of x ([n][w], int32 / float32 / float64).

    x holds the window [e0, e0+w) of per-rank vectors of E elements (default:
    the whole vector).  Returns the [n][w] result, or (result, counters) with
    per-rank byte counters ``sent_rs``, ``sent_ag``, ``reduced``.
    """
    if _general_ring(dims):
        if variant != VARIANT_BANDWIDTH or max_steps >= 0:
            raise OracleError(2)
        return gen_allreduce(x, E=E, e0=e0, counters=counters)
    if _general_torus(dims):
        if variant != VARIANT_BANDWIDTH or max_steps >= 0:
            raise OracleError(2)
        return gent_allreduce(dims, x, E=E, e0=e0, counters=counters)
    x = np.ascontiguousarray(x)
    if x.dtype not in _DTYPES or x.ndim != 2:
        raise TypeError("x must be a 2-D int32, float32 or float64 array")
    n, w = x.shape
    nn, _ = num_steps(dims)
    if n != nn:
        raise ValueError("x has %d rows, the topology has %d ranks" % (n, nn))
    if E is None:
        E = w
    out = np.empty_like(x)
    _, p, nd = _dims(dims)
    ctr = [np.zeros(n, np.int64) for _ in range(3)] if counters else [None] * 3
    ptr = [c.ctypes.data_as(ctypes.c_void_p) if c is not None else None for c in ctr]
    _check(_load().orc_allreduce(p, nd, ctypes.c_int(variant), ctypes.c_int(_DTYPES[x.dtype]), ctypes.c_int64(E),
                                 ctypes.c_int64(e0), ctypes.c_int64(e0 + w), x.ctypes.data_as(ctypes.c_void_p),
                                 out.ctypes.data_as(ctypes.c_void_p), ctypes.c_int(max_steps), *ptr))
    if counters:
        return out, {"sent_rs": ctr[0], "sent_ag": ctr[1], "reduced": ctr[2]}
    return out


def allreduce_algo(dims, variant, x, algo, E=None, e0=0, counters=False):
    """AllReduce of x by a comparator schedule (Bruck, Recursive Doubling, Swing, Bucket; ``| ALGO_MIRROR`` adds the
    mirrored sub-collective on the other half of the vector), executed message by message; as ``allreduce``."""
    x = np.ascontiguousarray(x)
    if x.dtype not in _DTYPES or x.ndim != 2:
        raise TypeError("x must be a 2-D int32, float32 or float64 array")
    n, w = x.shape
    if E is None:
        E = w
    out = np.empty_like(x)
    _, p, nd = _dims(dims)
    ctr = [np.zeros(n, np.int64) for _ in range(3)] if counters else [None] * 3
    ptr = [c.ctypes.data_as(ctypes.c_void_p) if c is not None else None for c in ctr]
    _check(_load().orc_allreduce_algo(p, nd, ctypes.c_int(variant), ctypes.c_int(algo), ctypes.c_int(_DTYPES[x.dtype]),
                                      ctypes.c_int64(E), ctypes.c_int64(e0), ctypes.c_int64(e0 + w),
                                      x.ctypes.data_as(ctypes.c_void_p), out.ctypes.data_as(ctypes.c_void_p), *ptr))
    if counters:
        return out, {"sent_rs": ctr[0], "sent_ag": ctr[1], "reduced": ctr[2]}
    return out


def link_loads(dims, variant, E, elem_size=4, algo=ALGO_TRIVANCE):
    """Per-step link loads: dict with msgs/bytes [T][n][D][2] and max_msgs/max_bytes [T]."""
    if _general_ring(dims, algo):
        if variant != VARIANT_BANDWIDTH:
            raise OracleError(2)
        return gen_link_loads(_general_ring(dims, algo), E, elem_size)
    if _general_torus(dims, algo):
        if variant != VARIANT_BANDWIDTH:
            raise OracleError(2)
        return gent_link_loads(dims, E, elem_size)
    a, p, nd = _dims(dims)
    n, s = num_steps(dims, algo)
    T = 2 * s if variant == VARIANT_BANDWIDTH else s
    D = a.size
    msgs = np.zeros((T, n, D, 2), np.int32)
    byts = np.zeros((T, n, D, 2), np.int64)
    mm = np.zeros(T, np.int32)
    mb = np.zeros(T, np.int64)
    _check(_load().orc_link_loads(p, nd, ctypes.c_int(variant), ctypes.c_int(algo), ctypes.c_int64(E),
                                  ctypes.c_int64(elem_size), msgs.ctypes.data_as(ctypes.c_void_p),
                                  byts.ctypes.data_as(ctypes.c_void_p), mm.ctypes.data_as(ctypes.c_void_p),
                                  mb.ctypes.data_as(ctypes.c_void_p)))
    return {"msgs": msgs, "bytes": byts, "max_msgs": mm, "max_bytes": mb}


def bytes_sent(dims, variant, E, elem_size=4, algo=ALGO_TRIVANCE):
    """[n] int64: bytes every node sends over the whole AllReduce."""
    if _general_ring(dims, algo):
        if variant != VARIANT_BANDWIDTH:
            raise OracleError(2)
        return gen_link_loads(_general_ring(dims, algo), E, elem_size)["sent"]
    if _general_torus(dims, algo):
        if variant != VARIANT_BANDWIDTH:
            raise OracleError(2)
        return gent_link_loads(dims, E, elem_size)["sent"]
    _, p, nd = _dims(dims)
    n, _ = num_steps(dims, algo)
    out = np.zeros(n, np.int64)
    _check(_load().orc_bytes_sent(p, nd, ctypes.c_int(variant), ctypes.c_int(algo), ctypes.c_int64(E),
                                  ctypes.c_int64(elem_size), out.ctypes.data_as(ctypes.c_void_p)))
    return out


def cost_model(dims, variant, E, elem_size, alpha, beta, algo=ALGO_TRIVANCE):
    """Sec. 2.1: C = steps * alpha + sum_k beta * m_k * c_k, with m_k * c_k = bytes on the most loaded
    link of step k; plus the optimality factors of Tables 1 and 2 (lambda, delta, theta)."""
    ll = link_loads(dims, variant, E, elem_size, algo)
    n = _general_ring(dims, algo) or (gent_num_steps(dims)[0] if _general_torus(dims, algo) else num_steps(dims, algo)[0])
    T = ll["max_bytes"].size
    tx = int(ll["max_bytes"].sum())
    sent = int(bytes_sent(dims, variant, E, elem_size, algo).max())
    m = float(E) * float(elem_size)
    D = len(np.atleast_1d(dims))
    return {"steps": T, "bytes_sent_per_node": sent, "tx_bytes": tx, "latency_term": T * alpha, "tx_term": beta * tx,
            "total": T * alpha + beta * tx, "lambda": T / (np.log(n) / np.log(3.0)), "delta": sent / (2.0 * m),
            "theta": tx / (m / D)}


# ------------------------------------------------------------------ rings of any size (Sec. 4.4)

def gen_num_steps(n):
    """(S, [dist_0 .. dist_{S-1}]) of the ring of n nodes: regular distances, then the final one."""
    s = ctypes.c_int()
    d = np.zeros(32, np.int32)
    _check(_load().orc_gen_num_steps(ctypes.c_int(n), ctypes.byref(s), d.ctypes.data_as(ctypes.c_void_p)))
    return s.value, [int(v) for v in d[:s.value]]


def gen_tree(n):
    """(par, stp), both [n][n]: par[b][v] = node v gets block b from (-1 for v = b), stp[b][v] = in which step."""
    par = np.zeros((n, n), np.int32)
    stp = np.zeros((n, n), np.int32)
    _check(_load().orc_gen_tree(ctypes.c_int(n), par.ctypes.data_as(ctypes.c_void_p), stp.ctypes.data_as(ctypes.c_void_p)))
    return par, stp


def gen_allreduce(x, E=None, e0=0, counters=False):
    """Bandwidth-optimal Trivance AllReduce on a ring of x.shape[0] nodes (any size >= 2); as ``allreduce``."""
    x = np.ascontiguousarray(x)
    if x.dtype not in _DTYPES or x.ndim != 2:
        raise TypeError("x must be a 2-D int32, float32 or float64 array")
    n, w = x.shape
    if E is None:
        E = w
    out = np.empty_like(x)
    ctr = [np.zeros(n, np.int64) for _ in range(3)] if counters else [None] * 3
    ptr = [c.ctypes.data_as(ctypes.c_void_p) if c is not None else None for c in ctr]
    _check(_load().orc_gen_allreduce(ctypes.c_int(n), ctypes.c_int(_DTYPES[x.dtype]), ctypes.c_int64(E), ctypes.c_int64(e0),
                                     ctypes.c_int64(e0 + w), x.ctypes.data_as(ctypes.c_void_p),
                                     out.ctypes.data_as(ctypes.c_void_p), *ptr))
    if counters:
        return out, {"sent_rs": ctr[0], "sent_ag": ctr[1], "reduced": ctr[2]}
    return out


def gen_link_loads(n, E, elem_size=4):
    """Link loads of that schedule: msgs/bytes [2S][n][1][2], max_msgs/max_bytes [2S], sent [n]."""
    S, _ = gen_num_steps(n)
    T = 2 * S
    msgs = np.zeros((T, n, 1, 2), np.int32)
    byts = np.zeros((T, n, 1, 2), np.int64)
    mm = np.zeros(T, np.int32)
    mb = np.zeros(T, np.int64)
    sent = np.zeros(n, np.int64)
    _check(_load().orc_gen_link_loads(ctypes.c_int(n), ctypes.c_int64(E), ctypes.c_int64(elem_size),
                                      msgs.ctypes.data_as(ctypes.c_void_p), byts.ctypes.data_as(ctypes.c_void_p),
                                      mm.ctypes.data_as(ctypes.c_void_p), mb.ctypes.data_as(ctypes.c_void_p),
                                      sent.ctypes.data_as(ctypes.c_void_p)))
    return {"msgs": msgs, "bytes": byts, "max_msgs": mm, "max_bytes": mb, "sent": sent}


# ------------------------------------------------------------------ tori with sides of any size (Sec. 4.4 + Sec. 5)

def gent_num_steps(dims):
    """(n, S): ranks and steps per phase (sum over dimensions of ceil(log3 side))."""
    _, p, nd = _dims(dims)
    n, s = ctypes.c_int(), ctypes.c_int()
    _check(_load().orc_gent_num_steps(p, nd, ctypes.byref(n), ctypes.byref(s)))
    return n.value, s.value


def gent_step_list(dims, c=0):
    """[(dim, dist), ...] of collective c: round-robin over the dimensions from c, each dimension's ring distances in order."""
    _, p, nd = _dims(dims)
    _, S = gent_num_steps(dims)
    d = np.zeros(S, np.int32)
    x = np.zeros(S, np.int32)
    _check(_load().orc_gent_step_list(p, nd, ctypes.c_int(c), d.ctypes.data_as(ctypes.c_void_p), x.ctypes.data_as(ctypes.c_void_p)))
    return [(int(a), int(b)) for a, b in zip(d, x)]


def gent_tree(dims, c=0):
    """(par, stp), both [n][n], of collective c: par[b][v] = node v gets block b from, stp[b][v] = in which of its steps."""
    _, p, nd = _dims(dims)
    n, _ = gent_num_steps(dims)
    par = np.zeros((n, n), np.int32)
    stp = np.zeros((n, n), np.int32)
    _check(_load().orc_gent_tree(p, nd, ctypes.c_int(c), par.ctypes.data_as(ctypes.c_void_p), stp.ctypes.data_as(ctypes.c_void_p)))
    return par, stp


def gent_allreduce(dims, x, E=None, e0=0, counters=False):
    """Bandwidth-optimal Trivance AllReduce on a torus with sides of any size >= 2; as ``allreduce``."""
    x = np.ascontiguousarray(x)
    if x.dtype not in _DTYPES or x.ndim != 2:
        raise TypeError("x must be a 2-D int32, float32 or float64 array")
    n, w = x.shape
    nn, _ = gent_num_steps(dims)
    if n != nn:
        raise ValueError("x has %d rows, the topology has %d ranks" % (n, nn))
    if E is None:
        E = w
    out = np.empty_like(x)
    _, p, nd = _dims(dims)
    ctr = [np.zeros(n, np.int64) for _ in range(3)] if counters else [None] * 3
    ptr = [c.ctypes.data_as(ctypes.c_void_p) if c is not None else None for c in ctr]
    _check(_load().orc_gent_allreduce(p, nd, ctypes.c_int(_DTYPES[x.dtype]), ctypes.c_int64(E), ctypes.c_int64(e0),
                                      ctypes.c_int64(e0 + w), x.ctypes.data_as(ctypes.c_void_p),
                                      out.ctypes.data_as(ctypes.c_void_p), *ptr))
    if counters:
        return out, {"sent_rs": ctr[0], "sent_ag": ctr[1], "reduced": ctr[2]}
    return out


def gent_link_loads(dims, E, elem_size=4):
    """Link loads of that schedule: msgs/bytes [2S][n][D][2], max_msgs/max_bytes [2S], sent [n]."""
    a, p, nd = _dims(dims)
    n, S = gent_num_steps(dims)
    T, D = 2 * S, a.size
    msgs = np.zeros((T, n, D, 2), np.int32)
    byts = np.zeros((T, n, D, 2), np.int64)
    mm = np.zeros(T, np.int32)
    mb = np.zeros(T, np.int64)
    sent = np.zeros(n, np.int64)
    _check(_load().orc_gent_link_loads(p, nd, ctypes.c_int64(E), ctypes.c_int64(elem_size),
                                       msgs.ctypes.data_as(ctypes.c_void_p), byts.ctypes.data_as(ctypes.c_void_p),
                                       mm.ctypes.data_as(ctypes.c_void_p), mb.ctypes.data_as(ctypes.c_void_p),
                                       sent.ctypes.data_as(ctypes.c_void_p)))
    return {"msgs": msgs, "bytes": byts, "max_msgs": mm, "max_bytes": mb, "sent": sent}
