"""Regenerates the optimality factors of Table 1 (rings) and Table 2 (tori) from tallied link loads.

``python -m paper_2602_17254_b200.tables [--ring N ...] [--torus A D ...]`` prints, for every algorithm and form the
library carries, the factors of Sec. 2.3 as ``trv_cost_model`` computes them from the per-step, per-link byte loads
(``trv_link_loads``, a GPU tally):

    Lambda = steps / log3 n,   Delta = bytes sent per node / 2m,   Theta = sum_k max_link_bytes_k / (m / D)

next to the closed forms the paper prints in Tables 1 and 2 (App. B).  The set-ups are the ones App. B counts: the
bandwidth-optimal one-port algorithms with their mirrored sub-collectives, the latency-optimal ones on a torus as ONE
collective that walks through the dimensions.  Needs a CUDA device (the tally is a kernel); marshalling only.
"""
import argparse
import math

from . import binding as B

LAT, BW = B.LATENCY_OPTIMAL, B.BANDWIDTH_OPTIMAL


def _pow(n, b):
    k = round(math.log(n, b))
    return b ** k == n


def _rows(dims):
    """(label, algo flags, variant, closed form of Theta as the paper prints it or None)."""
    D, a = len(dims), dims[0]
    n = a ** D
    rows = []
    if _pow(a, 3):
        rows.append(("Trivance (L)", B.ALGO_TRIVANCE, LAT, (D / 2) * (a - 1) if D > 1 else (a - 1) / 2))
        rows.append(("Trivance (B)", B.ALGO_TRIVANCE, BW, None))
        rows.append(("Bruck (L)", B.ALGO_BRUCK, LAT, None))
        rows.append(("Bruck (B)", B.ALGO_BRUCK, BW, None))
    if _pow(a, 2):
        single = B.ALGO_SINGLE if D > 1 else 0
        rows.append(("Rec.Doub. (L)", B.ALGO_RECDOUB | single, LAT, None))
        rows.append(("Swing (L)", B.ALGO_SWING | single, LAT, None))
        rows.append(("Rec.Doub. (B)", B.ALGO_RECDOUB | B.ALGO_MIRRORED, BW, None))
        rows.append(("Swing (B)", B.ALGO_SWING | B.ALGO_MIRRORED, BW, None))
    rows.append(("Bucket", B.ALGO_BUCKET | B.ALGO_MIRRORED, BW, (n - 1) / n))
    return rows


def table(dims, count=None):
    """List of dicts, one per algorithm, for the a^D torus (D = 1: ring) `dims`."""
    D = len(dims)
    n = math.prod(dims)
    # a vector every collective splits into whole blocks, so that the tally carries no rounding of block lengths
    count = count or 2 * D * n * 6
    out = []
    for label, algo, variant, closed in _rows(dims):
        try:
            plan = B.Plan(dims, variant, algo)
        except B.TrivanceError:
            continue
        c = plan.cost_model(count, 4, 0.0, 1.0)
        out.append({"algorithm": label, "steps": c.steps, "lambda": c.lambda_, "delta": c.delta, "theta": c.theta,
                    "paper_closed_form": closed})
        plan.destroy()
    return out


def _print(dims):
    name = "ring of %d" % dims[0] if len(dims) == 1 else "torus " + "x".join(str(a) for a in dims)
    print("%s (n = %d)" % (name, math.prod(dims)))
    print("  %-14s %6s %9s %8s %9s" % ("algorithm", "steps", "Lambda", "Delta", "Theta"))
    for r in table(dims):
        print("  %-14s %6d %9.3f %8.3f %9.3f" % (r["algorithm"], r["steps"], r["lambda"], r["delta"], r["theta"]))


def main():
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--ring", type=int, nargs="*", default=[9, 27, 81, 8, 64])
    ap.add_argument("--torus", type=int, nargs="*", default=[9, 2, 3, 3, 8, 2, 4, 3],
                    help="pairs: side, dimensions (9 2 = 9x9, 4 3 = 4x4x4)")
    args = ap.parse_args()
    for n in args.ring:
        _print((n,))
    for i in range(0, len(args.torus) - 1, 2):
        _print((args.torus[i],) * args.torus[i + 1])


if __name__ == "__main__":
    main()
