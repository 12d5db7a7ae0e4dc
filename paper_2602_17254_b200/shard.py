"""Element-range sharding of an AllReduce over several GPUs.

The AllReduce is element-wise, so every element column (all n simulated ranks x one element
index) is independent of every other.  GPU g of G therefore holds, for ALL n ranks, one
contiguous element range and calls ``trv_allreduce_ex`` with the global vector length and its
range's offset; slice and block membership follow the global element index, and nothing is
exchanged between GPUs.
"""


def element_shard(count, world, rank, align=4):
    """(offset, length) of the element range GPU `rank` of `world` holds.

    Cuts fall on multiples of `align` elements (16 bytes for 4-byte elements) so that every
    shard's buffers can start 16-byte aligned; the ranges tile [0, count) exactly.
    """
    if world < 1 or not 0 <= rank < world or count < 0 or align < 1:
        raise ValueError("bad shard request")

    def cut(g):
        if g >= world:
            return count
        c = (count * g) // world
        return min(count, (c // align) * align)

    lo, hi = cut(rank), cut(rank + 1)
    return lo, hi - lo
