"""Rank-sharded Trivance: every process (GPU) hosts a contiguous range of the n ranks and the partials of the ranks
at distance 3^k really travel between processes (Discussion and App. D: the deployment the paper aims at).

Process g of G hosts ranks [floor(g n / G), floor((g + 1) n / G)) as the rows of one ``[n_local, count]`` tensor.
Per schedule step the processes exchange, with ``torch.distributed`` point-to-point operations (NCCL between GPUs,
gloo in the CPU tests), exactly the messages the schedule defines -- the whole slice in the latency-optimal form
(Sec. 4.2), the blocks of the step's sets in the bandwidth-optimal form (Sec. 4.1, 4.3, and Sec. 4.4 for sides that
are no powers of three) -- and every process then runs the joint reductions of its own ranks:
``(from_left + own) + from_right`` with the library's ``trv_joint_reduce`` reading the received partials where they
were received.  Which rank sends which blocks to whom comes from the plan's host tables (``trv_plan_step``,
``trv_plan_send_set``, ``trv_plan_block_bounds``); this module holds the exchange bookkeeping only.

The arithmetic is injected: ``reduce_segments(left, own, right, out)`` gets lists of 1-D tensors (``None`` for a side
that sends nothing) and must write ``out[i] = (left[i] + own[i]) + right[i]``.  The default runs ``trv_joint_reduce``
on CUDA tensors; it refuses CPU tensors (there is no CPU path in the product).  The CPU tests pass a stand-in so that
the exchange logic can be checked with gloo ranks.
"""
import numpy as np

from . import binding

LATENCY, BANDWIDTH = binding.LATENCY_OPTIMAL, binding.BANDWIDTH_OPTIMAL


def rank_range(n, world, g):
    """Ranks [lo, hi) hosted by process g of `world`."""
    if world < 1 or not 0 <= g < world:
        raise ValueError("bad process index")
    return (g * n) // world, ((g + 1) * n) // world


def host_of(n, world, r):
    """The process hosting rank r."""
    g = min(world - 1, (r * world) // n)
    while rank_range(n, world, g)[0] > r:
        g -= 1
    while rank_range(n, world, g)[1] <= r:
        g += 1
    return g


def cuda_reduce_segments(left, own, right, out):
    """The product's arithmetic: trv_joint_reduce on the current CUDA stream."""
    import torch
    if not own:
        return
    if not all(t.is_cuda for t in own + out):
        raise RuntimeError("rank-sharded Trivance runs its reductions on CUDA tensors (no CPU path in the product)")
    dt = binding.INT32 if own[0].dtype == torch.int32 else binding.FLOAT32
    ptr = lambda ts: [0 if t is None else t.data_ptr() for t in ts]
    binding.joint_reduce(ptr(left), ptr(own), ptr(right), ptr(out), [t.numel() for t in own], dt,
                         torch.cuda.current_stream().cuda_stream)


class RankSharded:
    """AllReduce of ``local`` ([n_local, count], row i = rank lo + i) across the processes of a group, in place."""

    def __init__(self, plan, world, me, exchange, reduce_segments=cuda_reduce_segments):
        """exchange(sends, recvs): sends / recvs = lists of (process, tensor); performs all of them (the tensors of
        `recvs` are filled on return).  ``torch_exchange`` gives the torch.distributed one."""
        if plan.algo != binding.ALGO_TRIVANCE:
            raise ValueError("Trivance plans only")
        self.plan, self.world, self.me = plan, world, me
        self.exchange, self.reduce = exchange, reduce_segments
        self.n = plan.n
        self.lo, self.hi = rank_range(self.n, world, me)
        self.hosts = np.array([host_of(self.n, world, r) for r in range(self.n)])

    # ---- schedule tables (host integers from the plan)
    def _peers(self, c, row):
        return self.plan.peers(c, row)                  # [n][2]: left, right

    def _recv_masks(self, c, t):
        """[n][n] uint8: bit 0 = rank p gets a partial of block j from its left peer in Reduce-Scatter step t, bit 1 =
        from its right peer.  Regular schedules send the same set from both sides."""
        m = np.stack([self.plan.send_mask(c, t, p) for p in range(self.n)])
        general = any(_not_pow3(a) for a in self.plan.dims)
        return m if general else (m.astype(bool) * 3).astype(np.uint8)

    # ---- one exchange: every (source rank, destination rank, element ranges) triple; returns the received pieces
    def _swap(self, local, triples):
        """triples: list of (src, dst, [(e0, e1), ...]) over ALL ranks, the same list on every process.  Sends what my
        ranks owe to remote ranks, receives what remote ranks owe to mine.  Returns {(src, dst): tensor}: for a source I
        host myself a snapshot of its ranges, for a remote source the received buffer."""
        import torch
        got, sends, recvs = {}, {}, {}
        for src, dst, ranges in triples:
            hs, hd = self.hosts[src], self.hosts[dst]
            if hs != self.me and hd != self.me:
                continue
            length = sum(b - a for a, b in ranges)
            if hs == self.me:
                row = local[src - self.lo]
                piece = torch.cat([row[a:b] for a, b in ranges]) if ranges else row[:0].clone()
                if hd == self.me:
                    got[(src, dst)] = piece             # a copy: the source row may be overwritten in this step
                else:
                    sends.setdefault(int(hd), []).append(piece)
            else:
                buf = torch.empty(length, dtype=local.dtype, device=local.device)
                got[(src, dst)] = buf
                recvs.setdefault(int(hs), []).append(buf)
        # one message per pair of processes and direction: the pieces in the (common) order of the list
        out_msgs = [(q, torch.cat(ps) if ps else local.new_empty(0)) for q, ps in sorted(sends.items())]
        in_bufs = {q: torch.empty(sum(b.numel() for b in bs), dtype=local.dtype, device=local.device)
                   for q, bs in sorted(recvs.items())}
        self.exchange(out_msgs, sorted(in_bufs.items()))
        for q, bs in recvs.items():
            off = 0
            for b in bs:
                b.copy_(in_bufs[q][off:off + b.numel()])
                off += b.numel()
        return got

    def __call__(self, local, count=None):
        import torch
        plan = self.plan
        count = local.shape[1] if count is None else count
        if local.shape[0] != self.hi - self.lo:
            raise ValueError("local must hold one row per hosted rank")
        S = plan.rows if plan.variant == LATENCY else plan.rows // 2
        mine = range(self.lo, self.hi)
        for c in range(plan.nslices):
            bounds = plan.block_bounds(count, c)
            slo, shi = int(bounds[0]), int(bounds[-1])
            if shi <= slo:
                continue
            if plan.variant == LATENCY:
                for t in range(S):
                    peers = self._peers(c, t)
                    triples = [(int(peers[p][k]), p, [(slo, shi)]) for p in range(self.n) for k in (0, 1)]
                    got = self._swap(local, triples)
                    own = [local[p - self.lo][slo:shi] for p in mine]
                    self.reduce([got[(int(peers[p][0]), p)] for p in mine], own, [got[(int(peers[p][1]), p)] for p in mine], own)
                continue
            # ---- Reduce-Scatter
            masks = []
            for t in range(S):
                peers, m = self._peers(c, t), self._recv_masks(c, t)
                masks.append(m)
                triples, segs = [], []
                for p in range(self.n):
                    for k, bit in ((0, 1), (1, 2)):
                        blocks = np.nonzero(m[p] & bit)[0]
                        if k == 1 and peers[p][1] == peers[p][0]:
                            blocks = blocks[:0]          # both peers are one node: it sends once
                        rng = [(int(bounds[j]), int(bounds[j + 1])) for j in blocks if bounds[j + 1] > bounds[j]]
                        if rng:
                            triples.append((int(peers[p][k]), p, rng))
                got = self._swap(local, triples)
                L, O, R = [], [], []
                for p in mine:
                    row = local[p - self.lo]
                    fl, fr = got.get((int(peers[p][0]), p)), got.get((int(peers[p][1]), p))
                    if peers[p][1] == peers[p][0]:
                        fr = None
                    ol = orr = 0
                    for j in np.nonzero(m[p])[0]:
                        a, b = int(bounds[j]), int(bounds[j + 1])
                        if b <= a:
                            continue
                        has_l = bool(m[p][j] & 1) and fl is not None
                        has_r = bool(m[p][j] & 2) and fr is not None
                        L.append(fl[ol:ol + b - a] if has_l else None)
                        R.append(fr[orr:orr + b - a] if has_r else None)
                        O.append(row[a:b])
                        ol += (b - a) if has_l else 0
                        orr += (b - a) if has_r else 0
                self.reduce(L, O, R, O)
            # ---- AllGather: the mirror image; a rank gets back, from the peer it sent a partial to, the finished block
            for t in range(S - 1, -1, -1):
                peers, m = self._peers(c, t), masks[t]
                triples, plan_copy = [], {}
                for p in range(self.n):
                    for k, bit in ((0, 2), (1, 1)):     # my left peer got block j from ITS right peer (me): bit 1 of ITS mask
                        q = int(peers[p][k])
                        if k == 1 and peers[p][1] == peers[p][0]:
                            continue
                        blocks = [j for j in np.nonzero(m[q] & bit)[0] if bounds[j + 1] > bounds[j]]
                        if k == 0 and peers[p][1] == peers[p][0]:
                            blocks = [j for j in np.nonzero(m[q])[0] if bounds[j + 1] > bounds[j]]
                        if blocks:
                            rng = [(int(bounds[j]), int(bounds[j + 1])) for j in blocks]
                            triples.append((q, p, rng))
                            plan_copy[(q, p)] = rng
                got = self._swap(local, triples)
                for (q, p), rng in plan_copy.items():
                    if self.hosts[p] != self.me:
                        continue
                    row, piece, off = local[p - self.lo], got[(q, p)], 0
                    for a, b in rng:
                        row[a:b].copy_(piece[off:off + b - a])
                        off += b - a
        return local


def _not_pow3(a):
    while a % 3 == 0:
        a //= 3
    return a != 1


def torch_exchange(group=None):
    """exchange() over torch.distributed point-to-point operations (NCCL between GPUs, gloo on CPU)."""
    import torch.distributed as dist

    def exchange(sends, recvs):
        ops = [dist.P2POp(dist.isend, t, q, group) for q, t in sends if t.numel()]
        ops += [dist.P2POp(dist.irecv, t, q, group) for q, t in recvs if t.numel()]
        if ops:
            for w in dist.batch_isend_irecv(ops):
                w.wait()
    return exchange
