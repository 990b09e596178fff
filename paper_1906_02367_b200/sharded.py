"""The synchronisation round over several GPUs, one process per GPU (torch.distributed).

The masterless form the paper mentions in Section 1: every worker's record goes to all the others
and each aggregates for itself.  Worker r lives on rank r // (R / G); a rank compresses and packs its
own workers (qs_compress_feedback, qs_pack on a context that qs_set_sharding told its place in the
job), the packed records are exchanged with ONE all-gather (the only data-path collective: a few
tens of KB per worker; optionally in their gap-coded form, qs_recode_gaps / qs_decode_gaps), then every rank decodes the same R records in worker order
(qs_unpack_accumulate), so the replicas of x stay bit-identical, and broadcasts to its own workers
locally.  The gathered records land in this rank's memory before any kernel reads them.

Only host logic lives here: the partition, the masks, the collective.  The arithmetic is in the
library; `engine` is the object that runs it (a binding.Context by default).
"""
import numpy as np
import torch
import torch.distributed as dist


def partition(R, world):
    """(first worker, number of workers) of every rank: equal contiguous blocks."""
    if world < 1 or R % world != 0:
        raise ValueError("the number of workers must be a multiple of the number of ranks")
    per = R // world
    return [(g * per, per) for g in range(world)]


def local_mask(mask, base, count):
    """The part of a job-wide worker mask (None = everyone) that concerns this rank's workers."""
    if mask is None:
        return None
    m = np.ascontiguousarray(mask, dtype=np.uint8)
    return m[base:base + count].copy()


def gather_records(wire_local, R, group=None):
    """All ranks' packed records, rows ordered by global worker id (ranks hold contiguous blocks, so
    rank order is worker order).  wire_local: (R / G, stride) int32; returns (R, stride)."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    if world == 1:
        return wire_local
    out = torch.empty((R, wire_local.shape[1]), dtype=wire_local.dtype, device=wire_local.device)
    dist.all_gather_into_tensor(out, wire_local.contiguous(), group=group)
    return out


class ShardedRound:
    """One rank's share of a job of R workers.  x is this rank's replica of the global model; xw, mem
    (and anchors) hold this rank's workers only."""

    def __init__(self, R, engine, wire_local, rank=None, world=None, group=None, packed_local=None, records=None, nseg=1):
        """packed_local (R / G rows of qs_gap_words) and records (R rows of qs_wire_words) given: the
        records travel in their gap-coded form (qs_recode_gaps before the all-gather, qs_decode_gaps
        after it).  Rows are sized for the longest record there can be; what crosses the collective
        is cut to the longest record of the round (its bit count read back, the maximum agreed by a
        one-word all-reduce), so the exchange shrinks with the records.  nseg: segments per record."""
        self.packed_local, self.records = packed_local, records
        if (packed_local is None) != (records is None):
            raise ValueError("gap-coded exchange needs both packed_local and records")
        if packed_local is not None:
            self.gap_bits = torch.zeros(packed_local.shape[0], dtype=torch.int64, device=packed_local.device)
            self.packed_all = torch.zeros((int(R), packed_local.shape[1]), dtype=packed_local.dtype, device=packed_local.device)
            # words of a record of b bits: each directory entry holds 5 words against the 70 bits counted
            # for it, and each of a segment's streams (at most four) is padded to a word
            self.slack_words = 7 * int(nseg)
        self.exchanged_words = 0                  # per row, in the last round
        self.group = group
        self.world = world if world is not None else (dist.get_world_size(group) if dist.is_initialized() else 1)
        self.rank = rank if rank is not None else (dist.get_rank(group) if dist.is_initialized() else 0)
        self.R = int(R)
        self.base, self.count = partition(self.R, self.world)[self.rank]
        self.engine = engine
        self.wire_local = wire_local
        engine.set_sharding(self.base, self.R)

    def round(self, rnd, mask=None, bits_out=None):
        """Algorithm 1 (mask None) or Algorithm 2 (mask over the R workers of the job) for round rnd."""
        mine = local_mask(mask, self.base, self.count)
        if mine is None or mine.any():
            self.engine.compress_feedback(rnd, mine)
            self.engine.pack(self.wire_local, bits_out)
            if self.packed_local is not None:
                self.gap_bits.zero_()
                self.engine.recode_gaps(self.wire_local, self.packed_local, mine, self.gap_bits)
        if self.packed_local is not None:
            busy = mine is None or mine.any()
            longest = (int(self.gap_bits.max().item()) + 31) // 32 + self.slack_words if busy else 0
            width = torch.tensor([min(longest, self.packed_local.shape[1])], dtype=torch.int64, device=self.packed_local.device)
            if self.world > 1:
                dist.all_reduce(width, op=dist.ReduceOp.MAX, group=self.group)
            w = int(width.item())
            self.exchanged_words = w
            if w:
                self.packed_all[:, :w] = gather_records(self.packed_local[:, :w].contiguous(), self.R, self.group)
            self.engine.decode_gaps(self.packed_all, self.records, mask)
            records = self.records
        else:
            records = gather_records(self.wire_local, self.R, self.group)
            self.exchanged_words = int(self.wire_local.shape[1])
        self.engine.unpack_accumulate(records, mask)
        if mine is None or mine.any():
            self.engine.broadcast(mine)
        return records
