"""One N-gram module shared by sequences that live on several GPUs (one process per GPU).

Each rank holds a contiguous block of the batch (its context is created with seq_base = the global index
of its first sequence) and a full copy of the table.  A step is: verify locally, exchange the accepted
rows (Sec. 4.1's update records: a few KB per sequence, never the logits), apply the rows of ALL ranks in
global sequence order, draft locally.  Every copy of the table then equals the table of one context that
held the whole batch, and so does every draft.

Only marshalling and the collective live here; verification, update and drafting run in the library.
"""
import torch


def concat_rows(parts):
    """parts: per shard (ctx, ids, probs), in the order of their seq_base -> one (ctx, ids, probs)."""
    return tuple(torch.cat([p[i] for p in parts], dim=0) for i in range(3))


def gather_rows(dist, rows):
    """All ranks' (ctx, ids, probs) concatenated in rank order.  Every rank must pass the same shapes (same
    sequences per rank, same tree), and rank r must hold the sequences before those of rank r + 1."""
    if dist is None:
        return rows
    world = dist.get_world_size()
    out = []
    for t in rows:
        t = t.contiguous()
        buf = torch.empty((world * t.shape[0],) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device)
        dist.all_gather(list(buf.chunk(world, dim=0)), t)  # rank r's rows land in the r-th block of buf
        out.append(buf)
    return tuple(out)


class ShardedStand:
    """Wraps one rank's context (binding.Stand created with seq_base = rank * B)."""

    def __init__(self, stand, dist=None):
        self.stand = stand
        self.dist = dist
        if dist is not None:
            assert stand.seq_base == dist.get_rank() * stand.B, "rank r holds sequences [r * B, (r + 1) * B)"

    def verify(self, logits):
        """Local verification; returns this rank's rows for the exchange."""
        self.stand.verify_tree(logits)
        rows = self.stand.export_records()
        self.stand.skip_update()
        return rows

    def finish(self, all_rows):
        """Applies the rows of all ranks (already in global sequence order) and drafts the next tree."""
        self.stand.ngram_update_bulk(*all_rows, sync=False)
        return self.stand.draft_tree()

    def step(self, logits):
        rows = self.verify(logits)
        return self.finish(gather_rows(self.dist, rows))
