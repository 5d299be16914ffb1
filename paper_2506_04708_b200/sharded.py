"""One N-gram module shared by sequences that live on several GPUs (one process per GPU).

Each rank holds a contiguous block of the batch (its context is created with seq_base = the global index
of its first sequence) and a full copy of the table.  A step is: verify locally, exchange the accepted
rows (Sec. 4.1's update records: a few KB per sequence, never the logits; one gather of one packed buffer), apply the rows of ALL ranks in
global sequence order, draft locally.  Every copy of the table then equals the table of one context that
held the whole batch, and so does every draft.

Only marshalling and the collective live here; verification, update and drafting run in the library.
"""
import torch


def concat_rows(parts):
    """parts: per shard packed rows [rows, order_max + 2*topk], in the order of their seq_base -> one tensor."""
    return torch.cat(list(parts), dim=0)


def gather_rows(dist, rows, out=None):
    """All ranks' packed rows concatenated in rank order, with ONE collective.  Every rank must pass the same
    shape (same sequences per rank, same tree), and rank r must hold the sequences before those of rank r + 1."""
    if dist is None:
        return rows
    world = dist.get_world_size()
    rows = rows.contiguous()
    if out is None:
        out = torch.empty((world * rows.shape[0],) + tuple(rows.shape[1:]), dtype=rows.dtype, device=rows.device)
    dist.all_gather_into_tensor(out, rows)  # rank r's rows land in the r-th block
    return out


class ShardedStand:
    """Wraps one rank's context (binding.Stand created with seq_base = rank * B)."""

    def __init__(self, stand, dist=None):
        self.stand = stand
        self.dist = dist
        self._mine = self._all = None
        if dist is not None:
            assert stand.seq_base == dist.get_rank() * stand.B, "rank r holds sequences [r * B, (r + 1) * B)"
            rows, width = stand.B * (stand.D + 1), stand.n_max + 2 * stand.K
            self._mine = torch.empty((rows, width), dtype=torch.int32, device=stand.dev)
            self._all = torch.empty((dist.get_world_size() * rows, width), dtype=torch.int32, device=stand.dev)

    def verify(self, logits):
        """Local verification; returns this rank's packed rows for the exchange."""
        self.stand.verify_tree(logits)
        rows = self.stand.export_records_packed(out=self._mine)
        self.stand.skip_update()
        return rows

    def finish(self, all_rows):
        """Applies the rows of all ranks (already in global sequence order) and drafts the next tree."""
        self.stand.ngram_update_packed(all_rows)
        return self.stand.draft_tree()

    def step(self, logits):
        rows = self.verify(logits)
        return self.finish(gather_rows(self.dist, rows, self._all))
