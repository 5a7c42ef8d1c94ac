"""Oracle for the host-side rules (TEST INFRASTRUCTURE, not product code).

Plain Python restatements of two pieces of the paper that involve no data path:
the checkpoint protocol (Sec. 8, Algorithm 3) and peer-group formation (Sec. 4).
Nothing here is shared with the C++ library.

Parity status: pinned by the paper's own worked examples (the two-recipe trace of
Sec. 10: step 2 becomes the candidate, is promoted after the clean check at step
4, an SDC at step 5 recovers step 2; the (4,1,2,1,1,1) mesh whose groups are
{0,2,4,6} and {1,3,5,7}), by the retrieval rules stated in prose, and by
invariants (a checkpoint is verified only after K further accepted checks follow
its capture; peer groups partition the ranks).
"""
from itertools import product

HEALTHY, STRAGGLER, SDC, HANG, OTHER = range(5)
NONE = None


class Ledger:
    """Algorithm 3, state and both procedures, in the listing's own terms."""

    def __init__(self, K):
        assert K >= 1
        self.K, self.q = K, 0
        self.latest = self.candidate = self.verified = NONE
        self.persisted = []

    def checkpoint_save(self, f, captured, machines_accessible=True, replay_full_catalog=None):
        if f in (SDC, HANG):
            return ("retrieval",) + self.checkpoint_retrieval(f, machines_accessible, replay_full_catalog)
        self.latest = captured
        self.q += 1
        if self.q == self.K:
            self.q = 0
            self.verified = self.candidate
            self.persisted.append(self.latest)
            self.candidate = self.latest
            return ("boundary", self.candidate, self.verified)
        return ("captured",)

    def checkpoint_retrieval(self, f, machines_accessible=True, replay_full_catalog=None):
        """-> (role, checkpoint).  replay_full_catalog: None (not run), or a bool
        saying whether the sweep found an SDC."""
        if f == SDC or not machines_accessible:
            return ("verified", self.verified)
        if f == STRAGGLER:
            return ("latest", self.latest)
        if replay_full_catalog is None:
            return ("need_sweep", NONE)
        if replay_full_catalog:
            return ("verified", self.verified)
        return ("latest", self.latest)


def mesh_ranks(shape):
    """All ranks with their addresses, row-major over (d, s, t, p, c, e)."""
    return {rank: addr for rank, addr in enumerate(product(*[range(g) for g in shape]))}


def peer_group(shape, r):
    """-> (kind, sorted peers): G_rep when the data-replica degree exceeds one,
    else G_shard when the state-shard degree exceeds one, else the singleton."""
    ranks = mesh_ranks(shape)
    d, s, t, p, c, e = ranks[r]
    if shape[0] > 1:
        peers = [q for q, a in ranks.items() if a[1:] == (s, t, p, c, e)]
        return "replica", sorted(peers)
    if shape[1] > 1:
        peers = [q for q, a in ranks.items() if a[2:] == (t, p, c, e)]
        return "shard", sorted(peers)
    return "none", [r]


def rotating_slice(numel, slice_elems, step):
    """Window `step` of the rotation over a tensor of `numel` elements: the
    windows are the consecutive pieces range(0, numel, slice_elems), visited
    round-robin (the paper only says the slice rotates; this is the reading)."""
    windows = [(b, min(slice_elems, numel - b)) for b in range(0, numel, slice_elems)]
    return windows[step % len(windows)]
