"""Oracle for the host-side rules (TEST INFRASTRUCTURE, not product code).

Plain Python models of two pieces of the paper that involve no data path: the
checkpoint protocol (Sec. 8) and peer-group formation (Sec. 4).  The ledger is a
history-replay model: it keeps the list of boundary events and derives the three
roles from the list by the prose rule, so it shares neither code nor structure
with the C++ library (which keeps a counter and shifts roles at a boundary).

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
    """The checkpoint protocol of Sec. 8 as a model over the whole history.

    The object stores nothing but the list of boundary events it was given.  The
    three roles are recomputed from that list every time they are asked for, by
    the rule the prose states ("Checkpoint saving during training"):

      * only accepted checks (healthy, or a straggler that completed) capture
        state; an SDC or a hang captures nothing and leaves the count alone;
      * accepted checks are grouped into consecutive cycles of K; the capture of
        the check that closes a cycle is the one that is persisted;
      * latest   = capture of the most recent accepted check;
        candidate = capture persisted at the most recent cycle boundary;
        verified  = capture persisted one boundary earlier, i.e. the newest
                    persisted capture that has been FOLLOWED by K more accepted
                    checks (so 2K accepted checks lie between the start of its
                    own cycle and its promotion).
    """

    def __init__(self, K):
        assert K >= 1
        self.K = K
        self.history = []              # (outcome, captured id) for every boundary, in order

    # ---- views over the history ------------------------------------------------
    def _accepted(self):
        return [ck for f, ck in self.history if f not in (SDC, HANG)]

    def _persisted(self):
        a = self._accepted()
        return a[self.K - 1::self.K]   # capture of every K-th accepted check

    @property
    def q(self):
        return len(self._accepted()) % self.K

    @property
    def persisted(self):
        return self._persisted()

    @property
    def latest(self):
        a = self._accepted()
        return a[-1] if a else NONE

    @property
    def candidate(self):
        p = self._persisted()
        return p[-1] if p else NONE

    @property
    def verified(self):
        a = self._accepted()
        boundaries = len(a) // self.K              # cycles closed so far
        if boundaries < 2:
            return NONE
        pos = (boundaries - 1) * self.K - 1        # where the previous boundary's capture sits
        assert len(a) - 1 - pos >= self.K          # K accepted checks followed it: what makes it trusted
        return a[pos]

    # ---- the two procedures ------------------------------------------------------
    def checkpoint_save(self, f, captured, machines_accessible=True, replay_full_catalog=None):
        if f in (SDC, HANG):
            self.history.append((f, NONE))
            return ("retrieval",) + self.checkpoint_retrieval(f, machines_accessible, replay_full_catalog)
        n_before = len(self._persisted())
        self.history.append((f, captured))
        if len(self._persisted()) > n_before:
            return ("boundary", self.candidate, self.verified)
        return ("captured",)

    def checkpoint_retrieval(self, f, machines_accessible=True, replay_full_catalog=None):
        """-> (role, checkpoint), from the prose of "Checkpoint retrieval for failure
        recovery".  replay_full_catalog: None (the sweep has not run), or a bool
        saying whether it found an SDC."""
        newest_is_vouched_for = machines_accessible and f != SDC and (
            f == STRAGGLER or replay_full_catalog is False)
        undecidable_yet = machines_accessible and f not in (SDC, STRAGGLER) and replay_full_catalog is None
        if undecidable_yet:
            return ("need_sweep", NONE)
        return ("latest", self.latest) if newest_is_vouched_for else ("verified", self.verified)


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
