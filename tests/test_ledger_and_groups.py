"""Checkpoint ledger (Algorithm 3) and peer groups (Sec. 4): the oracle against
the paper's worked examples, then the library against the oracle.  Host-only
logic: no GPU is needed for any of it."""
import random

import pytest

from oracle import host_logic as H
from paper_2608_11034_b200 import binding as B, build

build.build()
NO = B.NO_CHECKPOINT


# ---------------------------------------------------------------- oracle pins

def test_oracle_two_recipe_trace_of_the_paper():
    """K = 2: step 2 becomes the candidate, it is promoted after the clean check
    at step 4, an SDC at step 5 recovers step 2."""
    L = H.Ledger(2)
    assert L.checkpoint_save(H.HEALTHY, 1) == ("captured",)
    assert L.checkpoint_save(H.HEALTHY, 2) == ("boundary", 2, None)
    assert (L.candidate, L.verified) == (2, None)
    assert L.checkpoint_save(H.HEALTHY, 3) == ("captured",)
    assert L.checkpoint_save(H.HEALTHY, 4) == ("boundary", 4, 2)
    assert (L.latest, L.candidate, L.verified) == (4, 4, 2)
    assert L.checkpoint_save(H.SDC, 5) == ("retrieval", "verified", 2)
    assert (L.latest, L.candidate, L.verified) == (4, 4, 2)        # nothing captured at step 5


def test_oracle_hand_derived_traces_k1_and_k3():
    """Worked by hand from the prose of Sec. 8.  K = 1 (static shapes): every accepted
    check closes a cycle, so the capture one boundary back is the verified one.  K = 3:
    captures 3 and 6 are persisted; 3 is verified once check 6 has been accepted."""
    L = H.Ledger(1)
    assert L.checkpoint_save(H.HEALTHY, 10) == ("boundary", 10, None)
    assert L.checkpoint_save(H.STRAGGLER, 11) == ("boundary", 11, 10)       # a completed straggler counts
    assert L.checkpoint_save(H.HANG, 12, True, None) == ("retrieval", "need_sweep", None)
    assert L.checkpoint_save(H.HANG, 12, True, False) == ("retrieval", "latest", 11)
    assert (L.latest, L.candidate, L.verified, L.q) == (11, 11, 10, 0)
    assert L.checkpoint_save(H.HEALTHY, 13) == ("boundary", 13, 11)

    L = H.Ledger(3)
    want = {1: ("captured",), 2: ("captured",), 3: ("boundary", 3, None), 4: ("captured",),
            5: ("captured",), 6: ("boundary", 6, 3), 7: ("captured",)}
    for step in range(1, 8):
        assert L.checkpoint_save(H.HEALTHY, step) == want[step]
    assert (L.latest, L.candidate, L.verified, L.q) == (7, 6, 3, 1)
    assert L.checkpoint_save(H.SDC, 8) == ("retrieval", "verified", 3)      # not 6: only one cycle followed it
    assert (L.latest, L.candidate, L.verified, L.q) == (7, 6, 3, 1)         # and nothing moved
    assert L.checkpoint_retrieval(H.STRAGGLER) == ("latest", 7)
    # an SDC in the middle of a cycle does not restart the count (the listing leaves q alone)
    assert L.checkpoint_save(H.HEALTHY, 9) == ("captured",)
    assert L.checkpoint_save(H.HEALTHY, 10) == ("boundary", 10, 6)


def test_oracle_retrieval_rules_from_the_prose():
    L = H.Ledger(1)
    for step in (1, 2, 3):
        L.checkpoint_save(H.HEALTHY, step)
    assert (L.latest, L.candidate, L.verified) == (3, 3, 2)
    assert L.checkpoint_retrieval(H.SDC) == ("verified", 2)                         # confirmed SDC
    assert L.checkpoint_retrieval(H.STRAGGLER, machines_accessible=False) == ("verified", 2)
    assert L.checkpoint_retrieval(H.STRAGGLER) == ("latest", 3)                     # slowness is not corruption
    assert L.checkpoint_retrieval(H.HANG) == ("need_sweep", None)
    assert L.checkpoint_retrieval(H.HANG, replay_full_catalog=False) == ("latest", 3)
    assert L.checkpoint_retrieval(H.OTHER, replay_full_catalog=True) == ("verified", 2)


@pytest.mark.parametrize("K", [1, 2, 3, 5])
def test_oracle_promotion_needs_two_accepted_cycles(K):
    L = H.Ledger(K)
    captured_at = {}
    for step in range(1, 6 * K + 1):
        L.checkpoint_save(H.HEALTHY, step)
        captured_at[step] = step
        if L.verified is not None:
            # at least K accepted checks were made after the verified checkpoint was captured,
            # and at least 2K since the cycle that produced it began
            assert step - L.verified >= K
            assert L.verified % K == 0 and L.candidate - L.verified == K
    assert L.verified == 5 * K


def test_oracle_mesh_example_of_the_paper():
    shape = (4, 1, 2, 1, 1, 1)
    ranks = H.mesh_ranks(shape)
    assert all(r == 2 * a[0] + a[2] for r, a in ranks.items())                      # rank = 2d + t
    assert H.peer_group(shape, 0) == ("replica", [0, 2, 4, 6])
    assert H.peer_group(shape, 1) == ("replica", [1, 3, 5, 7])
    assert H.peer_group((1, 4, 2, 1, 1, 1), 3) == ("shard", [1, 3, 5, 7])           # pure FSDP
    assert H.peer_group((1, 1, 2, 2, 1, 1), 3) == ("none", [3])


# ---------------------------------------------------------------- library vs oracle

def _lib_step(ledger, f, captured, acc, sweep):
    ev = B.scout_ledger_save(ledger, f, captured, acc, -1 if sweep is None else int(sweep))
    act = ev["action"]
    if act == B.LEDGER_CAPTURED:
        return ("captured",)
    if act == B.LEDGER_BOUNDARY:
        return ("boundary", ev["checkpoint"], None if ev["promoted"] == NO else ev["promoted"])
    if act == B.LEDGER_NEED_SWEEP:
        return ("retrieval", "need_sweep", None)
    role = {B.ROLE_LATEST: "latest", B.ROLE_VERIFIED: "verified"}[ev["role"]]
    return ("retrieval", role, None if ev["checkpoint"] == NO else ev["checkpoint"])


def test_ledger_matches_the_oracle_on_the_paper_trace_and_random_histories():
    rng = random.Random(8)
    for trial in range(300):
        K = rng.randrange(1, 5)
        L, ledger = H.Ledger(K), B.scout_ledger_create(K)
        for step in range(1, 40):
            if trial == 0:
                f = H.SDC if step == 5 else H.HEALTHY
            else:
                f = rng.choices([H.HEALTHY, H.STRAGGLER, H.SDC, H.HANG, H.OTHER], [12, 2, 1, 1, 1])[0]
            acc = rng.random() > 0.1
            sweep = rng.choice([None, False, True])
            assert _lib_step(ledger, f, step, acc, sweep) == L.checkpoint_save(f, step, acc, sweep)
            st = B.scout_ledger_state(ledger)
            want = [NO if x is None else x for x in (L.latest, L.candidate, L.verified)]
            assert [st["latest"], st["candidate"], st["verified"]] == want
            assert (st["q"], st["K"], st["n_persisted"]) == (L.q, K, len(L.persisted))
            if f != H.HEALTHY:
                ev = B.scout_ledger_retrieve(ledger, f, acc, -1 if sweep is None else int(sweep))
                role, ck = L.checkpoint_retrieval(f, acc, sweep)
                if role == "need_sweep":
                    assert ev["action"] == B.LEDGER_NEED_SWEEP
                else:
                    assert ev["role"] == {"latest": B.ROLE_LATEST, "verified": B.ROLE_VERIFIED}[role]
                    assert ev["checkpoint"] == (NO if ck is None else ck)
        B.scout_ledger_destroy(ledger)


def test_ledger_argument_checks_and_report_mapping():
    with pytest.raises(B.ScoutError):
        B.scout_ledger_create(0)
    ledger = B.scout_ledger_create(2)
    with pytest.raises(B.ScoutError):
        B.scout_ledger_save(ledger, 9, 1)
    with pytest.raises(B.ScoutError):
        B.scout_ledger_save(ledger, B.OUTCOME_HEALTHY, NO)
    with pytest.raises(B.ScoutError):
        B.scout_ledger_retrieve(ledger, B.OUTCOME_HEALTHY)
    B.scout_ledger_destroy(ledger)
    rep = {k: 0 for k in B.REPORT_DTYPE.names}
    for verdict, want in ((B.CERTIFIED, B.OUTCOME_HEALTHY), (B.VERDICT_ATTRIBUTED, B.OUTCOME_SDC),
                          (B.UNDECIDED, B.OUTCOME_SDC)):
        rep["verdict"] = verdict
        assert B.scout_outcome_from_report(rep) == want


@pytest.mark.parametrize("shape", [(4, 1, 2, 1, 1, 1), (1, 4, 2, 1, 1, 1), (2, 4, 2, 2, 1, 1),
                                   (3, 1, 1, 2, 2, 2), (1, 1, 2, 3, 1, 1), (16, 1, 1, 1, 1, 1),
                                   (2, 2, 2, 2, 2, 2)])
def test_peer_groups_match_the_oracle_and_partition_the_ranks(shape):
    n = B.scout_mesh_size(shape)
    ranks = H.mesh_ranks(shape)
    assert n == len(ranks)
    kinds = {"none": B.GROUP_NONE, "replica": B.GROUP_REPLICA, "shard": B.GROUP_SHARD}
    seen = {}
    for r in range(n):
        assert B.scout_mesh_coords(shape, r) == ranks[r]
        assert B.scout_mesh_rank(shape, ranks[r]) == r
        kind, peers = B.scout_peer_group(shape, r)
        okind, opeers = H.peer_group(shape, r)
        assert (kind, peers) == (kinds[okind], opeers)
        assert r in peers
        seen.setdefault(tuple(peers), set()).add(r)
    assert all(set(g) == members for g, members in seen.items())        # groups partition the ranks
    assert sum(len(g) for g in seen) == n


def test_peer_group_truncation_and_bad_arguments():
    kind, peers = B.scout_peer_group((8, 1, 1, 1, 1, 1), 3, cap=4)
    assert kind == B.GROUP_REPLICA and peers == [0, 1, 2, 3]
    with pytest.raises(B.ScoutError):
        B.scout_mesh_coords((2, 1, 1, 1, 1, 1), 2)
    with pytest.raises(B.ScoutError):
        B.scout_mesh_size((2, 0, 1, 1, 1, 1))


def test_rotating_slice_covers_every_element_once_per_rotation():
    for numel, slice_elems in ((1, 65536), (65536, 65536), (65537, 65536), (1_000_003, 65536), (10, 3)):
        n_windows = -(-numel // slice_elems)
        seen = []
        for step in range(2 * n_windows + 1):
            got = B.scout_rotating_slice(numel, slice_elems, step)
            assert got == H.rotating_slice(numel, slice_elems, step)
            seen.append(got)
        one_turn = seen[:n_windows]
        covered = [i for b, n in one_turn for i in range(b, b + n)] if numel < 10**5 else None
        if covered is not None:
            assert covered == list(range(numel))          # every element exactly once per rotation
        assert sum(n for _, n in one_turn) == numel
        assert seen[n_windows:2 * n_windows] == one_turn and seen[2 * n_windows] == seen[0]
    with pytest.raises(B.ScoutError):
        B.scout_rotating_slice(0, 65536, 0)


@pytest.mark.gpu
def test_signing_a_rotating_slice_localises_a_fault_inside_it():
    import torch
    import helpers
    from paper_2608_11034_b200 import inputs
    numel, slice_elems = 300_000, 65536
    spec = inputs.TensorSpec("param", (numel,), "f32", "normal", 0.02)
    w = inputs.Workload("slice", 0, "x", 3, 16384, [spec], 31)
    w.patches = [inputs.Patch(2, 0, 200_000, "xor", 1 << 13)]
    _, views = inputs.generate(w, "cuda")
    hits = {}
    for step in range(5):
        begin, count = B.scout_rotating_slice(numel, slice_elems, step)
        sw = inputs.Workload("slice", 0, "x", 3, 16384,
                             [inputs.TensorSpec("param", (count,), "f32", "normal", 0.02)], 31)
        sviews = [[views[r][0][begin:begin + count]] for r in range(3)]
        got = helpers.gpu_sign_vote(sw, sviews)
        hits[step] = got["outliers"]
    window = 200_000 // slice_elems
    chunk = (200_000 - window * slice_elems) * 4 // 16384
    assert hits == {0: [], 1: [], 2: [], 3: [(chunk, 2)], 4: []}
