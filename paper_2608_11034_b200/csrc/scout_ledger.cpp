// Host-only part of the library: the checkpoint ledger of Sec. 8 (the protocol
// Algorithm 3 summarises) and peer-group formation of Sec. 4.  No CUDA here.
#include <new>

#include "scout_ledger.h"

// The ledger is two small machines (Sec. 8, "Checkpoint saving during training" and
// "Checkpoint retrieval for failure recovery"):
//   * a cycle of K accepted checks.  Closing a cycle shifts the durable roles by
//     one place: what was persisted at the previous boundary has now seen a full
//     catalog of accepted checks after its capture and becomes trusted; the newest
//     capture is persisted in its place.
//   * a selector that answers "which role do we restart from" for a failure class.
//     It is a pure function of (failure class, machines reachable, emergency sweep
//     result) and is kept as a decision table.
struct DurableRoles {
    uint64_t awaiting = SCOUT_NO_CHECKPOINT;  // persisted, not yet followed by a full accepted cycle
    uint64_t trusted = SCOUT_NO_CHECKPOINT;   // persisted and followed by a full accepted cycle
};

struct scout_ledger {
    uint64_t newest_capture = SCOUT_NO_CHECKPOINT;
    DurableRoles durable;
    uint32_t accepted_in_cycle = 0, cycle_length = 1;
    uint64_t cycles_closed = 0;
};

namespace {

enum class Verdict { Accept, Reject };  // does this boundary's outcome allow a capture?
enum class Pick { Trusted, Newest, RunSweepFirst };

// Only a numerical disagreement or a hang blocks the capture; slowness alone does not.
Verdict judge(int outcome) {
    return (outcome == SCOUT_OUTCOME_SDC || outcome == SCOUT_OUTCOME_HANG) ? Verdict::Reject
                                                                         : Verdict::Accept;
}

// Decision table of the selector.  Rows: failure class.  Columns: machines
// reachable? then the sweep result (not run / clean / found SDC).
//   - a confirmed SDC never restarts from unverified state;
//   - an unreachable machine hides part of the newest capture, so it cannot be vouched for;
//   - a straggler is slow, not wrong: the newest capture is fine;
//   - anything else is decided by replaying the whole catalog once.
constexpr Pick T = Pick::Trusted, N = Pick::Newest, S = Pick::RunSweepFirst;
constexpr Pick kSelector[5][2][3] = {
    /* HEALTHY   */ {{T, T, T}, {S, N, T}},  // not a failure class; scout_ledger_retrieve rejects it
    /* STRAGGLER */ {{T, T, T}, {N, N, N}},
    /* SDC       */ {{T, T, T}, {T, T, T}},
    /* HANG      */ {{T, T, T}, {S, N, T}},
    /* OTHER     */ {{T, T, T}, {S, N, T}},
};

int select_restart_point(const scout_ledger *l, int failure, int reachable, int sweep,
                         scout_ledger_event_t *ev) {
    const int sweep_col = sweep < 0 ? 0 : (sweep == 0 ? 1 : 2);
    const Pick pick = kSelector[failure][reachable ? 1 : 0][sweep_col];
    ev->promoted = SCOUT_NO_CHECKPOINT;
    switch (pick) {
        case Pick::RunSweepFirst:
            ev->action = SCOUT_LEDGER_NEED_SWEEP;
            ev->role = SCOUT_ROLE_NONE;
            ev->checkpoint = SCOUT_NO_CHECKPOINT;
            break;
        case Pick::Trusted:
            ev->action = SCOUT_LEDGER_RETRIEVAL;
            ev->role = SCOUT_ROLE_VERIFIED;
            ev->checkpoint = l->durable.trusted;
            break;
        case Pick::Newest:
            ev->action = SCOUT_LEDGER_RETRIEVAL;
            ev->role = SCOUT_ROLE_LATEST;
            ev->checkpoint = l->newest_capture;
            break;
    }
    return SCOUT_OK;
}

// The K-th accepted check of a cycle arrived: shift the durable roles.
void close_cycle(scout_ledger *l, scout_ledger_event_t *ev) {
    const DurableRoles before = l->durable;
    l->durable.trusted = before.awaiting;
    l->durable.awaiting = l->newest_capture;  // the caller persists this id
    l->accepted_in_cycle = 0;
    l->cycles_closed += 1;
    ev->action = SCOUT_LEDGER_BOUNDARY;
    ev->checkpoint = l->durable.awaiting;
    ev->promoted = l->durable.trusted;
}

bool valid_outcome(int f) { return f >= SCOUT_OUTCOME_HEALTHY && f <= SCOUT_OUTCOME_OTHER; }

uint32_t degree(const scout_mesh_t *m, int i) {
    const uint32_t v[6] = {m->d, m->s, m->t, m->p, m->c, m->e};
    return v[i];
}
void set_coord(scout_mesh_t *m, int i, uint32_t x) {
    uint32_t *v[6] = {&m->d, &m->s, &m->t, &m->p, &m->c, &m->e};
    *v[i] = x;
}
bool valid_shape(const scout_mesh_t *m) {
    if (!m) return false;
    uint64_t n = 1;
    for (int i = 0; i < 6; ++i) {
        const uint32_t g = degree(m, i);
        if (g == 0) return false;
        if (n > (UINT64_MAX / g)) return false;
        n *= g;
    }
    return true;
}

}  // namespace

extern "C" {

int scout_ledger_create(uint32_t K, scout_ledger_t **out) {
    if (!out) return SCOUT_ERR_INVALID;
    *out = nullptr;
    if (K == 0) return SCOUT_ERR_INVALID;
    scout_ledger *l = new (std::nothrow) scout_ledger;
    if (!l) return SCOUT_ERR_NOMEM;
    l->cycle_length = K;
    *out = l;
    return SCOUT_OK;
}

int scout_ledger_destroy(scout_ledger_t *l) {
    delete l;
    return SCOUT_OK;
}

int scout_ledger_state(const scout_ledger_t *l, scout_ledger_state_t *s) {
    if (!l || !s) return SCOUT_ERR_INVALID;
    s->latest = l->newest_capture;
    s->candidate = l->durable.awaiting;
    s->verified = l->durable.trusted;
    s->q = l->accepted_in_cycle;
    s->K = l->cycle_length;
    s->n_persisted = l->cycles_closed;
    return SCOUT_OK;
}

int scout_ledger_save(scout_ledger_t *l, int f, uint64_t captured, int accessible, int sweep,
                      scout_ledger_event_t *ev) {
    if (!l || !ev || !valid_outcome(f)) return SCOUT_ERR_INVALID;
    if (judge(f) == Verdict::Reject)  // nothing is captured; the ledger itself is left as it is
        return select_restart_point(l, f, accessible, sweep, ev);
    if (captured == SCOUT_NO_CHECKPOINT) return SCOUT_ERR_INVALID;
    l->newest_capture = captured;
    ev->action = SCOUT_LEDGER_CAPTURED;
    ev->role = SCOUT_ROLE_NONE;
    ev->checkpoint = SCOUT_NO_CHECKPOINT;
    ev->promoted = SCOUT_NO_CHECKPOINT;
    if (++l->accepted_in_cycle == l->cycle_length) close_cycle(l, ev);
    return SCOUT_OK;
}

int scout_ledger_retrieve(const scout_ledger_t *l, int f, int accessible, int sweep,
                          scout_ledger_event_t *ev) {
    if (!l || !ev || !valid_outcome(f) || f == SCOUT_OUTCOME_HEALTHY) return SCOUT_ERR_INVALID;
    return select_restart_point(l, f, accessible, sweep, ev);
}

int scout_outcome_from_report(const scout_report_t *r, int *outcome) {
    if (!r || !outcome) return SCOUT_ERR_INVALID;
    *outcome = r->verdict == SCOUT_CERTIFIED ? SCOUT_OUTCOME_HEALTHY : SCOUT_OUTCOME_SDC;
    return SCOUT_OK;
}

int scout_mesh_size(const scout_mesh_t *shape, uint64_t *n) {
    if (!valid_shape(shape) || !n) return SCOUT_ERR_INVALID;
    uint64_t x = 1;
    for (int i = 0; i < 6; ++i) x *= degree(shape, i);
    *n = x;
    return SCOUT_OK;
}

int scout_mesh_coords(const scout_mesh_t *shape, uint64_t rank, scout_mesh_t *coords) {
    uint64_t n;
    if (scout_mesh_size(shape, &n) || !coords || rank >= n) return SCOUT_ERR_INVALID;
    for (int i = 5; i >= 0; --i) {  // e is the fastest-varying coordinate
        const uint32_t g = degree(shape, i);
        set_coord(coords, i, (uint32_t)(rank % g));
        rank /= g;
    }
    return SCOUT_OK;
}

int scout_mesh_rank(const scout_mesh_t *shape, const scout_mesh_t *coords, uint64_t *rank) {
    if (!valid_shape(shape) || !coords || !rank) return SCOUT_ERR_INVALID;
    uint64_t r = 0;
    for (int i = 0; i < 6; ++i) {
        if (degree(coords, i) >= degree(shape, i)) return SCOUT_ERR_INVALID;
        r = r * degree(shape, i) + degree(coords, i);
    }
    *rank = r;
    return SCOUT_OK;
}

int scout_peer_group(const scout_mesh_t *shape, uint64_t rank, uint64_t *peers, uint64_t cap,
                     uint64_t *n, int *kind) {
    scout_mesh_t at;
    if (!n || !kind || (cap && !peers)) return SCOUT_ERR_INVALID;
    int rc = scout_mesh_coords(shape, rank, &at);
    if (rc) return rc;
    int free_dim = -1;
    if (shape->d > 1) { free_dim = 0; *kind = SCOUT_GROUP_REPLICA; }
    else if (shape->s > 1) { free_dim = 1; *kind = SCOUT_GROUP_SHARD; }
    else { *kind = SCOUT_GROUP_NONE; }
    if (free_dim < 0) {
        *n = 1;
        if (cap) peers[0] = rank;
        return cap ? SCOUT_OK : SCOUT_ERR_TRUNCATED;
    }
    const uint32_t g = degree(shape, free_dim);
    *n = g;
    for (uint32_t x = 0; x < g && x < cap; ++x) {
        scout_mesh_t q = at;
        set_coord(&q, free_dim, x);
        scout_mesh_rank(shape, &q, &peers[x]);
    }
    return g > cap ? SCOUT_ERR_TRUNCATED : SCOUT_OK;
}

int scout_rotating_slice(uint64_t numel, uint64_t slice_elems, uint64_t step, uint64_t *begin,
                         uint64_t *count) {
    if (!begin || !count || numel == 0 || slice_elems == 0) return SCOUT_ERR_INVALID;
    const uint64_t n_windows = numel / slice_elems + (numel % slice_elems ? 1 : 0);
    const uint64_t w = step % n_windows;
    *begin = w * slice_elems;
    *count = numel - *begin < slice_elems ? numel - *begin : slice_elems;
    return SCOUT_OK;
}

}  // extern "C"
