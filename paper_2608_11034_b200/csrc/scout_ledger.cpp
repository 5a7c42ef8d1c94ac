// Host-only part of the library: the checkpoint ledger of Sec. 8 (Algorithm 3)
// and peer-group formation of Sec. 4.  No CUDA here.
#include <new>

#include "scout_ledger.h"

struct scout_ledger {
    uint64_t latest = SCOUT_NO_CHECKPOINT, candidate = SCOUT_NO_CHECKPOINT,
             verified = SCOUT_NO_CHECKPOINT;
    uint32_t q = 0, K = 1;
    uint64_t n_persisted = 0;
};

namespace {

// CheckpointRetrieval: which role answers failure class f.
int choose(const scout_ledger *l, int f, int accessible, int sweep, scout_ledger_event_t *ev) {
    ev->action = SCOUT_LEDGER_RETRIEVAL;
    ev->promoted = SCOUT_NO_CHECKPOINT;
    bool use_verified;
    if (f == SCOUT_OUTCOME_SDC || !accessible) {
        use_verified = true;
    } else if (f == SCOUT_OUTCOME_STRAGGLER) {
        use_verified = false;
    } else if (sweep < 0) {  // the full-catalog replay has to run before a choice is possible
        ev->action = SCOUT_LEDGER_NEED_SWEEP;
        ev->role = SCOUT_ROLE_NONE;
        ev->checkpoint = SCOUT_NO_CHECKPOINT;
        return SCOUT_OK;
    } else {
        use_verified = sweep != 0;
    }
    ev->role = use_verified ? SCOUT_ROLE_VERIFIED : SCOUT_ROLE_LATEST;
    ev->checkpoint = use_verified ? l->verified : l->latest;
    return SCOUT_OK;
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
    l->K = K;
    *out = l;
    return SCOUT_OK;
}

int scout_ledger_destroy(scout_ledger_t *l) {
    delete l;
    return SCOUT_OK;
}

int scout_ledger_state(const scout_ledger_t *l, scout_ledger_state_t *s) {
    if (!l || !s) return SCOUT_ERR_INVALID;
    s->latest = l->latest;
    s->candidate = l->candidate;
    s->verified = l->verified;
    s->q = l->q;
    s->K = l->K;
    s->n_persisted = l->n_persisted;
    return SCOUT_OK;
}

int scout_ledger_save(scout_ledger_t *l, int f, uint64_t captured, int accessible, int sweep,
                      scout_ledger_event_t *ev) {
    if (!l || !ev || !valid_outcome(f)) return SCOUT_ERR_INVALID;
    if (f == SCOUT_OUTCOME_SDC || f == SCOUT_OUTCOME_HANG) return choose(l, f, accessible, sweep, ev);
    if (captured == SCOUT_NO_CHECKPOINT) return SCOUT_ERR_INVALID;
    l->latest = captured;
    l->q += 1;
    ev->action = SCOUT_LEDGER_CAPTURED;
    ev->role = SCOUT_ROLE_NONE;
    ev->checkpoint = SCOUT_NO_CHECKPOINT;
    ev->promoted = SCOUT_NO_CHECKPOINT;
    if (l->q == l->K) {
        l->q = 0;
        l->verified = l->candidate;
        l->candidate = l->latest;  // persisted by the caller
        l->n_persisted += 1;
        ev->action = SCOUT_LEDGER_BOUNDARY;
        ev->checkpoint = l->candidate;
        ev->promoted = l->verified;
    }
    return SCOUT_OK;
}

int scout_ledger_retrieve(const scout_ledger_t *l, int f, int accessible, int sweep,
                          scout_ledger_event_t *ev) {
    if (!l || !ev || !valid_outcome(f) || f == SCOUT_OUTCOME_HEALTHY) return SCOUT_ERR_INVALID;
    return choose(l, f, accessible, sweep, ev);
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
