/*
 * scout_ledger.h - checkpoint ledger and peer-group formation (host-only part of
 * the library; no CUDA call is made by anything declared here).
 *
 * Ledger: the checkpoint protocol of Sec. 8 (Algorithm 3, "Checkpoint saving and
 * retrieval").  Three roles: latest (newest in-memory capture), candidate
 * (persisted, awaiting complete validation), verified (numerical trust supported
 * by replay evidence).  q counts accepted checks of the current cycle; at q = K
 * the previous candidate becomes verified and the latest capture is persisted as
 * the new candidate, so a candidate is promoted only after two consecutive
 * accepted cycles (2K checks).  Checkpoints are caller-chosen 64-bit ids.
 *
 * Peer groups: Sec. 4 ("Forming equivalent peer groups"), logical mesh address
 * r = (d, s, t, p, c, e).
 */
#ifndef SCOUT_LEDGER_H
#define SCOUT_LEDGER_H

#include "scout.h"

#ifdef __cplusplus
extern "C" {
#endif

/* job-wide outcome of a check / failure class */
enum { SCOUT_OUTCOME_HEALTHY = 0, SCOUT_OUTCOME_STRAGGLER = 1, SCOUT_OUTCOME_SDC = 2,
       SCOUT_OUTCOME_HANG = 3, SCOUT_OUTCOME_OTHER = 4 };
enum { SCOUT_ROLE_NONE = 0, SCOUT_ROLE_LATEST = 1, SCOUT_ROLE_CANDIDATE = 2, SCOUT_ROLE_VERIFIED = 3 };
enum { SCOUT_LEDGER_CAPTURED = 0,   /* accepted: latest replaced, q incremented             */
       SCOUT_LEDGER_BOUNDARY = 1,   /* accepted and q reached K: promote + persist           */
       SCOUT_LEDGER_RETRIEVAL = 2,  /* SDC or hang: nothing captured, a checkpoint was chosen */
       SCOUT_LEDGER_NEED_SWEEP = 3  /* retrieval needs the full-catalog replay result first  */ };
#define SCOUT_NO_CHECKPOINT UINT64_MAX

typedef struct scout_ledger scout_ledger_t;

typedef struct {
    uint64_t latest, candidate, verified; /* SCOUT_NO_CHECKPOINT when the role is empty */
    uint32_t q, K;
    uint64_t n_persisted;                 /* cycle boundaries so far */
} scout_ledger_state_t;

typedef struct {
    int32_t action;      /* SCOUT_LEDGER_*                                              */
    int32_t role;        /* retrieval: role of the chosen checkpoint, else SCOUT_ROLE_NONE */
    uint64_t checkpoint; /* retrieval: chosen id; boundary: id persisted as candidate    */
    uint64_t promoted;   /* boundary: id that became verified (may be SCOUT_NO_CHECKPOINT) */
} scout_ledger_event_t;

/* K >= 1: size of the recipe catalog (1 for models with static shapes). */
SCOUT_API int scout_ledger_create(uint32_t K, scout_ledger_t **out);
SCOUT_API int scout_ledger_destroy(scout_ledger_t *ledger);
SCOUT_API int scout_ledger_state(const scout_ledger_t *ledger, scout_ledger_state_t *state /*host*/);

/* CheckpointSave of Algorithm 3, called at every replay boundary.
 *   outcome             job-wide outcome f.  SDC or HANG: nothing is captured and
 *                       the call answers as scout_ledger_retrieve (q and the roles
 *                       are left as they are, as in the listing).  HEALTHY,
 *                       STRAGGLER ("completed straggler") or OTHER: `captured`
 *                       becomes latest and q is incremented; at q = K: q = 0,
 *                       verified = candidate, candidate = latest (persisted).
 *   captured            id of the state captured at this boundary
 *   machines_accessible, sweep_has_sdc   used only on the retrieval path */
SCOUT_API int scout_ledger_save(scout_ledger_t *ledger, int outcome, uint64_t captured,
                                int machines_accessible, int sweep_has_sdc,
                                scout_ledger_event_t *event /*host*/);

/* CheckpointRetrieval of Algorithm 3.  SDC, or a machine that cannot be reached:
 * verified.  STRAGGLER: latest.  Any other failure: the caller replays the full
 * catalog; sweep_has_sdc = 1: verified, 0: latest, -1 (not run yet): the event
 * says SCOUT_LEDGER_NEED_SWEEP and chooses nothing. */
SCOUT_API int scout_ledger_retrieve(const scout_ledger_t *ledger, int failure, int machines_accessible,
                                    int sweep_has_sdc, scout_ledger_event_t *event /*host*/);

/* Outcome of a certify run for the ledger: CERTIFIED -> HEALTHY; ATTRIBUTED or
 * UNDECIDED (replicas disagree) -> SDC. */
SCOUT_API int scout_outcome_from_report(const scout_report_t *report /*host*/, int *outcome);

/* ---- peer groups (Sec. 4) ---------------------------------------------------
 * A mesh is given by its six degrees in the order (d, s, t, p, c, e); absent
 * dimensions have degree 1.  Ranks are placed row-major in that order (e
 * fastest): the paper's example (4,1,2,1,1,1) puts position (d,t) at rank 2d+t. */
typedef struct { uint32_t d, s, t, p, c, e; } scout_mesh_t;
enum { SCOUT_GROUP_NONE = 0, SCOUT_GROUP_REPLICA = 1, SCOUT_GROUP_SHARD = 2 };

SCOUT_API int scout_mesh_size(const scout_mesh_t *shape, uint64_t *n_ranks);
SCOUT_API int scout_mesh_coords(const scout_mesh_t *shape, uint64_t rank, scout_mesh_t *coords);
SCOUT_API int scout_mesh_rank(const scout_mesh_t *shape, const scout_mesh_t *coords, uint64_t *rank);

/* Equivalent peers of `rank`, ascending along the free coordinate (the position
 * in this list is the bit position in C3's bitmap).  Data-replica degree > 1:
 * G_rep (s, t, p, c, e fixed, d free).  Otherwise state-shard degree > 1:
 * G_shard (t, p, c, e fixed, s free).  Otherwise the rank is a singleton:
 * kind = SCOUT_GROUP_NONE, n = 1.  peers: host array of `cap` entries; n gets
 * the group size even if cap is smaller (then SCOUT_ERR_TRUNCATED). */
SCOUT_API int scout_peer_group(const scout_mesh_t *shape, uint64_t rank, uint64_t *peers /*host*/,
                               uint64_t cap, uint64_t *n, int *kind);

/* ---- rotating slice (Sec. 9 "Optimizer boundary") -----------------------------
 * The optimizer-boundary check compares a rotating 64K-element slice of each
 * tensor instead of the whole tensor.  The paper does not say how the slice
 * moves; this library's reading: consecutive windows of `slice_elems` elements,
 * window `step` starting at (step mod n_windows) * slice_elems with
 * n_windows = ceil(numel / slice_elems); the last window is short; after it the
 * rotation starts again at element 0.  Signing a slice = a plan whose tensor is
 * (base + begin * element_size, count * element_size).
 *   begin, count   first element and length of the window for this step */
#define SCOUT_DEFAULT_SLICE_ELEMS 65536u
SCOUT_API int scout_rotating_slice(uint64_t numel, uint64_t slice_elems, uint64_t step,
                                   uint64_t *begin, uint64_t *count);

#ifdef __cplusplus
}
#endif
#endif /* SCOUT_LEDGER_H */
