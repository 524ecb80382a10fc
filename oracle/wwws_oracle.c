/*
 * CPU oracle for the batched WWW.Serve network step.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded restatement of what one step of the simulated
 * decentralized network computes: gossip peer synchronization, Proof-of-Stake
 * request dispatch, duel-and-judge and credit settlement.  It exists to check
 * the CUDA library and to be timed beside it as a CPU baseline; nothing in the
 * product may call it.  It shares no code with the CUDA path and keeps its own
 * data layout (an array of peer structs per replica).
 *
 * The method is a randomized protocol, not a shortcut to a closed form, so the
 * oracle takes the protocol's steps one at a time in the order the paper gives
 * them.  Each function names the passage it follows.  Where the paper is
 * silent the reading taken is stated next to the code.
 *
 * Pins (tests that tie this file to something other than itself):
 *   philox4x32_10      published known-answer vectors of the generator
 *   merge / gossip     semilattice laws, monotone versions, convergence to the
 *                      column-wise maximum, detection of departed peers, partner
 *                      choice uniform and independent across slots
 *   dispatch           candidate block follows the rank distribution,
 *                      first-pick frequency = s_i / sum s_j (Assumption 3),
 *                      interval check with big integers, Plackett-Luce order
 *                      probabilities by enumeration, stake 1:2:3:4 scenario
 *   duel-and-judge     closed-form win probabilities, Q_i of Assumption 3,
 *                      extra-request count identity N*alpha*p_d*(1+k)
 *   settlement         exact conservation of total credit, Lemma 1 mean payoff
 *   create             initial views: staleness recomputed from a second Philox written in
 *                      the test (itself checked against the published vectors), uniform on
 *                      0..init_stale_max by chi-square, diagonal current; offline bit,
 *                      advertised capacity (saturation included) and queue field against the
 *                      inputs; initial ledger and stake (tests/test_oracle_create.py)
 *   advance_time,      the queue model is a reading (the paper gives no formula); its
 *   latency/SLO (S4)   arithmetic is pinned to Lindley's recursion for the unfinished work
 *                      of a first-come-first-served server with batch arrivals, on random
 *                      job sizes and gaps; the priority window (half rate while active) is
 *                      recomputed peer by peer and window by window from the second Philox,
 *                      plus hand cases and the active-window frequency
 *
 *   all of the above   tests/test_oracle_mutations.py plants some fifty single mistakes (a dropped
 *                      term, a wrong sign or constant, an off-by-one, swapped operands) in copies of
 *                      this file and requires the pins to fail on each; the three that survived its
 *                      first run (advertised queue units, judges must be online, hop latency) got
 *                      pins of their own
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -shared -fPIC
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define OFFBIT (1ULL << 39)
#define WIN 32

enum { ST_ORIGIN = 1, ST_DRAW = 2, ST_PROBE = 3, ST_JUDGE = 4, ST_GOSSIP = 5, ST_CHURN = 6, ST_PRIO = 7, ST_INIT = 8 };

/* ---------- C0. Counter-based randomness: Philox4x32, 10 rounds (Salmon et al., SC'11) ---------- */

void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

typedef struct { uint32_t w[4]; } rnd4;

/* key = seed; counter = (index, slot, global replica, stage + 256*sub) */
static rnd4 draw(uint64_t seed, uint32_t index, uint32_t slot, uint32_t replica, uint32_t stage, uint32_t sub)
{
    uint32_t ctr[4] = { index, slot, replica, stage + 256u * sub };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    rnd4 r;
    orc_philox4x32_10(ctr, key, r.w);
    return r;
}

/* x uniform on [0,2^32) -> parts per million, -> integer below n, 64-bit x -> integer below S */
uint32_t orc_ppm(uint32_t x) { return (uint32_t)(((uint64_t)x * 1000000u) >> 32); }
uint32_t orc_below(uint32_t x, uint32_t n) { return (uint32_t)(((uint64_t)x * n) >> 32); }
uint64_t orc_mulhi64(uint64_t x, uint64_t s) { return (uint64_t)(((unsigned __int128)x * s) >> 64); }

/* ---------- C1. State ---------- */

typedef struct {
    uint32_t n_peers, n_replicas, replica_offset, pad0;
    uint64_t seed;
    uint32_t fanout_k, gossip_tries, max_probes, n_judges;
    uint32_t p_duel_ppm, p_noise_ppm, p_leave_ppm, p_join_ppm, p_prio_active_ppm;
    uint32_t prio_window_ms, util_window_ms, cap_ref_tok_s, slo_num, slo_den, hop_ms;
    uint32_t init_stale_max, flags, n_rank;
    int64_t reward_R, reward_add, penalty_P;
    const uint32_t *rank_cdf;
} orc_config;

typedef struct {
    const uint32_t *cap_true_tok_s, *quality_fx;
    const int64_t *credit0;
    const uint16_t *stake_pm, *offload_util_pm, *accept_util_pm;
    const uint32_t *offload_ppm, *accept_ppm;
    const uint8_t *misreport_mul, *prio_flag, *online0;
} orc_peer_init;

typedef struct {
    /* hidden */
    uint32_t cap_true, quality_fx; uint8_t misreport_mul, prio_flag;
    /* policy */
    uint16_t stake_pm, offload_util_pm, accept_util_pm; uint32_t offload_ppm, accept_ppm;
    /* dynamic */
    uint8_t online; uint32_t cap_eff; int64_t backlog; uint32_t ver;
    /* finalized ledger */
    int64_t credit, stake; uint32_t wins, duels; uint64_t served, served_local;
    /* pending (current block) */
    int64_t d_credit; uint32_t d_wins, d_duels;
    /* backlog added by the batch being settled */
    int64_t d_backlog;
    /* credits spent since the last finalization: in earlier batches of the block, in this batch so far */
    int64_t blk_spent, d_spent;
} peer_t;

enum { S_REQUESTS, S_LOCAL, S_FALLBACK, S_DROPPED, S_FAILED, S_DELEGATED, S_DUEL, S_DUEL_CANCELLED, S_DRAW,
       S_JUDGE_EVALS, S_PROBES, S_NEAR, S_SLO_MET, S_SUM_LAT, S_OFFLINE_MARKS, S_ROUNDS, S_BLOCKS, S_CREDIT_TOTAL,
       S_CHAIN_HEAD, S_PENDING_DIGEST, S_UNCOVERED, S_BLOCKS_REJECTED, S_N };

typedef struct {
    uint32_t inplay;       /* lanes still in play after the draws so far */
    uint32_t blk;
    uint8_t n_draws, n_probes, has_window;
} cont_t;

typedef struct {
    orc_config cfg;
    uint32_t *rank_cdf;
    uint32_t N, Rp;
    peer_t *peers;                 /* [Rp][N] */
    uint64_t *view, *view_new;     /* [Rp][N][N], row = observer, column = subject */
    uint32_t t_last_ms, round;
    int64_t *credit_total0;        /* [Rp] */
    uint64_t *stats;               /* [Rp][S_N] */
    /* requests (borrowed) and results (owned) */
    const uint32_t *origin, *t_ms; const uint16_t *len_in, *len_out; uint64_t Q;
    int32_t *exec_a, *exec_b, *judges; uint8_t *outcome, *flags; float *score_a, *score_sum;
    cont_t *cont;
    uint64_t batch_first, batch_count;
    int phase;                     /* 0 idle, 1 dispatched, 2 judged */
    int error;                     /* 0 ok, 4 range, 6 invariant */
} orc_net;

static uint64_t pack_entry(uint32_t ver, int offline, uint64_t adv_cap, uint64_t adv_q)
{
    if (adv_cap > (1u << 19) - 1) adv_cap = (1u << 19) - 1;
    if (adv_q > (1u << 20) - 1) adv_q = (1u << 20) - 1;
    return ((uint64_t)ver << 40) | (offline ? OFFBIT : 0) | (adv_cap << 20) | adv_q;
}

/* "keep the newer entry by version": only the owner issues a (version, payload)
 * pair and others can only raise the offline bit, so the newer of two entries
 * is the larger 64-bit value, offline winning at equal version. */
uint64_t orc_merge(uint64_t a, uint64_t b) { return a > b ? a : b; }

/* utilisation in per-mille: backlog as a fraction of util_window_ms of work at the current rate */
static uint32_t util_pm(const orc_net *n, const peer_t *p)
{
    if (p->cap_eff == 0) return 1000;
    uint64_t denom = (uint64_t)p->cap_eff * n->cfg.util_window_ms / 1000;
    if (denom < 1) denom = 1;
    uint64_t u = (uint64_t)p->backlog * 1000 / denom;
    return u > 1000 ? 1000 : (uint32_t)u;
}

static uint32_t cap_eff_at(const orc_net *n, const peer_t *p, uint32_t j, uint32_t rg, uint32_t now_ms)
{
    uint32_t w = now_ms / n->cfg.prio_window_ms;
    int active = p->prio_flag && orc_ppm(draw(n->cfg.seed, j, w, rg, ST_PRIO, 0).w[0]) < n->cfg.p_prio_active_ppm;
    return active ? p->cap_true / 2 : p->cap_true;
}

static uint64_t adv_cap_of(const peer_t *p) { return (uint64_t)p->cap_eff * p->misreport_mul; }

/* Credit Block Chain (Table "Structure of a Credit Block"): a block holds a list of credit
 * operations, its own id and its parent's id.  Here a block's operations are summarised by an
 * order-independent 64-bit digest (the wrapping sum of one hash per ledger record), and the block
 * id chains that digest to the parent id.  The mixer is the SplitMix64 finaliser (Steele, Lea,
 * Flood 2014); it stands in for the cryptographic hash, signatures are out of scope. */
#define GAMMA 0x9E3779B97F4A7C15ULL
uint64_t orc_mix64(uint64_t z)
{
    z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ULL;
    z ^= z >> 27; z *= 0x94D049BB133111EBULL;
    z ^= z >> 31;
    return z;
}
static uint64_t chain_key(const orc_net *n, uint32_t r) { return n->cfg.seed ^ ((uint64_t)(r + n->cfg.replica_offset) * GAMMA); }

/* one ledger record: request q moves `amount` credits on `peer`'s account; kind says why */
enum { OP_PAY = 1, OP_EARN = 2, OP_PAY_CHALLENGER = 3, OP_EARN_CHALLENGER = 4, OP_PENALTY = 5, OP_REWARD = 6, OP_JUDGE = 7 };
static void post(orc_net *n, uint32_t r, uint32_t q, uint32_t kind, uint32_t peer, int64_t amount)
{
    n->peers[(size_t)r * n->N + peer].d_credit += amount;
    uint64_t word = ((uint64_t)q << 32) | ((uint64_t)kind << 24) | peer;
    n->stats[(size_t)r * S_N + S_PENDING_DIGEST] += orc_mix64(orc_mix64(chain_key(n, r) ^ word) + (uint64_t)amount);
}

/* S5 finalize = commit of a credit block (Section "Credit-based Transaction System"):
 * pending operations are folded into the ledger, stake is re-derived, total credit is checked. */
static void finalize_replica(orc_net *n, uint32_t r)
{
    int64_t total = 0;
    for (uint32_t j = 0; j < n->N; ++j) {
        peer_t *p = &n->peers[(size_t)r * n->N + j];
        p->credit += p->d_credit; p->wins += p->d_wins; p->duels += p->d_duels;
        p->d_credit = 0; p->d_wins = 0; p->d_duels = 0;
        int64_t pos = p->credit > 0 ? p->credit : 0;
        p->stake = pos * p->stake_pm / 1000;
        total += p->credit;
    }
    uint64_t *st = &n->stats[(size_t)r * S_N];
    st[S_BLOCKS] += 1;
    st[S_CHAIN_HEAD] = orc_mix64(orc_mix64(st[S_CHAIN_HEAD] ^ chain_key(n, r)) + st[S_PENDING_DIGEST] + GAMMA * st[S_BLOCKS]);
    st[S_PENDING_DIGEST] = 0;
    if (total != n->credit_total0[r]) n->error = 6;
}

/* ---------- C2. Create ---------- */

orc_net *orc_create(const orc_config *cfg, const orc_peer_init *in)
{
    orc_net *n = (orc_net *)calloc(1, sizeof(orc_net));
    n->cfg = *cfg;
    n->N = cfg->n_peers; n->Rp = cfg->n_replicas;
    if (cfg->rank_cdf && cfg->n_rank) {
        n->rank_cdf = (uint32_t *)malloc(sizeof(uint32_t) * cfg->n_rank);
        memcpy(n->rank_cdf, cfg->rank_cdf, sizeof(uint32_t) * cfg->n_rank);
    }
    n->cfg.rank_cdf = n->rank_cdf;
    size_t NP = (size_t)n->Rp * n->N;
    n->peers = (peer_t *)calloc(NP, sizeof(peer_t));
    n->view = (uint64_t *)calloc(NP * n->N, sizeof(uint64_t));
    n->view_new = (uint64_t *)calloc(NP * n->N, sizeof(uint64_t));
    n->stats = (uint64_t *)calloc((size_t)n->Rp * S_N, sizeof(uint64_t));
    n->credit_total0 = (int64_t *)calloc(n->Rp, sizeof(int64_t));
    for (uint32_t r = 0; r < n->Rp; ++r) {
        uint32_t rg = r + cfg->replica_offset;
        for (uint32_t j = 0; j < n->N; ++j) {
            size_t x = (size_t)r * n->N + j;
            peer_t *p = &n->peers[x];
            p->cap_true = in->cap_true_tok_s[x]; p->quality_fx = in->quality_fx[x];
            p->misreport_mul = in->misreport_mul[x]; p->prio_flag = in->prio_flag[x];
            p->stake_pm = in->stake_pm[x]; p->offload_util_pm = in->offload_util_pm[x];
            p->accept_util_pm = in->accept_util_pm[x];
            p->offload_ppm = in->offload_ppm[x]; p->accept_ppm = in->accept_ppm[x];
            p->online = in->online0[x] ? 1 : 0;
            p->ver = cfg->init_stale_max + 1;
            p->cap_eff = cap_eff_at(n, p, j, rg, 0);
            p->backlog = 0;
            p->credit = 0; p->d_credit = in->credit0[x];
            n->credit_total0[r] += in->credit0[x];
        }
        finalize_replica(n, r);
        n->stats[(size_t)r * S_N + S_BLOCKS] = 0;
        n->stats[(size_t)r * S_N + S_CHAIN_HEAD] = orc_mix64(chain_key(n, r));      /* genesis id */
        /* every node starts knowing every peer, possibly by a version a few rounds old */
        for (uint32_t i = 0; i < n->N; ++i)
            for (uint32_t j = 0; j < n->N; ++j) {
                const peer_t *p = &n->peers[(size_t)r * n->N + j];
                uint32_t stale = (i == j) ? 0 : orc_below(draw(cfg->seed, i, j, rg, ST_INIT, 0).w[0], cfg->init_stale_max + 1);
                n->view[((size_t)r * n->N + i) * n->N + j] = pack_entry(p->ver - stale, !p->online, adv_cap_of(p), 0);
            }
    }
    return n;
}

void orc_destroy(orc_net *n)
{
    if (!n) return;
    free(n->rank_cdf); free(n->peers); free(n->view); free(n->view_new); free(n->stats); free(n->credit_total0);
    free(n->exec_a); free(n->exec_b); free(n->judges); free(n->outcome); free(n->flags);
    free(n->score_a); free(n->score_sum); free(n->cont);
    free(n);
}

void orc_bind_requests(orc_net *n, const uint32_t *origin, const uint32_t *t_ms, const uint16_t *len_in,
                       const uint16_t *len_out, uint64_t n_requests)
{
    n->origin = origin; n->t_ms = t_ms; n->len_in = len_in; n->len_out = len_out; n->Q = n_requests;
    size_t T = (size_t)n->Rp * n_requests;
    free(n->exec_a); free(n->exec_b); free(n->judges); free(n->outcome); free(n->flags);
    free(n->score_a); free(n->score_sum); free(n->cont);
    n->exec_a = (int32_t *)malloc(T * 4); n->exec_b = (int32_t *)malloc(T * 4); n->judges = (int32_t *)malloc(T * 16);
    memset(n->exec_a, 0xFF, T * 4); memset(n->exec_b, 0xFF, T * 4); memset(n->judges, 0xFF, T * 16);
    n->outcome = (uint8_t *)calloc(T, 1); n->flags = (uint8_t *)calloc(T, 1);
    n->score_a = (float *)calloc(T, 4); n->score_sum = (float *)calloc(T, 4);
    n->cont = (cont_t *)calloc(T, sizeof(cont_t));
    n->phase = 0;
}

/* ---------- C3. Advance simulated time (providers drain their queues; prioritized local load) ---------- */

void orc_advance_time(orc_net *n, uint32_t now_ms)
{
    uint32_t dt = now_ms - n->t_last_ms;
    for (uint32_t r = 0; r < n->Rp; ++r)
        for (uint32_t j = 0; j < n->N; ++j) {
            peer_t *p = &n->peers[(size_t)r * n->N + j];
            if (p->online) {
                int64_t done = (int64_t)((uint64_t)p->cap_eff * dt / 1000);
                p->backlog = p->backlog > done ? p->backlog - done : 0;
            }
            p->cap_eff = cap_eff_at(n, p, j, r + n->cfg.replica_offset, now_ms);
        }
    n->t_last_ms = now_ms;
}

/* ---------- C4. Gossip round (Appendix "Gossip-Driven Peer Synchronization") ---------- */

void orc_gossip_round(orc_net *n)
{
    const orc_config *c = &n->cfg;
    uint32_t N = n->N, t = n->round;
    uint64_t *self = (uint64_t *)malloc(sizeof(uint64_t) * N);
    for (uint32_t r = 0; r < n->Rp; ++r) {
        uint32_t rg = r + c->replica_offset;
        peer_t *P = &n->peers[(size_t)r * N];
        uint64_t *V = &n->view[(size_t)r * N * N], *Vn = &n->view_new[(size_t)r * N * N];
        uint64_t *st = &n->stats[(size_t)r * S_N];
        /* G0: peers leave (crash, queue lost) and join */
        for (uint32_t j = 0; j < N; ++j) {
            uint32_t x = orc_ppm(draw(c->seed, j, t, rg, ST_CHURN, 0).w[0]);
            if (P[j].online) { if (x < c->p_leave_ppm) { P[j].online = 0; P[j].backlog = 0; } }
            else if (x < c->p_join_ppm) P[j].online = 1;
        }
        /* G1: every online peer issues a new version of its own entry */
        for (uint32_t j = 0; j < N; ++j) {
            self[j] = 0;
            if (!P[j].online) continue;
            P[j].ver += 1;
            if (P[j].ver >= (1u << 24)) { n->error = 4; P[j].ver = (1u << 24) - 1; }
            self[j] = pack_entry(P[j].ver, 0, adv_cap_of(&P[j]), (uint64_t)P[j].backlog >> 4);
        }
        /* G2: pull the views of k partners believed online and reconcile entry by entry */
        memcpy(Vn, V, sizeof(uint64_t) * N * N);
        for (uint32_t i = 0; i < N; ++i) {
            if (!P[i].online) continue;
            uint64_t *row = &Vn[(size_t)i * N];
            row[i] = orc_merge(row[i], self[i]);
            for (uint32_t s = 0; s < c->fanout_k; ++s) {
                int64_t partner = -1;
                for (uint32_t a = 0; a < c->gossip_tries && partner < 0; ++a) {
                    uint32_t p = orc_below(draw(c->seed, i, t, rg, ST_GOSSIP, a).w[s], N);
                    uint64_t e = V[(size_t)i * N + p];
                    if (p != i && e != 0 && !(e & OFFBIT)) partner = p;
                }
                if (partner < 0) continue;
                uint32_t p = (uint32_t)partner;
                if (!P[p].online) {                      /* the pull fails: departure detected */
                    row[p] = orc_merge(row[p], V[(size_t)i * N + p] | OFFBIT);
                    st[S_OFFLINE_MARKS] += 1;
                } else {
                    const uint64_t *prow = &V[(size_t)p * N];
                    for (uint32_t col = 0; col < N; ++col) row[col] = orc_merge(row[col], prow[col]);
                    /* the pull itself tells the partner about the puller */
                    Vn[(size_t)p * N + i] = orc_merge(Vn[(size_t)p * N + i], self[i]);
                    /* full pairwise exchange (flag 8): the partner also reconciles with the puller's view */
                    if (c->flags & 8) {
                        const uint64_t *irow = &V[(size_t)i * N];
                        uint64_t *pnew = &Vn[(size_t)p * N];
                        for (uint32_t col = 0; col < N; ++col) pnew[col] = orc_merge(pnew[col], irow[col]);
                    }
                }
            }
        }
        st[S_ROUNDS] += 1;
    }
    free(self);
    uint64_t *tmp = n->view; n->view = n->view_new; n->view_new = tmp;   /* G3 */
    n->round += 1;
}

/* ---------- C5. Dispatch (Section "Request Routing and Node Design"; Assumption 3) ---------- */

typedef struct { uint64_t W[WIN]; float score[WIN]; } window_t;

/* D3: which 32-peer block of the id ring the origin samples from */
static uint32_t pick_block(const orc_net *n, uint32_t o, uint32_t w2)
{
    uint32_t n_blk = (n->N + WIN - 1) / WIN, rank;
    if (n->rank_cdf) {
        rank = 0;
        while (rank < n->cfg.n_rank && !(w2 < n->rank_cdf[rank])) ++rank;
        if (rank > n_blk - 1) rank = n_blk - 1;
    } else rank = orc_below(w2, n_blk);
    return (o / WIN + rank) % n_blk;
}

/* D4: fp32 score and integer weight of each candidate, from the origin's view and the shared ledger */
static void score_window(const orc_net *n, uint32_t r, uint32_t o, uint32_t blk, window_t *w)
{
    const peer_t *P = &n->peers[(size_t)r * n->N];
    const uint64_t *row = &n->view[((size_t)r * n->N + o) * n->N];
    float uwf = (float)n->cfg.util_window_ms / 1000.0f;
    for (uint32_t c = 0; c < WIN; ++c) {
        w->W[c] = 0; w->score[c] = 0.0f;
        uint32_t id = WIN * blk + c;
        if (id >= n->N || id == o) continue;
        uint64_t e = row[id];
        if (e == 0 || (e & OFFBIT)) continue;
        uint32_t advcap = (uint32_t)((e >> 20) & ((1u << 19) - 1)), advq = (uint32_t)(e & ((1u << 20) - 1));
        if (P[id].stake <= 0 || advcap == 0) continue;
        float sf = (float)P[id].stake;
        float rep = 1.0f;
        if (n->cfg.flags & 1) { float a = (float)(P[id].wins + 1), b = (float)(P[id].duels + 2); rep = a / b; }
        float spare = 1.0f;
        if (n->cfg.flags & 2) {
            float num = (float)(advq * 16u);
            float den = (float)advcap * uwf;
            float utilf = num / den;
            spare = 1.0f - utilf;
            if (!(spare > 0.0f)) spare = 0.0f;
        }
        float s1 = sf * rep;
        float score = s1 * spare;
        float scaled = score * 256.0f;
        uint64_t W = scaled >= 72057594037927936.0f ? (1ULL << 56) : (uint64_t)scaled;
        w->W[c] = W;
        w->score[c] = W ? score : 0.0f;
    }
}

void orc_window_weights(const orc_net *n, uint32_t r, uint64_t q, uint64_t *W_out, float *score_out, uint32_t *blk_out)
{
    uint32_t o = n->origin[(size_t)r * n->Q + q];
    rnd4 x = draw(n->cfg.seed, (uint32_t)q, 0, r + n->cfg.replica_offset, ST_ORIGIN, 0);
    uint32_t blk = pick_block(n, o, x.w[2]);
    window_t w; score_window(n, r, o, blk, &w);
    memcpy(W_out, w.W, sizeof w.W); memcpy(score_out, w.score, sizeof w.score); *blk_out = blk;
}

typedef struct { int lane; int near; } pick_t;

/* D5: one PoS draw among the lanes in play, by integer prefix sums.  lane = -1 when nothing is left. */
static pick_t pos_draw(const orc_net *n, uint32_t rg, uint32_t q, const window_t *w, cont_t *ct)
{
    pick_t out = { -1, 0 };
    uint64_t S = 0;
    for (int c = 0; c < WIN; ++c) if (ct->inplay >> c & 1) S += w->W[c];
    if (S == 0) return out;
    uint32_t d = ct->n_draws++;
    if (n->cfg.flags & 4) {
        /* greedy rule (a customised load-balancing rule of the Policy Manager): the highest
         * weight wins, the lowest lane on ties; flagged when the runner-up is within 1e-5 */
        int best = -1, second = -1;
        for (int c = 0; c < WIN; ++c) {
            if (!(ct->inplay >> c & 1) || w->W[c] == 0) continue;
            if (best < 0 || w->W[c] > w->W[best]) { second = best; best = c; }
            else if (second < 0 || w->W[c] > w->W[second]) second = c;
        }
        out.lane = best;
        out.near = second >= 0 && w->W[best] - w->W[second] <= w->W[best] / 100000;
        ct->inplay &= ~(1u << best);
        return out;
    }
    rnd4 y = draw(n->cfg.seed, q, d / 2, rg, ST_DRAW, 0);
    uint64_t u = ((uint64_t)y.w[2 * (d % 2)] << 32) | y.w[2 * (d % 2) + 1];
    uint64_t r64 = orc_mulhi64(u, S), acc = 0;
    for (int c = 0; c < WIN; ++c) {
        if (!(ct->inplay >> c & 1) || w->W[c] == 0) continue;
        uint64_t lo = acc; acc += w->W[c];
        if (acc > r64) {
            uint64_t m1 = r64 - lo, m2 = acc - 1 - r64, m = m1 < m2 ? m1 : m2;
            out.lane = c; out.near = m <= S / 100000;
            ct->inplay &= ~(1u << c);
            return out;
        }
    }
    return out; /* unreachable: r64 < S */
}

/* D6: the drawn candidate answers by its own policy and its true state */
static int probe(const orc_net *n, uint32_t rg, uint32_t q, const peer_t *p, int lane)
{
    if (!p->online || p->cap_eff == 0) return 0;
    if (!(util_pm(n, p) < p->accept_util_pm)) return 0;
    return orc_ppm(draw(n->cfg.seed, q, (uint32_t)lane / 4, rg, ST_PROBE, 0).w[lane % 4]) < p->accept_ppm;
}

/* draw-and-probe until a candidate accepts, the probe budget is spent or nobody is left */
static int find_executor(orc_net *n, uint32_t r, uint32_t q, const window_t *w, cont_t *ct, uint8_t *flag)
{
    uint32_t rg = r + n->cfg.replica_offset;
    const peer_t *P = &n->peers[(size_t)r * n->N];
    while (ct->n_probes < n->cfg.max_probes) {
        pick_t pk = pos_draw(n, rg, q, w, ct);
        if (pk.lane < 0) break;
        if (pk.near) *flag |= 1;
        ct->n_probes++;
        n->stats[(size_t)r * S_N + S_PROBES] += 1;
        uint32_t id = WIN * ct->blk + pk.lane;
        if (probe(n, rg, q, &P[id], pk.lane)) return (int)id;
    }
    return -1;
}

int orc_dispatch_batch(orc_net *n, uint64_t first, uint64_t count)
{
    if (!n->origin || first + count > n->Q || n->phase != 0) return 3;
    const orc_config *c = &n->cfg;
    for (uint32_t r = 0; r < n->Rp; ++r) {
        uint32_t rg = r + c->replica_offset;
        const peer_t *P = &n->peers[(size_t)r * n->N];
        for (uint64_t q = first; q < first + count; ++q) {
            size_t x = (size_t)r * n->Q + q;
            uint32_t o = n->origin[x];
            cont_t *ct = &n->cont[x];
            memset(ct, 0, sizeof *ct);
            n->exec_b[x] = -1; n->outcome[x] = 0; n->flags[x] = 0; n->score_a[x] = 0.0f; n->score_sum[x] = 0.0f;
            for (int k = 0; k < 4; ++k) n->judges[4 * x + k] = -1;
            if (o >= n->N || !P[o].online) { n->exec_a[x] = -3; continue; }        /* D1 */
            rnd4 rx = draw(c->seed, (uint32_t)q, 0, rg, ST_ORIGIN, 0);
            int offload = util_pm(n, &P[o]) >= P[o].offload_util_pm                   /* D2 */
                          && orc_ppm(rx.w[0]) < P[o].offload_ppm && P[o].credit >= c->reward_R;
            int local_code = P[o].cap_eff == 0 ? -4 : -1;
            if (!offload) { n->exec_a[x] = local_code; continue; }
            ct->blk = pick_block(n, o, rx.w[2]);                                    /* D3 */
            window_t w; score_window(n, r, o, ct->blk, &w);                         /* D4 */
            ct->has_window = 1; ct->inplay = 0;
            float sum = 0.0f;
            for (int l = 0; l < WIN; ++l) { if (w.W[l]) ct->inplay |= 1u << l; sum = sum + w.score[l]; }
            n->score_sum[x] = sum;
            int a = find_executor(n, r, (uint32_t)q, &w, ct, &n->flags[x]);        /* D5, D6 */
            if (a >= 0) { n->exec_a[x] = a; n->score_a[x] = w.score[a - (int)(WIN * ct->blk)]; }
            else n->exec_a[x] = P[o].cap_eff == 0 ? -4 : -2;
        }
    }
    n->batch_first = first; n->batch_count = count; n->phase = 1;
    return 0;
}

/* ---------- C6. Duel-and-judge (Section "Duel-and-Judge Mechanism"; Assumption 3) ---------- */

int orc_duel_judge(orc_net *n)
{
    if (n->phase != 1) return 3;
    const orc_config *c = &n->cfg;
    for (uint32_t r = 0; r < n->Rp; ++r) {
        uint32_t rg = r + c->replica_offset;
        const peer_t *P = &n->peers[(size_t)r * n->N];
        for (uint64_t q = n->batch_first; q < n->batch_first + n->batch_count; ++q) {
            size_t x = (size_t)r * n->Q + q;
            if (n->exec_a[x] < 0) continue;
            rnd4 rx = draw(c->seed, (uint32_t)q, 0, rg, ST_ORIGIN, 0);
            if (!(orc_ppm(rx.w[1]) < c->p_duel_ppm)) continue;                       /* J1 */
            cont_t *ct = &n->cont[x];
            window_t w; score_window(n, r, n->origin[x], ct->blk, &w);
            n->outcome[x] = 4;
            int b = find_executor(n, r, (uint32_t)q, &w, ct, &n->flags[x]);        /* J2: challenger */
            if (b < 0) continue;
            int nj = 0, jd[4];
            while (nj < (int)c->n_judges) {                                          /* J2: judges */
                pick_t pk = pos_draw(n, rg, (uint32_t)q, &w, ct);
                if (pk.lane < 0) break;
                if (pk.near) n->flags[x] |= 1;
                uint32_t id = WIN * ct->blk + pk.lane;
                if (P[id].online) jd[nj++] = (int)id;
            }
            if (nj == 0) continue;
            int a = n->exec_a[x], votes_a = 0;
            uint64_t thr = ((1ULL << 32) + P[a].quality_fx - P[b].quality_fx) >> 1;  /* J3 */
            for (int l = 0; l < nj; ++l) {
                rnd4 y = draw(c->seed, (uint32_t)q, (uint32_t)l, rg, ST_JUDGE, 0);
                int vote_a = (uint64_t)y.w[0] < thr;
                if (orc_ppm(y.w[1]) < c->p_noise_ppm) vote_a = !vote_a;
                votes_a += vote_a;
            }
            n->exec_b[x] = b;
            for (int l = 0; l < nj; ++l) n->judges[4 * x + l] = jd[l];
            n->outcome[x] = 2 * votes_a > nj ? 1 : (2 * votes_a < nj ? 2 : 3);
        }
    }
    n->phase = 2;
    return 0;
}

/* ---------- C8. Credit settlement (Section "Credit-based Transaction System"; Lemma 1) ---------- */

static uint64_t ceil_div(uint64_t a, uint64_t b) { return (a + b - 1) / b; }

int orc_settle_credits(orc_net *n, int finalize)
{
    if (n->phase != 2) return 3;
    const orc_config *c = &n->cfg;
    for (uint32_t r = 0; r < n->Rp; ++r) {
        peer_t *P = &n->peers[(size_t)r * n->N];
        uint64_t *st = &n->stats[(size_t)r * S_N];
        for (uint64_t q = n->batch_first; q < n->batch_first + n->batch_count; ++q) {
            size_t x = (size_t)r * n->Q + q;
            uint32_t o = n->origin[x];
            uint64_t li = n->len_in[x], lo = n->len_out[x], work = li + lo;
            int a = n->exec_a[x];
            st[S_REQUESTS] += 1;
            if (n->flags[x] & 1) st[S_NEAR] += 1;
            if (a == -3) { st[S_DROPPED] += 1; continue; }
            if (a == -4) { st[S_FAILED] += 1; continue; }
            uint32_t ex;
            /* exact intra-batch queueing (flag 16): a request waits behind the work that earlier
             * requests of the same batch put on its executor; otherwise only behind the batch-start queue */
            uint64_t ahead = (c->flags & 16) ? (uint64_t)P[a < 0 ? o : (uint32_t)a].d_backlog : 0;
            if (a < 0) {                                                     /* S1 served at the origin */
                st[a == -1 ? S_LOCAL : S_FALLBACK] += 1;
                P[o].d_backlog += (int64_t)work; P[o].served_local += 1; ex = o;
            } else {                                                         /* S2 credits-for-offloading */
                st[S_DELEGATED] += 1;
                if (c->flags & 16) {
                    /* in-block validation (Section "Credit-based Transaction System": a payer must not spend the
                     * same credits twice): a payment is covered only by the payer's finalized balance minus what it
                     * already spent in this block; earnings of the open block cannot be spent yet */
                    int64_t pay = c->reward_R * ((n->outcome[x] >= 1 && n->outcome[x] <= 3) ? 2 : 1);
                    if (P[o].credit - P[o].blk_spent - P[o].d_spent < pay) st[S_UNCOVERED] += 1;
                    P[o].d_spent += pay;
                }
                post(n, r, (uint32_t)q, OP_PAY, o, -c->reward_R); post(n, r, (uint32_t)q, OP_EARN, (uint32_t)a, c->reward_R);
                P[a].d_backlog += (int64_t)work; P[a].served += 1; ex = (uint32_t)a;
                uint8_t oc = n->outcome[x];
                if (oc != 0) st[S_DUEL] += 1;
                if (oc == 4) st[S_DUEL_CANCELLED] += 1;
                if (oc >= 1 && oc <= 3) {                                    /* S3 duel */
                    int b = n->exec_b[x], nj = 0;
                    post(n, r, (uint32_t)q, OP_PAY_CHALLENGER, o, -c->reward_R); post(n, r, (uint32_t)q, OP_EARN_CHALLENGER, (uint32_t)b, c->reward_R);
                    P[b].d_backlog += (int64_t)work; P[b].served += 1;
                    P[a].d_duels += 1; P[b].d_duels += 1;
                    for (int l = 0; l < 4; ++l) if (n->judges[4 * x + l] >= 0) {
                        P[n->judges[4 * x + l]].d_backlog += (int64_t)(li + 2 * lo); ++nj;
                    }
                    st[S_JUDGE_EVALS] += (uint64_t)nj;
                    if (oc == 3) st[S_DRAW] += 1;
                    else {
                        int win = oc == 1 ? a : b, lose = oc == 1 ? b : a;
                        int64_t pot = c->penalty_P - c->reward_add, share = pot / nj;
                        post(n, r, (uint32_t)q, OP_PENALTY, (uint32_t)lose, -c->penalty_P);
                        post(n, r, (uint32_t)q, OP_REWARD, (uint32_t)win, c->reward_add + (pot - share * nj));
                        P[win].d_wins += 1;
                        for (int l = 0; l < 4; ++l) if (n->judges[4 * x + l] >= 0) post(n, r, (uint32_t)q, OP_JUDGE + (uint32_t)l, (uint32_t)n->judges[4 * x + l], share);
                    }
                }
            }
            /* S4 latency estimate against the queue as it stood when the batch started */
            uint64_t lat = ceil_div(((uint64_t)P[ex].backlog + ahead + work) * 1000, P[ex].cap_eff) + (a >= 0 ? c->hop_ms : 0);
            uint64_t deadline = (uint64_t)c->slo_num * ceil_div(work * 1000, c->cap_ref_tok_s) / c->slo_den;
            st[S_SUM_LAT] += lat;
            if (lat <= deadline) st[S_SLO_MET] += 1;
        }
        /* majority validation (flag 32; Section "Credit-based Transaction System": a block is final once
         * a majority of peers confirm and append it): every online peer validates the proposed block; without
         * a majority the block stays open and its operations ride along with the next proposal */
        int commit = finalize;
        if (commit && (c->flags & 32)) {
            uint32_t online = 0;
            for (uint32_t j = 0; j < n->N; ++j) online += P[j].online;
            if (2 * online <= n->N) { commit = 0; st[S_BLOCKS_REJECTED] += 1; }
        }
        for (uint32_t j = 0; j < n->N; ++j) {
            P[j].backlog += P[j].d_backlog; P[j].d_backlog = 0;
            P[j].blk_spent = commit ? 0 : P[j].blk_spent + P[j].d_spent; P[j].d_spent = 0;
        }
        if (commit) finalize_replica(n, r);
    }
    n->phase = 0;
    return 0;
}

/* ---------- C7. Stats and table access ---------- */

void orc_stats(const orc_net *n, uint64_t *out /* [Rp+1][S_N], last row = totals */)
{
    memset(out, 0, sizeof(uint64_t) * (n->Rp + 1) * S_N);
    for (uint32_t r = 0; r < n->Rp; ++r) {
        memcpy(&out[(size_t)r * S_N], &n->stats[(size_t)r * S_N], sizeof(uint64_t) * S_N);
        int64_t tot = 0;
        for (uint32_t j = 0; j < n->N; ++j) tot += n->peers[(size_t)r * n->N + j].credit + n->peers[(size_t)r * n->N + j].d_credit;
        out[(size_t)r * S_N + S_CREDIT_TOTAL] = (uint64_t)tot;
        for (int k = 0; k < S_N; ++k) out[(size_t)n->Rp * S_N + k] += out[(size_t)r * S_N + k];
    }
}

int orc_error(const orc_net *n) { return n->error; }
uint32_t orc_stats_width(void) { return S_N; }
const uint64_t *orc_view(const orc_net *n) { return n->view; }
const int32_t *orc_exec_a(const orc_net *n) { return n->exec_a; }
const int32_t *orc_exec_b(const orc_net *n) { return n->exec_b; }
const int32_t *orc_judges(const orc_net *n) { return n->judges; }
const uint8_t *orc_outcome(const orc_net *n) { return n->outcome; }
const uint8_t *orc_flags(const orc_net *n) { return n->flags; }
const float *orc_score_a(const orc_net *n) { return n->score_a; }
const float *orc_score_sum(const orc_net *n) { return n->score_sum; }

/* copy one per-peer table, widened to int64, into out[Rp*N] */
enum { T_ONLINE, T_CAP_EFF, T_BACKLOG, T_VER, T_CREDIT, T_STAKE, T_WINS, T_DUELS, T_SERVED, T_SERVED_LOCAL,
       T_D_CREDIT, T_D_WINS, T_D_DUELS, T_BLK_SPENT };
int orc_table(const orc_net *n, int which, int64_t *out)
{
    size_t NP = (size_t)n->Rp * n->N;
    for (size_t x = 0; x < NP; ++x) {
        const peer_t *p = &n->peers[x];
        switch (which) {
        case T_ONLINE: out[x] = p->online; break;
        case T_CAP_EFF: out[x] = p->cap_eff; break;
        case T_BACKLOG: out[x] = p->backlog; break;
        case T_VER: out[x] = p->ver; break;
        case T_CREDIT: out[x] = p->credit; break;
        case T_STAKE: out[x] = p->stake; break;
        case T_WINS: out[x] = p->wins; break;
        case T_DUELS: out[x] = p->duels; break;
        case T_SERVED: out[x] = (int64_t)p->served; break;
        case T_SERVED_LOCAL: out[x] = (int64_t)p->served_local; break;
        case T_D_CREDIT: out[x] = p->d_credit; break;
        case T_D_WINS: out[x] = p->d_wins; break;
        case T_D_DUELS: out[x] = p->d_duels; break;
        case T_BLK_SPENT: out[x] = p->blk_spent; break;
        default: return 1;
        }
    }
    return 0;
}

/* test hooks: overwrite dynamic state of one peer (hand cases) */
void orc_poke_peer(orc_net *n, uint32_t r, uint32_t j, int online, int64_t backlog, int64_t cap_eff)
{
    peer_t *p = &n->peers[(size_t)r * n->N + j];
    if (online >= 0) p->online = (uint8_t)online;
    if (backlog >= 0) p->backlog = backlog;
    if (cap_eff >= 0) p->cap_eff = (uint32_t)cap_eff;
}
void orc_poke_view(orc_net *n, uint32_t r, uint32_t i, uint32_t j, uint64_t entry) { n->view[((size_t)r * n->N + i) * n->N + j] = entry; }
