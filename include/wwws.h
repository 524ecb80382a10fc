/*
 * wwws: batched simulation of the WWW.Serve decentralized LLM-serving network on one GPU.
 *
 * One network = n_replicas independent Monte-Carlo replicas of n_peers providers.  A step
 * of the network runs the paper's four mechanisms over a batch of user requests:
 *   gossip peer synchronization   (Appendix "Gossip-Driven Peer Synchronization")
 *   Proof-of-Stake dispatch       (Section "Request Routing and Node Design", Assumption 3)
 *   duel-and-judge                (Section "Duel-and-Judge Mechanism", Assumption 3)
 *   credit settlement             (Section "Credit-based Transaction System", Lemma 1)
 *
 * Conventions
 *   - Every call returns a wwws_status and never aborts.  wwws_last_error() gives text.
 *   - All device work is enqueued on the CUDA stream given at creation.  Calls are
 *     asynchronous except wwws_stats, wwws_export_*, wwws_import_table, wwws_step_host
 *     and wwws_destroy_network, which synchronise that stream.
 *   - The library allocates no device memory: the caller hands in one workspace of
 *     wwws_workspace_bytes() bytes (256-byte aligned) that must outlive the network.
 *   - "HOST" / "DEVICE" below say where a pointer must point.  Per-peer arrays are
 *     [n_replicas][n_peers]; per-request arrays are [n_replicas][n_requests], row-major.
 *   - Problems found on the device (version overflow, bad origin index, credit not
 *     conserved) set a device error word that the next synchronising call reports;
 *     no kernel traps.
 *   - A handle is not thread-safe.
 *   - A network lives on the GPU that holds its workspace.  Every call makes that GPU current
 *     while it runs and restores the caller's device before it returns.
 *   - All randomness is Philox4x32-10 with key = seed and counter
 *     (index, slot, replica_offset + replica, stage + 256*attempt), so results do not
 *     depend on launch shapes or on how replicas are split over processes.
 */
#ifndef WWWS_H
#define WWWS_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct wwws_network wwws_network; /* opaque */

typedef enum {
    WWWS_OK = 0,
    WWWS_ERR_ARG = 1,       /* null pointer, value out of range, bad origin index */
    WWWS_ERR_ALLOC = 2,     /* workspace too small or misaligned */
    WWWS_ERR_STATE = 3,     /* call order: dispatch -> duel_judge -> settle */
    WWWS_ERR_RANGE = 4,     /* a peer's version counter reached 2^24 */
    WWWS_ERR_CUDA = 5,      /* a CUDA runtime call failed */
    WWWS_ERR_INVARIANT = 6, /* total credit changed across a settlement */
    WWWS_ERR_TIMEOUT = 7,   /* reserved */
    WWWS_ERR_INDEX = 8      /* only from a library built with -DWWWS_CHECK_INDICES: an index that a kernel took from
                               device data (a partner id, a list offset, a candidate or executor id) was out of
                               range; the access was skipped and the results of that call are not to be trusted */
} wwws_status;

#define WWWS_WINDOW 32u      /* candidate-window width: peers per block of the id ring */
#define WWWS_MAX_JUDGES 4u
#define WWWS_FLAG_REPUTATION 1u /* multiply the PoS weight by the smoothed duel win rate */
#define WWWS_FLAG_LOAD 2u       /* multiply the PoS weight by the advertised spare-capacity fraction */
#define WWWS_FLAG_PUSH_PULL 8u  /* gossip as a full pairwise exchange: the pulled partner also merges the puller's
                                   view (Appendix "Gossip-Driven Peer Synchronization": two nodes exchange views) */
#define WWWS_FLAG_FIFO 16u      /* exact queueing inside a batch: a request's latency counts the work that earlier
                                   requests of the same batch put on its executor (executions, challenger runs,
                                   judge evaluations), not only the executor's queue at the start of the batch;
                                   also validates every payment against the payer's balance inside the open block
                                   (n_uncovered) */
#define WWWS_FLAG_MAJORITY 32u  /* a block is committed only if more than half of the peers are online to confirm it
                                   (Section "Credit-based Transaction System"); otherwise it stays open and its
                                   operations are committed with the next block that finds a majority */
#define WWWS_FLAG_GREEDY 4u     /* customised rule: instead of drawing in proportion to the weights, take the
                                   candidate with the highest weight (lowest id on ties), then the next one on
                                   refusal; flags bit 0 then marks a runner-up within 1e-5 (relative) of the pick */

/* Plain data, copied at creation.  Probabilities are in parts per million. */
typedef struct {
    uint32_t n_peers;          /* 2 .. 65535 */
    uint32_t n_replicas;       /* 1 .. 65535 */
    uint32_t replica_offset;   /* global index of replica 0 (replicas sharded over processes) */
    uint32_t max_batch;        /* largest `count` wwws_dispatch_batch will be given */
    uint64_t seed;
    uint32_t fanout_k;         /* gossip partners per round, 1..4 */
    uint32_t gossip_tries;     /* attempts to find a partner believed online, 1..64 */
    uint32_t max_probes;       /* willingness probes per request (executor + challenger), 1..15 */
    uint32_t n_judges;         /* judges per duel, 1..4 */
    uint32_t p_duel_ppm;       /* p_d of Assumption 2 */
    uint32_t p_noise_ppm;      /* a judge's vote is flipped with this probability */
    uint32_t p_leave_ppm;      /* per gossip round: an online peer crashes */
    uint32_t p_join_ppm;       /* per gossip round: an offline peer comes back */
    uint32_t p_prio_active_ppm;/* a peer with prio_flag runs its own prioritized load in a window */
    uint32_t prio_window_ms;   /* > 0 */
    uint32_t util_window_ms;   /* utilisation = backlog / (this much work at the current rate), > 0 */
    uint32_t cap_ref_tok_s;    /* reference rate of the SLO deadline, > 0 */
    uint32_t slo_num, slo_den; /* deadline = slo_num * ideal latency / slo_den, slo_den > 0 */
    uint32_t hop_ms;           /* network latency added to delegated requests */
    uint32_t init_stale_max;   /* initial views are 0..this many versions old, < 2^24 - 2 */
    uint32_t flags;            /* WWWS_FLAG_* */
    uint32_t n_rank;           /* entries in rank_cdf, 0 with rank_cdf == NULL */
    int64_t reward_R;          /* R of Assumption 2, > 0 */
    int64_t reward_add;        /* R_add, 0 < reward_add <= penalty_P */
    int64_t penalty_P;         /* P */
    const uint32_t* rank_cdf;  /* HOST, nondecreasing thresholds scaled to 2^32: the block rank of a request
                                  is the first index whose threshold exceeds a uniform 32-bit draw;
                                  NULL = uniform over blocks */
} wwws_config;

/* HOST arrays, each [n_replicas][n_peers]; copied at creation. */
typedef struct {
    const uint32_t* cap_true_tok_s; /* true service rate, tokens/s (0 = requester-only node) */
    const uint32_t* quality_fx;     /* hidden quality q_i of Assumption 1 as q * 2^32, clamped to 2^32-1 */
    const int64_t* credit0;         /* initial credit */
    const uint16_t* stake_pm;       /* fraction of credit staked, per mille (0..1000) */
    const uint16_t* offload_util_pm;/* offload when own utilisation >= this (per mille) */
    const uint16_t* accept_util_pm; /* accept delegated work while own utilisation < this */
    const uint32_t* offload_ppm;    /* offload frequency */
    const uint32_t* accept_ppm;     /* accept frequency */
    const uint8_t* misreport_mul;   /* advertised capacity = true capacity * this (1 = honest) */
    const uint8_t* prio_flag;       /* has a prioritized local load */
    const uint8_t* online0;         /* online at time 0 */
} wwws_peer_init;

/* DEVICE arrays [n_replicas][n_requests], caller-owned, read by the library. */
typedef struct {
    const uint32_t* origin; /* peer that received the user request, < n_peers */
    const uint16_t* len_in; /* prompt tokens */
    const uint16_t* len_out;/* generated tokens */
    uint64_t n_requests;    /* per replica, < 2^32 */
} wwws_requests;

/* DEVICE arrays [n_replicas][n_requests], caller-owned, written for the slots of each batch. */
typedef struct {
    int32_t* exec_a;   /* >= 0 executor; -1 served locally by policy; -2 locally because nobody was willing;
                          -3 dropped (origin offline or invalid); -4 failed (local, origin has no capacity) */
    int32_t* exec_b;   /* challenger of a decided duel, else -1 */
    int32_t* judges;   /* [..][4], -1 padded; judges of a decided duel */
    uint8_t* outcome;  /* 0 no duel, 1 executor won, 2 challenger won, 3 draw, 4 duel cancelled */
    uint8_t* flags;    /* bit 0: some draw of this request fell within 1e-5 (relative) of an interval end */
    float* score_a;    /* fp32 score of the executor (0 if none); may be NULL */
    float* score_sum;  /* fp32 sum of the window's scores, lane-ascending; may be NULL */
} wwws_results;

/* Counters, per replica and in total. */
typedef struct {
    uint64_t n_requests, n_local, n_fallback_local, n_dropped, n_failed, n_delegated, n_duel, n_duel_cancelled,
        n_draw, n_judge_evals, n_probes, n_near_boundary, slo_met, sum_latency_ms, n_offline_marks, rounds, blocks;
    int64_t credit_total; /* finalized + pending credit of all peers */
    uint64_t chain_head;     /* id of the last finalized credit block (Table "Structure of a Credit Block"):
                                hash of the parent id, the block's operations digest and its height */
    uint64_t pending_digest; /* order-independent digest (wrapping sum of per-record hashes) of the credit
                                operations settled since the last finalization */
    uint64_t n_uncovered;    /* with WWWS_FLAG_FIFO: payments that exceeded the payer's finalized balance minus
                                what it had already spent in the open block (double-spend check; counted only) */
    uint64_t blocks_rejected;/* with WWWS_FLAG_MAJORITY: finalizations refused for want of a majority */
} wwws_stats_t;

/* Per-peer tables for wwws_export_table / wwws_import_table; element type in the comment. */
typedef enum {
    WWWS_T_ONLINE = 0,   /* uint8  */
    WWWS_T_CAP_EFF,      /* uint32 */
    WWWS_T_BACKLOG,      /* int64  tokens queued */
    WWWS_T_VER,          /* uint32 */
    WWWS_T_CREDIT,       /* int64  finalized */
    WWWS_T_STAKE,        /* int64  */
    WWWS_T_WINS,         /* uint32 */
    WWWS_T_DUELS,        /* uint32 */
    WWWS_T_SERVED,       /* uint64 delegated executions */
    WWWS_T_SERVED_LOCAL, /* uint64 */
    WWWS_T_D_CREDIT,     /* int64  pending */
    WWWS_T_D_WINS,       /* uint32 pending */
    WWWS_T_D_DUELS,      /* uint32 pending */
    WWWS_T_BLK_SPENT,    /* int64  with WWWS_FLAG_FIFO: credits spent in the block that is still open */
    WWWS_T_COUNT
} wwws_table;

/* Bytes of device workspace a network with this configuration needs. */
wwws_status wwws_workspace_bytes(const wwws_config* cfg, uint64_t* bytes_out);

/* Build the network in `workspace` (DEVICE, 256-byte aligned, at least wwws_workspace_bytes()):
 * peers from `init`, every node knowing every peer by a version up to init_stale_max old.
 * `cuda_stream` is a cudaStream_t (NULL = default stream).  The library keeps the workspace
 * until wwws_destroy_network; the caller frees it afterwards. */
wwws_status wwws_create_network(const wwws_config* cfg, const wwws_peer_init* init, void* workspace,
                                uint64_t workspace_bytes, void* cuda_stream, wwws_network** out);
wwws_status wwws_destroy_network(wwws_network* net);

/* Attach request and result arrays (borrowed; must stay valid while used). */
wwws_status wwws_bind_requests(wwws_network* net, const wwws_requests* req, const wwws_results* res);

/* Simulated time moves to now_ms (>= the previous value): online peers drain their queues at
 * their effective rate; prioritized local load halves a peer's rate in the windows it is active
 * (Introduction: providers keep their own prioritized workloads). */
wwws_status wwws_advance_time(wwws_network* net, uint32_t now_ms);

/* One synchronous gossip round (Appendix "Gossip-Driven Peer Synchronization"): churn; every
 * online peer issues a new version of its own entry (online, advertised capacity and queue);
 * every online node pulls the views of fanout_k partners it believes online and keeps, entry
 * by entry, the newer one (64-bit max of the packed entry); a failed pull marks the partner
 * offline; a pull shows the puller's own entry to the partner. */
wwws_status wwws_gossip_round(wwws_network* net);

/* Dispatch requests [first, first+count) of every replica against the state at the call
 * (Section "Request Routing and Node Design"): local-or-delegate by the origin's policy; a
 * 32-peer candidate window scored in fp32 from the origin's gossiped view and the shared
 * ledger; executor drawn with probability proportional to the score (Assumption 3) by integer
 * prefix sums; the drawn peer probed against its true state and accept policy; redraw on
 * refusal.  Writes exec_a, flags, score_a, score_sum; resets exec_b, judges, outcome. */
wwws_status wwws_dispatch_batch(wwws_network* net, uint64_t first, uint64_t count);

/* Duel-and-judge for the batch last dispatched (Section "Duel-and-Judge Mechanism"): a
 * delegated request becomes a duel with probability p_duel; challenger and judges continue
 * the request's draw sequence; each judge votes for the executor with probability
 * (1 + q_A - q_B)/2 (Assumption 3, pairwise); the majority decides. */
wwws_status wwws_duel_judge(wwws_network* net);

/* Settle the batch (Section "Credit-based Transaction System", Lemma 1): R from origin to
 * each executor, loser pays P, winner earns R_add, judges share P - R_add; reputation and
 * queue updates; latency and SLO counters.  Credit and reputation changes stay pending until
 * a call with finalize != 0 commits the block: ledger folded, stakes re-derived, total credit
 * checked.  Must follow wwws_duel_judge. */
wwws_status wwws_settle_credits(wwws_network* net, int finalize);

/* One whole step in a single call, same results as
 * advance_time(now_ms); [gossip_round();] dispatch_batch; duel_judge; settle_credits(finalize)
 * with dispatch, duel and settlement fused into one kernel. */
wwws_status wwws_step(wwws_network* net, uint64_t first, uint64_t count, uint32_t now_ms, int do_gossip,
                      int finalize);

/* HOST mirrors of the request/result arrays, same [n_replicas][n_requests] layout. */
typedef struct {
    const uint32_t* origin; const uint16_t* len_in; const uint16_t* len_out;
    int32_t* exec_a; int32_t* exec_b; int32_t* judges; uint8_t* outcome; uint8_t* flags;
} wwws_host_io;

/* wwws_step with HOST buffers; synchronises before it returns.  totals_out (HOST, one record) may be NULL.
 * Two ways, with identical results.  Direct: if all eight buffers are page-locked and mapped into the device's
 * address space (cudaHostAlloc, cudaHostRegister), exact queueing (WWWS_FLAG_FIFO) is off and the batch is small
 * (n_replicas * count <= 98304, or WWWS_OPT_HOST_IO = 1), the kernels read the batch's requests from, and write
 * its results to, the host buffers themselves; the bound device arrays are not touched.  Staged: the batch's
 * request slices are copied to the bound device arrays on a second stream (created at the first such call)
 * while time advance and gossip run, the step runs on the device arrays, and the batch's results are copied
 * back on that stream while the block is folded.  Either way the total counters come back in totals_out. */
wwws_status wwws_step_host(wwws_network* net, const wwws_host_io* io, uint64_t first, uint64_t count,
                           uint32_t now_ms, int do_gossip, int finalize, wwws_stats_t* totals_out);

/* Counters: host_out is HOST [n_replicas + 1], the last record holds the totals. */
wwws_status wwws_stats(wwws_network* net, wwws_stats_t* host_out);

/* Copy one per-peer table to / from HOST memory ([n_replicas][n_peers] of the table's element
 * type; `bytes` must match).  Import is meant for checkpoint/resume and for setting up cases;
 * importing WWWS_T_CREDIT re-derives stakes. */
wwws_status wwws_export_table(wwws_network* net, wwws_table table, void* host_dst, uint64_t bytes);
wwws_status wwws_import_table(wwws_network* net, wwws_table table, const void* host_src, uint64_t bytes);

/* Copy rows [row_first, row_first + n_rows) of replica `replica`'s current view matrix to HOST
 * memory as n_rows * n_peers packed entries: bits 63..40 version, bit 39 offline, bits 38..20
 * advertised capacity (tokens/s), bits 19..0 advertised queue in 16-token units; 0 = unknown. */
wwws_status wwws_export_view_rows(wwws_network* net, uint32_t replica, uint32_t row_first, uint32_t n_rows,
                                  uint64_t* host_dst);

/* Checkpoint / resume.  A network's state is its per-peer tables (wwws_export_table), its view
 * matrices (wwws_export_view_rows), its counters (wwws_stats; the chain head lives there) and its
 * clock (simulated time and gossip round number).  Importing all of them into a network created
 * from the same configuration and peer arrays continues the run bit for bit.  host_src of
 * wwws_import_view_rows is n_rows * n_peers packed entries; host_src of wwws_import_stats is
 * HOST [n_replicas] (the totals record is not read).  None of these may be called inside a batch. */
wwws_status wwws_import_view_rows(wwws_network* net, uint32_t replica, uint32_t row_first, uint32_t n_rows,
                                  const uint64_t* host_src);
wwws_status wwws_export_clock(wwws_network* net, uint32_t* now_ms, uint32_t* round);
wwws_status wwws_import_clock(wwws_network* net, uint32_t now_ms, uint32_t round);
wwws_status wwws_import_stats(wwws_network* net, const wwws_stats_t* host_src);

/* Tuning options; results never depend on them. */
typedef enum {
    WWWS_OPT_REQUEST_KERNEL = 0,/* implementation of wwws_dispatch_batch / wwws_duel_judge: 0 chosen by launch size
                                   (default), 1 one warp per request (lane per candidate, warp-shuffle prefix sums),
                                   2 one thread per request (weights in shared memory, duels compacted per block) */
    WWWS_OPT_STEP_KERNEL = 1,   /* implementation of wwws_step's fused kernel: 0 chosen by launch size (default),
                                   1 eight lanes per request, 2 four lanes per request, 3 one thread per request,
                                   4 streaming phases (a warp takes a run of requests through origin / score /
                                   draw / vote / finish with full warps) */
    WWWS_OPT_STREAM_RUN = 2,    /* requests per warp of the streaming kernel: 0 chosen by launch size (default),
                                   else a multiple of 32 */
    WWWS_OPT_HOST_IO = 4,       /* wwws_step_host: 0 (default) chosen by batch size, 1 kernels read and write mapped host
                                   buffers directly where possible, 2 always staged copies */
    WWWS_OPT_LAUNCH_OVERLAP = 3 /* mask of the kernels that are launched so that their grid may be scheduled while the
                                   previous grid of the stream finishes (programmatic dependent launch; every kernel
                                   waits for its predecessor's completion before it touches memory): bit 0 time
                                   advance and the rest, bit 1 gossip, bit 2 request kernels, bit 3 fold.  Default: 15
                                   for networks of up to 32,768 peer-replicas (their steps are chains of launch
                                   latencies), 0 for larger ones */
} wwws_option;
wwws_status wwws_set_option(wwws_network* net, wwws_option option, int64_t value);

/* Kernels launched so far on behalf of this network. */
uint64_t wwws_kernel_launches(const wwws_network* net);

/* Optional per-kernel timing.  While enabled every kernel launch is bracketed by two CUDA
 * events on the network's stream.  wwws_profile(net, enable) clears the sums and switches
 * it; wwws_profile_read waits for the recorded events and writes, per kernel class
 * 0 .. wwws_profile_kernels()-1, the summed device time in milliseconds and the number of
 * launches (HOST arrays of that length).  wwws_profile_kernel_name gives the class's name. */
wwws_status wwws_profile(wwws_network* net, int enable);
wwws_status wwws_profile_read(wwws_network* net, double* ms_out, uint64_t* count_out);
uint32_t wwws_profile_kernels(void);
const char* wwws_profile_kernel_name(uint32_t kernel);

const char* wwws_last_error(const wwws_network* net);

/* wwws_gossip_round for callers that must not allocate.  (The paper has no counterpart: this
 * is a packaging variant of the round above, with identical results.)
 *
 * Who needs it: a program that embeds the library at a point where it cannot obtain device
 * memory - the whole GPU already belongs to another allocator's pool, allocation is not
 * allowed in that phase, or the device-wide synchronisation of cudaMalloc would stall its
 * loop.  The round's scratch (this round's self entries and partner lists, 24 bytes per
 * peer and replica) is taken from a fixed 1.5 MiB array inside the library image instead of
 * the workspace; every GPU that loads the library holds that array until the process exits.
 * The call itself allocates nothing on host or device paths of CUDA: no cudaMalloc, no
 * cudaFree, no allocating library routine.  Per-kernel timing (wwws_profile) creates CUDA
 * events, so while it is switched on this call returns WWWS_ERR_STATE instead of running.
 *
 * Limit: n_replicas * n_peers <= 65536; larger networks get WWWS_ERR_ARG and must use
 * wwws_gossip_round.  The first call on each device looks up the array's device address
 * (the call makes the network's device current for that, as every call of this library
 * does) and should be made before any stream capture begins; threads that make that first
 * call at the same time all find the same address.  All calls, from all
 * networks on a device, share the one array: two such rounds that overlap on the GPU (two
 * streams) race and give wrong views; run them one after another.  The array keeps the
 * previous round's contents; nothing in it has to start at zero, because each round
 * rewrites the entries of all its peers before reading them. */
wwws_status wwws_gossip_round_static(wwws_network* net);

#ifdef __cplusplus
}
#endif
#endif /* WWWS_H */
