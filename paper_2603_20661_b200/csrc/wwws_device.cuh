// Device-side state layout and small helpers shared by the wwws kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace wwws {

constexpr uint32_t kWin = 32;                 // candidate window = one warp
constexpr uint64_t kOffBit = 1ull << 39;
constexpr uint32_t kCapMax = (1u << 19) - 1;
constexpr uint32_t kQMax = (1u << 20) - 1;

// Random stages: the fourth counter word is stage + 256 * attempt.
enum : uint32_t { kOrigin = 1, kDraw = 2, kProbe = 3, kJudge = 4, kGossip = 5, kChurn = 6, kPrio = 7, kInit = 8 };

// Per-replica counters, in the order of wwws_stats_t.
enum : uint32_t { sRequests, sLocal, sFallback, sDropped, sFailed, sDelegated, sDuel, sDuelCancelled, sDraw,
                  sJudgeEvals, sProbes, sNear, sSloMet, sSumLat, sOfflineMarks, sRounds, sBlocks, sCreditTotal,
                  sChainHead, sPendingDigest, sUncovered, sBlocksRejected, sCount };

// Device error word codes (subset of wwws_status).
enum : uint32_t { eArg = 1, eRange = 4, eInvariant = 6, eIndex = 8 };

// Everything a kernel needs, passed by value.  Per-peer arrays are [Rp][N]; the view is
// [Rp][N][ld] with ld = N rounded up to 32 so that a candidate window is one aligned
// 256-byte segment; padding columns stay 0 ("never heard of").
struct Net {
    uint32_t N, Rp, ld, n_blk, replica_offset;
    uint32_t key0, key1;
    uint32_t fanout_k, gossip_tries, max_probes, n_judges;
    uint32_t p_duel, p_noise, p_leave, p_join, p_prio;
    uint32_t prio_window_ms, util_window_ms, cap_ref, slo_num, slo_den, hop_ms, flags, n_rank;
    int64_t R, R_add, P;
    int64_t judge_share[4];                      // (P - R_add) / n for n = 1..4 judges
    float uwf;                                   // util_window_ms / 1000 in fp32
    // view double buffer
    uint64_t* view; uint64_t* view_new;
    // hidden / policy (constant after creation)
    const uint32_t* cap_true; const uint32_t* quality; const uint16_t* stake_pm; const uint16_t* offload_util_pm;
    const uint16_t* accept_util_pm; const uint32_t* offload_ppm; const uint32_t* accept_ppm;
    const uint8_t* misreport; const uint8_t* prio_flag;
    // dynamic
    uint8_t* online; uint32_t* cap_eff; int64_t* backlog; uint32_t* ver;
    // ledger
    int64_t* credit; int64_t* stake; uint32_t* wins; uint32_t* duels;
    unsigned long long* served; unsigned long long* served_local;
    // pending block and pending queue growth
    long long* d_credit; uint32_t* d_wins; uint32_t* d_duels; long long* d_backlog;
    // derived: (float)stake * smoothed win rate, refreshed whenever the ledger is finalized; [Rp][ld], padding 0,
    // so that a candidate window's 32 weights are one aligned 128-byte segment
    float* w_led;
    // derived: what a probe and an origin decision need from a peer's true state and policy, in one word each
    // (see peer_gate); refreshed by every kernel that changes online, cap_eff, backlog or the finalized credit
    uint64_t* gate;
    // gossip scratch: this round's self entries and chosen partners
    uint64_t* self_entry; int32_t* partner;     // partner is [Rp][N][4]
    // reverse lists of the pairwise exchange: in-degree, list offset, fill cursor, puller ids [Rp][4N]
    uint32_t* in_deg; uint32_t* in_off; uint32_t* in_cursor; int32_t* pullers;
    // exact intra-batch queueing: work items (peer, tokens) of the batch [Rp][7*max_batch] (slot = request*7 + role; role 6 = the payment)
    // and, per peer, the list (request, tokens) of the items queued on it
    int2* fifo_items; uint2* fifo_list;
    // credits spent since the last finalization (earlier batches of the block / this batch), for in-block validation
    long long* blk_spent; long long* d_spent;
    // dispatch -> duel continuation, [Rp][max_batch]
    uint2* cont; uint32_t max_batch;
    const uint32_t* rank_cdf;
    unsigned long long* stats;                   // [Rp][sCount]
    const int64_t* credit_total0; long long* credit_check;   // [Rp]
    uint32_t* online_count;                      // [Rp] majority validation: peers online when a block is proposed
    uint32_t* fold_ticket;                       // [Rp] blocks of k_fold that have finished the replica
    uint32_t* err;                               // [2]: code, detail
    // bound requests / results
    const uint32_t* origin; const uint16_t* len_in; const uint16_t* len_out; uint64_t Q;
    int32_t* exec_a; int32_t* exec_b; int32_t* judges; uint8_t* outcome; uint8_t* rflags;
    float* score_a; float* score_sum;
};

// First statement of every kernel: let the next grid of the stream be scheduled already, then wait
// until the previous grid has completed and its memory operations are visible.  Without the
// programmatic-serialization launch attribute both instructions do nothing.
__device__ __forceinline__ void grid_dependency_enter()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

struct Rnd4 { uint32_t w[4]; };

// Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC'11).
__device__ __forceinline__ Rnd4 philox(uint32_t k0, uint32_t k1, uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3)
{
#pragma unroll
    for (int i = 0; i < 10; ++i) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0; c1 = lo1; c2 = hi0 ^ c3 ^ k1; c3 = lo0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    Rnd4 r; r.w[0] = c0; r.w[1] = c1; r.w[2] = c2; r.w[3] = c3;
    return r;
}

__device__ __forceinline__ Rnd4 draw(const Net& n, uint32_t index, uint32_t slot, uint32_t rg, uint32_t stage)
{
    return philox(n.key0, n.key1, index, slot, rg, stage);
}

__device__ __forceinline__ uint32_t ppm(uint32_t x) { return __umulhi(x, 1000000u); }
__device__ __forceinline__ uint32_t below(uint32_t x, uint32_t m) { return __umulhi(x, m); }

__device__ __forceinline__ uint64_t pack_entry(uint32_t ver, bool offline, uint64_t cap, uint64_t q)
{
    cap = cap > kCapMax ? kCapMax : cap;
    q = q > kQMax ? kQMax : q;
    return (uint64_t(ver) << 40) | (offline ? kOffBit : 0ull) | (cap << 20) | q;
}

// floor(min(1000, backlog*1000/denom)) >= thr  without the division.
__device__ __forceinline__ bool util_at_least(uint32_t cap_eff, int64_t backlog, uint32_t util_window_ms, uint32_t thr)
{
    if (thr == 0) return true;
    if (thr > 1000) return false;
    if (cap_eff == 0) return true;
    uint64_t denom = uint64_t(cap_eff) * util_window_ms / 1000u;
    if (denom < 1) denom = 1;
    return uint64_t(backlog) * 1000ull >= uint64_t(thr) * denom;
}

// A peer's "gate": everything a probe of the peer (low word) and a dispatch decision at the peer as
// origin (high word) read from its true state and policy, evaluated once per state change instead
// of once per request.
//   low  word: accept frequency in ppm if the peer would accept delegated work now (online, has
//              capacity, utilisation below its accept threshold), else 0: a probe is  ppm(u) < low
//   high word: bits 0..19 offload frequency in ppm if the peer, as origin, may offload now
//              (utilisation at or above its threshold and it can afford R), else 0;
//              bit 20 online; bit 21 no capacity
constexpr uint32_t kGateOnline = 1u << 20, kGateNoCap = 1u << 21, kGateFreq = (1u << 20) - 1u;
__device__ __forceinline__ void refresh_gate(const Net& n, size_t x, bool on, uint32_t cap, int64_t backlog, int64_t credit)
{
    const bool accepts = on && cap != 0 && !util_at_least(cap, backlog, n.util_window_ms, n.accept_util_pm[x]);
    const bool offloads = util_at_least(cap, backlog, n.util_window_ms, n.offload_util_pm[x]) && credit >= n.R;
    const uint32_t lo = accepts ? n.accept_ppm[x] : 0u;
    const uint32_t hi = (offloads ? n.offload_ppm[x] : 0u) | (on ? kGateOnline : 0u) | (cap == 0 ? kGateNoCap : 0u);
    n.gate[x] = uint64_t(hi) << 32 | lo;
}

__device__ __forceinline__ uint32_t cap_eff_at(const Net& n, uint32_t cap_true, bool prio, uint32_t j, uint32_t rg,
                                               uint32_t now_ms)
{
    if (!prio) return cap_true;
    const uint32_t w = now_ms / n.prio_window_ms;
    return ppm(draw(n, j, w, rg, kPrio).w[0]) < n.p_prio ? cap_true / 2 : cap_true;
}

// Credit block chain: SplitMix64 finaliser (Steele, Lea, Flood 2014) as the record and block hash.
constexpr uint64_t kGamma = 0x9E3779B97F4A7C15ull;
__host__ __device__ __forceinline__ uint64_t mix64(uint64_t z)
{
    z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ull;
    z ^= z >> 27; z *= 0x94D049BB133111EBull;
    z ^= z >> 31;
    return z;
}
__device__ __forceinline__ uint64_t chain_key(const Net& n, uint32_t r)
{
    return (uint64_t(n.key1) << 32 | n.key0) ^ (uint64_t(r + n.replica_offset) * kGamma);
}
// Hash of one ledger record: request q moves `amount` credits on `peer`'s account, for reason `kind`.
enum : uint32_t { opPay = 1, opEarn = 2, opPayChallenger = 3, opEarnChallenger = 4, opPenalty = 5, opReward = 6, opJudge = 7 };
static __device__ __noinline__ uint64_t record_hash(uint64_t key, uint32_t q, uint32_t kind, uint32_t peer, int64_t amount)
{
    return mix64(mix64(key ^ (uint64_t(q) << 32 | uint64_t(kind) << 24 | peer)) + uint64_t(amount));
}

__device__ __forceinline__ void set_error(const Net& n, uint32_t code, uint32_t detail)
{
    if (atomicCAS(&n.err[0], 0u, code) == 0u) n.err[1] = detail;
}

// Checked build (-DWWWS_CHECK_INDICES): every index that a kernel takes from device data (partner
// ids, list offsets, candidate and executor ids, queue slots) is range-checked before use; a bad
// one sets the device error word (code eIndex, detail = the site's tag) and the access is skipped.
// Nothing traps.  In the normal build the test compiles to `true`.
#ifdef WWWS_CHECK_INDICES
__device__ __forceinline__ bool index_ok(const Net& n, uint64_t i, uint64_t limit, uint32_t tag)
{
    if (i < limit) return true;
    set_error(n, eIndex, tag);
    return false;
}
#else
__device__ __forceinline__ bool index_ok(const Net&, uint64_t, uint64_t, uint32_t) { return true; }
#endif

}  // namespace wwws
