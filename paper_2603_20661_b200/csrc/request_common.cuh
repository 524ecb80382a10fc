// Pieces of the request path shared by the warp-per-request kernels (dispatch, duel, settle)
// and the thread-per-request fused step.
#pragma once
#include "wwws_internal.cuh"

namespace wwws {

constexpr unsigned kFull = 0xffffffffu;

// ---- per-block counters -------------------------------------------------------------------

struct BlockStats {
    unsigned long long c[sCount];
};

__device__ __forceinline__ void stats_begin(BlockStats& s)
{
    if (threadIdx.x < sCount) s.c[threadIdx.x] = 0;
    __syncthreads();
}
__device__ __forceinline__ void stats_add(BlockStats& s, uint32_t k, unsigned long long v)
{
    if (v) atomicAdd(&s.c[k], v);
}
__device__ __forceinline__ void stats_end(const Net& n, BlockStats& s, uint32_t r)
{
    __syncthreads();
    if (threadIdx.x < sCount) {
        const unsigned long long v = s.c[threadIdx.x];
        if (v) atomicAdd(&n.stats[size_t(r) * sCount + threadIdx.x], v);
    }
}

// D3: the block of the id ring this request samples from.
__device__ __forceinline__ uint32_t pick_block(const Net& n, uint32_t o, uint32_t w2)
{
    uint32_t rank;
    if (n.rank_cdf) {
        uint32_t lo = 0, hi = n.n_rank;           // first index with w2 < cdf[idx]
        while (lo < hi) {
            const uint32_t mid = (lo + hi) >> 1;
            if (w2 < __ldg(n.rank_cdf + mid)) hi = mid; else lo = mid + 1;
        }
        rank = lo > n.n_blk - 1 ? n.n_blk - 1 : lo;
    } else {
        rank = below(w2, n.n_blk);
    }
    return (o / kWin + rank) % n.n_blk;
}

// D4: fp32 score and integer weight of candidate `id` as the origin `o` sees it: view entry `e`
// of the origin's row, ledger weight `wl`.  Every fp32 operation is an explicitly rounded IEEE
// operation (no fused multiply-add), so a CPU computing the same expression in binary32 gets the
// same bits.  Returns the weight (0 = not eligible) and the score through `score`.
__device__ __forceinline__ uint64_t candidate_weight(const Net& n, uint32_t o, uint32_t id, uint64_t e, float wl, float& score)
{
    score = 0.0f;
    if (id >= n.N || id == o || e == 0 || (e & kOffBit)) return 0;
    const uint32_t advcap = uint32_t(e >> 20) & kCapMax, advq = uint32_t(e) & kQMax;
    if (!(wl > 0.0f) || advcap == 0) return 0;
    float spare = 1.0f;
    if (n.flags & 2u) {
        const float utilf = __fdiv_rn(__uint2float_rn(advq * 16u), __fmul_rn(__uint2float_rn(advcap), n.uwf));
        spare = __fsub_rn(1.0f, utilf);
        if (!(spare > 0.0f)) spare = 0.0f;
    }
    const float sc = __fmul_rn(wl, spare);
    const float scaled = __fmul_rn(sc, 256.0f);
    const uint64_t W = scaled >= 72057594037927936.0f ? (1ull << 56) : __float2ull_rz(scaled);
    if (W) score = sc;
    return W;
}

// fp32 score of one candidate (0 when it is not eligible or its integer weight truncates to 0),
// branch-free.  Same IEEE operations, in the same order, as candidate_weight().  Eligibility by
// the entry is one range test on its bits 20..39 (advertised capacity and offline bit): capacity
// in 1..2^19-1 and offline bit clear  <=>  (bits - 1) < 2^19 - 1; an entry that was never heard
// of (0) and a padding column have capacity 0.  A ledger weight is never negative, so a score of
// at least 2^-8 (integer weight >= 1) implies a positive weight.  The origin itself is taken out
// of its own window by the caller.
template <bool LOAD>
__device__ __forceinline__ float candidate_score(const Net& n, uint32_t elo, uint32_t ehi, float wl)
{
    const uint32_t t = __funnelshift_r(elo, ehi, 20);
    float spare = 1.0f;
    if (LOAD) {
        const float utilf = __fdiv_rn(__uint2float_rn((elo & kQMax) << 4), __fmul_rn(__uint2float_rn(t & kCapMax), n.uwf));
        spare = fmaxf(__fsub_rn(1.0f, utilf), 0.0f);                 // capacity 0 gives inf or NaN here, and 0 after the max
    }
    const float sc = __fmul_rn(wl, spare);
    const bool ok = ((t & 0xfffffu) - 1u) < kCapMax && sc >= 0.00390625f;
    return ok ? sc : 0.0f;
}

// The integer weight of a stored score: trunc(256 sc), at most 2^56 (the same value as weight_of()).
__device__ __forceinline__ unsigned long long weight_q(float sc)
{
    return __float2ull_rz(fminf(__fmul_rn(sc, 256.0f), 72057594037927936.0f));
}

// D1, D2 from the origin's gate word (see refresh_gate): true if the request goes to the network,
// else `code` is the local / dropped / failed code.  Same decisions as origin_offloads().
__device__ __forceinline__ bool origin_gate(const Net& n, uint32_t r, uint32_t o, const Rnd4& rx, int& code)
{
    code = -3;
    if (o >= n.N) { set_error(n, eArg, o); return false; }
    const uint32_t g = reinterpret_cast<const uint32_t*>(n.gate)[2 * (size_t(r) * n.N + o) + 1];
    if (!(g & kGateOnline)) return false;
    code = (g & kGateNoCap) ? -4 : -1;
    return ppm(rx.w[0]) < (g & kGateFreq);
}

// D6 from the drawn candidate's gate word: one load and the probe's random word.
__device__ __forceinline__ bool probe_gate(const Net& n, uint32_t r, uint32_t rg, uint32_t q, uint32_t blk, int pick)
{
    if (!index_ok(n, kWin * blk + uint32_t(pick), n.N, 410)) return false;
    const uint32_t thr = reinterpret_cast<const uint32_t*>(n.gate)[2 * (size_t(r) * n.N + kWin * blk + pick)];
    const Rnd4 y = draw(n, q, uint32_t(pick) >> 2, rg, kProbe);
    const uint32_t sel = uint32_t(pick) & 3u;
    return ppm(sel == 0 ? y.w[0] : sel == 1 ? y.w[1] : sel == 2 ? y.w[2] : y.w[3]) < thr;
}

// The integer weight that candidate_weight() derives from a score.
__device__ __forceinline__ uint64_t weight_of(float sc)
{
    const float scaled = __fmul_rn(sc, 256.0f);
    return scaled >= 72057594037927936.0f ? (1ull << 56) : __float2ull_rz(scaled);
}

// D6: the drawn candidate answers by its true state and its own accept policy.  All five values
// are loaded at once and the probe's random word is computed while they are in flight: one
// memory round trip per probe instead of a chain of dependent ones.
__device__ __forceinline__ bool probe_peer(const Net& n, uint32_t r, uint32_t rg, uint32_t q, uint32_t blk, int pick)
{
    const size_t x = size_t(r) * n.N + kWin * blk + pick;
    if (!index_ok(n, kWin * blk + uint32_t(pick), n.N, 409)) return false;
    const uint32_t cap = n.cap_eff[x];
    const uint8_t on = n.online[x];
    const int64_t queued = n.backlog[x];
    const uint32_t accept_util = n.accept_util_pm[x], accept_freq = n.accept_ppm[x];
    const Rnd4 y = draw(n, q, uint32_t(pick) >> 2, rg, kProbe);
    const uint32_t sel = uint32_t(pick) & 3u;                            // selected without indexing: the words stay in registers
    const uint32_t u = ppm(sel == 0 ? y.w[0] : sel == 1 ? y.w[1] : sel == 2 ? y.w[2] : y.w[3]);
    return on && cap != 0 && !util_at_least(cap, queued, n.util_window_ms, accept_util) && u < accept_freq;
}

// Origin side of dispatch (D1, D2).  Returns 1 if the request goes to the network, else
// writes the local / dropped / failed code to `code`.
__device__ __forceinline__ bool origin_offloads(const Net& n, uint32_t r, uint32_t o, const Rnd4& rx, int& code)
{
    if (o >= n.N) { set_error(n, eArg, o); code = -3; return false; }
    const size_t ox = size_t(r) * n.N + o;
    // independent loads first, decisions afterwards: one memory round trip
    const uint8_t on = n.online[ox];
    const uint32_t cap = n.cap_eff[ox];
    const int64_t queued = n.backlog[ox], credit = n.credit[ox];
    const uint32_t thr = n.offload_util_pm[ox], freq = n.offload_ppm[ox];
    if (!on) { code = -3; return false; }
    code = cap == 0 ? -4 : -1;
    return util_at_least(cap, queued, n.util_window_ms, thr) && ppm(rx.w[0]) < freq && credit >= n.R;
}

// 64-bit by 32-bit unsigned division; the common case (numerator below 2^32) takes the short
// 32-bit path instead of the long emulated 64-bit one.
static __device__ __noinline__ uint64_t udiv64_long(uint64_t t, uint32_t d) { return t / d; }   // one copy of the long path
__device__ __forceinline__ uint64_t udiv64by32(uint64_t t, uint32_t d)
{
    return (t >> 32) == 0 ? uint64_t(uint32_t(t) / d) : udiv64_long(t, d);
}

// ---- settlement of one request (one thread) ----------------------------------------------------

__device__ __forceinline__ void add64(long long* p, long long v) { atomicAdd((unsigned long long*)p, (unsigned long long)v); }

// Counters of the (at most two) requests a thread settles.  The twelve event counters other than
// the probe count stay below 8 per thread, so they are kept as 8-bit fields, four to a word, and
// a warp's sum of a field (at most 32 * 7) still fits its field: three reductions instead of twelve.
struct SettleAcc {
    uint32_t p[3];                 // field f of counter k: f = k below sProbes, k - 1 above
    uint32_t probes;
    unsigned long long sum_lat;
    unsigned long long digest;     // wrapping sum of the record hashes of this thread's requests
    __device__ __forceinline__ void add(uint32_t k, uint32_t v = 1u)
    {
        if (k == sProbes) { probes += v; return; }
        const uint32_t f = k < sProbes ? k : k - 1;
        p[f >> 2] += v << (8u * (f & 3u));
    }
};

// With exact intra-batch queueing (flag 16) the latency of a request depends on the work that
// earlier requests of the batch put on its executor, so settle_one only records the batch's work
// items (slot = request*7 + role: primary, challenger, four judges, and the origin's payment) and counts them per peer;
// k_fifo_latency computes the latencies once the per-peer lists are built.
__device__ __forceinline__ void fifo_emit(const Net& n, uint32_t r, uint32_t bidx, uint32_t role, int peer, uint32_t tokens)
{
    if (!index_ok(n, bidx, n.max_batch, 407)) return;
    n.fifo_items[(size_t(r) * n.max_batch + bidx) * 7 + role] = make_int2(peer, int(tokens));
    if (peer >= 0 && index_ok(n, uint32_t(peer), n.N, 408)) atomicAdd(&n.in_deg[size_t(r) * n.N + peer], 1u);
}

// S3 of a decided duel (outcome 1..3): the challenger's execution and payment, the judges' work,
// the reputation counters and the redistribution of the penalty.  Returns what the origin pays on
// top of the primary execution (R, for the challenger's run); the caller books it on the origin.
template <class Acc>
__device__ __forceinline__ long long settle_duel(const Net& n, uint32_t r, uint32_t q, uint32_t o, uint32_t li, uint32_t lo,
                                                 int a, int b, const int (&jd)[4], uint32_t oc, Acc& s)
{
    const size_t base = size_t(r) * n.N;
    const uint64_t key = chain_key(n, r);
    const uint64_t work = uint64_t(li) + lo;
#ifdef WWWS_CHECK_INDICES
    {
        bool ok = index_ok(n, uint32_t(a), n.N, 401) && index_ok(n, uint32_t(b), n.N, 402) && index_ok(n, o, n.N, 403);
        for (int l = 0; l < 4; ++l) if (jd[l] >= 0) ok = ok && index_ok(n, uint32_t(jd[l]), n.N, 404);
        if (!ok) return 0;
    }
#endif
    s.digest += record_hash(key, q, opPayChallenger, o, -n.R) + record_hash(key, q, opEarnChallenger, uint32_t(b), n.R);
    add64(&n.d_credit[base + b], n.R);
    add64(&n.d_backlog[base + b], (long long)work);
    atomicAdd(&n.served[base + b], 1ull);
    atomicAdd(&n.d_duels[base + a], 1u);
    atomicAdd(&n.d_duels[base + b], 1u);
    int nj = 0;
#pragma unroll
    for (int l = 0; l < 4; ++l)
        if (jd[l] >= 0) { add64(&n.d_backlog[base + jd[l]], (long long)(uint64_t(li) + 2ull * lo)); ++nj; }
    s.add(sJudgeEvals, uint32_t(nj));
    if (oc == 3) s.add(sDraw);
    else {
        const int win = oc == 1 ? a : b, lose = oc == 1 ? b : a;
        const long long pot = n.P - n.R_add, share = n.judge_share[nj - 1];
        const long long prize = n.R_add + (pot - share * nj);
        s.digest += record_hash(key, q, opPenalty, uint32_t(lose), -n.P) + record_hash(key, q, opReward, uint32_t(win), prize);
        add64(&n.d_credit[base + lose], -n.P);
        add64(&n.d_credit[base + win], prize);
        atomicAdd(&n.d_wins[base + win], 1u);
#pragma unroll
        for (int l = 0; l < 4; ++l)
            if (jd[l] >= 0) {
                s.digest += record_hash(key, q, opJudge + l, uint32_t(jd[l]), share);
                add64(&n.d_credit[base + jd[l]], share);
            }
    }
    return n.R;
}

// Settlement of one request.  `duel_booked`: the caller has already run settle_duel for this request
// (and booked its extra payment on the origin); everything else is still done here.
template <class Acc>
__device__ __forceinline__ void settle_one(const Net& n, uint32_t r, uint32_t q, uint32_t bidx, uint32_t o, uint32_t li, uint32_t lo,
                                           int a, int b, const int (&jd)[4], uint32_t oc, bool near, Acc& s, bool duel_booked = false)
{
    if (n.flags & 16u) {
        const bool served = a != -3 && a != -4, duel = a >= 0 && oc >= 1 && oc <= 3;
        fifo_emit(n, r, bidx, 0, served ? (a < 0 ? int(o) : a) : -1, li + lo);
        fifo_emit(n, r, bidx, 1, duel ? b : -1, li + lo);
#pragma unroll
        for (int l = 0; l < 4; ++l) fifo_emit(n, r, bidx, 2 + l, duel ? jd[l] : -1, li + 2u * lo);
        // the payment's slot carries the number of transactions of R (two for a duel); the amount stays 64-bit
        const uint32_t n_pay = duel ? 2u : 1u;
        fifo_emit(n, r, bidx, 6, a >= 0 ? int(o) : -1, n_pay);
        if (a >= 0) add64(&n.d_spent[size_t(r) * n.N + o], n.R * (long long)n_pay);
    }
    const size_t base = size_t(r) * n.N;
    const uint64_t work = uint64_t(li) + lo;
    s.add(sRequests);
    if (near) s.add(sNear);
    if (a == -3) { s.add(sDropped); return; }
    if (a == -4) { s.add(sFailed); return; }
    if (!index_ok(n, o, n.N, 405) || (a >= 0 && !index_ok(n, uint32_t(a), n.N, 406))) return;
    uint32_t ex;
    if (a < 0) {
        if (a == -1) s.add(sLocal); else s.add(sFallback);
        add64(&n.d_backlog[base + o], (long long)work);
        atomicAdd(&n.served_local[base + o], 1ull);
        ex = o;
    } else {
        s.add(sDelegated);
        const uint64_t key = chain_key(n, r);
        long long pay = n.R;
        s.digest += record_hash(key, q, opPay, o, -n.R) + record_hash(key, q, opEarn, uint32_t(a), n.R);
        add64(&n.d_credit[base + a], n.R);
        add64(&n.d_backlog[base + a], (long long)work);
        atomicAdd(&n.served[base + a], 1ull);
        ex = uint32_t(a);
        if (oc != 0) s.add(sDuel);
        if (oc == 4) s.add(sDuelCancelled);
        if (oc >= 1 && oc <= 3 && !duel_booked) pay += settle_duel(n, r, q, o, li, lo, a, b, jd, oc, s);
        add64(&n.d_credit[base + o], -pay);
    }
    if (n.flags & 16u) return;                       // latency and SLO are counted by k_fifo_latency
    const uint64_t cap = n.cap_eff[base + ex];
    const uint64_t t = (uint64_t(n.backlog[base + ex]) + work) * 1000ull, tq = udiv64by32(t, uint32_t(cap));
    const uint64_t lat = tq + (tq * cap != t ? 1 : 0) + (a >= 0 ? n.hop_ms : 0);
    const uint64_t ideal = udiv64by32(work * 1000ull + n.cap_ref - 1, n.cap_ref);
    const uint64_t deadline = udiv64by32(uint64_t(n.slo_num) * ideal, n.slo_den);
    s.sum_lat += lat;
    if (lat <= deadline) s.add(sSloMet);
}

__device__ __forceinline__ void acc_zero(SettleAcc& s)
{
    s.p[0] = s.p[1] = s.p[2] = 0; s.probes = 0;
    s.sum_lat = 0;
    s.digest = 0;
}

// Warp sums of a thread's counters, added to the block's counters by lane 0 (all lanes call).
__device__ __forceinline__ void acc_flush_warp(BlockStats& bs, const SettleAcc& s)
{
    const uint32_t w0 = __reduce_add_sync(kFull, s.p[0]), w1 = __reduce_add_sync(kFull, s.p[1]), w2 = __reduce_add_sync(kFull, s.p[2]);
    const uint32_t pr = __reduce_add_sync(kFull, s.probes);
    unsigned long long sl = s.sum_lat, dg = s.digest;
#pragma unroll
    for (int o = 16; o; o >>= 1) { sl += __shfl_down_sync(kFull, sl, o); dg += __shfl_down_sync(kFull, dg, o); }
    if ((threadIdx.x & 31) == 0) {
        const uint32_t w[3] = { w0, w1, w2 };
#pragma unroll
        for (uint32_t f = 0; f < 12; ++f) stats_add(bs, f < sProbes ? f : f + 1, (w[f >> 2] >> (8u * (f & 3u))) & 0xffu);
        stats_add(bs, sProbes, pr);
        stats_add(bs, sSumLat, sl);
        stats_add(bs, sPendingDigest, dg);
    }
}

}  // namespace wwws
