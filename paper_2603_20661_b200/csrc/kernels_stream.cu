// The fused step for large launches: dispatch + duel-and-judge + settlement as a stream of
// phases, so that every phase runs with (nearly) all 32 lanes of a warp busy.
//
// With one thread walking one request from start to end, lanes idle whenever their request is
// done with a part the others are still in: requests served locally sit through the scoring of
// the others, one refused probe keeps 31 lanes waiting for the redraw, one duel keeps them
// waiting for a challenger and three judges.  Here a warp owns a run of consecutive requests of
// one replica and takes them through five phases, each of which works on up to 32 DIFFERENT
// requests that are all at that point of the protocol:
//
//   origin   D1, D2, D3   online? offload? which candidate block?          -> score queue | finish queue
//   score    D4           the 32 candidates of the window, one thread per request (fp32 scores and
//                         four group sums into shared memory)                -> draw queue
//   draw     D5, D6, J2   ONE proportional draw, and what the request's stage does with the pick:
//                         probe it (executor, challenger) or check that it is online (judge)
//                                                                            -> draw | vote | finish queue
//   vote     J3, S3       judge votes and the duel's part of the settlement  -> finish queue
//   finish   S1, S2, S4   result record, settlement, counters
//
// The queues live in the warp's own shared memory, so there is no block-wide barrier and no
// atomic; a phase is run when 32 requests wait for it (later phases first, so queues stay short),
// and with fewer only once the warp's input is exhausted.  A request that was refused simply goes
// to the tail of the draw queue and its lane is taken by another request in the next round.
// Results are identical to the other step kernels: every random number is keyed by the request,
// never by the lane or the order of processing, and all updates are commutative.
#include "request_common.cuh"

namespace wwws {

#ifndef WWWS_STREAM_SLOTS
#define WWWS_STREAM_SLOTS 64
#endif
constexpr uint32_t kSlots = WWWS_STREAM_SLOTS;   // scored windows a warp holds at a time (draw + vote queues), 33..64
constexpr uint32_t kQ = 64;            // capacity of the score and finish queues

// meta word of a slot: draws used (8) | probes used (8) | stage (2) | judges found (3) | near-boundary (1)
// picks word of a slot: candidate index (5 bits each) of executor, challenger, judges 0..3
// where word: origin (16) | candidate block (11) | duel flag | origin has no capacity
constexpr uint32_t kWhereDuel = 1u << 27, kWhereNoCap = 1u << 28;
// finish entry: x = index in the batch, y = exec_a, z = exec_b (16 bits, 0xffff none) | block << 16,
// w = judges' candidate indices (4 x 5) | judges (3) << 20 | outcome (3) << 23 | near << 26 | probes (4) << 27

struct alignas(16) WarpPool {
    float S[kWin][kSlots];                     // scores still in play, [candidate][slot]
    unsigned long long G[4][kSlots];           // integer weight sums of the four 8-candidate groups
    unsigned long long ycache[kSlots];         // second 64-bit value of the draw pair in use
    uint4 q_fin[kQ];
    uint2 q_score[kQ];                         // (index in the batch, where word)
    uint32_t ident[kSlots], where[kSlots], meta[kSlots], picks[kSlots];
    uint8_t q_draw[kSlots], q_vote[kSlots], free_slots[kSlots];
};

struct Warp {                                  // warp-uniform scheduling state, in registers
    uint32_t sc_head, sc_n, dr_head, dr_n, vo_head, vo_n, fi_head, fi_n, n_free;
    uint32_t chunk, n_chunks, stride, count;   // next 32-request chunk of the batch this warp starts; chunks go round the replica's warps
    uint32_t r, rg, lane, lt;                  // replica, global replica, lane, mask of the lower lanes
    uint64_t first;
    size_t xbase, pbase;                       // replica's offset into the request arrays (+ first) and into the per-peer tables
};

// Counters of all the requests a thread finishes (a thread may finish hundreds).
struct WideAcc {
    uint32_t c[sSloMet + 1];                   // indexed by the counter's number, sRequests .. sSloMet (probes apart)
    uint32_t probes;
    unsigned long long sum_lat, digest;
    __device__ __forceinline__ void add(uint32_t k, uint32_t v = 1u)
    {
        if (k == sProbes) probes += v; else c[k] += v;
    }
};
static_assert(sProbes < sSloMet && sNear < sSloMet && sJudgeEvals < sSloMet, "the event counters come first");

struct E4 { uint32_t lo[4], hi[4]; };
__device__ __forceinline__ E4 ld_entries(const char* p)            // four view entries = 32 bytes, read once
{
    unsigned long long a, b, c, d;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u64 {%0,%1,%2,%3}, [%4];" : "=l"(a), "=l"(b), "=l"(c), "=l"(d) : "l"(p));
    E4 v;
    v.lo[0] = uint32_t(a); v.hi[0] = uint32_t(a >> 32); v.lo[1] = uint32_t(b); v.hi[1] = uint32_t(b >> 32);
    v.lo[2] = uint32_t(c); v.hi[2] = uint32_t(c >> 32); v.lo[3] = uint32_t(d); v.hi[3] = uint32_t(d >> 32);
    return v;
}

// ---- origin: D1, D2, D3 ---------------------------------------------------------------------------
template <bool SCORES>
__device__ __forceinline__ void phase_origin(const Net& n, WarpPool& p, Warp& w)
{
    const uint32_t m = min(32u, w.count - 32u * w.chunk);
    const bool active = w.lane < m;
    const uint32_t idx = 32u * w.chunk + w.lane;
    bool offload = false;
    int code = -3;
    uint32_t where = 0;
    if (active) {
        const size_t x = w.xbase + idx;
        const uint32_t o = n.origin[x];
        const Rnd4 rx = draw(n, uint32_t(w.first + idx), 0, w.rg, kOrigin);
        if (o >= n.N) set_error(n, eArg, o);
        else {
            const uint32_t g = reinterpret_cast<const uint32_t*>(n.gate)[2 * (w.pbase + o) + 1];
            if (g & kGateOnline) {
                code = (g & kGateNoCap) ? -4 : -1;
                if (ppm(rx.w[0]) < (g & kGateFreq)) {
                    offload = true;
                    where = o | pick_block(n, o, rx.w[2]) << 16 | (ppm(rx.w[1]) < n.p_duel ? kWhereDuel : 0u) | (code == -4 ? kWhereNoCap : 0u);
                }
            }
        }
        if (SCORES) {
            if (n.score_a) n.score_a[x] = 0.0f;
            if (n.score_sum) n.score_sum[x] = 0.0f;
        }
    }
    const uint32_t mo = __ballot_sync(kFull, offload), ml = __ballot_sync(kFull, active && !offload);
    if (offload) p.q_score[(w.sc_head + w.sc_n + __popc(mo & w.lt)) & (kQ - 1)] = make_uint2(idx, where);
    if (active && !offload) p.q_fin[(w.fi_head + w.fi_n + __popc(ml & w.lt)) & (kQ - 1)] = make_uint4(idx, uint32_t(code), 0xffffu, 0u);
    w.sc_n += __popc(mo); w.fi_n += __popc(ml); w.chunk += w.stride;
}

// ---- score: D4 ------------------------------------------------------------------------------------
template <bool SCORES, bool LOAD>
__device__ __forceinline__ void phase_score(const Net& n, WarpPool& p, Warp& w, uint32_t m)
{
    const bool active = w.lane < m;
    if (active) {
        const uint2 e = p.q_score[(w.sc_head + w.lane) & (kQ - 1)];
        uint32_t slot = p.free_slots[w.n_free - 1u - w.lane];
        if (!index_ok(n, slot, kSlots, 503)) slot = 0;
        const uint32_t o = e.y & 0xffffu, blk = (e.y >> 16) & 0x7ffu;
        const char* row = reinterpret_cast<const char*>(n.view + (w.pbase + o) * n.ld + kWin * blk);
        const float4* wl4 = reinterpret_cast<const float4*>(n.w_led + size_t(w.r) * n.ld + kWin * blk);
        const uint32_t self = (o >> 5) == blk ? (o & 31u) : 32u;
        float ssum = 0.0f;
#pragma unroll 1
        for (int g = 0; g < 4; ++g) {                                  // one 8-candidate group at a time: two 32-byte loads in flight
            E4 v[2];
            float4 f[2];
#pragma unroll
            for (int i = 0; i < 2; ++i) v[i] = ld_entries(row + 64 * g + 32 * i);
#pragma unroll
            for (int i = 0; i < 2; ++i) f[i] = __ldg(wl4 + 2 * g + i);
            unsigned long long gsum = 0;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const uint32_t c = 8u * g + k;
                const float wl = (k & 3) == 0 ? f[k >> 2].x : (k & 3) == 1 ? f[k >> 2].y : (k & 3) == 2 ? f[k >> 2].z : f[k >> 2].w;
                float sc = candidate_score<LOAD>(n, v[k >> 2].lo[k & 3], v[k >> 2].hi[k & 3], wl);
                if (SCORES) sc = self != c ? sc : 0.0f;            // the checked sum leaves the origin out as it goes
                p.S[c][slot] = sc;
                gsum += weight_q(sc);
                if (SCORES) ssum = __fadd_rn(ssum, sc);
            }
            p.G[g][slot] = gsum;
        }
        if (!SCORES && self < 32u) {
            // the origin is not a candidate of its own request: take it out of its window
            const unsigned long long ws = weight_q(p.S[self][slot]);
            p.S[self][slot] = 0.0f;
            p.G[self >> 3][slot] -= ws;
        }
        p.ident[slot] = e.x; p.where[slot] = e.y; p.meta[slot] = 0u; p.picks[slot] = 0u;
        if (SCORES && n.score_sum) n.score_sum[w.xbase + e.x] = ssum;
        p.q_draw[(w.dr_head + w.dr_n + w.lane) % kSlots] = uint8_t(slot);
    }
    w.sc_head += m; w.sc_n -= m; w.n_free -= m; w.dr_n += m;
}

// ---- draw: D5, D6, J2 -----------------------------------------------------------------------------
enum : int { kCont = 0, kFinNone = 1, kFinPlain = 2, kFinCancel = 3, kVote = 4, kIdle = 5 };

template <bool GREEDY, bool SCORES>
__device__ __forceinline__ void phase_draw(const Net& n, WarpPool& p, Warp& w, uint32_t m)
{
    const bool active = w.lane < m;
    // A batch normally takes every request one draw further and regroups.  Once the warp's input is
    // exhausted a partial batch has nothing left to fill its lanes with: then each lane takes its
    // request on, draw after draw, until it leaves the draw phase - fewer rounds at the end of a run,
    // which is what a launch that gives a warp only a chunk or two is made of.
    const bool run_on = m < 32u && w.chunk >= w.n_chunks;
    int kind = kIdle;
    uint32_t slot = 0;
    uint4 fin = make_uint4(0, 0, 0, 0);
    if (active) {
        slot = p.q_draw[(w.dr_head + w.lane) % kSlots];
        if (!index_ok(n, slot, kSlots, 501)) slot = 0;
        const uint32_t meta = p.meta[slot], where = p.where[slot], idx = p.ident[slot];
        uint32_t picks = p.picks[slot];
        uint32_t n_draws = meta & 0xffu, n_probes = (meta >> 8) & 0xffu, stage = (meta >> 16) & 3u, nj = (meta >> 18) & 7u;
        bool near = (meta >> 21) & 1u;
        const uint32_t blk = (where >> 16) & 0x7ffu, q = uint32_t(w.first + idx);
        const size_t cbase = w.pbase + kWin * blk;
        unsigned long long G0 = p.G[0][slot], G1 = p.G[1][slot], G2 = p.G[2][slot], G3 = p.G[3][slot];
#pragma unroll 1
        for (;;) {
            const unsigned long long S = G0 + G1 + G2 + G3;
            int pick = -1;
            if (S != 0) {
                const uint32_t k = n_draws++;
                uint32_t g;
                unsigned long long wp;
                if (GREEDY) {
                    // greedy rule: highest weight, lowest candidate on ties; flagged when the runner-up is within 1e-5
                    unsigned long long m1 = 0, m2 = 0;
#pragma unroll 4
                    for (int c = 0; c < int(kWin); ++c) {
                        const unsigned long long x = weight_q(p.S[c][slot]);
                        if (x > m1) { m2 = m1; m1 = x; pick = c; }
                        else if (x > m2) m2 = x;
                    }
                    if (m2 != 0 && m1 - m2 <= m1 / 100000ull) near = true;
                    g = uint32_t(pick) >> 3; wp = m1;
                } else {
                    unsigned long long u;
                    if (k & 1u) u = p.ycache[slot];
                    else {
                        const Rnd4 y = draw(n, q, k >> 1, w.rg, kDraw);
                        u = (unsigned long long)y.w[0] << 32 | y.w[1];
                        p.ycache[slot] = (unsigned long long)y.w[2] << 32 | y.w[3];
                    }
                    const unsigned long long r64 = __umul64hi(u, S);
                    // the group whose interval holds r64, then the candidate inside it, without branches:
                    // the pick is the number of inclusive prefix sums that do not exceed r64
                    const unsigned long long c1 = G0 + G1, c2 = c1 + G2;
                    g = uint32_t(r64 >= G0) + uint32_t(r64 >= c1) + uint32_t(r64 >= c2);
                    unsigned long long lo = g == 0 ? 0ull : g == 1 ? G0 : g == 2 ? c1 : c2, acc = lo;
                    uint32_t cnt = 0;
                    wp = 0;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const unsigned long long x = weight_q(p.S[8 * g + j][slot]);
                        const bool below = acc + x <= r64;                   // candidate j ends at or before r64
                        if (!below && cnt == uint32_t(j)) wp = x;            // the first one that does not is the pick
                        acc += x;
                        if (below) { lo = acc; ++cnt; }
                    }
                    pick = int(8u * g + cnt);
                    const unsigned long long d1 = r64 - lo, d2 = lo + wp - 1 - r64;
                    if ((d1 < d2 ? d1 : d2) <= S / 100000ull) near = true;
                    if (cnt >= 8u) pick = -1;                                // cannot happen: the group sums are the sums of the weights in play
                }
                if (pick >= 0) {
                    if (SCORES && stage == 0 && n.score_a) fin.x = __float_as_uint(p.S[pick][slot]);     // the executor's score, if this pick accepts
                    p.S[pick][slot] = 0.0f;
                    if (g == 0) G0 -= wp; else if (g == 1) G1 -= wp; else if (g == 2) G2 -= wp; else G3 -= wp;
                }
            }
            if (pick >= 0 && !index_ok(n, kWin * blk + uint32_t(pick), n.N, 502)) pick = -1;
            kind = kCont;
            if (pick < 0) kind = stage == 0 ? kFinNone : (stage == 2 && nj ? kVote : kFinCancel);
            else if (stage < 2) {
                ++n_probes;
                // D6: the drawn candidate answers by its true state and its own accept policy (its gate)
                const uint32_t thr = reinterpret_cast<const uint32_t*>(n.gate)[2 * (cbase + pick)];
                const Rnd4 y = draw(n, q, uint32_t(pick) >> 2, w.rg, kProbe);
                const uint32_t sel = uint32_t(pick) & 3u;
                const bool accepted = ppm(sel == 0 ? y.w[0] : sel == 1 ? y.w[1] : sel == 2 ? y.w[2] : y.w[3]) < thr;
                if (accepted) {
                    if (stage == 0) {
                        picks = uint32_t(pick);
                        if (SCORES && n.score_a) n.score_a[w.xbase + idx] = __uint_as_float(fin.x);
                        if (where & kWhereDuel) { stage = 1; if (n_probes >= n.max_probes) kind = kFinCancel; }
                        else kind = kFinPlain;
                    } else { picks |= uint32_t(pick) << 5; stage = 2; }
                } else if (n_probes >= n.max_probes) kind = stage == 0 ? kFinNone : kFinCancel;
            } else {
                if (n.online[cbase + pick]) { picks |= uint32_t(pick) << (10u + 5u * nj); ++nj; }
                if (nj >= n.n_judges) kind = kVote;
            }
            if (!(run_on && kind == kCont)) break;
        }
        if (kind == kCont || kind == kVote) {
            p.G[0][slot] = G0; p.G[1][slot] = G1; p.G[2][slot] = G2; p.G[3][slot] = G3;
            p.meta[slot] = n_draws | n_probes << 8 | stage << 16 | nj << 18 | (near ? 1u << 21 : 0u);
            p.picks[slot] = picks;
        } else {
            const int a = kind == kFinNone ? ((where & kWhereNoCap) ? -4 : -2) : int(kWin * blk + (picks & 31u));
            fin = make_uint4(idx, uint32_t(a), 0xffffu | blk << 16,
                             (kind == kFinCancel ? 4u << 23 : 0u) | (near ? 1u << 26 : 0u) | n_probes << 27);
        }
    }
    const bool to_fin = kind == kFinNone || kind == kFinPlain || kind == kFinCancel;
    __syncwarp();                               // every lane has read its queue entry: the ring's head may be reused by the pushes below
    const uint32_t mc = __ballot_sync(kFull, kind == kCont), mv = __ballot_sync(kFull, kind == kVote), mf = __ballot_sync(kFull, to_fin);
    w.dr_head += m; w.dr_n -= m;
    if (kind == kCont) p.q_draw[(w.dr_head + w.dr_n + __popc(mc & w.lt)) % kSlots] = uint8_t(slot);
    if (kind == kVote) p.q_vote[(w.vo_head + w.vo_n + __popc(mv & w.lt)) % kSlots] = uint8_t(slot);
    if (to_fin) {
        p.q_fin[(w.fi_head + w.fi_n + __popc(mf & w.lt)) & (kQ - 1)] = fin;
        p.free_slots[w.n_free + __popc(mf & w.lt)] = uint8_t(slot);
    }
    w.dr_n += __popc(mc); w.vo_n += __popc(mv); w.fi_n += __popc(mf); w.n_free += __popc(mf);
}

// ---- vote: J3 and the duel's part of the settlement (S3) --------------------------------------------
__device__ __forceinline__ void phase_vote(const Net& n, WarpPool& p, Warp& w, uint32_t m, WideAcc& acc)
{
    const bool active = w.lane < m;
    if (active) {
        uint32_t slot = p.q_vote[(w.vo_head + w.lane) % kSlots];
        if (!index_ok(n, slot, kSlots, 504)) slot = 0;
        const uint32_t meta = p.meta[slot], where = p.where[slot], idx = p.ident[slot], picks = p.picks[slot];
        const uint32_t blk = (where >> 16) & 0x7ffu, o = where & 0xffffu, q = uint32_t(w.first + idx);
        const uint32_t nj = (meta >> 18) & 7u;
        const int a = int(kWin * blk + (picks & 31u)), b = int(kWin * blk + ((picks >> 5) & 31u));
        int jd[4];
#pragma unroll
        for (int l = 0; l < 4; ++l) jd[l] = uint32_t(l) < nj ? int(kWin * blk + ((picks >> (10 + 5 * l)) & 31u)) : -1;
        const unsigned long long thr = ((1ull << 32) + n.quality[w.pbase + a] - n.quality[w.pbase + b]) >> 1;
        uint32_t votes_a = 0;
#pragma unroll 1
        for (uint32_t l = 0; l < nj; ++l) {
            const Rnd4 y = draw(n, q, l, w.rg, kJudge);
            bool va = (unsigned long long)y.w[0] < thr;
            if (ppm(y.w[1]) < n.p_noise) va = !va;
            votes_a += va;
        }
        const uint32_t oc = 2u * votes_a > nj ? 1u : (2u * votes_a < nj ? 2u : 3u);
        const size_t x = w.xbase + idx;
        const long long extra = settle_duel(n, w.r, q, o, n.len_in[x], n.len_out[x], a, b, jd, oc, acc);
        add64(&n.d_credit[w.pbase + o], -extra);
        p.q_fin[(w.fi_head + w.fi_n + w.lane) & (kQ - 1)] =
            make_uint4(idx, uint32_t(a), uint32_t(b) | blk << 16,
                       ((picks >> 10) & 0xfffffu) | nj << 20 | oc << 23 | ((meta >> 21) & 1u) << 26 | ((meta >> 8) & 15u) << 27);
        p.free_slots[w.n_free + w.lane] = uint8_t(slot);
    }
    w.vo_head += m; w.vo_n -= m; w.fi_n += m; w.n_free += m;
}

// ---- finish: result record, S1, S2, S4 -----------------------------------------------------------------
__device__ __forceinline__ void phase_finish(const Net& n, WarpPool& p, Warp& w, uint32_t m, WideAcc& acc)
{
    if (w.lane < m) {
        const uint4 e = p.q_fin[(w.fi_head + w.lane) & (kQ - 1)];
        const uint32_t idx = e.x, blk = e.z >> 16, nj = (e.w >> 20) & 7u, oc = (e.w >> 23) & 7u;
        const int a = int(e.y), b = (e.z & 0xffffu) == 0xffffu ? -1 : int(e.z & 0xffffu);
        const bool near = (e.w >> 26) & 1u;
        int jd[4];
#pragma unroll
        for (int l = 0; l < 4; ++l) jd[l] = uint32_t(l) < nj ? int(kWin * blk + ((e.w >> (5 * l)) & 31u)) : -1;
        const size_t x = w.xbase + idx;
        n.exec_a[x] = a; n.exec_b[x] = b; n.outcome[x] = uint8_t(oc); n.rflags[x] = near ? 1 : 0;
        *reinterpret_cast<int4*>(n.judges + 4 * x) = make_int4(jd[0], jd[1], jd[2], jd[3]);
        acc.probes += e.w >> 27;
        settle_one(n, w.r, uint32_t(w.first + idx), idx, n.origin[x], n.len_in[x], n.len_out[x], a, b, jd, oc, near, acc,
                   /*duel_booked=*/oc >= 1u && oc <= 3u);
    }
    w.fi_head += m; w.fi_n -= m;
}

enum : int { phOrigin, phScore, phDraw, phVote, phFinish, phDone };

template <bool GREEDY, bool SCORES, bool LOAD>
__global__ void __launch_bounds__(32, kSlots > 48 ? 16 : kSlots > 40 ? 19 : 22) k_step_stream(Net n, uint64_t first, uint32_t count)
{
    grid_dependency_enter();
    __shared__ WarpPool p;
    Warp w;
    w.lane = threadIdx.x; w.lt = (1u << w.lane) - 1u;
    w.r = blockIdx.y; w.rg = w.r + n.replica_offset; w.first = first;
    w.xbase = size_t(w.r) * n.Q + first; w.pbase = size_t(w.r) * n.N;
    w.count = count; w.n_chunks = (count + 31u) / 32u;
    w.chunk = blockIdx.x; w.stride = gridDim.x;
    w.sc_head = w.sc_n = w.dr_head = w.dr_n = w.vo_head = w.vo_n = w.fi_head = w.fi_n = 0;
    w.n_free = kSlots;
    p.free_slots[w.lane] = uint8_t(w.lane);
    if (w.lane + 32u < kSlots) p.free_slots[w.lane + 32] = uint8_t(w.lane + 32);
    WideAcc acc;
#pragma unroll
    for (int k = 0; k <= int(sSloMet); ++k) acc.c[k] = 0;
    acc.probes = 0; acc.sum_lat = 0; acc.digest = 0;

    // A phase runs when 32 requests wait for it, later phases first (queues stay short and never
    // overflow: whatever feeds the finish queue runs only while it holds fewer than 32 entries,
    // and the score queue is fed only while it holds fewer than 32).  Each phase's code exists once.
#pragma unroll 1
    for (;;) {
        int ph = phDone;
        uint32_t m = 32u;
        if (w.fi_n >= 32u) ph = phFinish;
        else if (w.vo_n >= 32u) ph = phVote;
        else if (w.dr_n >= 32u) ph = phDraw;
        else if (w.sc_n >= 32u) {
            if (w.n_free >= 32u) ph = phScore;
            // all windows taken: the draw and vote queues hold more than 32 between them, so the longer is at least half a warp
            else if (w.dr_n >= w.vo_n) { ph = phDraw; m = w.dr_n; }
            else { ph = phVote; m = w.vo_n; }
        }
        else if (w.chunk < w.n_chunks) ph = phOrigin;
        // input exhausted: what is left runs in partial batches, earlier phases first so that the later ones fill up
        else if (w.sc_n && w.n_free) { ph = phScore; m = min(w.sc_n, w.n_free); }
        else if (w.dr_n) { ph = phDraw; m = w.dr_n; }
        else if (w.vo_n) { ph = phVote; m = w.vo_n; }
        else if (w.fi_n) { ph = phFinish; m = w.fi_n; }
        if (ph == phDone) break;
        __syncwarp();
        switch (ph) {
        case phOrigin: phase_origin<SCORES>(n, p, w); break;
        case phScore: phase_score<SCORES, LOAD>(n, p, w, m); break;
        case phDraw: phase_draw<GREEDY, SCORES>(n, p, w, m); break;
        case phVote: phase_vote(n, p, w, m, acc); break;
        default: phase_finish(n, p, w, m, acc); break;
        }
    }

    // counters: one warp reduction and one atomic per counter
    unsigned long long* st = n.stats + size_t(w.r) * sCount;
#pragma unroll
    for (uint32_t k = 0; k <= sSloMet; ++k) {                       // c[] is indexed by the counter's number
        const uint32_t v = __reduce_add_sync(kFull, k == sProbes ? acc.probes : acc.c[k]);
        if (w.lane == 0 && v) atomicAdd(&st[k], (unsigned long long)v);
    }
    unsigned long long sl = acc.sum_lat, dg = acc.digest;
#pragma unroll
    for (int o = 16; o; o >>= 1) { sl += __shfl_down_sync(kFull, sl, o); dg += __shfl_down_sync(kFull, dg, o); }
    if (w.lane == 0) {
        if (sl) atomicAdd(&st[sSumLat], sl);
        if (dg) atomicAdd(&st[sPendingDigest], dg);
    }
}

// Warps per replica: all warps of the launch are resident at once (one wave: no tail), and a
// replica's 32-request chunks go round its warps, so every warp gets the same number of them
// (give or take one).  More chunks per warp is what lets the phases run full.
// `run` (WWWS_OPT_STREAM_RUN) instead fixes the requests per warp.
static uint32_t stream_warps_per_replica(const Net& n, uint32_t count, uint32_t run, int resident_warps)
{
    const uint32_t chunks = (count + 31u) / 32u;
    uint32_t g = run ? (count + run - 1u) / run : uint32_t(resident_warps) / n.Rp;
    if (g < 1u) g = 1u;
    return g > chunks ? chunks : g;
}

template <bool GREEDY, bool SCORES, bool LOAD>
static void launch_stream_variant(const Net& n, uint64_t first, uint32_t count, uint32_t run, const LaunchCtx& c)
{
    static const int resident = [] {
        int dev = 0, sms = 0, per_sm = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_step_stream<GREEDY, SCORES, LOAD>, 32, 0);
        return sms * per_sm > 0 ? sms * per_sm : 148 * 15;
    }();
    const dim3 grid(stream_warps_per_replica(n, count, run, resident), n.Rp);
    // A plain stream-ordered launch: this kernel wants the SM's whole shared memory, and blocks that
    // arrive while the previous kernel's blocks still hold the SM in another shared-memory
    // configuration get a fraction of the occupancy for their whole (long) life.
    LaunchCtx plain = c;
    plain.overlap = false;
    launch_kernel(plain, k_step_stream<GREEDY, SCORES, LOAD>, grid, 32, n, first, count);
}

template <bool GREEDY, bool SCORES>
static void launch_stream_load(const Net& n, uint64_t first, uint32_t count, uint32_t run, const LaunchCtx& c)
{
    if (n.flags & 2u) launch_stream_variant<GREEDY, SCORES, true>(n, first, count, run, c);
    else launch_stream_variant<GREEDY, SCORES, false>(n, first, count, run, c);
}

void launch_step_stream(const Net& n, uint64_t first, uint32_t count, uint32_t run, const LaunchCtx& c)
{
    Timed t(c, kStepFused);
    const bool scores = n.score_a || n.score_sum;
    if (n.flags & 4u) {
        if (scores) launch_stream_load<true, true>(n, first, count, run, c);
        else launch_stream_load<true, false>(n, first, count, run, c);
    } else {
        if (scores) launch_stream_load<false, true>(n, first, count, run, c);
        else launch_stream_load<false, false>(n, first, count, run, c);
    }
}

}  // namespace wwws
