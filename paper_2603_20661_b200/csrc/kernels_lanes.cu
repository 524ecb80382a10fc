// The fused step for small launches: L lanes per request instead of one thread.
//
// A launch of a few thousand requests leaves most of the GPU empty, and a thread that scores 32
// candidates and then walks the draw / probe / duel / settle chain alone is bound by the length of
// that chain.  Here a request is shared by L adjacent lanes (4 or 8): each lane scores 32 / L
// contiguous candidates and keeps their fp32 scores in registers (no shared memory for weights),
// a proportional draw is a prefix sum over the L lanes followed by a short scan inside the lane
// that owns the drawn interval, and everything that is the same for the whole request (origin
// decision, Philox words, the probe of the drawn peer, judge votes) is computed by all L lanes
// alike, so the group never diverges; lane 0 of the group writes the results and settles.
// Results are identical to the other request kernels: the intervals of a draw are the same
// candidate-ascending prefix sums, whoever holds them.
#include "request_common.cuh"

namespace wwws {

template <int L> struct Lanes {
    static constexpr int CP = 32 / L;                 // candidates per lane
    float sc[CP];                                     // scores still in play (0 = drawn or never eligible)
    uint64_t mine;                                    // sum of this lane's integer weights
    uint32_t n_draws, n_probes;
    bool near;
    Rnd4 y; uint32_t y_slot;
    unsigned gmask;                                   // the L lanes of this request within the warp
    uint32_t sub, lane0;                              // lane index inside the group; warp lane of the group's first lane
};

__device__ __forceinline__ uint64_t shfl64(unsigned mask, uint64_t v, int src)
{
    return uint64_t(__shfl_sync(mask, uint32_t(v >> 32), src)) << 32 | __shfl_sync(mask, uint32_t(v), src);
}

// Scores this lane's candidates of the window (o, blk); returns the lane-ascending fp32 sum of all
// 32 scores (the same order of additions as a single thread would use) when `want_sum`.
template <int L, bool LOAD>
__device__ __forceinline__ float score_lanes(const Net& n, Lanes<L>& w, uint32_t r, uint32_t o, uint32_t blk, bool want_sum)
{
    constexpr int CP = Lanes<L>::CP;
    const uint32_t c0 = w.sub * CP;
    const uint64_t* win = n.view + (size_t(r) * n.N + o) * n.ld + kWin * blk + c0;
    const float* wled = n.w_led + size_t(r) * n.ld;
    uint64_t e[CP];
#pragma unroll
    for (int j = 0; j < CP; j += 4) {
        const ulonglong4 e4 = *reinterpret_cast<const ulonglong4*>(win + j);
        e[j] = e4.x; e[j + 1] = e4.y; e[j + 2] = e4.z; e[j + 3] = e4.w;
    }
    w.mine = 0;
#pragma unroll
    for (int j = 0; j < CP; ++j) {
        const uint32_t id = kWin * blk + c0 + j;
        float sc = candidate_score<LOAD>(n, uint32_t(e[j]), uint32_t(e[j] >> 32), wled[id]);   // padding columns: entry 0, weight 0
        if (id == o) sc = 0.0f;                                            // the origin is not a candidate of its own request
        w.sc[j] = sc;
        w.mine += weight_q(sc);
    }
    float ssum = 0.0f;
    if (want_sum) {
        // candidate-ascending chain of additions, handed from lane to lane
        for (int l = 0; l < L; ++l) {
            if (int(w.sub) == l) {
#pragma unroll
                for (int j = 0; j < CP; ++j) ssum = __fadd_rn(ssum, w.sc[j]);
            }
            ssum = __shfl_sync(w.gmask, ssum, int(w.lane0) + l);
        }
    }
    return ssum;
}

// D5 for a group of lanes: returns the drawn candidate (0..31, the same in all lanes) or -1.
template <int L>
__device__ __forceinline__ int draw_lanes(const Net& n, Lanes<L>& w, uint32_t q, uint32_t rg)
{
    constexpr int CP = Lanes<L>::CP;
    // inclusive prefix sum of the lanes' weight sums, candidate-ascending
    uint64_t incl = w.mine;
#pragma unroll
    for (int d = 1; d < L; d <<= 1) {
        const uint64_t t = uint64_t(__shfl_up_sync(w.gmask, uint32_t(incl >> 32), d, L)) << 32 | __shfl_up_sync(w.gmask, uint32_t(incl), d, L);
        if (int(w.sub) >= d) incl += t;
    }
    const uint64_t S = shfl64(w.gmask, incl, int(w.lane0) + L - 1);
    if (S == 0) return -1;
    const uint32_t k = w.n_draws++;
    int pick = -1;
    bool near = false;
    if (n.flags & 4u) {
        // greedy rule: highest weight, lowest candidate on ties; flagged when the runner-up is within 1e-5
        uint64_t m = 0, m2 = 0;
        int at = 32;
#pragma unroll
        for (int j = 0; j < CP; ++j) {
            const uint64_t x = weight_q(w.sc[j]);
            if (x > m) { m2 = m; m = x; at = int(w.sub) * CP + j; }
            else if (x > m2) m2 = x;
        }
#pragma unroll
        for (int d = 1; d < L; d <<= 1) {
            const uint64_t om = uint64_t(__shfl_xor_sync(w.gmask, uint32_t(m >> 32), d)) << 32 | __shfl_xor_sync(w.gmask, uint32_t(m), d);
            const uint64_t om2 = uint64_t(__shfl_xor_sync(w.gmask, uint32_t(m2 >> 32), d)) << 32 | __shfl_xor_sync(w.gmask, uint32_t(m2), d);
            const int oat = __shfl_xor_sync(w.gmask, at, d);
            if (om > m || (om == m && oat < at)) { m2 = m > om2 ? m : om2; m = om; at = oat; }
            else m2 = om > m2 ? om : m2;
        }
        pick = at;
        near = m2 != 0 && m - m2 <= m / 100000ull;
        if (pick / CP == int(w.sub)) {
#pragma unroll
            for (int j = 0; j < CP; ++j) if (j == pick % CP) w.sc[j] = 0.0f;
            w.mine -= m;
        }
    } else {
        if (w.y_slot != (k >> 1)) { w.y = draw(n, q, k >> 1, rg, kDraw); w.y_slot = k >> 1; }
        const uint64_t u = (k & 1u) ? (uint64_t(w.y.w[2]) << 32 | w.y.w[3]) : (uint64_t(w.y.w[0]) << 32 | w.y.w[1]);
        const uint64_t r64 = __umul64hi(u, S);
        uint64_t lo = incl - w.mine;
        const bool owner = r64 >= lo && r64 < incl;                        // exactly one lane: the intervals tile [0, S)
        int local = -1;
        if (owner) {
            uint64_t wp = 0;
#pragma unroll
            for (int j = 0; j < CP; ++j) {
                const uint64_t x = weight_q(w.sc[j]);
                if (local < 0) {
                    if (r64 < lo + x) { local = j; wp = x; }
                    else lo += x;
                }
            }
            const uint64_t m1 = r64 - lo, m2 = lo + wp - 1 - r64;
            near = (m1 < m2 ? m1 : m2) <= S / 100000ull;
#pragma unroll
            for (int j = 0; j < CP; ++j) if (j == local) w.sc[j] = 0.0f;
            w.mine -= wp;
            local += int(w.sub) * CP;
        }
        const unsigned who = __ballot_sync(w.gmask, owner) & w.gmask;
        const int src = __ffs(who) - 1;
        pick = __shfl_sync(w.gmask, local, src);
        near = __shfl_sync(w.gmask, int(near), src) != 0;
    }
    if (near) w.near = true;
    return pick;
}

template <int L, bool LOAD>
__global__ void __launch_bounds__(128) k_step_lanes(Net n, uint64_t first, uint32_t count)
{
    grid_dependency_enter();
    constexpr int RPB = 128 / L;                       // requests per block
    __shared__ BlockStats bs;
    stats_begin(bs);                                   // barrier inside
    const uint32_t r = blockIdx.y, rg = r + n.replica_offset;
    const size_t pbase = size_t(r) * n.N;
    const uint32_t idx = blockIdx.x * RPB + threadIdx.x / L;
    SettleAcc acc; acc_zero(acc);
    Lanes<L> w;
    w.sub = threadIdx.x % L;
    w.lane0 = (threadIdx.x & 31u) - w.sub;
    w.gmask = (L == 32 ? 0xffffffffu : ((1u << L) - 1u)) << w.lane0;
    w.mine = 0; w.n_draws = 0; w.n_probes = 0; w.near = false; w.y_slot = 0xffffffffu;
#pragma unroll
    for (int j = 0; j < Lanes<L>::CP; ++j) w.sc[j] = 0.0f;

    if (idx < count) {                                 // the same for all lanes of a group
        const uint32_t q = uint32_t(first + idx);
        const size_t x = size_t(r) * n.Q + first + idx;
        const uint32_t o = n.origin[x];
        const Rnd4 rx = draw(n, q, 0, rg, kOrigin);
        int a, b = -1;
        int jd[4] = { -1, -1, -1, -1 };
        uint32_t oc = 0, blk = 0;
        float sa = 0.0f, ssum = 0.0f;
        if (origin_gate(n, r, o, rx, a)) {
            const int local_code = a;
            blk = pick_block(n, o, rx.w[2]);
            ssum = score_lanes<L, LOAD>(n, w, r, o, blk, n.score_sum != nullptr);
            // D5, D6: draw and probe until a peer accepts; for a duel go on with the challenger and the judges
            const bool duel = ppm(rx.w[1]) < n.p_duel;
            int found = -1, nj = 0, stage = 0;         // stage 0: executor, 1: challenger, 2: judges
            a = -1;
            for (;;) {
                if (stage < 2) { if (w.n_probes >= n.max_probes) break; }
                else if (nj >= int(n.n_judges)) break;
                const int pick = draw_lanes<L>(n, w, q, rg);
                if (pick < 0) break;
                const int id = int(kWin * blk + pick);
                if (stage < 2) {
                    w.n_probes++;
                    if (probe_gate(n, r, rg, q, blk, pick)) {
                        if (stage == 0) {
                            a = id;
                            if (!duel) break;
                            stage = 1;
                        } else { found = id; stage = 2; }
                    }
                } else if (n.online[pbase + id]) {
                    if (nj == 0) jd[0] = id; else if (nj == 1) jd[1] = id; else if (nj == 2) jd[2] = id; else jd[3] = id;
                    ++nj;
                }
            }
            if (a >= 0) {
                if (n.score_a) candidate_weight(n, o, uint32_t(a), n.view[(pbase + o) * n.ld + a], n.w_led[size_t(r) * n.ld + a], sa);
                if (duel) {
                    oc = 4;
                    if (found >= 0 && nj > 0) {
                        b = found;
                        const uint64_t thr = ((1ull << 32) + n.quality[pbase + a] - n.quality[pbase + b]) >> 1;
                        int votes_a = 0;
                        for (int l = 0; l < nj; ++l) {
                            const Rnd4 y = draw(n, q, uint32_t(l), rg, kJudge);
                            bool va = uint64_t(y.w[0]) < thr;
                            if (ppm(y.w[1]) < n.p_noise) va = !va;
                            votes_a += va;
                        }
                        oc = 2 * votes_a > nj ? 1u : (2 * votes_a < nj ? 2u : 3u);
                    } else jd[0] = jd[1] = jd[2] = jd[3] = -1;
                }
            } else a = local_code == -4 ? -4 : -2;
        }
        if (w.sub == 0) {
            n.exec_a[x] = a; n.exec_b[x] = b; n.outcome[x] = uint8_t(oc); n.rflags[x] = w.near ? 1 : 0;
            *reinterpret_cast<int4*>(n.judges + 4 * x) = make_int4(jd[0], jd[1], jd[2], jd[3]);
            if (n.score_a) n.score_a[x] = sa;
            if (n.score_sum) n.score_sum[x] = ssum;
            acc.probes += w.n_probes;
            settle_one(n, r, q, idx, o, n.len_in[x], n.len_out[x], a, b, jd, oc, w.near, acc);
        }
    }
    acc_flush_warp(bs, acc);
    stats_end(n, bs, r);
}

// Lanes per request for a launch of `total` requests over all replicas, or 0 when the launch is
// large enough for the streaming kernel.  Measured on 148 SMs (4,096-peer network, 1,000 requests per
// replica), 8 lanes / 4 lanes / streaming: 2,000 requests 20.9 / 24.0 / 25.1 us; 8,000: 23.0 / 26.1 /
// 25.4; 12,000: 24.4 / 27.1 / 26.8; 16,000: 30.6 / 27.5 / 27.1; 24,000: 36.0 / 29.1 / 27.8;
// 32,000: 41.5 / 38.7 / 29.1.  Four lanes per request are never the fastest any more and remain as
// an implementation that can be forced (WWWS_OPT_STEP_KERNEL).
int step_lanes_for(uint64_t total)
{
    return total <= 12288 ? 8 : 0;
}

void launch_step_lanes(const Net& n, uint64_t first, uint32_t count, int lanes, const LaunchCtx& c)
{
    Timed t(c, kStepFused);
    const bool load = (n.flags & 2u) != 0;
    if (lanes == 8) {
        if (load) launch_kernel(c, k_step_lanes<8, true>, dim3((count + 15) / 16, n.Rp), 128, n, first, count);
        else launch_kernel(c, k_step_lanes<8, false>, dim3((count + 15) / 16, n.Rp), 128, n, first, count);
    } else {
        if (load) launch_kernel(c, k_step_lanes<4, true>, dim3((count + 31) / 32, n.Rp), 128, n, first, count);
        else launch_kernel(c, k_step_lanes<4, false>, dim3((count + 31) / 32, n.Rp), 128, n, first, count);
    }
}

}  // namespace wwws
