// The fused step kernel: dispatch + duel-and-judge + settlement, one thread per request.
//
// Fusing is legal because every update of a batch goes to a pending column (d_credit, d_wins,
// d_duels, d_backlog) or a counter, while all decisions read the state as it stood when the
// batch started.
//
// A thread scores its request's 32 candidates serially (the window is 256 contiguous bytes of
// the origin's view row: eight 32-byte loads) and keeps the fp32 scores in shared memory (the
// integer weight is a function of the score alone and is recomputed where it is read: 4 bytes per
// candidate instead of 8), laid out [candidate][slot] so that lanes never conflict and so that ANY
// thread of the block can continue a request.  That is used for the duels: only a few requests per block become
// duels, so instead of letting every warp run the long duel code for one or two of its lanes,
// duel requests are queued in shared memory and picked up densely by the first threads of the
// block after a barrier.
#include "request_common.cuh"

namespace wwws {

// Resident 128-thread blocks per SM the register budget is set for: at 7 (72 registers) a
// 128,000-request launch is a single wave on 148 SMs; shared memory (18 KiB per block)
// would allow 12.
constexpr int kStepBlocksPerSM = 7;
// Unroll factor of the scoring loop over the four 8-candidate groups: 2 keeps two window loads in
// flight per thread at half the code of a full unroll.
constexpr int kScoreUnroll = 2;

template <int BT> struct StepShared {
    float S[kWin][BT];                   // fp32 scores of the candidates still in play, 0 = not in play
    BlockStats stats;
    uint32_t n_duel;
    uint16_t queue[BT];                  // slots whose request became a duel
    struct Ctx { int32_t a; uint32_t blk; uint32_t draws_probes_near; } ctx[BT];
};

// Draw state of one request, held by the thread that is working on it.
struct Draws {
    uint64_t G0, G1, G2, G3;             // sums of the four 8-candidate groups still in play
    uint32_t n_draws, n_probes;
    bool near;
    Rnd4 y; uint32_t y_slot;
};

// D5: one draw proportional to the weights still in play, by integer prefix sums: first the
// 8-candidate group, then the candidate inside it.  Returns the candidate or -1 if none is left.
template <int BT>
__device__ __forceinline__ int draw_candidate(const Net& n, StepShared<BT>& sh, uint32_t slot, Draws& d, uint32_t q, uint32_t rg)
{
    const uint64_t S = d.G0 + d.G1 + d.G2 + d.G3;
    if (S == 0) return -1;
    const uint32_t k = d.n_draws++;
    if (n.flags & 4u) {
        // greedy rule: highest weight, lowest lane on ties; flagged when the runner-up is within 1e-5
        uint64_t m = 0, m2 = 0;
        int pick = -1;
#pragma unroll 8
        for (int c = 0; c < int(kWin); ++c) {
            const uint64_t w = weight_of(sh.S[c][slot]);
            if (w > m) { m2 = m; m = w; pick = c; }
            else if (w > m2) m2 = w;
        }
        if (m2 != 0 && m - m2 <= m / 100000ull) d.near = true;
        sh.S[pick][slot] = 0.0f;
        const int g = pick >> 3;
        if (g == 0) d.G0 -= m; else if (g == 1) d.G1 -= m; else if (g == 2) d.G2 -= m; else d.G3 -= m;
        return pick;
    }
    if (d.y_slot != (k >> 1)) { d.y = draw(n, q, k >> 1, rg, kDraw); d.y_slot = k >> 1; }
    const uint64_t u = (k & 1u) ? (uint64_t(d.y.w[2]) << 32 | d.y.w[3]) : (uint64_t(d.y.w[0]) << 32 | d.y.w[1]);
    const uint64_t r64 = __umul64hi(u, S);
    uint64_t lo = 0;
    int g = 0;
    if (r64 >= lo + d.G0) { lo += d.G0; g = 1;
        if (r64 >= lo + d.G1) { lo += d.G1; g = 2;
            if (r64 >= lo + d.G2) { lo += d.G2; g = 3; } } }
    int pick = -1;
    uint64_t wp = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint64_t w = weight_of(sh.S[8 * g + j][slot]);
        if (pick < 0) {
            if (r64 < lo + w) { pick = 8 * g + j; wp = w; }
            else lo += w;
        }
    }
    const uint64_t m1 = r64 - lo, m2 = lo + wp - 1 - r64;
    if ((m1 < m2 ? m1 : m2) <= S / 100000ull) d.near = true;
    sh.S[pick][slot] = 0.0f;
    if (g == 0) d.G0 -= wp; else if (g == 1) d.G1 -= wp; else if (g == 2) d.G2 -= wp; else d.G3 -= wp;
    return pick;
}

// Scores the window of request (o, blk) into shared memory; returns the four group sums through d
// and the lane-ascending fp32 sum of the scores.
template <int BT>
__device__ __forceinline__ float score_window(const Net& n, StepShared<BT>& sh, uint32_t slot, uint32_t r, uint32_t o, uint32_t blk,
                                              uint32_t keep, Draws& d)
{
    const uint64_t* win = n.view + (size_t(r) * n.N + o) * n.ld + kWin * blk;
    const float* wled = n.w_led + size_t(r) * n.ld;
    float ssum = 0.0f;
#pragma unroll kScoreUnroll
    for (int g = 0; g < 4; ++g) {
        uint64_t gsum = 0;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int c0 = 8 * g + 4 * h;
            const ulonglong4 e4 = *reinterpret_cast<const ulonglong4*>(win + c0);     // 32 B of the window
            const uint64_t e[4] = { e4.x, e4.y, e4.z, e4.w };
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t id = kWin * blk + c0 + j;
                const float wl = id < n.N ? wled[id] : 0.0f;
                float sc;
                const uint64_t W = candidate_weight(n, o, id, e[j], wl, sc);              // sc = 0 when W = 0
                const bool in_play = keep >> (c0 + j) & 1u;                                // not drawn already (duel pass)
                sh.S[c0 + j][slot] = in_play ? sc : 0.0f;
                gsum += in_play ? W : 0ull;
                ssum = __fadd_rn(ssum, sc);                                                // lane-ascending fp32 sum
            }
        }
        if (g == 0) d.G0 = gsum; else if (g == 1) d.G1 = gsum; else if (g == 2) d.G2 = gsum; else d.G3 = gsum;
    }
    return ssum;
}

// What a launch does: the whole step, or one of the two calls it replaces on large batches.
enum : int { kModeFused = 0, kModeDispatch = 1, kModeDuel = 2 };

// The kernel makes two passes over the same code.  Pass 0: every thread takes its own request
// (origin decision, scoring, search for the executor).  Pass 1, after a barrier: the first
// threads of the block take the requests that became duels (search for the challenger, then the
// judges).  Both passes share one draw/probe loop, one result writer and one settlement, so the
// machine code holds each of those long sequences once: the kernel is bound by instruction
// fetch when many blocks at different points of a large program share an SM.
template <int BT, int MODE>
__global__ void __launch_bounds__(BT, BT == 128 ? kStepBlocksPerSM : 1) k_step_fused(Net n, uint64_t first, uint32_t count)
{
    grid_dependency_enter();
    __shared__ StepShared<BT> sh;
    stats_begin(sh.stats);                       // barrier inside
    if (threadIdx.x == 0) sh.n_duel = 0;
    __syncthreads();
    const uint32_t r = blockIdx.y, rg = r + n.replica_offset;
    const size_t pbase = size_t(r) * n.N;
    SettleAcc acc; acc_zero(acc);

#pragma unroll 1
    for (int pass = 0; pass < (MODE == kModeDispatch ? 1 : 2); ++pass) {
        uint32_t slot = threadIdx.x;             // the request of the block this thread works on
        bool search = false, finish = false, duel_if_found = false, scored = false;
        int a = -1, local_code = -1;
        uint32_t blk = 0, o = 0, probes0 = 0;
        float ssum = 0.0f;
        Draws d;
        d.G0 = d.G1 = d.G2 = d.G3 = 0; d.n_draws = 0; d.n_probes = 0; d.near = false; d.y_slot = 0xffffffffu;

        if (pass == 0) {
            const uint32_t idx = blockIdx.x * BT + slot;
            if (idx < count) {
                const uint32_t q = uint32_t(first + idx);
                const size_t x = size_t(r) * n.Q + first + idx;
                const Rnd4 rx = draw(n, q, 0, rg, kOrigin);
                if (MODE != kModeDuel) {
                    // ---- dispatch (D1..D4): origin decision and scoring ---------------------
                    o = n.origin[x];
                    finish = true;
                    if (origin_offloads(n, r, o, rx, a)) {
                        local_code = a;
                        blk = pick_block(n, o, rx.w[2]);
                        ssum = score_window<BT>(n, sh, slot, r, o, blk, 0xffffffffu, d);
                        scored = search = true;
                        duel_if_found = ppm(rx.w[1]) < n.p_duel;
                    }
                } else {
                    // ---- duel call: requests flagged as duels re-create their window and queue up
                    const int a0 = n.exec_a[x];
                    if (a0 >= 0 && index_ok(n, a0, n.N, 301) && ppm(rx.w[1]) < n.p_duel) {
                        const uint2 ct = n.cont[size_t(r) * n.max_batch + idx];
                        blk = pick_block(n, n.origin[x], rx.w[2]);
                        score_window<BT>(n, sh, slot, r, n.origin[x], blk, ct.x, d);
                        const uint32_t k = atomicAdd(&sh.n_duel, 1u);
                        sh.queue[k] = uint16_t(slot);
                        sh.ctx[slot].a = a0; sh.ctx[slot].blk = blk;
                        sh.ctx[slot].draws_probes_near = (ct.y & 0xffffu) | ((n.rflags[x] & 1u) << 16);
                    }
                }
            }
        } else {
            // ---- duel-and-judge (J2, J3) for the queued requests, densely ----------------------
            __syncthreads();
            if (threadIdx.x < sh.n_duel) {
                slot = sh.queue[threadIdx.x];
                a = sh.ctx[slot].a; blk = sh.ctx[slot].blk;
                const uint32_t packed = sh.ctx[slot].draws_probes_near;
                d.n_draws = packed & 0xffu; d.n_probes = (packed >> 8) & 0xffu; d.near = (packed >> 16) & 1u;
                probes0 = MODE == kModeDuel ? d.n_probes : 0u;
                uint64_t gs[4];
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    gs[g] = 0;
#pragma unroll
                    for (int j = 0; j < 8; ++j) gs[g] += weight_of(sh.S[8 * g + j][slot]);
                }
                d.G0 = gs[0]; d.G1 = gs[1]; d.G2 = gs[2]; d.G3 = gs[3];
                search = finish = true;
            }
        }
        const uint32_t idx = blockIdx.x * BT + slot;
        const uint32_t q = uint32_t(first + idx);
        const size_t x = size_t(r) * n.Q + first + idx;

        // ---- D5, D6 / J2: draw and probe until a peer accepts; in pass 1 go on drawing judges ------
        int found = -1, nj = 0;
        int jd[4] = { -1, -1, -1, -1 };
        if (search) {
            for (;;) {
                if (found < 0) { if (d.n_probes >= n.max_probes) break; }
                else if (pass == 0 || nj >= int(n.n_judges)) break;
                const int pick = draw_candidate(n, sh, slot, d, q, rg);
                if (pick < 0) break;
                const int id = int(kWin * blk + pick);
                if (found < 0) {
                    d.n_probes++;
                    if (probe_peer(n, r, rg, q, blk, pick)) found = id;
                } else if (n.online[pbase + id]) {
                    if (nj == 0) jd[0] = id; else if (nj == 1) jd[1] = id; else if (nj == 2) jd[2] = id; else jd[3] = id;
                    ++nj;
                }
            }
        }

        int b = -1;
        uint32_t oc = 0;
        if (pass == 0) {
            if (MODE != kModeDuel && finish) {
                bool duel = false;
                float sa = 0.0f;
                if (search) {
                    if (found >= 0) {
                        a = found;
                        duel = duel_if_found;
                        if (n.score_a) candidate_weight(n, o, uint32_t(a), n.view[(pbase + o) * n.ld + a], n.w_led[size_t(r) * n.ld + a], sa);
                    } else a = local_code == -4 ? -4 : -2;
                }
                n.exec_a[x] = a;
                if (n.score_a) n.score_a[x] = sa;
                if (n.score_sum) n.score_sum[x] = ssum;
                if (MODE == kModeFused && duel) {
                    const uint32_t k = atomicAdd(&sh.n_duel, 1u);
                    sh.queue[k] = uint16_t(slot);
                    sh.ctx[slot].a = a; sh.ctx[slot].blk = blk;
                    sh.ctx[slot].draws_probes_near = d.n_draws | (d.n_probes << 8) | (d.near ? 1u << 16 : 0u);
                    finish = false;                      // settled in pass 1
                }
            }
        } else if (finish) {
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
            o = n.origin[x];
        }

        // ---- results and settlement (S1..S4) of the request this pass completed -----------------
        if (finish) {
            n.exec_b[x] = b; n.outcome[x] = uint8_t(oc); n.rflags[x] = d.near ? 1 : 0;
            *reinterpret_cast<int4*>(n.judges + 4 * x) = make_int4(jd[0], jd[1], jd[2], jd[3]);
            acc.probes += d.n_probes - probes0;
            if (MODE == kModeFused) settle_one(n, r, q, idx, o, n.len_in[x], n.len_out[x], a, b, jd, oc, d.near, acc);
            if (MODE == kModeDispatch) {
                // continuation for the duel call: lanes still in play, draws and probes used
                uint32_t mask = 0;
                if (scored) {
#pragma unroll
                    for (int c = 0; c < int(kWin); ++c) mask |= (sh.S[c][slot] != 0.0f ? 1u : 0u) << c;
                }
                n.cont[size_t(r) * n.max_batch + idx] = make_uint2(mask, d.n_draws | (d.n_probes << 8));
            }
        }
    }

    // ---- counters: warp reduce, block reduce, one atomic per counter and block ---------------
    acc_flush_warp(sh.stats, acc);
    stats_end(n, sh.stats, r);
}

template <int MODE>
static void launch_by_size(const Net& n, uint64_t first, uint32_t count, const LaunchCtx& c)
{
    // small batches: small blocks, so that the requests spread over all SMs
    if (uint64_t(count) * n.Rp >= 148ull * 128 * 4)
        launch_kernel(c, k_step_fused<128, MODE>, dim3((count + 127) / 128, n.Rp), 128, n, first, count);
    else
        launch_kernel(c, k_step_fused<32, MODE>, dim3((count + 31) / 32, n.Rp), 32, n, first, count);
}

void launch_step_fused(const Net& n, uint64_t first, uint32_t count, const LaunchCtx& c, int step_kernel, uint32_t stream_run)
{
    if (step_kernel == 0) {
        // launches that leave most of the GPU empty share a request among several lanes; the others
        // are taken through the protocol phase by phase, with full warps
        const int lanes = step_lanes_for(uint64_t(count) * n.Rp);
        step_kernel = lanes == 8 ? 1 : lanes == 4 ? 2 : 4;
    }
    if (step_kernel == 1 || step_kernel == 2) { launch_step_lanes(n, first, count, step_kernel == 1 ? 8 : 4, c); return; }
    if (step_kernel == 4) { launch_step_stream(n, first, count, stream_run, c); return; }
    Timed t(c, kStepFused);
    launch_by_size<kModeFused>(n, first, count, c);
}

// Thread-per-request versions of the separate dispatch and duel calls (large batches).
void launch_dispatch_threads(const Net& n, uint64_t first, uint32_t count, const LaunchCtx& c)
{
    Timed t(c, kDispatch);
    launch_by_size<kModeDispatch>(n, first, count, c);
}
void launch_duel_threads(const Net& n, uint64_t first, uint32_t count, const LaunchCtx& c)
{
    Timed t(c, kDuel);
    launch_by_size<kModeDuel>(n, first, count, c);
}

}  // namespace wwws
