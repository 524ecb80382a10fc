// Per-request kernels: dispatch, duel-and-judge, settlement, and the fused step.
// One warp owns one request; lane c owns candidate c of the request's 32-peer window.
#include "request_common.cuh"

namespace wwws {

constexpr int kWarpsPerBlock = 8;

// ---- the candidate window of one request, spread over a warp -------------------------------

struct Window {
    uint32_t r, rg, q, o, blk;     // warp-uniform
    uint64_t W;                    // this lane's integer weight; 0 = not in play
    float score;                   // this lane's fp32 score (0 if never eligible)
    uint32_t n_draws, n_probes;    // warp-uniform
    bool near;                     // some consumed draw fell next to an interval end
    Rnd4 y; uint32_t y_slot;       // cached draw pair
};

// D4 for this lane's candidate.
__device__ __forceinline__ void score_lane(const Net& n, Window& w, uint32_t lane)
{
    const uint32_t id = kWin * w.blk + lane;
    const uint64_t e = n.view[(size_t(w.r) * n.N + w.o) * n.ld + id];     // id < ld always: coalesced 256 B per warp
    const float wl = n.w_led[size_t(w.r) * n.ld + id];                   // padding columns hold 0
    w.W = candidate_weight(n, w.o, id, e, wl, w.score);
}

__device__ __forceinline__ uint64_t warp_incl_scan(uint64_t v, uint32_t lane)
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint64_t t = __shfl_up_sync(kFull, v, o);
        if (lane >= uint32_t(o)) v += t;
    }
    return v;
}

// D5: one draw among the lanes in play, proportional to W, by integer prefix sums.
// Returns the picked lane (warp-uniform) or -1 if nothing is left; the pick leaves play.
__device__ __forceinline__ int pos_draw(const Net& n, Window& w, uint32_t lane)
{
    const uint64_t incl = warp_incl_scan(w.W, lane);
    const uint64_t S = __shfl_sync(kFull, incl, 31);
    if (S == 0) return -1;
    const uint32_t d = w.n_draws++;
    if (n.flags & 4u) {
        // greedy rule: highest weight, lowest lane on ties; flagged when the runner-up is within 1e-5
        uint64_t m = w.W;
#pragma unroll
        for (int o = 16; o; o >>= 1) { const uint64_t t = __shfl_xor_sync(kFull, m, o); m = t > m ? t : m; }
        const int pick = __ffs(__ballot_sync(kFull, w.W == m)) - 1;
        uint64_t m2 = lane == uint32_t(pick) ? 0 : w.W;
#pragma unroll
        for (int o = 16; o; o >>= 1) { const uint64_t t = __shfl_xor_sync(kFull, m2, o); m2 = t > m2 ? t : m2; }
        if (m2 != 0 && m - m2 <= m / 100000ull) w.near = true;
        if (lane == uint32_t(pick)) w.W = 0;
        return pick;
    }
    if (w.y_slot != (d >> 1)) { w.y = draw(n, w.q, d >> 1, w.rg, kDraw); w.y_slot = d >> 1; }
    const uint64_t u = (d & 1u) ? (uint64_t(w.y.w[2]) << 32 | w.y.w[3]) : (uint64_t(w.y.w[0]) << 32 | w.y.w[1]);
    const uint64_t r64 = __umul64hi(u, S);
    const int pick = __ffs(__ballot_sync(kFull, incl > r64)) - 1;
    const uint64_t hi = __shfl_sync(kFull, incl, pick), wp = __shfl_sync(kFull, w.W, pick);
    const uint64_t m1 = r64 - (hi - wp), m2 = hi - 1 - r64;
    if ((m1 < m2 ? m1 : m2) <= S / 100000ull) w.near = true;
    if (lane == uint32_t(pick)) w.W = 0;
    return pick;
}

// D6: the drawn candidate answers by its true state and its own accept policy.
__device__ __forceinline__ bool probe(const Net& n, const Window& w, int pick)
{
    return probe_peer(n, w.r, w.rg, w.q, w.blk, pick);
}

// Draw-and-probe until somebody accepts, the probe budget is spent or nobody is left.
__device__ __forceinline__ int find_executor(const Net& n, Window& w, uint32_t lane)
{
    while (w.n_probes < n.max_probes) {
        const int pick = pos_draw(n, w, lane);
        if (pick < 0) break;
        w.n_probes++;
        if (probe(n, w, pick)) return int(kWin * w.blk + pick);
    }
    return -1;
}

// J2 + J3 for a delegated request flagged as a duel.  Returns the outcome code.
__device__ __forceinline__ uint32_t run_duel(const Net& n, Window& w, uint32_t lane, int a, int& b, int (&jd)[4])
{
    b = find_executor(n, w, lane);
    jd[0] = jd[1] = jd[2] = jd[3] = -1;
    if (b < 0) return 4;
    int nj = 0;
    while (nj < int(n.n_judges)) {
        const int pick = pos_draw(n, w, lane);
        if (pick < 0) break;
        const int id = int(kWin * w.blk + pick);
        if (n.online[size_t(w.r) * n.N + id]) jd[nj++] = id;
    }
    if (nj == 0) { b = -1; return 4; }
    const uint64_t thr = ((1ull << 32) + n.quality[size_t(w.r) * n.N + a] - n.quality[size_t(w.r) * n.N + b]) >> 1;
    int votes_a = 0;
    for (int l = 0; l < nj; ++l) {
        const Rnd4 y = draw(n, w.q, uint32_t(l), w.rg, kJudge);
        bool va = uint64_t(y.w[0]) < thr;
        if (ppm(y.w[1]) < n.p_noise) va = !va;
        votes_a += va;
    }
    return 2 * votes_a > nj ? 1u : (2 * votes_a < nj ? 2u : 3u);
}

// ---- kernels ---------------------------------------------------------------------------------

__device__ __forceinline__ uint2 pack_cont(const Window& w, uint32_t mask) { return make_uint2(mask, w.n_draws | (w.n_probes << 8)); }

// Dispatch (D1..D6) of requests [first, first+count) of every replica.
__global__ void __launch_bounds__(kWarpsPerBlock * 32) k_dispatch(Net n, uint64_t first, uint32_t count)
{
    grid_dependency_enter();
    __shared__ BlockStats bs;
    stats_begin(bs);
    const uint32_t lane = threadIdx.x & 31, r = blockIdx.y;
    const uint32_t idx = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (idx < count) {
        const uint64_t q = first + idx;
        const size_t x = size_t(r) * n.Q + q;
        Window w;
        w.r = r; w.rg = r + n.replica_offset; w.q = uint32_t(q); w.o = n.origin[x];
        w.n_draws = 0; w.n_probes = 0; w.near = false; w.y_slot = 0xffffffffu; w.W = 0; w.score = 0.0f; w.blk = 0;
        const Rnd4 rx = draw(n, w.q, 0, w.rg, kOrigin);
        int a;
        float sa = 0.0f, ssum = 0.0f;
        if (origin_offloads(n, r, w.o, rx, a)) {
            const int local_code = a;
            w.blk = pick_block(n, w.o, rx.w[2]);
            score_lane(n, w, lane);
            if (n.score_sum) {
                for (int l = 0; l < 32; ++l) ssum = __fadd_rn(ssum, __shfl_sync(kFull, w.score, l));
            }
            a = find_executor(n, w, lane);
            if (a >= 0) sa = __shfl_sync(kFull, w.score, a & 31);
            else a = local_code == -4 ? -4 : -2;
        }
        const uint32_t mask = __ballot_sync(kFull, w.W != 0);
        if (lane == 0) {
            n.exec_a[x] = a; n.exec_b[x] = -1; n.outcome[x] = 0; n.rflags[x] = w.near ? 1 : 0;
            *reinterpret_cast<int4*>(n.judges + 4 * x) = make_int4(-1, -1, -1, -1);
            if (n.score_a) n.score_a[x] = sa;
            if (n.score_sum) n.score_sum[x] = ssum;
            n.cont[size_t(r) * n.max_batch + idx] = pack_cont(w, mask);
            stats_add(bs, sProbes, w.n_probes);
        }
    }
    stats_end(n, bs, r);
}

// Duel-and-judge (J1..J3) for the batch last dispatched.
__global__ void __launch_bounds__(kWarpsPerBlock * 32) k_duel(Net n, uint64_t first, uint32_t count)
{
    grid_dependency_enter();
    __shared__ BlockStats bs;
    stats_begin(bs);
    const uint32_t lane = threadIdx.x & 31, r = blockIdx.y;
    const uint32_t idx = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (idx < count) {
        const uint64_t q = first + idx;
        const size_t x = size_t(r) * n.Q + q;
        const int a = n.exec_a[x];
        if (a >= 0 && index_ok(n, a, n.N, 206)) {
            Window w;
            w.r = r; w.rg = r + n.replica_offset; w.q = uint32_t(q); w.o = n.origin[x];
            const Rnd4 rx = draw(n, w.q, 0, w.rg, kOrigin);
            if (ppm(rx.w[1]) < n.p_duel) {
                const uint2 ct = n.cont[size_t(r) * n.max_batch + idx];
                w.n_draws = ct.y & 0xffu; w.n_probes = ct.y >> 8; w.near = false; w.y_slot = 0xffffffffu;
                w.blk = pick_block(n, w.o, rx.w[2]);
                score_lane(n, w, lane);
                if (!(ct.x >> lane & 1u)) w.W = 0;
                const uint32_t probes0 = w.n_probes;
                int b, jd[4];
                const uint32_t oc = run_duel(n, w, lane, a, b, jd);
                if (lane == 0) {
                    n.outcome[x] = uint8_t(oc);
                    if (oc != 4) {
                        n.exec_b[x] = b;
                        *reinterpret_cast<int4*>(n.judges + 4 * x) = make_int4(jd[0], jd[1], jd[2], jd[3]);
                    }
                    if (w.near) n.rflags[x] |= 1;
                    stats_add(bs, sProbes, w.n_probes - probes0);
                }
            }
        }
    }
    stats_end(n, bs, r);
}

// Settlement (S1..S4) of the batch, one thread per request.
__global__ void __launch_bounds__(256) k_settle(Net n, uint64_t first, uint32_t count)
{
    grid_dependency_enter();
    __shared__ BlockStats bs;
    stats_begin(bs);
    const uint32_t r = blockIdx.y, idx = blockIdx.x * blockDim.x + threadIdx.x;
    SettleAcc s; acc_zero(s);
    if (idx < count) {
        const size_t x = size_t(r) * n.Q + first + idx;
        const int4 j4 = *reinterpret_cast<const int4*>(n.judges + 4 * x);
        const int jd[4] = { j4.x, j4.y, j4.z, j4.w };
        settle_one(n, r, uint32_t(first + idx), idx, n.origin[x], n.len_in[x], n.len_out[x], n.exec_a[x], n.exec_b[x], jd, n.outcome[x],
                   (n.rflags[x] & 1) != 0, s);
    }
    acc_flush_warp(bs, s);
    stats_end(n, bs, r);
}

// ---- exact intra-batch queueing (flag 16) -------------------------------------------------------

// Scatter the batch's work items into per-peer lists (offsets from the scan of in_deg).
__global__ void k_fifo_fill(Net n, uint32_t count)
{
    grid_dependency_enter();
    const uint32_t r = blockIdx.y, slot = blockIdx.x * blockDim.x + threadIdx.x;
    if (slot >= count * 7) return;
    const int2 item = n.fifo_items[size_t(r) * n.max_batch * 7 + slot];
    if (item.x < 0 || !index_ok(n, item.x, n.N, 201)) return;
    const size_t px = size_t(r) * n.N + item.x;
    const uint32_t k = atomicAdd(&n.in_cursor[px], 1u);
    if (!index_ok(n, uint64_t(n.in_off[px]) + k, 7ull * n.max_batch, 202)) return;
    // entry: (request, amount): tokens of queued work, or, with bit 31 set, the number of payments of R (role 6)
    n.fifo_list[size_t(r) * n.max_batch * 7 + n.in_off[px] + k] = make_uint2(slot / 7, uint32_t(item.y) | (slot % 7 == 6 ? 0x80000000u : 0u));
}

// Latency of every served request: it waits behind the batch-start queue of its executor and
// behind the items that earlier requests of the batch put there.
__global__ void __launch_bounds__(256) k_fifo_latency(Net n, uint64_t first, uint32_t count)
{
    grid_dependency_enter();
    __shared__ BlockStats bs;
    stats_begin(bs);
    const uint32_t r = blockIdx.y, idx = blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t met = 0, uncovered = 0;
    unsigned long long lat_sum = 0;
    if (idx < count) {
        const size_t x = size_t(r) * n.Q + first + idx;
        const int a = n.exec_a[x];
        if (a != -3 && a != -4 && index_ok(n, a < 0 ? n.origin[x] : uint32_t(a), n.N, 203)) {
            const uint32_t ex = a < 0 ? n.origin[x] : uint32_t(a);
            const size_t px = size_t(r) * n.N + ex;
            const uint2* list = n.fifo_list + size_t(r) * n.max_batch * 7 + n.in_off[px];
            const uint32_t len = index_ok(n, uint64_t(n.in_off[px]) + n.in_deg[px], 7ull * n.max_batch + 1, 204) ? n.in_deg[px] : 0u;
            uint64_t ahead = 0;
            for (uint32_t j = 0; j < len; ++j) { const uint2 it = list[j]; if (it.x < idx && !(it.y >> 31)) ahead += it.y; }
            if (a >= 0) {
                // in-block validation: the payment must fit the finalized balance minus what the
                // payer already spent in this block (earlier batches, earlier requests of this batch)
                const size_t ox = size_t(r) * n.N + n.origin[x];
                const uint2* mine = n.fifo_list + size_t(r) * n.max_batch * 7 + n.in_off[ox];
                const uint32_t mlen = index_ok(n, uint64_t(n.in_off[ox]) + n.in_deg[ox], 7ull * n.max_batch + 1, 205) ? n.in_deg[ox] : 0u;
                long long spent = n.blk_spent[ox];
                for (uint32_t j = 0; j < mlen; ++j) { const uint2 it = mine[j]; if (it.x < idx && (it.y >> 31)) spent += n.R * (long long)(it.y & 0x7fffffffu); }
                const uint32_t oc = n.outcome[x];
                const long long pay = n.R * ((oc >= 1 && oc <= 3) ? 2 : 1);
                uncovered = n.credit[ox] - spent < pay;
            }
            const uint64_t work = uint64_t(n.len_in[x]) + n.len_out[x], cap = n.cap_eff[px];
            const uint64_t t = (uint64_t(n.backlog[px]) + ahead + work) * 1000ull, tq = udiv64by32(t, uint32_t(cap));
            const uint64_t lat = tq + (tq * cap != t ? 1 : 0) + (a >= 0 ? n.hop_ms : 0);
            const uint64_t ideal = udiv64by32(work * 1000ull + n.cap_ref - 1, n.cap_ref);
            const uint64_t deadline = udiv64by32(uint64_t(n.slo_num) * ideal, n.slo_den);
            lat_sum = lat; met = lat <= deadline;
        }
    }
    const uint32_t m = __reduce_add_sync(kFull, met), unc = __reduce_add_sync(kFull, uncovered);
    for (int o = 16; o; o >>= 1) lat_sum += __shfl_down_sync(kFull, lat_sum, o);
    if ((threadIdx.x & 31) == 0) { stats_add(bs, sSloMet, m); stats_add(bs, sSumLat, lat_sum); stats_add(bs, sUncovered, unc); }
    stats_end(n, bs, r);
}

void launch_fifo(const Net& n, uint64_t first, uint32_t count, const LaunchCtx& c)
{
    launch_scan_in_degrees(n, c, kFifo);
    { Timed t(c, kFifo); launch_kernel(c, k_fifo_fill, dim3((count * 7 + 255) / 256, n.Rp), 256, n, count); }
    { Timed t(c, kFifo); launch_kernel(c, k_fifo_latency, dim3((count + 255) / 256, n.Rp), 256, n, first, count); }
}

// ---- batches to and from mapped host buffers ---------------------------------------------------------
// One thread per request, consecutive threads on consecutive requests: every warp reads or writes whole
// contiguous segments of the host buffers, so the bus carries full lines in request order.
__global__ void __launch_bounds__(256) k_host_batch_in(Net n, HostBatch h, uint64_t first, uint32_t count)
{
    grid_dependency_enter();
    const uint32_t idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= count) return;
    const size_t x = size_t(blockIdx.y) * n.Q + first + idx;
    const_cast<uint32_t*>(n.origin)[x] = h.origin[x];
    const_cast<uint16_t*>(n.len_in)[x] = h.len_in[x];
    const_cast<uint16_t*>(n.len_out)[x] = h.len_out[x];
}

__global__ void __launch_bounds__(256) k_host_batch_out(Net n, HostBatch h, uint64_t first, uint32_t count)
{
    grid_dependency_enter();
    const uint32_t idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= count) return;
    const size_t x = size_t(blockIdx.y) * n.Q + first + idx;
    h.exec_a[x] = n.exec_a[x];
    h.exec_b[x] = n.exec_b[x];
    reinterpret_cast<int4*>(h.judges)[x] = reinterpret_cast<const int4*>(n.judges)[x];
    h.outcome[x] = n.outcome[x];
    h.rflags[x] = n.rflags[x];
}

void launch_host_batch_in(const Net& n, const HostBatch& h, uint64_t first, uint32_t count, const LaunchCtx& c)
{
    Timed t(c, kHostBatch);
    launch_kernel(c, k_host_batch_in, dim3((count + 255) / 256, n.Rp), 256, n, h, first, count);
}
void launch_host_batch_out(const Net& n, const HostBatch& h, uint64_t first, uint32_t count, const LaunchCtx& c)
{
    Timed t(c, kHostBatch);
    launch_kernel(c, k_host_batch_out, dim3((count + 255) / 256, n.Rp), 256, n, h, first, count);
}

static dim3 warp_grid(const Net& n, uint32_t count) { return dim3((count + kWarpsPerBlock - 1) / kWarpsPerBlock, n.Rp); }

void launch_dispatch(const Net& n, uint64_t first, uint32_t count, const LaunchCtx& c)
{
    Timed t(c, kDispatch);
    launch_kernel(c, k_dispatch, warp_grid(n, count), kWarpsPerBlock * 32, n, first, count);
}
void launch_duel(const Net& n, uint64_t first, uint32_t count, const LaunchCtx& c)
{
    Timed t(c, kDuel);
    launch_kernel(c, k_duel, warp_grid(n, count), kWarpsPerBlock * 32, n, first, count);
}
void launch_settle(const Net& n, uint64_t first, uint32_t count, const LaunchCtx& c)
{
    Timed t(c, kSettle);
    launch_kernel(c, k_settle, dim3((count + 255) / 256, n.Rp), 256, n, first, count);
}
}  // namespace wwws
