// Per-peer kernels: initial state and views, time advance, queue fold, block finalization.
#include "wwws_internal.cuh"

namespace wwws {

// Reputation-weighted stake in fp32: (float)stake * (float)(wins+1) / (float)(duels+2), each
// operation rounded to nearest (no contraction), so the value equals the per-request formula.
__device__ __forceinline__ float ledger_weight(const Net& n, int64_t stake, uint32_t wins, uint32_t duels)
{
    if (stake <= 0) return 0.0f;
    const float sf = __ll2float_rn(stake);
    float rep = 1.0f;
    if (n.flags & 1u) rep = __fdiv_rn(__uint2float_rn(wins + 1u), __uint2float_rn(duels + 2u));
    return __fmul_rn(sf, rep);
}

__global__ void k_peer_init(Net n, const int64_t* __restrict__ credit0, const uint8_t* __restrict__ online0,
                            uint32_t init_stale_max)
{
    grid_dependency_enter();
    const uint32_t r = blockIdx.y, j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n.N) return;
    const size_t x = size_t(r) * n.N + j;
    n.online[x] = online0[x] ? 1 : 0;
    n.ver[x] = init_stale_max + 1;
    n.cap_eff[x] = cap_eff_at(n, n.cap_true[x], n.prio_flag[x] != 0, j, r + n.replica_offset, 0);
    n.backlog[x] = 0;
    const int64_t c = credit0[x];
    n.credit[x] = c;
    const int64_t st = (c > 0 ? c : 0) * int64_t(n.stake_pm[x]) / 1000;
    n.stake[x] = st;
    n.wins[x] = 0; n.duels[x] = 0; n.served[x] = 0; n.served_local[x] = 0;
    n.d_credit[x] = 0; n.d_wins[x] = 0; n.d_duels[x] = 0; n.d_backlog[x] = 0;
    n.blk_spent[x] = 0; n.d_spent[x] = 0;
    n.w_led[size_t(r) * n.ld + j] = ledger_weight(n, st, 0, 0);
    n.self_entry[x] = 0;
    refresh_gate(n, x, online0[x] != 0, n.cap_eff[x], 0, c);
}

// V[i][j] = entry of j at a version 0..init_stale_max old (own entry current).
__global__ void k_view_init(Net n, uint32_t init_stale_max)
{
    grid_dependency_enter();
    const uint32_t r = blockIdx.z, i = blockIdx.y;
    const uint32_t rg = r + n.replica_offset;
    uint64_t* row = n.view + (size_t(r) * n.N + i) * n.ld;
    for (uint32_t j = blockIdx.x * blockDim.x + threadIdx.x; j < n.ld; j += gridDim.x * blockDim.x) {
        uint64_t e = 0;
        if (j < n.N) {
            const size_t x = size_t(r) * n.N + j;
            uint32_t stale = 0;
            if (init_stale_max != 0 && i != j) stale = below(draw(n, i, j, rg, kInit).w[0], init_stale_max + 1);
            e = pack_entry(n.ver[x] - stale, n.online[x] == 0, uint64_t(n.cap_eff[x]) * n.misreport[x], 0);
        }
        row[j] = e;
    }
}

__global__ void k_advance(Net n, uint32_t dt_ms, uint32_t now_ms)
{
    grid_dependency_enter();
    const uint32_t r = blockIdx.y, j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n.N) return;
    const size_t x = size_t(r) * n.N + j;
    const uint32_t cap = n.cap_eff[x];
    const bool on = n.online[x] != 0;
    int64_t b = n.backlog[x];
    if (on) {
        const int64_t done = int64_t(uint64_t(cap) * dt_ms / 1000u);
        b = b > done ? b - done : 0;
        n.backlog[x] = b;
    }
    const uint32_t cap_now = cap_eff_at(n, n.cap_true[x], n.prio_flag[x] != 0, j, r + n.replica_offset, now_ms);
    n.cap_eff[x] = cap_now;
    refresh_gate(n, x, on, cap_now, b, n.credit[x]);
}

// Commit of replica r's block, run by the last block of k_fold to finish that replica: total
// credit must be what it was at creation; the chain head takes the block's operations digest.
__device__ void finalize_replica(const Net& n, uint32_t r)
{
    const long long total = (long long)atomicAdd((unsigned long long*)&n.credit_check[r], 0ull);
    if (total != n.credit_total0[r]) set_error(n, eInvariant, r);
    n.credit_check[r] = 0;
    unsigned long long* st = n.stats + size_t(r) * sCount;
    st[sBlocks] += 1;
    // block id = hash of (parent id, order-independent digest of the block's records, height)
    st[sChainHead] = mix64(mix64(st[sChainHead] ^ chain_key(n, r)) + st[sPendingDigest] + kGamma * st[sBlocks]);
    st[sPendingDigest] = 0;
}

// End of a settlement: queues take the batch's work; with `finalize` the pending block is
// folded into the ledger, stakes and derived weights are refreshed, credit is summed and the
// replica's block is committed.
// Majority validation: how many peers of each replica are online to confirm a proposed block.
__global__ void k_count_online(Net n)
{
    grid_dependency_enter();
    const uint32_t r = blockIdx.y, j = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t on = j < n.N && n.online[size_t(r) * n.N + j];
    const uint32_t c = __reduce_add_sync(0xffffffffu, on);
    if ((threadIdx.x & 31) == 0 && c) atomicAdd(&n.online_count[r], c);
}

// ADVANCE: the time advance of the next step in the same pass (the step's fold was deferred to the
// next step's call): one launch and one sweep over the per-peer tables instead of two.
template <bool ADVANCE>
__global__ void k_fold(Net n, int finalize_requested, uint32_t dt_ms, uint32_t now_ms)
{
    grid_dependency_enter();
    const uint32_t r = blockIdx.y, j = blockIdx.x * blockDim.x + threadIdx.x;
    // with majority validation the block is committed only if more than half of the peers are online
    const bool finalize = finalize_requested && (!(n.flags & 32u) || 2u * n.online_count[r] > n.N);
    long long csum = 0;
    if (j < n.N) {
        const size_t x = size_t(r) * n.N + j;
        // Most peers are untouched by a batch (16,000 requests on 262,144 peers): every table is
        // read, but written only where its value changes.
        const long long db = n.d_backlog[x];
        const int64_t queued_before = n.backlog[x], queued = queued_before + db;
        if (db) n.d_backlog[x] = 0;
        int64_t credit_now = n.credit[x];
        bool ledger_changed = false;
        if (n.flags & 16u) {
            n.in_deg[x] = 0;                         // per-peer item counts of the batch's queueing pass
            n.blk_spent[x] = finalize ? 0 : n.blk_spent[x] + n.d_spent[x];
            n.d_spent[x] = 0;
        }
        if (finalize) {
            const long long dc = n.d_credit[x];
            const uint32_t dw = n.d_wins[x], dd = n.d_duels[x];
            const int64_t c = credit_now + dc;
            if (dc) { n.credit[x] = c; n.d_credit[x] = 0; }
            if (dw | dd) {
                const uint32_t w = n.wins[x] + dw, d = n.duels[x] + dd;
                if (dw) { n.wins[x] = w; n.d_wins[x] = 0; }
                if (dd) { n.duels[x] = d; n.d_duels[x] = 0; }
            }
            if (dc || dw || dd) {                    // stake and ledger weight are functions of (credit, wins, duels)
                const int64_t st = (c > 0 ? c : 0) * int64_t(n.stake_pm[x]) / 1000;
                n.stake[x] = st;
                n.w_led[size_t(r) * n.ld + j] = ledger_weight(n, st, n.wins[x], n.duels[x]);
                ledger_changed = true;
            }
            csum = c;
            credit_now = c;
        }
        if (ADVANCE) {
            // C3 on top of the folded queue: drain at the rate in force, then the new window's rate
            const uint32_t cap = n.cap_eff[x];
            const bool on = n.online[x] != 0;
            int64_t b = queued;
            if (on) {
                const int64_t done = int64_t(uint64_t(cap) * dt_ms / 1000u);
                b = b > done ? b - done : 0;
            }
            if (b != queued_before) n.backlog[x] = b;
            const uint32_t cap_now = cap_eff_at(n, n.cap_true[x], n.prio_flag[x] != 0, j, r + n.replica_offset, now_ms);
            if (cap_now != cap) n.cap_eff[x] = cap_now;
            if (b != queued_before || cap_now != cap || ledger_changed) refresh_gate(n, x, on, cap_now, b, credit_now);
        } else {
            if (db) n.backlog[x] = queued;
            if (db || ledger_changed) refresh_gate(n, x, n.online[x] != 0, n.cap_eff[x], queued, credit_now);
        }
    }
    if (finalize) {
        // block sum of the committed credit, one atomic per block; the block that finishes a replica
        // last commits it (no second launch): thread 0 makes its sum visible, then takes a ticket
        __shared__ long long warp_sum[32];
        for (int o = 16; o; o >>= 1) csum += __shfl_down_sync(0xffffffffu, csum, o);
        if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = csum;
        __syncthreads();
        if (threadIdx.x == 0) {
            long long bsum = 0;
            for (uint32_t k = 0; k < (blockDim.x + 31) / 32; ++k) bsum += warp_sum[k];
            if (bsum) atomicAdd((unsigned long long*)&n.credit_check[r], (unsigned long long)bsum);
            __threadfence();
            if (atomicAdd(&n.fold_ticket[r], 1u) == gridDim.x - 1) {
                n.fold_ticket[r] = 0;
                __threadfence();
                finalize_replica(n, r);
            }
        }
    } else if (finalize_requested && blockIdx.x == 0 && threadIdx.x == 0) {
        n.stats[size_t(r) * sCount + sBlocksRejected] += 1;      // no majority: the block stays open
    }
}

// The online counts are consumed by one k_fold; clear them for the next proposal.
__global__ void k_clear_online_count(Net n)
{
    grid_dependency_enter();
    const uint32_t r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r < n.Rp) n.online_count[r] = 0;
}

// Re-derive stake and weight from the ledger as it stands (after a table import).
__global__ void k_rederive(Net n)
{
    grid_dependency_enter();
    const uint32_t r = blockIdx.y, j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n.N) return;
    const size_t x = size_t(r) * n.N + j;
    const int64_t c = n.credit[x];
    const int64_t st = (c > 0 ? c : 0) * int64_t(n.stake_pm[x]) / 1000;
    n.stake[x] = st;
    n.w_led[size_t(r) * n.ld + j] = ledger_weight(n, st, n.wins[x], n.duels[x]);
    refresh_gate(n, x, n.online[x] != 0, n.cap_eff[x], n.backlog[x], c);
}

// credit_total per replica = sum of finalized and pending credit.
__global__ void k_credit_total(Net n)
{
    grid_dependency_enter();
    const uint32_t r = blockIdx.y, j = blockIdx.x * blockDim.x + threadIdx.x;
    long long s = 0;
    if (j < n.N) { const size_t x = size_t(r) * n.N + j; s = n.credit[x] + n.d_credit[x]; }
    for (int o = 16; o; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
    if ((threadIdx.x & 31) == 0 && s) atomicAdd(&n.stats[size_t(r) * sCount + sCreditTotal], (unsigned long long)s);
}

__global__ void k_zero_credit_total(Net n)
{
    grid_dependency_enter();
    const uint32_t r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r < n.Rp) n.stats[size_t(r) * sCount + sCreditTotal] = 0;
}

static dim3 peer_grid(const Net& n) { return dim3((n.N + 255) / 256, n.Rp); }

void launch_peer_init(const Net& n, const int64_t* credit0, const uint8_t* online0, uint32_t init_stale_max, const LaunchCtx& c)
{
    { Timed t(c, kPeerInit); launch_kernel(c, k_peer_init, peer_grid(n), 256, n, credit0, online0, init_stale_max); }
    const uint32_t bx = (n.ld + 255) / 256 > 64 ? 64 : (n.ld + 255) / 256;
    // grid.y / grid.z limits (65535): rows go in y, replicas in z
    { Timed t(c, kViewInit); launch_kernel(c, k_view_init, dim3(bx, n.N, n.Rp), 256, n, init_stale_max); }
}

void launch_advance(const Net& n, uint32_t dt_ms, uint32_t now_ms, const LaunchCtx& c)
{
    Timed t(c, kAdvance);
    launch_kernel(c, k_advance, peer_grid(n), 256, n, dt_ms, now_ms);
}

void launch_fold(const Net& n, int finalize, const LaunchCtx& c)
{
    const bool majority = finalize && (n.flags & 32u);
    if (majority) { Timed t(c, kFold); launch_kernel(c, k_count_online, peer_grid(n), 256, n); }
    { Timed t(c, kFold); launch_kernel(c, k_fold<false>, peer_grid(n), 256, n, finalize, 0u, 0u); }
    if (majority) { Timed t(c, kFold); launch_kernel(c, k_clear_online_count, (n.Rp + 127) / 128, 128, n); }
}

// The fold of the previous step and the time advance of this one in a single launch (not with
// majority validation, whose online count needs a kernel of its own before the fold).
void launch_fold_advance(const Net& n, int finalize, uint32_t dt_ms, uint32_t now_ms, const LaunchCtx& c)
{
    Timed t(c, kFold);
    launch_kernel(c, k_fold<true>, peer_grid(n), 256, n, finalize, dt_ms, now_ms);
}

void launch_rederive(const Net& n, const LaunchCtx& c)
{
    Timed t(c, kRederive);
    launch_kernel(c, k_rederive, peer_grid(n), 256, n);
}

void launch_credit_total(const Net& n, const LaunchCtx& c)
{
    { Timed t(c, kCreditTotal); launch_kernel(c, k_zero_credit_total, (n.Rp + 127) / 128, 128, n); }
    { Timed t(c, kCreditTotal); launch_kernel(c, k_credit_total, peer_grid(n), 256, n); }
}

// ---- optional per-kernel event timing ------------------------------------------------------------

void Profiler::begin(int id, cudaStream_t s)
{
    Pair p;
    if (!pool.empty()) { p = pool.back(); pool.pop_back(); }
    else { cudaEventCreate(&p.a); cudaEventCreate(&p.b); }
    p.id = id;
    cudaEventRecord(p.a, s);
    used.push_back(p);
}
void Profiler::end(cudaStream_t s) { cudaEventRecord(used.back().b, s); }
void Profiler::collect()
{
    for (Pair& p : used) {
        cudaEventSynchronize(p.b);
        float t = 0.f;
        if (cudaEventElapsedTime(&t, p.a, p.b) == cudaSuccess) { ms[p.id] += t; count[p.id] += 1; }
        pool.push_back(p);
    }
    used.clear();
}
void Profiler::reset()
{
    collect();
    for (int k = 0; k < kKernelCount; ++k) { ms[k] = 0; count[k] = 0; }
}
Profiler::~Profiler()
{
    for (Pair& p : used) { cudaEventDestroy(p.a); cudaEventDestroy(p.b); }
    for (Pair& p : pool) { cudaEventDestroy(p.a); cudaEventDestroy(p.b); }
}

}  // namespace wwws
