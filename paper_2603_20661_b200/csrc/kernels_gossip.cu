// Gossip round: churn + self entries + partner choice (per peer), row merge (streaming
// 64-bit max over gathered rows), and the scattered single-entry updates.
#include <cstdlib>

#include "wwws_internal.cuh"

namespace wwws {

// G0 churn, G1 new version of the own entry, partner choice of G2 (reads the old view only).
__global__ void k_gossip_peer(Net n, uint32_t round)
{
    grid_dependency_enter();
    const uint32_t r = blockIdx.y, i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n.N) return;
    const uint32_t rg = r + n.replica_offset;
    const size_t x = size_t(r) * n.N + i;
    bool on = n.online[x] != 0;
    if (n.p_leave | n.p_join) {
        const uint32_t u = ppm(draw(n, i, round, rg, kChurn).w[0]);
        if (on) { if (u < n.p_leave) { on = false; n.backlog[x] = 0; n.online[x] = 0; refresh_gate(n, x, false, n.cap_eff[x], 0, n.credit[x]); } }
        else if (u < n.p_join) { on = true; n.online[x] = 1; refresh_gate(n, x, true, n.cap_eff[x], n.backlog[x], n.credit[x]); }
    }
    int32_t part[4] = { -1, -1, -1, -1 };
    uint64_t self = 0;
    if (on) {
        uint32_t v = n.ver[x] + 1;
        if (v >= (1u << 24)) { set_error(n, eRange, i); v = (1u << 24) - 1; }
        n.ver[x] = v;
        self = pack_entry(v, false, uint64_t(n.cap_eff[x]) * n.misreport[x], uint64_t(n.backlog[x]) >> 4);
        const uint64_t* row = n.view + x * n.ld;
        uint32_t open = (1u << n.fanout_k) - 1u;     // slots still looking for a partner
        for (uint32_t a = 0; a < n.gossip_tries && open; ++a) {
            const Rnd4 g = draw(n, i, round, rg, kGossip + 256u * a);
            // the candidates of all open slots first, their entries fetched together (one memory round
            // trip per attempt instead of one per slot), then the decisions
            uint32_t cand[4];
            uint64_t ent[4];
#pragma unroll
            for (uint32_t s = 0; s < 4; ++s) {
                cand[s] = below(g.w[s], n.N);
                ent[s] = (open >> s & 1u) ? row[cand[s]] : 0ull;
            }
#pragma unroll
            for (uint32_t s = 0; s < 4; ++s) {
                if (!(open >> s & 1u) || cand[s] == i) continue;
                if (ent[s] != 0 && !(ent[s] & kOffBit) && index_ok(n, cand[s], n.N, 101)) { part[s] = int32_t(cand[s]); open &= ~(1u << s); }
            }
        }
    }
    n.self_entry[x] = self;
    n.in_deg[x] = 0;
    *reinterpret_cast<int4*>(n.partner + x * 4) = make_int4(part[0], part[1], part[2], part[3]);
}

// Once every peer's churn is known, a chosen partner either answers (it is online) or not.  The
// partner list is rewritten in place so that the kernels that follow need no second lookup:
// p >= 0 = answered, -2 - p = chosen but dead, -1 = no partner in that slot.
__global__ void k_gossip_resolve(Net n)
{
    grid_dependency_enter();
    const uint32_t r = blockIdx.y, i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n.N) return;
    const size_t x = size_t(r) * n.N + i;
    int4 p4 = *reinterpret_cast<const int4*>(n.partner + x * 4);
    const uint8_t* on = n.online + size_t(r) * n.N;
    if (p4.x >= 0) { if (!index_ok(n, p4.x, n.N, 102)) p4.x = -1; else if (!on[p4.x]) p4.x = -2 - p4.x; }
    if (p4.y >= 0) { if (!index_ok(n, p4.y, n.N, 102)) p4.y = -1; else if (!on[p4.y]) p4.y = -2 - p4.y; }
    if (p4.z >= 0) { if (!index_ok(n, p4.z, n.N, 102)) p4.z = -1; else if (!on[p4.z]) p4.z = -2 - p4.z; }
    if (p4.w >= 0) { if (!index_ok(n, p4.w, n.N, 102)) p4.w = -1; else if (!on[p4.w]) p4.w = -2 - p4.w; }
    *reinterpret_cast<int4*>(n.partner + x * 4) = p4;
}

// Streaming merge: new row = max(old row, rows of the partners that answered).
//
// A row is read by its owner and by every node that pulls it (k+1 readers on average), so the
// order of the work decides how often it comes from HBM.  The matrix is cut into column panels
// narrow enough that one panel of all N rows stays in L2 (N * panel_cols * 8 bytes); blocks are
// numbered panel-major, so the blocks in flight at any time work on the same panel: the first
// reader of a row segment brings it in from HBM, the others hit L2.  HBM traffic per round drops
// from (k+2) * 8 * N^2 towards 2 * 8 * N^2 (each entry read once, written once).  Stores are
// streaming (evict-first) so that they do not push the panel out.
//
// A thread moves 32 bytes (four entries) per row it touches: one 256-bit load per source row.

constexpr int kMergeThreads = 128;
constexpr int kMergeIters = 4;                         // rows per thread

struct Q4 { uint64_t a, b, c, d; };                    // four entries = 32 bytes

__device__ __forceinline__ Q4 ld32(const char* p)
{
    Q4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u64 {%0,%1,%2,%3}, [%4];"
                 : "=l"(v.a), "=l"(v.b), "=l"(v.c), "=l"(v.d) : "l"(p));
    return v;
}
__device__ __forceinline__ void st32_stream(char* p, const Q4& v)
{
    asm volatile("st.global.cs.v4.u64 [%0], {%1,%2,%3,%4};" ::"l"(p), "l"(v.a), "l"(v.b), "l"(v.c), "l"(v.d) : "memory");
}
__device__ __forceinline__ uint64_t umax64(uint64_t a, uint64_t b) { return a > b ? a : b; }
__device__ __forceinline__ void join(Q4& x, const Q4& y)
{
    x.a = umax64(x.a, y.a); x.b = umax64(x.b, y.b); x.c = umax64(x.c, y.c); x.d = umax64(x.d, y.d);
}

// grid.x runs over (replica, panel, row group).  A thread owns one 32-byte column chunk of the
// panel and walks kMergeIters rows of the block's row group.  The sources of a row (the partners
// that answered; an offline row has none and is copied) were resolved by k_gossip_resolve, so a
// thread fetches them with one 16-byte load per row, all issued before the streaming part: no
// shared memory, no barrier, no dependent metadata loads.
// PUSH: full pairwise exchange, a row also takes the old rows of the nodes that pulled it
// (their ids come from the per-round reverse lists).
template <bool PUSH>
__global__ void __launch_bounds__(kMergeThreads, PUSH ? 6 : 8) k_gossip_merge(Net n, uint32_t panel_cols, uint32_t chunk_shift,
                                                                     uint32_t n_panels, uint32_t groups_per_panel)
{
    grid_dependency_enter();
    const uint32_t b = blockIdx.x;
    const uint32_t per_replica = n_panels * groups_per_panel;
    const uint32_t r = b / per_replica;
    const uint32_t rem = b - r * per_replica;
    const uint32_t panel = rem / groups_per_panel, group = rem - panel * groups_per_panel;
    const uint32_t rstep = kMergeThreads >> chunk_shift;                  // rows covered by one pass of the block
    const uint32_t row0 = group * rstep * kMergeIters + (threadIdx.x >> chunk_shift);
    const size_t rbase = size_t(r) * n.N;
    const uint32_t c = panel * panel_cols + 4u * (threadIdx.x & ((1u << chunk_shift) - 1u));
    if (c >= n.ld) return;
    int4 srcs[kMergeIters];
    uint2 ins[PUSH ? kMergeIters : 1];                                    // (offset, count) of the row's reverse list
#pragma unroll
    for (int it = 0; it < kMergeIters; ++it) {
        const uint32_t row = row0 + it * rstep;
        srcs[it] = row < n.N ? __ldg(reinterpret_cast<const int4*>(n.partner) + rbase + row) : make_int4(-1, -1, -1, -1);
        if (PUSH) ins[it] = row < n.N ? make_uint2(n.in_off[rbase + row], n.in_deg[rbase + row]) : make_uint2(0, 0);
    }
    const uint32_t ld8 = n.ld * 8u;
    const char* in = reinterpret_cast<const char*>(n.view + rbase * n.ld + c);
    char* out = reinterpret_cast<char*>(n.view_new + rbase * n.ld + c);
#pragma unroll
    for (int it = 0; it < kMergeIters; ++it) {
        const uint32_t row = row0 + it * rstep;
        if (row >= n.N) break;
        int4 src = srcs[it];
#ifdef WWWS_CHECK_INDICES
        if (src.x >= 0 && !index_ok(n, src.x, n.N, 103)) src.x = -1;
        if (src.y >= 0 && !index_ok(n, src.y, n.N, 103)) src.y = -1;
        if (src.z >= 0 && !index_ok(n, src.z, n.N, 103)) src.z = -1;
        if (src.w >= 0 && !index_ok(n, src.w, n.N, 103)) src.w = -1;
#endif
        Q4 acc = ld32(in + uint64_t(row) * ld8);
        Q4 v0, v1, v2, v3;
        if (src.x >= 0) v0 = ld32(in + uint64_t(uint32_t(src.x)) * ld8);
        if (src.y >= 0) v1 = ld32(in + uint64_t(uint32_t(src.y)) * ld8);
        if (src.z >= 0) v2 = ld32(in + uint64_t(uint32_t(src.z)) * ld8);
        if (src.w >= 0) v3 = ld32(in + uint64_t(uint32_t(src.w)) * ld8);
        if (src.x >= 0) join(acc, v0);
        if (src.y >= 0) join(acc, v1);
        if (src.z >= 0) join(acc, v2);
        if (src.w >= 0) join(acc, v3);
        if (PUSH) {
            const int32_t* who = n.pullers + rbase * 4 + ins[it].x;
            if (index_ok(n, uint64_t(ins[it].x) + ins[it].y, 4ull * n.N + 1, 104))
                for (uint32_t j = 0; j < ins[it].y; ++j)
                    if (index_ok(n, uint32_t(who[j]), n.N, 105)) join(acc, ld32(in + uint64_t(uint32_t(who[j])) * ld8));
        }
        st32_stream(out + uint64_t(row) * ld8, acc);
    }
}

// Reverse lists for the pairwise exchange: who pulled each node this round.
__global__ void k_gossip_indeg(Net n)
{
    grid_dependency_enter();
    const uint32_t r = blockIdx.y, i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n.N) return;
    const size_t x = size_t(r) * n.N + i;
    if (!n.online[x]) return;
    const int4 p4 = *reinterpret_cast<const int4*>(n.partner + x * 4);
    const int32_t p[4] = { p4.x, p4.y, p4.z, p4.w };
#pragma unroll
    for (int s = 0; s < 4; ++s)
        if (p[s] >= 0 && index_ok(n, p[s], n.N, 106)) atomicAdd(&n.in_deg[size_t(r) * n.N + p[s]], 1u);
}

// Exclusive prefix sum of the in-degrees of one replica (one block per replica).
__global__ void __launch_bounds__(1024) k_gossip_scan(Net n)
{
    grid_dependency_enter();
    __shared__ uint32_t warp_sum[32];
    __shared__ uint32_t carry;
    const uint32_t r = blockIdx.x, lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (uint32_t base = 0; base < n.N; base += 1024) {
        const uint32_t i = base + threadIdx.x;
        const uint32_t v = i < n.N ? n.in_deg[size_t(r) * n.N + i] : 0;
        uint32_t incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= uint32_t(o)) incl += t; }
        if (lane == 31) warp_sum[wid] = incl;
        __syncthreads();
        if (wid == 0) {
            uint32_t w = warp_sum[lane], wi = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_up_sync(0xffffffffu, wi, o); if (lane >= uint32_t(o)) wi += t; }
            warp_sum[lane] = wi - w;                                       // exclusive over warps
        }
        __syncthreads();
        const uint32_t excl = carry + warp_sum[wid] + incl - v;
        if (i < n.N) { n.in_off[size_t(r) * n.N + i] = excl; n.in_cursor[size_t(r) * n.N + i] = 0; }
        __syncthreads();
        if (threadIdx.x == 1023) carry = excl + v;
        __syncthreads();
    }
}

__global__ void k_gossip_fill(Net n)
{
    grid_dependency_enter();
    const uint32_t r = blockIdx.y, i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n.N) return;
    const size_t x = size_t(r) * n.N + i;
    if (!n.online[x]) return;
    const int4 p4 = *reinterpret_cast<const int4*>(n.partner + x * 4);
    const int32_t p[4] = { p4.x, p4.y, p4.z, p4.w };
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        if (p[s] < 0 || !index_ok(n, p[s], n.N, 107)) continue;
        const size_t px = size_t(r) * n.N + p[s];
        const uint32_t k = atomicAdd(&n.in_cursor[px], 1u);
        if (index_ok(n, uint64_t(n.in_off[px]) + k, 4ull * n.N, 108)) n.pullers[size_t(r) * n.N * 4 + n.in_off[px] + k] = int32_t(i);
    }
}

// The three single-entry updates of a round, applied after the row merge: own fresh entry,
// offline mark for a partner that did not answer, and the "hello" that shows the puller's entry
// to the partner.  None needs an atomic.  A peer that is online has just issued a new version,
// and nobody else can hold that version yet, so its fresh entry is the maximum wherever it
// lands: own entry and hellos are plain stores (two pullers of one partner write different
// columns).  An offline mark is a read-max-write of an element that only this thread writes: a
// hello into the same element would have to come from the dead partner, which sends none.
__global__ void k_gossip_fixup(Net n)
{
    grid_dependency_enter();
    const uint32_t r = blockIdx.y, i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n.N) return;
    const size_t x = size_t(r) * n.N + i;
    if (i == 0) atomicAdd(&n.stats[size_t(r) * sCount + sRounds], 1ull);
    n.in_deg[x] = 0;                                 // the reverse lists of this round are spent
    if (!n.online[x]) return;
    const uint64_t self = n.self_entry[x];
    uint64_t* vn = n.view_new;
    vn[x * n.ld + i] = self;
    const int4 p4 = *reinterpret_cast<const int4*>(n.partner + x * 4);
    const int32_t p[4] = { p4.x, p4.y, p4.z, p4.w };
    uint32_t marks = 0;
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        if (p[s] == -1) continue;
        if (p[s] < -1) {                             // chosen but dead: the pull failed
            const uint32_t dead = uint32_t(-2 - p[s]);
            if (index_ok(n, dead, n.N, 109)) {
                const uint64_t mark = n.view[x * n.ld + dead] | kOffBit, cur = vn[x * n.ld + dead];
                if (mark > cur) vn[x * n.ld + dead] = mark;
                ++marks;
            }
        } else if (index_ok(n, p[s], n.N, 110)) vn[(size_t(r) * n.N + p[s]) * n.ld + i] = self;
    }
    if (marks) atomicAdd(&n.stats[size_t(r) * sCount + sOfflineMarks], (unsigned long long)marks);
}

// per-peer exclusive prefix sums of in_deg into in_off (also clears in_cursor); shared with the
// intra-batch queueing of the settlement
void launch_scan_in_degrees(const Net& n, const LaunchCtx& c, int kernel_id)
{
    Timed t(c, kernel_id);
    launch_kernel(c, k_gossip_scan, n.Rp, 1024, n);
}

// Panel width: the widest power of two (32 .. 512 columns) whose panel of N rows fits the
// L2 budget; WWWS_PANEL_BYTES overrides the budget (tuning).
static uint32_t panel_columns(const Net& n)
{
    static const uint64_t budget = [] {
        const char* e = getenv("WWWS_PANEL_BYTES");
        const uint64_t v = e ? strtoull(e, nullptr, 10) : 0;
        return v ? v : (16ull << 20);
    }();
    uint32_t pc = 4 * kMergeThreads;                                      // one pass of the block covers at least one row segment
    while (pc > 32 && uint64_t(n.N) * pc * 8 > budget) pc >>= 1;
    return pc;
}

void launch_gossip(const Net& n, uint32_t round, const LaunchCtx& c)
{
    const dim3 pg((n.N + 127) / 128, n.Rp);
    { Timed t(c, kGossipPeer); launch_kernel(c, k_gossip_peer, pg, 128, n, round); }
    { Timed t(c, kGossipPeer); launch_kernel(c, k_gossip_resolve, pg, 128, n); }
    const uint32_t pc = panel_columns(n);
    uint32_t shift = 0;
    while ((4u << shift) < pc) ++shift;                                   // 32-byte chunks per row segment = pc / 4
    const uint32_t rows_per_block = (kMergeThreads >> shift) * kMergeIters;
    const uint32_t n_panels = (n.ld + pc - 1) / pc;
    const uint32_t groups = (n.N + rows_per_block - 1) / rows_per_block;
    const uint64_t blocks = uint64_t(n.Rp) * n_panels * groups;
    if (n.flags & 8u) {
        { Timed t(c, kGossipLists); launch_kernel(c, k_gossip_indeg, pg, 128, n); }
        { Timed t(c, kGossipLists); launch_kernel(c, k_gossip_scan, n.Rp, 1024, n); }
        { Timed t(c, kGossipLists); launch_kernel(c, k_gossip_fill, pg, 128, n); }
        Timed t(c, kGossipMerge);
        launch_kernel(c, k_gossip_merge<true>, uint32_t(blocks), kMergeThreads, n, pc, shift, n_panels, groups);
    } else {
        Timed t(c, kGossipMerge);
        launch_kernel(c, k_gossip_merge<false>, uint32_t(blocks), kMergeThreads, n, pc, shift, n_panels, groups);
    }
    { Timed t(c, kGossipFixup); launch_kernel(c, k_gossip_fixup, pg, 128, n); }
}

}  // namespace wwws
