// Gossip round: churn + self entries + partner choice (per peer), row merge (streaming
// 64-bit max over gathered rows), and the scattered single-entry updates.
#include "wwws_internal.cuh"

namespace wwws {

// G0 churn, G1 new version of the own entry, partner choice of G2 (reads the old view only).
__global__ void k_gossip_peer(Net n, uint32_t round)
{
    const uint32_t r = blockIdx.y, i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n.N) return;
    const uint32_t rg = r + n.replica_offset;
    const size_t x = size_t(r) * n.N + i;
    bool on = n.online[x] != 0;
    if (n.p_leave | n.p_join) {
        const uint32_t u = ppm(draw(n, i, round, rg, kChurn).w[0]);
        if (on) { if (u < n.p_leave) { on = false; n.backlog[x] = 0; n.online[x] = 0; } }
        else if (u < n.p_join) { on = true; n.online[x] = 1; }
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
#pragma unroll
            for (uint32_t s = 0; s < 4; ++s) {
                if (!(open >> s & 1u)) continue;
                const uint32_t p = below(g.w[s], n.N);
                if (p == i) continue;
                const uint64_t e = row[p];
                if (e != 0 && !(e & kOffBit)) { part[s] = int32_t(p); open &= ~(1u << s); }
            }
        }
    }
    n.self_entry[x] = self;
    *reinterpret_cast<int4*>(n.partner + x * 4) = make_int4(part[0], part[1], part[2], part[3]);
}

// Streaming merge.  One block handles `kTile` consecutive columns of one row: new row =
// max(old row, rows of the partners that answered).  16-byte vector accesses; the partner
// rows are independent loads, so each thread keeps (1+k) * kUnroll loads in flight.
constexpr int kMergeThreads = 256;
constexpr int kUnroll = 2;
constexpr int kTile = kMergeThreads * 2 * kUnroll;   // columns per block

__device__ __forceinline__ ulonglong2 ld16(const uint64_t* p)
{
    ulonglong2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u64 {%0,%1}, [%2];" : "=l"(v.x), "=l"(v.y) : "l"(p));
    return v;
}
__device__ __forceinline__ void st16(uint64_t* p, ulonglong2 v)
{
    asm volatile("st.global.L1::no_allocate.v2.u64 [%0], {%1,%2};" ::"l"(p), "l"(v.x), "l"(v.y) : "memory");
}
__device__ __forceinline__ uint64_t umax64(uint64_t a, uint64_t b) { return a > b ? a : b; }

__global__ void __launch_bounds__(kMergeThreads) k_gossip_merge(Net n, uint32_t tiles_per_row)
{
    const uint64_t blk = uint64_t(blockIdx.y) * gridDim.x + blockIdx.x;   // over Rp * N * tiles_per_row
    const uint64_t rowid = blk / tiles_per_row;                             // r * N + i
    if (rowid >= uint64_t(n.Rp) * n.N) return;
    const uint32_t tile = uint32_t(blk - rowid * tiles_per_row);
    const uint32_t r = uint32_t(rowid / n.N);
    const uint64_t* src[4];
    int ns = 0;
    if (n.online[rowid]) {
        const int4 p4 = *reinterpret_cast<const int4*>(n.partner + rowid * 4);
        const int32_t p[4] = { p4.x, p4.y, p4.z, p4.w };
#pragma unroll
        for (int s = 0; s < 4; ++s)
            if (p[s] >= 0 && n.online[size_t(r) * n.N + p[s]]) src[ns++] = n.view + (size_t(r) * n.N + p[s]) * n.ld;
    }
    const uint64_t* own = n.view + rowid * n.ld;
    uint64_t* out = n.view_new + rowid * n.ld;
    const uint32_t c0 = tile * kTile + threadIdx.x * 2;
    ulonglong2 acc[kUnroll];
    bool live[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
        const uint32_t c = c0 + u * kMergeThreads * 2;
        live[u] = c < n.ld;
        acc[u] = live[u] ? ld16(own + c) : make_ulonglong2(0, 0);
    }
    for (int s = 0; s < ns; ++s) {
        ulonglong2 v[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const uint32_t c = c0 + u * kMergeThreads * 2;
            v[u] = live[u] ? ld16(src[s] + c) : make_ulonglong2(0, 0);
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) { acc[u].x = umax64(acc[u].x, v[u].x); acc[u].y = umax64(acc[u].y, v[u].y); }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u)
        if (live[u]) st16(out + c0 + u * kMergeThreads * 2, acc[u]);
}

// The three single-entry updates of a round, all joins (max), applied after the row merge:
// own fresh entry, offline mark for a partner that did not answer, and the "hello" that shows
// the puller's entry to the partner.
__global__ void k_gossip_fixup(Net n)
{
    const uint32_t r = blockIdx.y, i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n.N) return;
    const size_t x = size_t(r) * n.N + i;
    if (i == 0) atomicAdd(&n.stats[size_t(r) * sCount + sRounds], 1ull);
    if (!n.online[x]) return;
    const uint64_t self = n.self_entry[x];
    unsigned long long* vn = reinterpret_cast<unsigned long long*>(n.view_new);
    atomicMax(vn + x * n.ld + i, self);
    const int4 p4 = *reinterpret_cast<const int4*>(n.partner + x * 4);
    const int32_t p[4] = { p4.x, p4.y, p4.z, p4.w };
    uint32_t marks = 0;
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        if (p[s] < 0) continue;
        const size_t px = size_t(r) * n.N + p[s];
        if (!n.online[px]) { atomicMax(vn + x * n.ld + p[s], n.view[x * n.ld + p[s]] | kOffBit); ++marks; }
        else atomicMax(vn + px * n.ld + i, self);
    }
    if (marks) atomicAdd(&n.stats[size_t(r) * sCount + sOfflineMarks], (unsigned long long)marks);
}

void launch_gossip(const Net& n, uint32_t round, const LaunchCtx& c)
{
    const dim3 pg((n.N + 127) / 128, n.Rp);
    { Timed t(c, kGossipPeer); k_gossip_peer<<<pg, 128, 0, c.stream>>>(n, round); }
    const uint32_t tiles = (n.ld + kTile - 1) / kTile;
    const uint64_t blocks = uint64_t(n.Rp) * n.N * tiles;
    const uint32_t gx = blocks > 65535u * 32u ? 65535u * 32u : uint32_t(blocks);   // x up to 2^31-1; keep y small
    const uint32_t gy = uint32_t((blocks + gx - 1) / gx);
    { Timed t(c, kGossipMerge); k_gossip_merge<<<dim3(gx, gy), kMergeThreads, 0, c.stream>>>(n, tiles); }
    { Timed t(c, kGossipFixup); k_gossip_fixup<<<pg, 128, 0, c.stream>>>(n); }
}

}  // namespace wwws
