// C-ABI of the wwws library: argument checks, workspace layout, call ordering, copies.
#include <atomic>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "../../include/wwws.h"
#include "wwws_internal.cuh"

using namespace wwws;

static_assert(sizeof(wwws_stats_t) == sCount * 8, "stats record and counter table must agree");

struct wwws_network {
    Net d;                       // device pointers and scalars
    wwws_config cfg;
    cudaStream_t stream;
    int device;                  // ordinal of the GPU that holds the workspace; every call runs there
    uint8_t* ws; uint64_t ws_bytes;
    uint32_t t_last_ms, round;
    int phase;                   // 0 idle, 1 dispatched, 2 judged
    uint64_t batch_first; uint32_t batch_count;
    bool bound;
    int request_kernel;          // 0 by launch size, 1 warp per request, 2 thread per request
    int step_kernel;             // fused step: 0 by launch size, 1/2 eight/four lanes per request, 3 one thread, 4 streaming phases
    uint32_t stream_run;         // requests per warp of the streaming kernel, 0 = by launch size
    uint64_t launches;
    Profiler prof;
    std::string err;
    bool fold_pending = false;   // wwws_step left its fold to the next call (see settle_pending)
    int fold_finalize = 0;
    int host_io = 0;             // wwws_step_host: 0 by batch size, 1 kernels use mapped host buffers, 2 staged copies
    cudaStream_t copy_stream = nullptr;          // staged host path: copies run beside the kernels
    cudaEvent_t ev_fork = nullptr, ev_in = nullptr, ev_step = nullptr;
    int overlap = 0;             // which launches may overlap their predecessor's tail (WWWS_OPT_LAUNCH_OVERLAP):
                                 // bit 0 time advance, 1 gossip, 2 request kernels, 3 fold; other kernels follow bit 0.
                                 // Set at creation: all for small networks, whose steps are a chain of launch latencies;
                                 // none for large ones, where a chain of early-resident waiting grids slowed the step down
                                 // (1,024 peers x 256 replicas: 0.47 ms per step plain, 0.61 ms with every launch overlapped)
    LaunchCtx ctx(int kind = 1) { return LaunchCtx{ stream, &launches, &prof, (overlap & kind) != 0 && !prof.enabled }; }
    struct TableInfo { void* ptr; uint32_t elem; } tables[WWWS_T_COUNT];
};

namespace {

thread_local std::string g_err;   // errors of calls that have no handle to keep them in

wwws_status fail(wwws_network* n, wwws_status st, const std::string& msg)
{
    if (n) n->err = msg; else g_err = msg;
    return st;
}

#define CUDA_TRY(net, call)                                                                      \
    do {                                                                                         \
        cudaError_t e_ = (call);                                                                 \
        if (e_ != cudaSuccess) return fail(net, WWWS_ERR_CUDA, std::string(#call) + ": " + cudaGetErrorString(e_)); \
    } while (0)

// Makes the network's GPU current for the duration of a call and puts the caller's back
// afterwards: a handle works whatever device the calling thread has selected.
struct DeviceScope {
    int prev = -1; bool switched = false; cudaError_t err;
    explicit DeviceScope(int want)
    {
        err = cudaGetDevice(&prev);
        if (err == cudaSuccess && prev != want) { err = cudaSetDevice(want); switched = err == cudaSuccess; }
    }
    ~DeviceScope() { if (switched) cudaSetDevice(prev); }
    DeviceScope(const DeviceScope&) = delete;
    DeviceScope& operator=(const DeviceScope&) = delete;
};
#define ON_DEVICE(net)                                                                           \
    DeviceScope device_scope_((net)->device);                                                    \
    if (device_scope_.err != cudaSuccess)                                                        \
        return fail(net, WWWS_ERR_CUDA, std::string("selecting the network's device: ") + cudaGetErrorString(device_scope_.err))

const char* check_config(const wwws_config* c)
{
    if (!c) return "config is NULL";
    if (c->n_peers < 2 || c->n_peers > 65535) return "n_peers must be 2..65535";
    if (c->n_replicas < 1 || c->n_replicas > 65535) return "n_replicas must be 1..65535";
    if (uint64_t(c->replica_offset) + c->n_replicas > 0xffffffffull) return "replica_offset + n_replicas overflows";
    if (c->max_batch < 1) return "max_batch must be >= 1";
    if (c->fanout_k < 1 || c->fanout_k > 4) return "fanout_k must be 1..4";
    if (c->gossip_tries < 1 || c->gossip_tries > 64) return "gossip_tries must be 1..64";
    if (c->max_probes < 1 || c->max_probes > 15) return "max_probes must be 1..15";
    if (c->n_judges < 1 || c->n_judges > WWWS_MAX_JUDGES) return "n_judges must be 1..4";
    if (c->p_duel_ppm > 1000000 || c->p_noise_ppm > 1000000 || c->p_leave_ppm > 1000000 || c->p_join_ppm > 1000000 ||
        c->p_prio_active_ppm > 1000000)
        return "probabilities are in ppm (0..1000000)";
    if (c->prio_window_ms == 0 || c->util_window_ms == 0 || c->cap_ref_tok_s == 0 || c->slo_den == 0)
        return "prio_window_ms, util_window_ms, cap_ref_tok_s and slo_den must be > 0";
    if (c->init_stale_max >= (1u << 24) - 2) return "init_stale_max must be < 2^24 - 2";
    if (c->reward_R <= 0 || c->reward_add <= 0 || c->reward_add > c->penalty_P) return "need R > 0 and 0 < R_add <= P";
    if (c->reward_R > (1ll << 40) || c->penalty_P > (1ll << 40)) return "rewards must be <= 2^40";
    if ((c->rank_cdf == nullptr) != (c->n_rank == 0)) return "rank_cdf and n_rank must be given together";
    if (c->n_rank > 65536) return "n_rank must be <= 65536";
    for (uint32_t i = 1; i < c->n_rank; ++i)
        if (c->rank_cdf[i] < c->rank_cdf[i - 1]) return "rank_cdf must be nondecreasing";
    return nullptr;
}

// Workspace carving: the same walk computes the size (base == nullptr) and the pointers.
struct Carver {
    uint8_t* base; uint64_t off;
    template <class T> T* take(uint64_t count)
    {
        off = (off + 255) & ~uint64_t(255);
        T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
        off += count * sizeof(T);
        return p;
    }
};

struct Staging {   // device copies of creation-only inputs, at the end of the workspace
    int64_t* credit0; uint8_t* online0;
};

void carve(const wwws_config& c, Carver& cv, Net& d, Staging& sg)
{
    const uint64_t N = c.n_peers, Rp = c.n_replicas, NP = N * Rp;
    const uint64_t ld = (N + kWin - 1) / kWin * kWin;
    d.view = cv.take<uint64_t>(NP * ld);
    d.view_new = cv.take<uint64_t>(NP * ld);
    d.cap_true = cv.take<uint32_t>(NP); d.quality = cv.take<uint32_t>(NP);
    d.stake_pm = cv.take<uint16_t>(NP); d.offload_util_pm = cv.take<uint16_t>(NP); d.accept_util_pm = cv.take<uint16_t>(NP);
    d.offload_ppm = cv.take<uint32_t>(NP); d.accept_ppm = cv.take<uint32_t>(NP);
    d.misreport = cv.take<uint8_t>(NP); d.prio_flag = cv.take<uint8_t>(NP);
    d.online = cv.take<uint8_t>(NP); d.cap_eff = cv.take<uint32_t>(NP); d.backlog = cv.take<int64_t>(NP);
    d.ver = cv.take<uint32_t>(NP);
    d.credit = cv.take<int64_t>(NP); d.stake = cv.take<int64_t>(NP); d.wins = cv.take<uint32_t>(NP);
    d.duels = cv.take<uint32_t>(NP);
    d.served = cv.take<unsigned long long>(NP); d.served_local = cv.take<unsigned long long>(NP);
    d.d_credit = cv.take<long long>(NP); d.d_wins = cv.take<uint32_t>(NP); d.d_duels = cv.take<uint32_t>(NP);
    d.d_backlog = cv.take<long long>(NP);
    d.w_led = cv.take<float>(Rp * ld);
    d.gate = cv.take<uint64_t>(NP);
    d.self_entry = cv.take<uint64_t>(NP); d.partner = cv.take<int32_t>(NP * 4);
    d.in_deg = cv.take<uint32_t>(NP); d.in_off = cv.take<uint32_t>(NP); d.in_cursor = cv.take<uint32_t>(NP);
    d.pullers = cv.take<int32_t>(NP * 4);
    d.fifo_items = cv.take<int2>(Rp * uint64_t(c.max_batch) * 7); d.fifo_list = cv.take<uint2>(Rp * uint64_t(c.max_batch) * 7);
    d.blk_spent = cv.take<long long>(NP); d.d_spent = cv.take<long long>(NP);
    d.cont = cv.take<uint2>(Rp * uint64_t(c.max_batch));
    d.rank_cdf = c.n_rank ? cv.take<uint32_t>(c.n_rank) : nullptr;
    d.stats = cv.take<unsigned long long>(Rp * sCount);
    d.credit_total0 = cv.take<int64_t>(Rp); d.credit_check = cv.take<long long>(Rp);
    d.fold_ticket = cv.take<uint32_t>(Rp); d.online_count = cv.take<uint32_t>(Rp);
    d.err = cv.take<uint32_t>(4);
    sg.credit0 = cv.take<int64_t>(NP); sg.online0 = cv.take<uint8_t>(NP);
    cv.off = (cv.off + 255) & ~uint64_t(255);
}

// Device-side problems surface at synchronising calls.
wwws_status check_device_error(wwws_network* n)
{
    uint32_t e[2] = { 0, 0 };
    CUDA_TRY(n, cudaMemcpyAsync(e, n->d.err, sizeof e, cudaMemcpyDeviceToHost, n->stream));
    CUDA_TRY(n, cudaStreamSynchronize(n->stream));
    if (e[0] == 0) return WWWS_OK;
    CUDA_TRY(n, cudaMemsetAsync(n->d.err, 0, 8, n->stream));
    char buf[160];
    switch (e[0]) {
    case eRange: snprintf(buf, sizeof buf, "version counter of peer %u reached 2^24", e[1]); return fail(n, WWWS_ERR_RANGE, buf);
    case eInvariant: snprintf(buf, sizeof buf, "total credit of replica %u changed across finalization", e[1]); return fail(n, WWWS_ERR_INVARIANT, buf);
    case eArg: snprintf(buf, sizeof buf, "request with origin index %u >= n_peers (dropped)", e[1]); return fail(n, WWWS_ERR_ARG, buf);
    case eIndex: snprintf(buf, sizeof buf, "checked build: an index taken from device data was out of range at site %u (access skipped)", e[1]); return fail(n, WWWS_ERR_INDEX, buf);
    default: snprintf(buf, sizeof buf, "device error word %u/%u", e[0], e[1]); return fail(n, WWWS_ERR_CUDA, buf);
    }
}

wwws_status launch_status(wwws_network* n, const char* what)
{
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(n, WWWS_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
    return WWWS_OK;
}

// wwws_step does not fold its batch (queues, block commit) itself: the next wwws_step does it in
// the same launch as its time advance.  Every other call that reads or changes the state folds
// first, so the deferral is never visible.
void settle_pending(wwws_network* n)
{
    if (!n->fold_pending) return;
    n->fold_pending = false;
    launch_fold(n->d, n->fold_finalize, n->ctx(8));
}

}  // namespace

extern "C" {

wwws_status wwws_workspace_bytes(const wwws_config* cfg, uint64_t* bytes_out)
{
    if (!bytes_out) return fail(nullptr, WWWS_ERR_ARG, "bytes_out is NULL");
    if (const char* m = check_config(cfg)) return fail(nullptr, WWWS_ERR_ARG, m);
    Carver cv{ nullptr, 0 }; Net d{}; Staging sg{};
    carve(*cfg, cv, d, sg);
    *bytes_out = cv.off;
    return WWWS_OK;
}

wwws_status wwws_create_network(const wwws_config* cfg, const wwws_peer_init* init, void* workspace,
                                uint64_t workspace_bytes, void* cuda_stream, wwws_network** out)
{
    if (!out) return fail(nullptr, WWWS_ERR_ARG, "out is NULL");
    *out = nullptr;
    if (const char* m = check_config(cfg)) return fail(nullptr, WWWS_ERR_ARG, m);
    if (!init) return fail(nullptr, WWWS_ERR_ARG, "peer init is NULL");
    const void* fields[] = { init->cap_true_tok_s, init->quality_fx, init->credit0, init->stake_pm, init->offload_util_pm,
                             init->accept_util_pm, init->offload_ppm, init->accept_ppm, init->misreport_mul,
                             init->prio_flag, init->online0 };
    for (const void* f : fields) if (!f) return fail(nullptr, WWWS_ERR_ARG, "a peer init array is NULL");
    const uint64_t NP = uint64_t(cfg->n_peers) * cfg->n_replicas;
    for (uint64_t x = 0; x < NP; ++x) {
        if (init->stake_pm[x] > 1000) return fail(nullptr, WWWS_ERR_ARG, "stake_pm must be <= 1000");
        if (init->offload_ppm[x] > 1000000 || init->accept_ppm[x] > 1000000) return fail(nullptr, WWWS_ERR_ARG, "frequencies are in ppm");
        if (init->credit0[x] > (1ll << 40) || init->credit0[x] < -(1ll << 40)) return fail(nullptr, WWWS_ERR_ARG, "|credit0| must be <= 2^40");
        if (init->misreport_mul[x] == 0) return fail(nullptr, WWWS_ERR_ARG, "misreport_mul must be >= 1");
    }
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255)) return fail(nullptr, WWWS_ERR_ALLOC, "workspace is NULL or not 256-byte aligned");
    // the GPU that holds the workspace is the network's GPU, whatever device is current now or later
    cudaPointerAttributes wa;
    if (cudaError_t e = cudaPointerGetAttributes(&wa, workspace); e != cudaSuccess) {
        cudaGetLastError();
        return fail(nullptr, WWWS_ERR_CUDA, std::string("cudaPointerGetAttributes(workspace): ") + cudaGetErrorString(e));
    }
    if (wa.type != cudaMemoryTypeDevice && wa.type != cudaMemoryTypeManaged)
        return fail(nullptr, WWWS_ERR_ARG, "workspace is not device memory");
    Carver cv{ static_cast<uint8_t*>(workspace), 0 };
    wwws_network* n = new (std::nothrow) wwws_network();
    if (!n) return fail(nullptr, WWWS_ERR_ALLOC, "host allocation failed");
    n->device = wa.device;
    struct Guard { wwws_network* n; ~Guard() { delete n; } } guard{ n };     // freed on every failure below
    DeviceScope device_scope_(n->device);
    if (device_scope_.err != cudaSuccess)
        return fail(nullptr, WWWS_ERR_CUDA, std::string("selecting the workspace's device: ") + cudaGetErrorString(device_scope_.err));
    Staging sg{};
    carve(*cfg, cv, n->d, sg);
    if (cv.off > workspace_bytes) return fail(nullptr, WWWS_ERR_ALLOC, "workspace too small");
    n->cfg = *cfg; n->cfg.rank_cdf = nullptr;
    n->stream = static_cast<cudaStream_t>(cuda_stream);
    n->overlap = uint64_t(cfg->n_peers) * cfg->n_replicas <= 32768 ? 15 : 0;
    n->ws = static_cast<uint8_t*>(workspace); n->ws_bytes = workspace_bytes;
    Net& d = n->d;
    d.N = cfg->n_peers; d.Rp = cfg->n_replicas; d.ld = (d.N + kWin - 1) / kWin * kWin; d.n_blk = d.ld / kWin;
    d.replica_offset = cfg->replica_offset;
    d.key0 = uint32_t(cfg->seed); d.key1 = uint32_t(cfg->seed >> 32);
    d.fanout_k = cfg->fanout_k; d.gossip_tries = cfg->gossip_tries; d.max_probes = cfg->max_probes; d.n_judges = cfg->n_judges;
    d.p_duel = cfg->p_duel_ppm; d.p_noise = cfg->p_noise_ppm; d.p_leave = cfg->p_leave_ppm; d.p_join = cfg->p_join_ppm;
    d.p_prio = cfg->p_prio_active_ppm;
    d.prio_window_ms = cfg->prio_window_ms; d.util_window_ms = cfg->util_window_ms; d.cap_ref = cfg->cap_ref_tok_s;
    d.slo_num = cfg->slo_num; d.slo_den = cfg->slo_den; d.hop_ms = cfg->hop_ms; d.flags = cfg->flags; d.n_rank = cfg->n_rank;
    d.R = cfg->reward_R; d.R_add = cfg->reward_add; d.P = cfg->penalty_P;
    for (int k = 0; k < 4; ++k) d.judge_share[k] = (d.P - d.R_add) / (k + 1);
    d.uwf = float(cfg->util_window_ms) / 1000.0f;
    d.max_batch = cfg->max_batch;

    wwws_network::TableInfo ti[WWWS_T_COUNT] = {
        { d.online, 1 }, { d.cap_eff, 4 }, { d.backlog, 8 }, { d.ver, 4 }, { d.credit, 8 }, { d.stake, 8 }, { d.wins, 4 },
        { d.duels, 4 }, { d.served, 8 }, { d.served_local, 8 }, { d.d_credit, 8 }, { d.d_wins, 4 }, { d.d_duels, 4 },
        { d.blk_spent, 8 } };
    memcpy(n->tables, ti, sizeof ti);

    cudaStream_t s = n->stream;
#define H2D(dst, src, T) CUDA_TRY(nullptr, cudaMemcpyAsync(const_cast<T*>(dst), src, NP * sizeof(T), cudaMemcpyHostToDevice, s))
    H2D(d.cap_true, init->cap_true_tok_s, uint32_t); H2D(d.quality, init->quality_fx, uint32_t);
    H2D(d.stake_pm, init->stake_pm, uint16_t); H2D(d.offload_util_pm, init->offload_util_pm, uint16_t);
    H2D(d.accept_util_pm, init->accept_util_pm, uint16_t);
    H2D(d.offload_ppm, init->offload_ppm, uint32_t); H2D(d.accept_ppm, init->accept_ppm, uint32_t);
    H2D(d.misreport, init->misreport_mul, uint8_t); H2D(d.prio_flag, init->prio_flag, uint8_t);
    H2D(sg.credit0, init->credit0, int64_t); H2D(sg.online0, init->online0, uint8_t);
#undef H2D
    if (cfg->n_rank)
        CUDA_TRY(nullptr, cudaMemcpyAsync(const_cast<uint32_t*>(d.rank_cdf), cfg->rank_cdf, cfg->n_rank * 4ull, cudaMemcpyHostToDevice, s));
    std::vector<int64_t> tot(d.Rp, 0);
    for (uint32_t r = 0; r < d.Rp; ++r)
        for (uint32_t j = 0; j < d.N; ++j) tot[r] += init->credit0[size_t(r) * d.N + j];
    CUDA_TRY(nullptr, cudaMemcpyAsync(const_cast<int64_t*>(d.credit_total0), tot.data(), d.Rp * 8ull, cudaMemcpyHostToDevice, s));
    {   // counters start at zero, each replica's chain at its genesis id
        std::vector<unsigned long long> st0(size_t(d.Rp) * sCount, 0);
        for (uint32_t r = 0; r < d.Rp; ++r)
            st0[size_t(r) * sCount + sChainHead] = mix64(cfg->seed ^ (uint64_t(r + cfg->replica_offset) * kGamma));
        CUDA_TRY(nullptr, cudaMemcpy(d.stats, st0.data(), st0.size() * 8, cudaMemcpyHostToDevice));
    }
    CUDA_TRY(nullptr, cudaMemsetAsync(d.credit_check, 0, d.Rp * 8ull, s));
    CUDA_TRY(nullptr, cudaMemsetAsync(d.fold_ticket, 0, d.Rp * 4ull, s));
    CUDA_TRY(nullptr, cudaMemsetAsync(d.online_count, 0, d.Rp * 4ull, s));
    CUDA_TRY(nullptr, cudaMemsetAsync(d.err, 0, 16, s));
    CUDA_TRY(nullptr, cudaMemsetAsync(d.partner, 0xff, NP * 16, s));
    CUDA_TRY(nullptr, cudaMemsetAsync(d.in_deg, 0, NP * 4, s));
    CUDA_TRY(nullptr, cudaMemsetAsync(d.w_led, 0, uint64_t(d.Rp) * d.ld * 4, s));   // padding columns stay 0
    launch_peer_init(d, sg.credit0, sg.online0, cfg->init_stale_max, n->ctx());
    if (cudaError_t e = cudaGetLastError(); e != cudaSuccess) return fail(nullptr, WWWS_ERR_CUDA, std::string("initialisation kernels: ") + cudaGetErrorString(e));
    // host staging (`tot`, the caller's arrays) must stay valid until the copies are done
    CUDA_TRY(nullptr, cudaStreamSynchronize(s));
    guard.n = nullptr;
    *out = n;
    return WWWS_OK;
}

wwws_status wwws_destroy_network(wwws_network* n)
{
    if (!n) return WWWS_OK;
    {
        DeviceScope scope(n->device);
        cudaStreamSynchronize(n->stream);
        if (n->copy_stream) {
            cudaStreamSynchronize(n->copy_stream);
            cudaEventDestroy(n->ev_fork); cudaEventDestroy(n->ev_in); cudaEventDestroy(n->ev_step);
            cudaStreamDestroy(n->copy_stream);
        }
    }
    delete n;
    return WWWS_OK;
}

wwws_status wwws_bind_requests(wwws_network* n, const wwws_requests* req, const wwws_results* res)
{
    if (!n) return fail(nullptr, WWWS_ERR_ARG, "network is NULL");
    if (!req || !res) return fail(n, WWWS_ERR_ARG, "requests or results is NULL");
    if (!req->origin || !req->len_in || !req->len_out) return fail(n, WWWS_ERR_ARG, "a request array is NULL");
    if (!res->exec_a || !res->exec_b || !res->judges || !res->outcome || !res->flags) return fail(n, WWWS_ERR_ARG, "a result array is NULL");
    if (req->n_requests == 0 || req->n_requests >= (1ull << 32)) return fail(n, WWWS_ERR_ARG, "n_requests must be 1..2^32-1");
    if (reinterpret_cast<uintptr_t>(res->judges) & 15) return fail(n, WWWS_ERR_ARG, "judges must be 16-byte aligned");
    if (n->phase != 0) return fail(n, WWWS_ERR_STATE, "a batch is in flight: settle it before rebinding");
    Net& d = n->d;
    d.origin = req->origin; d.len_in = req->len_in; d.len_out = req->len_out; d.Q = req->n_requests;
    d.exec_a = res->exec_a; d.exec_b = res->exec_b; d.judges = res->judges; d.outcome = res->outcome; d.rflags = res->flags;
    d.score_a = res->score_a; d.score_sum = res->score_sum;
    n->bound = true;
    return WWWS_OK;
}

wwws_status wwws_advance_time(wwws_network* n, uint32_t now_ms)
{
    if (!n) return fail(nullptr, WWWS_ERR_ARG, "network is NULL");
    if (now_ms < n->t_last_ms) return fail(n, WWWS_ERR_ARG, "time must not go back");
    if (n->phase != 0) return fail(n, WWWS_ERR_STATE, "advance_time inside a batch");
    ON_DEVICE(n);
    settle_pending(n);
    launch_advance(n->d, now_ms - n->t_last_ms, now_ms, n->ctx());
    n->t_last_ms = now_ms;
    return launch_status(n, "advance_time");
}

wwws_status wwws_gossip_round(wwws_network* n)
{
    if (!n) return fail(nullptr, WWWS_ERR_ARG, "network is NULL");
    if (n->phase != 0) return fail(n, WWWS_ERR_STATE, "gossip_round inside a batch");
    ON_DEVICE(n);
    settle_pending(n);
    launch_gossip(n->d, n->round, n->ctx());
    std::swap(n->d.view, n->d.view_new);
    n->round += 1;
    return launch_status(n, "gossip_round");
}

static wwws_status check_batch(wwws_network* n, uint64_t first, uint64_t count)
{
    if (!n) return fail(nullptr, WWWS_ERR_ARG, "network is NULL");
    if (!n->bound) return fail(n, WWWS_ERR_STATE, "no requests bound");
    if (n->phase != 0) return fail(n, WWWS_ERR_STATE, "previous batch not settled");
    if (count == 0 || count > n->cfg.max_batch) return fail(n, WWWS_ERR_ARG, "count must be 1..max_batch");
    if (first + count > n->d.Q || first + count < first) return fail(n, WWWS_ERR_ARG, "batch exceeds n_requests");
    return WWWS_OK;
}

// The separate dispatch and duel calls have two implementations with identical results: one warp
// per request (lane per candidate; shortest latency, best for small batches) and one thread per
// request (far fewer instructions per request; best from a few thousand requests per launch).
static bool threads_for(const wwws_network* n, uint64_t count)
{
    if (n->request_kernel == 1) return false;
    if (n->request_kernel == 2) return true;
    return count * n->d.Rp >= 8192;
}

wwws_status wwws_dispatch_batch(wwws_network* n, uint64_t first, uint64_t count)
{
    if (wwws_status st = check_batch(n, first, count)) return st;
    ON_DEVICE(n);
    settle_pending(n);
    if (threads_for(n, count)) launch_dispatch_threads(n->d, first, uint32_t(count), n->ctx());
    else launch_dispatch(n->d, first, uint32_t(count), n->ctx());
    n->batch_first = first; n->batch_count = uint32_t(count); n->phase = 1;
    return launch_status(n, "dispatch_batch");
}

wwws_status wwws_duel_judge(wwws_network* n)
{
    if (!n) return fail(nullptr, WWWS_ERR_ARG, "network is NULL");
    if (n->phase != 1) return fail(n, WWWS_ERR_STATE, "duel_judge must follow dispatch_batch");
    ON_DEVICE(n);
    if (threads_for(n, n->batch_count)) launch_duel_threads(n->d, n->batch_first, n->batch_count, n->ctx());
    else launch_duel(n->d, n->batch_first, n->batch_count, n->ctx());
    n->phase = 2;
    return launch_status(n, "duel_judge");
}

wwws_status wwws_settle_credits(wwws_network* n, int finalize)
{
    if (!n) return fail(nullptr, WWWS_ERR_ARG, "network is NULL");
    if (n->phase != 2) return fail(n, WWWS_ERR_STATE, "settle_credits must follow duel_judge");
    ON_DEVICE(n);
    launch_settle(n->d, n->batch_first, n->batch_count, n->ctx());
    if (n->d.flags & 16u) launch_fifo(n->d, n->batch_first, n->batch_count, n->ctx());
    launch_fold(n->d, finalize != 0, n->ctx());
    n->phase = 0;
    return launch_status(n, "settle_credits");
}

// One step; `inputs_ready` (may be null) is waited for before the request kernel, `results_ready`
// (may be null) is recorded right after it: the staged host path copies beside the other kernels.
static wwws_status step_impl(wwws_network* n, uint64_t first, uint64_t count, uint32_t now_ms, int do_gossip, int finalize,
                             cudaEvent_t inputs_ready, cudaEvent_t results_ready)
{
    if (n->fold_pending && !(n->d.flags & 32u)) {
        n->fold_pending = false;
        launch_fold_advance(n->d, n->fold_finalize, now_ms - n->t_last_ms, now_ms, n->ctx(1));
    } else {
        settle_pending(n);
        launch_advance(n->d, now_ms - n->t_last_ms, now_ms, n->ctx(1));
    }
    n->t_last_ms = now_ms;
    if (do_gossip) {
        launch_gossip(n->d, n->round, n->ctx(2));
        std::swap(n->d.view, n->d.view_new);
        n->round += 1;
    }
    if (inputs_ready) CUDA_TRY(n, cudaStreamWaitEvent(n->stream, inputs_ready, 0));
    launch_step_fused(n->d, first, uint32_t(count), n->ctx(4), n->step_kernel, n->stream_run);
    if (results_ready) CUDA_TRY(n, cudaEventRecord(results_ready, n->stream));
    if (n->d.flags & 16u) launch_fifo(n->d, first, uint32_t(count), n->ctx(4));
    n->fold_pending = true;                      // folded by the next call, whichever it is
    n->fold_finalize = finalize != 0;
    return launch_status(n, "step");
}

wwws_status wwws_step(wwws_network* n, uint64_t first, uint64_t count, uint32_t now_ms, int do_gossip, int finalize)
{
    if (wwws_status st = check_batch(n, first, count)) return st;
    if (now_ms < n->t_last_ms) return fail(n, WWWS_ERR_ARG, "time must not go back");
    ON_DEVICE(n);
    return step_impl(n, first, count, now_ms, do_gossip, finalize, nullptr, nullptr);
}

wwws_status wwws_step_host(wwws_network* n, const wwws_host_io* io, uint64_t first, uint64_t count, uint32_t now_ms,
                           int do_gossip, int finalize, wwws_stats_t* totals_out)
{
    if (wwws_status st = check_batch(n, first, count)) return st;
    if (!io || !io->origin || !io->len_in || !io->len_out || !io->exec_a || !io->exec_b || !io->judges || !io->outcome || !io->flags)
        return fail(n, WWWS_ERR_ARG, "a host buffer is NULL");
    ON_DEVICE(n);
    if (now_ms < n->t_last_ms) return fail(n, WWWS_ERR_ARG, "time must not go back");
    // Large batches go through staged copies even when the buffers are mapped: result records written
    // across the bus request by request, in the order the kernel finishes them, cost more than two
    // small copy kernels that run beside the others (measured per step, direct / staged: 64,000
    // requests 0.67 / 0.70 ms, 128,000 requests 0.94 / 0.62 ms).
    const bool want_direct = n->host_io == 1 || (n->host_io == 0 && count * n->d.Rp <= 98304);
    // are all eight buffers page-locked and mapped into the device's address space?
    const void* host[8] = { io->origin, io->len_in, io->len_out, io->exec_a, io->exec_b, io->judges, io->outcome, io->flags };
    void* dev[8];
    bool mapped = true;
    for (int k = 0; k < 8 && mapped; ++k) {
        cudaPointerAttributes a;
        if (cudaPointerGetAttributes(&a, host[k]) != cudaSuccess) { cudaGetLastError(); mapped = false; }
        else if (a.type != cudaMemoryTypeHost || !a.devicePointer) mapped = false;
        else dev[k] = a.devicePointer;
    }
    if (mapped && (reinterpret_cast<uintptr_t>(dev[5]) & 15) != 0) mapped = false;
    HostBatch hb{};
    if (mapped) {
        hb.origin = static_cast<const uint32_t*>(dev[0]); hb.len_in = static_cast<const uint16_t*>(dev[1]);
        hb.len_out = static_cast<const uint16_t*>(dev[2]);
        hb.exec_a = static_cast<int32_t*>(dev[3]); hb.exec_b = static_cast<int32_t*>(dev[4]); hb.judges = static_cast<int32_t*>(dev[5]);
        hb.outcome = static_cast<uint8_t*>(dev[6]); hb.rflags = static_cast<uint8_t*>(dev[7]);
    }
    if (!(n->d.flags & 16u) && want_direct && mapped) {
        // Page-locked, mapped host buffers are read and written by the kernels themselves: no copies,
        // and the result stores travel while the step runs.  (With exact queueing the results are
        // read again by later kernels, which is better done from device memory.)
        Net& d = n->d;
        const Net saved = d;
        d.origin = hb.origin; d.len_in = hb.len_in; d.len_out = hb.len_out;
        d.exec_a = hb.exec_a; d.exec_b = hb.exec_b; d.judges = hb.judges; d.outcome = hb.outcome; d.rflags = hb.rflags;
        d.score_a = nullptr; d.score_sum = nullptr;
        const wwws_status st = step_impl(n, first, count, now_ms, do_gossip, finalize, nullptr, nullptr);
        d.origin = saved.origin; d.len_in = saved.len_in; d.len_out = saved.len_out;
        d.exec_a = saved.exec_a; d.exec_b = saved.exec_b; d.judges = saved.judges; d.outcome = saved.outcome; d.rflags = saved.rflags;
        d.score_a = saved.score_a; d.score_sum = saved.score_sum;
        if (st) return st;
        if (totals_out) {
            std::vector<wwws_stats_t> all(d.Rp + 1);
            if (wwws_status st2 = wwws_stats(n, all.data())) return st2;
            *totals_out = all[d.Rp];
            return WWWS_OK;
        }
        return check_device_error(n);
    }
    // Staged path: the batch's request slices go to the bound device arrays on a second stream while
    // time advance and gossip run; the request kernel waits for them; the results travel back on the
    // second stream while the block is folded and the counters are read.  Mapped buffers are moved by
    // two small kernels (whole 128-byte lines across the bus, in request order), others by strided copies.
    if (!n->copy_stream) {
        CUDA_TRY(n, cudaStreamCreateWithFlags(&n->copy_stream, cudaStreamNonBlocking));
        CUDA_TRY(n, cudaEventCreateWithFlags(&n->ev_fork, cudaEventDisableTiming));
        CUDA_TRY(n, cudaEventCreateWithFlags(&n->ev_in, cudaEventDisableTiming));
        CUDA_TRY(n, cudaEventCreateWithFlags(&n->ev_step, cudaEventDisableTiming));
    }
    const Net& d = n->d;
    cudaStream_t cs = n->copy_stream;
    LaunchCtx cctx = n->ctx(0);
    cctx.stream = cs;
    const size_t Q = d.Q, Rp = d.Rp, c = count;
    // the batch is one strided slice per array: Rp rows of `count` elements, pitch n_requests
#define COPY2D(dst, src, T, W, kind) CUDA_TRY(n, cudaMemcpy2DAsync((void*)((dst) + first * (W)), Q * sizeof(T) * (W), (src) + first * (W), Q * sizeof(T) * (W), c * sizeof(T) * (W), Rp, kind, cs))
    CUDA_TRY(n, cudaEventRecord(n->ev_fork, n->stream));               // whatever still reads the device arrays comes first
    CUDA_TRY(n, cudaStreamWaitEvent(cs, n->ev_fork, 0));
    if (mapped) launch_host_batch_in(d, hb, first, uint32_t(count), cctx);
    else {
        COPY2D(d.origin, io->origin, uint32_t, 1, cudaMemcpyHostToDevice);
        COPY2D(d.len_in, io->len_in, uint16_t, 1, cudaMemcpyHostToDevice);
        COPY2D(d.len_out, io->len_out, uint16_t, 1, cudaMemcpyHostToDevice);
    }
    CUDA_TRY(n, cudaEventRecord(n->ev_in, cs));
    if (wwws_status st = step_impl(n, first, count, now_ms, do_gossip, finalize, n->ev_in, n->ev_step)) { cudaStreamSynchronize(cs); return st; }
    CUDA_TRY(n, cudaStreamWaitEvent(cs, n->ev_step, 0));
    if (mapped) launch_host_batch_out(d, hb, first, uint32_t(count), cctx);
    else {
        COPY2D(io->exec_a, d.exec_a, int32_t, 1, cudaMemcpyDeviceToHost);
        COPY2D(io->exec_b, d.exec_b, int32_t, 1, cudaMemcpyDeviceToHost);
        COPY2D(io->judges, d.judges, int32_t, 4, cudaMemcpyDeviceToHost);
        COPY2D(io->outcome, d.outcome, uint8_t, 1, cudaMemcpyDeviceToHost);
        COPY2D(io->flags, d.rflags, uint8_t, 1, cudaMemcpyDeviceToHost);
    }
#undef COPY2D
    wwws_status st = WWWS_OK;
    if (totals_out) {
        std::vector<wwws_stats_t> all(Rp + 1);
        st = wwws_stats(n, all.data());
        if (!st) *totals_out = all[Rp];
    } else st = check_device_error(n);
    CUDA_TRY(n, cudaStreamSynchronize(cs));
    if (cudaError_t e = cudaGetLastError(); e != cudaSuccess && !st) return fail(n, WWWS_ERR_CUDA, std::string("step_host copies: ") + cudaGetErrorString(e));
    return st;
}

wwws_status wwws_stats(wwws_network* n, wwws_stats_t* host_out)
{
    if (!n) return fail(nullptr, WWWS_ERR_ARG, "network is NULL");
    if (!host_out) return fail(n, WWWS_ERR_ARG, "host_out is NULL");
    ON_DEVICE(n);
    settle_pending(n);
    launch_credit_total(n->d, n->ctx());
    if (wwws_status st = launch_status(n, "stats")) return st;
    CUDA_TRY(n, cudaMemcpyAsync(host_out, n->d.stats, uint64_t(n->d.Rp) * sizeof(wwws_stats_t), cudaMemcpyDeviceToHost, n->stream));
    if (wwws_status st = check_device_error(n)) return st;   // synchronises
    uint64_t* tot = reinterpret_cast<uint64_t*>(&host_out[n->d.Rp]);
    memset(tot, 0, sizeof(wwws_stats_t));
    for (uint32_t r = 0; r < n->d.Rp; ++r) {
        const uint64_t* row = reinterpret_cast<const uint64_t*>(&host_out[r]);
        for (uint32_t k = 0; k < sCount; ++k) tot[k] += row[k];
    }
    return WWWS_OK;
}

wwws_status wwws_export_table(wwws_network* n, wwws_table t, void* host_dst, uint64_t bytes)
{
    if (!n) return fail(nullptr, WWWS_ERR_ARG, "network is NULL");
    if (!host_dst || int(t) < 0 || t >= WWWS_T_COUNT) return fail(n, WWWS_ERR_ARG, "bad table or NULL destination");
    const uint64_t need = uint64_t(n->d.N) * n->d.Rp * n->tables[t].elem;
    if (bytes != need) return fail(n, WWWS_ERR_ARG, "bytes does not match the table size");
    ON_DEVICE(n);
    settle_pending(n);
    CUDA_TRY(n, cudaMemcpyAsync(host_dst, n->tables[t].ptr, need, cudaMemcpyDeviceToHost, n->stream));
    return check_device_error(n);
}

wwws_status wwws_import_table(wwws_network* n, wwws_table t, const void* host_src, uint64_t bytes)
{
    if (!n) return fail(nullptr, WWWS_ERR_ARG, "network is NULL");
    if (!host_src || int(t) < 0 || t >= WWWS_T_COUNT) return fail(n, WWWS_ERR_ARG, "bad table or NULL source");
    if (n->phase != 0) return fail(n, WWWS_ERR_STATE, "import inside a batch");
    const uint64_t need = uint64_t(n->d.N) * n->d.Rp * n->tables[t].elem;
    if (bytes != need) return fail(n, WWWS_ERR_ARG, "bytes does not match the table size");
    ON_DEVICE(n);
    settle_pending(n);
    CUDA_TRY(n, cudaMemcpyAsync(n->tables[t].ptr, host_src, need, cudaMemcpyHostToDevice, n->stream));
    if (t == WWWS_T_CREDIT || t == WWWS_T_WINS || t == WWWS_T_DUELS || t == WWWS_T_ONLINE || t == WWWS_T_CAP_EFF || t == WWWS_T_BACKLOG)
        launch_rederive(n->d, n->ctx());           // stakes, ledger weights and the peers' gates follow the tables
    CUDA_TRY(n, cudaStreamSynchronize(n->stream));
    return launch_status(n, "import_table");
}

wwws_status wwws_export_view_rows(wwws_network* n, uint32_t replica, uint32_t row_first, uint32_t n_rows, uint64_t* host_dst)
{
    if (!n) return fail(nullptr, WWWS_ERR_ARG, "network is NULL");
    if (!host_dst) return fail(n, WWWS_ERR_ARG, "host_dst is NULL");
    if (replica >= n->d.Rp || uint64_t(row_first) + n_rows > n->d.N) return fail(n, WWWS_ERR_ARG, "rows out of range");
    ON_DEVICE(n);
    if (n_rows == 0) return WWWS_OK;
    const uint64_t* src = n->d.view + (uint64_t(replica) * n->d.N + row_first) * n->d.ld;
    CUDA_TRY(n, cudaMemcpy2DAsync(host_dst, n->d.N * 8ull, src, n->d.ld * 8ull, n->d.N * 8ull, n_rows, cudaMemcpyDeviceToHost, n->stream));
    return check_device_error(n);
}

wwws_status wwws_import_view_rows(wwws_network* n, uint32_t replica, uint32_t row_first, uint32_t n_rows, const uint64_t* host_src)
{
    if (!n) return fail(nullptr, WWWS_ERR_ARG, "network is NULL");
    if (!host_src) return fail(n, WWWS_ERR_ARG, "host_src is NULL");
    if (n->phase != 0) return fail(n, WWWS_ERR_STATE, "import inside a batch");
    if (replica >= n->d.Rp || uint64_t(row_first) + n_rows > n->d.N) return fail(n, WWWS_ERR_ARG, "rows out of range");
    ON_DEVICE(n);
    if (n_rows == 0) return WWWS_OK;
    uint64_t* dst = n->d.view + (uint64_t(replica) * n->d.N + row_first) * n->d.ld;
    CUDA_TRY(n, cudaMemcpy2DAsync(dst, n->d.ld * 8ull, host_src, n->d.N * 8ull, n->d.N * 8ull, n_rows, cudaMemcpyHostToDevice, n->stream));
    CUDA_TRY(n, cudaStreamSynchronize(n->stream));
    return WWWS_OK;
}

wwws_status wwws_export_clock(wwws_network* n, uint32_t* now_ms, uint32_t* round)
{
    if (!n) return fail(nullptr, WWWS_ERR_ARG, "network is NULL");
    if (!now_ms || !round) return fail(n, WWWS_ERR_ARG, "output pointer is NULL");
    *now_ms = n->t_last_ms; *round = n->round;
    return WWWS_OK;
}

wwws_status wwws_import_clock(wwws_network* n, uint32_t now_ms, uint32_t round)
{
    if (!n) return fail(nullptr, WWWS_ERR_ARG, "network is NULL");
    if (n->phase != 0) return fail(n, WWWS_ERR_STATE, "import inside a batch");
    n->t_last_ms = now_ms; n->round = round;
    return WWWS_OK;
}

wwws_status wwws_import_stats(wwws_network* n, const wwws_stats_t* host_src)
{
    if (!n) return fail(nullptr, WWWS_ERR_ARG, "network is NULL");
    if (!host_src) return fail(n, WWWS_ERR_ARG, "host_src is NULL");
    if (n->phase != 0) return fail(n, WWWS_ERR_STATE, "import inside a batch");
    ON_DEVICE(n);
    settle_pending(n);
    CUDA_TRY(n, cudaMemcpyAsync(n->d.stats, host_src, uint64_t(n->d.Rp) * sizeof(wwws_stats_t), cudaMemcpyHostToDevice, n->stream));
    CUDA_TRY(n, cudaStreamSynchronize(n->stream));
    return WWWS_OK;
}

wwws_status wwws_set_option(wwws_network* n, wwws_option option, int64_t value)
{
    if (!n) return fail(nullptr, WWWS_ERR_ARG, "network is NULL");
    switch (option) {
    case WWWS_OPT_REQUEST_KERNEL:
        if (value < 0 || value > 2) return fail(n, WWWS_ERR_ARG, "WWWS_OPT_REQUEST_KERNEL takes 0 (by size), 1 (warp) or 2 (thread)");
        n->request_kernel = int(value);
        return WWWS_OK;
    case WWWS_OPT_STEP_KERNEL:
        if (value < 0 || value > 4) return fail(n, WWWS_ERR_ARG, "WWWS_OPT_STEP_KERNEL takes 0 (by size), 1 (8 lanes), 2 (4 lanes), 3 (thread) or 4 (streaming)");
        n->step_kernel = int(value);
        return WWWS_OK;
    case WWWS_OPT_HOST_IO:
        if (value < 0 || value > 2) return fail(n, WWWS_ERR_ARG, "WWWS_OPT_HOST_IO takes 0 (by batch size), 1 (mapped buffers) or 2 (staged copies)");
        n->host_io = int(value);
        return WWWS_OK;
    case WWWS_OPT_LAUNCH_OVERLAP:
        if (value < 0 || value > 15) return fail(n, WWWS_ERR_ARG, "WWWS_OPT_LAUNCH_OVERLAP takes a mask 0..15");
        n->overlap = int(value);
        return WWWS_OK;
    case WWWS_OPT_STREAM_RUN:
        if (value < 0 || value > 65536 || value % 32) return fail(n, WWWS_ERR_ARG, "WWWS_OPT_STREAM_RUN takes 0 (by size) or a multiple of 32 up to 65536");
        n->stream_run = uint32_t(value);
        return WWWS_OK;
    default:
        return fail(n, WWWS_ERR_ARG, "unknown option");
    }
}

uint64_t wwws_kernel_launches(const wwws_network* n) { return n ? n->launches : 0; }

wwws_status wwws_profile(wwws_network* n, int enable)
{
    if (!n) return fail(nullptr, WWWS_ERR_ARG, "network is NULL");
    ON_DEVICE(n);
    n->prof.reset();
    n->prof.enabled = enable != 0;
    return WWWS_OK;
}

wwws_status wwws_profile_read(wwws_network* n, double* ms_out, uint64_t* count_out)
{
    if (!n) return fail(nullptr, WWWS_ERR_ARG, "network is NULL");
    if (!ms_out || !count_out) return fail(n, WWWS_ERR_ARG, "output array is NULL");
    ON_DEVICE(n);
    n->prof.collect();
    for (int k = 0; k < kKernelCount; ++k) { ms_out[k] = n->prof.ms[k]; count_out[k] = n->prof.count[k]; }
    return WWWS_OK;
}

uint32_t wwws_profile_kernels(void) { return kKernelCount; }

const char* wwws_profile_kernel_name(uint32_t k)
{
    static const char* names[kKernelCount] = { "k_peer_init", "k_view_init", "k_advance", "k_fold",
        "k_rederive", "k_credit_total", "k_gossip_peer", "k_gossip_merge", "k_gossip_fixup", "k_gossip_lists", "k_fifo", "k_dispatch", "k_duel",
        "k_settle", "k_step_fused", "k_host_batch" };
    return k < kKernelCount ? names[k] : "";
}

const char* wwws_last_error(const wwws_network* n) { return n ? n->err.c_str() : g_err.c_str(); }

}  // extern "C"

// ---- gossip round whose scratch lives in the library image --------------------------------------
//
// Some programs that embed this library may not allocate device memory at the point where
// they call it: all of the GPU's memory already belongs to another allocator (an inference
// server's pool), an allocation is not permitted in that phase of the program, or the
// device-wide synchronisation that cudaMalloc implies is not acceptable inside their loop.
// For them the scratch of a gossip round (this round's self entries and partner lists) sits
// in a fixed array that every GPU holds from the moment it loads the library until exit.

namespace {

constexpr uint64_t kStaticPeers = 65536;                       // n_replicas * n_peers limit
constexpr uint64_t kStaticSelfBytes = kStaticPeers * sizeof(uint64_t);
constexpr uint64_t kStaticPartnerBytes = kStaticPeers * 4 * sizeof(int32_t);
static __device__ __align__(256) unsigned char g_gossip_scratch[kStaticSelfBytes + kStaticPartnerBytes];  // 1.5 MiB

constexpr int kMaxDevices = 64;
std::atomic<void*> g_gossip_scratch_addr[kMaxDevices];         // per device, filled on first use; handles on
                                                               // several threads may resolve it at once (same value)

}  // namespace

extern "C" wwws_status wwws_gossip_round_static(wwws_network* n)
{
    if (!n) return fail(nullptr, WWWS_ERR_ARG, "network is NULL");
    if (n->phase != 0) return fail(n, WWWS_ERR_STATE, "gossip_round inside a batch");
    if (n->prof.enabled) return fail(n, WWWS_ERR_STATE, "per-kernel timing creates CUDA events: switch wwws_profile off for the round that allocates nothing");
    const uint64_t peers = uint64_t(n->d.N) * n->d.Rp;
    if (peers > kStaticPeers) {
        char buf[160];
        snprintf(buf, sizeof buf, "n_replicas * n_peers = %llu exceeds the built-in scratch of %llu peers; use wwws_gossip_round",
                 (unsigned long long)peers, (unsigned long long)kStaticPeers);
        return fail(n, WWWS_ERR_ARG, buf);
    }
    const int dev = n->device;
    if (dev < 0 || dev >= kMaxDevices) return fail(n, WWWS_ERR_ARG, "device ordinal beyond 63");
    ON_DEVICE(n);
    settle_pending(n);
    void* p = g_gossip_scratch_addr[dev].load(std::memory_order_acquire);
    if (!p) {
        // In host code the array's name is only a handle for the runtime; the address the
        // kernels need comes from the runtime, for the device that is current now (the
        // network's own, selected just above).
        CUDA_TRY(n, cudaGetSymbolAddress(&p, g_gossip_scratch));
        g_gossip_scratch_addr[dev].store(p, std::memory_order_release);
    }
    unsigned char* base = static_cast<unsigned char*>(p);
    Net d = n->d;                                              // same network, scratch pointers redirected
    d.self_entry = reinterpret_cast<uint64_t*>(base);
    d.partner = reinterpret_cast<int32_t*>(base + kStaticSelfBytes);
    launch_gossip(d, n->round, n->ctx());
    std::swap(n->d.view, n->d.view_new);
    n->round += 1;
    return launch_status(n, "gossip_round_static");
}
