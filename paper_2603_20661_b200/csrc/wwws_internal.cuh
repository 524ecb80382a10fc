// Launchers of the wwws kernels (internal to the library) and the optional per-kernel timer.
#pragma once
#include <vector>

#include "wwws_device.cuh"

namespace wwws {

// Kernel classes, for launch counts and optional event timing.
enum KernelId : int { kPeerInit, kViewInit, kAdvance, kFold, kRederive, kCreditTotal, kGossipPeer,
                      kGossipMerge, kGossipFixup, kGossipLists, kFifo, kDispatch, kDuel, kSettle, kStepFused, kHostBatch, kKernelCount };

// When enabled, every launch is bracketed by two events on the launching stream; read()
// synchronises and returns the summed device time per kernel class.
struct Profiler {
    bool enabled = false;
    struct Pair { cudaEvent_t a, b; int id; };
    std::vector<Pair> used;
    std::vector<Pair> pool;
    double ms[kKernelCount] = {};
    uint64_t count[kKernelCount] = {};
    void begin(int id, cudaStream_t s);
    void end(cudaStream_t s);
    void collect();              // synchronises the events recorded so far
    void reset();
    ~Profiler();
};

struct LaunchCtx {
    cudaStream_t stream;
    uint64_t* launches;          // total kernels launched
    Profiler* prof;
    bool overlap;                // launch with programmatic stream serialization (see launch_kernel)
};

struct Timed {                   // RAII bracket around one launch
    const LaunchCtx& c;
    Timed(const LaunchCtx& ctx, int id) : c(ctx) { *c.launches += 1; if (c.prof && c.prof->enabled) c.prof->begin(id, c.stream); }
    ~Timed() { if (c.prof && c.prof->enabled) c.prof->end(c.stream); }
};

// Every kernel of the library is launched through here.  With `overlap` the launch carries the
// programmatic-stream-serialization attribute: the grid may be scheduled while its predecessor in
// the stream is still running, and its threads hold at grid_dependency_enter() (the first
// statement of every kernel) until the predecessor has completed and its writes are visible.
// What overlaps is the launch latency and the block scheduling, not the work.
template <class... P, class... A>
inline void launch_kernel(const LaunchCtx& c, void (*kernel)(P...), dim3 grid, dim3 block, A&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = 0; cfg.stream = c.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = c.overlap ? 1 : 0;
    cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...);
}

// Device-side addresses of a caller's mapped host buffers ([Rp][Q] like the bound arrays).
struct HostBatch {
    const uint32_t* origin; const uint16_t* len_in; const uint16_t* len_out;
    int32_t* exec_a; int32_t* exec_b; int32_t* judges; uint8_t* outcome; uint8_t* rflags;
};
void launch_host_batch_in(const Net& n, const HostBatch& h, uint64_t first, uint32_t count, const LaunchCtx& c);
void launch_host_batch_out(const Net& n, const HostBatch& h, uint64_t first, uint32_t count, const LaunchCtx& c);

void launch_peer_init(const Net& n, const int64_t* credit0, const uint8_t* online0, uint32_t init_stale_max, const LaunchCtx& c);
void launch_advance(const Net& n, uint32_t dt_ms, uint32_t now_ms, const LaunchCtx& c);
void launch_fold(const Net& n, int finalize, const LaunchCtx& c);
void launch_fold_advance(const Net& n, int finalize, uint32_t dt_ms, uint32_t now_ms, const LaunchCtx& c);
void launch_rederive(const Net& n, const LaunchCtx& c);
void launch_credit_total(const Net& n, const LaunchCtx& c);
void launch_gossip(const Net& n, uint32_t round, const LaunchCtx& c);
void launch_scan_in_degrees(const Net& n, const LaunchCtx& c, int kernel_id);
void launch_fifo(const Net& n, uint64_t first, uint32_t count, const LaunchCtx& c);
void launch_dispatch(const Net& n, uint64_t first, uint32_t count, const LaunchCtx& c);
void launch_duel(const Net& n, uint64_t first, uint32_t count, const LaunchCtx& c);
void launch_settle(const Net& n, uint64_t first, uint32_t count, const LaunchCtx& c);
// step_kernel: 0 chosen by launch size, 1 eight lanes per request, 2 four lanes, 3 one thread per request,
// 4 streaming phases; stream_run: requests per warp of the streaming kernel, 0 = by launch size
void launch_step_fused(const Net& n, uint64_t first, uint32_t count, const LaunchCtx& c, int step_kernel = 0, uint32_t stream_run = 0);
void launch_step_stream(const Net& n, uint64_t first, uint32_t count, uint32_t per_warp, const LaunchCtx& c);
int step_lanes_for(uint64_t total_requests);
void launch_step_lanes(const Net& n, uint64_t first, uint32_t count, int lanes, const LaunchCtx& c);
void launch_dispatch_threads(const Net& n, uint64_t first, uint32_t count, const LaunchCtx& c);
void launch_duel_threads(const Net& n, uint64_t first, uint32_t count, const LaunchCtx& c);

}  // namespace wwws
