// Device executors of a broadcast plan (sm_100a): every message of the plan is a copy of `len`
// bytes at `offset` from the source rank's buffer to the same offset of the destination rank's
// buffer (Section III-A: scatter and native ring; Section IV: tuned ring).
//
// Two facts about the schedule shape the kernels:
//   * source and destination of a message use the SAME byte offset (the listing displaces both
//     sides by chunk index x scatter_size), so with 16-byte aligned rank buffers both sides are
//     co-aligned: a range splits into <= 15 head bytes, 16-byte words, <= 15 tail bytes;
//   * a byte of the message at some rank depends only on the same byte at the rank it is copied
//     from, so messages that cover different byte ranges never depend on one another.
//
// WALK executor (one launch): the message is cut into segments on a fixed grid of byte offsets,
// split further at chunk boundaries.  A warp takes such a slice and performs every message of the
// plan that covers the slice's chunk, restricted to the slice, in an order that respects the
// plan's dependencies: load from the source rank's buffer, store to the destination rank's
// buffer.  Each thread always handles the same bytes of the slice, so whatever a hop reads was
// stored earlier by the same thread: program order per thread is the only ordering the schedule
// needs.  Loads bypass L1 (.cg) so that every hop really re-reads the source rank's buffer from
// the L2/HBM level.
//
// STEPS / GRAPH executors: one launch per plan step, the messages of the step cut into tiles.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "plan_internal.h"

namespace {

constexpr int kThreads = 256;             // threads per block, both executors
constexpr int kStepWordsPerThread = 4;    // STEPS executor: 256 x 4 x 16 B = 16 KiB tiles
constexpr uint64_t kStepTile = (uint64_t)kThreads * kStepWordsPerThread * 16;

thread_local int t_last_cuda_error = 0;

#define CUDA_TRY(expr)                                        \
    do {                                                      \
        cudaError_t e_ = (expr);                              \
        if (e_ != cudaSuccess) {                              \
            t_last_cuda_error = (int)e_;                      \
            return e_ == cudaErrorMemoryAllocation ? BCAST_ERR_NOMEM : BCAST_ERR_CUDA; \
        }                                                     \
    } while (0)

// The P rank-buffer pointers travel as a kernel argument (copied at launch), so a launch never
// depends on a device-side table that a later call could overwrite.
template <int MAXP>
struct RankPtrs {
    uint8_t *p[MAXP];
};

struct DevXfer {      // one message, device copy
    uint64_t off, len;
    uint16_t src, dst;
    uint32_t pad;
};

struct WalkSlice {    // one warp's share of the message: segment `seg` of the fixed grid of
    uint32_t seg;     // 32 * U * 16-byte segments, cut down to the bytes of relative chunk `chunk`
    uint32_t chunk;   // (selects the hop list)
};

// ---- memory operations.  volatile + "memory": the compiler must keep loads and stores of
// successive hops in program order, because a hop may read what the previous hop wrote.
__device__ __forceinline__ uint4 ld16(const uint8_t *p)
{
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st16(uint8_t *p, const uint4 &v)
{
    asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint32_t ld1(const uint8_t *p)
{
    uint32_t v;
    asm volatile("ld.global.cg.u8 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st1(uint8_t *p, uint32_t v)
{
    asm volatile("st.global.u8 [%0], %1;" :: "l"(p), "r"(v) : "memory");
}

// Split [lo, hi) into head bytes [lo, head_end), 16-byte words [a0, a1) and tail bytes
// [tail_begin, hi).  Offsets are relative to buffers that are themselves 16-byte aligned.
struct Split {
    uint64_t a0, head_end, tail_begin;
    uint32_t nwords, nhead, ntail;
};
__device__ __forceinline__ Split split16(uint64_t lo, uint64_t hi)
{
    Split s;
    s.a0 = (lo + 15) & ~(uint64_t)15;
    const uint64_t a1 = hi & ~(uint64_t)15;
    s.head_end = s.a0 < hi ? s.a0 : hi;
    s.tail_begin = a1 > s.head_end ? a1 : s.head_end;
    s.nwords = a1 > s.a0 ? (uint32_t)((a1 - s.a0) >> 4) : 0u;
    s.nhead = (uint32_t)(s.head_end - lo);
    s.ntail = (uint32_t)(hi - s.tail_begin);
    return s;
}

// ------------------------------------------------------------------------------------- WALK
// The message is cut on a fixed grid of segments of 32 x U words (U x 512 bytes), and every
// segment further at chunk boundaries: a slice is the part of one segment that lies in one chunk.
// A warp owns a slice and walks it through the chunk's hop list on its own: warps never wait for
// one another.  Slices are dealt round-robin with the block index running fastest (slice w goes to
// block w mod G, then to that block's warp (w / G) mod 8): all SMs get the same share, and the
// slices in flight at any time are neighbours in the message.  Lanes map to the fixed 16-byte words of the segment,
// whatever the chunk's first byte is, so a warp's 512-byte accesses stay aligned to cache lines;
// the <= 15 bytes before the first whole word and after the last one go one byte per lane.
// The (src, dst) pair of hop h+1 is fetched while the loads of hop h are in flight.
constexpr int kWarpsPerBlock = kThreads / 32;

// One slice, all its hops, by one warp with U words per lane (the register path).
template <int U, int MAXP>
__device__ __forceinline__ void walk_slice(const RankPtrs<MAXP> &bufs, const WalkSlice sl, uint64_t scatter_size,
                                           uint64_t nbytes, const uint32_t *__restrict__ hops,
                                           const int *__restrict__ hop_begin, uint32_t lane)
{
    constexpr uint64_t kSeg = 32ull * U * 16;
    const uint64_t seg_lo = (uint64_t)sl.seg * kSeg, seg_hi = seg_lo + kSeg;
    const uint64_t lo = max(min((uint64_t)sl.chunk * scatter_size, nbytes), seg_lo);
    const uint64_t hi = min(min(((uint64_t)sl.chunk + 1) * scatter_size, nbytes), seg_hi);
    if (lo >= hi) return;
    const uint32_t *hp = hops + hop_begin[sl.chunk];
    const int nh = hop_begin[sl.chunk + 1] - hop_begin[sl.chunk];
    if (nh <= 0) return;
    const uint64_t base = seg_lo + (uint64_t)lane * 16;

    uint32_t e = __ldg(hp);
    const uint8_t *s = bufs.p[e & 0xffffu];
    uint8_t *d = bufs.p[e >> 16];
    if (lo == seg_lo && hi == seg_hi) {
        // whole segment: every lane moves U words per hop, no predicates
        for (int h = 0; h < nh; h++) {
            uint4 v[U];
#pragma unroll
            for (int u = 0; u < U; u++) v[u] = ld16(s + base + (uint64_t)u * 512);
            e = __ldg(hp + min(h + 1, nh - 1));              // next hop, while the loads are in flight
            const uint8_t *s_next = bufs.p[e & 0xffffu];
            uint8_t *d_next = bufs.p[e >> 16];
#pragma unroll
            for (int u = 0; u < U; u++) st16(d + base + (uint64_t)u * 512, v[u]);
            s = s_next;
            d = d_next;
        }
    } else {
        // ragged slice (a chunk starts or ends inside the segment): predicated words, plus the
        // bytes of the partial words at either end
        const uint64_t body_lo = (lo + 15) & ~(uint64_t)15, body_hi = hi & ~(uint64_t)15;
        const uint64_t head_end = body_lo < hi ? body_lo : hi;
        const uint64_t tail_begin = body_hi > head_end ? body_hi : head_end;
        const uint32_t nhead = (uint32_t)(head_end - lo), nedge = nhead + (uint32_t)(hi - tail_begin);
        bool ok[U];
#pragma unroll
        for (int u = 0; u < U; u++) {
            const uint64_t o = base + (uint64_t)u * 512;
            ok[u] = o >= body_lo && o + 16 <= body_hi;
        }
        const bool has_edge = lane < nedge;
        const uint64_t eoff = lane < nhead ? lo + lane : tail_begin + (lane - nhead);
        for (int h = 0; h < nh; h++) {
            uint4 v[U];
            uint32_t b = 0;
#pragma unroll
            for (int u = 0; u < U; u++)
                if (ok[u]) v[u] = ld16(s + base + (uint64_t)u * 512);
            if (has_edge) b = ld1(s + eoff);
            e = __ldg(hp + min(h + 1, nh - 1));
            const uint8_t *s_next = bufs.p[e & 0xffffu];
            uint8_t *d_next = bufs.p[e >> 16];
#pragma unroll
            for (int u = 0; u < U; u++)
                if (ok[u]) st16(d + base + (uint64_t)u * 512, v[u]);
            if (has_edge) st1(d + eoff, b);
            s = s_next;
            d = d_next;
        }
    }
}

template <int U, int MAXP>
__global__ void __launch_bounds__(kThreads)
bcast_walk_kernel(const __grid_constant__ RankPtrs<MAXP> bufs, const WalkSlice *__restrict__ slices,
                  long long n_slices, uint64_t scatter_size, uint64_t nbytes,
                  const uint32_t *__restrict__ hops, const int *__restrict__ hop_begin)
{
    const uint32_t lane = threadIdx.x & 31u;
    const long long total_warps = (long long)gridDim.x * kWarpsPerBlock;
    // slice w goes to block w mod gridDim.x: every SM gets the same number of slices (+-1)
    for (long long w = (long long)(threadIdx.x >> 5) * gridDim.x + blockIdx.x; w < n_slices; w += total_warps)
        walk_slice<U, MAXP>(bufs, slices[w], scatter_size, nbytes, hops, hop_begin, lane);
}

// ------------------------------------------------------------------------------------- WALK, bulk copies
// The same walk for large messages, with the data moved by the bulk-copy engine (TMA, untiled
// cp.async.bulk) instead of through registers: whole 16 KiB segments of the fixed grid go
// global -> shared -> global, one worker thread per segment.  A hop is: expect 16 KiB on the
// worker's mbarrier, bulk load from the source rank's buffer, wait, bulk store to the destination
// rank's buffer, wait until the store has completed (not merely been read out of shared memory:
// the next hop may load those very bytes again).  Two memory round trips per hop instead of one
// are paid for with more bytes in flight (kBulkWorkers x 16 KiB per block); the longer contiguous
// runs are what DRAM likes better.  Segments that a chunk boundary cuts are left to a second warp
// of every block, which walks them as 4 KiB register slices.
// Every address and size handed to a bulk copy is a multiple of 16 bytes (rank buffers are
// 16-byte aligned, segment offsets and sizes are multiples of 16 KiB).  No cluster multicast.
constexpr uint32_t kBulkSeg = 16384;
constexpr int kBulkWorkers = 4;               // worker threads (lanes 0..3 of warp 0) and segments in flight per block
constexpr int kBulkThreads = 64;              // warp 0: bulk workers; warp 1: register slices
constexpr int kBulkSpinLimit = 1 << 24;       // mbarrier polls before a worker gives up

template <int MAXP>
__global__ void __launch_bounds__(kBulkThreads)
bcast_walk_bulk_kernel(const __grid_constant__ RankPtrs<MAXP> bufs, const WalkSlice *__restrict__ bulk_slices,
                       long long n_bulk, const WalkSlice *__restrict__ reg_slices, long long n_reg,
                       uint64_t scatter_size, uint64_t nbytes, const uint32_t *__restrict__ hops,
                       const int *__restrict__ hop_begin, int *status)
{
    extern __shared__ __align__(128) uint8_t bulk_smem[];
    __shared__ __align__(8) uint64_t bulk_bar[kBulkWorkers];
    const uint32_t lane = threadIdx.x & 31u;

    if (threadIdx.x >= 32) {
        // warp 1: the segments cut by chunk boundaries, as register slices of 8 words per lane
        for (long long w = blockIdx.x; w < n_reg; w += gridDim.x)
            walk_slice<8, MAXP>(bufs, reg_slices[w], scatter_size, nbytes, hops, hop_begin, lane);
        return;
    }
    if (lane >= kBulkWorkers) return;

    const uint32_t sbuf = (uint32_t)__cvta_generic_to_shared(bulk_smem + (size_t)lane * kBulkSeg);
    const uint32_t sbar = (uint32_t)__cvta_generic_to_shared(&bulk_bar[lane]);
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(sbar) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    uint32_t phase = 0;
    const long long total = (long long)gridDim.x * kBulkWorkers;
    for (long long w = (long long)lane * gridDim.x + blockIdx.x; w < n_bulk; w += total) {
        const WalkSlice sl = bulk_slices[w];
        const uint64_t off = (uint64_t)sl.seg * kBulkSeg;
        const uint32_t *hp = hops + hop_begin[sl.chunk];
        const int nh = hop_begin[sl.chunk + 1] - hop_begin[sl.chunk];
        for (int h = 0; h < nh; h++) {
            const uint32_t e = __ldg(hp + h);
            const uint8_t *s = bufs.p[e & 0xffffu] + off;
            uint8_t *d = bufs.p[e >> 16] + off;
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(sbar), "r"(kBulkSeg) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         :: "r"(sbuf), "l"(s), "r"(kBulkSeg), "r"(sbar) : "memory");
            uint32_t arrived = 0;
            for (int spin = 0; spin < kBulkSpinLimit && !arrived; spin++)
                asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                             : "=r"(arrived) : "r"(sbar), "r"(phase) : "memory");
            if (!arrived) {
                // the load never reported completion: flag it for the host and stop this worker
                // (nothing else of this worker is in flight: its last store was waited for)
                atomicExch(status, 1);
                return;
            }
            phase ^= 1u;
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" :: "l"(d), "r"(sbuf), "r"(kBulkSeg) : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        }
    }
}

// ------------------------------------------------------------------------------------- STEPS
// blockIdx.y selects a message of the step, blockIdx.x a tile of the fixed offset grid inside it.
template <int MAXP>
__global__ void __launch_bounds__(kThreads)
bcast_step_kernel(const __grid_constant__ RankPtrs<MAXP> bufs, const DevXfer *__restrict__ xfers)
{
    const DevXfer x = xfers[blockIdx.y];
    const uint64_t end = x.off + x.len;
    const uint64_t tile = x.off / kStepTile + blockIdx.x;
    const uint64_t lo = max(x.off, tile * kStepTile);
    const uint64_t hi = min(end, (tile + 1) * kStepTile);
    if (lo >= hi) return;
    const uint8_t *s = bufs.p[x.src];
    uint8_t *d = bufs.p[x.dst];
    const Split sp = split16(lo, hi);
    const int tid = threadIdx.x;
    const uint64_t base = sp.a0 + (uint64_t)tid * 16;
    uint4 v[kStepWordsPerThread];
#pragma unroll
    for (int u = 0; u < kStepWordsPerThread; u++)
        if ((uint32_t)(tid + u * kThreads) < sp.nwords) v[u] = ld16(s + base + (uint64_t)u * kThreads * 16);
#pragma unroll
    for (int u = 0; u < kStepWordsPerThread; u++)
        if ((uint32_t)(tid + u * kThreads) < sp.nwords) st16(d + base + (uint64_t)u * kThreads * 16, v[u]);
    if ((uint32_t)tid < sp.nhead) st1(d + lo + tid, ld1(s + lo + tid));
    else if ((uint32_t)tid < sp.nhead + sp.ntail) {
        const uint64_t o = sp.tail_begin + (tid - sp.nhead);
        st1(d + o, ld1(s + o));
    }
}

}  // namespace

// ======================================================================================= host
struct StepLaunch {
    int64_t first;     // index of the step's first message in d_xfers
    unsigned count;    // messages in the step (gridDim.y)
    unsigned tiles;    // most tiles any message of the step spans (gridDim.x); 0: nothing to copy
};

struct bcast_device_state {
    int device = -1;
    int sm_count = 0;
    // STEPS / GRAPH
    DevXfer *d_xfers = nullptr;
    std::vector<StepLaunch> steps;
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t graph_exec = nullptr;
    std::vector<void *> graph_bufs;
    // WALK
    WalkSlice *d_slices = nullptr;
    uint32_t *d_hops = nullptr;        // dependency order
    uint32_t *d_hops_plan = nullptr;   // plan order
    int *d_hop_begin = nullptr;
    long long n_slices = 0;
    int walk_u = 0, walk_grid = 0;
    // WALK with bulk copies
    WalkSlice *d_bulk_slices = nullptr, *d_reg_slices = nullptr;
    long long n_bulk = 0, n_reg = 0;
    int bulk_grid = 0;
    int *d_status = nullptr;           // set by a kernel whose bounded wait ran out
    // argument check cache
    std::vector<void *> checked_bufs;
};

void bcast_device_state_free(bcast_device_state *dev)
{
    if (!dev) return;
    int cur = -1;
    const bool switched = cudaGetDevice(&cur) == cudaSuccess && cur != dev->device && dev->device >= 0 &&
                          cudaSetDevice(dev->device) == cudaSuccess;
    if (dev->graph_exec) cudaGraphExecDestroy(dev->graph_exec);
    if (dev->graph) cudaGraphDestroy(dev->graph);
    cudaFree(dev->d_xfers);
    cudaFree(dev->d_slices);
    cudaFree(dev->d_bulk_slices);
    cudaFree(dev->d_reg_slices);
    cudaFree(dev->d_status);
    cudaFree(dev->d_hops);
    cudaFree(dev->d_hops_plan);
    cudaFree(dev->d_hop_begin);
    if (switched) cudaSetDevice(cur);
    delete dev;
}

namespace {

int env_int(const char *name, int fallback)
{
    const char *v = std::getenv(name);
    return (v && *v) ? std::atoi(v) : fallback;
}

template <typename T>
int upload(T **d_ptr, const std::vector<T> &h)
{
    const size_t bytes = std::max<size_t>(h.size(), 1) * sizeof(T);
    CUDA_TRY(cudaMalloc((void **)d_ptr, bytes));
    if (!h.empty()) CUDA_TRY(cudaMemcpy(*d_ptr, h.data(), h.size() * sizeof(T), cudaMemcpyHostToDevice));
    return BCAST_OK;
}

template <int U, int MAXP>
int walk_occupancy(int *blocks_per_sm)
{
    CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, bcast_walk_kernel<U, MAXP>, kThreads, 0));
    return BCAST_OK;
}

// Tables of the STEPS executor: the messages themselves and one launch shape per step.
int build_step_tables(const bcast_plan_t &p, bcast_device_state &ds)
{
    std::vector<DevXfer> hx(p.xfers.size());
    for (size_t i = 0; i < p.xfers.size(); i++) {
        const bcast_xfer_t &x = p.xfers[i];
        hx[i] = DevXfer{x.offset, x.len, (uint16_t)x.src_rank, (uint16_t)x.dst_rank, 0u};
    }
    const int nsteps = (int)p.step_begin.size() - 1;
    ds.steps.resize(nsteps);
    for (int s = 0; s < nsteps; s++) {
        StepLaunch sl{p.step_begin[s], (unsigned)(p.step_begin[s + 1] - p.step_begin[s]), 0u};
        for (int64_t i = p.step_begin[s]; i < p.step_begin[s + 1]; i++) {
            const bcast_xfer_t &x = p.xfers[i];
            if (!x.len) continue;
            const uint64_t t = (x.offset + x.len - 1) / kStepTile - x.offset / kStepTile + 1;
            sl.tiles = std::max<unsigned>(sl.tiles, (unsigned)t);
        }
        ds.steps[s] = sl;
    }
    return upload(&ds.d_xfers, hx);
}

// Host form of the WALK executor's tables: per chunk the list of (src, dst) hops in plan order,
// and the tiles (fixed grid of `256 * u * 16`-byte offsets, split at chunk boundaries).
struct WalkTables {
    std::vector<WalkSlice> slices;
    std::vector<uint32_t> hops;        // per chunk, dependency order (see order_by_dependency)
    std::vector<uint32_t> hops_plan;   // per chunk, plan order
    std::vector<int> hop_begin;        // [P + 1], by relative chunk index; the same for both
};

// Re-order the hops of one chunk without breaking any dependency, so that a rank's copy is read
// soon after it was written and is still in L2 then.
//
// In plan order the scatter hops come first and the ring hops later, so in the tuned ring every
// copy that the scatter left at an inner node of the tree is read a second time ~P hops after it
// was written, from DRAM.  The hops of a chunk form a tree: hop h hangs below the hop that wrote
// its source rank (`dep` in the plan), or below the root's original data.  If no rank is written
// twice, any order that puts a hop after its parent performs the same copies with the same result:
// the data a hop reads is final once written.  The order chosen here is level order (breadth
// first): all hops that read the same copy are neighbours, and the branches of the tree (the
// ring segments that start at the root and at each inner node of the scatter tree) advance in
// turn, so a copy is read again at most one level -- a handful of hops -- after it was written.
// Chunks in which some rank is written more than once (native ring: redundant re-receives) keep
// plan order, where write-after-read order matters.
void order_by_dependency(const bcast_plan_t &p, const std::vector<int64_t> &plan_order, std::vector<int64_t> &out)
{
    const int n = (int)plan_order.size();
    out = plan_order;
    std::vector<int> writer(p.P, -1);
    for (int h = 0; h < n; h++) {
        const int dst = p.xfers[plan_order[h]].dst_rank;
        if (writer[dst] >= 0) return;                 // written twice: keep plan order
        writer[dst] = h;
    }
    std::vector<int> depth(n), index(n);
    for (int h = 0; h < n; h++) {
        const int parent = writer[p.xfers[plan_order[h]].src_rank];
        if (parent > h) return;                       // would read a copy before it exists: keep plan order
        depth[h] = parent < 0 ? 0 : depth[parent] + 1;
        index[h] = h;
    }
    std::stable_sort(index.begin(), index.end(), [&](int a, int b) { return depth[a] < depth[b]; });
    for (int i = 0; i < n; i++) out[i] = plan_order[index[i]];
}

// For every relative chunk: the plan's messages that move bytes of it, in plan order.
void messages_by_chunk(const bcast_plan_t &p, std::vector<std::vector<int64_t>> &per_chunk)
{
    auto chunk_begin = [&](int c) { return std::min<uint64_t>((uint64_t)c * p.S, p.nbytes); };
    per_chunk.assign(p.P, {});
    for (size_t i = 0; i < p.xfers.size(); i++) {
        const bcast_xfer_t &x = p.xfers[i];
        if (!x.len) continue;
        for (int c = x.chunk; c < x.chunk + x.nchunks; c++)
            if (chunk_begin(c + 1) > chunk_begin(c)) per_chunk[c].push_back((int64_t)i);
    }
}

int make_walk_tables(const bcast_plan_t &p, int u, WalkTables &t)
{
    const int P = p.P;
    auto chunk_begin = [&](int c) { return std::min<uint64_t>((uint64_t)c * p.S, p.nbytes); };
    auto encode = [&](int64_t i) { return (uint32_t)p.xfers[i].src_rank | ((uint32_t)p.xfers[i].dst_rank << 16); };
    std::vector<std::vector<int64_t>> per_chunk;
    messages_by_chunk(p, per_chunk);
    t.hop_begin.assign(P + 1, 0);
    t.hops.clear();
    t.hops_plan.clear();
    std::vector<int64_t> reordered;
    for (int c = 0; c < P; c++) {
        t.hop_begin[c] = (int)t.hops.size();
        order_by_dependency(p, per_chunk[c], reordered);
        for (int64_t i : reordered) t.hops.push_back(encode(i));
        for (int64_t i : per_chunk[c]) t.hops_plan.push_back(encode(i));
    }
    t.hop_begin[P] = (int)t.hops.size();

    const uint64_t seg = 32ull * u * 16;
    t.slices.clear();
    for (int c = 0; c < P; c++) {
        const uint64_t b = chunk_begin(c), e = chunk_begin(c + 1);
        if (e <= b || per_chunk[c].empty()) continue;
        for (uint64_t g = b / seg; g * seg < e; g++) t.slices.push_back(WalkSlice{(uint32_t)g, (uint32_t)c});
    }
    return BCAST_OK;
}

// Number of slices for U words per lane, without building the list.
long long count_walk_slices(const bcast_plan_t &p, int u)
{
    const uint64_t seg = 32ull * u * 16;
    long long n = 0;
    for (int c = 0; c < p.P; c++) {
        const uint64_t b = std::min<uint64_t>((uint64_t)c * p.S, p.nbytes);
        const uint64_t e = std::min<uint64_t>((uint64_t)(c + 1) * p.S, p.nbytes);
        if (e > b) n += (long long)((e - 1) / seg - b / seg + 1);
    }
    return n;
}

int walk_blocks_per_sm(int u, int P, int *bps)
{
    if (P <= 128)
        return u == 8 ? walk_occupancy<8, 128>(bps) : u == 4 ? walk_occupancy<4, 128>(bps)
             : u == 2 ? walk_occupancy<2, 128>(bps) : walk_occupancy<1, 128>(bps);
    return u == 8 ? walk_occupancy<8, BCAST_MAX_RANKS>(bps) : u == 4 ? walk_occupancy<4, BCAST_MAX_RANKS>(bps)
         : u == 2 ? walk_occupancy<2, BCAST_MAX_RANKS>(bps) : walk_occupancy<1, BCAST_MAX_RANKS>(bps);
}

// Launch shape of the WALK executor: words per lane (U) and blocks.
// Measured on B200: an SM's share of the work takes the same time whether 8 or 16 warps carry it
// (the SM's load/store path is the limit), so what matters is that every SM gets the same share
// -- the grid is a multiple of the SM count and slices are dealt SM by SM -- and that not more is
// in flight than needed: about 32 KB per SM (8 warps x 8 words x 512 B) saturate the memory
// system; more concurrent slices scatter the DRAM writes further and, with level-order hops,
// push the copies that are still to be re-read out of L2.
//   * Message larger than that (more than 1.4 rounds of SMs x 32 KB): U = 8, one block per SM,
//     several rounds.
//   * Smaller: everything is in flight at once and the run time is one walk down the longest hop
//     list at memory latency; take the smallest U whose slices fit the resident warps (the most
//     warps, the fewest words each).
//   * Very few ranks (P <= 4): at most three hops per slice, close to a plain copy: as many
//     bytes in flight as the SMs hold.
// BCAST_WALK_WORDS and BCAST_WALK_BLOCKS_PER_SM override the choice (for experiments).
struct WalkShape {
    int u = 1, grid = 1;
};

int choose_walk_shape(const bcast_plan_t &p, int sm_count, WalkShape *shape)
{
    const int forced_u = env_int("BCAST_WALK_WORDS", 0);
    const int forced_bps = env_int("BCAST_WALK_BLOCKS_PER_SM", 0);
    const bool u_ok = forced_u == 1 || forced_u == 2 || forced_u == 4 || forced_u == 8;
    int rc, resident = 1, u = 0, bps = 0;
    if (u_ok || forced_bps > 0) {
        u = u_ok ? forced_u : 8;
        if ((rc = walk_blocks_per_sm(u, p.P, &resident))) return rc;
        bps = forced_bps > 0 ? std::min(forced_bps, resident) : resident;
    } else if (p.P <= 4) {
        u = 2;
        if ((rc = walk_blocks_per_sm(u, p.P, &resident))) return rc;
        bps = resident;
    } else if (count_walk_slices(p, 8) * 5 > (long long)sm_count * kWarpsPerBlock * 7) {   // > 1.4 rounds
        u = 8;
        bps = 1;
    } else {
        for (int cand : {1, 2, 4, 8}) {
            if ((rc = walk_blocks_per_sm(cand, p.P, &resident))) return rc;
            const long long slices = count_walk_slices(p, cand);
            if (slices <= (long long)sm_count * resident * kWarpsPerBlock) {
                u = cand;
                bps = (int)std::max<long long>(1, (slices + (long long)sm_count * kWarpsPerBlock - 1) /
                                                      ((long long)sm_count * kWarpsPerBlock));
                break;
            }
        }
        if (!u) { u = 8; bps = 1; }
    }
    const long long slices = std::max<long long>(1, count_walk_slices(p, u));
    shape->u = u;
    shape->grid = (int)std::min<long long>(slices, (long long)sm_count * std::max(1, bps));
    return BCAST_OK;
}

// Slices of the bulk-copy walk: every whole 16 KiB segment that lies inside one chunk is a bulk
// slice; what is left of the segments that a chunk boundary (or the end of the message) cuts
// becomes register slices on the 4 KiB grid of walk_slice<8>.
void make_bulk_slices(const bcast_plan_t &p, std::vector<WalkSlice> &bulk, std::vector<WalkSlice> &reg)
{
    constexpr uint64_t kReg = 32ull * 8 * 16;
    bulk.clear();
    reg.clear();
    for (int c = 0; c < p.P; c++) {
        const uint64_t b = std::min<uint64_t>((uint64_t)c * p.S, p.nbytes);
        const uint64_t e = std::min<uint64_t>((uint64_t)(c + 1) * p.S, p.nbytes);
        for (uint64_t g = b / kBulkSeg; b < e && g * kBulkSeg < e; g++) {
            const uint64_t lo = std::max(b, g * kBulkSeg), hi = std::min(e, (g + 1) * kBulkSeg);
            if (hi - lo == kBulkSeg) {
                bulk.push_back(WalkSlice{(uint32_t)g, (uint32_t)c});
                continue;
            }
            for (uint64_t q = lo / kReg; q * kReg < hi; q++) reg.push_back(WalkSlice{(uint32_t)q, (uint32_t)c});
        }
    }
}

int build_bulk_tables(const bcast_plan_t &p, bcast_device_state &ds)
{
    std::vector<WalkSlice> bulk, reg;
    make_bulk_slices(p, bulk, reg);
    ds.n_bulk = (long long)bulk.size();
    ds.n_reg = (long long)reg.size();
    int rc;
    if ((rc = upload(&ds.d_bulk_slices, bulk))) return rc;
    if ((rc = upload(&ds.d_reg_slices, reg))) return rc;
    CUDA_TRY(cudaMalloc((void **)&ds.d_status, sizeof(int)));
    CUDA_TRY(cudaMemset(ds.d_status, 0, sizeof(int)));
    // three blocks of four workers per SM: 192 KB of segments in flight per SM
    const size_t smem = (size_t)kBulkWorkers * kBulkSeg;
    int resident = 0;
    if (p.P <= 128) {
        CUDA_TRY(cudaFuncSetAttribute(bcast_walk_bulk_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, bcast_walk_bulk_kernel<128>, kBulkThreads, smem));
    } else {
        CUDA_TRY(cudaFuncSetAttribute(bcast_walk_bulk_kernel<BCAST_MAX_RANKS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, bcast_walk_bulk_kernel<BCAST_MAX_RANKS>, kBulkThreads, smem));
    }
    const int bps = std::max(1, std::min(resident, env_int("BCAST_BULK_BLOCKS_PER_SM", 3)));
    const long long want = std::max<long long>(1, std::max((ds.n_bulk + kBulkWorkers - 1) / kBulkWorkers, ds.n_reg));
    ds.bulk_grid = (int)std::min<long long>(want, (long long)ds.sm_count * bps);
    return BCAST_OK;
}

// Device tables of the WALK executor, cached in the plan's device state.
int build_walk_tables(const bcast_plan_t &p, bcast_device_state &ds)
{
    WalkShape shape;
    int rc = choose_walk_shape(p, ds.sm_count, &shape);
    if (rc) return rc;
    ds.walk_u = shape.u;
    ds.walk_grid = shape.grid;
    WalkTables t;
    if ((rc = make_walk_tables(p, ds.walk_u, t))) return rc;
    ds.n_slices = (long long)t.slices.size();
    if ((rc = upload(&ds.d_slices, t.slices))) return rc;
    if ((rc = upload(&ds.d_hops, t.hops))) return rc;
    if ((rc = upload(&ds.d_hops_plan, t.hops_plan))) return rc;
    if ((rc = upload(&ds.d_hop_begin, t.hop_begin))) return rc;
    return BCAST_OK;
}

int get_state(const bcast_plan_t &p, bcast_device_state **out)
{
    int device = -1;
    CUDA_TRY(cudaGetDevice(&device));
    if (p.dev) {
        if (p.dev->device != device) return BCAST_ERR_INVAL;
        *out = p.dev;
        return BCAST_OK;
    }
    bcast_device_state *ds = new (std::nothrow) bcast_device_state();
    if (!ds) return BCAST_ERR_NOMEM;
    ds->device = device;
    int rc = BCAST_OK;
    cudaError_t e = cudaDeviceGetAttribute(&ds->sm_count, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess) { t_last_cuda_error = (int)e; rc = BCAST_ERR_CUDA; }
    try {
        if (!rc) rc = build_step_tables(p, *ds);
        if (!rc) rc = build_walk_tables(p, *ds);
        if (!rc) rc = build_bulk_tables(p, *ds);
    } catch (const std::bad_alloc &) {
        rc = BCAST_ERR_NOMEM;
    }
    if (rc) { bcast_device_state_free(ds); return rc; }
    p.dev = ds;
    *out = ds;
    return BCAST_OK;
}

// NULL, misaligned or overlapping rank buffers are refused before anything is launched.
int validate_bufs(void *const *rank_bufs, size_t P, uint64_t nbytes)
{
    std::vector<uintptr_t> a(P);
    for (size_t k = 0; k < P; k++) {
        a[k] = (uintptr_t)rank_bufs[k];
        if (!a[k] || (a[k] & 15)) return BCAST_ERR_INVAL;
    }
    std::sort(a.begin(), a.end());
    for (size_t k = 1; k < P; k++)
        if (a[k] - a[k - 1] < std::max<uint64_t>(nbytes, 1)) return BCAST_ERR_INVAL;
    return BCAST_OK;
}

// Every rank buffer must be memory of the current device (or managed memory): a host pointer
// handed to the kernels would fault the GPU.  Only the first byte of each buffer can be checked.
int validate_device_memory(void *const *rank_bufs, size_t P)
{
    int device = -1;
    CUDA_TRY(cudaGetDevice(&device));
    for (size_t k = 0; k < P; k++) {
        cudaPointerAttributes attr;
        const cudaError_t e = cudaPointerGetAttributes(&attr, rank_bufs[k]);
        if (e != cudaSuccess) {
            cudaGetLastError();   // not a sticky error: clear it
            return BCAST_ERR_INVAL;
        }
        if (attr.type == cudaMemoryTypeManaged) continue;
        if (attr.type != cudaMemoryTypeDevice || attr.device != device) return BCAST_ERR_INVAL;
    }
    return BCAST_OK;
}

// Both checks, skipped when the pointers are the ones that passed them last time.
int check_bufs(void *const *rank_bufs, const bcast_plan_t &p, bcast_device_state &ds)
{
    const size_t P = (size_t)p.P;
    if (ds.checked_bufs.size() == P && std::memcmp(ds.checked_bufs.data(), rank_bufs, P * sizeof(void *)) == 0)
        return BCAST_OK;
    int rc = validate_bufs(rank_bufs, P, p.nbytes);
    if (!rc) rc = validate_device_memory(rank_bufs, P);
    if (rc) return rc;
    ds.checked_bufs.assign(rank_bufs, rank_bufs + P);
    return BCAST_OK;
}

template <int MAXP>
void fill_ptrs(RankPtrs<MAXP> &rp, void *const *rank_bufs, int P)
{
    for (int k = 0; k < P; k++) rp.p[k] = (uint8_t *)rank_bufs[k];
    for (int k = P; k < MAXP; k++) rp.p[k] = nullptr;
}

struct WalkLaunch {     // everything one WALK launch needs besides the rank pointers
    int u, grid;
    const WalkSlice *slices;
    long long n_slices;
    uint64_t scatter_size, nbytes;
    const uint32_t *hops;
    const int *hop_begin;
};

template <int MAXP>
int launch_walk_tables(const WalkLaunch &w, void *const *rank_bufs, int P, cudaStream_t st)
{
    RankPtrs<MAXP> rp;
    fill_ptrs(rp, rank_bufs, P);
#define BCAST_WALK_LAUNCH(U_)                                                                       \
    bcast_walk_kernel<U_, MAXP><<<w.grid, kThreads, 0, st>>>(rp, w.slices, w.n_slices, w.scatter_size, \
                                                             w.nbytes, w.hops, w.hop_begin)
    switch (w.u) {
    case 8: BCAST_WALK_LAUNCH(8); break;
    case 4: BCAST_WALK_LAUNCH(4); break;
    case 2: BCAST_WALK_LAUNCH(2); break;
    default: BCAST_WALK_LAUNCH(1); break;
    }
#undef BCAST_WALK_LAUNCH
    CUDA_TRY(cudaGetLastError());
    return BCAST_OK;
}

int launch_walk(const bcast_plan_t &p, const bcast_device_state &ds, void *const *rank_bufs, bool plan_order,
                cudaStream_t st)
{
    const WalkLaunch w{ds.walk_u, ds.walk_grid, ds.d_slices, ds.n_slices, p.S, p.nbytes,
                       plan_order ? ds.d_hops_plan : ds.d_hops, ds.d_hop_begin};
    return p.P <= 128 ? launch_walk_tables<128>(w, rank_bufs, p.P, st)
                      : launch_walk_tables<BCAST_MAX_RANKS>(w, rank_bufs, p.P, st);
}

template <int MAXP>
int launch_walk_bulk_tables(const bcast_plan_t &p, const bcast_device_state &ds, void *const *rank_bufs, cudaStream_t st)
{
    RankPtrs<MAXP> rp;
    fill_ptrs(rp, rank_bufs, p.P);
    bcast_walk_bulk_kernel<MAXP><<<ds.bulk_grid, kBulkThreads, (size_t)kBulkWorkers * kBulkSeg, st>>>(
        rp, ds.d_bulk_slices, ds.n_bulk, ds.d_reg_slices, ds.n_reg, p.S, p.nbytes, ds.d_hops, ds.d_hop_begin, ds.d_status);
    CUDA_TRY(cudaGetLastError());
    return BCAST_OK;
}

int launch_walk_bulk(const bcast_plan_t &p, const bcast_device_state &ds, void *const *rank_bufs, cudaStream_t st)
{
    return p.P <= 128 ? launch_walk_bulk_tables<128>(p, ds, rank_bufs, st)
                      : launch_walk_bulk_tables<BCAST_MAX_RANKS>(p, ds, rank_bufs, st);
}

template <int MAXP>
int launch_steps(const bcast_device_state &ds, void *const *rank_bufs, int P, cudaStream_t st)
{
    RankPtrs<MAXP> rp;
    fill_ptrs(rp, rank_bufs, P);
    for (const StepLaunch &sl : ds.steps) {
        if (!sl.tiles) continue;
        bcast_step_kernel<MAXP><<<dim3(sl.tiles, sl.count), kThreads, 0, st>>>(rp, ds.d_xfers + sl.first);
        CUDA_TRY(cudaGetLastError());
    }
    return BCAST_OK;
}

int launch_graph(bcast_device_state &ds, void *const *rank_bufs, int P, cudaStream_t st)
{
    const bool same = ds.graph_exec && ds.graph_bufs.size() == (size_t)P &&
                      std::memcmp(ds.graph_bufs.data(), rank_bufs, (size_t)P * sizeof(void *)) == 0;
    if (!same) {
        if (ds.graph_exec) { cudaGraphExecDestroy(ds.graph_exec); ds.graph_exec = nullptr; }
        if (ds.graph) { cudaGraphDestroy(ds.graph); ds.graph = nullptr; }
        cudaStream_t cap = nullptr;
        CUDA_TRY(cudaStreamCreateWithFlags(&cap, cudaStreamNonBlocking));
        int rc = BCAST_OK;
        cudaError_t e = cudaStreamBeginCapture(cap, cudaStreamCaptureModeThreadLocal);
        if (e == cudaSuccess) {
            rc = P <= 128 ? launch_steps<128>(ds, rank_bufs, P, cap) : launch_steps<BCAST_MAX_RANKS>(ds, rank_bufs, P, cap);
            e = cudaStreamEndCapture(cap, &ds.graph);
        }
        cudaStreamDestroy(cap);
        if (rc) return rc;
        CUDA_TRY(e);
        CUDA_TRY(cudaGraphInstantiate(&ds.graph_exec, ds.graph, 0));
        ds.graph_bufs.assign(rank_bufs, rank_bufs + P);
    }
    CUDA_TRY(cudaGraphLaunch(ds.graph_exec, st));
    return BCAST_OK;
}

}  // namespace

extern "C" {

int bcast_exec_mode(void *const *rank_bufs, const bcast_plan_t *plan, void *cuda_stream, int mode)
{
    if (!rank_bufs || !plan) return BCAST_ERR_INVAL;
    if (mode != BCAST_EXEC_WALK && mode != BCAST_EXEC_STEPS && mode != BCAST_EXEC_GRAPH &&
        mode != BCAST_EXEC_WALK_PLAN_ORDER && mode != BCAST_EXEC_WALK_BULK && mode != BCAST_EXEC_AUTO)
        return BCAST_ERR_INVAL;
    const bcast_plan_t &p = *plan;
    bcast_device_state *ds = nullptr;
    int rc = get_state(p, &ds);
    if (rc) return rc;
    try {
        rc = check_bufs(rank_bufs, p, *ds);
    } catch (const std::bad_alloc &) {
        rc = BCAST_ERR_NOMEM;
    }
    if (rc) return rc;
    if (p.total_bytes == 0) return BCAST_OK;   // P = 1 or an empty message: nothing moves
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int P = p.P;
    // The bulk-copy walk needs ~4x the bytes in flight of the register walk.  With plan-order hops
    // (native, doubling) a segment is re-read on the very next hop and that still fits in L2; with
    // the tuned variant's level-order hops the re-read comes up to a tree level later and no longer
    // does (measured: 11-20 % slower than the register walk), so the tuned variant stays with registers.
    // It also needs at least two rounds of its own to pay: below that (about 58 MB on 148 SMs) the
    // register walk is as fast or faster (16 MiB messages: 11 % faster).
    if (mode == BCAST_EXEC_AUTO) {
        const bool bulk_pays = ds->n_bulk >= 2ll * ds->bulk_grid * kBulkWorkers;
        mode = bulk_pays && p.variant != BCAST_TUNED ? BCAST_EXEC_WALK_BULK : BCAST_EXEC_WALK;
    }
    switch (mode) {
    case BCAST_EXEC_WALK_BULK:
        return launch_walk_bulk(p, *ds, rank_bufs, st);
    case BCAST_EXEC_WALK:
    case BCAST_EXEC_WALK_PLAN_ORDER: {
        return launch_walk(p, *ds, rank_bufs, mode == BCAST_EXEC_WALK_PLAN_ORDER, st);
    }
    case BCAST_EXEC_STEPS:
        return P <= 128 ? launch_steps<128>(*ds, rank_bufs, P, st) : launch_steps<BCAST_MAX_RANKS>(*ds, rank_bufs, P, st);
    default:
        try {
            return launch_graph(*ds, rank_bufs, P, st);
        } catch (const std::bad_alloc &) {
            return BCAST_ERR_NOMEM;
        }
    }
}

int bcast_exec(void *const *rank_bufs, const bcast_plan_t *plan, void *cuda_stream)
{
    return bcast_exec_mode(rank_bufs, plan, cuda_stream, BCAST_EXEC_AUTO);
}

int bcast_exec_host(void *const *rank_bufs, const bcast_plan_t *plan, void *cuda_stream, int mode,
                    const void *host_message, void *const *host_out)
{
    if (!rank_bufs || !plan) return BCAST_ERR_INVAL;
    const bcast_plan_t &p = *plan;
    if (p.nbytes && !host_message) return BCAST_ERR_INVAL;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // validate the buffers before the first copy touches them
    bcast_device_state *ds = nullptr;
    int rc = get_state(p, &ds);
    if (rc) return rc;
    try {
        rc = check_bufs(rank_bufs, p, *ds);
    } catch (const std::bad_alloc &) {
        rc = BCAST_ERR_NOMEM;
    }
    if (rc) return rc;
    if (p.nbytes)
        CUDA_TRY(cudaMemcpyAsync(rank_bufs[p.root], host_message, p.nbytes, cudaMemcpyHostToDevice, st));
    rc = bcast_exec_mode(rank_bufs, plan, cuda_stream, mode);
    if (rc) return rc;
    if (host_out && p.nbytes)
        for (int k = 0; k < p.P; k++)
            if (host_out[k])
                CUDA_TRY(cudaMemcpyAsync(host_out[k], rank_bufs[k], p.nbytes, cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaStreamSynchronize(st));
    return BCAST_OK;
}

int64_t bcast_plan_walk_order(const bcast_plan_t *plan, int chunk, int mode, int64_t *out, int64_t cap)
{
    if (!plan || chunk < 0 || chunk >= plan->P || cap < 0 || (cap > 0 && !out)) return BCAST_ERR_INVAL;
    if (mode != BCAST_EXEC_WALK && mode != BCAST_EXEC_WALK_PLAN_ORDER) return BCAST_ERR_INVAL;
    try {
        std::vector<std::vector<int64_t>> per_chunk;
        messages_by_chunk(*plan, per_chunk);
        std::vector<int64_t> order = per_chunk[chunk];
        if (mode == BCAST_EXEC_WALK) order_by_dependency(*plan, per_chunk[chunk], order);
        for (int64_t i = 0; i < (int64_t)order.size() && i < cap; i++) out[i] = order[i];
        return (int64_t)order.size();
    } catch (const std::bad_alloc &) {
        return BCAST_ERR_NOMEM;
    }
}

int64_t bcast_exec_num_launches(const bcast_plan_t *plan, int mode)
{
    if (!plan || plan->total_bytes == 0) return 0;
    if (mode == BCAST_EXEC_WALK || mode == BCAST_EXEC_WALK_PLAN_ORDER || mode == BCAST_EXEC_WALK_BULK ||
        mode == BCAST_EXEC_AUTO)
        return 1;
    if (mode != BCAST_EXEC_STEPS && mode != BCAST_EXEC_GRAPH) return 0;
    // a step launches a kernel unless all of its messages are empty
    int64_t n = 0;
    const int nsteps = (int)plan->step_begin.size() - 1;
    for (int s = 0; s < nsteps; s++) {
        bool any = false;
        for (int64_t i = plan->step_begin[s]; i < plan->step_begin[s + 1] && !any; i++) any = plan->xfers[i].len != 0;
        n += any;
    }
    return n;
}

int bcast_exec_status(const bcast_plan_t *plan)
{
    if (!plan) return BCAST_ERR_INVAL;
    if (!plan->dev || !plan->dev->d_status) return BCAST_OK;     // never executed: nothing to report
    int flag = 0;
    CUDA_TRY(cudaMemcpy(&flag, plan->dev->d_status, sizeof(int), cudaMemcpyDeviceToHost));
    if (!flag) return BCAST_OK;
    CUDA_TRY(cudaMemset(plan->dev->d_status, 0, sizeof(int)));
    return BCAST_ERR_TIMEOUT;
}

int bcast_last_cuda_error(void) { return t_last_cuda_error; }

}  // extern "C"

// ============================================================== execution without allocation
// Scratch of bcast_exec_static(): lives in the library's device image, one copy per GPU that
// loads it.  In host code this name is only a handle; the device address comes from
// cudaGetSymbolAddress (once per device) and is what the kernel receives.
static __device__ __align__(256) unsigned char g_static_scratch[BCAST_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
unsigned char *g_static_addr[kMaxDevices] = {};   // device address of g_static_scratch, per device
int g_static_sms[kMaxDevices] = {};
std::vector<void *> g_static_checked;             // rank buffers that last passed the device-memory check

inline size_t round256(size_t x) { return (x + 255) & ~(size_t)255; }

// Device address of the scratch on the current device; looked up on the first call per device.
int static_scratch(unsigned char **addr, int *sm_count)
{
    int device = -1;
    CUDA_TRY(cudaGetDevice(&device));
    if (device < 0 || device >= kMaxDevices) return BCAST_ERR_INVAL;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_addr[device]) {
        void *p = nullptr;
        CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
        int sms = 0;
        CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
        g_static_addr[device] = (unsigned char *)p;
        g_static_sms[device] = sms;
    }
    *addr = g_static_addr[device];
    *sm_count = g_static_sms[device];
    return BCAST_OK;
}

int exec_static(void *const *rank_bufs, const bcast_plan_t &p, cudaStream_t st)
{
    int rc = validate_bufs(rank_bufs, (size_t)p.P, p.nbytes);
    if (rc) return rc;
    {
        // the device-memory check costs a driver call per buffer: remember the last set that passed
        std::lock_guard<std::mutex> lock(g_static_mu);
        if (g_static_checked.size() != (size_t)p.P ||
            std::memcmp(g_static_checked.data(), rank_bufs, (size_t)p.P * sizeof(void *)) != 0) {
            if ((rc = validate_device_memory(rank_bufs, (size_t)p.P))) return rc;
            g_static_checked.assign(rank_bufs, rank_bufs + p.P);
        }
    }
    if (p.total_bytes == 0) return BCAST_OK;
    unsigned char *scratch = nullptr;
    int sms = 0;
    if ((rc = static_scratch(&scratch, &sms))) return rc;

    // tables on the host; if they do not fit, try the largest slices before giving up
    WalkShape shape;
    if ((rc = choose_walk_shape(p, sms, &shape))) return rc;
    WalkTables t;
    size_t off_slices = 0, off_hops = 0, total = 0;
    for (;;) {
        if ((rc = make_walk_tables(p, shape.u, t))) return rc;
        off_slices = round256(t.hop_begin.size() * sizeof(int));
        off_hops = off_slices + round256(t.slices.size() * sizeof(WalkSlice));
        total = off_hops + round256(t.hops.size() * sizeof(uint32_t));
        if (total <= BCAST_STATIC_SCRATCH_BYTES) break;
        if (shape.u == 8) return BCAST_ERR_CAPACITY;
        shape.u = 8;
        shape.grid = std::max(1, std::min<int>(shape.grid, (int)((count_walk_slices(p, 8) + kWarpsPerBlock - 1) / kWarpsPerBlock)));
    }

    // one image of the three tables; a single stream-ordered copy puts it in place (the source is
    // pageable host memory, which the runtime stages before returning).  Nothing in the array has
    // to start at zero: the kernel only reads it.
    std::vector<unsigned char> img(total, 0);
    std::memcpy(img.data(), t.hop_begin.data(), t.hop_begin.size() * sizeof(int));
    std::memcpy(img.data() + off_slices, t.slices.data(), t.slices.size() * sizeof(WalkSlice));
    std::memcpy(img.data() + off_hops, t.hops.data(), t.hops.size() * sizeof(uint32_t));
    CUDA_TRY(cudaMemcpyAsync(scratch, img.data(), total, cudaMemcpyHostToDevice, st));

    const WalkLaunch w{shape.u, shape.grid, (const WalkSlice *)(scratch + off_slices), (long long)t.slices.size(),
                       p.S, p.nbytes, (const uint32_t *)(scratch + off_hops), (const int *)scratch};
    return p.P <= 128 ? launch_walk_tables<128>(w, rank_bufs, p.P, st)
                      : launch_walk_tables<BCAST_MAX_RANKS>(w, rank_bufs, p.P, st);
}

}  // namespace

extern "C" int bcast_exec_static(void *const *rank_bufs, const bcast_plan_t *plan, void *cuda_stream)
{
    if (!rank_bufs || !plan) return BCAST_ERR_INVAL;
    try {
        return exec_static(rank_bufs, *plan, (cudaStream_t)cuda_stream);
    } catch (const std::bad_alloc &) {
        return BCAST_ERR_NOMEM;
    }
}
