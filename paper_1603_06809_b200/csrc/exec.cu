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
// WALK executor (one launch): the message is cut into tiles on a fixed grid of byte offsets, split
// further at chunk boundaries.  A thread block takes a tile and performs, in plan order, every
// message that covers the tile's chunk, restricted to the tile: load from the source rank's
// buffer, store to the destination rank's buffer.  Each thread always handles the same bytes of
// the tile, so the load of hop h+1 reads what the same thread stored in hop h or earlier:
// program order per thread is the only ordering the schedule needs.  Loads bypass L1 (.cg) so that
// every hop really re-reads the source rank's buffer from the L2/HBM level.
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
constexpr int kMaxHops = BCAST_MAX_RANKS + 16;   // a chunk is covered by <= L + P - 1 messages

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

struct WalkItem {     // one tile of one chunk: bytes [lo, hi) of the message
    uint64_t lo, hi;
    int32_t chunk;    // relative chunk index: selects the hop list
    int32_t pad;
};

struct WalkCtl {      // work counter of the WALK executor; both fields are 0 between launches
    unsigned int ticket, done;
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
template <int U, int MAXP>
__global__ void __launch_bounds__(kThreads)
bcast_walk_kernel(const __grid_constant__ RankPtrs<MAXP> bufs, const WalkItem *__restrict__ items, int n_items,
                  const uint32_t *__restrict__ hops, const int *__restrict__ hop_begin, WalkCtl *ctl)
{
    __shared__ uint32_t s_hops[kMaxHops];
    __shared__ int s_item;
    const int tid = threadIdx.x;

    for (;;) {
        if (tid == 0) s_item = (int)atomicAdd(&ctl->ticket, 1u);
        __syncthreads();
        const int it = s_item;
        if (it >= n_items) break;
        const WalkItem item = items[it];
        const int hb = hop_begin[item.chunk];
        const int nh = hop_begin[item.chunk + 1] - hb;
        for (int h = tid; h < nh; h += kThreads) s_hops[h] = hops[hb + h];
        __syncthreads();

        const Split sp = split16(item.lo, item.hi);
        const uint64_t base = sp.a0 + (uint64_t)tid * 16;
        if (sp.nwords == (uint32_t)(kThreads * U) && sp.nhead == 0 && sp.ntail == 0) {
            // full tile: every thread moves U words per hop, no predicates
            for (int h = 0; h < nh; h++) {
                const uint32_t e = s_hops[h];
                const uint8_t *s = bufs.p[e & 0xffffu] + base;
                uint8_t *d = bufs.p[e >> 16] + base;
                uint4 v[U];
#pragma unroll
                for (int u = 0; u < U; u++) v[u] = ld16(s + (uint64_t)u * kThreads * 16);
#pragma unroll
                for (int u = 0; u < U; u++) st16(d + (uint64_t)u * kThreads * 16, v[u]);
            }
        } else {
            // ragged tile (chunk boundary or end of message): predicated words plus edge bytes,
            // one byte per thread (at most 15 head + 15 tail bytes)
            const uint32_t nedge = sp.nhead + sp.ntail;
            const bool has_edge = (uint32_t)tid < nedge;
            const uint64_t eoff = (uint32_t)tid < sp.nhead ? item.lo + tid : sp.tail_begin + (tid - sp.nhead);
            for (int h = 0; h < nh; h++) {
                const uint32_t e = s_hops[h];
                const uint8_t *s = bufs.p[e & 0xffffu];
                uint8_t *d = bufs.p[e >> 16];
                uint4 v[U];
                uint32_t b = 0;
#pragma unroll
                for (int u = 0; u < U; u++)
                    if ((uint32_t)(tid + u * kThreads) < sp.nwords) v[u] = ld16(s + base + (uint64_t)u * kThreads * 16);
                if (has_edge) b = ld1(s + eoff);
#pragma unroll
                for (int u = 0; u < U; u++)
                    if ((uint32_t)(tid + u * kThreads) < sp.nwords) st16(d + base + (uint64_t)u * kThreads * 16, v[u]);
                if (has_edge) st1(d + eoff, b);
            }
        }
        __syncthreads();   // s_item and s_hops are rewritten by the next round
    }

    // the last block to leave puts the counters back to zero for the next launch
    if (tid == 0) {
        __threadfence();
        const unsigned int d = atomicAdd(&ctl->done, 1u);
        if (d == gridDim.x - 1) {
            __threadfence();
            ctl->ticket = 0;
            ctl->done = 0;
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
    int64_t nonempty_steps = 0;
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t graph_exec = nullptr;
    std::vector<void *> graph_bufs;
    // WALK
    WalkItem *d_items = nullptr;
    uint32_t *d_hops = nullptr;
    int *d_hop_begin = nullptr;
    WalkCtl *d_ctl = nullptr;
    int n_items = 0, walk_u = 0, walk_grid = 0;
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
    cudaFree(dev->d_items);
    cudaFree(dev->d_hops);
    cudaFree(dev->d_hop_begin);
    cudaFree(dev->d_ctl);
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
    ds.nonempty_steps = 0;
    for (int s = 0; s < nsteps; s++) {
        StepLaunch sl{p.step_begin[s], (unsigned)(p.step_begin[s + 1] - p.step_begin[s]), 0u};
        for (int64_t i = p.step_begin[s]; i < p.step_begin[s + 1]; i++) {
            const bcast_xfer_t &x = p.xfers[i];
            if (!x.len) continue;
            const uint64_t t = (x.offset + x.len - 1) / kStepTile - x.offset / kStepTile + 1;
            sl.tiles = std::max<unsigned>(sl.tiles, (unsigned)t);
        }
        ds.steps[s] = sl;
        ds.nonempty_steps += sl.tiles > 0;
    }
    return upload(&ds.d_xfers, hx);
}

// Host form of the WALK executor's tables: per chunk the list of (src, dst) hops in plan order,
// and the tiles (fixed grid of `256 * u * 16`-byte offsets, split at chunk boundaries).
struct WalkTables {
    std::vector<WalkItem> items;
    std::vector<uint32_t> hops;
    std::vector<int> hop_begin;   // [P + 1], by relative chunk index
};

int make_walk_tables(const bcast_plan_t &p, int u, WalkTables &t)
{
    const int P = p.P;
    auto chunk_begin = [&](int c) { return std::min<uint64_t>((uint64_t)c * p.S, p.nbytes); };
    std::vector<std::vector<uint32_t>> per_chunk(P);
    for (const bcast_xfer_t &x : p.xfers) {
        if (!x.len) continue;
        const uint32_t e = (uint32_t)x.src_rank | ((uint32_t)x.dst_rank << 16);
        for (int c = x.chunk; c < x.chunk + x.nchunks; c++)
            if (chunk_begin(c + 1) > chunk_begin(c)) per_chunk[c].push_back(e);
    }
    t.hop_begin.assign(P + 1, 0);
    t.hops.clear();
    for (int c = 0; c < P; c++) {
        if ((int)per_chunk[c].size() > kMaxHops) return BCAST_ERR_INVAL;
        t.hop_begin[c] = (int)t.hops.size();
        t.hops.insert(t.hops.end(), per_chunk[c].begin(), per_chunk[c].end());
    }
    t.hop_begin[P] = (int)t.hops.size();

    const uint64_t tile = (uint64_t)kThreads * u * 16;
    t.items.clear();
    for (int c = 0; c < P; c++) {
        const uint64_t b = chunk_begin(c), e = chunk_begin(c + 1);
        if (e <= b || per_chunk[c].empty()) continue;
        for (uint64_t g = b / tile; g * tile < e; g++)
            t.items.push_back(WalkItem{std::max(b, g * tile), std::min(e, (g + 1) * tile), c, 0});
    }
    return BCAST_OK;
}

// words per thread: large tiles when the message is big enough to fill the GPU with them
int choose_walk_words(uint64_t nbytes, int sm_count)
{
    const int forced = env_int("BCAST_WALK_WORDS", 0);
    if (forced == 1 || forced == 2 || forced == 4 || forced == 8) return forced;
    for (int cand : {4, 2}) {
        const uint64_t tile = (uint64_t)kThreads * cand * 16;
        if (nbytes / tile >= (uint64_t)sm_count * 8) return cand;
    }
    return 1;
}

int walk_blocks_per_sm(int u, int P, int *bps)
{
    if (P <= 128)
        return u == 8 ? walk_occupancy<8, 128>(bps) : u == 4 ? walk_occupancy<4, 128>(bps)
             : u == 2 ? walk_occupancy<2, 128>(bps) : walk_occupancy<1, 128>(bps);
    return u == 8 ? walk_occupancy<8, BCAST_MAX_RANKS>(bps) : u == 4 ? walk_occupancy<4, BCAST_MAX_RANKS>(bps)
         : u == 2 ? walk_occupancy<2, BCAST_MAX_RANKS>(bps) : walk_occupancy<1, BCAST_MAX_RANKS>(bps);
}

// Device tables of the WALK executor, cached in the plan's device state.
int build_walk_tables(const bcast_plan_t &p, bcast_device_state &ds)
{
    ds.walk_u = choose_walk_words(p.nbytes, ds.sm_count);
    WalkTables t;
    int rc = make_walk_tables(p, ds.walk_u, t);
    if (rc) return rc;
    ds.n_items = (int)t.items.size();
    int bps = 1;
    if ((rc = walk_blocks_per_sm(ds.walk_u, p.P, &bps))) return rc;
    const int cap = env_int("BCAST_WALK_BLOCKS_PER_SM", bps);
    ds.walk_grid = std::max(1, std::min(ds.n_items, ds.sm_count * std::max(1, std::min(cap, bps))));

    if ((rc = upload(&ds.d_items, t.items))) return rc;
    if ((rc = upload(&ds.d_hops, t.hops))) return rc;
    if ((rc = upload(&ds.d_hop_begin, t.hop_begin))) return rc;
    CUDA_TRY(cudaMalloc((void **)&ds.d_ctl, sizeof(WalkCtl)));
    CUDA_TRY(cudaMemset(ds.d_ctl, 0, sizeof(WalkCtl)));
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

// The same check, skipped when the pointers are the ones that passed it last time.
int check_bufs(void *const *rank_bufs, const bcast_plan_t &p, bcast_device_state &ds)
{
    const size_t P = (size_t)p.P;
    if (ds.checked_bufs.size() == P && std::memcmp(ds.checked_bufs.data(), rank_bufs, P * sizeof(void *)) == 0)
        return BCAST_OK;
    const int rc = validate_bufs(rank_bufs, P, p.nbytes);
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

template <int MAXP>
int launch_walk_tables(int u, int grid, void *const *rank_bufs, int P, const WalkItem *items, int n_items,
                       const uint32_t *hops, const int *hop_begin, WalkCtl *ctl, cudaStream_t st)
{
    RankPtrs<MAXP> rp;
    fill_ptrs(rp, rank_bufs, P);
    switch (u) {
    case 8: bcast_walk_kernel<8, MAXP><<<grid, kThreads, 0, st>>>(rp, items, n_items, hops, hop_begin, ctl); break;
    case 4: bcast_walk_kernel<4, MAXP><<<grid, kThreads, 0, st>>>(rp, items, n_items, hops, hop_begin, ctl); break;
    case 2: bcast_walk_kernel<2, MAXP><<<grid, kThreads, 0, st>>>(rp, items, n_items, hops, hop_begin, ctl); break;
    default: bcast_walk_kernel<1, MAXP><<<grid, kThreads, 0, st>>>(rp, items, n_items, hops, hop_begin, ctl); break;
    }
    CUDA_TRY(cudaGetLastError());
    return BCAST_OK;
}

template <int MAXP>
int launch_walk(const bcast_device_state &ds, void *const *rank_bufs, int P, cudaStream_t st)
{
    return launch_walk_tables<MAXP>(ds.walk_u, ds.walk_grid, rank_bufs, P, ds.d_items, ds.n_items, ds.d_hops,
                                    ds.d_hop_begin, ds.d_ctl, st);
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
    if (mode != BCAST_EXEC_WALK && mode != BCAST_EXEC_STEPS && mode != BCAST_EXEC_GRAPH) return BCAST_ERR_INVAL;
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
    switch (mode) {
    case BCAST_EXEC_WALK:
        return P <= 128 ? launch_walk<128>(*ds, rank_bufs, P, st) : launch_walk<BCAST_MAX_RANKS>(*ds, rank_bufs, P, st);
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
    return bcast_exec_mode(rank_bufs, plan, cuda_stream, BCAST_EXEC_WALK);
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

int64_t bcast_exec_num_launches(const bcast_plan_t *plan, int mode)
{
    if (!plan || plan->total_bytes == 0) return 0;
    if (mode == BCAST_EXEC_WALK) return 1;
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
    if (p.total_bytes == 0) return BCAST_OK;
    unsigned char *scratch = nullptr;
    int sms = 0;
    if ((rc = static_scratch(&scratch, &sms))) return rc;

    // tables on the host; if they do not fit, try the largest tile before giving up
    WalkTables t;
    int u = choose_walk_words(p.nbytes, sms);
    size_t off_hop_begin = 0, off_items = 0, off_hops = 0, total = 0;
    for (;;) {
        if ((rc = make_walk_tables(p, u, t))) return rc;
        off_hop_begin = round256(sizeof(WalkCtl));
        off_items = off_hop_begin + round256(t.hop_begin.size() * sizeof(int));
        off_hops = off_items + round256(t.items.size() * sizeof(WalkItem));
        total = off_hops + round256(t.hops.size() * sizeof(uint32_t));
        if (total <= BCAST_STATIC_SCRATCH_BYTES) break;
        if (u == 8) return BCAST_ERR_CAPACITY;
        u = 8;
    }
    int bps = 1;
    if ((rc = walk_blocks_per_sm(u, p.P, &bps))) return rc;
    const int n_items = (int)t.items.size();
    const int grid = std::max(1, std::min(n_items, sms * std::max(1, bps)));

    // one image: zeroed work counter, then the three tables; a single stream-ordered copy puts it
    // in place (the source is pageable host memory, which the runtime stages before returning)
    std::vector<unsigned char> img(total, 0);
    std::memcpy(img.data() + off_hop_begin, t.hop_begin.data(), t.hop_begin.size() * sizeof(int));
    std::memcpy(img.data() + off_items, t.items.data(), t.items.size() * sizeof(WalkItem));
    std::memcpy(img.data() + off_hops, t.hops.data(), t.hops.size() * sizeof(uint32_t));
    CUDA_TRY(cudaMemcpyAsync(scratch, img.data(), total, cudaMemcpyHostToDevice, st));

    WalkCtl *ctl = (WalkCtl *)scratch;
    const int *hop_begin = (const int *)(scratch + off_hop_begin);
    const WalkItem *items = (const WalkItem *)(scratch + off_items);
    const uint32_t *hops = (const uint32_t *)(scratch + off_hops);
    return p.P <= 128 ? launch_walk_tables<128>(u, grid, rank_bufs, p.P, items, n_items, hops, hop_begin, ctl, st)
                      : launch_walk_tables<BCAST_MAX_RANKS>(u, grid, rank_bufs, p.P, items, n_items, hops, hop_begin, ctl, st);
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
