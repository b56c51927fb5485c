// Host side of the device executors: device tables of a plan, launch shapes, argument checks and
// the bcast_exec* entry points.  The kernels are in kernels.cuh, the table builders (slices, hop
// orders, dual lists) in walk_tables.cpp.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "exec_internal.h"
#include "kernels.cuh"
#include "plan_internal.h"
#include "walk_tables.h"

using namespace bcast_dev;

namespace {

thread_local int t_last_cuda_error = 0;

#define CUDA_TRY(expr)                                        \
    do {                                                      \
        cudaError_t e_ = (expr);                              \
        if (e_ != cudaSuccess) {                              \
            t_last_cuda_error = (int)e_;                      \
            return e_ == cudaErrorMemoryAllocation ? BCAST_ERR_NOMEM : BCAST_ERR_CUDA; \
        }                                                     \
    } while (0)

}  // namespace

// ======================================================================================= state
struct StepLaunch {
    int64_t first;     // index of the step's first message in d_xfers
    unsigned count;    // messages in the step (gridDim.y)
    unsigned tiles;    // most tiles any message of the step spans (gridDim.x); 0: nothing to copy
};

struct bcast_device_state {
    int device = -1;
    int sm_count = 0;
    std::mutex mu;                     // guards the host-side caches below (checked_bufs, graph_*)
    // STEPS / GRAPH
    DevXfer *d_xfers = nullptr;
    std::vector<StepLaunch> steps;
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t graph_exec = nullptr;
    std::vector<void *> graph_bufs;
    // WALK: hop lists and dual lists (shared by the register and the bulk walk)
    uint32_t *d_hops = nullptr, *d_hops_plan = nullptr;
    int32_t *d_hop_msg = nullptr, *d_hop_msg_plan = nullptr;
    int *d_hop_begin = nullptr, *d_dual_begin = nullptr;
    DualSlot *d_dual = nullptr;
    DualMsg *d_dual_msg = nullptr;
    // WALK: slices of the register walk and its launch shape
    WalkSlice *d_slices = nullptr;
    long long n_slices = 0;
    int walk_u = 0, walk_grid = 0, walk_group = 1;
    long long walk_grouped = 0;
    // WALK with bulk copies
    WalkSlice *d_bulk_slices = nullptr, *d_reg_slices = nullptr;
    long long n_bulk = 0, n_reg = 0;
    int bulk_grid = 0, bulk_spin_limit = kBulkSpinLimit;
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
    cudaFree(dev->d_hops);
    cudaFree(dev->d_hops_plan);
    cudaFree(dev->d_hop_msg);
    cudaFree(dev->d_hop_msg_plan);
    cudaFree(dev->d_hop_begin);
    cudaFree(dev->d_dual_begin);
    cudaFree(dev->d_dual);
    cudaFree(dev->d_dual_msg);
    cudaFree(dev->d_slices);
    cudaFree(dev->d_bulk_slices);
    cudaFree(dev->d_reg_slices);
    cudaFree(dev->d_status);
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

// ---- kernel instantiations by run-time parameters
template <int MAXP, bool TRACE>
const void *walk_kernel(int u)
{
    switch (u) {
    case 1: return (const void *)bcast_walk_kernel<1, MAXP, TRACE>;
    case 2: return (const void *)bcast_walk_kernel<2, MAXP, TRACE>;
    case 3: return (const void *)bcast_walk_kernel<3, MAXP, TRACE>;
    case 4: return (const void *)bcast_walk_kernel<4, MAXP, TRACE>;
    case 5: return (const void *)bcast_walk_kernel<5, MAXP, TRACE>;
    case 6: return (const void *)bcast_walk_kernel<6, MAXP, TRACE>;
    case 7: return (const void *)bcast_walk_kernel<7, MAXP, TRACE>;
    default: return (const void *)bcast_walk_kernel<8, MAXP, TRACE>;
    }
}
// Tracing is a test facility: it only exists for the large pointer table.
const void *walk_kernel(int u, int P, bool trace)
{
    if (trace) return walk_kernel<BCAST_MAX_RANKS, true>(u);
    return P <= 128 ? walk_kernel<128, false>(u) : walk_kernel<BCAST_MAX_RANKS, false>(u);
}
const void *bulk_kernel(int P, bool trace)
{
    if (trace) return (const void *)bcast_walk_bulk_kernel<BCAST_MAX_RANKS, true>;
    return P <= 128 ? (const void *)bcast_walk_bulk_kernel<128, false> : (const void *)bcast_walk_bulk_kernel<BCAST_MAX_RANKS, false>;
}
const void *step_kernel(int P, bool trace)
{
    if (trace) return (const void *)bcast_step_kernel<BCAST_MAX_RANKS, true>;
    return P <= 128 ? (const void *)bcast_step_kernel<128, false> : (const void *)bcast_step_kernel<BCAST_MAX_RANKS, false>;
}

// Launch `kernel`, whose first parameter is a RankPtrs<128> or RankPtrs<BCAST_MAX_RANKS> (chosen
// like the kernel itself) filled from rank_bufs; `rest` are pointers to the remaining arguments.
int launch_with_ptrs(const void *kernel, dim3 grid, dim3 block, size_t smem, cudaStream_t st, void *const *rank_bufs, int P,
                     bool trace, std::initializer_list<void *> rest)
{
    void *args[8];
    size_t n = 1;
    for (void *a : rest) args[n++] = a;
    if (P <= 128 && !trace) {
        RankPtrs<128> rp;
        for (int k = 0; k < 128; k++) rp.p[k] = k < P ? (uint8_t *)rank_bufs[k] : nullptr;
        args[0] = &rp;
        CUDA_TRY(cudaLaunchKernel(kernel, grid, block, args, smem, st));
    } else {
        RankPtrs<BCAST_MAX_RANKS> rp;
        for (int k = 0; k < BCAST_MAX_RANKS; k++) rp.p[k] = k < P ? (uint8_t *)rank_bufs[k] : nullptr;
        args[0] = &rp;
        CUDA_TRY(cudaLaunchKernel(kernel, grid, block, args, smem, st));
    }
    return BCAST_OK;
}

// ======================================================================================= tables
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

int walk_blocks_per_sm(int u, int P, int *bps)
{
    CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(bps, walk_kernel(u, P, false), kThreads, 0));
    return BCAST_OK;
}

// Launch shape of the WALK executor: words per lane (U, 1..8: segments of U x 512 bytes) and blocks.
// Measured on B200: an SM's share of the work takes the same time whether 8 or 16 warps carry it
// (the SM's load/store path is the limit), so what matters is that every SM gets the same share
// -- the grid is a multiple of the SM count and slices are dealt SM by SM -- and that not more is
// in flight than needed: about 32 KB per SM (8 warps x 8 words x 512 B) saturate the memory
// system; more concurrent slices scatter the DRAM writes further and, with level-order hops,
// push the copies that are still to be re-read out of L2.
//   * Message larger than that (more than 1.4 rounds of SMs x 32 KB): U = 8, one block per SM,
//     several rounds.  (Smaller segments that would fill the last round better were measured and
//     lose: 3.5 rounds of 4 KiB segments beat 4.0 rounds of 3.5 KiB ones by 6 %.)
//   * Smaller: everything is in flight at once and the run time is one walk down the longest hop
//     list at memory latency; take the smallest U whose slices fit the resident warps (the most
//     warps, the fewest words each).
//   * Very few ranks (P <= 4): at most three hops per slice, close to a plain copy: as many
//     bytes in flight as the SMs hold (U = 6 for P <= 3, U = 2 for P = 4, all resident blocks).
// BCAST_WALK_WORDS and BCAST_WALK_BLOCKS_PER_SM override the choice (for experiments).
struct WalkShape {
    int u = 1, grid = 1;
    bool many_rounds = false;     // the bandwidth regime: one block per SM, several rounds of slices
};

int choose_shape(bool few_hops, const std::function<long long(int)> &slices_for, int P, int sm_count, WalkShape *shape)
{
    const int forced_u = env_int("BCAST_WALK_WORDS", 0);
    const int forced_bps = env_int("BCAST_WALK_BLOCKS_PER_SM", 0);
    const bool u_ok = forced_u >= 1 && forced_u <= kMaxWords;
    int rc, resident = 1, u = 0, bps = 0;
    if (u_ok || forced_bps > 0) {
        u = u_ok ? forced_u : kMaxWords;
        if ((rc = walk_blocks_per_sm(u, P, &resident))) return rc;
        bps = forced_bps > 0 ? std::min(forced_bps, resident) : resident;
    } else if (few_hops) {
        u = P <= 3 ? 6 : 2;
        if ((rc = walk_blocks_per_sm(u, P, &resident))) return rc;
        bps = resident;
    } else if (slices_for(kMaxWords) * 5 > (long long)sm_count * kWarpsPerBlock * 7) {   // > 1.4 rounds
        u = kMaxWords;
        bps = 1;
        shape->many_rounds = true;
    } else {
        for (int cand = 1; cand <= kMaxWords; cand++) {
            if ((rc = walk_blocks_per_sm(cand, P, &resident))) return rc;
            const long long slices = slices_for(cand);
            if (slices <= (long long)sm_count * resident * kWarpsPerBlock) {
                u = cand;
                bps = (int)std::max<long long>(1, (slices + (long long)sm_count * kWarpsPerBlock - 1) /
                                                      ((long long)sm_count * kWarpsPerBlock));
                break;
            }
        }
        if (!u) { u = kMaxWords; bps = 1; }
    }
    const long long slices = std::max<long long>(1, slices_for(u));
    shape->u = u;
    shape->grid = (int)std::min<long long>(slices, (long long)sm_count * std::max(1, bps));
    return BCAST_OK;
}

// In the bandwidth regime the eight warps of a block take eight neighbouring slices at a time (32 KiB
// of every destination buffer written by one SM at about the same time) when the hop lists are long:
// measured +1..3 % of the copy rate for P >= 24 (config 4: 0.936 -> 0.960), -1..5 % for P <= 16.
// BCAST_WALK_GROUP overrides (for experiments).
int walk_group_for(const WalkShape &shape, int P)
{
    return std::max(1, env_int("BCAST_WALK_GROUP", shape.many_rounds && P >= 24 ? kWarpsPerBlock : 1));
}

int choose_walk_shape(const bcast_plan_t &p, int sm_count, WalkShape *shape)
{
    return choose_shape(p.P <= 4, [&](int u) { return count_slices(p, 512ull * u, true, nullptr); }, p.P, sm_count, shape);
}

// Hop lists and dual lists, then the slices of the register walk for the chosen shape.
int build_walk_tables(const bcast_plan_t &p, bcast_device_state &ds)
{
    HopLists lists;
    whole_plan_hops(p, lists);
    WalkTables t;
    make_walk_tables(p, lists, t);
    int rc;
    if ((rc = upload(&ds.d_hops, t.hops))) return rc;
    if ((rc = upload(&ds.d_hops_plan, t.hops_plan))) return rc;
    if ((rc = upload(&ds.d_hop_msg, t.hop_msg))) return rc;
    if ((rc = upload(&ds.d_hop_msg_plan, t.hop_msg_plan))) return rc;
    if ((rc = upload(&ds.d_hop_begin, t.hop_begin))) return rc;
    if ((rc = upload(&ds.d_dual, t.dual))) return rc;
    if ((rc = upload(&ds.d_dual_msg, t.dual_msg))) return rc;
    if ((rc = upload(&ds.d_dual_begin, t.dual_begin))) return rc;

    WalkShape shape;
    if ((rc = choose_walk_shape(p, ds.sm_count, &shape))) return rc;
    ds.walk_u = shape.u;
    ds.walk_grid = shape.grid;
    std::vector<WalkSlice> slices;
    make_slices(p, 512ull * ds.walk_u, env_int("BCAST_WALK_DUAL", 1) != 0, nullptr, slices);
    ds.n_slices = (long long)slices.size();
    ds.walk_group = walk_group_for(shape, p.P);
    ds.walk_grouped = ds.n_slices / ((long long)ds.walk_group * ds.walk_grid) * ds.walk_group * ds.walk_grid;
    return upload(&ds.d_slices, slices);
}

int build_bulk_tables(const bcast_plan_t &p, bcast_device_state &ds)
{
    std::vector<WalkSlice> bulk, reg;
    make_bulk_slices(p, kBulkSeg, 512ull * kBulkRegWords, bulk, reg);
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
    for (bool trace : {false, true})
        CUDA_TRY(cudaFuncSetAttribute(bulk_kernel(p.P, trace), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, bulk_kernel(p.P, false), kBulkThreads, smem));
    const int bps = std::max(1, std::min(resident, env_int("BCAST_BULK_BLOCKS_PER_SM", 3)));
    const long long want = std::max<long long>(1, std::max((ds.n_bulk + kBulkWorkers - 1) / kBulkWorkers, ds.n_reg));
    ds.bulk_grid = (int)std::min<long long>(want, (long long)ds.sm_count * bps);
    ds.bulk_spin_limit = std::max(0, env_int("BCAST_BULK_SPIN_LIMIT", kBulkSpinLimit));
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

// ======================================================================================= checks
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

// Both checks, skipped when the pointers are the ones that passed them last time (the cache
// assumes that those buffers are still allocated).
int check_bufs(void *const *rank_bufs, const bcast_plan_t &p, bcast_device_state &ds)
{
    const size_t P = (size_t)p.P;
    std::lock_guard<std::mutex> lock(ds.mu);
    if (ds.checked_bufs.size() == P && std::memcmp(ds.checked_bufs.data(), rank_bufs, P * sizeof(void *)) == 0)
        return BCAST_OK;
    int rc = validate_bufs(rank_bufs, P, p.nbytes);
    if (!rc) rc = validate_device_memory(rank_bufs, P);
    if (rc) return rc;
    ds.checked_bufs.assign(rank_bufs, rank_bufs + P);
    return BCAST_OK;
}

// ======================================================================================= launches
WalkDev walk_dev(const bcast_plan_t &p, const bcast_device_state &ds, bool plan_order, const WalkSlice *slices,
                 long long n_slices, unsigned long long *trace)
{
    WalkDev w;
    w.slices = slices;
    w.n_slices = n_slices;
    w.hops = plan_order ? ds.d_hops_plan : ds.d_hops;
    w.hop_begin = ds.d_hop_begin;
    w.dual = ds.d_dual;
    w.dual_begin = ds.d_dual_begin;
    w.hop_msg = plan_order ? ds.d_hop_msg_plan : ds.d_hop_msg;
    w.dual_msg = ds.d_dual_msg;
    w.trace = trace;
    w.scatter_size = p.S;
    w.nbytes = p.nbytes;
    w.group = 1;
    w.grouped = 0;
    return w;
}

int launch_walk(const bcast_plan_t &p, const bcast_device_state &ds, void *const *rank_bufs, bool plan_order,
                cudaStream_t st, unsigned long long *trace)
{
    WalkDev w = walk_dev(p, ds, plan_order, ds.d_slices, ds.n_slices, trace);
    w.group = ds.walk_group;
    w.grouped = ds.walk_grouped;
    return launch_with_ptrs(walk_kernel(ds.walk_u, p.P, trace != nullptr), dim3(ds.walk_grid), dim3(kThreads), 0, st,
                            rank_bufs, p.P, trace != nullptr, {&w});
}

int launch_walk_bulk(const bcast_plan_t &p, const bcast_device_state &ds, void *const *rank_bufs, cudaStream_t st,
                     unsigned long long *trace)
{
    WalkDev w = walk_dev(p, ds, env_int("BCAST_BULK_PLAN_ORDER", 0) != 0, ds.d_reg_slices, ds.n_reg, trace);
    BulkDev b{ds.d_bulk_slices, ds.n_bulk, ds.bulk_spin_limit, ds.d_status};
    return launch_with_ptrs(bulk_kernel(p.P, trace != nullptr), dim3(ds.bulk_grid), dim3(kBulkThreads),
                            (size_t)kBulkWorkers * kBulkSeg, st, rank_bufs, p.P, trace != nullptr, {&w, &b});
}

int launch_steps(const bcast_plan_t &p, const bcast_device_state &ds, void *const *rank_bufs, cudaStream_t st,
                 unsigned long long *trace)
{
    for (const StepLaunch &sl : ds.steps) {
        if (!sl.tiles) continue;
        const DevXfer *x = ds.d_xfers + sl.first;
        long long first = sl.first;
        int rc = launch_with_ptrs(step_kernel(p.P, trace != nullptr), dim3(sl.tiles, sl.count), dim3(kThreads), 0, st,
                                  rank_bufs, p.P, trace != nullptr, {&x, &first, &trace});
        if (rc) return rc;
    }
    return BCAST_OK;
}

int launch_graph(const bcast_plan_t &p, bcast_device_state &ds, void *const *rank_bufs, cudaStream_t st)
{
    const int P = p.P;
    std::lock_guard<std::mutex> lock(ds.mu);
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
            rc = launch_steps(p, ds, rank_bufs, cap, nullptr);
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

bool known_mode(int mode)
{
    return mode == BCAST_EXEC_WALK || mode == BCAST_EXEC_STEPS || mode == BCAST_EXEC_GRAPH ||
           mode == BCAST_EXEC_WALK_PLAN_ORDER || mode == BCAST_EXEC_WALK_BULK || mode == BCAST_EXEC_AUTO;
}

// The bulk-copy walk needs ~4x the bytes in flight of the register walk.  With plan-order hops
// (native, doubling) a segment is re-read on the very next hop and that still fits in L2; with
// the tuned variant's level-order hops the re-read comes up to a tree level later and no longer
// does (measured: 20-25 % slower than the register walk), so the tuned variant stays with registers.
// For the others it pays only for very large messages on many ranks (measured: 128 MiB, P >= 128:
// 0.95-0.96 of the copy rate against 0.93-0.94; at 64 MiB, or with P <= 64, the register walk is as
// fast or faster): at least four rounds of its own (about 116 MB on 148 SMs) and P >= 64.
int resolve_auto(const bcast_plan_t &p, const bcast_device_state &ds)
{
    const bool bulk_pays = p.P >= 64 && ds.n_bulk >= 4ll * ds.bulk_grid * kBulkWorkers;
    return bulk_pays && p.variant != BCAST_TUNED ? BCAST_EXEC_WALK_BULK : BCAST_EXEC_WALK;
}

int exec_checked(void *const *rank_bufs, const bcast_plan_t *plan, void *cuda_stream, int mode, unsigned long long *trace)
{
    if (!rank_bufs || !plan || !known_mode(mode)) return BCAST_ERR_INVAL;
    if (trace && mode == BCAST_EXEC_GRAPH) return BCAST_ERR_INVAL;
    const bcast_plan_t &p = *plan;
    bcast_device_state *ds = nullptr;
    int rc = get_state(p, &ds);
    if (rc) return rc;
    try {
        rc = check_bufs(rank_bufs, p, *ds);
        if (rc) return rc;
        if (p.total_bytes == 0) return BCAST_OK;   // P = 1 or an empty message: nothing moves
        cudaStream_t st = (cudaStream_t)cuda_stream;
        if (mode == BCAST_EXEC_AUTO) mode = resolve_auto(p, *ds);
        switch (mode) {
        case BCAST_EXEC_WALK_BULK: return launch_walk_bulk(p, *ds, rank_bufs, st, trace);
        case BCAST_EXEC_WALK:
        case BCAST_EXEC_WALK_PLAN_ORDER: return launch_walk(p, *ds, rank_bufs, mode == BCAST_EXEC_WALK_PLAN_ORDER, st, trace);
        case BCAST_EXEC_STEPS: return launch_steps(p, *ds, rank_bufs, st, trace);
        default: return launch_graph(p, *ds, rank_bufs, st);
        }
    } catch (const std::bad_alloc &) {
        return BCAST_ERR_NOMEM;
    }
}

}  // namespace

// ======================================================================================= for shard.cpp
int bcast_internal_walk_shape(bool few_hops, const std::function<long long(int)> &slices_for, int P, int sm_count, int *u,
                              int *grid, int *group)
{
    WalkShape shape;
    const int rc = choose_shape(few_hops, slices_for, P, sm_count, &shape);
    *u = shape.u;
    *grid = shape.grid;
    *group = walk_group_for(shape, P);
    return rc;
}

int bcast_internal_launch_walk(const WalkDev &w, int u, int grid, void *const *rank_bufs, int P, void *cuda_stream)
{
    WalkDev copy = w;
    const bool trace = w.trace != nullptr;
    return launch_with_ptrs(walk_kernel(u, P, trace), dim3(grid), dim3(kThreads), 0, (cudaStream_t)cuda_stream, rank_bufs, P,
                            trace, {&copy});
}

int bcast_internal_validate_bufs(void *const *rank_bufs, size_t P, uint64_t nbytes) { return validate_bufs(rank_bufs, P, nbytes); }

int bcast_internal_cuda_failed(int cuda_error)
{
    t_last_cuda_error = cuda_error;
    return cuda_error == (int)cudaErrorMemoryAllocation ? BCAST_ERR_NOMEM : BCAST_ERR_CUDA;
}

// ======================================================================================= C ABI
extern "C" {

int bcast_exec_mode(void *const *rank_bufs, const bcast_plan_t *plan, void *cuda_stream, int mode)
{
    return exec_checked(rank_bufs, plan, cuda_stream, mode, nullptr);
}

int bcast_exec(void *const *rank_bufs, const bcast_plan_t *plan, void *cuda_stream)
{
    return exec_checked(rank_bufs, plan, cuda_stream, BCAST_EXEC_AUTO, nullptr);
}

int bcast_exec_traced(void *const *rank_bufs, const bcast_plan_t *plan, void *cuda_stream, int mode,
                      uint64_t *device_msg_bytes)
{
    if (!device_msg_bytes) return BCAST_ERR_INVAL;
    static_assert(sizeof(unsigned long long) == sizeof(uint64_t), "counter width");
    return exec_checked(rank_bufs, plan, cuda_stream, mode, (unsigned long long *)device_msg_bytes);
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

int64_t bcast_plan_walk_pairing(const bcast_plan_t *plan, int chunk, int64_t *out, int64_t cap)
{
    if (!plan || chunk < 0 || chunk + 1 >= plan->P || cap < 0 || (cap > 0 && !out)) return BCAST_ERR_INVAL;
    try {
        std::vector<std::vector<int64_t>> per_chunk;
        messages_by_chunk(*plan, per_chunk);
        if (per_chunk[chunk].empty() || per_chunk[chunk + 1].empty()) return 0;
        std::vector<DualMsg> slots;
        pair_hops(*plan, per_chunk[chunk], per_chunk[chunk + 1], slots);
        for (int64_t i = 0; i < (int64_t)slots.size() && i < cap; i++) {
            out[2 * i] = slots[i].a;
            out[2 * i + 1] = slots[i].b;
        }
        return (int64_t)slots.size();
    } catch (const std::bad_alloc &) {
        return BCAST_ERR_NOMEM;
    }
}

int64_t bcast_plan_walk_slices(const bcast_plan_t *plan, int words, int64_t *out, int64_t cap)
{
    if (!plan || words < 1 || words > kMaxWords || cap < 0 || (cap > 0 && !out)) return BCAST_ERR_INVAL;
    try {
        std::vector<WalkSlice> slices;
        if (plan->total_bytes) make_slices(*plan, 512ull * words, true, nullptr, slices);
        if ((long long)slices.size() != (plan->total_bytes ? count_slices(*plan, 512ull * words, true, nullptr) : 0))
            return BCAST_ERR_INVAL;                       // the two must agree: the launch shape relies on it
        for (int64_t i = 0; i < (int64_t)slices.size() && i < cap; i++) {
            out[3 * i] = slices[i].seg;
            out[3 * i + 1] = slices[i].ref >> kSliceKindShift;
            out[3 * i + 2] = slices[i].ref & kSliceRefMask;
        }
        return (int64_t)slices.size();
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

// Host image of the five tables the WALK kernel reads, laid out as they will sit in the scratch.
// Built on a plan's first bcast_exec_static call and kept in ordinary host memory with the plan.
struct bcast_static_image {
    std::vector<unsigned char> bytes;
    size_t off_dual_begin = 0, off_slices = 0, off_hops = 0, off_dual = 0;
    long long n_slices = 0;
    int u = 0, grid = 0, sm_count = 0, group = 1;
    long long grouped = 0;
};

void bcast_static_image_free(bcast_static_image *img) { delete img; }

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
unsigned char *g_static_addr[kMaxDevices] = {};   // device address of g_static_scratch, per device
int g_static_sms[kMaxDevices] = {};
std::vector<void *> g_static_checked[kMaxDevices];   // rank buffers that last passed the device-memory check, per device

inline size_t round256(size_t x) { return (x + 255) & ~(size_t)255; }

// Device address of the scratch on the current device; looked up on the first call per device.
int static_scratch(int device, unsigned char **addr, int *sm_count)
{
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

// Assemble the image: with the boundary (dual) lists if everything fits, else without them (cut
// segments then go as ragged slices), else with the largest slices; BCAST_ERR_CAPACITY if nothing fits.
int make_static_image(const bcast_plan_t &p, int sm_count, bcast_static_image &img)
{
    WalkShape shape;
    int rc = choose_walk_shape(p, sm_count, &shape);
    if (rc) return rc;
    HopLists lists;
    whole_plan_hops(p, lists);
    WalkTables t;
    make_walk_tables(p, lists, t);
    std::vector<WalkSlice> slices;
    for (int attempt = 0; attempt < 4; attempt++) {
        const bool use_dual = (attempt & 1) == 0;
        const int u = attempt < 2 ? shape.u : kMaxWords;
        if (attempt >= 2 && shape.u == kMaxWords) break;
        make_slices(p, 512ull * u, use_dual, nullptr, slices);
        const size_t dual_bytes = use_dual ? t.dual.size() * sizeof(DualSlot) : 0;
        img.off_dual_begin = round256(t.hop_begin.size() * sizeof(int));
        img.off_slices = img.off_dual_begin + round256(t.dual_begin.size() * sizeof(int));
        img.off_hops = img.off_slices + round256(slices.size() * sizeof(WalkSlice));
        img.off_dual = img.off_hops + round256(t.hops.size() * sizeof(uint32_t));
        const size_t total = img.off_dual + round256(dual_bytes);
        if (total > BCAST_STATIC_SCRATCH_BYTES) continue;
        img.bytes.assign(total, 0);
        std::memcpy(img.bytes.data(), t.hop_begin.data(), t.hop_begin.size() * sizeof(int));
        std::memcpy(img.bytes.data() + img.off_dual_begin, t.dual_begin.data(), t.dual_begin.size() * sizeof(int));
        std::memcpy(img.bytes.data() + img.off_slices, slices.data(), slices.size() * sizeof(WalkSlice));
        std::memcpy(img.bytes.data() + img.off_hops, t.hops.data(), t.hops.size() * sizeof(uint32_t));
        if (dual_bytes) std::memcpy(img.bytes.data() + img.off_dual, t.dual.data(), dual_bytes);
        img.n_slices = (long long)slices.size();
        img.u = u;
        img.grid = (int)std::max<long long>(1, std::min<long long>(shape.grid, img.n_slices));
        img.group = u == shape.u ? walk_group_for(shape, p.P) : 1;                            // as in build_walk_tables
        img.grouped = img.n_slices / ((long long)img.group * img.grid) * img.group * img.grid;
        img.sm_count = sm_count;
        return BCAST_OK;
    }
    return BCAST_ERR_CAPACITY;
}

int exec_static(void *const *rank_bufs, const bcast_plan_t &p, cudaStream_t st)
{
    int rc = validate_bufs(rank_bufs, (size_t)p.P, p.nbytes);
    if (rc) return rc;
    int device = -1;
    CUDA_TRY(cudaGetDevice(&device));
    if (device < 0 || device >= kMaxDevices) return BCAST_ERR_INVAL;
    // the copy into the scratch below must not become part of a captured graph: its source and the
    // one shared array would both be stale by the time the graph is replayed
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    CUDA_TRY(cudaStreamIsCapturing(st, &cap));
    if (cap != cudaStreamCaptureStatusNone) return BCAST_ERR_INVAL;

    std::lock_guard<std::mutex> lock(g_static_mu);
    // the device-memory check costs a driver call per buffer: remember the last set that passed
    std::vector<void *> &checked = g_static_checked[device];
    if (checked.size() != (size_t)p.P || std::memcmp(checked.data(), rank_bufs, (size_t)p.P * sizeof(void *)) != 0) {
        if ((rc = validate_device_memory(rank_bufs, (size_t)p.P))) return rc;
        checked.assign(rank_bufs, rank_bufs + p.P);
    }
    if (p.total_bytes == 0) return BCAST_OK;
    unsigned char *scratch = nullptr;
    int sms = 0;
    if ((rc = static_scratch(device, &scratch, &sms))) return rc;

    if (p.static_img && p.static_img->sm_count != sms) { delete p.static_img; p.static_img = nullptr; }
    if (!p.static_img) {
        bcast_static_image *img = new bcast_static_image();
        if ((rc = make_static_image(p, sms, *img))) { delete img; return rc; }
        p.static_img = img;
    }
    const bcast_static_image &img = *p.static_img;

    // one stream-ordered copy puts the tables in place.  The source is pageable host memory owned by
    // the plan: the runtime stages it before returning (which may wait for earlier work on the
    // stream).  Nothing in the array has to start at zero: the kernel only reads it.
    CUDA_TRY(cudaMemcpyAsync(scratch, img.bytes.data(), img.bytes.size(), cudaMemcpyHostToDevice, st));

    WalkDev w;
    w.slices = (const WalkSlice *)(scratch + img.off_slices);
    w.n_slices = img.n_slices;
    w.hops = (const uint32_t *)(scratch + img.off_hops);
    w.hop_begin = (const int *)scratch;
    w.dual = (const DualSlot *)(scratch + img.off_dual);
    w.dual_begin = (const int *)(scratch + img.off_dual_begin);
    w.hop_msg = nullptr;
    w.dual_msg = nullptr;
    w.trace = nullptr;
    w.scatter_size = p.S;
    w.nbytes = p.nbytes;
    w.group = img.group;
    w.grouped = img.grouped;
    return launch_with_ptrs(walk_kernel(img.u, p.P, false), dim3(img.grid), dim3(kThreads), 0, st, rank_bufs, p.P, false, {&w});
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
