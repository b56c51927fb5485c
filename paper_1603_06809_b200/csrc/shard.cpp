// The P virtual ranks of a plan spread over G GPUs (one NVSwitch domain): host-side partition of
// the plan and an executor that needs no waiting inside any kernel.
//
// Every rank's buffer lives in the memory of the GPU that owns the rank.  A message is performed by
// the GPU that owns its DESTINATION: that GPU's kernel loads from the source rank's buffer (its own
// memory, or a peer's through an ordinary peer load) and stores into its own memory, so whatever
// crosses NVLink lands in local memory before anything re-reads it.  Per byte column the messages
// still form the chains and trees of Sections III-A and IV; a chain only leaves a GPU where the
// ring passes from the last rank of one group to the first rank of the next.
//
// Phases.  For every (message, chunk) pair -- a hop of that chunk's byte columns -- the phase is
//     phase(hop) = phase(the hop that wrote the source copy) + (1 if source and destination are
//                  on different GPUs else 0),   the root's own data having phase 0.
// So a hop of phase k reads either something written by its own GPU in a phase <= k (ordered by
// the stream, and inside one kernel by each thread's program order, as in the one-GPU walk) or
// something written by another GPU in phase k-1.  Running phase after phase, with every GPU's
// phase-k kernel ordered after all phase-(k-1) kernels (CUDA events between the GPUs' streams, or
// a host barrier between processes), honours every dependency of the plan.  With contiguous rank
// groups the ring has about G phases, and in each of them every GPU walks about P/G hops of the
// chunks that are passing through it.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstring>
#include <new>
#include <vector>

#include "exec_internal.h"
#include "plan_internal.h"
#include "walk_tables.h"

namespace {

#define SHARD_TRY(expr)                                                    \
    do {                                                                   \
        cudaError_t e_ = (expr);                                           \
        if (e_ != cudaSuccess) return bcast_internal_cuda_failed((int)e_); \
    } while (0)

struct ShardKernel {               // one (phase, gpu) launch
    HopLists lists;                // per chunk: the hops of this phase whose destination the GPU owns
    std::vector<char> active;      // per chunk: any hop here?
    bool any = false;
    // device side (on the GPU's device), built at the first execution
    bool built = false;
    int u = 0, grid = 0, group = 1;
    long long n_slices = 0, grouped = 0;
    WalkSlice *d_slices = nullptr;
    uint32_t *d_hops = nullptr;
    int32_t *d_hop_msg = nullptr;
    int *d_hop_begin = nullptr, *d_dual_begin = nullptr;
    DualSlot *d_dual = nullptr;
    DualMsg *d_dual_msg = nullptr;
    cudaEvent_t done = nullptr;
};

template <typename T>
int upload(T **d_ptr, const std::vector<T> &h)
{
    const size_t bytes = std::max<size_t>(h.size(), 1) * sizeof(T);
    SHARD_TRY(cudaMalloc((void **)d_ptr, bytes));
    if (!h.empty()) SHARD_TRY(cudaMemcpy(*d_ptr, h.data(), h.size() * sizeof(T), cudaMemcpyHostToDevice));
    return BCAST_OK;
}

}  // namespace

struct bcast_shard {
    const bcast_plan_t *plan = nullptr;
    int G = 0, n_phases = 0;
    std::vector<int32_t> rank_gpu;                 // [P]
    std::vector<int32_t> msg_phase_first, msg_phase_last;   // [num_xfers]: phases of a message's hops (one per chunk it carries)
    std::vector<int32_t> msg_gpu;                  // [num_xfers]: the GPU that performs the message (owner of dst_rank)
    std::vector<ShardKernel> kernels;              // [n_phases * G]
    uint64_t crossing_bytes = 0;
    int64_t crossing_msgs = 0;
    std::vector<int> devices;                      // CUDA device of every GPU of the partition, fixed at the first execution
    ShardKernel &at(int phase, int gpu) { return kernels[(size_t)phase * G + gpu]; }
};

namespace {

void partition(bcast_shard &sh)
{
    const bcast_plan_t &p = *sh.plan;
    const int P = p.P, G = sh.G;
    const size_t nx = p.xfers.size();
    sh.msg_phase_first.assign(nx, -1);
    sh.msg_phase_last.assign(nx, -1);
    sh.msg_gpu.assign(nx, 0);
    for (size_t i = 0; i < nx; i++) {
        const bcast_xfer_t &x = p.xfers[i];
        sh.msg_gpu[i] = sh.rank_gpu[x.dst_rank];
        if (sh.rank_gpu[x.src_rank] != sh.rank_gpu[x.dst_rank]) {
            sh.crossing_bytes += x.len;
            sh.crossing_msgs += 1;
        }
    }
    HopLists whole;
    whole_plan_hops(p, whole);
    // phase of every hop, chunk by chunk, following the chunk's messages in plan order
    std::vector<std::vector<int32_t>> hop_phase(P);          // parallel to whole.plan_order[c]
    std::vector<int32_t> at_rank(P), of_msg(nx, -1);
    int max_phase = -1;
    for (int c = 0; c < P; c++) {
        std::fill(at_rank.begin(), at_rank.end(), -1);
        at_rank[p.root] = 0;
        hop_phase[c].resize(whole.plan_order[c].size());
        for (size_t h = 0; h < whole.plan_order[c].size(); h++) {
            const int64_t m = whole.plan_order[c][h];
            const bcast_xfer_t &x = p.xfers[m];
            const int32_t from = at_rank[x.src_rank] < 0 ? 0 : at_rank[x.src_rank];   // (a valid plan never sends what is not there)
            const int32_t ph = from + (sh.rank_gpu[x.src_rank] != sh.rank_gpu[x.dst_rank] ? 1 : 0);
            hop_phase[c][h] = ph;
            at_rank[x.dst_rank] = ph;
            max_phase = std::max(max_phase, (int)ph);
            if (sh.msg_phase_first[m] < 0 || ph < sh.msg_phase_first[m]) sh.msg_phase_first[m] = ph;
            sh.msg_phase_last[m] = std::max(sh.msg_phase_last[m], ph);
        }
    }
    sh.n_phases = max_phase + 1;
    sh.kernels.assign((size_t)sh.n_phases * G, ShardKernel());
    for (ShardKernel &k : sh.kernels) {
        k.lists.plan_order.assign(P, {});
        k.lists.walk_order.assign(P, {});
        k.active.assign(P, 0);
    }
    for (int c = 0; c < P; c++) {
        for (size_t h = 0; h < whole.plan_order[c].size(); h++) {
            const int64_t m = whole.plan_order[c][h];
            of_msg[m] = hop_phase[c][h];
            ShardKernel &k = sh.at(hop_phase[c][h], sh.msg_gpu[m]);
            k.lists.plan_order[c].push_back(m);
            k.active[c] = 1;
            k.any = true;
        }
        // the same hops in the order the one-GPU walk takes them (a filtered valid order is valid)
        for (int64_t m : whole.walk_order[c]) sh.at(of_msg[m], sh.msg_gpu[m]).lists.walk_order[c].push_back(m);
    }
}

void free_kernel(ShardKernel &k)
{
    cudaFree(k.d_slices);
    cudaFree(k.d_hops);
    cudaFree(k.d_hop_msg);
    cudaFree(k.d_hop_begin);
    cudaFree(k.d_dual_begin);
    cudaFree(k.d_dual);
    cudaFree(k.d_dual_msg);
    if (k.done) cudaEventDestroy(k.done);
    k = ShardKernel();
}

// Device tables and launch shape of one (phase, gpu) kernel, on the current device.
int build_kernel(const bcast_plan_t &p, ShardKernel &k)
{
    int device = -1, sms = 0;
    SHARD_TRY(cudaGetDevice(&device));
    SHARD_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    WalkTables t;
    make_walk_tables(p, k.lists, t);
    int rc = bcast_internal_walk_shape(false, [&](int u) { return count_slices(p, 512ull * u, true, &k.active); }, p.P, sms,
                                       &k.u, &k.grid, &k.group);
    if (rc) return rc;
    std::vector<WalkSlice> slices;
    make_slices(p, 512ull * k.u, true, &k.active, slices);
    k.n_slices = (long long)slices.size();
    k.grouped = k.n_slices / ((long long)k.group * k.grid) * k.group * k.grid;
    if ((rc = upload(&k.d_slices, slices))) return rc;
    if ((rc = upload(&k.d_hops, t.hops))) return rc;
    if ((rc = upload(&k.d_hop_msg, t.hop_msg))) return rc;
    if ((rc = upload(&k.d_hop_begin, t.hop_begin))) return rc;
    if ((rc = upload(&k.d_dual, t.dual))) return rc;
    if ((rc = upload(&k.d_dual_msg, t.dual_msg))) return rc;
    if ((rc = upload(&k.d_dual_begin, t.dual_begin))) return rc;
    SHARD_TRY(cudaEventCreateWithFlags(&k.done, cudaEventDisableTiming));
    k.built = true;
    return BCAST_OK;
}

int launch_kernel(const bcast_plan_t &p, ShardKernel &k, void *const *rank_bufs, cudaStream_t st, unsigned long long *trace)
{
    if (!k.built) {
        const int rc = build_kernel(p, k);
        if (rc) return rc;
    }
    WalkDev w;
    w.slices = k.d_slices;
    w.n_slices = k.n_slices;
    w.hops = k.d_hops;
    w.hop_begin = k.d_hop_begin;
    w.dual = k.d_dual;
    w.dual_begin = k.d_dual_begin;
    w.hop_msg = k.d_hop_msg;
    w.dual_msg = k.d_dual_msg;
    w.trace = trace;
    w.scatter_size = p.S;
    w.nbytes = p.nbytes;
    w.group = k.group;
    w.grouped = k.grouped;
    return bcast_internal_launch_walk(w, k.u, k.grid, rank_bufs, p.P, st);
}

// Every rank buffer must be device (or managed) memory of the device that its owner GPU is mapped to.
int check_placement(const bcast_shard &sh, void *const *rank_bufs, const int *devices)
{
    for (int r = 0; r < sh.plan->P; r++) {
        cudaPointerAttributes attr;
        if (cudaPointerGetAttributes(&attr, rank_bufs[r]) != cudaSuccess) {
            cudaGetLastError();
            return BCAST_ERR_INVAL;
        }
        if (attr.type == cudaMemoryTypeManaged) continue;
        if (attr.type != cudaMemoryTypeDevice || attr.device != devices[sh.rank_gpu[r]]) return BCAST_ERR_INVAL;
    }
    return BCAST_OK;
}

// Every device of the partition must be able to load from every other one's memory: enable peer
// access where it is not enabled yet (one process driving all GPUs; with one process per GPU the
// IPC mappings the caller opens do this).
int enable_peer_access(const int *devices, int G)
{
    int cur = -1;
    SHARD_TRY(cudaGetDevice(&cur));
    for (int a = 0; a < G; a++)
        for (int b = 0; b < G; b++) {
            if (devices[a] == devices[b]) continue;
            int can = 0;
            SHARD_TRY(cudaDeviceCanAccessPeer(&can, devices[a], devices[b]));
            if (!can) { cudaSetDevice(cur); return BCAST_ERR_INVAL; }
            SHARD_TRY(cudaSetDevice(devices[a]));
            const cudaError_t e = cudaDeviceEnablePeerAccess(devices[b], 0);
            if (e == cudaErrorPeerAccessAlreadyEnabled) cudaGetLastError();      // fine: clear it
            else if (e != cudaSuccess) { cudaSetDevice(cur); return bcast_internal_cuda_failed((int)e); }
        }
    SHARD_TRY(cudaSetDevice(cur));
    return BCAST_OK;
}

int fix_devices(bcast_shard &sh, const int *devices)
{
    if (sh.devices.empty()) {
        const int rc = enable_peer_access(devices, sh.G);
        if (rc) return rc;
        sh.devices.assign(devices, devices + sh.G);
        return BCAST_OK;
    }
    return std::memcmp(sh.devices.data(), devices, sizeof(int) * (size_t)sh.G) == 0 ? BCAST_OK : BCAST_ERR_INVAL;
}

}  // namespace

extern "C" {

int bcast_shard_create(const bcast_plan_t *plan, int num_gpus, const int32_t *rank_gpu, bcast_shard_t **out)
{
    if (!out) return BCAST_ERR_INVAL;
    *out = nullptr;
    if (!plan || num_gpus < 1 || num_gpus > plan->P) return BCAST_ERR_INVAL;
    bcast_shard *sh = nullptr;
    try {
        sh = new bcast_shard();
        sh->plan = plan;
        sh->G = num_gpus;
        sh->rank_gpu.resize(plan->P);
        for (int r = 0; r < plan->P; r++) {
            const int32_t g = rank_gpu ? rank_gpu[r] : (int32_t)((int64_t)r * num_gpus / plan->P);   // contiguous groups
            if (g < 0 || g >= num_gpus) { delete sh; return BCAST_ERR_INVAL; }
            sh->rank_gpu[r] = g;
        }
        partition(*sh);
    } catch (const std::bad_alloc &) {
        delete sh;
        return BCAST_ERR_NOMEM;
    }
    *out = sh;
    return BCAST_OK;
}

void bcast_shard_free(bcast_shard_t *shard)
{
    if (!shard) return;
    int cur = -1;
    const bool have = cudaGetDevice(&cur) == cudaSuccess;
    for (int k = 0; k < shard->n_phases; k++)
        for (int g = 0; g < shard->G; g++) {
            ShardKernel &sk = shard->at(k, g);
            if (!sk.built) continue;
            if (!shard->devices.empty()) cudaSetDevice(shard->devices[g]);
            free_kernel(sk);
        }
    if (have) cudaSetDevice(cur);
    delete shard;
}

int32_t bcast_shard_num_gpus(const bcast_shard_t *s) { return s ? s->G : 0; }
int32_t bcast_shard_num_phases(const bcast_shard_t *s) { return s ? s->n_phases : 0; }
const int32_t *bcast_shard_rank_gpu(const bcast_shard_t *s) { return s ? s->rank_gpu.data() : nullptr; }
const int32_t *bcast_shard_msg_gpu(const bcast_shard_t *s) { return s ? s->msg_gpu.data() : nullptr; }
const int32_t *bcast_shard_msg_phase(const bcast_shard_t *s, int last)
{
    return s ? (last ? s->msg_phase_last.data() : s->msg_phase_first.data()) : nullptr;
}
uint64_t bcast_shard_crossing_bytes(const bcast_shard_t *s) { return s ? s->crossing_bytes : 0; }
int64_t bcast_shard_crossing_msgs(const bcast_shard_t *s) { return s ? s->crossing_msgs : 0; }

int64_t bcast_shard_hops(const bcast_shard_t *s, int phase, int gpu, int chunk, int64_t *out, int64_t cap)
{
    if (!s || phase < 0 || phase >= s->n_phases || gpu < 0 || gpu >= s->G || chunk < 0 || chunk >= s->plan->P || cap < 0 ||
        (cap > 0 && !out))
        return BCAST_ERR_INVAL;
    const std::vector<int64_t> &l = s->kernels[(size_t)phase * s->G + gpu].lists.walk_order[chunk];
    for (int64_t i = 0; i < (int64_t)l.size() && i < cap; i++) out[i] = l[i];
    return (int64_t)l.size();
}

int bcast_shard_exec_phase(bcast_shard_t *shard, void *const *rank_bufs, int phase, int gpu, void *cuda_stream,
                           uint64_t *device_msg_bytes)
{
    if (!shard || !rank_bufs || phase < 0 || phase >= shard->n_phases || gpu < 0 || gpu >= shard->G) return BCAST_ERR_INVAL;
    const bcast_plan_t &p = *shard->plan;
    try {
        int rc = bcast_internal_validate_bufs(rank_bufs, (size_t)p.P, p.nbytes);
        if (rc) return rc;
        ShardKernel &k = shard->at(phase, gpu);
        if (!k.any || p.total_bytes == 0) return BCAST_OK;
        return launch_kernel(p, k, rank_bufs, (cudaStream_t)cuda_stream, (unsigned long long *)device_msg_bytes);
    } catch (const std::bad_alloc &) {
        return BCAST_ERR_NOMEM;
    }
}

int bcast_shard_exec(bcast_shard_t *shard, void *const *rank_bufs, const int *gpu_device, void *const *cuda_streams,
                     uint64_t *device_msg_bytes)
{
    if (!shard || !rank_bufs || !gpu_device || !cuda_streams) return BCAST_ERR_INVAL;
    const bcast_plan_t &p = *shard->plan;
    const int G = shard->G;
    int cur = -1;
    SHARD_TRY(cudaGetDevice(&cur));
    int rc = BCAST_OK;
    try {
        if ((rc = bcast_internal_validate_bufs(rank_bufs, (size_t)p.P, p.nbytes))) return rc;
        if ((rc = check_placement(*shard, rank_bufs, gpu_device))) return rc;
        if ((rc = fix_devices(*shard, gpu_device))) return rc;
        if (p.total_bytes == 0) return BCAST_OK;
        // a previous execution of this partition may still be running on the other GPUs' streams:
        // nothing of this one starts on a GPU before all of that has finished
        for (int g = 0; g < G && !rc; g++)
            for (int o = 0; o < G && !rc; o++) {
                if (o == g) continue;
                for (int ph = shard->n_phases - 1; ph >= 0; ph--) {
                    ShardKernel &last = shard->at(ph, o);
                    if (!last.built) continue;
                    cudaError_t e = cudaSetDevice(gpu_device[g]);
                    if (e == cudaSuccess) e = cudaStreamWaitEvent((cudaStream_t)cuda_streams[g], last.done, 0);
                    if (e != cudaSuccess) rc = bcast_internal_cuda_failed((int)e);
                    break;
                }
            }
        for (int ph = 0; ph < shard->n_phases && !rc; ph++)
            for (int g = 0; g < G && !rc; g++) {
                ShardKernel &k = shard->at(ph, g);
                if (!k.any) continue;
                cudaError_t e = cudaSetDevice(gpu_device[g]);
                if (e != cudaSuccess) { rc = bcast_internal_cuda_failed((int)e); break; }
                cudaStream_t st = (cudaStream_t)cuda_streams[g];
                // everything another GPU wrote in the previous phase must have landed
                for (int o = 0; o < G && ph > 0 && !rc; o++) {
                    ShardKernel &prev = shard->at(ph - 1, o);
                    if (o == g || !prev.any || !prev.done) continue;
                    e = cudaStreamWaitEvent(st, prev.done, 0);
                    if (e != cudaSuccess) rc = bcast_internal_cuda_failed((int)e);
                }
                if (!rc) rc = launch_kernel(p, k, rank_bufs, st, (unsigned long long *)device_msg_bytes);
                if (!rc) {
                    e = cudaEventRecord(k.done, st);
                    if (e != cudaSuccess) rc = bcast_internal_cuda_failed((int)e);
                }
            }
    } catch (const std::bad_alloc &) {
        rc = BCAST_ERR_NOMEM;
    }
    cudaSetDevice(cur);
    return rc;
}

}  // extern "C"
