// Host-side planner: the control flow of the scatter-ring-allgather broadcast turned into data.
//
// The schedule is derived from the closed form of the binomial tree rather than by running the
// per-process loops of the paper's listing: relative rank r >= 1 roots a sub-tree of
//     s(r) = min(lowbit(r), P - r)        (lowbit = largest power of two dividing r)
// chunks, receives the byte range of chunks [r, r + s(r)) from relative rank r - lowbit(r) in the
// scatter (Section III-A, Figs. 1-2), and in ring step i receives chunk (r - i) mod P from its
// left neighbour (Section III-A, Fig. 3).  The tuned ring (Section IV) keeps exactly the receives
// of chunks outside [r, r + s(r)), i.e. steps i <= P - s(r); the root (s = P) never receives.
// The recursive-doubling variant (Section I; power-of-two P) replaces the ring by log2 P exchanges:
// in exchange i relative rank r receives from r xor 2^i the block of 2^i chunks that starts at the
// partner's rank with its low i bits cleared.
#include <algorithm>
#include <new>

#include "plan_internal.h"

namespace {

inline int lowbit(int x) { return x & -x; }

struct Geometry {
    int P, root;
    uint64_t n, S;
    int abs_rank(int r) const { return (r + root) % P; }
    int rel_rank(int k) const { return (k - root + P) % P; }
    uint64_t chunk_begin(int c) const { return std::min<uint64_t>((uint64_t)c * S, n); }   // c in [0, P]
    int subtree(int r) const { return r == 0 ? P : std::min(lowbit(r), P - r); }
};

void count(bcast_plan_t &p, const bcast_xfer_t &x)
{
    p.bytes_sent[x.phase][x.src_rank] += x.len;
    p.bytes_recv[x.phase][x.dst_rank] += x.len;
    p.msgs_sent[x.phase][x.src_rank] += 1;
    p.msgs_recv[x.phase][x.dst_rank] += 1;
    p.total_bytes += x.len;
}

void build(bcast_plan_t &p)
{
    const Geometry g{p.P, p.root, p.nbytes, p.S};
    const int P = p.P;
    for (int ph = 0; ph < 2; ph++) {
        p.bytes_sent[ph].assign(P, 0); p.bytes_recv[ph].assign(P, 0);
        p.msgs_sent[ph].assign(P, 0);  p.msgs_recv[ph].assign(P, 0);
    }
    p.L = 0;
    while ((1 << p.L) < P) p.L++;
    const bool doubling = p.variant == BCAST_DOUBLING;
    const int nsteps = P > 1 ? p.L + (doubling ? p.L : P - 1) : 0;
    p.step_begin.assign(nsteps + 1, 0);
    if (P == 1) return;

    size_t ring_msgs = doubling ? (size_t)P * p.L : (size_t)P * (P - 1);
    if (p.variant == BCAST_TUNED) {
        ring_msgs = (size_t)P * P;
        for (int r = 0; r < P; r++) ring_msgs -= g.subtree(r);
    }
    p.xfers.reserve((size_t)(P - 1) + ring_msgs);

    // delivered[r]: index of the message that brought relative rank r its scatter range (-1: root)
    std::vector<int64_t> delivered(P, -1);

    // ---- scatter: the message into relative rank r happens at the level whose mask is lowbit(r)
    for (int t = 0; t < p.L; t++) {
        const int mask = 1 << (p.L - 1 - t);
        p.step_begin[t] = (int64_t)p.xfers.size();
        // receivers of this level are the odd multiples of mask; list them by absolute rank
        for (int k = 0; k < P; k++) {
            const int r = g.rel_rank(k);
            if (r == 0 || lowbit(r) != mask) continue;
            bcast_xfer_t x{};
            x.phase = BCAST_PHASE_SCATTER;
            x.step = t;
            x.src_rank = g.abs_rank(r - mask);
            x.dst_rank = k;
            x.chunk = r;
            x.nchunks = g.subtree(r);
            x.offset = g.chunk_begin(r);
            x.len = g.chunk_begin(r + x.nchunks) - x.offset;
            x.dep = delivered[r - mask];
            delivered[r] = (int64_t)p.xfers.size();
            count(p, x);
            p.xfers.push_back(x);
        }
    }

    if (doubling) {
        // ---- recursive doubling: exchange i, receiver r takes the block of 2^i chunks from r xor 2^i
        std::vector<std::vector<int64_t>> into(p.L, std::vector<int64_t>(P, -1));   // [exchange][relative rank]
        for (int i = 0; i < p.L; i++) {
            const int mask = 1 << i;
            p.step_begin[p.L + i] = (int64_t)p.xfers.size();
            for (int k = 0; k < P; k++) {
                const int r = g.rel_rank(k), q = r ^ mask;     // receiver, sender (relative)
                const int block = (q >> i) << i;
                bcast_xfer_t x{};
                x.phase = BCAST_PHASE_RING;
                x.step = i;
                x.src_rank = g.abs_rank(q);
                x.dst_rank = k;
                x.chunk = block;
                x.nchunks = mask;
                x.offset = g.chunk_begin(block);
                x.len = g.chunk_begin(block + mask) - x.offset;
                // who last wrote the block's first chunk into the sender: the exchange that brought it
                // the sub-block starting there (the highest set bit of q below bit i), else the scatter
                const int low = q & (mask - 1);
                if (low == 0) {
                    x.dep = delivered[q];
                } else {
                    int j = 0;
                    while ((2 << j) <= low) j++;
                    x.dep = into[j][q];
                }
                into[i][r] = (int64_t)p.xfers.size();
                count(p, x);
                p.xfers.push_back(x);
            }
        }
        p.step_begin[nsteps] = (int64_t)p.xfers.size();
        return;
    }

    // ---- ring: step i, receiver r takes chunk (r - i) mod P from r - 1
    std::vector<int64_t> prev(P, -1), cur(P, -1);   // index of the ring message into r in step i-1 / i
    for (int i = 1; i < P; i++) {
        p.step_begin[p.L + i - 1] = (int64_t)p.xfers.size();
        std::fill(cur.begin(), cur.end(), (int64_t)-1);
        for (int k = 0; k < P; k++) {
            const int r = g.rel_rank(k);
            if (p.variant == BCAST_TUNED && i > P - g.subtree(r)) continue;   // r already holds that chunk
            const int q = (r - 1 + P) % P;                                     // sender, relative
            const int c = ((r - i) % P + P) % P;
            bcast_xfer_t x{};
            x.phase = BCAST_PHASE_RING;
            x.step = i - 1;
            x.src_rank = g.abs_rank(q);
            x.dst_rank = k;
            x.chunk = c;
            x.nchunks = 1;
            x.offset = g.chunk_begin(c);
            x.len = g.chunk_begin(c + 1) - x.offset;
            // the sender forwards what reached it in the previous ring step; if nothing did (first
            // step, or the sender had stopped receiving) it holds the chunk from the scatter
            x.dep = (i >= 2 && prev[q] >= 0) ? prev[q] : delivered[q];
            cur[r] = (int64_t)p.xfers.size();
            count(p, x);
            p.xfers.push_back(x);
        }
        std::swap(prev, cur);
    }
    p.step_begin[nsteps] = (int64_t)p.xfers.size();
}

}  // namespace

extern "C" {

int bcast_plan(int P, int root, uint64_t nbytes, int variant, bcast_plan_t **out)
{
    if (!out) return BCAST_ERR_INVAL;
    *out = nullptr;
    if (P < 1 || P > BCAST_MAX_RANKS || root < 0 || root >= P) return BCAST_ERR_INVAL;
    if (variant != BCAST_NATIVE && variant != BCAST_TUNED && variant != BCAST_DOUBLING) return BCAST_ERR_INVAL;
    if (variant == BCAST_DOUBLING && (P & (P - 1)) != 0) return BCAST_ERR_INVAL;
    if (nbytes > (UINT64_MAX >> 1) - (uint64_t)P) return BCAST_ERR_INVAL;
    bcast_plan_t *p = nullptr;
    try {
        p = new bcast_plan_t();
        p->P = P; p->root = root; p->variant = variant; p->nbytes = nbytes;
        p->S = (nbytes + (uint64_t)P - 1) / (uint64_t)P;
        build(*p);
    } catch (const std::bad_alloc &) {
        delete p;
        return BCAST_ERR_NOMEM;
    }
    *out = p;
    return BCAST_OK;
}

void bcast_plan_free(bcast_plan_t *plan)
{
    if (!plan) return;
    bcast_device_state_free(plan->dev);
    bcast_static_image_free(plan->static_img);
    delete plan;
}

int32_t bcast_plan_num_ranks(const bcast_plan_t *p) { return p ? p->P : 0; }
int32_t bcast_plan_root(const bcast_plan_t *p) { return p ? p->root : 0; }
int32_t bcast_plan_variant(const bcast_plan_t *p) { return p ? p->variant : 0; }
uint64_t bcast_plan_nbytes(const bcast_plan_t *p) { return p ? p->nbytes : 0; }
uint64_t bcast_plan_scatter_size(const bcast_plan_t *p) { return p ? p->S : 0; }
int64_t bcast_plan_num_xfers(const bcast_plan_t *p) { return p ? (int64_t)p->xfers.size() : 0; }
int32_t bcast_plan_num_steps(const bcast_plan_t *p) { return p ? (int32_t)p->step_begin.size() - 1 : 0; }
const bcast_xfer_t *bcast_plan_xfers(const bcast_plan_t *p) { return p ? p->xfers.data() : nullptr; }
const int64_t *bcast_plan_step_begin(const bcast_plan_t *p) { return p ? p->step_begin.data() : nullptr; }
uint64_t bcast_plan_total_bytes(const bcast_plan_t *p) { return p ? p->total_bytes : 0; }

#define BCAST_COUNTER_VIEW(name)                                                     \
    const uint64_t *bcast_plan_##name(const bcast_plan_t *p, int phase)              \
    {                                                                                \
        if (!p || (phase != BCAST_PHASE_SCATTER && phase != BCAST_PHASE_RING)) return nullptr; \
        return p->name[phase].data();                                                \
    }
BCAST_COUNTER_VIEW(bytes_sent)
BCAST_COUNTER_VIEW(bytes_recv)
BCAST_COUNTER_VIEW(msgs_sent)
BCAST_COUNTER_VIEW(msgs_recv)
#undef BCAST_COUNTER_VIEW

const char *bcast_strerror(int code)
{
    switch (code) {
    case BCAST_OK: return "success";
    case BCAST_ERR_INVAL: return "invalid argument";
    case BCAST_ERR_NOMEM: return "out of memory";
    case BCAST_ERR_CUDA: return "CUDA runtime error";
    case BCAST_ERR_CAPACITY: return "plan tables exceed the built-in scratch of bcast_exec_static";
    case BCAST_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
    default: return "unknown error code";
    }
}

}  // extern "C"
