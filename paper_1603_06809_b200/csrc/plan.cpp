// Host-side planner: the control flow of the scatter-ring-allgather broadcast turned into data.
//
// The schedule is derived from the closed form of the binomial tree rather than by running the
// per-process loops of the paper's listing: relative rank r >= 1 roots a sub-tree of
//     s(r) = min(lowbit(r), P - r)        (lowbit = largest power of two dividing r)
// chunks, receives the byte range of chunks [r, r + s(r)) from relative rank r - lowbit(r) in the
// scatter (Section III-A, Figs. 1-2), and in ring step i receives chunk (r - i) mod P from its
// left neighbour (Section III-A, Fig. 3).  The tuned ring (Section IV) keeps exactly the receives
// of chunks outside [r, r + s(r)), i.e. steps i <= P - s(r); the root (s = P) never receives.
// The node-aware broadcast (Section II) wraps the same scatter + ring, run between the node leaders,
// into two rounds of binomial-tree broadcasts inside the nodes.
// The recursive-doubling variant (Section I; power-of-two P) replaces the ring by log2 P exchanges:
// in exchange i relative rank r receives from r xor 2^i the block of 2^i chunks that starts at the
// partner's rank with its low i bits cleared.
#include <algorithm>
#include <new>

#include "plan_internal.h"

namespace {

inline int lowbit(int x) { return x & -x; }
inline int levels_of(int size) { int L = 0; while ((1 << L) < size) L++; return L; }

// The processes that run a scatter + allgather: all P ranks (relative rank r = absolute rank
// (r + root) mod P), or the node leaders of the node-aware broadcast (Section II).
struct Group {
    int size = 0;
    std::vector<int> abs_of_rel;      // [size]
    std::vector<int> rel_of_abs;      // [P], -1 for ranks outside the group
    int subtree(int r) const { return r == 0 ? size : std::min(lowbit(r), size - r); }
};

struct Builder {
    bcast_plan_t &p;
    std::vector<int64_t> writer0;     // per absolute rank: the message that last wrote chunk 0 there (-1: none)
    explicit Builder(bcast_plan_t &plan) : p(plan), writer0(plan.P, -1) {}

    uint64_t chunk_begin(int c) const { return std::min<uint64_t>((uint64_t)c * p.S, p.nbytes); }   // c in [0, chunks]

    void emit(bcast_xfer_t x)
    {
        x.offset = chunk_begin(x.chunk);
        x.len = chunk_begin(x.chunk + x.nchunks) - x.offset;
        p.bytes_sent[x.phase][x.src_rank] += x.len;
        p.bytes_recv[x.phase][x.dst_rank] += x.len;
        p.msgs_sent[x.phase][x.src_rank] += 1;
        p.msgs_recv[x.phase][x.dst_rank] += 1;
        p.total_bytes += x.len;
        if (x.chunk == 0) writer0[x.dst_rank] = (int64_t)p.xfers.size();
        p.xfers.push_back(x);
    }

    void begin_step() { p.step_begin.push_back((int64_t)p.xfers.size()); }

    // Scatter down the binomial tree of the group (Section III-A, Figs. 1-2): the message into
    // relative rank r happens at the level whose mask is lowbit(r).  delivered[r]: index of the
    // message that brought relative rank r what it sends on (on entry: [0] for the group's root).
    void scatter(const Group &g, std::vector<int64_t> &delivered)
    {
        const int L = levels_of(g.size);
        for (int t = 0; t < L; t++) {
            const int mask = 1 << (L - 1 - t);
            begin_step();
            // receivers of this level are the odd multiples of mask; list them by absolute rank
            for (int k = 0; k < p.P; k++) {
                const int r = g.rel_of_abs[k];
                if (r <= 0 || lowbit(r) != mask) continue;
                bcast_xfer_t x{};
                x.phase = BCAST_PHASE_SCATTER;
                x.step = t;
                x.src_rank = g.abs_of_rel[r - mask];
                x.dst_rank = k;
                x.chunk = r;
                x.nchunks = g.subtree(r);
                x.dep = delivered[r - mask];
                delivered[r] = (int64_t)p.xfers.size();
                emit(x);
            }
        }
    }

    // Ring allgather (Section III-A Fig. 3; tuned: Section IV): step i, receiver r takes chunk
    // (r - i) mod size from r - 1; the tuned ring keeps the receives of chunks outside [r, r + s(r)).
    void ring(const Group &g, bool tuned, const std::vector<int64_t> &delivered)
    {
        const int n = g.size;
        std::vector<int64_t> prev(n, -1), cur(n, -1);   // index of the ring message into r in step i-1 / i
        for (int i = 1; i < n; i++) {
            begin_step();
            std::fill(cur.begin(), cur.end(), (int64_t)-1);
            for (int k = 0; k < p.P; k++) {
                const int r = g.rel_of_abs[k];
                if (r < 0) continue;
                if (tuned && i > n - g.subtree(r)) continue;                    // r already holds that chunk
                const int q = (r - 1 + n) % n;                                   // sender, relative
                bcast_xfer_t x{};
                x.phase = BCAST_PHASE_RING;
                x.step = i - 1;
                x.src_rank = g.abs_of_rel[q];
                x.dst_rank = k;
                x.chunk = ((r - i) % n + n) % n;
                x.nchunks = 1;
                // the sender forwards what reached it in the previous ring step; if nothing did (first
                // step, or the sender had stopped receiving) it holds the chunk from before the ring
                x.dep = (i >= 2 && prev[q] >= 0) ? prev[q] : delivered[q];
                cur[r] = (int64_t)p.xfers.size();
                emit(x);
            }
            std::swap(prev, cur);
        }
    }

    // Recursive doubling (Section I; power-of-two group): exchange i, receiver r takes the block of
    // 2^i chunks from r xor 2^i.
    void doubling(const Group &g, const std::vector<int64_t> &delivered)
    {
        const int n = g.size, L = levels_of(n);
        std::vector<std::vector<int64_t>> into(L, std::vector<int64_t>(n, -1));   // [exchange][relative rank]
        for (int i = 0; i < L; i++) {
            const int mask = 1 << i;
            begin_step();
            for (int k = 0; k < p.P; k++) {
                const int r = g.rel_of_abs[k];
                if (r < 0) continue;
                const int q = r ^ mask;                            // sender (relative)
                const int block = (q >> i) << i;
                bcast_xfer_t x{};
                x.phase = BCAST_PHASE_RING;
                x.step = i;
                x.src_rank = g.abs_of_rel[q];
                x.dst_rank = k;
                x.chunk = block;
                x.nchunks = mask;
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
                emit(x);
            }
        }
    }

    // Binomial-tree broadcasts of the whole message (Section II), several disjoint groups level by
    // level at the same time: in a group of `size` processes the member of relative rank r >= 1
    // receives from r - lowbit(r) at level L - 1 - log2(lowbit(r)), L = ceil(log2 size).
    void tree_bcasts(int phase, const std::vector<std::vector<int>> &groups)
    {
        int levels = 0;
        for (const auto &m : groups) levels = std::max(levels, levels_of((int)m.size()));
        std::vector<std::pair<int, bcast_xfer_t>> step;          // (dst, message) of one level
        for (int t = 0; t < levels; t++) {
            step.clear();
            for (const auto &m : groups) {
                const int size = (int)m.size(), L = levels_of(size);
                if (t >= L) continue;
                const int mask = 1 << (L - 1 - t);
                for (int r = mask; r < size; r += 2 * mask) {      // the odd multiples of mask
                    bcast_xfer_t x{};
                    x.phase = phase;
                    x.step = t;
                    x.src_rank = m[r - mask];
                    x.dst_rank = m[r];
                    x.chunk = 0;
                    x.nchunks = p.chunks;
                    step.emplace_back(m[r], x);
                }
            }
            std::sort(step.begin(), step.end(), [](const auto &a, const auto &b) { return a.first < b.first; });
            begin_step();
            for (auto &e : step) {
                e.second.dep = writer0[e.second.src_rank];
                emit(e.second);
            }
        }
    }
};

Group whole_communicator(int P, int root)
{
    Group g;
    g.size = P;
    g.abs_of_rel.resize(P);
    g.rel_of_abs.resize(P);
    for (int r = 0; r < P; r++) {
        g.abs_of_rel[r] = (r + root) % P;
        g.rel_of_abs[(r + root) % P] = r;
    }
    return g;
}

void build(bcast_plan_t &p)
{
    const int P = p.P;
    for (int ph = 0; ph < 4; ph++) {
        p.bytes_sent[ph].assign(P, 0); p.bytes_recv[ph].assign(P, 0);
        p.msgs_sent[ph].assign(P, 0);  p.msgs_recv[ph].assign(P, 0);
    }
    p.step_begin.clear();
    Builder b(p);
    if (P > 1 && p.ranks_per_node == 0) {
        const Group g = whole_communicator(P, p.root);
        p.L = levels_of(P);
        std::vector<int64_t> delivered(P, -1);
        b.scatter(g, delivered);
        if (p.variant == BCAST_DOUBLING) b.doubling(g, delivered);
        else b.ring(g, p.variant == BCAST_TUNED, delivered);
    } else if (P > 1) {
        // node-aware (Section II): nodes are blocks of ranks_per_node consecutive ranks, a node's
        // leader is its lowest rank
        const int c = p.ranks_per_node, nodes = p.chunks, root_node = p.root / c;
        auto node_ranks = [&](int node) {
            std::vector<int> m;
            for (int k = node * c; k < std::min((node + 1) * c, P); k++) m.push_back(k);
            return m;
        };
        // 1. tree broadcast in the root's node, rooted at the root
        std::vector<int> first = node_ranks(root_node);
        std::rotate(first.begin(), first.begin() + (p.root - root_node * c), first.end());
        b.tree_bcasts(BCAST_PHASE_NODE_FIRST, {first});
        // 2. scatter + ring between the leaders, nodes numbered relative to the root's node
        Group g;
        g.size = nodes;
        g.abs_of_rel.resize(nodes);
        g.rel_of_abs.assign(P, -1);
        for (int q = 0; q < nodes; q++) {
            g.abs_of_rel[q] = ((root_node + q) % nodes) * c;
            g.rel_of_abs[g.abs_of_rel[q]] = q;
        }
        p.L = levels_of(nodes);
        std::vector<int64_t> delivered(nodes, -1);
        delivered[0] = b.writer0[g.abs_of_rel[0]];        // how the root node's leader got the message (-1: it is the root)
        b.scatter(g, delivered);
        b.ring(g, p.variant == BCAST_TUNED, delivered);
        // 3. tree broadcasts in all the other nodes, from their leaders
        std::vector<std::vector<int>> others;
        for (int node = 0; node < nodes; node++)
            if (node != root_node) others.push_back(node_ranks(node));
        b.tree_bcasts(BCAST_PHASE_NODE_LAST, others);
    }
    p.step_begin.push_back((int64_t)p.xfers.size());
}

int make_plan(int P, int root, uint64_t nbytes, int variant, int ranks_per_node, bcast_plan_t **out)
{
    if (!out) return BCAST_ERR_INVAL;
    *out = nullptr;
    if (P < 1 || P > BCAST_MAX_RANKS || root < 0 || root >= P || ranks_per_node < 0) return BCAST_ERR_INVAL;
    if (variant != BCAST_NATIVE && variant != BCAST_TUNED && variant != BCAST_DOUBLING) return BCAST_ERR_INVAL;
    if (variant == BCAST_DOUBLING && ((P & (P - 1)) != 0 || ranks_per_node)) return BCAST_ERR_INVAL;
    if (nbytes > (UINT64_MAX >> 1) - (uint64_t)P) return BCAST_ERR_INVAL;
    bcast_plan_t *p = nullptr;
    try {
        p = new bcast_plan_t();
        p->P = P; p->root = root; p->variant = variant; p->nbytes = nbytes;
        p->ranks_per_node = ranks_per_node;
        p->chunks = ranks_per_node ? (P + ranks_per_node - 1) / ranks_per_node : P;
        p->S = (nbytes + (uint64_t)p->chunks - 1) / (uint64_t)p->chunks;
        build(*p);
    } catch (const std::bad_alloc &) {
        delete p;
        return BCAST_ERR_NOMEM;
    }
    *out = p;
    return BCAST_OK;
}

}  // namespace

extern "C" {

int bcast_plan(int P, int root, uint64_t nbytes, int variant, bcast_plan_t **out)
{
    return make_plan(P, root, nbytes, variant, 0, out);
}

int bcast_plan_smp(int P, int root, uint64_t nbytes, int variant, int ranks_per_node, bcast_plan_t **out)
{
    if (ranks_per_node < 1) {
        if (out) *out = nullptr;
        return BCAST_ERR_INVAL;
    }
    return make_plan(P, root, nbytes, variant, ranks_per_node, out);
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
int32_t bcast_plan_ranks_per_node(const bcast_plan_t *p) { return p ? p->ranks_per_node : 0; }
int32_t bcast_plan_num_chunks(const bcast_plan_t *p) { return p ? p->chunks : 0; }
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
        if (!p || phase < 0 || phase > BCAST_PHASE_NODE_LAST) return nullptr;        \
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
