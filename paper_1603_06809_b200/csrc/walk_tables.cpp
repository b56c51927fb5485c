// Host-side tables of the WALK executors (see walk_tables.h).
#include "walk_tables.h"

#include <algorithm>

namespace {

inline uint64_t chunk_begin(const bcast_plan_t &p, int c) { return std::min<uint64_t>((uint64_t)c * p.S, p.nbytes); }

inline uint32_t encode_hop(const bcast_plan_t &p, int64_t i)
{
    return (uint32_t)p.xfers[i].src_rank | ((uint32_t)p.xfers[i].dst_rank << 16);
}

inline bool is_active(const std::vector<char> *active, uint64_t c) { return !active || (*active)[(size_t)c] != 0; }

// Classify segment g of the `seg`-byte grid and append its slice(s).
void classify_segment(const bcast_plan_t &p, uint64_t seg, uint64_t g, bool use_dual, const std::vector<char> *active,
                      std::vector<WalkSlice> &ragged, std::vector<WalkSlice> &dual, std::vector<WalkSlice> &full)
{
    const uint64_t lo = g * seg, hi = std::min(lo + seg, p.nbytes);
    if (lo >= hi || p.S == 0) return;
    const uint64_t c0 = lo / p.S, c1 = (hi - 1) / p.S;      // chunks that overlap the segment: all non-empty
    const bool whole = hi == lo + seg;
    if (c0 == c1) {
        if (is_active(active, c0))
            (whole ? full : ragged).push_back(WalkSlice{(uint32_t)g, (uint32_t)c0 | ((whole ? kSliceFull : kSliceRagged) << kSliceKindShift)});
    } else if (c1 == c0 + 1 && whole && use_dual && is_active(active, c0) && is_active(active, c1)) {
        dual.push_back(WalkSlice{(uint32_t)g, (uint32_t)c0 | (kSliceDual << kSliceKindShift)});
    } else {
        for (uint64_t c = c0; c <= c1; c++)
            if (is_active(active, c)) ragged.push_back(WalkSlice{(uint32_t)g, (uint32_t)c | (kSliceRagged << kSliceKindShift)});
    }
}

}  // namespace

void messages_by_chunk(const bcast_plan_t &p, std::vector<std::vector<int64_t>> &per_chunk)
{
    per_chunk.assign(p.P, {});
    for (size_t i = 0; i < p.xfers.size(); i++) {
        const bcast_xfer_t &x = p.xfers[i];
        if (!x.len) continue;
        for (int c = x.chunk; c < x.chunk + x.nchunks; c++)
            if (chunk_begin(p, c + 1) > chunk_begin(p, c)) per_chunk[c].push_back((int64_t)i);
    }
}

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

// Two neighbouring chunks meet inside one 16-byte word (and one 32-byte sector) of every rank
// buffer unless the scatter size happens to be a multiple of 32.  If the two parts of that sector
// are written at different times, each write is a partial-sector write and the next read of the
// sector has to wait for the rest of it to be fetched from DRAM.  A warp that carries both parts
// can write them with one instruction whenever the two chunks' lists have a hop into the same
// rank side by side.  In the ring the hop of chunk c+1 into a rank comes one step before the hop
// of chunk c into it, so the lists are merged here with a small look-ahead: both keep their own
// order (which is all the plan's dependencies need, the two byte ranges being disjoint), and a
// slot holds a hop of each list when they write the same rank.
void pair_hops(const bcast_plan_t &p, const std::vector<int64_t> &lower, const std::vector<int64_t> &upper,
               std::vector<DualMsg> &slots)
{
    constexpr size_t kLookAhead = 8;
    auto dst = [&](int64_t i) { return p.xfers[i].dst_rank; };
    slots.clear();
    size_t i = 0, j = 0;
    const size_t na = lower.size(), nb = upper.size();
    while (i < na || j < nb) {
        if (i == na) { slots.push_back(DualMsg{-1, (int32_t)upper[j++]}); continue; }
        if (j == nb) { slots.push_back(DualMsg{(int32_t)lower[i++], -1}); continue; }
        if (dst(lower[i]) == dst(upper[j])) { slots.push_back(DualMsg{(int32_t)lower[i++], (int32_t)upper[j++]}); continue; }
        size_t ka = 0, kb = 0;
        for (size_t k = 1; k <= kLookAhead && i + k < na && !ka; k++)
            if (dst(lower[i + k]) == dst(upper[j])) ka = k;
        for (size_t k = 1; k <= kLookAhead && j + k < nb && !kb; k++)
            if (dst(upper[j + k]) == dst(lower[i])) kb = k;
        if (ka && (!kb || ka <= kb)) {
            for (size_t k = 0; k < ka; k++) slots.push_back(DualMsg{(int32_t)lower[i++], -1});
        } else if (kb) {
            for (size_t k = 0; k < kb; k++) slots.push_back(DualMsg{-1, (int32_t)upper[j++]});
        } else {
            slots.push_back(DualMsg{(int32_t)lower[i++], (int32_t)upper[j++]});   // no partner near: two partial writes
        }
    }
}

void whole_plan_hops(const bcast_plan_t &p, HopLists &lists)
{
    messages_by_chunk(p, lists.plan_order);
    lists.walk_order.assign(p.P, {});
    for (int c = 0; c < p.P; c++) order_by_dependency(p, lists.plan_order[c], lists.walk_order[c]);
}

void make_walk_tables(const bcast_plan_t &p, const HopLists &lists, WalkTables &t)
{
    const int P = p.P;
    t.hop_begin.assign(P + 1, 0);
    t.hops.clear(); t.hops_plan.clear(); t.hop_msg.clear(); t.hop_msg_plan.clear();
    for (int c = 0; c < P; c++) {
        t.hop_begin[c] = (int)t.hops.size();
        for (int64_t i : lists.walk_order[c]) { t.hops.push_back(encode_hop(p, i)); t.hop_msg.push_back((int32_t)i); }
        for (int64_t i : lists.plan_order[c]) { t.hops_plan.push_back(encode_hop(p, i)); t.hop_msg_plan.push_back((int32_t)i); }
    }
    t.hop_begin[P] = (int)t.hops.size();

    t.dual_begin.assign(P + 1, 0);
    t.dual.clear(); t.dual_msg.clear();
    std::vector<DualMsg> slots;
    for (int c = 0; c < P; c++) {
        t.dual_begin[c] = (int)t.dual.size();
        if (c + 1 >= P || lists.plan_order[c].empty() || lists.plan_order[c + 1].empty()) continue;
        pair_hops(p, lists.plan_order[c], lists.plan_order[c + 1], slots);
        const size_t first = t.dual.size();
        for (const DualMsg &s : slots) {
            t.dual.push_back(DualSlot{s.a < 0 ? kNoHop : encode_hop(p, s.a), s.b < 0 ? kNoHop : encode_hop(p, s.b)});
            t.dual_msg.push_back(s);
        }
        // mark the slots that come kDualAhead before a slot with two different hops (see kHopAheadFlag)
        for (size_t i = 0; i + kDualAhead < slots.size(); i++) {
            const DualSlot &ahead = t.dual[first + i + kDualAhead];
            if ((ahead.a & ~kHopAheadFlag) == (ahead.b & ~kHopAheadFlag)) continue;
            DualSlot &now = t.dual[first + i];
            if (now.a != kNoHop) now.a |= kHopAheadFlag;
            if (now.b != kNoHop) now.b |= kHopAheadFlag;
        }
    }
    t.dual_begin[P] = (int)t.dual.size();
}

void make_slices(const bcast_plan_t &p, uint64_t seg_bytes, bool use_dual, const std::vector<char> *active,
                 std::vector<WalkSlice> &slices)
{
    std::vector<WalkSlice> ragged, dual, full;
    const uint64_t nseg = (p.nbytes + seg_bytes - 1) / seg_bytes;
    for (uint64_t g = 0; g < nseg; g++) classify_segment(p, seg_bytes, g, use_dual, active, ragged, dual, full);
    slices.clear();
    slices.reserve(ragged.size() + dual.size() + full.size());
    slices.insert(slices.end(), ragged.begin(), ragged.end());
    slices.insert(slices.end(), dual.begin(), dual.end());
    slices.insert(slices.end(), full.begin(), full.end());
}

long long count_slices(const bcast_plan_t &p, uint64_t seg_bytes, bool use_dual, const std::vector<char> *active)
{
    if (p.nbytes == 0 || p.S == 0) return 0;
    if (active) {                                   // a partial walk: count what make_slices would make
        std::vector<WalkSlice> ragged, dual, full;
        const uint64_t nseg = (p.nbytes + seg_bytes - 1) / seg_bytes;
        for (uint64_t g = 0; g < nseg; g++) classify_segment(p, seg_bytes, g, use_dual, active, ragged, dual, full);
        return (long long)(ragged.size() + dual.size() + full.size());
    }
    // every segment is one slice, except those that are cut into ragged slices per chunk
    const uint64_t nseg = (p.nbytes + seg_bytes - 1) / seg_bytes;
    long long n = (long long)nseg;
    for (int c = 1; c < p.P; c++) {
        const uint64_t b = (uint64_t)c * p.S;
        if (b >= p.nbytes) break;
        if (b % seg_bytes == 0) continue;                                  // boundary on the grid: cuts nothing
        const uint64_t g = b / seg_bytes;
        const uint64_t lo = g * seg_bytes, hi = std::min(lo + seg_bytes, p.nbytes);
        const uint64_t c0 = lo / p.S, c1 = (hi - 1) / p.S;
        const bool dual = c1 == c0 + 1 && hi == lo + seg_bytes && use_dual;
        if (!dual) n += 1;                                                 // each boundary inside adds one ragged slice
    }
    return n;
}

void make_bulk_slices(const bcast_plan_t &p, uint64_t bulk_seg, uint64_t reg_seg, std::vector<WalkSlice> &bulk,
                      std::vector<WalkSlice> &reg)
{
    std::vector<WalkSlice> ragged, dual, full;
    bulk.clear();
    reg.clear();
    if (p.S == 0) return;
    const uint64_t per = bulk_seg / reg_seg;
    const uint64_t nseg = (p.nbytes + bulk_seg - 1) / bulk_seg;
    for (uint64_t g = 0; g < nseg; g++) {
        const uint64_t lo = g * bulk_seg, hi = std::min(lo + bulk_seg, p.nbytes);
        const uint64_t c0 = lo / p.S, c1 = (hi - 1) / p.S;
        if (c0 == c1 && hi == lo + bulk_seg) {
            bulk.push_back(WalkSlice{(uint32_t)g, (uint32_t)c0});
            continue;
        }
        for (uint64_t q = g * per; q < (g + 1) * per && q * reg_seg < p.nbytes; q++)
            classify_segment(p, reg_seg, q, true, nullptr, ragged, dual, full);
    }
    reg.insert(reg.end(), ragged.begin(), ragged.end());
    reg.insert(reg.end(), dual.begin(), dual.end());
    reg.insert(reg.end(), full.begin(), full.end());
}
