// Host-side tables of the WALK executors: how the message is cut into slices and in which order
// the messages of the plan ("hops") are performed on every slice.  Integers only; no CUDA.
#pragma once
#include <cstdint>
#include <vector>

#include "plan_internal.h"

// One warp's unit of work: the part of segment `seg` (fixed grid of `seg_bytes`-byte segments
// over the message) that `ref` describes.
//   kSliceFull    the whole segment lies in relative chunk `ref & kSliceRefMask`
//   kSliceRagged  only the bytes of that chunk which fall into the segment (the segment holds a
//                 chunk boundary or the end of the message)
//   kSliceDual    the whole segment, which holds exactly one chunk boundary: the bytes below it
//                 belong to chunk `ref & kSliceRefMask`, the bytes above it to the next chunk
struct WalkSlice {
    uint32_t seg;
    uint32_t ref;
};
constexpr uint32_t kSliceFull = 0u, kSliceRagged = 1u, kSliceDual = 2u;
constexpr int kSliceKindShift = 30;
constexpr uint32_t kSliceRefMask = (1u << kSliceKindShift) - 1u;

// A hop is src_rank | dst_rank << 16.  A slot of a dual list holds one hop of the lower chunk
// (a) and one of the upper chunk (b), either of which may be absent.
constexpr uint32_t kNoHop = 0xffffffffu;
// Dual slots only: bit 15 of a hop says that the slot kDualAhead places further on holds two
// different hops (or one), i.e. will store only part of the sector around the boundary; the warp
// then asks L2 for that sector now.  Ranks need 10 bits, so the source rank is hop & kHopRankMask.
constexpr uint32_t kHopAheadFlag = 0x8000u, kHopRankMask = 0x3ffu;
constexpr int kDualAhead = 6;
struct DualSlot {
    uint32_t a, b;
};
struct DualMsg {       // indices into the plan's message array, -1 where the slot has no hop
    int32_t a, b;
};

// Device pointers of the tables one WALK launch reads (filled by the host, passed by value).
struct WalkDev {
    const WalkSlice *slices;
    long long n_slices;
    const uint32_t *hops;        // per chunk, the order in use
    const int *hop_begin;
    const DualSlot *dual;        // per chunk boundary
    const int *dual_begin;
    const int32_t *hop_msg;      // traced launches only: plan message of every hop / slot
    const DualMsg *dual_msg;
    unsigned long long *trace;   // traced launches only: bytes stored per plan message
    uint64_t scatter_size, nbytes;
    // How slices are dealt to blocks: the first `grouped` slices of the list in runs of `group`
    // neighbours (run j goes to block j mod gridDim.x), the rest one by one (group = 1: all one by one).
    int group;
    long long grouped;
};

// Per relative chunk, the plan messages ("hops") a walk performs on the bytes of that chunk: in
// the order the full and ragged slices take them, and in plan order (what the dual lists are
// merged from).  A walk over a part of the plan (one GPU's share of one phase) has shorter lists.
struct HopLists {
    std::vector<std::vector<int64_t>> walk_order, plan_order;
};

struct WalkTables {
    // per relative chunk c: hops [hop_begin[c], hop_begin[c+1]) in dependency order / plan order,
    // and beside every hop the index of the plan message it performs
    std::vector<uint32_t> hops, hops_plan;
    std::vector<int32_t> hop_msg, hop_msg_plan;
    std::vector<int> hop_begin;                       // [P + 1]
    // per chunk boundary (c, c+1): slots [dual_begin[c], dual_begin[c+1])
    std::vector<DualSlot> dual;
    std::vector<DualMsg> dual_msg;
    std::vector<int> dual_begin;                      // [P + 1]
};

// For every relative chunk: the plan's messages that move bytes of it, in plan order.
void messages_by_chunk(const bcast_plan_t &p, std::vector<std::vector<int64_t>> &per_chunk);

// Re-order the hops of one chunk into the level order of its dependency tree where that is legal
// (no rank written twice); otherwise `out` = `plan_order`.
void order_by_dependency(const bcast_plan_t &p, const std::vector<int64_t> &plan_order, std::vector<int64_t> &out);

// Merge the plan-order hop lists of two neighbouring chunks into one list of slots; the order
// inside each list is kept, and hops of the two lists that write the same rank share a slot
// wherever the lists allow it.
void pair_hops(const bcast_plan_t &p, const std::vector<int64_t> &lower, const std::vector<int64_t> &upper,
               std::vector<DualMsg> &slots);

// The hop lists of the whole plan: plan order, and level order of the dependency tree where legal.
void whole_plan_hops(const bcast_plan_t &p, HopLists &lists);

// Device-table images (hop lists and dual lists) from hop lists; independent of the segment size.
void make_walk_tables(const bcast_plan_t &p, const HopLists &lists, WalkTables &t);

// The slices of the message for segments of `seg_bytes` bytes, restricted to segments
// [seg_first, seg_last) (pass 0, UINT64_MAX for all).  Order: ragged slices first, then dual
// slices, then full slices, each group in message order (the slow kinds start first).
// `use_dual` = false cuts every segment that holds a boundary into ragged slices instead.
// `active` (NULL: all): per relative chunk, whether the walk has any hop for it; bytes of inactive
// chunks get no slice, and a boundary segment is a dual slice only if both its chunks are active.
void make_slices(const bcast_plan_t &p, uint64_t seg_bytes, bool use_dual, const std::vector<char> *active,
                 std::vector<WalkSlice> &slices);

// Number of slices make_slices() would produce.
long long count_slices(const bcast_plan_t &p, uint64_t seg_bytes, bool use_dual, const std::vector<char> *active);

// Slices of the bulk-copy walk: every whole 16 KiB segment inside one chunk is a bulk slice (kind
// kSliceFull on the 16 KiB grid); the other 16 KiB segments are cut on the 4 KiB grid into
// register slices of any kind.
void make_bulk_slices(const bcast_plan_t &p, uint64_t bulk_seg, uint64_t reg_seg, std::vector<WalkSlice> &bulk,
                      std::vector<WalkSlice> &reg);
