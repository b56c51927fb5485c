// Device code of the broadcast executors (sm_100a): every message of the plan is a copy of `len`
// bytes at `offset` from the source rank's buffer to the same offset of the destination rank's
// buffer (Section III-A: scatter and native ring; Section IV: tuned ring).
//
// Two facts about the schedule shape the kernels:
//   * source and destination of a message use the SAME byte offset (the listing displaces both
//     sides by chunk index x scatter_size), so with 16-byte aligned rank buffers both sides are
//     co-aligned;
//   * a byte of the message at some rank depends only on the same byte at the rank it is copied
//     from, so messages that cover different byte ranges never depend on one another.
//
// WALK executor (one launch): the message is cut into segments on a fixed grid of byte offsets.
// A warp takes a segment and performs every message of the plan that covers it, restricted to the
// segment, in an order that respects the plan's dependencies: load from the source rank's buffer,
// store to the destination rank's buffer.  Each thread always handles the same bytes of the
// segment, so whatever a hop reads was stored earlier by the same thread: program order per thread
// is the only ordering the schedule needs.  Loads bypass L1 (.cg) so that every hop really
// re-reads the source rank's buffer from the L2/HBM level.
//
// STEPS / GRAPH executors: one launch per plan step, the messages of the step cut into tiles.
//
// With TRACE every kernel also adds, per message of the plan, the bytes it stored for it to a
// counter array (one 64-bit counter per message), so that a test can see that each message was
// performed in full; without TRACE none of that code exists.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "walk_tables.h"

namespace bcast_dev {

constexpr int kThreads = 256;             // threads per block of the walk and step kernels
constexpr int kWarpsPerBlock = kThreads / 32;
constexpr int kMaxWords = 8;              // most 16-byte words per lane of a walk slice
constexpr int kStepWordsPerThread = 4;    // STEPS executor: 256 x 4 x 16 B = 16 KiB tiles
constexpr uint64_t kStepTile = (uint64_t)kThreads * kStepWordsPerThread * 16;

// The P rank-buffer pointers travel as a kernel argument (copied at launch), so a launch never
// depends on a device-side pointer table that a later call could overwrite.
template <int MAXP>
struct RankPtrs {
    uint8_t *p[MAXP];
};

struct DevXfer {      // one message, device copy (STEPS executor)
    uint64_t off, len;
    uint16_t src, dst;
    uint32_t pad;
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

// Ask L2 to fetch the line that holds *p.  Used ahead of a store that will cover only part of a
// 32-byte sector: a sector that sits in L2 partly written makes the next read of it wait for
// DRAM, whereas a partial write into a sector that is already complete in L2 leaves it complete.
__device__ __forceinline__ void prefetch_l2(const uint8_t *p)
{
    asm volatile("prefetch.global.L2 [%0];" :: "l"(p) : "memory");
}
constexpr int kPrefetchAhead = 6;         // hops between that request and the partial store

// Warp-wide: add the bytes the lanes stored for plan message `msg` to its counter.
__device__ __forceinline__ void trace_add(unsigned long long *trace, int msg, uint32_t lane_bytes)
{
    const uint32_t total = __reduce_add_sync(0xffffffffu, lane_bytes);
    if ((threadIdx.x & 31u) == 0 && msg >= 0 && total) atomicAdd(trace + msg, (unsigned long long)total);
}

// ------------------------------------------------------------------------------------- WALK
// The message is cut on a fixed grid of segments of 32 x U words (U x 512 bytes).  Lanes map to
// the fixed 16-byte words of the segment, whatever a chunk's first byte is, so a warp's 512-byte
// accesses stay aligned to cache lines.  The (src, dst) pair of hop h+1 is fetched while the loads
// of hop h are in flight.

// A segment that lies inside one chunk: every lane moves U words per hop, no predicates.
template <int U, int MAXP, bool TRACE>
__device__ __forceinline__ void walk_full(const RankPtrs<MAXP> &bufs, uint32_t seg, uint32_t chunk, const WalkDev &t,
                                          uint32_t lane)
{
    constexpr uint64_t kSeg = 32ull * U * 16;
    const int h0 = t.hop_begin[chunk];
    const int nh = t.hop_begin[chunk + 1] - h0;
    if (nh <= 0) return;
    const uint32_t *hp = t.hops + h0;
    const uint64_t base = (uint64_t)seg * kSeg + (uint64_t)lane * 16;
    uint32_t e = __ldg(hp);
    const uint8_t *s = bufs.p[e & 0xffffu];
    uint8_t *d = bufs.p[e >> 16];
    for (int h = 0; h < nh; h++) {
        uint4 v[U];
#pragma unroll
        for (int u = 0; u < U; u++) v[u] = ld16(s + base + (uint64_t)u * 512);
        e = __ldg(hp + min(h + 1, nh - 1));              // next hop, while the loads are in flight
        const uint8_t *s_next = bufs.p[e & 0xffffu];
        uint8_t *d_next = bufs.p[e >> 16];
#pragma unroll
        for (int u = 0; u < U; u++) st16(d + base + (uint64_t)u * 512, v[u]);
        if constexpr (TRACE) trace_add(t.trace, t.hop_msg[h0 + h], 16u * U);
        s = s_next;
        d = d_next;
    }
}

// The bytes of one chunk inside a segment that the chunk does not fill (several chunk boundaries
// in the segment, or the end of the message): predicated words, plus the bytes of the partial
// words at either end, one byte per lane.
template <int U, int MAXP, bool TRACE>
__device__ __forceinline__ void walk_ragged(const RankPtrs<MAXP> &bufs, uint32_t seg, uint32_t chunk, const WalkDev &t,
                                            uint32_t lane)
{
    constexpr uint64_t kSeg = 32ull * U * 16;
    const uint64_t seg_lo = (uint64_t)seg * kSeg, seg_hi = seg_lo + kSeg;
    const uint64_t lo = max(min((uint64_t)chunk * t.scatter_size, t.nbytes), seg_lo);
    const uint64_t hi = min(min(((uint64_t)chunk + 1) * t.scatter_size, t.nbytes), seg_hi);
    if (lo >= hi) return;
    const int h0 = t.hop_begin[chunk];
    const int nh = t.hop_begin[chunk + 1] - h0;
    if (nh <= 0) return;
    const uint32_t *hp = t.hops + h0;
    const uint64_t base = seg_lo + (uint64_t)lane * 16;
    const uint64_t body_lo = (lo + 15) & ~(uint64_t)15, body_hi = hi & ~(uint64_t)15;
    const uint64_t head_end = body_lo < hi ? body_lo : hi;
    const uint64_t tail_begin = body_hi > head_end ? body_hi : head_end;
    const uint32_t nhead = (uint32_t)(head_end - lo), nedge = nhead + (uint32_t)(hi - tail_begin);
    bool ok[U];
    uint32_t lane_bytes = 0;
#pragma unroll
    for (int u = 0; u < U; u++) {
        const uint64_t o = base + (uint64_t)u * 512;
        ok[u] = o >= body_lo && o + 16 <= body_hi;
        lane_bytes += ok[u] ? 16u : 0u;
    }
    const bool has_edge = lane < nedge;
    lane_bytes += has_edge ? 1u : 0u;
    const uint64_t eoff = lane < nhead ? lo + lane : tail_begin + (lane - nhead);
    uint32_t e = __ldg(hp);
    const uint8_t *s = bufs.p[e & 0xffffu];
    uint8_t *d = bufs.p[e >> 16];
    // the first and the last sector of the range may be written in part only: have them in L2 first
    for (int h = (int)lane; h < min(nh, kPrefetchAhead); h += 32) {
        uint8_t *dn = bufs.p[__ldg(hp + h) >> 16];
        prefetch_l2(dn + lo);
        prefetch_l2(dn + hi - 1);
    }
    uint32_t ahead = __ldg(hp + min(kPrefetchAhead, nh - 1));
    for (int h = 0; h < nh; h++) {
        uint4 v[U];
        uint32_t b = 0;
#pragma unroll
        for (int u = 0; u < U; u++)
            if (ok[u]) v[u] = ld16(s + base + (uint64_t)u * 512);
        if (has_edge) b = ld1(s + eoff);
        if (lane < 2 && h + kPrefetchAhead < nh) {
            uint8_t *dn = bufs.p[ahead >> 16];
            prefetch_l2(lane ? dn + hi - 1 : dn + lo);
        }
        ahead = __ldg(hp + min(h + 1 + kPrefetchAhead, nh - 1));   // fetched a hop early: nothing waits for it
        e = __ldg(hp + min(h + 1, nh - 1));
        const uint8_t *s_next = bufs.p[e & 0xffffu];
        uint8_t *d_next = bufs.p[e >> 16];
#pragma unroll
        for (int u = 0; u < U; u++)
            if (ok[u]) st16(d + base + (uint64_t)u * 512, v[u]);
        if (has_edge) st1(d + eoff, b);
        if constexpr (TRACE) trace_add(t.trace, t.hop_msg[h0 + h], lane_bytes);
        s = s_next;
        d = d_next;
    }
}

// Bytes [0, nb) of a 32-bit lane from `a`, the rest from `b` (nb may be <= 0 or >= 4).
__device__ __forceinline__ uint32_t low_bytes_from(uint32_t a, uint32_t b, int nb)
{
    if (nb <= 0) return b;
    if (nb >= 4) return a;
    const uint32_t m = (1u << (8 * nb)) - 1u;
    return (a & m) | (b & ~m);
}
// Store bytes [from, to) of the 16-byte word `v` to p[from..to), one st.u8 each.
__device__ __forceinline__ void store_bytes(uint8_t *p, const uint4 &v, uint32_t from, uint32_t to)
{
    const uint32_t c[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (uint32_t b = 0; b < 16; b++)
        if (b >= from && b < to) st1(p + b, (c[b >> 2] >> (8 * (b & 3))) & 0xffu);
}

// A whole segment that holds exactly one chunk boundary (`cut` bytes into it): the words below it
// follow the hops of chunk c, the words above it those of chunk c+1, slot by slot of the
// boundary's dual list.
//   * A slot whose two hops are the same (src, dst) pair -- every ring step once the lists are
//     aligned -- moves the segment as one piece, exactly like a full slice.
//   * Otherwise every lane takes source, destination and predicate from the side its word is on.
//     The 16-byte word that straddles the boundary (if the boundary is not a multiple of 16)
//     belongs to one lane, which loads it from both sources; when the two hops write the same
//     rank it stores the word whole -- its low `cut % 16` bytes from the lower chunk's source, the
//     rest from the upper chunk's -- in the same warp instruction as its neighbours, so that the
//     32-byte sector around the boundary is written in one piece and never sits half-written in
//     L2 (a read of a half-written sector has to wait for DRAM).  With one hop only, or two
//     different destinations, the parts go out byte by byte.
template <int U, int MAXP, bool TRACE>
__device__ __forceinline__ void walk_dual(const RankPtrs<MAXP> &bufs, uint32_t seg, uint32_t c, const WalkDev &t,
                                          uint32_t lane)
{
    constexpr uint64_t kSeg = 32ull * U * 16;
    const uint64_t seg_lo = (uint64_t)seg * kSeg;
    const uint32_t cut = (uint32_t)(((uint64_t)c + 1) * t.scatter_size - seg_lo);   // 0 < cut < kSeg
    const int s0 = t.dual_begin[c];
    const int ns = t.dual_begin[c + 1] - s0;
    if (ns <= 0) return;
    const DualSlot *sp = t.dual + s0;
    const uint64_t base = seg_lo + (uint64_t)lane * 16;
    const uint32_t k = cut & 15u;                                   // bytes of the straddling word below the boundary
    const bool strad = k != 0 && lane == ((cut >> 4) & 31u);        // this lane owns the straddling word ...
    const int su = (int)(cut >> 9);                                 // ... as its word number su
    const uint64_t so = seg_lo + (cut & ~15u);
    uint32_t bytes_a = 0, bytes_b = 0;
    if constexpr (TRACE) {
#pragma unroll
        for (int u = 0; u < U; u++) {
            const uint32_t o = lane * 16u + (uint32_t)u * 512u;
            bytes_a += o + 16 <= cut ? 16u : 0u;
            bytes_b += o >= cut ? 16u : 0u;
        }
        if (strad) { bytes_a += k; bytes_b += 16u - k; }
    }
    DualSlot e = sp[0];
    // slots whose two hops differ store only part of the sector around the boundary: have it in L2
    // first.  The scatter hops, where most such slots are, come first: one request per lane now;
    // for the others the table flags the slot kDualAhead places before.
    auto prefetch_cut = [&](int slot) {
        const DualSlot a = sp[slot];
        if (a.a == a.b) return;
        if (a.a != kNoHop) prefetch_l2(bufs.p[a.a >> 16] + seg_lo + cut - 1);
        if (a.b != kNoHop) prefetch_l2(bufs.p[a.b >> 16] + seg_lo + cut);
    };
    if ((int)lane < min(ns, kDualAhead)) prefetch_cut((int)lane);
    for (int h = 0; h < ns; h++) {
        const DualSlot cur = e;
        if (cur.a == cur.b) {
            // the same hop for both chunks: the segment moves as one piece
            const uint8_t *s = bufs.p[cur.a & kHopRankMask];
            uint8_t *d = bufs.p[cur.a >> 16];
            uint4 v[U];
#pragma unroll
            for (int u = 0; u < U; u++) v[u] = ld16(s + base + (uint64_t)u * 512);
            e = sp[min(h + 1, ns - 1)];                  // next slot, while the loads are in flight
            if (lane == 0 && (cur.a & kHopAheadFlag)) prefetch_cut(h + kDualAhead);
#pragma unroll
            for (int u = 0; u < U; u++) st16(d + base + (uint64_t)u * 512, v[u]);
        } else {
            const bool ha = cur.a != kNoHop, hb = cur.b != kNoHop;
            const uint8_t *sa = bufs.p[ha ? (cur.a & kHopRankMask) : 0u], *sb = bufs.p[hb ? (cur.b & kHopRankMask) : 0u];
            uint8_t *da = bufs.p[ha ? (cur.a >> 16) : 0u], *db = bufs.p[hb ? (cur.b >> 16) : 0u];
            const bool whole = ha && hb && da == db;     // the straddling word can be stored in one piece
            uint4 v[U], wa = make_uint4(0, 0, 0, 0), wb = wa;
#pragma unroll
            for (int u = 0; u < U; u++) {
                const uint32_t o = lane * 16u + (uint32_t)u * 512u;
                const bool upper = o >= cut;             // else lower, or the straddling word (loaded from the lower source here)
                if (upper ? hb : ha) v[u] = ld16((upper ? sb : sa) + base + (uint64_t)u * 512);
            }
            if (strad && hb) wb = ld16(sb + so);
            e = sp[min(h + 1, ns - 1)];
            if (lane == 0 && ((ha ? cur.a : cur.b) & kHopAheadFlag)) prefetch_cut(h + kDualAhead);
#pragma unroll
            for (int u = 0; u < U; u++) {
                const uint32_t o = lane * 16u + (uint32_t)u * 512u;
                const bool upper = o >= cut, mine = strad && u == su;
                if (mine) {
                    wa = v[u];
                    v[u].x = low_bytes_from(wa.x, wb.x, (int)k);
                    v[u].y = low_bytes_from(wa.y, wb.y, (int)k - 4);
                    v[u].z = low_bytes_from(wa.z, wb.z, (int)k - 8);
                    v[u].w = low_bytes_from(wa.w, wb.w, (int)k - 12);
                }
                if (mine ? whole : (upper ? hb : ha)) st16((upper ? db : da) + base + (uint64_t)u * 512, v[u]);
            }
            if (strad && !whole) {
                if (ha) store_bytes(da + so, wa, 0u, k);
                if (hb) store_bytes(db + so, wb, k, 16u);
            }
        }
        if constexpr (TRACE) {
            const DualMsg m = t.dual_msg[s0 + h];
            trace_add(t.trace, m.a, cur.a != kNoHop ? bytes_a : 0u);
            trace_add(t.trace, m.b, cur.b != kNoHop ? bytes_b : 0u);
        }
    }
}

template <int U, int MAXP, bool TRACE>
__device__ __forceinline__ void walk_slice(const RankPtrs<MAXP> &bufs, const WalkSlice sl, const WalkDev &t, uint32_t lane)
{
    const uint32_t kind = sl.ref >> kSliceKindShift, c = sl.ref & kSliceRefMask;
    if (kind == kSliceFull) walk_full<U, MAXP, TRACE>(bufs, sl.seg, c, t, lane);
    else if (kind == kSliceDual) walk_dual<U, MAXP, TRACE>(bufs, sl.seg, c, t, lane);
    else walk_ragged<U, MAXP, TRACE>(bufs, sl.seg, c, t, lane);
}

// Slices are dealt round-robin over the blocks -- one by one (slice w belongs to block
// w mod gridDim.x) or, for the first `grouped` slices of the list, in runs of `group` neighbours
// (run j belongs to block j mod gridDim.x; with group = warps per block an SM then works on one
// contiguous piece of the message at a time) -- so that every SM gets the same share and the
// slices in flight at any time are neighbours in the message.  Inside a block the warps draw the
// block's slices in order from a ticket counter in shared memory, so a warp that got a slow
// slice (a partial sector at the end of the message, an L2 miss) does not hold up the others.
// Warps never wait for one another.
template <int U, int MAXP, bool TRACE>
__global__ void __launch_bounds__(kThreads)
bcast_walk_kernel(const __grid_constant__ RankPtrs<MAXP> bufs, const __grid_constant__ WalkDev t)
{
    __shared__ int ticket;
    if (threadIdx.x == 0) ticket = 0;
    __syncthreads();
    const uint32_t lane = threadIdx.x & 31u;
    for (;;) {
        int k = 0;
        if (lane == 0) k = atomicAdd(&ticket, 1);
        k = __shfl_sync(0xffffffffu, k, 0);
        // ticket k of this block -> slice index w
        const long long in_runs = t.grouped / gridDim.x;          // tickets of a block that fall into the grouped part
        long long w;
        if (k < in_runs)
            w = ((long long)(k / t.group) * gridDim.x + blockIdx.x) * t.group + (k % t.group);
        else
            w = t.grouped + (k - in_runs) * gridDim.x + blockIdx.x;
        if (w >= t.n_slices) break;
        walk_slice<U, MAXP, TRACE>(bufs, t.slices[w], t, lane);
    }
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
//
// Every wait on the copy engine is bounded.  A worker polls its mbarrier at most `spin_limit`
// times; if the load has not arrived by then it raises the status flag (the host reports it as a
// timeout) and goes on polling under a second, much larger bound, so that it does not leave
// while its own copy may still be landing in shared memory.  If that bound runs out too, the
// worker stops: the copy is lost and the rank buffers stay incomplete.
constexpr uint32_t kBulkSeg = 16384;
constexpr int kBulkWorkers = 4;               // worker threads (lanes 0..3 of warp 0) and segments in flight per block
constexpr int kBulkThreads = 64;              // warp 0: bulk workers; warp 1: register slices
constexpr int kBulkRegWords = 8;              // register slices of the bulk walk: 4 KiB
constexpr int kBulkSpinLimit = 1 << 22;       // default first bound (polls)
constexpr int kBulkSpinLimitLate = 1 << 26;   // second bound, after the flag has been raised

struct BulkDev {
    const WalkSlice *bulk_slices;
    long long n_bulk;
    int spin_limit;
    int *status;
};

__device__ __forceinline__ bool mbar_poll(uint32_t sbar, uint32_t phase, int limit)
{
    uint32_t arrived = 0;
    for (int spin = 0; spin < limit && !arrived; spin++)
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                     : "=r"(arrived) : "r"(sbar), "r"(phase) : "memory");
    return arrived != 0;
}

template <int MAXP, bool TRACE>
__global__ void __launch_bounds__(kBulkThreads)
bcast_walk_bulk_kernel(const __grid_constant__ RankPtrs<MAXP> bufs, const __grid_constant__ WalkDev t,
                       const __grid_constant__ BulkDev bk)
{
    extern __shared__ __align__(128) uint8_t bulk_smem[];
    __shared__ __align__(8) uint64_t bulk_bar[kBulkWorkers];
    const uint32_t lane = threadIdx.x & 31u;

    if (threadIdx.x >= 32) {
        // warp 1: the 16 KiB segments cut by chunk boundaries, as register slices of 8 words per lane
        for (long long w = blockIdx.x; w < t.n_slices; w += gridDim.x)
            walk_slice<kBulkRegWords, MAXP, TRACE>(bufs, t.slices[w], t, lane);
        return;
    }
    if (lane >= kBulkWorkers) return;

    const uint32_t sbuf = (uint32_t)__cvta_generic_to_shared(bulk_smem + (size_t)lane * kBulkSeg);
    const uint32_t sbar = (uint32_t)__cvta_generic_to_shared(&bulk_bar[lane]);
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(sbar) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    uint32_t phase = 0;
    const long long total = (long long)gridDim.x * kBulkWorkers;
    for (long long w = (long long)lane * gridDim.x + blockIdx.x; w < bk.n_bulk; w += total) {
        const WalkSlice sl = bk.bulk_slices[w];
        const uint32_t chunk = sl.ref & kSliceRefMask;
        const uint64_t off = (uint64_t)sl.seg * kBulkSeg;
        const int h0 = t.hop_begin[chunk];
        const int nh = t.hop_begin[chunk + 1] - h0;
        for (int h = 0; h < nh; h++) {
            const uint32_t e = __ldg(t.hops + h0 + h);
            const uint8_t *s = bufs.p[e & 0xffffu] + off;
            uint8_t *d = bufs.p[e >> 16] + off;
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(sbar), "r"(kBulkSeg) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         :: "r"(sbuf), "l"(s), "r"(kBulkSeg), "r"(sbar) : "memory");
            if (!mbar_poll(sbar, phase, bk.spin_limit)) {
                atomicExch(bk.status, 1);                                   // tell the host, then keep waiting
                if (!mbar_poll(sbar, phase, kBulkSpinLimitLate)) return;    // the load never came: give up
            }
            phase ^= 1u;
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" :: "l"(d), "r"(sbuf), "r"(kBulkSeg) : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
            if constexpr (TRACE) atomicAdd(t.trace + t.hop_msg[h0 + h], (unsigned long long)kBulkSeg);
        }
    }
}

// ------------------------------------------------------------------------------------- STEPS
// blockIdx.y selects a message of the step, blockIdx.x a tile of the fixed offset grid inside it.
// `first_msg`: plan index of the step's first message (TRACE only).
template <int MAXP, bool TRACE>
__global__ void __launch_bounds__(kThreads)
bcast_step_kernel(const __grid_constant__ RankPtrs<MAXP> bufs, const DevXfer *__restrict__ xfers, long long first_msg,
                  unsigned long long *trace)
{
    const DevXfer x = xfers[blockIdx.y];
    const uint64_t end = x.off + x.len;
    const uint64_t tile = x.off / kStepTile + blockIdx.x;
    const uint64_t lo = max(x.off, tile * kStepTile);
    const uint64_t hi = min(end, (tile + 1) * kStepTile);
    if (lo >= hi) return;
    const uint8_t *s = bufs.p[x.src];
    uint8_t *d = bufs.p[x.dst];
    // head bytes [lo, a0), 16-byte words [a0, a1), tail bytes [a1, hi); offsets are relative to
    // buffers that are themselves 16-byte aligned
    const uint64_t a0 = min((lo + 15) & ~(uint64_t)15, hi);
    const uint64_t a1 = max(hi & ~(uint64_t)15, a0);
    const uint32_t nwords = (uint32_t)((a1 - a0) >> 4), nhead = (uint32_t)(a0 - lo), ntail = (uint32_t)(hi - a1);
    const int tid = threadIdx.x;
    const uint64_t base = a0 + (uint64_t)tid * 16;
    uint32_t lane_bytes = 0;
    uint4 v[kStepWordsPerThread];
#pragma unroll
    for (int u = 0; u < kStepWordsPerThread; u++)
        if ((uint32_t)(tid + u * kThreads) < nwords) v[u] = ld16(s + base + (uint64_t)u * kThreads * 16);
#pragma unroll
    for (int u = 0; u < kStepWordsPerThread; u++)
        if ((uint32_t)(tid + u * kThreads) < nwords) {
            st16(d + base + (uint64_t)u * kThreads * 16, v[u]);
            lane_bytes += 16u;
        }
    if ((uint32_t)tid < nhead) {
        st1(d + lo + tid, ld1(s + lo + tid));
        lane_bytes += 1u;
    } else if ((uint32_t)tid < nhead + ntail) {
        const uint64_t o = a1 + (tid - nhead);
        st1(d + o, ld1(s + o));
        lane_bytes += 1u;
    }
    if constexpr (TRACE) trace_add(trace, (int)(first_msg + blockIdx.y), lane_bytes);
}

}  // namespace bcast_dev
