/*
 * bcast.h -- C ABI of the scatter-ring-allgather broadcast over P virtual ranks whose
 * receive buffers all live in the memory of one GPU.
 *
 * The method is the large-message / medium-message-non-power-of-two broadcast of MPICH as
 * described in "A Bandwidth-saving Optimization for MPI Broadcast Collective Operation"
 * (Zhou, Marjanovic, Niethammer, Gracia): the root's message is cut into P chunks of
 * scatter_size = ceil(nbytes / P) bytes and scattered down a binomial tree (Section III-A,
 * Figs. 1-2); a (P-1)-step ring allgather then completes every rank's buffer, either the
 * NATIVE "enclosed" ring in which every rank receives in every step (Section III-A, Fig. 3)
 * or the TUNED "non-enclosed" ring in which a rank never receives a chunk it already holds
 * from the scatter (Section IV, Figs. 4-5 and the listing).
 *
 * bcast_plan()  turns that control flow into data: an ordered list of messages
 *               (src_rank, dst_rank, chunk, offset, len) grouped into steps, plus per-rank
 *               byte and message counters.  Host only, integers only.
 * bcast_exec()  performs the messages of a plan as device-to-device copies between the P rank
 *               buffers, honouring the step order: a byte is copied out of a rank's buffer only
 *               after the message that delivers it to that rank has been performed.
 *
 * General conventions
 *   - Every function returns BCAST_OK (0) or a negative BCAST_ERR_* code; nothing throws
 *     across this boundary.  bcast_strerror() gives a static string for a code.
 *   - "host" / "device" is stated for every pointer.  Ranks are ABSOLUTE ranks 0..P-1 unless a
 *     field says "relative" (relative rank r = (rank - root + P) mod P, Section IV listing).
 *   - A plan is immutable once created.  It may be executed any number of times; executions of
 *     the same plan may overlap on the GPU if they use different rank buffers (the device-side
 *     tables a plan caches are only read), except in BCAST_EXEC_GRAPH mode, whose captured graph
 *     is bound to one set of buffers at a time.  The first execution of a plan (which builds those
 *     tables) must not race with another call on the same plan; later calls on one plan may come
 *     from several host threads (the plan's host-side caches are locked).  The rank-buffer check
 *     is skipped for the set of pointers that passed it last, on the assumption that those
 *     buffers are still allocated.
 *   - Environment variables override what the library would choose, for experiments and tests
 *     only; they are read when a plan is executed for the first time (the last one at every call):
 *     BCAST_WALK_WORDS (1..8 sixteen-byte words per lane of the register walk, i.e. segments of
 *     512 B .. 4 KiB), BCAST_WALK_BLOCKS_PER_SM, BCAST_WALK_GROUP (neighbouring slices that a block
 *     of the register walk takes at a time), BCAST_BULK_BLOCKS_PER_SM, BCAST_WALK_DUAL (0: walk a
 *     segment that holds a chunk boundary in two parts instead of with the merged list of
 *     bcast_plan_walk_pairing), BCAST_BULK_SPIN_LIMIT (polls of the bulk-copy kernel's first wait
 *     bound, see bcast_exec_status; 0 makes every wait report a timeout and then complete under the
 *     second bound), BCAST_BULK_PLAN_ORDER (1: the bulk walk takes the hops in plan order).
 *   - The library keeps no other global state.  There is no CPU fallback: without a CUDA device
 *     the bcast_exec* calls fail with BCAST_ERR_CUDA.
 */
#ifndef BCAST_B200_H
#define BCAST_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define BCAST_MAX_RANKS 1024 /* largest accepted P */

/* variant: what follows the scatter.  NATIVE / TUNED: the ring allgather of Section III-A / IV.
   DOUBLING: the recursive-doubling allgather that MPICH uses for medium messages on a power-of-two
   number of processes (named in Section I; the standard hypercube exchange): log2 P exchanges, in
   exchange i relative rank r swaps with r xor 2^i the block of 2^i chunks around each of them. */
enum { BCAST_NATIVE = 0, BCAST_TUNED = 1, BCAST_DOUBLING = 2 };
/* phase of a message; BCAST_PHASE_RING is the allgather phase (ring steps, or doubling exchanges).
   The node-aware broadcast (bcast_plan_smp) has two more: the tree broadcast inside the root's node,
   which comes before the scatter, and the tree broadcasts inside the other nodes, which come last. */
enum { BCAST_PHASE_SCATTER = 0, BCAST_PHASE_RING = 1, BCAST_PHASE_NODE_FIRST = 2, BCAST_PHASE_NODE_LAST = 3 };

enum {
    BCAST_OK = 0,
    BCAST_ERR_INVAL = -1,  /* bad argument (range, null, misaligned or overlapping buffers) */
    BCAST_ERR_NOMEM = -2,  /* host or device allocation failed                              */
    BCAST_ERR_CUDA = -3,   /* a CUDA runtime call failed; see bcast_last_cuda_error()       */
    BCAST_ERR_CAPACITY = -4, /* bcast_exec_static only: the plan's tables exceed the built-in scratch */
    BCAST_ERR_TIMEOUT = -5   /* bcast_exec_status only: a bounded wait inside a kernel ran out          */
};

/* How bcast_exec_mode() runs a plan.  All modes perform exactly the plan's messages. */
enum {
    /* One launch for the whole plan.  The message is cut into segments on a fixed grid of byte
       offsets; a warp takes a segment and carries it through every message of the plan that
       covers it (scatter hops and ring hops), re-reading it from the source rank's buffer at
       every hop.  Messages that cover different byte ranges are independent, so no waiting
       between warps is needed.  A segment that holds the boundary between two chunks is carried
       through both chunks' messages at once (bcast_plan_walk_pairing).  The hops of a segment
       run in an order that respects every `dep` of the plan (no copy is read before the message
       that delivers it has been performed) but is not the plan's step order where a different
       order keeps the data in L2: see BCAST_EXEC_WALK_PLAN_ORDER. */
    BCAST_EXEC_WALK = 0,
    /* One launch per plan step (ceil(log2 P) + P - 1 launches) on the caller's stream; inside a
       launch the messages of that step are cut into tiles and copied in parallel. */
    BCAST_EXEC_STEPS = 1,
    /* The same per-step launches, captured once into a CUDA graph and replayed. */
    BCAST_EXEC_GRAPH = 2,
    /* BCAST_EXEC_WALK with the hops of every slice strictly in plan order (all scatter levels,
       then the ring steps in ascending order).  Same copies, same result; in the tuned variant
       the copies the scatter left at inner tree nodes are then re-read from DRAM instead of L2. */
    BCAST_EXEC_WALK_PLAN_ORDER = 3,
    /* BCAST_EXEC_WALK for large messages, with the data moved by the bulk-copy engine (TMA):
       whole 16 KiB segments go global -> shared -> global, one worker thread and one mbarrier per
       segment, twelve segments in flight per SM; segments cut by a chunk boundary are walked through
       registers as in BCAST_EXEC_WALK.  Same copies, same hop order, same result.  Its waits on the
       copy engine are bounded: see bcast_exec_status(). */
    BCAST_EXEC_WALK_BULK = 4,
    /* The fastest of the above for the plan at hand; what bcast_exec() uses.  BCAST_EXEC_WALK_BULK
       for very large messages on many ranks (the bulk walk has at least four rounds of work, about
       116 MB on 148 SMs, and P >= 64) unless the variant is the tuned one (whose hop order re-reads a
       segment up to a tree level later, by which time the bulk path's larger working set has left
       L2); otherwise BCAST_EXEC_WALK. */
    BCAST_EXEC_AUTO = 5
};

/* One message of the schedule.  Plain data, 48 bytes, host memory. */
typedef struct {
    int32_t phase;     /* BCAST_PHASE_SCATTER or BCAST_PHASE_RING                                   */
    int32_t step;      /* scatter: tree level 0..L-1 (L = ceil(log2 P)); ring: i-1 for ring step i;
                          doubling: exchange 0..log2(P)-1                                            */
    int32_t src_rank;  /* absolute rank whose buffer is read                                        */
    int32_t dst_rank;  /* absolute rank whose buffer is written                                     */
    int32_t chunk;     /* RELATIVE index of the (first) chunk carried; chunk c = bytes
                          [min(c*S, nbytes), min((c+1)*S, nbytes)) of the message                    */
    int32_t nchunks;   /* ring: 1; scatter: the destination's own chunk plus its descendants';
                          doubling exchange i: 2^i                                                   */
    uint64_t offset;   /* first byte, the same in the source and the destination buffer             */
    uint64_t len;      /* bytes; 0 for chunks past the end of a short message (still a message)      */
    int64_t dep;       /* index (into the plan's message array) of the message that last wrote this
                          range into src_rank's buffer, -1 if it is the root's original data         */
} bcast_xfer_t;

typedef struct bcast_plan bcast_plan_t; /* opaque; created and freed by the library */

/*
 * bcast_plan -- build the schedule of one broadcast.
 *   Scatter: Section III-A, Figs. 1-2 (binomial tree; L = ceil(log2 P) levels; in level t with
 *   mask m = 2^(L-1-t) every relative rank r that is a multiple of 2m and has r+m < P sends the
 *   chunks [r+m, min(r+2m, P)) to relative rank r+m).  Ring: Section III-A Fig. 3 (native) or
 *   Section IV Figs. 4-5 and listing (tuned): in ring step i = 1..P-1 relative rank r receives
 *   chunk (r-i) mod P from its left neighbour; in the tuned ring only while it still lacks it.
 *   P        number of ranks, 1..BCAST_MAX_RANKS.  P = 1 gives an empty plan.
 *   root     absolute rank that owns the message, 0..P-1
 *   nbytes   message size; 0 is valid (all messages have len 0)
 *   variant  BCAST_NATIVE, BCAST_TUNED, or BCAST_DOUBLING (P must then be a power of two)
 *   out      host pointer that receives the plan; the caller releases it with bcast_plan_free()
 * Messages are ordered by (phase, step, dst_rank); a rank receives at most one message per step.
 * Errors: BCAST_ERR_INVAL (arguments out of range, out == NULL), BCAST_ERR_NOMEM.
 */
int bcast_plan(int P, int root, uint64_t nbytes, int variant, bcast_plan_t **out);

/*
 * bcast_plan_smp -- the node-aware broadcast that MPICH uses for medium messages on a
 * non-power-of-two number of processes (Section II): a binomial-tree broadcast inside the root's
 * node, the scatter-ring-allgather between the nodes, a binomial-tree broadcast inside every other
 * node.  The paper names the three phases and no more; the readings taken here:
 *   - a node is a block of ranks_per_node consecutive absolute ranks (the last one may be smaller);
 *     its leader is its lowest rank;
 *   - first phase (BCAST_PHASE_NODE_FIRST): the binomial tree of Figs. 1-2 over the root's node,
 *     rooted at the root (relative ranks inside the node), the whole message on every edge;
 *   - second phase (BCAST_PHASE_SCATTER, BCAST_PHASE_RING): scatter and native or tuned ring between
 *     the node leaders, nodes numbered relative to the root's node; the message is cut into as many
 *     chunks as there are nodes, scatter_size = ceil(nbytes / nodes);
 *   - third phase (BCAST_PHASE_NODE_LAST): in every other node the same kind of tree from the
 *     leader, all nodes level by level at the same time (a step holds one level of every node).
 *   variant         BCAST_NATIVE or BCAST_TUNED: the ring between the leaders
 *   ranks_per_node  >= 1; 1 gives the schedule of bcast_plan(), >= P a single tree broadcast
 * Messages are ordered by (NODE_FIRST steps, SCATTER steps, RING steps, NODE_LAST steps), inside a
 * step by dst_rank; `chunk` counts chunks of scatter_size bytes, relative to the root's node; `dep`
 * of a whole-message send names the message that last wrote the first chunk into its source.
 * All executors run such a plan like any other.  Errors: as bcast_plan.
 */
int bcast_plan_smp(int P, int root, uint64_t nbytes, int variant, int ranks_per_node, bcast_plan_t **out);

/* Release a plan and the device tables it cached (the device it was executed on must still be
   usable).  NULL is ignored. */
void bcast_plan_free(bcast_plan_t *plan);

/* Read-only views of a plan.  All returned pointers are HOST pointers owned by the plan and
   valid until bcast_plan_free(); a NULL plan (or a bad phase) gives 0 / NULL. */
int32_t bcast_plan_num_ranks(const bcast_plan_t *plan);          /* P                               */
int32_t bcast_plan_root(const bcast_plan_t *plan);
int32_t bcast_plan_variant(const bcast_plan_t *plan);
int32_t bcast_plan_ranks_per_node(const bcast_plan_t *plan);     /* 0 unless made by bcast_plan_smp     */
int32_t bcast_plan_num_chunks(const bcast_plan_t *plan);         /* P, or the number of nodes           */
uint64_t bcast_plan_nbytes(const bcast_plan_t *plan);
uint64_t bcast_plan_scatter_size(const bcast_plan_t *plan);      /* S = ceil(nbytes / num_chunks) (Section IV listing) */
int64_t bcast_plan_num_xfers(const bcast_plan_t *plan);          /* number of messages               */
int32_t bcast_plan_num_steps(const bcast_plan_t *plan);          /* L + (P-1) (doubling: 2L); 0 for P = 1;
                                                                    node-aware: tree levels + L + (nodes-1) + tree levels */
const bcast_xfer_t *bcast_plan_xfers(const bcast_plan_t *plan);  /* [num_xfers], canonical order      */
const int64_t *bcast_plan_step_begin(const bcast_plan_t *plan);  /* [num_steps+1]: messages of step s
                                                                    are [step_begin[s], step_begin[s+1]) */
/* Per-rank counters of one phase, indexed by absolute rank, [P] each.  Message counts include
   zero-length messages (Section IV counts ring messages this way: 56 vs 44 for P = 8). */
const uint64_t *bcast_plan_bytes_sent(const bcast_plan_t *plan, int phase);
const uint64_t *bcast_plan_bytes_recv(const bcast_plan_t *plan, int phase);
const uint64_t *bcast_plan_msgs_sent(const bcast_plan_t *plan, int phase);
const uint64_t *bcast_plan_msgs_recv(const bcast_plan_t *plan, int phase);
uint64_t bcast_plan_total_bytes(const bcast_plan_t *plan);       /* sum of len over all messages      */

/*
 * bcast_exec -- perform a plan's messages on the GPU (Sections III-A and IV: the data movement
 * of the scatter and of the ring allgather; every message is the copy of `len` bytes at `offset`
 * from src_rank's buffer to the same offset of dst_rank's buffer).
 *   rank_bufs    HOST array of P DEVICE pointers, one buffer of at least nbytes bytes per absolute
 *                rank, all on the current device, 16-byte aligned, pairwise disjoint.  The array is
 *                read before the call returns; the buffers stay owned by the caller.
 *   plan         from bcast_plan()
 *   cuda_stream  a cudaStream_t (NULL = the default stream).  The call only enqueues work and
 *                does not synchronise; errors of the kernels themselves surface at the caller's
 *                next synchronisation.
 * On entry rank_bufs[root][0..nbytes) holds the message; other contents are arbitrary.  When the
 * enqueued work has completed, rank_bufs[k][0..nbytes) equals the message for every k and no byte
 * outside those ranges has been written.
 * The first execution of a plan allocates and fills the plan's device tables (cudaMalloc and
 * blocking copies); later executions allocate nothing.
 * Errors: BCAST_ERR_INVAL (NULL arguments, NULL/misaligned/overlapping buffers, a buffer that is not
 * device or managed memory of the current device, a device other than the one the plan was first
 * executed on), BCAST_ERR_NOMEM, BCAST_ERR_CUDA.  Arguments are checked before anything is
 * launched; the extent of a buffer cannot be checked.
 */
int bcast_exec(void *const *rank_bufs, const bcast_plan_t *plan, void *cuda_stream);

/* bcast_exec (which uses BCAST_EXEC_AUTO) with an explicit execution mode; same contract.
   BCAST_EXEC_GRAPH captures and instantiates its graph on the first call and again whenever
   rank_bufs differs from the previous call. */
int bcast_exec_mode(void *const *rank_bufs, const bcast_plan_t *plan, void *cuda_stream, int mode);

/*
 * bcast_exec_host -- the same broadcast for a caller whose data lives in HOST memory.
 *   host_message  HOST pointer to nbytes bytes; copied into rank_bufs[root] first
 *   host_out      HOST array of P HOST pointers (or NULL); after the broadcast the buffer of
 *                 every rank k with host_out[k] != NULL is copied to host_out[k] (nbytes each)
 *   rank_bufs, plan, cuda_stream, mode   as for bcast_exec_mode(); the device buffers are the
 *                 working storage of the P ranks
 * Copies use cudaMemcpyAsync on cuda_stream (pinned host memory makes them asynchronous and
 * fast); the call returns after cudaStreamSynchronize, so on return host_out is filled.
 * Errors: as bcast_exec, plus BCAST_ERR_INVAL for a NULL host_message when nbytes > 0.
 */
int bcast_exec_host(void *const *rank_bufs, const bcast_plan_t *plan, void *cuda_stream, int mode,
                    const void *host_message, void *const *host_out);

/*
 * bcast_exec_static -- bcast_exec for callers that must not allocate device memory.
 * (The paper has no counterpart to this entry point; it exists for the sake of such callers.)
 *
 * Who needs it: programs that hand all device memory to their own pool at start-up and may not
 * call cudaMalloc afterwards (a raw allocation can fail or fragment the pool's address space),
 * services that run under a fixed memory budget, and latency-critical code for which the implicit
 * device-wide synchronisation of cudaMalloc / cudaFree is not acceptable.  bcast_exec() allocates
 * the plan's device tables on a plan's first execution; this call never allocates: it runs the
 * same one-launch WALK kernel, with the tables it needs (slice list, per-chunk hop lists and
 * their offsets) placed in a fixed array of BCAST_STATIC_SCRATCH_BYTES bytes that is part of the
 * library's device image.  Every GPU on which the library is loaded holds that array until the
 * process exits.
 *   rank_bufs, plan, cuda_stream   as for bcast_exec(); inputs and outputs are still the caller's.
 * Behaviour to know about:
 *   - Plans whose tables do not fit (roughly: 8 B per slice of the message -- slices are 512 B to
 *     4 KiB -- plus 4 B per (chunk, message) pair, about 4*P*P bytes, plus, when there is room, 8 B
 *     per (chunk boundary, message) pair for the lists of bcast_plan_walk_pairing) are refused
 *     with BCAST_ERR_CAPACITY before anything is copied or launched.  The call tries, in this
 *     order: everything; without the boundary lists (segments that hold a chunk boundary are then
 *     walked in two parts, which is slower for odd scatter sizes, never wrong); the largest slices.
 *     All configurations up to P = 256 ranks with messages up to 256 MiB fit; P = 1024 does not.
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress) and
 *     remembers it.
 *   - Never call it on a stream that is being captured into a CUDA graph: the call returns
 *     BCAST_ERR_INVAL in that case.  (It copies the tables into the one shared array; recorded into
 *     a graph, that copy would be replayed later from memory that may have changed.)
 *   - Every call re-writes the array (stream-ordered on cuda_stream) from host memory that the plan
 *     keeps, so its previous contents never matter; nothing in it has to start at zero (the kernel
 *     only reads it).  The copy's source is ordinary pageable memory, so the call may block the
 *     host until earlier work on cuda_stream has finished; unlike bcast_exec it is not purely
 *     asynchronous.
 *     Because all calls share the one array, two calls whose GPU work overlaps in time (different
 *     streams, or different host threads) race on it: serialise them.
 *   - The rank buffers are checked like in bcast_exec; the set that passed last is remembered per
 *     device, on the assumption that those buffers stay allocated.
 *   - No cudaMalloc, cudaFree or other allocating CUDA call is made; ordinary host heap memory is
 *     used to assemble the tables (once per plan).
 * Errors: BCAST_ERR_INVAL as for bcast_exec or for a capturing stream, BCAST_ERR_CAPACITY, BCAST_ERR_CUDA.
 */
#define BCAST_STATIC_SCRATCH_BYTES (2u << 20)
int bcast_exec_static(void *const *rank_bufs, const bcast_plan_t *plan, void *cuda_stream);

/*
 * bcast_plan_walk_order -- the order in which BCAST_EXEC_WALK (or BCAST_EXEC_WALK_PLAN_ORDER)
 * performs the messages that move bytes of one chunk.  Host only; needs no GPU.
 *   chunk   relative chunk index 0..P-1
 *   mode    BCAST_EXEC_WALK or BCAST_EXEC_WALK_PLAN_ORDER
 *   out     HOST array of cap entries (may be NULL if cap = 0); receives indices into
 *           bcast_plan_xfers(): every message with len > 0 whose chunk range contains `chunk` and
 *           whose part of it is non-empty, each exactly once
 * Returns the number of such messages (also when it exceeds cap; then only cap are written) or a
 * negative BCAST_ERR_* code.  In both modes a message comes after the message named by its `dep`
 * (Sections III-A and IV: a process can only pass on what it has received).
 */
int64_t bcast_plan_walk_order(const bcast_plan_t *plan, int chunk, int mode, int64_t *out, int64_t cap);

/*
 * bcast_plan_walk_pairing -- how the WALK executors carry the messages of two neighbouring chunks
 * through a segment that holds the boundary between them.  Host only; needs no GPU.
 * Chunks c and c+1 meet inside one 32-byte sector of every rank buffer unless scatter_size is a
 * multiple of 32 (Section IV listing: scatter_size = ceil(nbytes / P), so usually it is not).  One
 * warp takes the whole segment and walks a merged list of slots; a slot holds a message of chunk c,
 * a message of chunk c+1, or one of each.  Inside each chunk the messages keep plan order (so every
 * message still comes after the one named by its `dep`); a slot holds two messages preferably when
 * both write the same rank, because then the sector around the boundary is written in one piece.
 *   chunk   lower chunk c of the boundary, 0..P-2
 *   out     HOST array of 2*cap entries (may be NULL if cap = 0): for slot i, out[2i] is the index
 *           (into bcast_plan_xfers()) of the message of chunk c and out[2i+1] that of chunk c+1,
 *           -1 where the slot has none
 * Returns the number of slots (also when it exceeds cap), 0 if either chunk is empty, or a
 * negative BCAST_ERR_* code.
 */
int64_t bcast_plan_walk_pairing(const bcast_plan_t *plan, int chunk, int64_t *out, int64_t cap);

/*
 * bcast_plan_walk_slices -- the units of work of the WALK executor for segments of words x 512
 * bytes.  Host only; needs no GPU.
 *   words   16-byte words per lane, 1..8
 *   out     HOST array of 3*cap entries (may be NULL if cap = 0): per slice its segment index, its
 *           kind (0: the whole segment, inside one chunk; 1: the bytes of one chunk in a segment
 *           that the chunk does not fill; 2: a whole segment that holds one chunk boundary, see
 *           bcast_plan_walk_pairing) and its (lower) chunk
 * The slices of a plan cover every byte of every non-empty chunk exactly once.  Returns their
 * number (also when it exceeds cap) or a negative BCAST_ERR_* code.
 */
int64_t bcast_plan_walk_slices(const bcast_plan_t *plan, int words, int64_t *out, int64_t cap);

/*
 * bcast_exec_traced -- bcast_exec_mode that also counts, on the device, the bytes it copies for
 * every message of the plan (Sections III-A and IV count messages and their bytes per process;
 * this is the executor's own account of them, as opposed to the planner's).
 *   device_msg_bytes   DEVICE array of bcast_plan_num_xfers() 64-bit counters, zeroed by the
 *                      caller; the kernels add to counter i the bytes they store for message i.
 *                      When the enqueued work has completed, counter i equals xfers[i].len if and
 *                      only if message i was performed in full exactly once.
 *   mode               any mode but BCAST_EXEC_GRAPH
 * Slower than bcast_exec_mode (one atomic per warp and hop); meant for tests and audits.
 * Errors: as bcast_exec_mode, plus BCAST_ERR_INVAL for a NULL counter array or BCAST_EXEC_GRAPH.
 */
int bcast_exec_traced(void *const *rank_bufs, const bcast_plan_t *plan, void *cuda_stream, int mode,
                      uint64_t *device_msg_bytes);

/*
 * ---- The ranks of a plan spread over several GPUs of one NVLink/NVSwitch domain ----------------
 * (Section V measures the broadcast where ring neighbours sit on different nodes; here the P ranks
 * are dealt to G GPUs and a message whose source and destination are on different GPUs crosses
 * NVLink.)  Every rank's buffer lives in the memory of the GPU that owns the rank.  A message is
 * performed by the GPU that owns its destination rank: its kernel loads from the source rank's
 * buffer -- local memory or a peer's, by ordinary peer loads, never a multicast load -- and stores
 * into its own memory.  The work is cut into phases: a hop (message restricted to one chunk) whose
 * source copy was written by another GPU runs one phase after the hop that wrote it; hops inside one
 * GPU keep the order of the one-GPU walk.  Phase k+1 of every GPU is ordered after phase k of all
 * GPUs, by CUDA events between streams (bcast_shard_exec, one process drives all GPUs) or by whatever
 * barrier the caller has between processes (bcast_shard_exec_phase, one process per GPU).  No kernel
 * ever waits for another kernel.
 */
typedef struct bcast_shard bcast_shard_t; /* opaque; created and freed by the library */

/*
 * bcast_shard_create -- partition a plan over num_gpus GPUs.  Host only; needs no GPU.
 *   plan      must outlive the partition
 *   num_gpus  1..P
 *   rank_gpu  HOST array [P]: the GPU (0..num_gpus-1) that owns each absolute rank, or NULL for
 *             contiguous groups (rank r on GPU floor(r * num_gpus / P))
 * Errors: BCAST_ERR_INVAL, BCAST_ERR_NOMEM.
 */
int bcast_shard_create(const bcast_plan_t *plan, int num_gpus, const int32_t *rank_gpu, bcast_shard_t **out);
/* Release a partition and its device tables.  NULL is ignored. */
void bcast_shard_free(bcast_shard_t *shard);

/* Read-only views; HOST pointers owned by the partition. */
int32_t bcast_shard_num_gpus(const bcast_shard_t *shard);
int32_t bcast_shard_num_phases(const bcast_shard_t *shard);          /* 0 for a plan that moves nothing */
const int32_t *bcast_shard_rank_gpu(const bcast_shard_t *shard);     /* [P]                                */
const int32_t *bcast_shard_msg_gpu(const bcast_shard_t *shard);      /* [num_xfers]: GPU that performs it  */
/* [num_xfers]: the phase of a message's hops; last = 0 gives the earliest, last != 0 the latest (they
   differ only for a message whose chunks reached its source in different phases); -1 for a message
   that moves nothing */
const int32_t *bcast_shard_msg_phase(const bcast_shard_t *shard, int last);
/* Bytes (sum of len) and number of the messages whose source and destination ranks are on different
   GPUs: what crosses NVLink.  The tuned ring saves here exactly what it saves in total. */
uint64_t bcast_shard_crossing_bytes(const bcast_shard_t *shard);
int64_t bcast_shard_crossing_msgs(const bcast_shard_t *shard);
/* The messages (indices into bcast_plan_xfers) that GPU `gpu` performs in phase `phase` on the bytes
   of relative chunk `chunk`, in execution order; two-call protocol like bcast_plan_walk_order. */
int64_t bcast_shard_hops(const bcast_shard_t *shard, int phase, int gpu, int chunk, int64_t *out, int64_t cap);

/*
 * bcast_shard_exec -- perform the whole plan from one process that drives all GPUs.
 *   rank_bufs     HOST array of P DEVICE pointers; rank r's buffer must be memory of device
 *                 gpu_device[rank_gpu[r]]; alignment and disjointness as for bcast_exec.  Where the
 *                 devices differ the first call enables peer access between them (BCAST_ERR_INVAL if
 *                 two of them cannot reach each other)
 *   gpu_device    HOST array [num_gpus]: CUDA device ordinal of every GPU of the partition (they may
 *                 repeat: several, or all, "GPUs" of the partition on one device); fixed by the first call
 *   cuda_streams  HOST array [num_gpus] of cudaStream_t, stream g on device gpu_device[g]; streams of
 *                 GPUs mapped to one device may be the same stream or different ones.  The message
 *                 must be in rank_bufs[root] before the work enqueued here starts on the root's GPU
 *                 (enqueue its copy on that GPU's stream, or synchronise first).
 *   device_msg_bytes  NULL, or counters as for bcast_exec_traced, reachable from every device used
 * Asynchronous: when all the streams have been synchronised, every rank buffer holds the message.
 * The first call builds device tables (cudaMalloc) on every device.  Errors: as bcast_exec.
 */
int bcast_shard_exec(bcast_shard_t *shard, void *const *rank_bufs, const int *gpu_device, void *const *cuda_streams,
                     uint64_t *device_msg_bytes);

/*
 * bcast_shard_exec_phase -- enqueue only GPU `gpu`'s kernel of phase `phase`, on the current device
 * and the given stream: the building block for one process per GPU.  The caller runs the phases in
 * ascending order and makes sure that phase k of every GPU has completed before any GPU starts phase
 * k+1 (stream synchronisation plus a barrier between the processes); rank_bufs holds, for ranks owned
 * by other GPUs, pointers through which this device can read their buffers (peer or IPC mappings).
 * A (phase, gpu) pair without work enqueues nothing.  Errors: as bcast_exec.
 */
int bcast_shard_exec_phase(bcast_shard_t *shard, void *const *rank_bufs, int phase, int gpu, void *cuda_stream,
                           uint64_t *device_msg_bytes);

/*
 * bcast_exec_status -- did a kernel of this plan give up on a bounded wait?
 * The bulk-copy kernel (BCAST_EXEC_WALK_BULK) polls an mbarrier for the arrival of every load; the
 * number of polls is limited, so that a copy that never completes ends the kernel instead of
 * hanging the GPU.  A worker whose first limit runs out sets a flag in the plan's device state and
 * goes on waiting under a second, much larger limit (it must not leave while its own copy may still
 * be landing in the block's shared memory); if the load arrives after all, the worker carries on
 * and the rank buffers end up complete; if the second limit runs out too, the worker stops and the
 * rank buffers are incomplete.  Call this after the stream has been synchronised: it reads the flag
 * (a blocking 4-byte copy), clears it, and returns BCAST_ERR_TIMEOUT if it was set, else BCAST_OK.
 * The other executors have no waits and never set it.
 */
int bcast_exec_status(const bcast_plan_t *plan);

/* Number of kernel launches one execution of the plan enqueues in the given mode (0 if nothing
   has to move); a CUDA-graph replay counts the kernels inside the graph. */
int64_t bcast_exec_num_launches(const bcast_plan_t *plan, int mode);

/* Static description of an error code. */
const char *bcast_strerror(int code);

/* The cudaError_t (as int) of the most recent failed CUDA call on this thread, 0 if none. */
int bcast_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* BCAST_B200_H */
