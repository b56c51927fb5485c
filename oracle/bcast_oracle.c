/*
 * bcast_oracle.c -- TEST INFRASTRUCTURE, NOT PART OF THE PRODUCT.
 *
 * A plain, slow, single-threaded CPU simulation of the scatter-ring-allgather
 * broadcast over P simulated processes, each with its own host buffer, written
 * from the paper "A Bandwidth-saving Optimization for MPI Broadcast Collective
 * Operation" (Zhou, Marjanovic, Niethammer, Gracia).  It exists so that tests,
 * the smoke check and the CPU-baseline leg of the benchmark have something to
 * compare the CUDA library against.  It shares no code, header or table with
 * that library, and nothing in the library may call it.
 *
 * What it follows:
 *   - Section III-A (Figs. 1-2):  binomial scatter, the root's message cut into
 *     P chunks of scatter_size = ceil(nbytes / P) bytes.
 *   - Section III-A (Fig. 3):     native "enclosed" ring allgather, P-1 steps,
 *     every process sends and receives in every step.
 *   - Section IV (Figs. 4-5 and the description of the method): tuned
 *     "non-enclosed" ring allgather; each process knows which chunks it owned when
 *     the scatter ended and a transfer of such a chunk to it does not take place.
 *     The (step, flag) pair of the description is read off the simulated behaviour.
 *   - Section I: for medium messages on a power-of-two number of processes MPICH
 *     follows the scatter with a recursive-doubling allgather instead of the ring.
 *     The paper only names it; the exchange pattern simulated here is the standard
 *     one of that algorithm (Thakur, Rabenseifner, Gropp, "Optimization of
 *     Collective Communication Operations in MPICH"): in step i = 0..log2(P)-1 a
 *     process exchanges, with the process whose relative rank differs in bit i, the
 *     block of 2^i chunks that starts at its own relative rank with the low i bits
 *     cleared.  Third variant (2); power-of-two P only.
 *
 *   - Section II: for medium messages on a non-power-of-two number of processes MPICH's
 *     broadcast is aware of the nodes: first a binomial-tree broadcast inside the root's
 *     node, then the scatter-ring-allgather between the nodes, finally a binomial-tree
 *     broadcast inside every other node.  Simulated by oracle_bcast_simulate_smp() with
 *     nodes = blocks of consecutive ranks (see the readings below).
 *
 * The simulation keeps, for every process, the set of chunks it holds; a message
 * is only formed from what its sender holds (checked before anything is copied).
 * No blocking, fusion or reordering: one memcpy per message, steps in the
 * paper's order.
 *
 * Readings taken where the paper is silent (each also listed in the design
 * notes of the repository):
 *   - nbytes = count * length of the listing's signature.
 *   - the opaque binomial_tree() call is the tree of Figs. 1-2: in level t
 *     (mask m = 2^(L-1-t), L = ceil(log2 P)) every relative rank r that is a
 *     multiple of 2m and has r + m < P sends the chunks [r+m, min(r+2m, P))
 *     to relative rank r + m.
 *   - chunk indices and displacements are RELATIVE to the root (the listing
 *     displaces by the relative rank); src/dst ranks are absolute.
 *   - zero-length messages (chunks past the end of a short message) are still
 *     messages: the listing clamps the count to 0 and still makes the call.
 *     Their offset is reported clipped to nbytes.
 *   - inside one step, messages are listed by ascending destination rank.
 *   - a "message transfer" in the paper's 56/44 and 90/75 counts is a ring
 *     message; scatter messages are counted separately.
 *   - node-aware broadcast (Section II names the three phases and nothing else): a node
 *     is a block of ranks_per_node consecutive ranks (the last one may be smaller); a
 *     node's leader is its lowest rank; the first broadcast runs down a binomial tree
 *     rooted at the root over the root's node (relative ranks inside the node, the
 *     tree of Figs. 1-2 with the whole message on every edge); the scatter-ring runs
 *     between the leaders, nodes numbered relative to the root's node, with
 *     scatter_size = ceil(nbytes / number of nodes); the last broadcast runs in every
 *     other node from its leader, all nodes level by level at the same time.
 *
 * Pinned by tests/test_oracle_pins.py against the worked examples of
 * Figs. 1-5, the printed message counts, closed forms, MPI broadcast
 * semantics and a brute-force ownership enumeration; the recursive-doubling
 * variant, for which the paper prints nothing, against the textbook hypercube
 * exchange with explicit ownership sets, its byte budget, and the two-process
 * case where it must coincide with the ring.  Nothing is unpinned.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORC_OK = 0, ORC_E_ARG = -1, ORC_E_NOMEM = -2, ORC_E_CAP = -3,
       ORC_E_NOT_HELD = -4,      /* a sender did not hold what it sends          */
       ORC_E_UNMATCHED = -5,     /* a send without the matching receive          */
       ORC_E_OVERLAP = -7,       /* a step reads a range that the step writes    */
       ORC_E_INCOMPLETE = -8,    /* some process misses a chunk at the end       */
       ORC_E_MISMATCH = -9 };    /* some buffer differs from the root's message  */

/* schedule record: 9 x int64, in this order */
enum { F_PHASE = 0, F_STEP, F_SRC, F_DST, F_CHUNK, F_NCHUNKS, F_OFFSET, F_LEN, F_DEP, F_NFIELDS };
enum { PH_SCATTER = 0, PH_RING = 1, PH_NODE_FIRST = 2, PH_NODE_LAST = 3 };   /* 2, 3: node-aware variant only */
enum { SEND_ONLY = 0, RECV_ONLY = 1 };

typedef struct {
    int P, root;
    int C;                        /* number of chunks the message is cut into (P, or the number of nodes) */
    int G;                        /* size of the group that runs the scatter and the ring ...            */
    const int *member;            /* ... and its processes (absolute ranks) by relative rank, or NULL:
                                     all P processes, relative rank r = absolute rank (r + root) mod P   */
    uint64_t n, S;
    uint8_t *const *buf;          /* NULL: schedule and counters only */
    int64_t *sched, cap, len;
    uint64_t *bytes_sent, *bytes_recv, *msgs_sent, *msgs_recv;   /* [2][P] */
    uint8_t *holds;               /* holds[k*C + c]: process k (absolute) holds chunk c (relative) */
    int *rd_lo, *rd_hi;           /* per process: chunk range read from it in the current step */
    int64_t *writer;              /* writer[k*C + c]: schedule index of the message that last wrote it, -1 = never */
} sim_t;

static uint64_t umin(uint64_t a, uint64_t b) { return a < b ? a : b; }

/* first byte of relative chunk c, clipped to the message (Section IV listing: disp = rel * scatter_size) */
static uint64_t chunk_begin(const sim_t *s, int c) { return umin((uint64_t)c * s->S, s->n); }

/* length of relative chunk c: min(scatter_size, nbytes - c*scatter_size), clamped at 0 (listing) */
static uint64_t chunk_len(const sim_t *s, int c)
{
    uint64_t b = (uint64_t)c * s->S;
    if (b >= s->n) return 0;
    return umin(s->S, s->n - b);
}

/* relative rank r of the group <-> absolute rank */
static int abs_of(const sim_t *s, int r) { return s->member ? s->member[r] : (r + s->root) % s->P; }
static int rel_of(const sim_t *s, int k)
{
    if (!s->member) return k >= s->root ? k - s->root : k - s->root + s->P;
    for (int r = 0; r < s->G; r++)
        if (s->member[r] == k) return r;
    return -1;
}

typedef struct { int src, dst, chunk, nchunks; } pending_t;

static int by_dst(const void *a, const void *b)
{
    return ((const pending_t *)a)->dst - ((const pending_t *)b)->dst;
}

/* Deliver the messages of one step: check, record, count, copy. */
static int deliver_step(sim_t *s, int phase, int step, pending_t *m, int nm)
{
    const int P = s->P, C = s->C;
    qsort(m, (size_t)nm, sizeof *m, by_dst);

    /* a process can only send what has arrived at it in an earlier step */
    for (int a = 0; a < nm; a++)
        for (int c = m[a].chunk; c < m[a].chunk + m[a].nchunks; c++)
            if (!s->holds[(size_t)m[a].src * C + c]) return ORC_E_NOT_HELD;
    /* all sends of a step see the buffers as they were when the step began: nothing a message
       of this step writes may be read by a message of this step, so that copying the messages
       one after the other equals copying them at once */
    for (int k = 0; k < P; k++) s->rd_lo[k] = s->rd_hi[k] = 0;      /* chunk range read from process k */
    for (int a = 0; a < nm; a++) {
        if (s->rd_hi[m[a].src] != s->rd_lo[m[a].src]) return ORC_E_UNMATCHED;   /* one send per process and step */
        s->rd_lo[m[a].src] = m[a].chunk; s->rd_hi[m[a].src] = m[a].chunk + m[a].nchunks;
    }
    for (int a = 0; a < nm; a++)
        if (m[a].chunk < s->rd_hi[m[a].dst] && s->rd_lo[m[a].dst] < m[a].chunk + m[a].nchunks)
            return ORC_E_OVERLAP;

    for (int a = 0; a < nm; a++) {
        const int c0 = m[a].chunk, c1 = c0 + m[a].nchunks;
        const uint64_t off = chunk_begin(s, c0);
        uint64_t len = 0;
        for (int c = c0; c < c1; c++) len += chunk_len(s, c);
        if (s->len + a >= s->cap) return ORC_E_CAP;
        int64_t *rec = s->sched + (s->len + a) * F_NFIELDS;
        rec[F_PHASE] = phase;  rec[F_STEP] = step;
        rec[F_SRC] = m[a].src; rec[F_DST] = m[a].dst;
        rec[F_CHUNK] = c0;     rec[F_NCHUNKS] = m[a].nchunks;
        rec[F_OFFSET] = (int64_t)off; rec[F_LEN] = (int64_t)len;
        rec[F_DEP] = s->writer[(size_t)m[a].src * C + c0];

        s->bytes_sent[(size_t)phase * P + m[a].src] += len;
        s->bytes_recv[(size_t)phase * P + m[a].dst] += len;
        s->msgs_sent[(size_t)phase * P + m[a].src] += 1;
        s->msgs_recv[(size_t)phase * P + m[a].dst] += 1;

        if (s->buf && len) memcpy(s->buf[m[a].dst] + off, s->buf[m[a].src] + off, (size_t)len);
    }
    /* ownership changes only after every message of the step has been read */
    for (int a = 0; a < nm; a++) {
        /* records of this step were appended in the same order as m[] */
        const int64_t idx = s->len + a;
        for (int c = m[a].chunk; c < m[a].chunk + m[a].nchunks; c++) {
            s->holds[(size_t)m[a].dst * C + c] = 1;
            s->writer[(size_t)m[a].dst * C + c] = idx;
        }
    }
    s->len += nm;
    return ORC_OK;
}

/* Section III-A, Figs. 1-2: binomial scatter from relative rank 0 of the group (all P processes,
   or the node leaders of the node-aware variant). */
static int scatter_phase(sim_t *s, int L, pending_t *m)
{
    const int P = s->G;
    for (int t = 0; t < L; t++) {
        const int mask = 1 << (L - 1 - t);
        int nm = 0;
        for (int r = 0; r < P; r += 2 * mask) {          /* roots of the sub-trees alive at this level */
            if (r + mask >= P) continue;                 /* no process there (non-power-of-two P)   */
            const int hi = (r + 2 * mask < P) ? r + 2 * mask : P;
            m[nm].src = abs_of(s, r);
            m[nm].dst = abs_of(s, r + mask);
            m[nm].chunk = r + mask;                      /* the child gets its own chunk ...         */
            m[nm].nchunks = hi - (r + mask);             /* ... and those of all its descendants     */
            nm++;
        }
        int rc = deliver_step(s, PH_SCATTER, t, m, nm);
        if (rc) return rc;
    }
    return ORC_OK;
}

/* Section III-A (Fig. 3) and Section IV (Figs. 4-5): the ring allgather, P-1 steps.
 *
 * Native ("enclosed") ring: in the first step every process passes its own chunk to its right
 * neighbour and takes the left neighbour's; in every later step it passes on what came in the
 * step before.  Every process sends and receives in every step, whatever it already holds.
 *
 * Tuned ("non-enclosed") ring: the same rotation of chunks, but each process knows the set of
 * chunks it owned when the scatter ended (the sets drawn above the processes in Figs. 3-5) and
 * "only receives those missing data chunks": a transfer takes place only if the receiver did not
 * own the chunk then, and its left neighbour does not send it otherwise.  A skipped transfer does
 * not disturb the rotation: the receiver has the chunk anyway and it is what it passes on next.
 *
 * Alongside the messages the phase records, per process, the last step in which it received and
 * the last step in which it sent; step_and_flag() below reads the listing's (step, flag) pair off
 * those.
 */
static int ring_phase(sim_t *s, int tuned, pending_t *m, int *last_recv, int *last_send)
{
    const int P = s->G, C = s->C;                        /* processes on the ring; chunks per process set */
    int rc = ORC_OK;
    uint8_t *owned_after_scatter = malloc((size_t)s->P * (size_t)C);
    int *passes = malloc(sizeof(int) * (size_t)P), *arrives = malloc(sizeof(int) * (size_t)P);
    if (!owned_after_scatter || !passes || !arrives) { rc = ORC_E_NOMEM; goto out; }
    memcpy(owned_after_scatter, s->holds, (size_t)s->P * (size_t)C);
    for (int q = 0; q < P; q++) {                        /* q: position on the ring = relative rank */
        passes[q] = q;                                   /* step 1: the process's own chunk */
        if (last_recv) last_recv[abs_of(s, q)] = 0;
        if (last_send) last_send[abs_of(s, q)] = 0;
    }

    for (int i = 1; i < P; i++) {
        int nm = 0;
        for (int q = 0; q < P; q++) {
            const int k = abs_of(s, q), qr = (q + 1) % P, right = abs_of(s, qr);
            const int chunk = passes[q];
            arrives[qr] = chunk;                         /* due at the right neighbour in this step */
            if (tuned && owned_after_scatter[(size_t)right * C + chunk]) continue;   /* it has that one: nothing is sent */
            m[nm].src = k; m[nm].dst = right; m[nm].chunk = chunk; m[nm].nchunks = 1;
            nm++;
            if (last_send) last_send[k] = i;
            if (last_recv) last_recv[right] = i;
        }
        rc = deliver_step(s, PH_RING, i - 1, m, nm);
        if (rc) goto out;
        for (int q = 0; q < P; q++) passes[q] = arrives[q];   /* forward what was due in this step */
    }
out:
    free(owned_after_scatter); free(passes); free(arrives);
    return rc;
}

/* Section IV, second step of the description ("each process computes out the related step ..."):
 * a process takes part in the two-sided exchange up to ring step P - step and from step
 * P - step + 1 on only sends (flag 0) or only receives (flag 1).  Read off what the process
 * does in the tuned ring: the two-sided part ends with the earlier of its last receive and its
 * last send; the flag says which side goes on afterwards (when the sending side ends first, or
 * both end together, the process is on the receiving side from then on). */
static void step_and_flag(int P, int last_recv, int last_send, int *step, int *flag)
{
    const int two_sided_until = last_recv < last_send ? last_recv : last_send;
    *step = P - two_sided_until;
    *flag = last_send <= last_recv ? RECV_ONLY : SEND_ONLY;
}

/* Section I (named only) -- recursive-doubling allgather after the scatter; P a power of two. */
static int doubling_phase(sim_t *s, pending_t *m)
{
    const int P = s->P;
    int rc = ORC_OK;
    int *wants_from = malloc(sizeof(int) * (size_t)P), *wants_chunk = malloc(sizeof(int) * (size_t)P);
    if (!wants_from || !wants_chunk) { rc = ORC_E_NOMEM; goto out; }
    for (int i = 0, mask = 1; mask < P; i++, mask <<= 1) {
        /* every process posts its receive: from the partner, the partner's current block */
        for (int k = 0; k < P; k++) {
            const int r = rel_of(s, k), partner = r ^ mask;
            wants_from[k] = abs_of(s, partner);
            wants_chunk[k] = (partner >> i) << i;
        }
        /* every process sends its own current block to the partner */
        int nm = 0;
        for (int k = 0; k < P; k++) {
            const int r = rel_of(s, k), partner = abs_of(s, r ^ mask);
            const int my_block = (r >> i) << i;
            if (wants_from[partner] != k || wants_chunk[partner] != my_block) { rc = ORC_E_UNMATCHED; goto out; }
            m[nm].src = k; m[nm].dst = partner; m[nm].chunk = my_block; m[nm].nchunks = mask;
            nm++;
        }
        rc = deliver_step(s, PH_RING, i, m, nm);
        if (rc) goto out;
    }
out:
    free(wants_from); free(wants_chunk);
    return rc;
}

/* Section II: "an intra-node broadcast ... following a binomial tree".  One step of such broadcasts,
 * for several disjoint groups at once: in level t of a group of `size` processes (mask m =
 * 2^(L-1-t), L = ceil(log2 size): the tree of Figs. 1-2) every relative rank r that is a multiple of
 * 2m and has r + m < size passes the WHOLE message (all C chunks) to relative rank r + m.
 * groups[g] lists the processes of group g by relative rank; groups with fewer levels than t+1 are
 * idle.  Returns the number of messages formed (0: no group has a level t), or a negative code. */
static int tree_bcast_step(sim_t *s, int phase, int t, int ngroups, int *const *groups, const int *sizes, pending_t *m)
{
    int nm = 0;
    for (int g = 0; g < ngroups; g++) {
        int L = 0;
        while ((1 << L) < sizes[g]) L++;
        if (t >= L) continue;
        const int mask = 1 << (L - 1 - t);
        for (int r = 0; r + mask < sizes[g]; r += 2 * mask) {
            m[nm].src = groups[g][r];
            m[nm].dst = groups[g][r + mask];
            m[nm].chunk = 0;
            m[nm].nchunks = s->C;
            nm++;
        }
    }
    if (nm == 0) return 0;
    const int rc = deliver_step(s, phase, t, m, nm);
    return rc ? rc : nm;
}

/*
 * Simulate one broadcast.
 *   P, root, nbytes   communicator size, root rank, message bytes
 *   tuned             0: native ring (Section III-A), 1: tuned ring (Section IV),
 *                     2: recursive-doubling allgather in place of the ring (Section I; P must be
 *                        a power of two)
 *   per_node          0: no node awareness (everything above).  >= 1: the node-aware broadcast of
 *                     Section II with nodes of per_node consecutive ranks: binomial-tree broadcast in
 *                     the root's node, scatter + (native or tuned) ring between the node leaders with
 *                     the message cut into as many chunks as there are nodes, binomial-tree
 *                     broadcast in every other node (tuned = 2 is not defined here)
 *   buf               P host buffers of nbytes each; buf[root] holds the message.  NULL: no data is
 *                     moved, only the schedule and the counters are produced.
 *   sched, cap        room for cap records of 9 int64 (phase, step, src, dst, chunk, nchunks,
 *                     offset, len, dep); *nsched receives the number written
 *   bytes_sent ...    four arrays [nphases][P] (phase, absolute rank), zeroed here; nphases is 2
 *                     without node awareness and 4 with it
 * Returns ORC_OK or a negative ORC_E_* code.
 */
static int simulate(int P, int root, uint64_t nbytes, int tuned, int per_node, uint8_t *const *buf,
                    int64_t *sched, int64_t cap, int64_t *nsched,
                    uint64_t *bytes_sent, uint64_t *bytes_recv,
                    uint64_t *msgs_sent, uint64_t *msgs_recv, int *last_recv, int *last_send)
{
    if (P < 1 || root < 0 || root >= P || !sched || !nsched || cap < 0 || per_node < 0 ||
        !bytes_sent || !bytes_recv || !msgs_sent || !msgs_recv)
        return ORC_E_ARG;
    if (tuned < 0 || tuned > 2 || (tuned == 2 && ((P & (P - 1)) != 0 || per_node))) return ORC_E_ARG;

    const int nnodes = per_node ? (P + per_node - 1) / per_node : 0;
    const int C = per_node ? nnodes : P;                      /* chunks: one per process on the ring */
    const int nphases = per_node ? 4 : 2;
    sim_t s;
    memset(&s, 0, sizeof s);
    s.P = P; s.root = root; s.n = nbytes; s.C = C; s.G = P; s.member = NULL;
    s.S = (nbytes + (uint64_t)C - 1) / (uint64_t)C;          /* scatter_size, Section IV listing */
    s.buf = buf; s.sched = sched; s.cap = cap; s.len = 0;
    s.bytes_sent = bytes_sent; s.bytes_recv = bytes_recv; s.msgs_sent = msgs_sent; s.msgs_recv = msgs_recv;
    memset(bytes_sent, 0, sizeof(uint64_t) * (size_t)nphases * (size_t)P);
    memset(bytes_recv, 0, sizeof(uint64_t) * (size_t)nphases * (size_t)P);
    memset(msgs_sent, 0, sizeof(uint64_t) * (size_t)nphases * (size_t)P);
    memset(msgs_recv, 0, sizeof(uint64_t) * (size_t)nphases * (size_t)P);

    int rc = ORC_OK;
    pending_t *m = malloc(sizeof(pending_t) * (size_t)P);
    s.holds = calloc((size_t)P * (size_t)C, 1);
    s.writer = malloc(sizeof(int64_t) * (size_t)P * (size_t)C);
    s.rd_lo = malloc(sizeof(int) * (size_t)P);
    s.rd_hi = malloc(sizeof(int) * (size_t)P);
    int *order = malloc(sizeof(int) * (size_t)P * 2);         /* node-aware: processes by node, leaders */
    int **groups = malloc(sizeof(int *) * (size_t)(nnodes + 1));
    int *sizes = malloc(sizeof(int) * (size_t)(nnodes + 1));
    if (!m || !s.holds || !s.writer || !s.rd_lo || !s.rd_hi || !order || !groups || !sizes) { rc = ORC_E_NOMEM; goto out; }
    for (size_t x = 0; x < (size_t)P * (size_t)C; x++) s.writer[x] = -1;
    for (int c = 0; c < C; c++) s.holds[(size_t)root * C + c] = 1;   /* the root has the whole message */

    if (per_node) {
        /* Section II, first phase: binomial-tree broadcast inside the root's node, rooted at the root */
        const int root_node = root / per_node;
        const int first = root_node * per_node, size = (first + per_node <= P ? per_node : P - first);
        for (int r = 0; r < size; r++) order[r] = first + (root - first + r) % size;    /* relative rank r of the node */
        groups[0] = order; sizes[0] = size;
        for (int t = 0;; t++) {
            rc = tree_bcast_step(&s, PH_NODE_FIRST, t, 1, groups, sizes, m);
            if (rc < 0) goto out;
            if (rc == 0) break;
        }
        /* second phase: scatter and ring between the node leaders (lowest rank of each node),
           nodes numbered relative to the root's node */
        int *leaders = order + P;
        for (int q = 0; q < nnodes; q++) leaders[q] = ((root_node + q) % nnodes) * per_node;
        s.G = nnodes; s.member = leaders;
        /* the leader of the root's node now stands for the root: it holds the whole message */
        for (int c = 0; c < C; c++)
            if (!s.holds[(size_t)leaders[0] * C + c]) { rc = ORC_E_NOT_HELD; goto out; }
    }

    int L = 0;
    while ((1 << L) < s.G) L++;                               /* ceil(log2) scatter levels */

    rc = scatter_phase(&s, L, m);
    if (rc) goto out;
    rc = tuned == 2 ? doubling_phase(&s, m) : ring_phase(&s, tuned, m, last_recv, last_send);
    if (rc) goto out;

    if (per_node) {
        /* third phase: binomial-tree broadcast inside every other node, from its leader, all nodes at once */
        const int root_node = root / per_node;
        int ng = 0;
        for (int node = 0; node < nnodes; node++) {
            if (node == root_node) continue;
            const int first = node * per_node, size = (first + per_node <= P ? per_node : P - first);
            int *list = order + first;                        /* the node's own stretch of `order` (the root's node is done with it) */
            for (int r = 0; r < size; r++) list[r] = first + r;
            groups[ng] = list; sizes[ng] = size; ng++;
        }
        for (int t = 0; ng; t++) {
            rc = tree_bcast_step(&s, PH_NODE_LAST, t, ng, groups, sizes, m);
            if (rc < 0) goto out;
            if (rc == 0) break;
        }
        rc = ORC_OK;
    }

    /* MPI broadcast semantics (Section III-A): on return every process has the root's message */
    for (size_t x = 0; x < (size_t)P * (size_t)C; x++)
        if (!s.holds[x]) { rc = ORC_E_INCOMPLETE; goto out; }
    if (buf && nbytes)
        for (int k = 0; k < P; k++)
            if (memcmp(buf[k], buf[root], (size_t)nbytes) != 0) { rc = ORC_E_MISMATCH; goto out; }
out:
    if (rc > 0) rc = ORC_OK;
    *nsched = s.len;
    free(m); free(s.holds); free(s.writer); free(s.rd_lo); free(s.rd_hi); free(order); free(groups); free(sizes);
    return rc;
}

int oracle_bcast_simulate(int P, int root, uint64_t nbytes, int tuned, uint8_t *const *buf,
                          int64_t *sched, int64_t cap, int64_t *nsched,
                          uint64_t *bytes_sent, uint64_t *bytes_recv,
                          uint64_t *msgs_sent, uint64_t *msgs_recv)
{
    return simulate(P, root, nbytes, tuned, 0, buf, sched, cap, nsched, bytes_sent, bytes_recv,
                    msgs_sent, msgs_recv, NULL, NULL);
}

/* The node-aware broadcast of Section II; counter arrays are [4][P] (phases 0..3, see PH_*). */
int oracle_bcast_simulate_smp(int P, int root, uint64_t nbytes, int tuned, int ranks_per_node, uint8_t *const *buf,
                              int64_t *sched, int64_t cap, int64_t *nsched,
                              uint64_t *bytes_sent, uint64_t *bytes_recv,
                              uint64_t *msgs_sent, uint64_t *msgs_recv)
{
    if (ranks_per_node < 1) return ORC_E_ARG;
    return simulate(P, root, nbytes, tuned, ranks_per_node, buf, sched, cap, nsched, bytes_sent, bytes_recv,
                    msgs_sent, msgs_recv, NULL, NULL);
}

/* scatter_size for the caller's convenience (Section IV listing) */
uint64_t oracle_bcast_scatter_size(int P, uint64_t nbytes)
{
    return P < 1 ? 0 : (nbytes + (uint64_t)P - 1) / (uint64_t)P;
}

/*
 * (step, flag) of every relative rank 0..P-1 in the tuned ring (Section IV), exposed so that tests
 * can pin the pair on its own.  Obtained by simulating the tuned broadcast of a P-byte message
 * from root 0 without data and reading off when each process last received and last sent.
 * P = 1 has no ring: step = 1, flag = RECV_ONLY by the convention of step_and_flag().
 */
int oracle_bcast_step_flag(int P, int *step, int *flag)
{
    if (P < 1 || !step || !flag) return ORC_E_ARG;
    int rc = ORC_E_NOMEM;
    const int64_t cap = (int64_t)P * P + 1;
    int64_t nsched = 0;
    int64_t *sched = malloc(sizeof(int64_t) * F_NFIELDS * (size_t)cap);
    uint64_t *cnt = malloc(sizeof(uint64_t) * 8 * (size_t)P);
    int *last_recv = malloc(sizeof(int) * (size_t)P), *last_send = malloc(sizeof(int) * (size_t)P);
    if (sched && cnt && last_recv && last_send) {
        rc = simulate(P, 0, (uint64_t)P, 1, 0, NULL, sched, cap, &nsched, cnt, cnt + 2 * P, cnt + 4 * P, cnt + 6 * P,
                      last_recv, last_send);
        for (int r = 0; !rc && r < P; r++) step_and_flag(P, last_recv[r], last_send[r], &step[r], &flag[r]);
    }
    free(sched); free(cnt); free(last_recv); free(last_send);
    return rc;
}
