"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU needed).

Each test states which passage of the paper it pins.  None of them re-types the oracle's own
formulas: they use the printed worked examples (tests/golden), closed forms obtained another way
(lowest-set-bit sub-tree sizes, recursive halving), MPI broadcast semantics, and a brute-force
ownership enumeration.
"""
import numpy as np
import pytest

from helpers import golden_lines

NATIVE, TUNED = 0, 1
SCATTER, RING = 0, 1


# ----------------------------------------------------------------------------- independent maths
def lowbit(x):
    return x & -x


def subtree(P, r):
    """Number of chunks relative rank r holds after the scatter: itself and its descendants."""
    return P if r == 0 else min(lowbit(r), P - r)


def halving_tree(lo, hi, out, depth_of_mask, L):
    """Binomial scatter by recursive halving: the owner `lo` of chunks [lo, hi) gives the upper part
    to the process in the middle, at the level that belongs to the distance between them."""
    size = hi - lo
    if size <= 1:
        return
    h = 1
    while h * 2 < size:
        h *= 2
    out.append((L - 1 - depth_of_mask[h], lo, lo + h, tuple(range(lo + h, hi))))
    halving_tree(lo + h, hi, out, depth_of_mask, L)
    halving_tree(lo, lo + h, out, depth_of_mask, L)


def brute_force(P):
    """Relative-rank messages of scatter, native ring and tuned ring by explicit chunk ownership."""
    L = (P - 1).bit_length()
    depth = {1 << b: b for b in range(L + 1)}
    scatter = []
    halving_tree(0, P, scatter, depth, L)
    scatter.sort()
    holds = [set() for _ in range(P)]
    holds[0] = set(range(P))
    for level, src, dst, chunks in scatter:
        assert set(chunks) <= holds[src]
        holds[dst] |= set(chunks)
    after_scatter = [set(h) for h in holds]
    native, tuned = [], []
    carry = list(range(P))                    # step 1: everyone passes on its own chunk
    for i in range(1, P):
        arriving = [carry[(r - 1) % P] for r in range(P)]
        for r in range(P):
            c = arriving[r]
            assert c in holds[(r - 1) % P]    # the sender really has it
            native.append((i, (r - 1) % P, r, c))
            if c not in holds[r]:             # useful transfer: the receiver lacks the chunk
                tuned.append((i, (r - 1) % P, r, c))
        for r in range(P):
            holds[r].add(arriving[r])
        carry = arriving                      # steps 2..P-1: forward what came in
    assert all(h == set(range(P)) for h in holds)
    return scatter, after_scatter, native, tuned


def rel_rows(res, phase):
    """Oracle schedule rows of one phase as relative-rank tuples (step1based, src, dst, chunk, nchunks)."""
    P, root = res.P, res.root
    rows = res.phase_rows(phase)
    return [(int(s) + 1, (int(a) - root) % P, (int(b) - root) % P, int(c), int(nc))
            for _, s, a, b, c, nc, *_ in rows]


# ----------------------------------------------------------------------------- worked examples
@pytest.mark.parametrize("P,fixture", [(8, "fig1_scatter_p8.txt"), (10, "fig2_scatter_p10.txt")])
def test_scatter_worked_examples(oracle, P, fixture):
    """Section III-A, Figs. 1-2: who sends which chunk set to whom in which scatter step."""
    want = sorted((int(s), int(a), int(b), tuple(int(c) for c in cs.split(",")))
                  for s, a, b, cs in golden_lines(fixture))
    res = oracle.simulate(P, 0, 4 * P, NATIVE)
    got = sorted((s, a, b, tuple(range(c, c + nc))) for s, a, b, c, nc in rel_rows(res, SCATTER))
    assert got == want
    assert max(s for s, *_ in got) == (P - 1).bit_length()        # ceil(log2 P) steps


@pytest.mark.parametrize("P,fixture", [(8, "fig4_tuned_ring_p8.txt"), (10, "fig5_tuned_ring_p10.txt")])
def test_tuned_ring_worked_examples(oracle, P, fixture):
    """Section IV, Figs. 4-5: printed message counts and the per-process receive narratives."""
    nat = rel_rows(oracle.simulate(P, 0, 4 * P, NATIVE), RING)
    tun = rel_rows(oracle.simulate(P, 0, 4 * P, TUNED), RING)
    for key, *val in golden_lines(fixture):
        if key == "native_messages":
            assert len(nat) == int(val[0])
        elif key == "tuned_messages":
            assert len(tun) == int(val[0])
        elif key == "steps":
            assert max(s for s, *_ in tun) == int(val[0]) == max(s for s, *_ in nat)
        elif key == "recv_none":
            assert not [m for m in tun if m[2] == int(val[0])]
        elif key == "recv_seq":
            proc, seq = int(val[0]), [int(c) for c in val[1].split(",")]
            mine = sorted(m for m in tun if m[2] == proc)
            assert [m[3] for m in mine] == seq
            assert [m[0] for m in mine] == list(range(1, len(seq) + 1))   # consecutive steps from step 1
        elif key == "last_recv_step":
            proc = int(val[0])
            assert max(m[0] for m in tun if m[2] == proc) == int(val[1])
        else:
            raise AssertionError(key)


def test_native_ring_shape(oracle):
    """Section III-A, Fig. 3: P messages in each of the P-1 steps; step 1 passes the own chunk to the
    right neighbour, later steps forward what arrived the step before."""
    for P in (2, 3, 5, 8, 10, 13):
        nat = rel_rows(oracle.simulate(P, 0, 3 * P + 1, NATIVE), RING)
        assert len(nat) == P * (P - 1)
        for i in range(1, P):
            step = [m for m in nat if m[0] == i]
            assert len(step) == P
            assert sorted(m[2] for m in step) == list(range(P))
            assert all(m[2] == (m[1] + 1) % P and m[4] == 1 for m in step)
        first = {m[1]: m[3] for m in nat if m[0] == 1}
        assert first == {r: r for r in range(P)}
        got = {(m[0], m[2]): m[3] for m in nat}
        sent = {(m[0], m[1]): m[3] for m in nat}
        for i in range(2, P):
            for r in range(P):
                assert sent[(i, r)] == got[(i - 1, r)]


# ----------------------------------------------------------------------------- brute force
@pytest.mark.parametrize("P", list(range(1, 17)) + [24, 33])
def test_against_brute_force_ownership(oracle, P):
    """Sections III-A and IV: the scatter leaves every process with its own chunk and those of its
    descendants; the tuned ring is the native ring minus exactly the transfers whose receiver
    already holds the chunk (no useful transfer dropped, no useless one kept)."""
    scatter, after_scatter, native, tuned = brute_force(P)
    for r in range(P):
        assert after_scatter[r] == set(range(r, r + subtree(P, r)))
    nat = oracle.simulate(P, 0, 5 * P + 3, NATIVE)
    tun = oracle.simulate(P, 0, 5 * P + 3, TUNED)
    want_sc = sorted((lvl + 1, a, b, cs[0], len(cs)) for lvl, a, b, cs in scatter)
    assert sorted(rel_rows(nat, SCATTER)) == want_sc
    assert sorted(rel_rows(tun, SCATTER)) == want_sc
    assert sorted(rel_rows(nat, RING)) == sorted((i, a, b, c, 1) for i, a, b, c in native)
    assert sorted(rel_rows(tun, RING)) == sorted((i, a, b, c, 1) for i, a, b, c in tuned)
    assert len(native) - len(tuned) == sum(subtree(P, r) for r in range(P)) - P if P > 1 else True


# ----------------------------------------------------------------------------- closed forms
@pytest.mark.parametrize("P", [2, 3, 7, 8, 10, 12, 16, 24, 33, 64, 100, 128, 255, 256])
def test_message_count_closed_forms(oracle, P):
    """Ring message counts: native P(P-1) (Section III-A); tuned P^2 - sum of sub-tree sizes, which
    for a power of two is P(P-1) - (P/2) log2 P (Section IV: 56-12 for P=8)."""
    nat = oracle.simulate(P, P - 1, 12288, NATIVE)
    tun = oracle.simulate(P, P - 1, 12288, TUNED)
    sigma = sum(subtree(P, r) for r in range(P))
    assert len(nat.phase_rows(RING)) == P * (P - 1)
    assert len(tun.phase_rows(RING)) == P * P - sigma
    assert len(nat.phase_rows(SCATTER)) == len(tun.phase_rows(SCATTER)) == P - 1
    if P & (P - 1) == 0:
        lg = P.bit_length() - 1
        assert P * (P - 1) - len(tun.phase_rows(RING)) == (P // 2) * lg


def test_step_flag_closed_form(oracle):
    """Section IV, the (step, flag) pair: what the oracle reads off its simulated tuned ring agrees
    with the sub-tree-size closed form (which is what the listing's mask loop evaluates to) for
    every relative rank of every P <= 300 (and a few larger P)."""
    for P in list(range(2, 301)) + [511, 512, 513, 1000, 1024]:
        pairs = oracle.step_flags(P)
        for r in range(P):
            step, flag = pairs[r]
            if r == 0:
                assert (step, flag) == (P, oracle.SEND_ONLY)
            elif r == P - 1:
                assert (step, flag) == (P, oracle.RECV_ONLY)
            elif r % 2 == 0:
                assert (step, flag) == (subtree(P, r), oracle.SEND_ONLY)
            else:
                assert (step, flag) == (subtree(P, r + 1), oracle.RECV_ONLY)


CASES = [(8, 0, 1 << 20), (12, 5, 256 << 10), (64, 17, (16 << 20) + 13), (100, 63, 64 << 20),
         (255, 254, 12 << 10), (7, 6, 512 << 10), (33, 32, 4 << 20), (3, 1, 5), (5, 2, 3), (4, 0, 0)]


@pytest.mark.parametrize("P,root,n", CASES)
def test_byte_budget(oracle, P, root, n):
    """Every byte of every non-root buffer is written exactly once by scatter + tuned ring, so the
    tuned total is (P-1)*nbytes; the native ring alone already moves (P-1)*nbytes (each of its P-1
    steps moves every chunk once) and the scatter comes on top.  Per process: Section IV's point
    that a process only receives the chunks it lacks."""
    nat = oracle.simulate(P, root, n, NATIVE)
    tun = oracle.simulate(P, root, n, TUNED)
    S = -(-n // P)
    assert nat.scatter_size == tun.scatter_size == S

    def span(a, b):                       # bytes of chunks [a, b)
        return min(b * S, n) - min(a * S, n)
    scatter_bytes = sum(span(r, r + subtree(P, r)) for r in range(1, P))
    assert int(nat.col("len")[nat.col("phase") == SCATTER].sum()) == scatter_bytes
    assert int(nat.col("len")[nat.col("phase") == RING].sum()) == (P - 1) * n
    assert int(tun.col("len").sum()) == (P - 1) * n
    for k in range(P):
        r = (k - root) % P
        own = span(r, r + subtree(P, r))
        assert int(tun.bytes_recv[:, k].sum()) == (0 if r == 0 else n)
        assert int(tun.bytes_recv[RING, k]) == n - own
        assert int(nat.bytes_recv[RING, k]) == n - span(r, r + 1)
        assert int(nat.bytes_recv[SCATTER, k]) == (0 if r == 0 else own)
    for res in (nat, tun):
        assert res.bytes_sent.sum() == res.bytes_recv.sum() == res.col("len").sum()
        assert res.msgs_sent.sum() == res.msgs_recv.sum() == len(res.schedule)
        # counters agree with the schedule, rank by rank
        for ph in (SCATTER, RING):
            rows = res.phase_rows(ph)
            for k in range(P):
                assert int(res.bytes_sent[ph, k]) == int(rows[rows[:, 2] == k][:, 7].sum())
                assert int(res.bytes_recv[ph, k]) == int(rows[rows[:, 3] == k][:, 7].sum())
                assert int(res.msgs_sent[ph, k]) == int((rows[:, 2] == k).sum())
                assert int(res.msgs_recv[ph, k]) == int((rows[:, 3] == k).sum())


# ----------------------------------------------------------------------------- semantics
@pytest.mark.parametrize("P,root,n", [(1, 0, 100), (2, 1, 1), (3, 0, 2), (5, 3, 4), (8, 0, 1 << 12),
                                      (10, 7, 12345), (12, 5, 1 << 14), (16, 15, 65521), (33, 8, 100003),
                                      (255, 254, 12288), (64, 17, 262145 * 2 + 7), (7, 2, 0)])
@pytest.mark.parametrize("variant", [NATIVE, TUNED])
def test_broadcast_semantics(oracle, P, root, n, variant):
    """Section III-A: after the broadcast every process holds the root's message; nothing else is
    touched (chunk ranges tile [0, nbytes) and never reach past it)."""
    rng = np.random.default_rng(P * 1000 + root)
    msg = rng.integers(0, 256, size=n, dtype=np.uint8)
    res = oracle.simulate(P, root, n, variant, message=msg)
    assert res.bufs.shape == (P, n)
    assert (res.bufs == msg[None, :]).all()
    S = res.scatter_size
    off, ln, ch, nch = res.col("offset"), res.col("len"), res.col("chunk"), res.col("nchunks")
    assert ((off + ln) <= n).all() and (off >= 0).all() and (ln >= 0).all()
    assert (off == np.minimum(ch * S, n)).all()
    assert (off + ln == np.minimum((ch + nch) * S, n)).all()
    assert ((ch >= 0) & (ch + nch <= P)).all()


def test_schedule_geometry(oracle):
    """Chunk c is bytes [min(cS, n), min((c+1)S, n)) with S = ceil(n / P) (Section IV listing); a
    message carries whole chunks, never reaches past the message, and empty chunks still give
    messages (of length 0, offset clipped to n)."""
    for P, root, n, variant in [(8, 0, 4096, TUNED), (12, 5, 262144, NATIVE), (255, 254, 12288, TUNED),
                                (10, 9, 7, NATIVE), (5, 2, 0, TUNED), (64, 17, (16 << 20) + 13, TUNED)]:
        res = oracle.simulate(P, root, n, variant)
        S = -(-n // P)
        assert res.scatter_size == S
        off, ln, ch, nch = res.col("offset"), res.col("len"), res.col("chunk"), res.col("nchunks")
        assert ((off + ln) <= n).all() and (off >= 0).all() and (ln >= 0).all()
        assert (off == np.minimum(ch * S, n)).all()
        assert (off + ln == np.minimum((ch + nch) * S, n)).all()
        assert ((ch >= 0) & (nch >= 1) & (ch + nch <= P)).all()
        assert (res.msgs_recv.sum(axis=0)[[k for k in range(P) if k != root]] >= 1).all() or P == 1


def test_validity_of_every_send(oracle):
    """A chunk is sent only after it has arrived at the sender: replay the schedule in order and
    check holdings; `dep` names the message that last delivered the chunk to the sender (-1: the
    root's original data) and always lies in an earlier step."""
    for P, root, variant in [(8, 0, TUNED), (10, 3, TUNED), (12, 5, NATIVE), (13, 12, TUNED), (16, 1, NATIVE)]:
        res = oracle.simulate(P, root, 7 * P + 2, variant)
        holds = {(root, c): -1 for c in range(P)}
        sched = res.schedule
        key_of = lambda row: (int(row[0]), int(row[1]))
        i = 0
        while i < len(sched):
            j = i
            while j < len(sched) and key_of(sched[j]) == key_of(sched[i]):
                j += 1
            for x in range(i, j):               # all sends of a step read the state before the step
                ph, st, src, dst, c, nc, off, ln, dep = (int(v) for v in sched[x])
                for cc in range(c, c + nc):
                    assert (src, cc) in holds
                assert dep == holds[(src, c)]
                assert dep < i
            for x in range(i, j):
                ph, st, src, dst, c, nc, off, ln, dep = (int(v) for v in sched[x])
                for cc in range(c, c + nc):
                    holds[(dst, cc)] = x
            i = j
        assert len(holds) == P * P


def test_canonical_order(oracle):
    """Messages are listed by (phase, step, destination rank); a process receives at most one
    message per step, so the order is total."""
    for P, root, variant in [(12, 5, TUNED), (12, 5, NATIVE), (33, 32, TUNED)]:
        sch = oracle.simulate(P, root, 1000, variant).schedule
        keys = [(int(r[0]), int(r[1]), int(r[3])) for r in sch]
        assert keys == sorted(keys) and len(set(keys)) == len(keys)


def test_tuned_is_subset_of_native(oracle):
    """The tuned ring uses the same steps as the native ring and only leaves transfers out
    (Section IV); byte for byte it never moves more."""
    for P, root, n in [(8, 0, 1 << 16), (12, 5, 262144), (24, 23, 12288), (100, 63, 1 << 20)]:
        nat = oracle.simulate(P, root, n, NATIVE)
        tun = oracle.simulate(P, root, n, TUNED)
        strip = lambda res: {tuple(int(v) for v in r[:8]) for r in res.schedule}
        assert strip(tun) <= strip(nat)
        assert (tun.bytes_recv <= nat.bytes_recv).all() and (tun.bytes_sent <= nat.bytes_sent).all()
        assert (tun.msgs_recv <= nat.msgs_recv).all() and (tun.msgs_sent <= nat.msgs_sent).all()


def test_root_rotation(oracle):
    """Relative ranks (Section IV listing): the schedule for root rho is the schedule for root 0 with
    every rank rotated by rho; chunk indices, offsets and lengths do not change."""
    P, n = 12, 256 << 10
    for variant in (NATIVE, TUNED):
        base = oracle.simulate(P, 0, n, variant)
        base_rows = sorted(tuple(int(v) for v in r[:8]) for r in base.schedule)
        for root in range(P):
            res = oracle.simulate(P, root, n, variant)
            rows = sorted((int(r[0]), int(r[1]), (int(r[2]) - root) % P, (int(r[3]) - root) % P,
                           int(r[4]), int(r[5]), int(r[6]), int(r[7])) for r in res.schedule)
            assert rows == base_rows
            assert (np.roll(res.bytes_recv, -root, axis=1) == base.bytes_recv).all()
            assert (np.roll(res.msgs_sent, -root, axis=1) == base.msgs_sent).all()


def test_degenerate_inputs(oracle):
    """P = 1 moves nothing; nbytes = 0 keeps every message with length 0; nbytes < P leaves the
    trailing chunks empty but still scheduled."""
    r = oracle.simulate(1, 0, 1000, TUNED, message=np.arange(1000, dtype=np.uint8) % 251)
    assert len(r.schedule) == 0
    r = oracle.simulate(6, 2, 0, TUNED, message=np.zeros(0, dtype=np.uint8))
    assert len(r.schedule) == 5 + (36 - sum(subtree(6, x) for x in range(6))) and r.col("len").sum() == 0
    r = oracle.simulate(255, 254, 12288, NATIVE)
    assert r.scatter_size == 49
    lens = {int(c): int(l) for c, l, nc in zip(r.col("chunk"), r.col("len"), r.col("nchunks")) if nc == 1}
    assert lens[250] == 38 and all(lens[c] == 0 for c in range(251, 255)) and lens[249] == 49
    with pytest.raises(oracle.OracleError):
        oracle.simulate(4, 4, 10, TUNED)
    with pytest.raises(oracle.OracleError):
        oracle.simulate(0, 0, 10, TUNED)


# ----------------------------------------------------------------------------- recursive doubling
DOUBLING = 2


def test_doubling_equals_ring_for_two_processes(oracle):
    """With two processes the one exchange of recursive doubling is the one step of the ring (each
    sends its own chunk to the other): the schedules must be identical, `dep` included."""
    for root, n in ((0, 10), (1, 10), (1, 1), (0, 4097)):
        a = oracle.simulate(2, root, n, NATIVE)
        b = oracle.simulate(2, root, n, DOUBLING)
        assert np.array_equal(a.schedule, b.schedule)
        assert np.array_equal(a.bytes_recv, b.bytes_recv) and np.array_equal(a.msgs_sent, b.msgs_sent)


@pytest.mark.parametrize("P", [1, 2, 4, 8, 16, 32, 64, 256])
def test_doubling_against_textbook_hypercube_exchange(oracle, P):
    """Section I names the recursive-doubling allgather; its textbook definition: in step i every
    process exchanges with the process whose (relative) rank differs in bit i everything both have
    gathered so far, i.e. the aligned block of 2^i chunks around each of them, so that after step i
    every process holds the aligned block of 2^(i+1) chunks around itself.  Checked with explicit
    ownership sets on top of the scatter's holdings."""
    root, n = P // 3, 11 * P + 5
    res = oracle.simulate(P, root, n, DOUBLING)
    lg = P.bit_length() - 1
    rows = rel_rows(res, RING)
    assert len(rows) == P * lg
    holds = [set(range(r, r + subtree(P, r))) for r in range(P)]
    for i in range(lg):
        step = [m for m in rows if m[0] == i + 1]
        assert len(step) == P
        assert sorted(m[2] for m in step) == list(range(P))        # everybody receives once
        arriving = {}
        for _, src, dst, c, nc in step:
            assert dst == src ^ (1 << i)                           # partner differs in bit i
            block = set(range(c, c + nc))
            assert block == set(range((src >> i) << i, ((src >> i) << i) + (1 << i)))
            assert block <= holds[src]                             # the sender has gathered it
            arriving[dst] = block
        for r in range(P):
            holds[r] |= arriving[r]
            lo = (r >> (i + 1)) << (i + 1)
            assert set(range(lo, lo + (2 << i))) <= holds[r]
    assert all(h == set(range(P)) for h in holds)


@pytest.mark.parametrize("P,root,n", [(4, 1, 3), (8, 0, 1 << 20), (16, 15, 65521), (64, 17, (16 << 20) + 13), (256, 255, 12288)])
def test_doubling_byte_budget_and_semantics(oracle, P, root, n, with_data=True):
    """Every process receives, over the log2 P exchanges, each chunk but its own exactly once: n minus
    its own chunk's bytes, (P-1)*n in total for the phase -- as many bytes as the native ring moves,
    in log2 P steps instead of P-1.  With data: every buffer ends up equal to the root's message."""
    small = with_data and n <= (1 << 20)
    msg = np.random.default_rng(P).integers(0, 256, size=n, dtype=np.uint8) if small else None
    res = oracle.simulate(P, root, n, DOUBLING, message=msg)
    S = -(-n // P)

    def span(a, b):
        return min(b * S, n) - min(a * S, n)
    assert int(res.col("len")[res.col("phase") == RING].sum()) == (P - 1) * n
    for k in range(P):
        r = (k - root) % P
        assert int(res.bytes_recv[RING, k]) == n - span(r, r + 1)
        assert int(res.bytes_sent[RING, k]) == sum(span((r >> i) << i, ((r >> i) << i) + (1 << i)) for i in range(P.bit_length() - 1))
        assert int(res.msgs_recv[RING, k]) == int(res.msgs_sent[RING, k]) == P.bit_length() - 1
    nat = oracle.simulate(P, root, n, NATIVE)
    assert np.array_equal(res.phase_rows(SCATTER), nat.phase_rows(SCATTER))      # same scatter
    if small:
        assert (res.bufs == msg[None, :]).all()


def test_doubling_needs_power_of_two(oracle):
    for P in (3, 6, 12, 100, 255):
        with pytest.raises(oracle.OracleError):
            oracle.simulate(P, 0, 1000, DOUBLING)
    with pytest.raises(oracle.OracleError):
        oracle.simulate(8, 0, 1000, 3)


def test_doubling_root_rotation_and_validity(oracle):
    P, n = 16, 12345
    base = oracle.simulate(P, 0, n, DOUBLING)
    base_rows = sorted(tuple(int(v) for v in r[:8]) for r in base.schedule)
    for root in range(P):
        res = oracle.simulate(P, root, n, DOUBLING)
        rows = sorted((int(r[0]), int(r[1]), (int(r[2]) - root) % P, (int(r[3]) - root) % P,
                       int(r[4]), int(r[5]), int(r[6]), int(r[7])) for r in res.schedule)
        assert rows == base_rows
        keys = [(int(r[0]), int(r[1]), int(r[3])) for r in res.schedule]
        assert keys == sorted(keys) and len(set(keys)) == len(keys)
        for x, row in enumerate(res.schedule):
            assert -1 <= int(row[8]) < x


# ----------------------------------------------------------------------------- node-aware broadcast
# Section II: tree broadcast in the root's node, scatter-ring between the nodes, tree broadcast in the
# other nodes.  The paper prints no worked example for it, so the pins are structural: the trees
# against recursive halving (the tree of Figs. 1-2, pinned above, carrying the whole message), the
# part between the nodes against the plain schedule of as many processes as there are nodes (pinned
# above by Figs. 1-5), explicit holder sets, byte budgets and MPI semantics.
NODE_FIRST, NODE_LAST = 2, 3
SMP_CASES = [(12, 5, 1000, 4), (12, 0, 4096, 3), (10, 7, 777, 3), (24, 13, 24 * 100 + 1, 6), (9, 2, 64, 4), (16, 15, 5000, 4),
             (7, 3, 50, 2), (33, 20, 33 * 31, 8), (6, 5, 3, 5)]


def tree_by_halving(members):
    """(level, src, dst) of a binomial broadcast over `members` (relative rank order), by recursive halving."""
    size = len(members)
    if size <= 1:
        return set()
    L = (size - 1).bit_length()
    depth = {1 << b: b for b in range(L + 1)}
    edges = []
    halving_tree(0, size, edges, depth, L)
    return {(level, members[src], members[dst]) for level, src, dst, _ in edges}


@pytest.mark.parametrize("P,root,n,c", SMP_CASES)
def test_node_aware_structure(oracle, P, root, n, c):
    nodes = [list(range(f, min(f + c, P))) for f in range(0, P, c)]
    k = len(nodes)
    root_node = root // c
    leaders = [nd[0] for nd in nodes]
    S = -(-n // k)
    for variant in (NATIVE, TUNED):
        res = oracle.simulate(P, root, n, variant, ranks_per_node=c)
        assert res.scatter_size == S
        sch = res.schedule
        phase = sch[:, 0]
        # the phases come in the order of Section II: first tree, scatter, ring, last trees
        order = [int(p) for i, p in enumerate(phase) if i == 0 or p != phase[i - 1]]
        assert order == [p for p in (NODE_FIRST, SCATTER, RING, NODE_LAST) if (phase == p).any()]
        # first tree: over the root's node, rooted at the root, the whole message on every edge
        rn = nodes[root_node]
        members = [rn[(rn.index(root) + r) % len(rn)] for r in range(len(rn))]
        first = sch[phase == NODE_FIRST]
        assert {(int(r[1]), int(r[2]), int(r[3])) for r in first} == tree_by_halving(members)
        assert (first[:, 4] == 0).all() and (first[:, 5] == k).all() and (first[:, 6] == 0).all() and (first[:, 7] == n).all()
        # last trees: in every other node from its lowest rank, all nodes level by level together
        want = set()
        for i, nd in enumerate(nodes):
            if i != root_node:
                want |= tree_by_halving(nd)
        last = sch[phase == NODE_LAST]
        assert {(int(r[1]), int(r[2]), int(r[3])) for r in last} == want
        assert (last[:, 7] == n).all() and (last[:, 5] == k).all()
        # between the nodes only leaders talk
        inter = sch[(phase == SCATTER) | (phase == RING)]
        assert set(inter[:, 2].tolist()) | set(inter[:, 3].tolist()) <= set(leaders)
        # holder sets: nothing is sent that has not arrived; in the end everybody holds every chunk
        holds = [set() for _ in range(P)]
        holds[root] = set(range(k))
        i = 0
        while i < len(sch):
            j = i
            while j < len(sch) and (sch[j, 0], sch[j, 1]) == (sch[i, 0], sch[i, 1]):
                j += 1
            for row in sch[i:j]:
                assert set(range(int(row[4]), int(row[4] + row[5]))) <= holds[int(row[2])]
            for row in sch[i:j]:
                holds[int(row[3])] |= set(range(int(row[4]), int(row[4] + row[5])))
            i = j
        assert all(h == set(range(k)) for h in holds)
        # byte budget
        assert int(first[:, 7].sum()) == (len(rn) - 1) * n
        assert int(last[:, 7].sum()) == sum(len(nd) - 1 for i, nd in enumerate(nodes) if i != root_node) * n
        if variant == TUNED:
            assert int(inter[:, 7].sum()) == (k - 1) * n             # every other leader receives the message once
            assert int(sch[:, 7].sum()) == (P - 1) * n               # and every process but the root, in total
            per_rank = np.bincount(sch[:, 3], weights=sch[:, 7], minlength=P)
            assert all(int(per_rank[r]) == (0 if r == root else n) for r in range(P))
        for ph in range(4):
            rows = sch[phase == ph]
            assert np.array_equal(res.bytes_recv[ph], np.bincount(rows[:, 3], weights=rows[:, 7], minlength=P).astype(np.uint64))
            assert np.array_equal(res.msgs_sent[ph], np.bincount(rows[:, 2], minlength=P).astype(np.uint64))
    # data
    msg = np.random.default_rng(P * 1000 + c).integers(0, 256, size=n, dtype=np.uint8)
    res = oracle.simulate(P, root, n, TUNED, message=msg, ranks_per_node=c)
    assert (res.bufs == msg[None, :]).all()


def test_node_aware_leader_ring_is_the_plain_ring_of_the_nodes(oracle):
    """With P = c * k, what happens between the nodes is the plain scatter-ring of k processes
    (the one Figs. 1-5 pin), process j standing for the leader of node j."""
    for c, k, root, n in [(4, 8, 13, 8 * 512 + 3), (3, 10, 29, 10 * 100), (2, 12, 0, 4099), (5, 3, 7, 100)]:
        P = c * k
        for variant in (NATIVE, TUNED):
            smp = oracle.simulate(P, root, n, variant, ranks_per_node=c)
            plain = oracle.simulate(k, root // c, n, variant)
            inter = smp.schedule[(smp.schedule[:, 0] == SCATTER) | (smp.schedule[:, 0] == RING)]
            assert len(inter) == len(plain.schedule)
            a = inter.copy()
            a[:, 2] //= c
            a[:, 3] //= c
            assert (inter[:, 2] % c == 0).all() and (inter[:, 3] % c == 0).all()
            assert np.array_equal(a[:, :8], plain.schedule[:, :8])          # all but `dep`


def test_node_aware_degenerate_cases(oracle):
    """One process per node: nothing but the plain scatter-ring.  One node: nothing but a tree
    broadcast, ceil(log2 P) steps, P - 1 messages of the whole message."""
    for P, root, n in [(8, 3, 1000), (10, 0, 77), (5, 4, 5)]:
        for variant in (NATIVE, TUNED):
            a = oracle.simulate(P, root, n, variant, ranks_per_node=1)
            b = oracle.simulate(P, root, n, variant)
            assert np.array_equal(a.schedule, b.schedule)
        one = oracle.simulate(P, root, n, TUNED, ranks_per_node=P + 3)
        assert (one.schedule[:, 0] == NODE_FIRST).all() and len(one.schedule) == P - 1
        assert int(one.schedule[:, 1].max()) + 1 == (P - 1).bit_length()
        assert (one.schedule[:, 7] == n).all() and one.scatter_size == n
        members = [(root + r) % P for r in range(P)]
        assert {(int(r[1]), int(r[2]), int(r[3])) for r in one.schedule} == tree_by_halving(members)
    with pytest.raises(oracle.OracleError):
        oracle.simulate(8, 0, 100, 2, ranks_per_node=2)              # no recursive doubling between nodes here


@pytest.mark.parametrize("P,root,n,c", SMP_CASES)
def test_node_aware_dep_names_the_last_writer(oracle, P, root, n, c):
    """`dep` of every message of the node-aware schedule is the message that last wrote the first chunk
    it carries into its source (-1: the root's own data), and lies in an earlier step; messages of one
    step are listed by destination."""
    k = -(-P // c)
    for variant in (NATIVE, TUNED):
        sched = oracle.simulate(P, root, n, variant, ranks_per_node=c).schedule
        holds = {(root, cc): -1 for cc in range(k)}
        i = 0
        while i < len(sched):
            j = i
            while j < len(sched) and (sched[j, 0], sched[j, 1]) == (sched[i, 0], sched[i, 1]):
                j += 1
            assert list(sched[i:j, 3]) == sorted(sched[i:j, 3]) and len(set(sched[i:j, 3])) == j - i
            for x in range(i, j):
                src, first, dep = int(sched[x, 2]), int(sched[x, 4]), int(sched[x, 8])
                assert dep == holds[(src, first)] and dep < i
            for x in range(i, j):
                for cc in range(int(sched[x, 4]), int(sched[x, 4] + sched[x, 5])):
                    holds[(int(sched[x, 3]), cc)] = x
            i = j
        assert len(holds) == P * k
