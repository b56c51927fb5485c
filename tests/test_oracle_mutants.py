"""Do the pins of the oracle notice a mistake?  Each case below plants one plausible mistake into a
copy of oracle/bcast_oracle.c (on the CPU, in a temporary build), routes the oracle's Python front
end to that build and runs the schedule-level pins of tests/test_oracle_pins.py: at least one of
them, or one of the oracle's own consistency checks, must fail."""
import os
import subprocess

import pytest

import test_oracle_pins as pins
from helpers import ROOT

SRC = os.path.join(ROOT, "oracle", "bcast_oracle.c")

# (name, text in the source, replacement)
MUTANTS = [
    ("scatter_size_rounds_down", "s.S = (nbytes + (uint64_t)C - 1) / (uint64_t)C;", "s.S = C ? nbytes / (uint64_t)C : 0;"),
    ("scatter_levels_in_reverse", "const int mask = 1 << (L - 1 - t);\n        int nm = 0;", "const int mask = 1 << t;\n        int nm = 0;"),
    ("child_keeps_only_its_own_chunk", "m[nm].nchunks = hi - (r + mask);", "m[nm].nchunks = 1;"),
    ("tuned_ring_skips_nothing", "if (tuned && owned_after_scatter[(size_t)right * C + chunk]) continue;",
     "if (0 && tuned && owned_after_scatter[(size_t)right * C + chunk]) continue;"),
    ("tuned_ring_skips_by_what_the_sender_owned", "if (tuned && owned_after_scatter[(size_t)right * C + chunk]) continue;",
     "if (tuned && owned_after_scatter[(size_t)k * C + chunk]) continue;"),
    ("skipped_transfer_stalls_the_rotation", "arrives[qr] = chunk;                         /* due",
     "arrives[qr] = (tuned && owned_after_scatter[(size_t)right * C + chunk]) ? passes[qr] : chunk;   /* due"),
    ("ring_turns_the_other_way", "const int k = abs_of(s, q), qr = (q + 1) % P, right = abs_of(s, qr);",
     "const int k = abs_of(s, q), qr = (q + P - 1) % P, right = abs_of(s, qr);"),
    ("ring_chunk_by_absolute_rank", "passes[q] = q;                                   /* step 1", "passes[q] = abs_of(s, q);                        /* step 1"),
    ("ring_keeps_passing_the_own_chunk", "for (int q = 0; q < P; q++) passes[q] = arrives[q];", "(void)arrives;"),
    ("send_only_and_recv_only_swapped", "*flag = last_send <= last_recv ? RECV_ONLY : SEND_ONLY;",
     "*flag = last_send <= last_recv ? SEND_ONLY : RECV_ONLY;"),
    ("step_from_the_receiving_side_only", "const int two_sided_until = last_recv < last_send ? last_recv : last_send;",
     "const int two_sided_until = last_recv; (void)last_send;"),
    ("two_sided_phase_one_step_long", "*step = P - two_sided_until;", "*step = P - two_sided_until - 1;"),
    ("dep_forgotten", "rec[F_DEP] = s->writer[(size_t)m[a].src * C + c0];", "rec[F_DEP] = -1;"),
    ("messages_sorted_by_sender", "return ((const pending_t *)a)->dst - ((const pending_t *)b)->dst;",
     "return ((const pending_t *)b)->src - ((const pending_t *)a)->src;"),
    ("sent_bytes_booked_to_receiver", "s->bytes_sent[(size_t)phase * P + m[a].src] += len;",
     "s->bytes_sent[(size_t)phase * P + m[a].dst] += len;"),
    ("empty_messages_dropped_from_counts", "s->msgs_recv[(size_t)phase * P + m[a].dst] += 1;",
     "s->msgs_recv[(size_t)phase * P + m[a].dst] += len ? 1 : 0;"),
    ("doubling_sends_one_chunk_of_the_block", "m[nm].nchunks = mask;", "m[nm].nchunks = 1;"),
    ("doubling_partner_by_relative_rank", "wants_from[k] = abs_of(s, partner);", "wants_from[k] = partner;"),
    ("doubling_block_of_the_wrong_size", "const int my_block = (r >> i) << i;", "const int my_block = (r >> (i + 1)) << (i + 1);"),
    # ---- the node-aware broadcast (Section II)
    ("node_tree_passes_one_chunk_only", "m[nm].nchunks = s->C;", "m[nm].nchunks = 1;"),
    ("node_tree_levels_in_reverse", "const int mask = 1 << (L - 1 - t);\n        for (int r = 0; r + mask < sizes[g]; r += 2 * mask) {",
     "const int mask = 1 << t;\n        for (int r = 0; r + mask < sizes[g]; r += 2 * mask) {"),
    ("first_tree_rooted_at_the_node_leader", "order[r] = first + (root - first + r) % size;", "order[r] = first + r;"),
    ("leaders_not_relative_to_the_root_node", "leaders[q] = ((root_node + q) % nnodes) * per_node;", "leaders[q] = q * per_node;"),
    ("last_trees_also_in_the_root_node", "if (node == root_node) continue;", "if (0 && node == root_node) continue;"),
    ("node_chunks_as_many_as_processes", "const int C = per_node ? nnodes : P;", "const int C = P; (void)nnodes;"),
    ("offset_not_clipped", "static uint64_t chunk_begin(const sim_t *s, int c) { return umin((uint64_t)c * s->S, s->n); }",
     "static uint64_t chunk_begin(const sim_t *s, int c) { return (uint64_t)c * s->S; }"),
]


def schedule_level_pins(oracle):
    """The pins that need no data movement (a broken oracle must never be allowed to memcpy)."""
    yield lambda: pins.test_scatter_worked_examples(oracle, 8, "fig1_scatter_p8.txt")
    yield lambda: pins.test_scatter_worked_examples(oracle, 10, "fig2_scatter_p10.txt")
    yield lambda: pins.test_tuned_ring_worked_examples(oracle, 8, "fig4_tuned_ring_p8.txt")
    yield lambda: pins.test_tuned_ring_worked_examples(oracle, 10, "fig5_tuned_ring_p10.txt")
    yield lambda: pins.test_native_ring_shape(oracle)
    for P in (1, 2, 3, 5, 8, 10, 12, 16, 33):
        yield lambda P=P: pins.test_against_brute_force_ownership(oracle, P)
    for P in (2, 7, 12, 64, 100, 255):
        yield lambda P=P: pins.test_message_count_closed_forms(oracle, P)
    yield lambda: pins.test_step_flag_closed_form(oracle)
    for case in pins.CASES:
        yield lambda case=case: pins.test_byte_budget(oracle, *case)
    yield lambda: pins.test_validity_of_every_send(oracle)
    yield lambda: pins.test_canonical_order(oracle)
    yield lambda: pins.test_tuned_is_subset_of_native(oracle)
    yield lambda: pins.test_root_rotation(oracle)
    yield lambda: pins.test_schedule_geometry(oracle)
    yield lambda: pins.test_doubling_equals_ring_for_two_processes(oracle)
    for P in (1, 2, 8, 64):
        yield lambda P=P: pins.test_doubling_against_textbook_hypercube_exchange(oracle, P)
    for case in ((4, 1, 3), (16, 15, 65521), (64, 17, (16 << 20) + 13)):
        yield lambda case=case: pins.test_doubling_byte_budget_and_semantics(oracle, *case, with_data=False)
    yield lambda: pins.test_doubling_root_rotation_and_validity(oracle)
    for case in pins.SMP_CASES:
        yield lambda case=case: pins.test_node_aware_structure(oracle, *case)
    yield lambda: pins.test_node_aware_degenerate_cases(oracle)
    for case in pins.SMP_CASES[:3]:
        yield lambda case=case: pins.test_node_aware_dep_names_the_last_writer(oracle, *case)
    yield lambda: pins.test_node_aware_leader_ring_is_the_plain_ring_of_the_nodes(oracle)


def test_the_unbroken_oracle_passes_the_same_pins(oracle):
    for pin in schedule_level_pins(oracle):
        pin()


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_pins_catch_planted_mistake(oracle, tmp_path, name, old, new):
    src = open(SRC).read()
    assert src.count(old) == 1, "mutation site not found (or not unique) in the oracle source"
    broken_c = tmp_path / "broken.c"
    broken_c.write_text(src.replace(old, new))
    broken_so = tmp_path / "libbroken.so"
    subprocess.check_call(["gcc", "-O1", "-shared", "-fPIC", "-o", str(broken_so), str(broken_c)])
    oracle.use_build(str(broken_so))
    try:
        caught = None
        for pin in schedule_level_pins(oracle):
            try:
                pin()
            except (AssertionError, oracle.OracleError, KeyError, ValueError, IndexError) as e:
                caught = e
                break
        assert caught is not None, f"no pin noticed the planted mistake '{name}'"
    finally:
        oracle.use_build(None)
