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
    ("scatter_size_rounds_down", "s.S = (nbytes + (uint64_t)P - 1) / (uint64_t)P;", "s.S = P ? nbytes / (uint64_t)P : 0;"),
    ("scatter_levels_in_reverse", "const int mask = 1 << (L - 1 - t);", "const int mask = 1 << t;"),
    ("child_keeps_only_its_own_chunk", "m[nm].nchunks = hi - (r + mask);", "m[nm].nchunks = 1;"),
    ("two_sided_phase_one_step_short", "if (!tuned || step[k] <= P - i)", "if (!tuned || step[k] < P - i)"),
    ("two_sided_phase_one_step_long", "if (!tuned || step[k] <= P - i)", "if (!tuned || step[k] <= P - i + 1)"),
    ("send_only_and_recv_only_swapped", "*flag = RECV_ONLY;                           /* them",
     "*flag = SEND_ONLY;                           /* them"),
    ("ring_turns_the_other_way", "jnext[k] = (P + k - 1) % P;", "jnext[k] = (k + 1) % P;"),
    ("ring_chunk_by_absolute_rank", "const int rel_j = rel_of(s, j[k]);", "const int rel_j = j[k];"),
    ("step_from_own_rank_only", "if (rr % mask == 0) {", "if (0 && rr % mask == 0) {"),
    ("dep_forgotten", "rec[F_DEP] = s->writer[(size_t)m[a].src * P + c0];", "rec[F_DEP] = -1;"),
    ("messages_sorted_by_sender", "return ((const pending_t *)a)->dst - ((const pending_t *)b)->dst;",
     "return ((const pending_t *)b)->src - ((const pending_t *)a)->src;"),
    ("sent_bytes_booked_to_receiver", "s->bytes_sent[(size_t)phase * P + m[a].src] += len;",
     "s->bytes_sent[(size_t)phase * P + m[a].dst] += len;"),
    ("empty_messages_dropped_from_counts", "s->msgs_recv[(size_t)phase * P + m[a].dst] += 1;",
     "s->msgs_recv[(size_t)phase * P + m[a].dst] += len ? 1 : 0;"),
    ("doubling_sends_one_chunk_of_the_block", "m[nm].nchunks = mask;", "m[nm].nchunks = 1;"),
    ("doubling_partner_by_relative_rank", "wants_from[k] = abs_of(s, partner);", "wants_from[k] = partner;"),
    ("doubling_block_of_the_wrong_size", "const int my_block = (r >> i) << i;", "const int my_block = (r >> (i + 1)) << (i + 1);"),
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
