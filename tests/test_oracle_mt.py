"""The all-cores CPU baseline (oracle/bcast_oracle_mt.c) replays the oracle's schedule with a team of
threads; it must leave exactly the buffers the single-threaded oracle leaves."""
import numpy as np
import pytest

from paper_1603_06809_b200 import workloads as W


@pytest.mark.parametrize("variant", [0, 1, 2], ids=["native", "tuned", "doubling"])
@pytest.mark.parametrize("P,root,n", [(8, 0, 1 << 16), (12, 5, 256 * 1024 + 5), (16, 15, 40001), (33, 32, 700), (7, 3, 5)])
@pytest.mark.parametrize("threads", [1, 3, 8])
def test_threaded_replay_equals_the_oracle(oracle, variant, P, root, n, threads):
    if variant == 2 and P & (P - 1):
        pytest.skip("recursive doubling needs a power of two")
    msg = W.message_bytes(77 + P, n)
    ref = oracle.simulate(P, root, n, variant, message=msg)
    bufs = np.empty((P, n), dtype=np.uint8)
    for k in range(P):
        bufs[k, :] = W.poison_byte(k)
    bufs[root, :] = msg
    seconds = oracle.replay_mt(P, ref.schedule, bufs, threads)
    assert seconds >= 0.0
    assert np.array_equal(bufs, ref.bufs)
    assert (bufs == msg[None, :]).all()


def test_threaded_replay_rejects_bad_records(oracle):
    bufs = np.zeros((4, 64), dtype=np.uint8)
    bad = np.zeros((1, 9), dtype=np.int64)
    bad[0, 2] = 9                                   # source rank out of range
    with pytest.raises(oracle.OracleError):
        oracle.replay_mt(4, bad, bufs, 2)
