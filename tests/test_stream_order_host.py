"""Host logic that keeps stream order although kernels overlap on the GPU: per stream the library
remembers the byte ranges of the calls that may still be running and tells a new call whether it has
to wait.  cconv_stream_order_probe registers calls with that bookkeeping without launching anything,
so the rules can be checked without a GPU:

  * a call waits when its Image or Filter meets the Out of a call that may still be running, and --
    if it may write beside earlier calls -- when its Out meets any of their arrays;
  * calls that are provably complete are forgotten: walking back from the newest call, everything
    behind sm_count SMs' worth of resident CTAs (counted by memory or by thread slots);
  * an ordinary launch, and a call that waits, complete everything before them.
"""
import itertools

import pytest

from paper_1802_06905_b200 import binding

INPUTS, OUT = 1, 2
NONE, INPUTS_EARLY, DEEP = 0, 1, 2
_keys = itertools.count(0x7E570000)


def key():
    return next(_keys) << 8          # a fresh fake stream per test


def R(lo, n=0x1000):
    return (lo, lo + n)


def probe(k, image, filt, out, how=DEEP, sms=28.0, threads=0.0, sm_count=148):
    return binding.stream_order_probe(k, image, filt, out, how, sms, threads, sm_count)


def test_independent_calls_do_not_wait():
    k = key()
    for i in range(12):
        base = 0x100000 * (i + 1)
        assert probe(k, R(base), R(base + 0x10000), R(base + 0x20000)) == 0


def test_read_after_write_image_and_filter():
    k = key()
    assert probe(k, R(0x1000), R(0x3000), R(0x5000)) == 0
    assert probe(k, R(0x5800, 0x100), R(0x9000), R(0xA000)) == INPUTS          # Image inside the earlier Out
    k = key()
    assert probe(k, R(0x1000), R(0x3000), R(0x5000)) == 0
    assert probe(k, R(0x7000), R(0x4FFF, 2), R(0xA000)) == INPUTS              # Filter overlaps it by one byte
    k = key()
    assert probe(k, R(0x1000), R(0x3000), R(0x5000)) == 0
    assert probe(k, R(0x7000), R(0x6000), R(0xA000)) == 0                      # adjacent ranges do not meet


def test_write_after_read_and_write_after_write_for_calls_that_write_early():
    k = key()
    assert probe(k, R(0x1000), R(0x3000), R(0x5000)) == 0
    assert probe(k, R(0x7000), R(0x9000), R(0x1800, 0x10)) == OUT              # Out over the earlier Image
    k = key()
    assert probe(k, R(0x1000), R(0x3000), R(0x5000)) == 0
    assert probe(k, R(0x7000), R(0x9000), R(0x3000)) == OUT                    # ... Filter
    k = key()
    assert probe(k, R(0x1000), R(0x3000), R(0x5000)) == 0
    assert probe(k, R(0x7000), R(0x9000), R(0x5000)) == OUT                    # ... Out
    k = key()
    assert probe(k, R(0x1000), R(0x3000), R(0x5000)) == 0
    assert probe(k, R(0x5000), R(0x9000), R(0x1000)) == (INPUTS | OUT)


def test_calls_that_write_only_after_earlier_calls_are_complete_check_their_inputs_only():
    k = key()
    assert probe(k, R(0x1000), R(0x3000), R(0x5000)) == 0
    assert probe(k, R(0x7000), R(0x9000), R(0x5000), how=INPUTS_EARLY) == 0    # same Out: no wait needed
    k = key()
    assert probe(k, R(0x1000), R(0x3000), R(0x5000)) == 0
    assert probe(k, R(0x5000), R(0x9000), R(0xB000), how=INPUTS_EARLY) == INPUTS
    # such a call completes everything before it: only itself stays on the list
    assert probe(k, R(0x20000), R(0x30000), R(0x1000)) == 0                    # the first call is forgotten
    assert probe(k, R(0xB000), R(0x30000), R(0x40000)) == INPUTS               # the second is not


def test_calls_behind_a_full_machine_of_resident_ctas_are_forgotten():
    """A call may still be running only while the CTAs of all calls registered after it fit the SMs
    together (each of them keeps its CTAs resident until the call in front of it is complete).  Calls
    of 28 SMs each: with five later calls (140 SMs) call 0 may still run, with six (168) it cannot."""
    outs = [R(0x100000 * (i + 1)) for i in range(8)]
    k = key()
    for i in range(6):
        assert probe(k, R(0x10), R(0x20), outs[i]) == 0
    assert probe(k, R(0x10), R(0x20), outs[0]) == OUT         # five calls behind call 0: 140 < 148
    k = key()
    for i in range(7):
        assert probe(k, R(0x10), R(0x20), outs[i]) == 0
    assert probe(k, R(0x10), R(0x20), outs[0]) == 0           # six: call 0 is forgotten, no write-after-write
    assert probe(k, R(0x10), R(0x20), outs[3]) == OUT         # call 3 is not


def test_either_resource_proves_completion():
    k = key()
    for i in range(3):                                        # pooling-like calls: 91 SMs' worth of thread slots
        assert probe(k, R(0x100 * (i + 1)), None, R(0x100000 * (i + 1)), sms=0.0, threads=91.0) == 0
    assert probe(k, R(0xA00), None, R(0x100000), sms=0.0, threads=91.0) == 0       # two calls behind the first: 182
    k = key()
    for i in range(2):
        assert probe(k, R(0x100 * (i + 1)), None, R(0x100000 * (i + 1)), sms=0.0, threads=91.0) == 0
    assert probe(k, R(0xA00), None, R(0x100000), sms=0.0, threads=91.0) == OUT     # one call behind it: 91
    k = key()
    assert probe(k, R(0x100), None, R(0x100000), sms=0.0, threads=30.0) == 0
    assert probe(k, R(0x200), None, R(0x200000), sms=100.0, threads=0.0) == 0
    assert probe(k, R(0x300), None, R(0x300000), sms=40.0, threads=100.0) == 0
    # behind the first call: memory 140, threads 100 -- neither reaches 148: it may still run
    assert probe(k, R(0x400), None, R(0x100000), sms=1.0, threads=1.0) == OUT
    k = key()
    assert probe(k, R(0x100), None, R(0x100000), sms=0.0, threads=30.0) == 0
    assert probe(k, R(0x200), None, R(0x200000), sms=100.0, threads=0.0) == 0
    assert probe(k, R(0x300), None, R(0x300000), sms=48.0, threads=100.0) == 0
    assert probe(k, R(0x400), None, R(0x100000), sms=1.0, threads=1.0) == 0        # memory 148: forgotten


def test_an_ordinary_launch_completes_everything_before_it():
    k = key()
    assert probe(k, R(0x1000), R(0x3000), R(0x5000)) == 0
    assert probe(k, R(0x5000), R(0x3000), R(0x1000), how=NONE) == 0
    assert probe(k, R(0x5000), R(0x9000), R(0xB000)) == 0


def test_a_call_that_waits_clears_the_list_and_a_full_list_makes_the_next_call_wait():
    k = key()
    assert probe(k, R(0x1000), R(0x3000), R(0x5000)) == 0
    assert probe(k, R(0x5000), R(0x9000), R(0xB000)) == INPUTS
    assert probe(k, R(0x20000), R(0x30000), R(0x1000)) == 0   # the first call went with the wait
    k = key()
    n = 0
    while True:                                               # tiny grids: nothing is ever forgotten
        h = probe(k, R(0x10), R(0x20), R(0x100000 * (n + 1)), sms=0.01)
        n += 1
        if h:
            break
        assert n < 10000
    assert h == (INPUTS | OUT) and 100 <= n <= 1000           # the bounded list filled up
    assert probe(k, R(0x10), R(0x20), R(0x100000)) == 0        # ... and starts afresh


def test_streams_are_independent_and_bad_arguments_are_rejected():
    k1, k2 = key(), key()
    assert probe(k1, R(0x1000), R(0x3000), R(0x5000)) == 0
    assert probe(k2, R(0x5000), R(0x3000), R(0x1000)) == 0
    lib = binding.load_library()
    assert lib.cconv_stream_order_probe(None, None, None, None, None, None, None, 3, 0.0, 0.0, 148) == binding.EINVAL
    assert lib.cconv_stream_order_probe(None, None, None, None, None, None, None, 2, 0.0, 0.0, 0) == binding.EINVAL
