"""qsim_simulate_static, the entry point for callers that may not allocate device memory.

Some users of the library run where cudaMalloc is not an option: inside a serving process whose allocator
already owns the card, or in a section that cannot take cudaMalloc's device-wide synchronisation.  For
them the library carries a 32 MiB built-in scratch array and an entry point that allocates nothing.
This file checks, through the C ABI, that it returns what the allocating entry point (qsim_simulate)
returns - twice in a row, since the array keeps the previous call's contents - and that a problem too
large for the array is refused with a clear message.  It is collected last on purpose.
"""
import numpy as np
import pytest

from qsim_inputs import presets
from qsim_inputs.spec import PLACE_RANDOM

from parity import assert_parity

pytestmark = pytest.mark.gpu


def test_static_entry_point_matches_the_allocating_one_on_two_calls_in_a_row():
    from paper_2602_02987_b200 import simulate_host, simulate_static
    # first a table-driven case, then a different, smaller one that reuses the same scratch bytes
    first = presets.cfg1(R=4, horizon_iters=400).with_(qcap=512)
    second = presets.paper_instance(n=12, R=6, placement=PLACE_RANDOM).with_(qcap=256)
    for inp, horizon in ((first, 400), (second, 3000)):
        want = simulate_host(inp, horizon)
        got = simulate_static(inp, horizon)
        assert_parity(got, want, what=f"static vs allocating ({inp.name})")
        for k in ("arrivals", "done_mixed", "done_solo", "tokens_out_completed"):
            assert np.array_equal(got["_totals"][k], want["_totals"][k])
        assert int(got["events"].sum()) > 1000
    # and the first case again: stale contents of the second call must not leak into it
    again = simulate_static(first, 400)
    assert_parity(again, simulate_host(first, 400), what="static, third call")


def test_static_entry_point_refuses_what_does_not_fit():
    from paper_2602_02987_b200 import QSimError, simulate_static
    big = presets.cfg1(R=1024)
    with pytest.raises(QSimError, match="built-in scratch"):
        simulate_static(big, 10)
