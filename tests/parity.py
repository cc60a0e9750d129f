"""Element-by-element comparison of the CUDA library's statistics with the oracle's."""
import numpy as np

INT_KEYS = ("arrivals", "admitted", "prefill_done", "placed_mixed", "placed_solo", "done_mixed", "done_solo",
            "abandoned_p", "abandoned_d", "overflow", "overflow_d", "tokens_in_prefilled", "tokens_in_completed",
            "tokens_out_completed", "Qp", "X", "Qd", "Ym", "Ys", "iters_mixed", "iters_solo", "events",
            "hist_ttft", "hist_tpot")
F64_KEYS = ("area_Qp", "area_X", "area_Qd", "area_Ym", "area_Ys", "sum_ttft", "sum_tpot", "busy_mixed",
            "busy_solo", "T_elapsed")
# fp64 statistics: clocks are bit-identical by construction; sums may be taken in another order
RTOL = 1e-9


def assert_parity(gpu: dict, ref: dict, rows=None, what=""):
    """Integer statistics bit-exact, fp64 statistics within 1e-9 relative.  rows: replications to compare."""
    for k in INT_KEYS:
        if k not in ref:
            continue
        a, b = gpu[k], ref[k]
        if rows is not None:
            a, b = a[rows], b[rows]
        if not np.array_equal(a, b):
            bad = np.argwhere(a != b)
            raise AssertionError(f"{what}: integer statistic {k} differs at {bad[:5].tolist()}: "
                                 f"gpu {a[tuple(bad[0])]} oracle {b[tuple(bad[0])]}")
    for k in F64_KEYS:
        a, b = gpu[k], ref[k]
        if rows is not None:
            a, b = a[rows], b[rows]
        if not np.allclose(a, b, rtol=RTOL, atol=1e-300):
            err = np.abs(a - b) / np.maximum(np.abs(b), 1e-300)
            raise AssertionError(f"{what}: fp64 statistic {k} off by {err.max():.3e} relative")
