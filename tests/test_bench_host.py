"""Host-side pieces of bench.py that need no GPU: the clock-sample window and its summary."""
import datetime
import time

import bench


def _line(ts, sm, cap):
    stamp = datetime.datetime.fromtimestamp(ts).strftime("%Y/%m/%d %H:%M:%S.%f")[:-3]
    return f"{stamp}, {sm}, 1965, 612.5, Not Active, Not Active, Not Active, {'Active' if cap else 'Not Active'}"


def test_clock_samples_are_cut_to_the_timed_window():
    now = time.time()
    text = "\n".join(_line(now + 0.1 * i, 1000 + 10 * i, cap=(i == 7)) for i in range(20)) + "\ngarbage, line\n"
    rows = bench.ClockSampler.parse(text, now + 0.45, now + 1.05)
    assert [r[1] for r in rows] == [1050.0, 1060.0, 1070.0, 1080.0, 1090.0, 1100.0]
    out = bench.ClockSampler.summarise(rows, True)
    assert out["samples"] == 6 and out["sm_mhz"] == 1075.0 and out["sm_max_mhz"] == 1965.0
    assert out["reasons"] == ["sw_power_cap"] and out["in_timed_region"] is True
    # without a window every well-formed line counts; the malformed one is dropped
    assert len(bench.ClockSampler.parse(text)) == 20
    empty = bench.ClockSampler.summarise([], False)
    assert empty["samples"] == 0 and empty["sm_mhz"] is None and empty["reasons"] == []
