"""Host-side pieces of the benchmark that need no GPU: the clock record keeps only samples stamped inside a
timed region and reports throttle reasons seen there."""
import datetime
import importlib.util
import pathlib

_spec = importlib.util.spec_from_file_location("bench", pathlib.Path(__file__).resolve().parents[1] / "bench.py")
bench = importlib.util.module_from_spec(_spec)
_spec.loader.exec_module(bench)


class _Proc:
    def terminate(self):
        pass


class _Thread:
    def join(self, timeout=None):
        pass


def _line(ts, clk, cap="Not Active", therm="Not Active"):
    return (f"{ts:%Y/%m/%d %H:%M:%S.%f}"[:-3] + f", 0, {clk}, 1965, 300.0, 0x0, Not Active, {therm}, Not Active, {cap}\n")


def _sampler(lines, windows):
    s = bench.ClockSampler(0)
    s.proc, s.t, s.lines, s.windows, s.INTERVAL_MS = _Proc(), _Thread(), lines, windows, 1
    return s


def test_only_samples_inside_a_timed_region_count():
    t0 = datetime.datetime(2026, 1, 1, 12, 0, 0)
    ms = lambda k: t0 + datetime.timedelta(milliseconds=k)
    lines = [_line(ms(0), 300), _line(ms(25), 1900), _line(ms(50), 1950, cap="Active"), _line(ms(75), 1700),
             _line(ms(100), 1600, therm="Active"), "garbage\n"]
    rec = _sampler(lines, [(ms(20), ms(30), False), (ms(40), ms(80), True)]).stop()
    assert rec["samples"] == 3 and rec["samples_in_headline_region"] == 2
    assert rec["sm_mhz"] == 1900 and rec["sm_mhz_headline_region"] == (1950 + 1700) / 2
    assert rec["sm_max_mhz"] == 1965 and rec["reasons"] == ["sw_power_cap"]      # the thermal one lies outside
    assert "note" not in rec


def test_a_region_between_two_samples_is_flagged():
    t0 = datetime.datetime(2026, 1, 1, 12, 0, 0)
    ms = lambda k: t0 + datetime.timedelta(milliseconds=k)
    rec = _sampler([_line(ms(0), 1000), _line(ms(100), 1200)], [(ms(40), ms(60), True)]).stop()
    assert rec["samples"] == 2 and rec["samples_in_headline_region"] == 0 and "note" in rec
    assert rec["sm_mhz"] == 1100
