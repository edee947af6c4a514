"""Host-side pieces of the benchmark that need no GPU: the clock record keeps only samples stamped inside a
timed region and reports throttle reasons seen there; `--gpus N` started as a plain process starts its N ranks
itself; the oracle arm's line says that its value is extrapolated from a bounded sample."""
import datetime
import importlib.util
import json
import pathlib
import subprocess
import sys

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


BENCH = str(pathlib.Path(__file__).resolve().parents[1] / "bench.py")


def test_gpus_flag_starts_the_ranks_itself():
    """No outer launcher, no WORLD_SIZE: `--gpus 2` must come back with a line from a 2-rank job (host-only stub step
    over gloo: rank r sleeps r + 1 ms per step, so the reported time is the slower rank's)."""
    import os
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, BENCH, "--gpus", "2", "--steps", "5", "--warmup", "0", "--stub-step"],
                       capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(ln) for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                                            # rank 0 alone prints
    assert lines[0]["n_gpus"] == 2 and lines[0]["steps"] == 5 and lines[0]["ms_per_step"] >= 2.0


def test_reference_arm_says_that_its_value_is_extrapolated(monkeypatch, capsys):
    class _Sample:
        def __init__(self, w):
            pass

        def run(self):
            return 7000.0, 16, "stub sample"
    monkeypatch.setattr(bench, "OracleSample", _Sample)
    monkeypatch.delenv("RANK", raising=False)
    import argparse
    bench.run_reference(argparse.Namespace(config=2, warmup=1, steps=3, gpus=1))
    line = json.loads(capsys.readouterr().out.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["extrapolated"] is True and line["timed_passes"] == 3
    assert line["timed_s"] < 1.0 and line["value"] == 7000.0 and line["steps"] == 3
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
