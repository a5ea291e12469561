"""The peak micro-kernels (cert_peak_microbench): they measure the roofline denominators bench.py reports against.
Run in a child process with a time limit, as bench.py runs them."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_CODE = r"""
import json
from paper_2507_20055_b200 import binding
out = {k: binding.peak_microbench(k, 3.0) for k in (0, 1, 2, 3)}
assert binding.lib.cert_peak_microbench(4, 3.0, None, None, None, None) == 1     # bad kind
assert binding.lib.cert_peak_microbench(0, 0.0, None, None, None, None) == 1     # no output pointer, bad duration
print("PEAKS " + json.dumps(out))
"""


def test_peak_microbench_rates_are_the_units_nominal_rates_per_cycle():
    r = subprocess.run([sys.executable, "-c", _CODE], cwd=ROOT, capture_output=True, text=True, timeout=180)
    assert r.returncode == 0, r.stdout[-1500:] + r.stderr[-1500:]
    peaks = json.loads([x for x in r.stdout.splitlines() if x.startswith("PEAKS ")][-1][6:])
    # flop per cycle per SM from the kernel's own clock reading: the documented rates of the three units on 148 SMs
    for kind, nominal in (("0", 8192.0), ("1", 4096.0), ("2", 256.0)):
        tflops, mhz, ms = peaks[kind]
        assert 1.0 < ms < 50.0 and 500.0 < mhz < 2100.0
        per_cycle = tflops * 1e12 / (mhz * 1e6) / 148.0
        assert 0.85 * nominal <= per_cycle <= 1.02 * nominal, (kind, per_cycle)
    # what an SM takes in from L2 through bulk copies: tens of bytes per cycle (the fp16-split contraction in two
    # passes needs 64 at full MMA rate, in one pass 43)
    tbs, mhz, ms = peaks["3"]
    assert 1.0 < ms < 50.0 and 500.0 < mhz < 2100.0
    per_cycle = tbs * 1e12 / (mhz * 1e6) / 148.0
    assert 20.0 <= per_cycle <= 200.0, per_cycle
