"""Run by test_checked_build.py in a process of its own with NSP_LIBRARY pointing at libnsp_checked.so (the same
kernels compiled with -DNSP_CHECKED: every index computed for a global access is verified, a bad one is recorded as
NSP_ERR_DEVICE_ASSERT and skipped).

Part 1: parity cases through the checked kernels: results match the oracle and no check fires.
Part 2: failure detection inside a real attention kernel, without a fault: the forward launch is told to leave out one
V tile load, the plan's wait limit is two million clocks; the wait behind the missing tile runs out, every role of the
kernel unwinds, the launch ends, the status record names the wait, the plan refuses further work, and a fresh plan on
the same context still matches the oracle."""
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))
sys.path.insert(0, str(ROOT / "tests"))

import numpy as np  # noqa: E402
import torch  # noqa: E402

import parity_util as P  # noqa: E402
from paper_2609_22755_b200 import binding as B  # noqa: E402
from paper_2609_22755_b200 import workloads as W  # noqa: E402

assert B.LIB_PATH.name == "libnsp_checked.so", B.LIB_PATH
assert hasattr(B.lib(), "nsp_checked_withhold_load")

base = W.ragged()
cases = [W.config(1), base, W.config(4, twin=True),
         W.custom(base.lengths.tolist(), base.hq.tolist(), base.hkv.tolist(), seed=2, head_dim=64),
         # short segments that share first tiles (per-row LSE addresses)
         W.custom([5, 60, 63, 1, 127, 2, 64, 7, 0, 9, 200, 16, 16, 16], [8] * 7 + [4] * 7, [2] * 7 + [4] * 7, seed=3)]
for w in cases:
    run = P.GpuRun(w)
    run.forward()
    run.backward()
    assert run.status() == (0, 0, 0, 0), run.status()
    P.compare_full(w, run.results(), P.oracle_full(w, run.host))
    print("checked build:", w.name, "ok")

w = W.config(1)
run = P.GpuRun(w)
B.nsp_plan_set_wait_limit(run.plan, 2_000_000)
B.nsp_checked_withhold_load(run.plan, True)
run.forward()
torch.cuda.synchronize()  # the launch ends by itself
try:
    run.forward()
    raise SystemExit("the plan accepted work after a device-side timeout")
except B.NspError as e:
    assert e.code == B.NSP_ERR_DEVICE_TIMEOUT, e
code, item, where, aux = B.nsp_device_status(run.plan)
assert code == B.NSP_ERR_DEVICE_TIMEOUT and 1 <= where <= 6, (code, item, where, aux)
print("withheld load: status", (code, item, where, aux))
run2 = P.GpuRun(w)
run2.forward()
run2.backward()
assert run2.status() == (0, 0, 0, 0)
P.compare_full(w, run2.results(), P.oracle_full(w, run2.host))
print("fresh plan after the timeout: ok")
