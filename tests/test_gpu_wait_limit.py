"""The path on which a device-side wait gives up.  Every mbarrier wait of the attention kernel is bounded; when one
runs out the CTA raises the device status word, drains its copies, frees its tensor memory and returns.  A test-only
copy of the library (20 ms limit, and a switch that makes one V tile never arrive, once) runs that path in a child
process: the launch must return, `hyperattn_last_device_status` must report the timeout exactly once, and an ordinary
call afterwards - which needs all the tensor memory of every SM again - must give the same result as before."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys, time
import torch
import paper_2310_05869_b200 as ha
L = ha.lib()
g = torch.Generator(device="cuda"); g.manual_seed(3)
q, k, v = (torch.randn((1, 4, 4096, 64), device="cuda", generator=g, dtype=torch.float32).to(torch.bfloat16) for _ in range(3))
args = dict(block=256, samples=256, hash_bits=7, causal=True, n0=1024, seed=0)
ref, ref_lse = ha.forward(q, k, v, **args)
torch.cuda.synchronize()
assert ha.last_device_status() == 0
assert L.hyperattn_test_arm_drop(1) == 0
t0 = time.time()
ha.forward(q, k, v, **args)                 # one V tile never arrives: the wait for it runs out
torch.cuda.synchronize()                    # the launch returns
dt = time.time() - t0
assert dt < 5.0, dt
assert ha.last_device_status() == -6        # HYPERATTN_DEVICE_TIMEOUT, reported ...
assert ha.last_device_status() == 0         # ... once
out, lse = ha.forward(q, k, v, **args)      # needs every SM's tensor memory again
torch.cuda.synchronize()
assert ha.last_device_status() == 0
assert torch.equal(out, ref) and torch.equal(lse, ref_lse)
print("wait limit path ok, gave up after %.3f s" % dt)
"""


def test_a_wait_that_runs_out_is_reported_once_and_leaves_the_device_usable():
    from paper_2310_05869_b200 import build as B
    lib = B.WAIT_TEST_LIB if os.path.exists(B.WAIT_TEST_LIB) else B.build_wait_test_library()     # (built by the package's build step)
    env = dict(os.environ, HYPERATTN_LIB=lib, PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    res = subprocess.run([sys.executable, "-c", CHILD], env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-4000:]
    assert "wait limit path ok" in res.stdout
