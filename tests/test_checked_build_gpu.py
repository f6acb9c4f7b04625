"""The bounds-checked build of the library (-DSGP_CHECKED): every table index and every global offset is tested
before use; a violation sets SGP_STATUS_BOUNDS in the device status word and the access is skipped.  Nothing
traps.  The small-shape and pitch/alignment parity tests are run once under that build in a child process (the
library is chosen at import time through SGP_CHECKED=1), and one corrupted table entry -- injected from the host
through a hook that only this build has -- must be caught, not dereferenced."""
import os
import subprocess
import sys

import pytest

from conftest import ROOT

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def checked_env():
    from paper_1811_10792_b200 import build
    build.build_checked()
    return dict(os.environ, SGP_CHECKED="1")


def test_small_shapes_under_the_checked_build(checked_env):
    r = subprocess.run([sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider",
                        os.path.join(ROOT, "tests", "test_parity_gpu.py"), "-k",
                        "small_shapes or pitch_and_alignment or config1 or degenerate or custom_weighted or complete_graph_shared"],
                       env=checked_env, capture_output=True, text=True, timeout=1500, cwd=ROOT)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout


_POKE = r"""
import sys, torch
sys.path.insert(0, %(root)r)
from paper_1811_10792_b200 import binding, inputs
assert binding.LIB_PATH.endswith("libsgp_checked.so")
for n, variant in ((8, 1), (8, 3), (128, 1)):                       # table in the constant bank, and in global memory
    w = inputs.sweep_workload(n, 40_000)
    X = inputs.initial_x(w, device="cuda:0").contiguous()
    W = torch.ones(n, device="cuda:0"); M = torch.zeros_like(X); Z = torch.empty_like(X)
    G = inputs.gradient(w, 0, torch.empty_like(X))
    with binding.Sgp(n, w.d, binding.graph_desc(w)) as h:
        h.set_option("variant", variant)
        h.step(X, W, M, G, Z, 0, w.lr, w.momentum, 0.0, True)
        assert h.device_status() == 0
        h.set_option("poke_table", n + 1000)                        # an in-neighbour index far outside [0, n)
        h.step(X, W, M, G, Z, 10, w.lr, w.momentum, 0.0, True)      # step 10 uses slot 0 again (period 10)
        torch.cuda.synchronize()                                    # no fault: the access was skipped
        assert h.device_status() & binding.SGP_STATUS_BOUNDS, (n, variant)
        assert torch.isfinite(X).all().item()
# the skipped entry is a lost message: with the per-step bracket on, the step's weight sum and column sums no longer
# match what they were before the step, and both conservation bits are raised (Sec. 2, 1^T P = 1^T)
n = 8
w = inputs.sweep_workload(n, 40_000)
X = inputs.initial_x(w, device="cuda:0").contiguous()
W = torch.ones(n, device="cuda:0"); M = torch.zeros_like(X); Z = torch.empty_like(X)
G = inputs.gradient(w, 0, torch.empty_like(X))
with binding.Sgp(n, w.d, binding.graph_desc(w)) as h:
    h.set_option("check_steps", 1)
    for k in range(3):
        h.step(X, W, M, G, Z, k, w.lr, w.momentum, 0.0, True)
    assert h.device_status() == 0
    h.set_option("poke_table", n + 1000)
    h.step(X, W, M, G, Z, 10, w.lr, w.momentum, 0.0, True)
    st = h.device_status()
    assert st & binding.SGP_STATUS_WEIGHT_SUM and st & binding.SGP_STATUS_COLUMN_SUM, st
print("poke ok")
"""


def test_out_of_range_table_entry_is_caught_not_dereferenced(checked_env):
    r = subprocess.run([sys.executable, "-c", _POKE % {"root": ROOT}], env=checked_env, capture_output=True, text=True,
                       timeout=600, cwd=ROOT)
    assert r.returncode == 0 and "poke ok" in r.stdout, r.stdout[-2000:] + r.stderr[-3000:]


def test_release_build_has_no_hook(checked_env):
    from paper_1811_10792_b200 import binding
    import torch
    if binding.LIB_PATH.endswith("libsgp_checked.so"):
        pytest.skip("this process already runs the checked build")
    with binding.Sgp(4, 100, binding.GraphDesc.exp_peers(1)) as h:
        with pytest.raises(binding.SgpError):
            h.set_option("poke_table", 7)
