"""The product kernels are chosen by problem size (persistent single-CTA tiles, cluster split-K for
small problems, CTA pairs for large ones).  The small parity shapes would never reach the CTA-pair
kernel or the unsplit kernel on their own, so the tensor-core parity cases are run again in child
processes with the selection forced through the library's environment switches (read once per
process, hence the child processes).  The same goes for the intermediate-label loss, which the
tensor-core path takes inside the last forward product's epilogue: SEG_NO_FUSED_LOSS runs the separate
loss kernel; and for the optimizer update, which the persistent tensor-core kernels apply inside the
weight-gradient product when SEG_FUSED_UPDATE asks for it (with SEG_NO_SPLITK every weight gradient runs
in such a kernel, with SEG_PAIR_MIN_TILES=1 the larger ones in the CTA-pair kernel); and for the output path of the persistent kernels, staged through shared memory and written by
bulk tensor stores by default, per-lane stores with SEG_NO_STAGED_EPILOGUE.  Small fp32 segments run
their whole step in two launches; SEG_NO_SMALL_FUSED sends them through the launch-by-launch path, so
the fp32 cases run once more that way."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("env", [{"SEG_PAIR_MIN_TILES": "1"}, {"SEG_NO_SPLITK": "1", "SEG_NO_PAIRS": "1"},
                                 {"SEG_NO_GRAPH": "1"}, {"SEG_NO_FORK": "1"}, {"SEG_NO_PDL": "1"},
                                 {"SEG_NO_FUSED_LOSS": "1"}, {"SEG_FUSED_UPDATE": "1"},
                                 {"SEG_FUSED_UPDATE": "1", "SEG_NO_SPLITK": "1", "SEG_PAIR_MIN_TILES": "1"},
                                 {"SEG_NO_STAGED_EPILOGUE": "1"}, {"SEG_NO_STAGED_EPILOGUE": "1", "SEG_PAIR_MIN_TILES": "1"}])
def test_tensor_core_cases_with_forced_kernel_selection(env):
    child_env = dict(os.environ, **env)
    res = subprocess.run([sys.executable, "-m", "pytest", "tests/test_gpu_parity.py", "-m", "gpu", "-q", "-x",
                          "-k", "tensor_core"], cwd=ROOT, env=child_env, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-1000:]


@pytest.mark.parametrize("env", [{"SEG_NO_SMALL_FUSED": "1"}, {"SEG_NO_GRAPH": "1"}, {"SEG_NO_PDL": "1"}])
def test_fp32_cases_with_switches(env):
    """The fp32 cases once more: launch by launch (no two-launch step for small segments), and the two-launch step
    without the captured graph and without programmatic dependent launches."""
    child_env = dict(os.environ, **env)
    res = subprocess.run([sys.executable, "-m", "pytest", "tests/test_gpu_parity.py", "-m", "gpu", "-q", "-x",
                          "-k", "fp32 or tiny or reproducible or replayed or class_index"], cwd=ROOT, env=child_env,
                         capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-1000:]
