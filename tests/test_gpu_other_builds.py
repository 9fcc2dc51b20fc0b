"""The small parity cases once more under the bounds-checked build of the library
(-DATREX_DEBUG_BOUNDS): every index the ingest kernels form into the key table, the spill buffers
and their shared-memory arrays is range checked there, and a violation would come back as
ATREX_ERR_BOUNDS from finalize / stats.  Stands in for a memory checker; nothing traps."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_parity_cases_under_the_bounds_checked_build():
    import importlib.util
    spec = importlib.util.spec_from_file_location("atrex_build", os.path.join(ROOT, "paper_2607_14541_b200", "build.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    lib = mod.build_checked()
    env = dict(os.environ, ATREX_AGG_LIBRARY=lib)
    probe = subprocess.run([sys.executable, "-c", "import paper_2607_14541_b200 as p; print(p.atrex_build_has_bounds_checks())"],
                           cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)
    assert probe.returncode == 0 and probe.stdout.strip() == "1", probe.stderr[-2000:]
    run = subprocess.run([sys.executable, "-m", "pytest", "tests/test_gpu_parity.py", "-x", "-q", "-k",
                          "five_configs or misaligned or carry or invalid_records or full_u32 or largest_geometry or crowded or exactly_to_max_keys or merge_of_partial or every_partition_count"],
                         cwd=ROOT, env=env, capture_output=True, text=True, timeout=1200)
    assert run.returncode == 0, run.stdout[-3000:] + run.stderr[-2000:]
    assert " passed" in run.stdout


@pytest.mark.parametrize("variant", ["ring4"])
def test_parity_cases_under_the_scatter_variants(variant):
    """The scatter pass's build-time variant -- the shared-memory record ring filled by bulk asynchronous
    copies -- is slower than the default and therefore not what ships, but it is kept buildable and
    exact: the same parity cases, bit for bit against the oracle."""
    import importlib.util
    spec = importlib.util.spec_from_file_location("atrex_build", os.path.join(ROOT, "paper_2607_14541_b200", "build.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    lib = mod.build_variant_if_stale(variant, mod.VARIANTS[variant])
    env = dict(os.environ, ATREX_AGG_LIBRARY=lib)
    run = subprocess.run([sys.executable, "-m", "pytest", "tests/test_gpu_parity.py", "-x", "-q", "-k",
                          "five_configs or misaligned or carry or invalid_records or full_u32 or many_small_calls"],
                         cwd=ROOT, env=env, capture_output=True, text=True, timeout=1200)
    assert run.returncode == 0, run.stdout[-3000:] + run.stderr[-2000:]
    assert " passed" in run.stdout


def test_the_regular_build_has_no_checks():
    import paper_2607_14541_b200 as p
    assert p.atrex_build_has_bounds_checks() == 0 or os.environ.get("ATREX_AGG_LIBRARY")
