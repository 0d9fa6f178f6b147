"""The debug library (libswitchhead_debug.so, -DSH_DEBUG): index checks on every list entry, tile
field and expert index the kernels read, plus the launch-structure switches.  Each case runs in a
child process (tests/debug_driver.py) because the library and its switches are fixed when the
binding is imported / the weights are set."""
import os
import subprocess
import sys

import pytest

from paper_2312_07987_b200 import build

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_case(case, extra_env=None):
    lib = build.build(debug=True)
    env = dict(os.environ, SWITCHHEAD_LIB=lib, **(extra_env or {}))
    res = subprocess.run([sys.executable, "-m", "tests.debug_driver", case], cwd=ROOT, env=env,
                         capture_output=True, text=True, timeout=1200)
    assert res.returncode == 0 and "DEBUG_DRIVER_OK" in res.stdout, res.stdout[-2000:] + res.stderr[-4000:]


@pytest.mark.parametrize("env", [{}, {"SH_NO_PDL": "1"}, {"SH_NO_PDL": "1", "SH_NO_OVERLAP": "1"}, {"SH_NO_PERSISTENT": "1"},
                                 {"SH_ATTN_ADJACENT": "1"}, {"SH_O_SINGLE": "1"}, {"SH_O_MASKED": "1"}, {"SH_V_BY_EXPERT": "1"}, {"SH_QK_SINGLE": "1"}, {"SH_QK_ONE_GRID": "1"},
                                 {"SH_SORT_SEPARATE": "1"}, {"SH_SIMT_STAGES": "31"},
                                 # the launch structure without the one-grid front (gate + sort and Q/K as kernels of their own)
                                 {"SH_NO_FRONT": "1"}, {"SH_NO_FRONT": "1", "SH_NO_PDL": "1"},
                                 {"SH_NO_FRONT": "1", "SH_NO_PDL": "1", "SH_NO_OVERLAP": "1"}, {"SH_NO_FRONT": "1", "SH_QK_SINGLE": "1"},
                                 {"SH_NO_FRONT": "1", "SH_QK_ONE_GRID": "1"}, {"SH_NO_FRONT": "1", "SH_SORT_SEPARATE": "1"},
                                 {"SH_NO_FRONT": "1", "SH_NO_PERSISTENT": "1"}],
                         ids=lambda e: "+".join(sorted(e)) or "default")
def test_launch_structure_switches_keep_the_result(env):
    run_case("switches", env)


def test_sparse_output_projection_shapes_with_index_checks_and_against_the_masked_kernel():
    run_case("sparse_o")
    run_case("sparse_o", {"SH_O_MASKED": "1"})
    run_case("sparse_o", {"SH_V_BY_EXPERT": "1"})
    run_case("sparse_o", {"SH_NO_FRONT": "1"})


def test_key_and_query_experts_with_index_checks():
    run_case("moe_qk")


def test_index_checks_stay_silent_on_edge_shapes():
    run_case("edges")


def test_index_check_records_a_bad_value_and_the_layer_recovers():
    run_case("index_selftest")
