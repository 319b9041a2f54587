"""The pins must reject a wrong oracle: each planted mistake (compiled into a private copy of the oracle with
-DORC_MUTATION=n, on the CPU) has to fail at least one of the oracle's pin tests.  Mutation 0 (none) must pass."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

# mutation -> a pin test that must catch it
MUTATIONS = {
    1: "tests/test_oracle_formats.py::test_e2m1_midpoints_round_to_even_code",
    2: "tests/test_oracle_formats.py::test_enumeration_counts",
    3: "tests/test_oracle_quantize.py::test_scale_is_absmax_over_q",
    4: "tests/test_oracle_quantize.py::test_uniform_data_closed_form_and_decision",
    5: "tests/test_oracle_layer.py::test_against_library_matmul",
    6: "tests/test_oracle_quantize.py::test_selection_strict_less_first_wins_ties",
    7: "tests/test_oracle_formats.py::test_all_midpoints_and_grid_points",
    8: "tests/test_oracle_formats.py::test_int_rounding_ties_to_even_and_clamp",
    9: "tests/test_oracle_blocks.py::test_block_equals_the_slice_scored_as_its_own_tensor",
}


def _run(mutation, target, tmp_path):
    lib = tmp_path / f"liborc_mut{mutation}.so"
    subprocess.run(["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", f"-DORC_MUTATION={mutation}",
                    "-o", str(lib), os.path.join(ROOT, "oracle", "mofq_oracle.c"), "-lm"], check=True)
    env = dict(os.environ, MOFQ_ORACLE_LIB=str(lib))
    return subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider", target], cwd=ROOT, env=env,
                          capture_output=True, text=True)


@pytest.mark.parametrize("mutation", sorted(MUTATIONS))
def test_pins_catch_planted_mistake(mutation, tmp_path):
    r = _run(mutation, MUTATIONS[mutation], tmp_path)
    assert r.returncode != 0, f"mutation {mutation} slipped through {MUTATIONS[mutation]}"
    assert "failed" in r.stdout


def test_unmutated_copy_passes(tmp_path):
    r = _run(0, "tests/test_oracle_formats.py::test_e2m1_midpoints_round_to_even_code", tmp_path)
    assert r.returncode == 0, r.stdout[-2000:]
