"""The pins must reject a wrong oracle: each planted mistake has to fail at least one of the oracle's pin tests.

The oracle source itself carries no test hooks.  A mistake is planted by editing a private copy of
``oracle/mofq_oracle.c`` (one exact text replacement, which must match exactly once), compiling that copy on the CPU
and pointing the pin test at it.  The unedited copy must pass."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SOURCE = os.path.join(ROOT, "oracle", "mofq_oracle.c")

# name -> (text in the oracle, what the mistake replaces it with, a pin test that must catch it)
MUTATIONS = {
    "fp_ties_away_from_zero": (
        "double m = nearbyint(ldexp(a, f.M - e));",
        "double m = floor(ldexp(a, f.M - e) + 0.5);",
        "tests/test_oracle_formats.py::test_e2m1_midpoints_round_to_even_code"),
    "e4m3_top_code_is_a_value": (
        "if (f.top_reserved == 2 && e == emax_field && m == (1 << f.M) - 1) return NAN;",
        "",
        "tests/test_oracle_formats.py::test_enumeration_counts"),
    "scale_uses_q_plus_one": (
        "float Q = (float)f.fmt_max;",
        "float Q = (float)f.fmt_max + 1.0f;",
        "tests/test_oracle_quantize.py::test_scale_is_absmax_over_q"),
    "inverse_scale_from_rounded_scale": (
        "*inv = Q / absmax;",
        "*inv = 1.0f / *scale;",
        "tests/test_oracle_quantize.py::test_scale_pair_is_two_correctly_rounded_quotients"),
    "mse_divides_by_rows": (
        "sse / (double)(rows * cols)",
        "sse / (double)rows",
        "tests/test_oracle_quantize.py::test_uniform_data_closed_form_and_decision"),
    "layer_output_reads_w_transposed": (
        "y += Xd[t * in + i] * Wd[o * in + i];",
        "y += Xd[t * in + i] * Wd[(i * out + o) % (out * in)];",
        "tests/test_oracle_layer.py::test_against_library_matmul"),
    "selection_takes_ties": (
        "if (errors[i] < min_error)",
        "if (errors[i] <= min_error)",
        "tests/test_oracle_quantize.py::test_selection_strict_less_first_wins_ties"),
    "subnormals_flushed": (
        "double m = nearbyint(ldexp(a, f.M - e));",
        "if (a < ldexp(1.0, 1 - f.bias)) a = 0.0;\n        double m = nearbyint(ldexp(a, f.M - e));",
        "tests/test_oracle_formats.py::test_all_midpoints_and_grid_points"),
    "int_ties_away_from_zero": (
        "double q = nearbyint((double)t);",
        "double q = t >= 0 ? floor((double)t + 0.5) : ceil((double)t - 0.5);",
        "tests/test_oracle_formats.py::test_int_rounding_ties_to_even_and_clamp"),
    "blocks_numbered_group_major": (
        "sse_out[r * per_row + b] = sse;",
        "sse_out[b * rows + r] = sse;",
        "tests/test_oracle_blocks.py::test_block_equals_the_slice_scored_as_its_own_tensor"),
}


def _run(edit, target, tmp_path):
    text = open(SOURCE).read()
    if edit is not None:
        old, new = edit
        assert text.count(old) == 1, f"the oracle no longer contains exactly one {old!r}: update this test"
        text = text.replace(old, new)
    src = tmp_path / "mofq_oracle_copy.c"
    src.write_text(text)
    lib = tmp_path / "liborc_copy.so"
    subprocess.run(["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", "-o", str(lib), str(src), "-lm"], check=True)
    env = dict(os.environ, MOFQ_ORACLE_LIB=str(lib))
    return subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider", target], cwd=ROOT, env=env,
                          capture_output=True, text=True)


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_pins_catch_planted_mistake(name, tmp_path):
    old, new, target = MUTATIONS[name]
    r = _run((old, new), target, tmp_path)
    assert r.returncode != 0, f"planted mistake {name} slipped through {target}"
    assert "failed" in r.stdout


def test_unedited_copy_passes(tmp_path):
    r = _run(None, "tests/test_oracle_formats.py::test_e2m1_midpoints_round_to_even_code", tmp_path)
    assert r.returncode == 0, r.stdout[-2000:]
