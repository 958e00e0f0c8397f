"""Each pin must be able to fail: one mistake at a time is planted in a COPY of the oracle's
source (on the CPU, in a temporary folder) and the pin that is meant to catch it is run against
that copy in a child process, which has to fail; the unchanged copy has to pass."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "aaac_oracle.c")

# (name, text in the source, what it becomes, the pin that must notice)
MUTATIONS = [
    ("selection tie goes to table 1",
     "int sigma = (E[1] < E[0]) ? 1 : 0;", "int sigma = (E[1] <= E[0]) ? 1 : 0;",
     "test_zero_rounds_fixed_grid_is_round_to_nearest"),
    ("importance dropped from the group error",
     "E[r] += (double)I[k] * (d * d);", "E[r] += (d * d);",
     "test_selection_and_codes_are_brute_force_optimal"),
    ("equidistant entries: the larger one wins",
     "if (d < bd || (d == bd && T[i] < T[best])) { bd = d; best = i; }", "if (d <= bd) { bd = d; best = i; }",
     "test_pack_counts_weights_half_way_between_two_entries"),
    ("nibble order swapped",
     "if (e & 1) codes[e >> 1]", "if (!(e & 1)) codes[e >> 1]",
     "test_sign_bit_round_trip_and_dequant"),
    ("Eq. 10 offset doubled",
     "const double d = 1.0 / (2.0 * (M - 1));", "const double d = 1.0 / (1.0 * (M - 1));",
     "test_quantile_init_matches_numpy"),
    ("INT4 scale divides by 8",
     "s = bf16_to_f32(f32_to_bf16(a / 7.f));", "s = bf16_to_f32(f32_to_bf16(a / 8.f));",
     "test_int4_scales_absmax_over_7_and_range"),
    ("grid start: last entry of T1 a full step up",
     "T01[2 * M - 1] = T01[M - 1] + 0.5 * (T01[M - 1] - T01[M - 2]);",
     "T01[2 * M - 1] = T01[M - 1] + 1.0 * (T01[M - 1] - T01[M - 2]);",
     "test_grid_start_second_table_is_the_first_moved_up_half_a_step"),
    ("grid start: T1 a full step up",
     "T01[M + i] = 0.5 * (T01[i] + T01[i + 1]);", "T01[M + i] = T01[i + 1];",
     "test_grid_start_second_table_is_the_first_moved_up_half_a_step"),
    ("half-way count also counts duplicate entries",
     "if (T01[sigma * M + i] != T01[sigma * M + idx[k]] && fabs(x - T01[sigma * M + i]) == d) { ++t1; break; }",
     "if (i != idx[k] && fabs(x - T01[sigma * M + i]) == d) { ++t1; break; }",
     "test_pack_counts_weights_half_way_between_two_entries"),
    ("centroid not weighted by the importance",
     "p[sigma * M + idx[k]] += (double)imp[k] * (double)w[k];", "p[sigma * M + idx[k]] += (double)w[k];",
     "test_identical_tables_reduce_to_single_codebook_weighted_kmeans"),
    ("tables rounded to BF16 by truncation",
     "u += 0x7FFFu + ((u >> 16) & 1u);", "u += 0u;",
     "test_bf16_rounding_matches_ml_dtypes"),
]


def _run_pin(src_path, pin):
    env = dict(os.environ, AAAC_ORACLE_SRC=src_path)
    return subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_oracle_pins.py"), "-x", "-q",
                           "-k", pin, "-p", "no:cacheprovider"], cwd=ROOT, env=env, capture_output=True, text=True)


def test_unchanged_copy_passes(tmp_path):
    dst = tmp_path / "oracle_copy.c"
    dst.write_text(open(SRC).read())
    pins = " or ".join(sorted({m[3] for m in MUTATIONS}))
    r = _run_pin(str(dst), pins)
    assert r.returncode == 0, r.stdout[-2000:]


@pytest.mark.parametrize("name,old,new,pin", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_fails_its_pin(tmp_path, name, old, new, pin):
    text = open(SRC).read()
    assert text.count(old) == 1, f"the source no longer holds exactly one copy of: {old}"
    dst = tmp_path / "oracle_mutated.c"
    dst.write_text(text.replace(old, new))
    r = _run_pin(str(dst), pin)
    assert r.returncode == 1, f"{name}: the pin {pin} did not fail\n{r.stdout[-1500:]}"
    assert "failed" in r.stdout
