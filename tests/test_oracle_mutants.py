"""Plant one plausible mistake at a time in a copy of the oracle's source (on the CPU)
and check that the pins notice: a pin suite that lets a mutant through pins nothing."""
import ctypes
import os
import subprocess

import pytest

from oracle import ref
from tests.oracle_pins import ALL_PINS

MUTANTS = {
    "mean_not_divided": ("float Dnew = acc / fK;", "float Dnew = acc;"),
    "update_sign": ("r[j] = std::fmaf(-s->mu, mnew, r[j]);", "r[j] = std::fmaf(s->mu, mnew, r[j]);"),
    "dropped_worker": ("for (int i = 1; i < s->K; ++i) acc", "for (int i = 2; i < s->K; ++i) acc"),
    "no_delay": ("if (s->D_valid) s->w[j] = s->w[j] + s->D[j];", "s->w[j] = s->w[j] + Dnew;"),
    "replicas_not_recloned": ("for (int i = 0; i < s->K; ++i) s->r[i][j] = s->w[j];", ""),
    "momentum_operands_swapped": ("std::fmaf(s->beta, m[j], gd)", "std::fmaf(s->beta, gd, m[j])"),
    "decay_on_gradient": ("std::fmaf(s->lambda, r[j], g[j])", "std::fmaf(s->lambda, g[j], g[j])"),
    "merge_resets_momentum": ("for (int i = 0; i < s->K; ++i) s->r[i][j] = s->w[j];",
                              "for (int i = 0; i < s->K; ++i) { s->r[i][j] = s->w[j]; s->m[i][j] = 0.f; }"),
    "global_subtracted_once": ("acc = acc + (s->r[i][j] - s->w[j]);", "acc = acc + s->r[i][j];"),
    "inactive_rows_not_zeroed": ("for (int64_t j = seg_start; j < seg_start + rows * cols; ++j) g[j] = 0.f;", ""),
    "clone_before_commit": [("float Dnew = acc / fK;",
                             "float Dnew = acc / fK; for (int i = 0; i < s->K; ++i) s->r[i][j] = s->w[j];"),
                            ("        for (int i = 0; i < s->K; ++i) s->r[i][j] = s->w[j];\n", "")],
    "accum_not_reset": ("s->a[i][j] = 0.f;", ""),
    "accum_sum_not_mean": ("s->synced[j] = sum / fK;", "s->synced[j] = sum;"),
    "accum_commit_without_lr": ("s->w[j] = std::fmaf(-s->mu, s->synced[j], s->w[j]);", "s->w[j] = s->w[j] - s->synced[j];"),
    "accum_commit_not_delayed": ("if (s->synced_valid) s->w[j] = std::fmaf(-s->mu, s->synced[j], s->w[j]);",
                                 "s->w[j] = std::fmaf(-s->mu, s->a[0][j], s->w[j]);"),
    "accum_replica_not_updated": ("r[j] = std::fmaf(-s->mu, g[j], r[j]);\n        a[j]", "a[j]"),
    "accum_first_worker_twice": ("for (int i = 1; i < s->K; ++i) sum = sum + s->a[i][j];",
                                 "for (int i = 1; i < s->K; ++i) sum = sum + s->a[0][j];"),
    "pending_overwritten_early": ("float Dnew = acc / fK;", "float Dnew = acc / fK; s->D[j] = Dnew;"),
}


def _build_mutant(tmp_path, name):
    edits = MUTANTS[name]
    if isinstance(edits, tuple):
        edits = [edits]
    src = open(os.path.join(os.path.dirname(ref.__file__), "hpsgd_ref.cpp")).read()
    for old, new in edits:
        assert src.count(old) == 1, "mutation site for %s not found exactly once" % name
        src = src.replace(old, new)
    path = tmp_path / (name + ".cpp")
    path.write_text(src)
    lib = tmp_path / (name + ".so")
    subprocess.run(["g++", *ref.CXXFLAGS, "-o", str(lib), str(path)], check=True, capture_output=True)
    return ref.load(str(lib))


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_pins_catch_mutant(tmp_path, name):
    lib = _build_mutant(tmp_path, name)
    caught = []
    for pin in ALL_PINS:
        try:
            pin(lib)
        except AssertionError:
            caught.append(pin.__name__)
    assert caught, "no pin noticed the planted mistake %r" % name
