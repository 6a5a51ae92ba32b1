"""The two forms of elm_express_prefill on bf16 inputs in fp32 mode - one attention launch per round over a list
gathered once, and windows of 512 tokens - compute the same thing: same coresets, outputs equal up to the bf16
rounding of differently ordered sums.  The form is chosen when the library is loaded (ELM_PREFILL_ROUNDS), so each
runs in a process of its own."""
import os
import subprocess
import sys

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)


def _run(tmp_path, rounds):
    path = str(tmp_path / f"prefill_rounds{rounds}.npz")
    env = dict(os.environ, ELM_PREFILL_ROUNDS=str(rounds), PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    subprocess.run([sys.executable, os.path.join(HERE, "_prefill_forms_child.py"), path], check=True, env=env, cwd=ROOT,
                   timeout=600)
    return np.load(path)


def test_one_launch_per_round_equals_windows(tmp_path):
    sys.path.insert(0, HERE)
    from _prefill_forms_child import SHAPES
    a, b = _run(tmp_path, 1), _run(tmp_path, 0)
    for i, shape in enumerate(SHAPES):
        assert np.array_equal(a[f"idx{i}"], b[f"idx{i}"]), shape
        Oa, Ob = a[f"O{i}"], b[f"O{i}"]
        assert not np.isnan(Oa).any() and not np.isnan(Ob).any()
        diff = np.max(np.abs(Oa - Ob)) / np.max(np.abs(Ob))
        print(shape, f"max difference {diff:.3e} of the largest output; launches {int(a[f'launches{i}'])} / {int(b[f'launches{i}'])}")
        assert diff <= 1e-2, shape
        # the one-launch form really ran (far fewer launches than one per window)
        assert a[f"launches{i}"] < b[f"launches{i}"], shape
