"""The bounds-checked build (-DFQ_CHECKED: every kernel verifies the indices it computes, skips an access that would
fall outside its buffer and reports FQ_ERR_BOUNDS) runs a fixed set of calls in a child process: no check fires,
every result is bit-identical to the normal build's, and the guard words around every output are untouched."""
import os
import subprocess
import sys

import pytest
import torch

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))


def test_checked_build_fires_no_check_and_matches_the_normal_build(tmp_path):
    import paper_2501_07139_b200 as P
    from paper_2501_07139_b200.build import LIB_CHECKED
    import fq_checked_cases as cases
    assert os.path.exists(LIB_CHECKED), "libflexq_checked.so not built (python -m paper_2501_07139_b200.build --checked)"
    assert os.path.basename(P.lib_path()) == "libflexq.so"
    normal = cases.run_cases(P)
    assert bool(normal["guards_intact"][0])
    out = tmp_path / "checked.pt"
    env = dict(os.environ, FLEXQ_LIBRARY="checked")
    r = subprocess.run([sys.executable, os.path.join(HERE, "fq_checked_cases.py"), str(out)], env=env,
                       capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]         # (the child asserts fq_status() == 0 after each group)
    checked = torch.load(out)
    assert bool(checked["guards_intact"][0])
    assert set(checked) == set(normal)
    for key in normal:
        assert torch.equal(normal[key], checked[key]), key
