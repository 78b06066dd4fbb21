"""Parity under the bounds-checked build of the library (-DEG_DEBUG).

compute-sanitizer is not available where these tests run, so the library can be compiled with
index checks of its own: every index a kernel forms into a table (tile records, per-replica
modes, pipeline stages, partial sums, entry slots) is compared with the table's size first; a
miss sets a bit of the context's error word -- which the next synchronising call reports as an
error -- and the access is skipped.  Here a slice of the parity suite (ragged sizes, dense and
Top-K, the guessed and the repeated Top-K route, the single-launch kernel, more neighbours,
intermittent delivery, momentum, the pipelined kernel walking tiles handed out by a counter, quantised messages) runs against that build in a child process: it must pass, which
includes every eg_stats / eg_last_decisions call returning EG_OK, i.e. the error word staying 0.
"""
import os
import subprocess
import sys

import pytest

from paper_2103_07454_b200 import build

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SLICE = ("test_ragged_dense and (True-7 or False-64 or True-3 or False-5) or test_ragged_topk and (3-frac0 or 8-frac1) "
         "or test_topk_guess_and_exact_repeat and (5-True or -8-False) or test_topk_degenerate "
         "or test_more_neighbours_per_side and (9-4 or 16-8) or test_intermittent_delivery_topk "
         "or test_momentum_with_topk_and_history or test_history_and_horizon and 4-1.0 "
         "or test_graph_replay and walking_cap or test_quantised_messages_ragged and 5-True "
         "or test_quantised_topk_messages and 8-True")


def test_parity_slice_under_the_bounds_checked_build():
    lib = build.build_debug()
    env = dict(os.environ, EG_LIBRARY=lib, EG_EXPECT_DEBUG="1")
    run = subprocess.run([sys.executable, "-m", "pytest", os.path.join("tests", "test_gpu_parity.py"), "-q", "-x",
                          "-m", "gpu", "-p", "no:cacheprovider", "-k", SLICE],
                         cwd=ROOT, env=env, capture_output=True, text=True, timeout=1200)
    tail = run.stdout[-3000:] + run.stderr[-1000:]
    assert run.returncode == 0, tail
    assert " passed" in run.stdout and "failed" not in run.stdout, tail
    passed = int(run.stdout.rsplit(" passed", 1)[0].split()[-1])
    assert passed >= 30, tail
