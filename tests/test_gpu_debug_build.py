"""The debug build of the library (-DKVSINK_DEBUG: index checks that raise a status bit and skip the access, never a
trap) runs the same parity cases as the release build with a clean status word.  It runs in a process of its own because
a process binds one build of the library."""
import os
import subprocess
import sys

import pytest

from paper_2508_04257_b200 import build as kv_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SCRIPT = r"""
import sys
sys.path.insert(0, sys.argv[1]); sys.path.insert(0, sys.argv[1] + "/tests")
import torch
import paper_2508_04257_b200 as kv
from paper_2508_04257_b200 import binding, synth
from parity_util import run_both
assert binding.lib()._name.endswith("libkvsink_debug.so")
TINY = synth.WORKLOADS["tiny"]
run_both(TINY, appends=3)
for bits, group, hq, hkv in ((2, 128, 4, 4), (3, 64, 8, 2), (4, 64, 16, 2), (2, 64, 6, 2)):
    wl = TINY.scaled(bits=bits, head_dim=128, group=group, n_q_heads=hq, n_kv_heads=hkv, batch=2, seq=3 * group + 37, topk=5, pfn_n=2, seed=99 + bits)
    r = run_both(wl, appends=2)          # asserts parity and a zero status word
print("debug build ok")
"""


@pytest.mark.gpu
def test_debug_build_runs_the_path_with_a_clean_status_word():
    if not os.path.exists(kv_build.DEBUG_LIB):
        pytest.skip("libkvsink_debug.so has not been built (python -m paper_2508_04257_b200.build --debug)")
    env = dict(os.environ, KVSINK_LIB=kv_build.DEBUG_LIB)
    r = subprocess.run([sys.executable, "-c", SCRIPT, ROOT], capture_output=True, text=True, env=env, timeout=600)
    assert r.returncode == 0 and "debug build ok" in r.stdout, r.stdout[-1500:] + r.stderr[-3000:]
