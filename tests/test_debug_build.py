"""The -DMOE_DEBUG build of the library (index guards in the routing kernel, a
canary after every workspace section, both reported by moe_route_poll as
MOE_ERR_INTERNAL) stands in for a memory checker.  The small parity cases run
against it in a child process -- the binding picks the library named by
MOE_ROUTE_LIB -- and must pass without a guard or canary report; a canary
overwritten from the host must be reported."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

from paper_2609_39137_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
pytestmark = pytest.mark.gpu


def _is_debug_library():
    return binding.load().moe_debug_build() == 1


def test_small_parity_cases_pass_on_the_debug_build():
    if _is_debug_library():
        pytest.skip("already running against the debug build")
    lib = build.build(debug=True)
    env = dict(os.environ, MOE_ROUTE_LIB=lib)
    select = ("test_route_matches_oracle or test_route_edge_shapes or chunk_split_scheduling or random_shapes "
              "or gives_up or exact_ties or canary or one_launch or non_finite")
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-v", "-m", "gpu", "-p", "no:cacheprovider",
                        os.path.join("tests", "test_gpu_parity.py"), os.path.join("tests", "test_debug_build.py"),
                        "-k", select], env=env, cwd=ROOT, capture_output=True, text=True, timeout=1200)
    assert r.returncode == 0, (r.stdout[-4000:] + r.stderr[-2000:])
    assert "test_overwritten_canary_is_reported_by_poll PASSED" in r.stdout     # the child really ran the debug library
    assert r.stdout.count(" PASSED") >= 40 and " FAILED" not in r.stdout


def test_overwritten_canary_is_reported_by_poll():
    if not _is_debug_library():
        pytest.skip("needs the debug build (run by test_small_parity_cases_pass_on_the_debug_build)")
    r = binding.Router(2, 768, 10, 64, 256)
    assert r.poll(raise_on_error=False) == binding.MOE_OK
    ws = r.workspace
    # the canaries are 256-byte runs of 0xC5 on 256-byte boundaries, written by moe_route_init
    blocks = ws[: (ws.numel() // 256) * 256].view(-1, 256)
    guards = torch.nonzero((blocks == 0xC5).all(dim=1)).flatten()
    assert guards.numel() >= 8
    victim = int(guards[3])
    ws[victim * 256 + 17] = 0                      # what a stray write past the end of a section would do
    assert r.poll(raise_on_error=False) == binding.MOE_ERR_INTERNAL
    assert "canary" in r.lib.moe_last_error(r.h).decode()
    ws[victim * 256 + 17] = 0xC5
    assert r.poll(raise_on_error=False) == binding.MOE_OK
