"""Failure paths that no healthy run takes, exercised in their safe forms: a bounded device-side wait that is made to
run out (a one-thread kernel waiting on a barrier nobody signals: nothing is starved, nothing hangs), and the checking
build of the library (every index read from memory is range-checked and counted, never trapped on)."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

from paper_1701_06538_b200 import binding as B
from paper_1701_06538_b200 import build as moe_build
from paper_1701_06538_b200 import synth

from helpers import act_empty, cfg_of, dev, dev_act, f32, host, i32, small_workload

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_a_bounded_wait_that_runs_out_reports_timeout_and_leaves_the_context_usable():
    w = small_workload("timeout", T=512, d=64, h=64, n=4, k=2, act="bf16", seed=71)
    cfg = cfg_of(w)
    S = B.moe_query_sizes(cfg)
    ws = B.empty_bytes(S.ws_bytes)
    B.moe_debug_wait_timeout(ws, 1_000_000)          # one millisecond on a barrier nobody arrives at
    assert B.moe_check_status(ws) == 5                # MOE_ERR_TIMEOUT, read back on the host
    assert B.lib().moe_status_string(5) == b"device-side wait timed out"
    # the kernel returned normally: the same workspace and context carry on, and the next call clears the word
    I = synth.make_all(w)
    from oracle import moe_oracle as O
    D = O.dispatch(I["x"], np.stack([np.arange(w.T) % w.n, (np.arange(w.T) + 1) % w.n], 1).astype(np.int32), w.n)
    hid, ys = act_empty(w, S.R, w.h), act_empty(w, S.R, w.d)
    B.moe_expert_ffn(cfg, dev_act(D.xs, w), dev(D.offsets), dev_act(I["W1"], w), dev_act(I["b1"], w), dev_act(I["W2"], w),
                     dev_act(I["b2"], w), hid, ys, ws)
    assert B.moe_check_status(ws) == 0
    assert torch.isfinite(ys.float()).all()
    with pytest.raises(B.MoeError):                   # the limit is capped: nobody can park a kernel for long
        B.moe_debug_wait_timeout(ws, 10 ** 9)


def run_on_checking_build(args, expect_violations):
    lib = moe_build.build_checking()
    env = dict(os.environ, MOE_B200_LIB=lib, MOE_EXPECT_VIOLATIONS="1" if expect_violations else "0")
    return subprocess.run([sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider"] + args,
                          cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)


def test_checking_build_sees_no_out_of_range_index_on_the_small_and_odd_shapes():
    """The stage tests (ragged, k = 1, k = n, empty experts, largest n, screened and unscreened gates) and the
    hierarchical ones, run once on the library compiled with -DMOE_BOUNDS_CHECK: same results (the tests' own
    assertions), and the index checks must not have fired."""
    res = run_on_checking_build(["tests/test_gpu_stages.py", "tests/test_gpu_hier.py", "tests/test_gpu_layer.py", "-k",
                                 "not many_batches and not badly_scaled and not drops_expert_ids and not pure_chain"], False)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-2000:]
    assert "checking build: 0 out-of-range" in res.stdout


def test_checking_build_counts_what_the_guards_skip():
    """Positive control: caller-made expert ids outside [0, n) are dropped in every build; the checking build counts them."""
    res = run_on_checking_build(["tests/test_gpu_stages.py", "-k", "drops_expert_ids"], True)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-2000:]
