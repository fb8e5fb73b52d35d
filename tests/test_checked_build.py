"""The checked build of the library (-DBAOC_CHECKED): every CTA of the streaming kernels validates its tile and the
ranges it will touch before touching memory, and records the first violation instead of faulting.  It stands in for a
memory checker where none can be run.  The checked library is a second shared object, chosen at import by
BAOC_CHECKED=1, so the GPU cases run in child processes."""
import os
import subprocess
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

# the odd-size and mixed cases of the parity suite: every kernel of the window, of the finalize and of the step, every
# update path, ragged tails, one-element blocks, sampling, re-configuration, both routes of the select's last pass and
# the repeated select
CASES = ("odd_sizes or each_configuration or stateless_bf16 or factored_with or finalize_from_shared or sampled_statistics "
         "or quantile_select or bias_corrected or extreme_shapes or least_alignment "
         "or reconfigure or configure_from_window or toy_pipeline or grouped_factored or nonfinite or coupled_decay "
         "or dynamic_codebook or adafactor")


def _child(args, timeout=1500):
    env = dict(os.environ, BAOC_CHECKED="1")
    return subprocess.run([sys.executable] + args, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


@pytest.mark.gpu
def test_parity_cases_run_clean_under_the_checked_build():
    from paper_2605_04711_b200 import build
    build.build(checked=True)
    r = _child(["-m", "pytest", "tests/test_gpu_parity.py", "-m", "gpu", "-x", "-q", "-k", CASES])
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "failed" not in r.stdout


@pytest.mark.gpu
def test_a_violation_is_recorded_and_the_context_stays_usable():
    from paper_2605_04711_b200 import build
    build.build(checked=True)
    code = (
        "import torch\n"
        "from paper_2605_04711_b200 import binding as B, harness as H, workloads as W\n"
        "assert B.CHECKED and B.check_status()['enabled'] == 1\n"
        "assert B.check_selftest() == 0\n"
        "st = B.check_status()\n"
        "assert st['code'] == 4 and st['kernel'] == 10 and st['a'] == 99 and st['b'] == 48 and st['c'] == 32 and st['d'] == 64, st\n"
        "assert B.check_status()['code'] == 0\n"                       # the record was cleared by the read
        "wl = W.make_workload('toy', seed=0)\n"
        "s = H.Session(wl, n_grad_sets=1); s.init_params(); s.fill_grads(1); s.sample_stats(0); s.sample_stats(0)\n"
        "risk, _ = s.risk(); s.configure([i % 3 for i in range(len(wl.blocks))]); s.step(0, 1)\n"
        "torch.cuda.synchronize()\n"
        "assert B.check_status()['code'] == 0 and s.verify_guards()\n"
        "print('ok')\n")
    r = _child(["-c", code], timeout=600)
    assert r.returncode == 0 and r.stdout.strip().endswith("ok"), r.stdout[-2000:] + r.stderr[-2000:]


def test_the_normal_build_reports_checks_disabled():
    from paper_2605_04711_b200 import binding as B
    assert not B.CHECKED
    assert B.check_status() == {"enabled": 0, "code": 0, "kernel": 0, "a": 0, "b": 0, "c": 0, "d": 0}
    assert B.check_selftest() == B.E_STATE


def test_both_builds_export_the_same_symbols():
    import ctypes
    from paper_2605_04711_b200 import binding as B, build
    lib = ctypes.CDLL(build.build(checked=True))
    for name in B.EXPORTS:
        assert hasattr(lib, name), name


def test_guard_bytes_detect_an_overrun():
    """The harness puts guard bytes around every device buffer; the check itself, on host memory: a write one byte past
    either end is seen, writes inside are not."""
    from paper_2605_04711_b200 import harness as H
    whole, view = H.guarded_alloc(1000, "cpu", fill_zero=True)
    assert view.numel() == 1000 and H.guards_intact(whole)
    view.fill_(7)
    assert H.guards_intact(whole)
    whole[H.GUARD_BYTES + 1000] = 0                                   # one past the end
    assert not H.guards_intact(whole)
    whole[H.GUARD_BYTES + 1000] = H.GUARD_BYTE
    assert H.guards_intact(whole)
    whole[H.GUARD_BYTES - 1] = 1                                      # one before the start
    assert not H.guards_intact(whole)
