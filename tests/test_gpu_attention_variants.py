"""The attention kernel is chosen by problem size (one or two query tiles per CTA on the tcgen05
path, mma.sync for head dimension 64), so the small parity cases never reach some of the kernels
that the full-size runs use, e.g. the two-query-tile kernel reading two key sources (shared affix
storage), and switches such as the grouping of four requests per decode-pass tile have a second path.  The choice is read from the environment once per process; each case below runs the
attention-heavy parity tests in a child process with one kernel forced."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SELECT = ("shared or layer_step or recompute_then_scatter or duplicate_row or full_size or idempotent or "
          "generate_block or decode_over_shared")


@pytest.mark.parametrize("switch", ["ACACHE_ATTN_TC2Q=2", "ACACHE_ATTN_TC2Q=0", "ACACHE_ATTN_TC=0", "ACACHE_ATTN_GROUP=0"])
def test_parity_with_one_attention_kernel_forced(switch):
    name, value = switch.split("=")
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
           "tests/test_gpu_parity.py", "tests/test_gpu_predict_commit.py", "tests/test_gpu_generate.py", "-k", SELECT]
    r = subprocess.run(cmd, cwd=ROOT, env={**os.environ, name: value}, capture_output=True, text=True, timeout=1200)
    assert r.returncode == 0, (r.stdout[-3000:], r.stderr[-1000:])
    assert " passed" in r.stdout and "no tests ran" not in r.stdout


@pytest.mark.parametrize("switch", ["ACACHE_SCORE_SMALL=0", "ACACHE_SCORE_TC=0", "ACACHE_KEEP_WQ=0", "ACACHE_SCORE_FUSED=0", "ACACHE_SCORE_ONEPASS=0"])
def test_parity_with_one_scoring_path_forced(switch):
    """Short affixes are scored by the one-launch cluster kernel and long ones on tcgen05; with either switched off
    the two mma.sync kernels take their place; a probe at head dimension 128 takes its scores out of its own attention, with
    that switched off the separate kernels score it.  The scoring, layer-step and probe parity cases must hold on every path."""
    name, value = switch.split("=")
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
           "tests/test_gpu_parity.py", "tests/test_gpu_multilayer.py", "tests/test_gpu_configs.py", "-k",
           "score_anchors or layer_step or full_size or probe or sweep_points or full_context"]
    r = subprocess.run(cmd, cwd=ROOT, env={**os.environ, name: value}, capture_output=True, text=True, timeout=1200)
    assert r.returncode == 0, (r.stdout[-3000:], r.stderr[-1000:])
    assert " passed" in r.stdout and "no tests ran" not in r.stdout


@pytest.mark.parametrize("csize", [1, 2, 4, 8])
def test_scoring_with_every_cluster_size_forced(csize):
    """The one-pass tcgen05 scoring kernel picks its cluster size (CTAs per head and request) from the problem; each size is
    forced in turn over the scoring cases (ragged and empty key ranges per CTA, both normalisers, a cache shared by the batch)
    and the full-context layer-steps."""
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
           "tests/test_gpu_parity.py", "tests/test_gpu_configs.py", "-k", "score_anchors or full_context"]
    r = subprocess.run(cmd, cwd=ROOT, env={**os.environ, "ACACHE_SCORE_CLUSTER": str(csize)}, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, (r.stdout[-3000:], r.stderr[-1000:])
    assert " passed" in r.stdout and "no tests ran" not in r.stdout
