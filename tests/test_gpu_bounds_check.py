"""The range-checked build of the library (-DDP_BOUNDS_CHECK): every index a kernel computes from
data -- the gathered column of the tied cross term, the sorted positions of the scatter, ranks and
partial-sum slots -- is compared with its array's extent before the access.  The small-shape
parity tests (ragged T, K tails, odd widths, frequent tokens) are run once more in a child process
that loads that build: every one of them asserts a clean device status, so an index outside its
array anywhere fails here.  No memory checker may be run on this machine; this stands in for one."""
import os
import subprocess
import sys

import pytest
import torch

from paper_2609_40335_b200 import binding as dp

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CHECK_LIB = os.path.join(ROOT, "paper_2609_40335_b200", "libdp_ghost_check.so")

SELECT = ("test_tied_cross_term or test_embed_norms_and_first_occurrence or test_clip_accumulate_embed "
          "or test_linear_norms_bf16_tensor_core or test_pair_and_single_cta_gram_kernels_agree "
          "or test_clip_accumulate_bf16_tensor_core or test_vector_parameter "
          "or test_step_graph_with_positions_and_full_parameter_set or test_cfg1_end_to_end_fp32")


def _child(code):
    env = dict(os.environ, DP_GHOST_LIB=CHECK_LIB, PYTHONPATH=ROOT)
    return subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=900)


def test_normal_build_is_not_checked_and_probe_is_silent():
    assert dp.load().dp_debug_bounds_checked() == 0
    st = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    dp._check(dp.load().dp_debug_bounds_probe(7, 3, st.data_ptr(), torch.cuda.current_stream().cuda_stream), "probe")
    torch.cuda.synchronize()
    assert int(st.item()) == 0


def test_checked_build_reports_an_index_outside_its_array():
    if not os.path.exists(CHECK_LIB):
        from paper_2609_40335_b200 import build
        build.build(check=True)
    r = _child(
        "import torch\n"
        "from paper_2609_40335_b200 import binding as dp\n"
        "L = dp.load(); assert L.dp_debug_bounds_checked() == 1\n"
        "st = torch.zeros(1, dtype=torch.int32, device='cuda:0')\n"
        "s = torch.cuda.current_stream().cuda_stream\n"
        "for idx, n, want in ((2, 3, 0), (3, 3, dp.DP_DEV_BOUNDS), (-1, 3, dp.DP_DEV_BOUNDS)):\n"
        "    st.zero_(); dp._check(L.dp_debug_bounds_probe(idx, n, st.data_ptr(), s), 'probe')\n"
        "    torch.cuda.synchronize(); assert int(st.item()) == want, (idx, n, int(st.item()))\n"
        "print('probe ok')\n")
    assert r.returncode == 0 and "probe ok" in r.stdout, r.stdout + r.stderr


def test_small_shape_parity_suite_is_clean_under_the_checked_build():
    if not os.path.exists(CHECK_LIB):
        from paper_2609_40335_b200 import build
        build.build(check=True)
    env = dict(os.environ, DP_GHOST_LIB=CHECK_LIB)
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_parity.py"),
                        "-x", "-q", "-m", "gpu", "-k", SELECT, "-p", "no:cacheprovider"],
                       env=env, cwd=ROOT, capture_output=True, text=True, timeout=1500)
    tail = (r.stdout + r.stderr)[-1500:]
    assert r.returncode == 0, tail
    assert " passed" in r.stdout and "failed" not in r.stdout, tail
