"""The range-checked debug build (-DSP_DEBUG), the stand-in for a memory checker: the small parity tests run under
it in a child process (same results, status word clean), and lists that point outside their range are caught by its
checks: reported as SP_ERR_RANGE with the id of the check, with every access kept inside the caller's buffers."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _debug_env():
    from paper_2505_19578_b200 import build
    lib = build.build(debug=True)
    env = dict(os.environ, SHAREPREFILL_LIB=lib)
    return env, lib


def test_small_parity_tests_pass_under_the_range_checked_build():
    env, lib = _debug_env()
    r = subprocess.run([sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "tests/test_gpu_parity.py", "-k",
                        "dense_pivot or block_sparse or prefill_tiny or degenerate or block_mask"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout


_BAD_LIST = r'''
import sys, torch
from paper_2505_19578_b200 import binding
assert binding.LIB_PATH.endswith("libshareprefill_debug.so"), binding.LIB_PATH
for d, B, where in ((128, 128, 50), (64, 64, 60)):
    N = 8 * B
    Nb = N // B
    g = torch.Generator().manual_seed(1)
    q = torch.randn(2, N, d, generator=g).to(torch.bfloat16).cuda()
    k = torch.randn(1, N, d, generator=g).to(torch.bfloat16).cuda()
    out = torch.zeros_like(q)
    counts = torch.ones(1, Nb, dtype=torch.int32)
    idx = torch.full((1, Nb, Nb), -1, dtype=torch.int32)
    for i in range(Nb):
        idx[0, i, 0] = i
    idx[0, 3, 0] = 6            # a key-block after the diagonal of row-block 3
    ctx = binding.Context()
    ctx.sp_block_sparse_attn(q, k, k, [0, 1], [0, 0], counts.cuda(), idx.cuda(), B, out)
    torch.cuda.synchronize()
    code, where_got = ctx.status()
    assert (code, where_got) == (binding.SP_ERR_RANGE, where), (d, B, code, where_got)
    # the status is cleared by the read and a well-formed call then works
    idx[0, 3, 0] = 3
    out.fill_(float("nan"))
    ctx.sp_block_sparse_attn(q, k, k, [0, 1], [0, 0], counts.cuda(), idx.cuda(), B, out)
    torch.cuda.synchronize()
    assert ctx.status() == (0, 0) and torch.isfinite(out.float()).all()
print("range checks ok")
'''


def test_out_of_range_list_is_reported_not_followed():
    env, lib = _debug_env()
    r = subprocess.run([sys.executable, "-c", _BAD_LIST], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "range checks ok" in r.stdout, r.stdout[-2000:] + r.stderr[-3000:]
