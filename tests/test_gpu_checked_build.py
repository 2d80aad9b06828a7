"""The bounds-checked build of the library (-DSB_CHECKED): every store or load whose index comes
from data (a permutation entry, a sorted position, a look-back offset, a block's word offset, a
score record) is compared with the size of its buffer first; a failing index is latched in the
context's status word, the access is skipped (a gather reads entry 0 instead) and the next sync
reports SB_ERR_INVALID with the index and the limit.

The checked library is a second .so beside the product's; child processes load it through
SCALEBITS_LIB, so that the process running the rest of the suite keeps the product build."""
import os
import subprocess
import sys
import textwrap

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _checked_env():
    from paper_2602_17698_b200 import build
    assert os.path.exists(build.LIB_CHECKED), \
        "the checked library is missing: build it with __graft_entry__.build()"
    env = dict(os.environ)
    env["SCALEBITS_LIB"] = build.LIB_CHECKED
    env["PYTHONPATH"] = ROOT + os.pathsep + env.get("PYTHONPATH", "")
    return env


def test_parity_cases_pass_under_the_checked_build():
    """The kernel-level parity file and the first-order file, run through the checked library:
    same results, and no check fires on valid inputs."""
    probe = subprocess.run([sys.executable, "-c",
                            "from paper_2602_17698_b200 import binding; print(int(binding.checked_build()))"],
                           cwd=ROOT, env=_checked_env(), capture_output=True, text=True, timeout=600)
    assert probe.returncode == 0 and probe.stdout.strip() == "1", probe.stdout + probe.stderr
    run = subprocess.run([sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider",
                          "tests/test_gpu_parity.py", "tests/test_gpu_first_order.py"],
                         cwd=ROOT, env=_checked_env(), capture_output=True, text=True, timeout=1800)
    assert run.returncode == 0, run.stdout[-4000:] + run.stderr[-2000:]
    assert " passed" in run.stdout and "failed" not in run.stdout


CHILD = textwrap.dedent("""
    import torch
    from paper_2602_17698_b200 import binding
    from paper_2602_17698_b200.binding import Context, SbError, SB_ERR_INVALID
    assert binding.checked_build(), "this script must only ever run against the checked library"
    torch.cuda.set_device(0)
    dev = "cuda:0"
    R, C = 256, 512
    g = torch.Generator(device="cpu").manual_seed(0)
    # the matrix is a view of a larger allocation: whatever happened, index R or C stays inside it
    big = torch.randn((R + 8, C + 64), generator=g).to(torch.bfloat16).to(dev)
    W = big[:R, :C]
    ctx = Context()
    rp = torch.randperm(R, generator=g).to(torch.int32).to(dev)
    cp = torch.randperm(C, generator=g).to(torch.int32).to(dev)
    good = ctx.permute_matrix(W, rp, cp)
    ctx.sync()
    assert torch.equal(good, W[rp.long()][:, cp.long()])
    for which in ("row", "col"):
        bad_r, bad_c = rp.clone(), cp.clone()
        if which == "row":
            bad_r[17] = R                      # one entry past the last row
        else:
            bad_c[33] = C                      # one entry past the last column
        ctx.permute_matrix(W, bad_r, bad_c)
        try:
            ctx.sync()
        except SbError as e:
            assert e.status == SB_ERR_INVALID, e
            limit = R if which == "row" else C
            assert f"index {limit} outside [0, {limit})" in str(e), e
        else:
            raise AssertionError("a permutation entry outside the matrix was not reported")
        again = ctx.permute_matrix(W, rp, cp)  # the context stays usable and the status is clear
        ctx.sync()
        assert torch.equal(again, good)
    ctx.close()
    print("checked-ok")
""")


def test_a_permutation_entry_outside_the_matrix_is_caught_not_followed():
    run = subprocess.run([sys.executable, "-c", CHILD], cwd=ROOT, env=_checked_env(),
                         capture_output=True, text=True, timeout=600)
    assert run.returncode == 0 and "checked-ok" in run.stdout, run.stdout[-3000:] + run.stderr[-3000:]
