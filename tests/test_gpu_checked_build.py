"""The checked build (-DDL_BOUNDS=1): stores through computed indices are compared with their buffers first; an
index outside is skipped and recorded, nothing traps.  The chained path must run clean under it (any recorded
index fails run_chained's final status check), with the same parity as the normal build; a deliberate store one
word past a buffer must be skipped and reported.  Runs in a child process, since the library is chosen at import."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys, torch
sys.path.insert(0, %r)
from paper_2412_00876_b200 import build, binding as dl
build.build(checked=True)
assert dl.lib().dl_build_is_checked() == 1
from tests import path_check as pc
pc.run_chained(1)
pc.run_chained(2, n_decode=8)
pc.run_chained(3, n_decode=6, B=3, L=2, ragged=True)
ctx = dl.Context(256, 4, 128, 64, torch.bfloat16, 0, max_batch=4, max_rows=64, cap=64)
assert ctx.selftest_bounds() == dl.DL_OK
torch.cuda.synchronize()
code, detail = ctx.device_status()
assert code == dl.DL_ERR_BOUNDS, code
assert detail == ((0x7e << 48) | 64), hex(detail)
# the context is still usable
q = torch.zeros(4, 4, 128, dtype=torch.bfloat16, device="cuda")
kc = torch.zeros(4, 4, 64, 128, dtype=torch.bfloat16, device="cuda")
ln = torch.zeros(4, dtype=torch.int32, device="cuda")
out = torch.empty_like(q)
ctx.sparse_attn_decode(q, q, q, kc, kc.clone(), ln, None, 0.1, out)
torch.cuda.synchronize()
ctx.close()
print("checked build ok")
""" % ROOT


def test_chained_path_runs_clean_under_the_checked_build_and_a_bad_index_is_caught():
    env = dict(os.environ, DL_SPARSE_CHECKED="1")
    r = subprocess.run([sys.executable, "-c", CHILD], capture_output=True, text=True, env=env, cwd=ROOT, timeout=900)
    assert r.returncode == 0 and "checked build ok" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]


def test_normal_build_has_no_checked_selftest():
    import torch
    from paper_2412_00876_b200 import binding as dl
    if dl.lib().dl_build_is_checked():
        pytest.skip("running against the checked build")
    ctx = dl.Context(256, 4, 128, 64, torch.bfloat16, 0, max_batch=4, max_rows=64, cap=64)
    assert ctx.selftest_bounds() == dl.DL_ERR_UNSUPPORTED
    ctx.close()
