"""The debug build of the library (-DBRACE_DEBUG): its ring kernels check the index ranges they are
about to use and report through a status word instead of trapping.  The release build is what every
other test runs; here the debug build runs whole rounds (hop by hop and fused, sign and sum rules,
ragged and granule-1 layouts, the round without a workspace) in a child process, must give the same bits
as the release build, and must report that no check failed.  The release build answers
BRACE_ERR_UNSUPPORTED to the status query."""

import json
import os
import subprocess
import sys

import pytest
import torch

from paper_2501_17392_b200 import brace as B
from paper_2501_17392_b200 import build as brace_build

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import hashlib, json, sys
import torch
from paper_2501_17392_b200 import brace as B, workloads as W
digest = hashlib.sha256()
cases = [(20, 300_001, 128, B.RULE_SIGN_CONSENSUS), (5, 1_003, 1, B.RULE_SIGN_CONSENSUS), (9, 70_000, 128, B.RULE_SUM),
         (130, 40_000, 128, B.RULE_SIGN_CONSENSUS), (3, 2, 128, B.RULE_SIGN_CONSENSUS)]
for n, d, G, rule in cases:
    g = torch.Generator(device="cuda").manual_seed(n * 7 + d)
    ld = W.round_up(d, 128)
    U = torch.zeros((n, ld), dtype=torch.float32, device="cuda")
    U[:, :d].normal_(generator=g)
    for mode in (B.AGG_STEPWISE, B.AGG_AUTO):
        ctx = B.Brace(n, 0, d, B.default_params(rule=rule, lam=1.0, granule=G, agg_mode=mode))
        out = ctx.new_output()
        ctx.aggregate(U, out)
        torch.cuda.synchronize()
        digest.update(out.cpu().numpy().tobytes())
        ctx.close()
p = B.default_params(lam=1.0, agg_mode=B.AGG_FUSED)
U = torch.randn((20, 300_032), device="cuda", generator=torch.Generator(device="cuda").manual_seed(5))
out = torch.zeros((20, 9_376), dtype=torch.int32, device="cuda")
B.aggregate_static(20, 300_001, p, U, out)
torch.cuda.synchronize()
digest.update(out.cpu().numpy().tobytes())
status, code = B.debug_status()
print(json.dumps({"digest": digest.hexdigest(), "status": status, "code": code}))
"""


def run_child(library):
    env = dict(os.environ)
    env["BRACE_LIBRARY"] = library
    env["PYTHONPATH"] = ROOT + os.pathsep + env.get("PYTHONPATH", "")
    res = subprocess.run([sys.executable, "-c", CHILD], capture_output=True, text=True, env=env, cwd=ROOT, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    return json.loads(res.stdout.strip().splitlines()[-1])


def test_debug_build_same_bits_and_no_failed_check():
    assert torch.cuda.is_available(), "this test needs a CUDA device"
    release = run_child(brace_build.build())
    debug = run_child(brace_build.build_debug())
    assert release["status"] == B.ERR_UNSUPPORTED and release["code"] == 0
    assert debug["status"] == B.OK and debug["code"] == 0
    assert debug["digest"] == release["digest"]
