"""The checking build of the library (-DLSA_CHECK): caller-given cache row numbers outside the cache are reported
(LSA_ERR_INDEX through lsa_status) and skipped instead of being read.  Runs in a child process that loads
liblsa_check.so; the normal build, which trusts its inputs, is never given such a list."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import json, sys, torch
sys.path.insert(0, sys.argv[1])
from paper_2608_01662_b200.configs import CONFIGS
from paper_2608_01662_b200.workload import PrefillWorkload
dev = torch.device("cuda:0")
res = {}
for name, base in (("mla", CONFIGS["cfg2"].replace(L=2048, M=8, Ksp=256, W=128, R=1, seed=5)), ("small", CONFIGS["cfg1"])):
    cfg = base.replace(name="chk_" + name)
    wl = PrefillWorkload(cfg, dev)
    wl.prepare()
    wl.step()
    good = wl.out[0].clone()
    # the caches as views of larger allocations: even a check that missed could not read outside device memory
    def roomy(x):
        big = torch.zeros((x.shape[0] + 256, x.shape[1]), dtype=x.dtype, device=dev)
        big[:x.shape[0]] = x
        return big[:x.shape[0]]
    k = wl.k[0]
    view = roomy(k)
    v = view if wl.v[0].data_ptr() == k.data_ptr() else roomy(wl.v[0])
    out = torch.empty_like(good)
    def attend(idx):
        wl.ctx.sparse_attn(wl.q[0], view, v, idx, wl.n_sparse, 0, wl.n_query, wl.n_key, out)
        torch.cuda.synchronize()
        return wl.ctx.status()
    r = {"clean_status": attend(wl.sparse_idx), "clean_equal": bool(torch.equal(out, good))}
    bad = wl.sparse_idx.clone()
    q_bad = cfg.L - 7                      # a late query: its sparse list is full
    bad[q_bad, 3] = wl.n_key               # one row past the end
    bad[q_bad - 1, 0] = -5                 # not the padding value
    r["bad_status"] = attend(bad)
    r["finite"] = bool(torch.isfinite(out.float()).all())
    r["after_status"] = attend(wl.sparse_idx)
    r["after_equal"] = bool(torch.equal(out, good))
    res[name] = r
print("RESULT " + json.dumps(res))
"""


def test_checking_build_reports_rows_outside_the_cache(cuda_device):
    from paper_2608_01662_b200 import build
    lib = build.build(check=True)
    env = dict(os.environ, LSA_LIBRARY=lib)
    pr = subprocess.run([sys.executable, "-c", CHILD, ROOT], env=env, capture_output=True, text=True, timeout=600)
    assert pr.returncode == 0, pr.stderr[-2000:]
    line = [l for l in pr.stdout.splitlines() if l.startswith("RESULT ")][-1]
    res = json.loads(line[len("RESULT "):])
    for name, r in res.items():
        assert r["clean_status"] == 0 and r["clean_equal"], (name, r)        # the checks change nothing on good input
        assert r["bad_status"] == -7 and r["finite"], (name, r)               # LSA_ERR_INDEX, reported once, nothing read
        assert r["after_status"] == 0 and r["after_equal"], (name, r)         # the status word was cleared by the read
