"""lsa_index_static, the no-allocation variant of the indexer, against lsa_index (needs a B200).

Collected last on purpose: if it fails under `pytest -x`, every other test has already run.
The variant keeps its page-score scratch in a fixed device array inside the library, for callers that
cannot obtain device memory (an engine that owns the whole GPU, a plugin without an allocator).  It must
return exactly what lsa_index returns, on a first call (which looks up the array's address) and on a
second call that reuses the array with the first call's contents still in it.
"""
import pytest
import torch

from paper_2608_01662_b200 import binding
from paper_2608_01662_b200.configs import CONFIGS
from paper_2608_01662_b200.workload import PrefillWorkload

pytestmark = pytest.mark.gpu


def _run_static(wl, q0, n):
    idx = torch.full((n, wl.cfg.Ksp), -7, dtype=torch.int32, device=wl.device)
    cnt = torch.full((n,), -7, dtype=torch.int32, device=wl.device)
    binding.index_static(wl.params, wl.q_idx[q0 - wl.q_pos0:], wl.w[q0 - wl.q_pos0:], wl.keys["k"], wl.keys.get("scale"),
                         wl.kmean, q0, n, wl.n_key, idx, cnt)
    torch.cuda.synchronize()
    assert binding.index_static_status(wl.device) == 0     # no bounded device-side wait ran out
    return idx, cnt


def test_static_scratch_indexer_matches_workspace_indexer_twice(cuda_device):
    # first call: fp8 keys, 6000 tokens (ragged last page), hierarchical stage active
    cfg_a = CONFIGS["cfg3"].replace(name="na_fp8", L=6000, M=8, Ksp=512, W=384, R=1, seed=21)
    a = PrefillWorkload(cfg_a, cuda_device)
    a.prepare()
    a.index()
    idx, cnt = _run_static(a, 0, cfg_a.L)
    assert torch.equal(idx, a.sparse_idx) and torch.equal(cnt, a.n_sparse)      # integer work: exact

    # second call right after, different shape and bf16 keys: the array still holds call one's scores
    cfg_b = CONFIGS["cfg1"].replace(name="na_bf16", seed=22)
    b = PrefillWorkload(cfg_b, cuda_device)
    b.prepare()
    b.index()
    idx, cnt = _run_static(b, 0, cfg_b.L)
    assert torch.equal(idx, b.sparse_idx) and torch.equal(cnt, b.n_sparse)
    # a query sub-range with an offset, again on the shared array
    idx, cnt = _run_static(a, 4000, 1500)
    assert torch.equal(idx, a.sparse_idx[4000:5500]) and torch.equal(cnt, a.n_sparse[4000:5500])


def test_static_scratch_refuses_misaligned_pointers_before_any_launch(cuda_device):
    """The kernels read q_idx, w, k_idx and kmean with 16-byte vector loads: a pointer off by two bytes is refused with
    LSA_ERR_SHAPE by the host-side checks (the same ones lsa_index makes); nothing reaches the GPU."""
    cfg = CONFIGS["cfg1"]
    params = binding.make_params(cfg)
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device=cuda_device)
    ok, off = buf[256:], buf[258:]
    out = torch.zeros(64, dtype=torch.int32, device=cuda_device)
    for which in range(4):
        ptrs = [off if i == which else ok for i in range(4)]     # q_idx, w, k_idx, kmean
        with pytest.raises(binding.LsaError) as e:
            binding.index_static(params, ptrs[0], ptrs[1], ptrs[2], None, ptrs[3], 0, 4, 64, out, out)
        assert e.value.code == -2
    torch.cuda.synchronize()
    assert binding.index_static_status(cuda_device) == 0


def test_static_scratch_capacity_is_enforced(cuda_device):
    """A call whose page-score matrix would not fit the fixed array is refused before anything is launched."""
    cfg = CONFIGS["cfg2"]                           # 32768 queries x 512 pages x 4 B = 64 MiB > 8 MiB
    params = binding.make_params(cfg)
    dummy = torch.zeros(64, dtype=torch.int32, device=cuda_device)   # never touched: the size check comes first
    with pytest.raises(binding.LsaError) as e:
        binding.index_static(params, dummy, dummy, dummy, None, dummy, 0, cfg.L, cfg.L, dummy, dummy)
    assert e.value.code == -6
    assert binding.STATIC_SCRATCH_BYTES == 8 << 20
    torch.cuda.synchronize()
