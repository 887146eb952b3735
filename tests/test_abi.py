"""The C-ABI library builds, loads and exports every symbol include/lsa.h declares (no GPU needed)."""
import ctypes
import os
import re

from paper_2608_01662_b200 import binding, build
from paper_2608_01662_b200.configs import CONFIGS

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "lsa.h")).read()
    return sorted(set(re.findall(r"^LSA_API [\w\s\*]*?\b(lsa_\w+)\(", text, flags=re.M)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    handle = ctypes.CDLL(path)
    names = _declared()
    assert len(names) >= 14
    for n in names:
        assert hasattr(handle, n), n
    assert set(names) == set(binding.EXPORTS), set(names) ^ set(binding.EXPORTS)


def test_host_only_entry_points():
    lib = binding.lib()
    assert lib.lsa_strerror(0) == b"ok" and lib.lsa_strerror(-3).startswith(b"workspace")
    for name, cfg in CONFIGS.items():
        p = binding.make_params(cfg)
        n = binding.workspace_bytes(p, cfg.L or cfg.batch, cfg.L or cfg.ctx_hi, cfg.batch)
        assert n % 256 == 0 and n > 0
    p = binding.make_params(CONFIGS["cfg3"])
    assert ctypes.sizeof(p) == p.struct_size == 80
    # cfg3: page scores (131072 queries x 1024 pages x 4 B) + the e4m3 keys widened to bf16 (131072 x 128 x 2 B)
    assert binding.workspace_bytes(p, 131072, 131072) == 131072 * 1024 * 4 + 131072 * 128 * 2 + 256
    # q_chunk bounds the scratch
    p5 = binding.make_params(CONFIGS["cfg5"])
    assert binding.workspace_bytes(p5, 1 << 20, 1 << 20) == 16384 * 4096 * 4 + (1 << 20) * 128 * 2 + 256
    assert binding.host_stage_bytes(p, 4096) > 4096 * 64 * (576 + 512) * 2 * 4


def test_bad_parameters_return_codes():
    import pytest
    cfg = CONFIGS["cfg2"]
    # M * P: 8192 is served by the large-budget path; 2^19 tokens, an odd multiple of 64, or the 8-head indexer are not
    for bad in (cfg.replace(P=96), cfg.replace(B=3), cfg.replace(M=8192), cfg.replace(M=129), cfg.replace(Ksp=2050),
                cfg.replace(H=32), cfg.replace(d_I=96), CONFIGS["cfg1"].replace(M=128), CONFIGS["cfg4"].replace(M=128)):
        with pytest.raises(binding.LsaError) as e:
            binding.workspace_bytes(binding.make_params(bad), 16, 1024)
        assert e.value.code == -2
    assert binding.workspace_bytes(binding.make_params(cfg.replace(M=128)), 16, 1024) > 16 * 128 * 64 * 4
    p = binding.make_params(cfg)
    p.struct_size = 12
    with pytest.raises(binding.LsaError) as e:
        binding.workspace_bytes(p, 16, 1024)
    assert e.value.code == -1
