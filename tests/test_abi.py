"""The C-ABI library loads and exports every symbol the public header declares (no GPU needed)."""
import re
from pathlib import Path

import numpy as np
import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    from paper_2604_12247_b200 import build, binding
    build.build()
    return binding.lib()


def declared_functions():
    text = (ROOT / "include" / "specbound.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sb_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2604_12247_b200 import binding
    names = declared_functions()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), f"{n} declared in specbound.h but not exported"
    assert set(names) == set(binding.EXPORTS)


def test_host_only_helpers(lib):
    from paper_2604_12247_b200 import binding, inputs
    T = binding.tau_schedule(0.2, 32)
    assert T[-1] == pytest.approx(1.0) and T[0] == pytest.approx(1.2 - 0.00625, rel=1e-6)   # Eq. 1
    assert binding.model_speedup(32, 0.9, 8, 10) == pytest.approx(1.608, abs=5e-4)            # Eq. 5
    assert lib.sb_strerror(-3).decode() == "capacity exceeded"
    cfg = binding.make_config(inputs.LLAMA2_7B, 1040)
    ws = lib.sb_workspace_bytes(cfg)
    kv = 2 * 32 * (17 * 64) * 4096 * 2          # K and V, 32 layers, 17 pages of 64, bf16
    # scratch beside the cache: decode buffers, the 128-row prefill pass (split-K partials of 16 blocks), sampling rows
    assert kv < ws < kv + (192 << 20)
    bad = binding.make_config(inputs.LLAMA2_7B, 1040, kv_page=48)
    assert lib.sb_workspace_bytes(bad) == 0      # page size must be a power of two
    assert lib.sb_create(bad, None, 0, None, None) == -1


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2604_12247_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", tmp_path / "nope.so")
    with pytest.raises(ImportError):
        binding.lib()


def test_sampling_uniforms_equal_the_oracles_generator(lib):
    """Host function of the library (no GPU): both sides implement the same counter-based generator."""
    from oracle import oracle
    from paper_2604_12247_b200 import binding
    for seed in (0, 1, 2 ** 63 + 12345, 2 ** 64 - 1):
        for pos in (0, 1, 511, 1023, 10 ** 9):
            assert binding.sample_uniform(seed, pos) == oracle.uniform(seed, pos)
