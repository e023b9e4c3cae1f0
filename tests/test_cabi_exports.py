"""The C-ABI library loads and exports every function the public header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = []
    inc = os.path.join(ROOT, "include")
    for f in sorted(os.listdir(inc)):
        if f.endswith(".h"):
            text = open(os.path.join(inc, f)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b(tts_gpt_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


@pytest.fixture(scope="module")
def lib():
    from paper_2607_21042_b200 import build, binding
    build.build()
    return binding.load()


def test_header_declares_the_five_calls():
    d = _declared()
    for n in ("tts_gpt_create", "tts_gpt_prefill", "tts_gpt_decode_step", "tts_gpt_release_stream",
              "tts_gpt_destroy"):
        assert n in d


def test_every_declared_symbol_is_exported(lib):
    for n in _declared():
        assert hasattr(lib, n), n


def test_binding_lists_every_declared_symbol():
    from paper_2607_21042_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()


def test_query_workspace_and_config_errors_need_no_gpu(lib):
    from paper_2607_21042_b200 import binding, cases
    cfg = cases.workload(2).cfg
    n = binding.query_workspace(cfg)
    # bf16 weights twice (965 MB in the streaming layout for small batches + 985 MB as tensor-core
    # operand images for more than 16 rows) + 32 pages * 7.86 MB of KV + activations
    assert 2.1e9 < n < 2.4e9
    bad = cases.GPTConfig(**{**cfg.as_dict(), "head_dim": 32})
    with pytest.raises(binding.TtsGptError) as e:
        binding.query_workspace(bad)
    assert e.value.code == binding.E_UNSUPPORTED
    bad = cases.GPTConfig(**{**cfg.as_dict(), "max_streams": 129})
    with pytest.raises(binding.TtsGptError) as e:
        binding.query_workspace(bad)
    assert e.value.code == binding.E_ARG
    # quantized formats need less: 264 MB packed + 985 MB of bf16 integer images for the tensor cores
    n4 = binding.query_workspace(cases.workload(4).cfg)
    assert n4 < 16 * 32 * 7.9e6 + 1.4e9


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    from paper_2607_21042_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(OSError):
        binding.load()
