"""The C ABI library loads and exports every symbol the header declares (no GPU needed)."""
import os
import re

import pytest

from paper_2609_12378_b200 import binding, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "ckks_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ckks_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported():
    lib = binding.load()
    names = _declared()
    assert len(names) >= 19
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == sorted(n for n in names)


def test_status_strings():
    lib = binding.load()
    seen = {lib.ckks_status_string(c).decode() for c in range(0, -10, -1)}
    assert len(seen) == 10 and "ok" in seen


def test_parameter_validation_happens_before_any_cuda_call():
    q, p = inputs.prime_chain(10, 4, 2)
    bad = [
        dict(log_n=9, q=q, p=p, dnum=2),                         # ring too small
        dict(log_n=17, q=q, p=p, dnum=2),                        # ring too large
        dict(log_n=10, q=[int(q[0]), int(q[0])], p=p, dnum=1),   # duplicate prime
        dict(log_n=10, q=q, p=p[:1], dnum=2),                    # K < alpha
        dict(log_n=10, q=[(1 << 50) - 27], p=p, dnum=1),         # not 1 mod 2N / not in the chain
        dict(log_n=11, q=q, p=p, dnum=2) if int(q[0]) % 4096 != 1 else dict(log_n=9, q=q, p=p, dnum=2),
        dict(log_n=10, q=q, p=p, dnum=0),
    ]
    for kw in bad:
        with pytest.raises(binding.CkksError) as e:
            binding.Context(**kw)
        assert e.value.code == binding.ERR_UNSUPPORTED, kw


def test_missing_library_is_a_loud_error(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libckks_b200.so")
    with pytest.raises(RuntimeError):
        binding.load()
