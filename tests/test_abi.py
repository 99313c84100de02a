"""The C-ABI library loads without a GPU, exports every declared symbol, and its host-side
logic (parameter admissibility) agrees with the oracle's statement of the constraints."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2604_02292_b200 import build
    build.build()
    from paper_2604_02292_b200 import binding as b
    return b


def _declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(hccs_[a-z0-9_]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported(binding):
    declared = _declared_symbols()
    assert {"hccs_params_upload", "hccs_forward", "hccs_attention_fused"} <= declared
    lib = ctypes.CDLL(binding.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
    assert set(binding.EXPORTS) == declared


def test_status_strings(binding):
    names = {binding.hccs_status_string(i) for i in range(7)}
    assert len(names) == 7 and all(n.startswith("HCCS_") for n in names)
    assert "unknown" in binding.hccs_status_string(99)


def test_params_check_matches_oracle_constraints(binding):
    from oracle import hccs_oracle as orc
    rng = np.random.default_rng(0)
    for n in (1, 2, 7, 64, 100, 128, 512, 1024, 4096, 32767):
        bmax = 32767 // n
        cases = []
        for _ in range(300):
            cases.append((int(rng.integers(-2, bmax + 4)), int(rng.integers(-2, 131)),
                          int(rng.integers(-1, 131))))
        f = -(-256 // n)
        for S, D in ((0, 1), (1, 1), (1, 127), (2, 50), (127, 1), (128, 1), (0, 128), (0, 0)):
            for dB in (-1, 0, 1):
                cases.append((S * D + f + dB, S, D))
                cases.append((bmax + dB, S, D))
        for (B, S, D) in cases:
            st, bad = binding.hccs_params_check([(B, S, D)], n)
            want_ok = orc.check_params(B, S, D, n) == 0
            assert (st == binding.HCCS_OK) == want_ok, (n, B, S, D, st)
            assert st in (binding.HCCS_OK, binding.HCCS_ERR_CONSTRAINT)
            assert bad == (-1 if want_ok else 0)
    # first offending head is reported
    st, bad = binding.hccs_params_check([(300, 3, 85), (300, 3, 85), (200, 3, 85)], 64)
    assert (st, bad) == (binding.HCCS_ERR_CONSTRAINT, 2)
    assert binding.hccs_params_check([(300, 3, 85)], 0)[0] == binding.HCCS_ERR_INVALID_ARG
    assert binding.hccs_params_check([(1, 0, 1)], 32768)[0] == binding.HCCS_ERR_INVALID_ARG


def test_null_arguments_are_rejected_without_a_gpu(binding):
    lib = binding.raw()
    assert lib.hccs_create(None, 0) == binding.HCCS_ERR_INVALID_ARG
    assert lib.hccs_destroy(None) == binding.HCCS_ERR_INVALID_ARG
    assert lib.hccs_forward(None, None, None, 1, 1, 1, 1, 0, None) == binding.HCCS_ERR_INVALID_ARG
    assert lib.hccs_params_upload(None, None, 1, 64, 0, None, None) == binding.HCCS_ERR_INVALID_ARG
    assert lib.hccs_last_cuda_error(None) == 0 and lib.hccs_launch_count(None) == 0
