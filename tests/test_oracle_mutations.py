"""The pins must notice a mistake anywhere in the oracle: each case below plants one plausible mistake in
a copy of ``oracle/hccs_oracle.c`` (a dropped clamp, a wrong sign, shift or constant, a mask or an index
off by one, a transposed operand), builds the copy, lets the oracle's Python front end call it, and runs
the pins of ``test_oracle_pins.py`` and ``test_oracle_attention.py`` until one fails.  A mistake that every
pin accepts fails this test.  Everything here runs on the CPU; the real library is put back afterwards."""
import inspect
import os
import subprocess

import pytest

import test_oracle_attention as attention_pins
import test_oracle_pins as row_pins
from oracle import hccs_oracle as orc

SRC = os.path.join(os.path.dirname(os.path.abspath(orc.__file__)), "hccs_oracle.c")

# (name, text in the C file, its replacement)
MUTANTS = [
    ("distance clamp dropped", "        if (delta > D) delta = D;\n", ""),
    ("score sign", "        s = B - S * delta;", "        s = B + S * delta;"),
    ("distance sign", "        delta = m - (int64_t)x[i];", "        delta = (int64_t)x[i] - m;"),
    ("row maximum becomes minimum", "(int64_t)x[i] > m) m = (int64_t)x[i];", "(int64_t)x[i] < m) m = (int64_t)x[i];"),
    ("mask ignored by the maximum", "        if (valid && !valid[i]) continue;\n        if (n_valid == 0 ||",
     "        if (n_valid == 0 ||"),
    ("int8 path shifts by 14", "prod >> (ORACLE_INV_SHIFT + out_shift)", "prod >> (ORACLE_INV_SHIFT - 1 + out_shift)"),
    ("leading-bit position off by one", "        return Tprime >> k;", "        return Tprime >> (k + 1);"),
    ("leading-bit result not saturated", "q > ORACLE_T_U8)\n                q = ORACLE_T_U8;", "q > 100000)\n                q = ORACLE_T_U8;"),
    ("causal rule off by one", "!(j <= i + (Lk - Lq))", "!(j < i + (Lk - Lq))"),
    ("causal rule aligned at the top left", "!(j <= i + (Lk - Lq))", "!(j <= i)"),
    ("head of a row", "int64_t h = (r / Lq) % H;", "int64_t h = r % H;"),
    ("key length includes one key too many", "!(j < (int64_t)key_len[b])", "!(j <= (int64_t)key_len[b])"),
    ("requantisation truncates", "    if (sh > 0) t += (int64_t)1 << (sh - 1);\n", ""),
    ("output requantisation takes the wrong head", "Mo[bh % H], sh);", "Mo[0], sh);"),
]


def _pins():
    """Every pin with its parameter sets: (callable, kwargs)."""
    out = []
    for mod in (row_pins, attention_pins):
        for name, fn in sorted(vars(mod).items()):
            if not name.startswith("test_") or not callable(fn):
                continue
            marks = [m for m in getattr(fn, "pytestmark", []) if m.name == "parametrize"]
            if not marks:
                out.append((fn, {}))
                continue
            (mark,) = marks
            arg = mark.args[0]
            for value in mark.args[1]:
                out.append((fn, {arg: value}))
    return out


def _constant_of(name):
    text = open(SRC).read()
    return name in text


def test_the_unchanged_file_passes_every_pin(tmp_path):
    """The harness itself: a plain copy of the C file, built and loaded the same way, passes."""
    lib = tmp_path / "copy.so"
    subprocess.run(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", SRC, "-o", str(lib)], check=True)
    try:
        orc.use_library(str(lib))
        for fn, kwargs in _pins():
            fn(**kwargs)
    finally:
        orc.use_library(None)


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_a_planted_mistake_is_noticed(tmp_path, name, old, new):
    text = open(SRC).read()
    assert text.count(old) == 1, f"the text to replace for '{name}' must occur exactly once in the oracle"
    src = tmp_path / "mutant.c"
    src.write_text(text.replace(old, new))
    lib = tmp_path / "mutant.so"
    subprocess.run(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", str(src), "-o", str(lib)], check=True)
    noticed_by = None
    try:
        orc.use_library(str(lib))
        for fn, kwargs in _pins():
            try:
                fn(**kwargs)
            except (AssertionError, OverflowError, ValueError, IndexError):
                noticed_by = fn.__name__
                break
    finally:
        orc.use_library(None)
    assert noticed_by is not None, f"no pin noticed the mistake '{name}'"
