"""Plant one plausible mistake at a time in a copy of the oracle's C source and check that
the pins notice.  A pin set that lets a mutant through is too weak to trust."""
import os
import subprocess
import sys

import pytest

import oracle
import test_oracle_pins as pins

SRC = os.path.join(os.path.dirname(oracle.__file__), "slimspec_oracle.c")

# (name, text in the source, replacement)
MUTANTS = [
    ("down_wrong_stride_A", "const uint16_t *Ai = A + (size_t)i * r;", "const uint16_t *Ai = A + (size_t)i * d;"),
    ("down_transposed_A", "zm[j] += hv * bf16_to_double(Ai[j]);", "zm[j] += hv * bf16_to_double(A[(size_t)j * d + i]);"),
    ("down_dropped_last_term", "for (int i = 0; i < d; ++i) {\n            double hv = bf16_to_double(h[(size_t)m * d + i]);\n            const uint16_t *Ai",
     "for (int i = 0; i < d - 1; ++i) {\n            double hv = bf16_to_double(h[(size_t)m * d + i]);\n            const uint16_t *Ai"),
    ("up_sign", "lm[v] += zj * bf16_to_double(Bj[v]);", "lm[v] -= zj * bf16_to_double(Bj[v]);"),
    ("up_wrong_row_of_z", "double zj = z[(size_t)m * r + j];", "double zj = z[j];"),
    ("up_transposed_B", "lm[v] += zj * bf16_to_double(Bj[v]);", "lm[v] += zj * bf16_to_double(B[(size_t)v * r + j]);"),
    ("full_wrong_stride_W", "const uint16_t *Wi = W + (size_t)i * V;", "const uint16_t *Wi = W + (size_t)i * d;"),
    ("softmax_no_max_shift", "double l = mx + log(s);", "double l = log(s);"),
    ("softmax_log_dropped", "double l = mx + log(s);", "double l = mx + s;"),
    ("softmax_first_term_lost", "for (int v = 0; v < V; ++v) s += exp(lm[v] - mx);", "for (int v = 1; v < V; ++v) s += exp(lm[v] - mx);"),
    ("topk_ascending", "if (x->val > y->val) return -1;          /* larger value first */\n    if (x->val < y->val) return 1;",
     "if (x->val > y->val) return 1;\n    if (x->val < y->val) return -1;"),
    ("topk_ties_to_higher_id", "return (x->id > y->id) - (x->id < y->id);", "return (x->id < y->id) - (x->id > y->id);"),
    ("topk_next_off_by_one", "next_val[m] = (k < V) ? p[k].val", "next_val[m] = (k < V) ? p[k - 1].val"),
    ("bf16_low_half", "uint32_t w = ((uint32_t)bits) << 16;", "uint32_t w = ((uint32_t)bits) << 15;"),
]

PIN_FUNCS = [getattr(pins, n) for n in dir(pins) if n.startswith("test_")]


def run_pins():
    """Names of the pins that fail against the currently bound oracle build."""
    failed = []
    for f in PIN_FUNCS:
        marks = [m for m in getattr(f, "pytestmark", []) if m.name == "parametrize"]
        cases = [dict(zip(marks[0].args[0].split(","), c)) for c in marks[0].args[1]] if marks else [{}]
        for kw in cases:
            try:
                f(**kw)
            except (AssertionError, ValueError, MemoryError):
                failed.append(f.__name__)
                break
    return failed


def test_unmutated_source_passes_every_pin():
    assert run_pins() == []


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_pins_catch_planted_mistake(tmp_path, name, old, new):
    src = open(SRC).read()
    assert src.count(old) == 1, "mutation site must be unique: %s" % name
    c = tmp_path / "mutant.c"
    c.write_text(src.replace(old, new))
    so = tmp_path / ("mutant_%s.so" % name)
    subprocess.check_call(["gcc", "-O1", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", str(so), str(c), "-lm"])
    # A mutant may read out of bounds and crash, so it runs in a child process; a crash
    # counts as noticed, a clean run that reports no failed pin does not.
    code = ("import sys; sys.path[:0] = [%r, %r]; import oracle, test_oracle_mutants as t; "
            "oracle._lib = oracle._bind(%r); f = t.run_pins(); print('FAILED', f); "
            "sys.exit(0 if not f else 3)") % (os.path.dirname(os.path.dirname(SRC)), os.path.dirname(__file__), str(so))
    rc = subprocess.run([sys.executable, "-c", code], capture_output=True, timeout=300).returncode
    assert rc != 0, "no pin noticed mutant %s" % name
