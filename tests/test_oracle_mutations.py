"""The pins must be able to fail: each case plants one plausible mistake in a copy of the
oracle's C source (on the CPU, nothing else is touched), builds it, points the wrapper at
the mutated library and checks that at least one pin test then fails."""
import ctypes
import os
import subprocess

import pytest

import oracle
from oracle import fda_oracle as wrapper
import test_oracle_pins as pins

SRC = os.path.join(os.path.dirname(wrapper.__file__), "fda_oracle.c")

MUTATIONS = {
    "sign rule flipped": ("return (g & 1u) ? -1 : +1;", "return (g & 1u) ? +1 : -1;"),
    "Horner term dropped": ("    g = mul_add_mod_p(g, x, c[4]);\n", ""),
    "bucket uses b as multiplier": ("mul_add_mod_p(c[0], j % FDA_P, c[1])", "mul_add_mod_p(c[1], j % FDA_P, c[0])"),
    "no reduction mod p before mod m": ("return (uint64_t)(t % (u128)FDA_P);", "return (uint64_t)t;"),
    "sketch row index transposed": ("S[2 + (size_t)i * m + c] += (double)s * u;", "S[2 + (size_t)c * l + i] += (double)s * u;"),
    "drift sign": ("double u = (double)wk[j] - (double)w_t0[j];      /* drift, Table 1 */",
                   "double u = (double)wk[j] + (double)w_t0[j];      /* drift, Table 1 */"),
    "norm not squared": ("sq += u * u;                                     /* ||u||^2        */",
                         "sq += u;                                     /* ||u||^2        */"),
    "projection ignores xi": ("if (xi) pr += (double)xi[j] * u;", "if (xi) pr += u;"),
    "state sum not averaged": ("Sbar[e] = acc / (double)K;", "Sbar[e] = acc;"),
    "mean instead of median": ("double med = (l & 1) ? sorted[l / 2] : 0.5 * (sorted[l / 2 - 1] + sorted[l / 2]);",
                               "double med = 0.0; for (int i = 0; i < l; ++i) med += sorted[i] / l;"),
    "epsilon factor inverted": ("est = med / (1.0 + epsilon);", "est = med * (1.0 + epsilon);"),
    "linear estimate not squared": ("est = Sbar[1] * Sbar[1];", "est = Sbar[1];"),
    "trigger not strict": ("out[3] = (out[2] > theta) ? 1.0 : 0.0;", "out[3] = (out[2] >= theta) ? 1.0 : 0.0;"),
    "average divides by K-1": ("avg[j - j_begin] = acc / (double)K;", "avg[j - j_begin] = acc / (double)(K > 1 ? K - 1 : 1);"),
    "direction not normalised": ("xi[j] = norm > 0.0 ? (w_new[j] - (double)w_old[j]) / norm : 0.0;",
                                 "xi[j] = (w_new[j] - (double)w_old[j]);"),
}

PIN_TESTS = [getattr(pins, n) for n in dir(pins) if n.startswith("test_") and n != "test_workload_expectations"]


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_pins_catch_a_planted_mistake(name, tmp_path, monkeypatch):
    old, new = MUTATIONS[name]
    src = open(SRC).read()
    assert src.count(old) == 1, "mutation target must be unique in the oracle source"
    mutated = tmp_path / "mutant.c"
    mutated.write_text(src.replace(old, new))
    lib_path = tmp_path / "libmutant.so"
    subprocess.check_call(["gcc", "-O1", "-std=gnu11", "-shared", "-fPIC", "-w", "-o", str(lib_path), str(mutated), "-lm"])
    good = wrapper._load()
    bad = ctypes.CDLL(str(lib_path))
    for fn in ("fda_oracle_hash", "fda_oracle_local_state", "fda_oracle_combine", "fda_oracle_average",
               "fda_oracle_variance", "fda_oracle_direction"):
        getattr(bad, fn).argtypes = getattr(good, fn).argtypes
        getattr(bad, fn).restype = getattr(good, fn).restype
    monkeypatch.setattr(wrapper, "_lib", bad)
    caught = 0
    for t in PIN_TESTS:
        try:
            t()
        except (AssertionError, ValueError):
            caught += 1
        except Exception:
            caught += 1
    assert caught >= 1, "no pin noticed: " + name
    monkeypatch.setattr(wrapper, "_lib", good)
    assert oracle.state_len(5, 250) == 1252
