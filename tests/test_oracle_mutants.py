"""Do the pins bite?  Each case plants one plausible mistake in a COPY of the oracle's source
(on the CPU, in a temporary directory), builds it and runs the pin tests against the mutant: at
least one pin must fail.  The real oracle is never modified."""
from __future__ import annotations

import ctypes
import inspect
import itertools
import os
import subprocess

import pytest

import oracle
from tests import test_oracle_pins as pins

SRC = os.path.join(os.path.dirname(oracle.__file__), "outer_sync_oracle.c")

# (name, text in the oracle, replacement)
MUTANTS = [
    ("sign of the outer gradient", "(input_kind == 1 ? x : t0 - x)", "(input_kind == 1 ? x : x - t0)"),
    ("nesterov look-ahead term dropped", "t1 = t0 - outer_lr * (delta + outer_momentum * m1);",
     "t1 = t0 - outer_lr * m1;"),
    ("momentum not decayed", "m1 = outer_momentum * (double)mo[k] + delta;\n                        t1 = t0 - outer_lr * (delta",
     "m1 = (double)mo[k] + delta;\n                        t1 = t0 - outer_lr * (delta"),
    ("mean divides by all paths of the module instead of the reporting ones", "alpha[r] = w / total_weight;",
     "alpha[r] = w / (path_weights ? total_weight : (double)n_members);"),
    ("uniform weights used instead of shard sizes", "double w = path_weights ? (double)path_weights[reporters[r]] : 1.0;",
     "double w = 1.0; (void)path_weights;"),
    ("masked paths still contribute", "if (reported && !reported[i])\n                    continue;",
     "if (0 && reported && !reported[i])\n                    continue;"),
    ("write-back skips paths that did not report", "for (int32_t s = 0; s < n_members; ++s)\n                    write_copy(path_ptrs[members[s]]",
     "for (int32_t s = 0; s < n_members; ++s)\n                    if (!reported || reported[members[s]]) write_copy(path_ptrs[members[s]]"),
    ("empty module still decays its momentum", "const int update = (n_reporters > 0 && total_weight > 0.0);",
     "const int update = 1; if (!(n_reporters > 0 && total_weight > 0.0)) { n_reporters = 0; }"),
    ("level offset inside a path copy not advanced", "        level_base += n;\n    }\n    free(members)",
     "        level_base += 0;\n    }\n    free(members)"),
    ("module offset inside theta not advanced", "            module_base += n;\n        }\n        level_base",
     "            module_base += 0;\n        }\n        level_base"),
    ("bf16 cast truncates", "if (lower > 0x8000u || (lower == 0x8000u && (upper & 1u)))", "if (0)"),
    ("bf16 cast rounds a NaN like a number", "if ((bits & 0x7fffffffu) > 0x7f800000u)", "if (0)"),
    ("bf16 ties round away from zero", "(lower == 0x8000u && (upper & 1u))", "(lower == 0x8000u)"),
    ("learning rate applied twice to momentum", "t1 = t0 - outer_lr * (delta + outer_momentum * m1);",
     "t1 = t0 - outer_lr * (delta + outer_lr * outer_momentum * m1);"),
    ("module scale ignored", "delta *= scale;", "delta *= 1.0; (void)scale;"),
    ("level flag ignored", "if (level_sync && !level_sync[l]) {", "if (0 && level_sync && !level_sync[l]) {"),
    ("heavy ball uses the nesterov step", "t1 = t0 - outer_lr * m1;\n                    } else if (optimizer == 2)",
     "t1 = t0 - outer_lr * (delta + outer_momentum * m1);\n                    } else if (optimizer == 2)"),
    ("sgd touches the momentum buffer", "m1 = (double)mo[k];\n                        t1 = t0 - outer_lr * delta;",
     "m1 = delta;\n                        t1 = t0 - outer_lr * delta;"),
    ("adam without bias correction", "(m1 / c1) / (sqrt(v1 / c2) + eps)", "(m1) / (sqrt(v1) + eps)"),
    ("adam eps inside the square root", "(sqrt(v1 / c2) + eps)", "sqrt(v1 / c2 + eps)"),
    ("adam weight decay not decoupled", "t1 = t0 * (1.0 - outer_lr * wd) - outer_lr * (m1 / c1)",
     "t1 = t0 - outer_lr * (m1 / c1 + wd * t0)"),
    ("path table read transposed", "if (path_to_module[(int64_t)i * num_levels + l] != e)",
     "if (path_to_module[((int64_t)l * num_paths + i) % ((int64_t)num_paths * num_levels)] != e)"),
    ("every contributor gets the first coefficient", "delta += alpha[r] *", "delta += alpha[0] *"),
    ("theta rounded to bf16 before it is stored", "th[k] = new_theta;",
     "th[k] = new_theta; if (path_dtype == ORACLE_BF16) { uint32_t b = ((uint32_t)narrow_bf16(new_theta)) << 16; memcpy(&th[k], &b, 4); }"),
    ("gradient inputs treated as copies", "(input_kind == 1 ? x : t0 - x)", "(t0 - x)"),
]


def pin_calls():
    """Every pin test with every parameter combination, as zero-argument callables."""
    calls = []
    for name, fn in inspect.getmembers(pins, inspect.isfunction):
        if not name.startswith("test_") or name == "test_path_table_matches_the_papers_toy_figure":
            continue
        marks = [m for m in getattr(fn, "pytestmark", []) if m.name == "parametrize"]
        if not marks:
            calls.append((name, fn, {}))
            continue
        names, values = [], []
        for m in marks:
            keys = [k.strip() for k in m.args[0].split(",")]
            names.append(keys)
            values.append([v if isinstance(v, (tuple, list)) and len(keys) > 1 else (v,) for v in m.args[1]])
        for combo in itertools.product(*values):
            kw = {}
            for keys, vals in zip(names, combo):
                kw.update(dict(zip(keys, vals)))
            calls.append((name, fn, kw))
    return calls


def build_mutant(tmp_path, old, new):
    text = open(SRC).read()
    assert text.count(old) == 1, "mutation site must be unique in the oracle: %r" % old
    src = tmp_path / "mutant.c"
    src.write_text(text.replace(old, new))
    lib = str(tmp_path / "libmutant.so")
    subprocess.check_call(["gcc", "-O1", "-std=c99", "-fopenmp", "-shared", "-fPIC", "-o", lib, str(src), "-lm"])
    return lib


@pytest.fixture
def restore_oracle():
    oracle._load()
    real = oracle._lib
    yield
    oracle._lib = real


def test_the_unmodified_source_passes_every_pin_through_this_harness(tmp_path, restore_oracle):
    lib = build_mutant(tmp_path, "delta *= scale;", "delta *= scale; /* unchanged */")
    swap_in(lib)
    for name, fn, kw in pin_calls():
        call(fn, kw, tmp_path)


def swap_in(lib_path):
    real = oracle._lib
    lib = ctypes.CDLL(lib_path)
    for fname in ("oracle_outer_sync", "oracle_outer_sync_ex", "oracle_max_threads"):
        getattr(lib, fname).restype = getattr(real, fname).restype
        getattr(lib, fname).argtypes = getattr(real, fname).argtypes
    oracle._lib = lib


def call(fn, kw, tmp_path):
    if "tmp_path" in inspect.signature(fn).parameters:
        kw = dict(kw, tmp_path=tmp_path)
    fn(**kw)


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_a_planted_mistake_is_caught_by_some_pin(name, old, new, tmp_path, restore_oracle):
    swap_in(build_mutant(tmp_path, old, new))
    caught = []
    for tname, fn, kw in pin_calls():
        try:
            call(fn, kw, tmp_path)
        except AssertionError:
            caught.append(tname)
        except ValueError:
            caught.append(tname)
    assert caught, "no pin noticed: " + name
