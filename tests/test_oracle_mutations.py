"""The pins are only worth something if a plausible mistake in the oracle fails them.  Each case plants one
mistake in a COPY of the oracle (never in the tree), runs the pin files against that copy in a child process
and expects them to fail.  CPU only; the mistakes are planted in the oracle, nothing here touches a GPU."""
import os
import shutil
import subprocess
import sys

import pytest

from tests.conftest import ROOT

CPP = os.path.join("oracle", "pe_oracle.cpp")
COARSEN = os.path.join("oracle", "pe_coarsen_oracle.py")
PY = os.path.join("oracle", "pe_oracle.py")

# (name, file, text to find, replacement, pin files that must catch it)
MUTATIONS = [
    ("link class looked up the wrong way round", CPP, "link_class[(size_t)x[p] * D + j]", "link_class[(size_t)j * D + x[p]]",
     ["test_oracle_pins.py"]),
    ("communication delay dropped", CPP, "            t += comm ? comm[(size_t)b * L + cls] : 0;", "            t += 0;",
     ["test_oracle_pins.py"]),
    ("delay charged inside one machine too", CPP, "        if (x[p] != j) {", "        if (true) {", ["test_oracle_pins.py"]),
    ("machine chain dropped (Eqs. 7-8)", CPP, "s[i] = r > free_at[j] ? r : free_at[j];", "s[i] = r;", ["test_oracle_pins.py"]),
    ("memory adjustment with the wrong sign", CPP, "lvl[j] += mem_delta[i];", "lvl[j] -= mem_delta[i];", ["test_oracle_pins.py"]),
    ("peak forgets the level before the first operation", CPP, "for (int32_t j = 0; j < D; ++j) peak[j] = lvl[j];",
     "for (int32_t j = 0; j < D; ++j) peak[j] = -(1 << 30);", ["test_oracle_pins.py"]),
    ("weights not resident from the start (Eq. 16)", CPP, "for (int32_t i = 0; i < V; ++i) lvl[x[i]] += mem_weight[i];", ";",
     ["test_oracle_pins.py"]),
    ("makespan taken over starts", CPP, "if (e[i] > z) z = e[i];", "if (s[i] > z) z = s[i];", ["test_oracle_pins.py"]),
    ("busy time counts every machine", CPP, "busy_j[j] += d_i;", "for (int32_t jj = 0; jj < D; ++jj) busy_j[jj] += d_i;",
     ["test_oracle_pins.py"]),
    ("heterogeneous table indexed the wrong way round", CPP, "dur_by_machine[(size_t)i * D + j]", "dur_by_machine[(size_t)j * V + i]",
     ["test_hetero_pins.py"]),
    ("heterogeneous table ignored", CPP, "dur_by_machine ? dur_by_machine[(size_t)i * D + j] : dur[i]", "dur[i]", ["test_hetero_pins.py"]),
    ("decode: largest rank first", CPP, "std::greater<int64_t>> ready;", "std::less<int64_t>> ready;", ["test_decode_pins.py"]),
    ("decode: rank of list entry off by one", CPP, "rank[i] = r;", "rank[i] = (r + 1) % V;", ["test_decode_pins.py"]),
    ("decode: duplicates not flagged", CPP, "if (i >= (uint32_t)V || rank[i] >= 0) { ok = false; continue; }",
     "if (i >= (uint32_t)V) { ok = false; continue; }", ["test_decode_pins.py"]),
    ("exclusive: channel never occupied", CPP, "            chan = t;\n", "", ["test_contention_pins.py"]),
    ("exclusive: transfer ignores when the source ends", CPP, "const int32_t c_start = t > chan ? t : chan;",
     "const int32_t c_start = chan;", ["test_contention_pins.py"]),
    ("exclusive: one channel per receiving machine", CPP, "int32_t& chan = chan_free[(size_t)x[p] * D + j];",
     "int32_t& chan = chan_free[(size_t)j];", ["test_contention_pins.py"]),
    ("coarsening: redundant edges not set aside", COARSEN, "        red = _two_hop_redundant(succ)\n        best = None",
     "        red = set()\n        best = None", ["test_coarsen.py"]),
    ("coarsening: head may have several inputs", COARSEN, "            if len(ins) != 1:", "            if len(ins) < 1:", ["test_coarsen.py"]),
    ("coarsening: unrelated means no direct edge only", COARSEN, "if v in reach[u] or u in reach[v]:", "if v in succ[u] or u in succ[v]:",
     ["test_coarsen.py"]),
    ("coarsening: largest pair first", COARSEN, "                key = (dur[u] + dur[v], u, v)\n                if best is None or key < best:\n                    best = key\n        return None if best is None else (best[1], best[2])\n\n    def merge",
     "                key = (-dur[u] - dur[v], u, v)\n                if best is None or key < best:\n                    best = key\n        return None if best is None else (best[1], best[2])\n\n    def merge",
     ["test_coarsen.py"]),
    ("coarsening: merged communication is the smaller one", COARSEN, "succ[keep][x] = [max(a, b_) for a, b_ in zip(succ[keep][x], c)]",
     "succ[keep][x] = [min(a, b_) for a, b_ in zip(succ[keep][x], c)]", ["test_coarsen.py"]),
    ("top-k: ties to the largest index", PY, "if best_c < 0 or int(makespan[c]) < int(makespan[best_c]):",
     "if best_c < 0 or int(makespan[c]) <= int(makespan[best_c]):", ["test_oracle_pins.py"]),
]


@pytest.fixture(scope="module")
def tree(tmp_path_factory):
    """A copy of what the pin files import: oracle/, tests/ and the input generators (no CUDA library needed
    by the files used here, except test_coarsen.py's library half, which is deselected)."""
    work = str(tmp_path_factory.mktemp("mutants"))
    for d in ("oracle", "tests", "paper_2503_09357_b200"):
        shutil.copytree(os.path.join(ROOT, d), os.path.join(work, d),
                        ignore=shutil.ignore_patterns("_build", "__pycache__", "libpe_oracle.so", "csrc", ".pytest_cache"))
    return work


def run_pins(work, files):
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider", "-k",
           "not test_library_matches and not test_library_on_the and not test_library_argument"]   # (pe_coarsen itself)
    cmd += [os.path.join("tests", f) for f in files]
    return subprocess.run(cmd, cwd=work, capture_output=True, text=True).returncode


def test_the_unmodified_copy_passes(tree):
    assert run_pins(tree, ["test_oracle_pins.py", "test_hetero_pins.py", "test_decode_pins.py", "test_contention_pins.py",
                           "test_coarsen.py"]) == 0


@pytest.mark.parametrize("name,rel,find,repl,files", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_a_planted_mistake_fails_the_pins(tree, name, rel, find, repl, files):
    path = os.path.join(tree, rel)
    original = open(os.path.join(ROOT, rel)).read()
    assert find in original, f"the text to mutate is gone from {rel}: {find!r}"
    try:
        open(path, "w").write(original.replace(find, repl, 1))
        assert run_pins(tree, files) != 0, f"the pins did not notice: {name}"
    finally:
        open(path, "w").write(original)
        so = os.path.join(tree, "oracle", "libpe_oracle.so")
        if os.path.exists(so):
            os.remove(so)                     # rebuilt from the restored source by the next case
