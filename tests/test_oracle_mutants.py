"""Planted mistakes: each mutant is a copy of the oracle's C source with one plausible error
(a swapped operand, a wrong tie-break, a wrong eviction order, ...).  The pins of
test_oracle_pins.py / test_oracle_policies.py / test_oracle_neuron_pruning.py must fail on every one of them -- that is what
makes them pins.  The mistakes are planted in the CPU oracle only."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "dip_oracle.c")

MUTANTS = {
    "silu_on_up_branch": ("h32[j] = (float)(u[j] * orc_silu(g[j]));", "h32[j] = (float)(g[j] * orc_silu(u[j]));"),
    "dense_silu_on_up_branch": ("glu[j] = u * orc_silu(g);", "glu[j] = g * orc_silu(u);"),
    "tie_to_higher_index": ("return a->idx < b->idx ? -1 : (a->idx > b->idx ? 1 : 0);\n}\n\nint orc_topk_mask",
                            "return a->idx > b->idx ? -1 : (a->idx < b->idx ? 1 : 0);\n}\n\nint orc_topk_mask"),
    "keeps_smallest": ("return a->key > b->key ? -1 : 1;", "return a->key < b->key ? -1 : 1;"),
    "penalty_on_resident": ("float w = resident ? 1.0f : gamma;", "float w = resident ? gamma : 1.0f;"),
    "evicts_most_recent": ("return a->stamp < b->stamp ? -1 : 1;", "return a->stamp > b->stamp ? -1 : 1;"),
    "transposed_weight_index": ("size_t e = (size_t)j * (size_t)d_in + (size_t)i;", "size_t e = (size_t)i * (size_t)d_out + (size_t)j;"),
    "mask_ignored_in_matvec": ("            if (m[i])\n                acc += orc_weight(type, w, scales, d_out, d_in, j, i) * (double)v[i];",
                               "            acc += orc_weight(type, w, scales, d_out, d_in, j, i) * (double)v[i];"),
    "int4_zero_point_off_by_one": ("return (double)(q - 8) * s;", "return (double)(q - 7) * s;"),
    "hits_against_new_state": ("    int misses = k - hits;\n    int free_slots = capacity - *n_resident;\n    int n_evict = misses - free_slots;\n    if (n_evict < 0)\n        n_evict = 0;\n    int evictable = *n_resident - hits;\n    if (n_evict > evictable)\n        n_evict = evictable;\n\n    /* least recently used first",
                               "    int misses = k - hits;\n    int free_slots = capacity - *n_resident;\n    int n_evict = misses;\n    if (n_evict < 0)\n        n_evict = 0;\n    int evictable = *n_resident - hits;\n    if (n_evict > evictable)\n        n_evict = evictable;\n\n    /* least recently used first"),
    "lfu_evicts_most_used": ("            v[nv].stamp = count[i];", "            v[nv].stamp = -count[i];"),
    "belady_evicts_soonest": ("                if (next > far) {", "                if (far < 0 || next < far) {"),
    "gate_pruning_ranks_raw_gate": ("p32[j] = (float)(by == 0 ? orc_silu(acc) : acc);", "p32[j] = (float)acc;"),
    "gate_and_up_pruning_swapped": ("const void *Wp = by == 0 ? Wg : Wu;", "const void *Wp = by == 0 ? Wu : Wg;"),
    "pruned_neurons_reach_down": ("    orc_masked_matvec(type, Wd, Sd, d_model, d_ff, h32, m, y);\n    return 0;\n}\n\n/* ------------------------------------------------------------------ *\n * Layer chaining",
                                  "    memset(m, 1, (size_t)d_ff);\n    orc_masked_matvec(type, Wd, Sd, d_model, d_ff, h32, m, y);\n    return 0;\n}\n\n/* ------------------------------------------------------------------ *\n * Layer chaining"),
}


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_pins_kill_mutant(name, tmp_path):
    old, new = MUTANTS[name]
    text = open(SRC).read()
    assert text.count(old) == 1, "mutation site not found exactly once: " + name
    src = tmp_path / "mutant.c"
    lib = tmp_path / "libmutant.so"
    src.write_text(text.replace(old, new))
    subprocess.run(["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC", "-std=c11", str(src), "-o",
                    str(lib), "-lm"], check=True)
    env = dict(os.environ, DIP_ORACLE_LIB=str(lib))
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                        os.path.join(ROOT, "tests", "test_oracle_pins.py"),
                        os.path.join(ROOT, "tests", "test_oracle_policies.py"),
                        os.path.join(ROOT, "tests", "test_oracle_neuron_pruning.py")],
                       cwd=ROOT, env=env, capture_output=True, text=True)
    assert r.returncode != 0, "the pins passed on a broken oracle (%s)" % name
    assert "failed" in r.stdout
