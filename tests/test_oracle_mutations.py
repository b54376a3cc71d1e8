"""The pins must bite: each planted mistake in the CPU checker has to fail at
least one of them.

Every case copies oracle/placeto_oracle.c, plants one plausible mistake (a
dropped term, a swapped direction, a wrong index ...), compiles the copy and
runs the pin tests of tests/test_oracle_pins.py against it. The mistakes live
in the checker, on the CPU, only.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import pytest

from oracle import oracle
from tests import test_oracle_pins as pins

SRC = os.path.join(os.path.dirname(oracle.__file__), "placeto_oracle.c")

# (name, text in the checker, replacement)
MUTATIONS = [
    ("directions swapped",
     "const int *ptr = down ? g->par_ptr : g->chi_ptr, *nbr = down ? g->par : g->chi;",
     "const int *ptr = down ? g->chi_ptr : g->par_ptr, *nbr = down ? g->chi : g->par;"),
    ("bias dropped", "real s = (real)b[j];", "real s = 0;"),
    ("hidden layer not activated",
     "for (int j = 0; j < M->hidden_dim; ++j) t[j] = activate(t[j], M->act);", ""),
    ("features before embedding in the message input",
     "memcpy(in, H + ((size_t)u * B + b) * d, sizeof(real) * (size_t)d);\n"
     "            memcpy(in + d, X + ((size_t)u * B + b) * F, sizeof(real) * (size_t)F);",
     "memcpy(in + F, H + ((size_t)u * B + b) * d, sizeof(real) * (size_t)d);\n"
     "            memcpy(in, X + ((size_t)u * B + b) * F, sizeof(real) * (size_t)F);"),
    ("raw features not re-injected",
     "memcpy(in + d, X + ((size_t)u * B + b) * F, sizeof(real) * (size_t)F);\n            mlp(f, in, msg);",
     "memset(in + d, 0, sizeof(real) * (size_t)F);\n            mlp(f, in, msg);"),
    ("ancestor and descendant sets swapped",
     "int i = anc[u] ? 0 : (desc[u] ? 1 : 2);\n            mlp(&l[i], e, y);",
     "int i = anc[u] ? 1 : (desc[u] ? 0 : 2);\n            mlp(&l[i], e, y);"),
    ("current node pooled as parallel",
     "if (u == c) { memcpy(z, e, sizeof(real) * (size_t)E); continue; }",
     "if (u == c) { memcpy(z, e, sizeof(real) * (size_t)E); }"),
    ("repeated edges counted twice", "if (i == a || tmp[i] != tmp[i - 1]) out[w++] = tmp[i];",
     "out[w++] = tmp[i];"),
    ("is-current and is-placed swapped",
     "x[2 + m] = (cur[b] == v) ? 1 : 0;\n            x[3 + m] = placed[(size_t)b * n + v] ? 1 : 0;",
     "x[3 + m] = (cur[b] == v) ? 1 : 0;\n            x[2 + m] = placed[(size_t)b * n + v] ? 1 : 0;"),
    ("weights read transposed", "(real)W[(size_t)k * out + j] * v[k]",
     "(real)W[(size_t)(in == out ? j * in + k : k * out + j)] * v[k]"),
    ("reachability not transitive", "if (!mark[w]) { mark[w] = 1; stack[top++] = w; }",
     "if (!mark[w]) { mark[w] = 1; }"),
    ("embedding halves swapped in the node embedding",
     "memcpy(e, H_down + ((size_t)u * B + b) * d, sizeof(real) * (size_t)d);\n"
     "            memcpy(e + d, H_up + ((size_t)u * B + b) * d, sizeof(real) * (size_t)d);",
     "memcpy(e + d, H_down + ((size_t)u * B + b) * d, sizeof(real) * (size_t)d);\n"
     "            memcpy(e, H_up + ((size_t)u * B + b) * d, sizeof(real) * (size_t)d);"),
    ("softmax not normalised", "probs[(size_t)b * m + k] /= tot;", "(void)tot;"),
    ("one-hot off by one", "(dev[(size_t)b * n + v] == k) ? 1 : 0", "(dev[(size_t)b * n + v] == k + 1) ? 1 : 0"),
    ("synchronous rounds update in place",
     "memcpy(in, prev + ((size_t)u * B + b) * d, sizeof(real) * (size_t)d);",
     "memcpy(in, H + ((size_t)u * B + b) * d, sizeof(real) * (size_t)d);"),
    ("synchronous rounds start from the bias-only state instead of zeros",
     "for (size_t i = 0; i < tot; ++i) H[i] = 0;\n        for (int r = 0; r < rounds; ++r) {",
     "for (size_t i = 0; i < tot; ++i) H[i] = 0;\n        for (int r = -1; r < rounds; ++r) {"),
    ("sum over neighbours replaced by the last neighbour", "for (int j = 0; j < d; ++j) s[j] += msg[j];\n        }\n        mlp(gg,",
     "for (int j = 0; j < d; ++j) s[j] = msg[j];\n        }\n        mlp(gg,"),
]

# the pins, cheapest first (the exhaustive four-node brute force is left to the pin suite itself)
PINS = [
    pins.test_diamond_fixture,
    pins.test_feature_layout,
    pins.test_path_counting,
    lambda: pins.test_chain_closed_form(2),
    lambda: pins.test_general_dag_linear_solve(False),
    lambda: pins.test_general_dag_linear_solve(True),
    pins.test_single_node_is_plain_mlp,
    pins.test_softmax_properties,
    pins.test_groups_partition_and_match_closure,
    pins.test_pooling_sum_identity,
    pins.test_simple_partitioner_special_case,
    pins.test_influence_sets,
    lambda: pins.test_brute_force_random_small_dags(5, 1),
    lambda: pins.test_brute_force_random_small_dags(6, 2),
    lambda: pins.test_synchronous_rounds_truncated_series(2),
]


def _load(path):
    lib = ctypes.CDLL(path)
    for fn in ("oracle_features", "oracle_embed", "oracle_embed_sync", "oracle_policy",
               "oracle_group_sizes", "oracle_real_bytes"):
        getattr(lib, fn).restype = ctypes.c_int
    return lib


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(name, old, new, tmp_path):
    source = open(SRC).read()
    assert source.count(old) >= 1, "mutation target not found: " + name
    mutated = tmp_path / "mutant.c"
    mutated.write_text(source.replace(old, new))
    lib_path = str(tmp_path / "libmutant.so")
    subprocess.run(["gcc", "-O1", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-DORACLE_REAL=double",
                    str(mutated), "-o", lib_path, "-lm"], check=True)
    oracle.build()
    good = oracle._lib("double")
    oracle._LIBS["double"] = _load(lib_path)
    try:
        caught = None
        for pin in PINS:
            try:
                pin()
            except (AssertionError, ValueError) as e:
                caught = (pin, e)
                break
    finally:
        oracle._LIBS["double"] = good
    assert caught is not None, "no pin noticed: " + name
    # and the untouched checker still passes the pin that caught the mutant
    caught[0]()
