"""The pins must be able to fail: deliberately broken copies of the oracle (one changed line each) are built and
the pin tests are run against them; every copy has to be caught, and the unchanged copy has to pass."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "avsg_oracle.c")

MUTATIONS = [
    ("unchanged", None, None),
    ("no pre-decay of the first token", "if (g == 0) decay_all(t);", "(void)g;"),
    ("hits are not refreshed", "if (m[i]) t->life[o[i]] = t->L;", "if (0) t->life[o[i]] = t->L;"),
    ("a lifetime of 0 counts as dead", "if (t->life[j] < 0) e[n++] = (int32_t)j;", "if (t->life[j] <= 0) e[n++] = (int32_t)j;"),
    ("lifetimes do not saturate", "if (t->life[j] > -1) t->life[j] -= 1;", "t->life[j] -= 1;"),
    ("a new entry gets no lifetime", "        t->life[j] = t->L;\n        o[i] = j;", "        o[i] = j;"),
    ("invalidation spares id == N", "if (t->c[j] >= N) t->c[j] = -1;", "if (t->c[j] > N) t->c[j] = -1;"),
    ("dead slots are taken from the end", "int32_t j = e[k++];", "int32_t j = e[n_dead - 1 - k++];"),
    ("a dead slot cannot be hit", "if (t->c[j] == x) return (int32_t)j;", "if (t->c[j] == x && t->life[j] >= 0) return (int32_t)j;"),
    ("misses are placed in reverse order", "for (uint32_t i = 0; i < K; ++i) {\n        if (x[i] < 0 || m[i]) continue;",
     "for (uint32_t i = K; i-- > 0;) {\n        if (x[i] < 0 || m[i]) continue;"),
    ("later tokens are pre-decayed too", "if (g == 0) decay_all(t);", "decay_all(t);"),
    ("hits are refreshed after the allocation instead of before",
     ["if (m[i]) t->life[o[i]] = t->L;", "    t->tokens++;\n    t->hits += valid"],
     ["if (0) t->life[o[i]] = t->L;",
      "    for (uint32_t i = 0; i < K; ++i) if (m[i]) t->life[o[i]] = t->L;\n    t->tokens++;\n    t->hits += valid"]),
    ("padding counts as a miss", "if (x[i] >= 0) { valid++; n_g += 1 - (int32_t)m[i]; }",
     "{ valid += x[i] >= 0; n_g += 1 - (int32_t)m[i]; }"),
    ("Eq. 6 drops the remainder", "*end = *begin + q + (c < r ? 1 : 0);", "*end = *begin + q;"),
    ("Eq. 13 ignores the remainder", "return B / C + (c < B % C ? 1u : 0u);", "return B / C;"),
    ("Eq. 14 rounds the upper end up", "*end = (uint64_t)(c + 1) * n_positions / C;",
     "*end = ((uint64_t)(c + 1) * n_positions + C - 1) / C;"),
    ("the gather steps through the host rows by row_bytes instead of the stride",
     "host_kv + (uint64_t)list[k].x * row_stride, t->row_bytes);", "host_kv + (uint64_t)list[k].x * t->row_bytes, t->row_bytes);"),
    ("transfer-all-K ignores the host row stride",
     "host_kv + (uint64_t)X[p] * row_stride, t->row_bytes);", "host_kv + (uint64_t)X[p] * t->row_bytes, t->row_bytes);"),
    ("reset forgets the counters",
     "    t->steps = t->tokens = t->hits = t->misses = t->rows_copied = t->extra_decays = 0;\n}", "}"),
    ("reset leaves the rows", "    memset(t->rows, 0, (size_t)t->S * t->row_bytes);\n    t->steps = ", "    t->steps = "),
    ("reset leaves the lifetimes",
     "for (uint32_t j = 0; j < t->S; ++j) { t->c[j] = -1; t->life[j] = -1; }\n    memset(",
     "for (uint32_t j = 0; j < t->S; ++j) { t->c[j] = -1; }\n    memset("),
    ("transfer-all-K keeps a padding row", "if (X[p] < 0) { O[p] = -1; continue; }", "if (X[p] < 0) { O[p] = (int32_t)p; continue; }"),
]

# the paper-literal Hash-State mode (Eq. 2-4, 8-11, Alg. 2), against its own pins
LITERAL_MUTATIONS = [
    ("unchanged", None, None),
    ("the probe visits R buckets instead of R + 1", "for (uint32_t r = 0; r <= t->R; ++r) {\n        const uint32_t o = t->q[h] % S;",
     "for (uint32_t r = 0; r < t->R; ++r) {\n        const uint32_t o = t->q[h] % S;"),
    ("the probe step is not forced odd", "const uint32_t d = ((t->a2 * (uint32_t)x) % S) | 1u;",
     "const uint32_t d = ((t->a2 * (uint32_t)x) % S);"),
    ("the step of UpdateState is not forced odd", "const uint32_t d = ((t->a2 * (uint32_t)x[i]) % S) | 1u;",
     "const uint32_t d = ((t->a2 * (uint32_t)x[i]) % S);"),
    ("reclamation ignores the fingerprint", " || phi_h != ((uint32_t)t->c[o] % F);", ";"),
    ("reclamation ignores the invalid bit", "return b == 1 || lit_life(t->q[o]) < 0", "return lit_life(t->q[o]) < 0"),
    ("reclamation ignores the lifetime", "return b == 1 || lit_life(t->q[o]) < 0 || ", "return b == 1 || "),
    ("hits are not refreshed", "if (m[i]) t->q[o[i]] = lit_set_life(t->q[o[i]], t->L);", "if (0) t->q[o[i]] = lit_set_life(t->q[o[i]], t->L);"),
    ("the bucket word keeps no fingerprint", "| (((uint32_t)x[i] % F) << t->m) | (uint32_t)o[i];", "| (uint32_t)o[i];"),
]


def _run_pins(tmp_path, pins, label, old, new):
    text = open(SRC).read()
    if old is not None:
        olds, news = (old, new) if isinstance(old, list) else ([old], [new])
        for o, n in zip(olds, news):
            assert text.count(o) >= 1, "the line to change was not found"
            text = text.replace(o, n, 1)          # the first occurrence is the exact oracle's (the literal mode follows it)
    src, lib = tmp_path / "avsg_oracle.c", tmp_path / "libavsg_oracle_variant.so"
    src.write_text(text)
    subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-o", str(lib), str(src)])
    env = dict(os.environ, AVSG_ORACLE_LIB=str(lib))
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", pins), "-x", "-q",
                        "-p", "no:cacheprovider"], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    if old is None:
        assert r.returncode == 0, r.stdout[-2000:]
    else:
        assert r.returncode != 0, "no pin noticed: " + label


@pytest.mark.parametrize("label,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_pins_catch_a_broken_oracle(tmp_path, label, old, new):
    _run_pins(tmp_path, "test_oracle_pins.py", label, old, new)


@pytest.mark.parametrize("label,old,new", LITERAL_MUTATIONS, ids=[m[0] for m in LITERAL_MUTATIONS])
def test_pins_catch_a_broken_literal_oracle(tmp_path, label, old, new):
    _run_pins(tmp_path, "test_oracle_literal.py", label, old, new)
