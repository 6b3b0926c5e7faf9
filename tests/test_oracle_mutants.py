"""Do the pins have teeth?  Each case plants ONE plausible mistake in a copy of the oracle's C
source (on the CPU; the product is not involved), builds it, routes the oracle front end
through it and expects at least one pin of the regular oracle tests to fail."""
import os
import subprocess

import pytest

import oracle
import test_oracle_pairs as t_pairs
import test_oracle_policies as t_pol
import test_oracle_rope as t_rope
import test_oracle_score as t_score
import test_oracle_select as t_sel
import test_oracle_step as t_step

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(os.path.dirname(HERE), "oracle", "sirllm_oracle.c")
GOLDEN = os.path.join(HERE, "golden")

MUTANTS = {
    "entropy: sign of the log-sum term":
        ("return (m - logit_at(row, dtype, id)) + log(s);", "return (m - logit_at(row, dtype, id)) - log(s);"),
    "entropy: max shift dropped":
        ("s += exp(logit_at(row, dtype, v) - m);", "s += exp(logit_at(row, dtype, v));"),
    "entropy: base-2 logarithm":
        ("return (m - logit_at(row, dtype, id)) + log(s);", "return (m - logit_at(row, dtype, id)) + log2(s);"),
    "entropy: score of the arg-max instead of the realised token":
        ("return (m - logit_at(row, dtype, id)) + log(s);", "return (m - m) + log(s);"),
    "pairs: tile maxima ignored":
        ("S += (double)pairs[2 * i + 1] * exp((double)pairs[2 * i] - M);", "S += (double)pairs[2 * i + 1];"),
    "range pair: every rank claims the target logit":
        ("(id >= 0 && (int64_t)id >= v0 && (int64_t)id < v1) ? (float)logit_at(row, dtype, id) : 0.0f;",
         "(id >= 0) ? (float)logit_at(row, dtype, id) : 0.0f;"),
    "range pair: sum not taken relative to the range's maximum":
        ("        for (int64_t v = v0; v < v1; ++v)\n            s += exp(logit_at(row, dtype, v) - m);",
         "        for (int64_t v = v0; v < v1; ++v)\n            s += exp(logit_at(row, dtype, v));"),
    "range pair: maximum of the whole row":
        ("    for (int64_t v = v0; v < v1; ++v) {\n        double z = logit_at(row, dtype, v);",
         "    for (int64_t v = 0; v < v1; ++v) {\n        double z = logit_at(row, dtype, v);"),
    "decay: applied to the old scores only":
        ("    l += T;\n    oracle_decay(E, l, eta);", "    oracle_decay(E, l, eta);\n    l += T;"),
    "decay: applied twice per round":
        ("    l += T;\n    oracle_decay(E, l, eta);", "    l += T;\n    oracle_decay(E, l, eta);\n    oracle_decay(E, l, eta);"),
    "decay: not an fp32 product (double kept until the cache is read)":
        ("volatile float p = E[i] * eta;", "volatile float p = (float)((double)E[i] * (double)eta * 1.0000001);"),
    "select: ties go to the newer slot":
        ("return (a->slot > b->slot) - (a->slot < b->slot);", "return (a->slot < b->slot) - (a->slot > b->slot);"),
    "select: lowest scores kept":
        ("return a->key > b->key ? -1 : 1;", "return a->key > b->key ? 1 : -1;"),
    "select: recent window one slot short":
        ("int32_t lo = n_sink, hi = l - n_recent, k = budget - n_sink - n_recent;\n    int32_t n_mid = hi - lo;\n    ranked_t *mid = malloc(sizeof(ranked_t) * (size_t)(n_mid > 0 ? n_mid : 1));\n    for (int32_t i = lo; i < hi; ++i) {\n        mid[i - lo].key = oracle_order_key(E[i]);",
         "int32_t lo = n_sink, hi = l - n_recent + 1, k = budget - n_sink - n_recent;\n    int32_t n_mid = hi - lo;\n    ranked_t *mid = malloc(sizeof(ranked_t) * (size_t)(n_mid > 0 ? n_mid : 1));\n    for (int32_t i = lo; i < hi; ++i) {\n        mid[i - lo].key = oracle_order_key(E[i]);"),
    "select: n_sink + 1 sink slots (the formula as printed)":
        ("int32_t lo = n_sink, hi = l - n_recent, k = budget - n_sink - n_recent;\n    int32_t n_mid = hi - lo;\n    ranked_t *mid = malloc(sizeof(ranked_t) * (size_t)(n_mid > 0 ? n_mid : 1));\n    for (int32_t i = lo; i < hi; ++i) {\n        mid[i - lo].key = oracle_order_key(E[i]);",
         "int32_t lo = n_sink + 1, hi = l - n_recent, k = budget - n_sink - n_recent - 1;\n    int32_t n_mid = hi - lo;\n    ranked_t *mid = malloc(sizeof(ranked_t) * (size_t)(n_mid > 0 ? n_mid : 1));\n    for (int32_t i = lo; i < hi; ++i) {\n        mid[i - lo].key = oracle_order_key(E[i]);"),
    "select: evicts already at the threshold":
        ("    if (l <= threshold) {\n        for (int32_t i = 0; i < l; ++i)\n            keep[i] = i;\n        return l;\n    }\n    int32_t lo = n_sink, hi = l - n_recent, k",
         "    if (l < threshold) {\n        for (int32_t i = 0; i < l; ++i)\n            keep[i] = i;\n        return l;\n    }\n    int32_t lo = n_sink, hi = l - n_recent, k"),
    "order key: raw bit pattern":
        ("return (u & 0x80000000u) ? ~u : (u | 0x80000000u);", "return u;"),
    "gather: identity instead of X[Id]":
        ("(const char *)src + (size_t)keep[j] * (size_t)row_bytes, (size_t)row_bytes);",
         "(const char *)src + (size_t)j * (size_t)row_bytes, (size_t)row_bytes);"),
    "round: scores not compacted with the cache":
        ("    memcpy(E, E2, sizeof(float) * (size_t)n_keep);", "    (void)E2;"),
    "round: tags not compacted with the cache":
        ("        memcpy(serial, s2, sizeof(int64_t) * (size_t)n_keep);", "        (void)s2;"),
    "round: only the first plane of a cache is compacted":
        ("        for (int64_t p = 0; p < n_planes; ++p) {\n            char *plane", "        for (int64_t p = 0; p < 1; ++p) {\n            char *plane"),
    "round: the V cache is left as it was":
        ("    for (int c = 0; c < 2; ++c) {\n        if (!caches[c])", "    for (int c = 0; c < 1; ++c) {\n        if (!caches[c])"),
    "round: new scores appended after the decay":
        ("    l += T;\n    oracle_decay(E, l, eta);", "    oracle_decay(E, l + T, eta);\n    for (int32_t t = 0; t < T; ++t)\n        E[l + t] = new_e[t];\n    l += T;"),
    "interval policy: interval from the retained size":
        ("    int32_t interval = l / budget;", "    int32_t interval = budget / (l - budget + 1) + 1;"),
    "random policy: round not part of the counter":
        ("uint32_t ctr[4] = {(uint32_t)i, (uint32_t)round, (uint32_t)stream, 0u}, out[4];",
         "uint32_t ctr[4] = {(uint32_t)i, 0u, (uint32_t)stream, 0u}, out[4];"),
    "rope: rotation the wrong way round":
        ("        *px = x * c - y * s;\n        *py = x * s + y * c;", "        *px = x * c + y * s;\n        *py = -x * s + y * c;"),
    "rope: frequencies base^(-i/d)":
        ("double theta = pow(base, -2.0 * (double)i / (double)d);", "double theta = pow(base, -1.0 * (double)i / (double)d);"),
    "rope: turned by the new position instead of the shift":
        ("        int32_t delta = j - keep[j];", "        int32_t delta = j;"),
    "rope: storage rounding truncates":
        ("return ldexp(nearbyint(ldexp(m, keep)), e - keep);", "return ldexp(trunc(ldexp(m, keep)), e - keep);"),
    "philox: nine rounds":
        ("for (int r = 0; r < 10; ++r) {", "for (int r = 0; r < 9; ++r) {"),
}


def _pins():
    """The regular pins, as plain callables."""
    calls = []
    for mod in (t_score, t_sel, t_step, t_pairs, t_pol, t_rope):
        for name in sorted(dir(mod)):
            fn = getattr(mod, name)
            if not name.startswith("test_") or not callable(fn):
                continue
            marks = [m for m in getattr(fn, "pytestmark", []) if m.name == "parametrize"]
            inner = getattr(fn, "hypothesis", None)
            target = fn
            if marks:
                argnames, values = marks[0].args[0], marks[0].args[1]
                n = len([a for a in argnames.split(",")])
                for v in values:
                    args = v if n > 1 else (v,)
                    calls.append((f"{name}[{v}]", lambda f=target, a=tuple(args): f(*a)))
            elif "golden_dir" in fn.__code__.co_varnames[:fn.__code__.co_argcount]:
                calls.append((name, lambda f=target: f(GOLDEN)))
            else:
                calls.append((name, lambda f=target: f()))
            del inner
    return calls


def test_the_unmodified_oracle_passes_every_pin_called_this_way():
    for name, call in _pins():
        call()


@pytest.mark.parametrize("label", sorted(MUTANTS))
def test_every_planted_mistake_is_caught(label, tmp_path):
    old, new = MUTANTS[label]
    src = open(SRC).read()
    assert old in src, "mutation site not found"
    mutated = tmp_path / "mutant.c"
    mutated.write_text(src.replace(old, new, 1))        # the first site (oracle_select / oracle_step)
    lib = tmp_path / "libmutant.so"
    subprocess.check_call(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-shared", "-fPIC", "-o",
                           str(lib), str(mutated), "-lm"])
    caught = []
    with oracle.use_library(str(lib)):
        for name, call in _pins():
            try:
                call()
            except AssertionError:
                caught.append(name)
            except Exception as exc:          # a broken oracle may also raise elsewhere
                caught.append(f"{name} ({type(exc).__name__})")
    assert caught, f"no pin noticed: {label}"
