"""The pins are only worth something if a plausible mistake in the oracle fails one of them.

Each case plants one mistake in a COPY of the oracle's C source (a dropped term, a wrong sign or
index, a swapped operand, an off-by-one), compiles the copy on the CPU, loads it through a private
copy of the oracle's Python front end, and runs the pin tests of the affected part against it: at
least one of them must fail.  The unmodified source must pass the same tests through the same route.
"""
import importlib.util
import os
import subprocess
import sys

import pytest

from tests import test_oracle_attention, test_oracle_fp8, test_oracle_plan, test_oracle_prune, test_oracle_score, test_oracle_topk

_ORACLE_DIR = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "oracle")


def _load_variant(tmp_path, name, old=None, new=None):
    src = open(os.path.join(_ORACLE_DIR, "kvzap_oracle.c")).read()
    if old is not None:
        assert src.count(old) == 1, "mutation site not found exactly once: %r" % old
        src = src.replace(old, new)
    c_path = os.path.join(tmp_path, name + ".c")
    so_path = os.path.join(tmp_path, name + ".so")
    with open(c_path, "w") as f:
        f.write(src)
    subprocess.run(["gcc", "-O1", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-o", so_path, c_path, "-lm"], check=True)
    spec = importlib.util.spec_from_file_location("kvzap_oracle_" + name, os.path.join(_ORACLE_DIR, "kvzap_oracle.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    mod._LIB = so_path
    mod.build = lambda force=False: so_path          # the variant is already built
    return mod


def _pins(module, prefix=""):
    """Zero-argument callables for the module's tests that take only the `oracle` fixture (parametrised
    ones are run over their own parameter lists)."""
    out = []
    for name in sorted(dir(module)):
        fn = getattr(module, name)
        if not name.startswith("test_") or not callable(fn) or not name.startswith("test_" + prefix):
            continue
        marks = [m for m in getattr(fn, "pytestmark", []) if m.name == "parametrize"]
        code = fn.__code__
        args = code.co_varnames[:code.co_argcount]
        if "oracle" not in args:
            continue
        combos = [{}]
        for m in marks:
            keys = [k.strip() for k in m.args[0].split(",")]
            combos = [dict(c, **dict(zip(keys, v if len(keys) > 1 else (v,)))) for c in combos for v in m.args[1]]
        if set(args) - {"oracle"} - set(combos[0].keys()):
            continue                                   # needs a fixture this harness does not provide
        for c in combos:
            out.append((name, c, fn))
    return out


def _failures(mod, pins):
    failed = []
    for name, kwargs, fn in pins:
        try:
            fn(oracle=mod, **kwargs)
        except AssertionError:
            failed.append(name)
        except Exception as e:                         # a mutant may also crash a pin outright (shape errors, ...)
            failed.append(name + ":" + type(e).__name__)
    return failed


SCORE = _pins(test_oracle_score)
PRUNE = _pins(test_oracle_prune)
TOPK = _pins(test_oracle_topk)
ATTN = _pins(test_oracle_attention)
PLAN = _pins(test_oracle_plan)
FP8 = _pins(test_oracle_fp8)

MUTANTS = [
    # name, pins, text in the source, replacement
    ("linear_drops_bias", SCORE, "double acc = b ? (double)b[h] : 0.0;\n            for (int k = 0; k < Dh; ++k)\n                acc += bf16_to_double(X[t * Dh + k])",
     "double acc = 0.0;\n            for (int k = 0; k < Dh; ++k)\n                acc += bf16_to_double(X[t * Dh + k])"),
    ("linear_wrong_weight_row", SCORE, "bf16_to_double(W[(int64_t)h * Dh + k]);", "bf16_to_double(W[(int64_t)(H - 1 - h) * Dh + k]);"),
    ("mlp_drops_b1", SCORE, "for (int j = 0; j < N1; ++j) z[j] = b1 ? (double)b1[j] : 0.0;", "for (int j = 0; j < N1; ++j) z[j] = 0.0;"),
    ("mlp_drops_b2", SCORE, "double acc = b2 ? (double)b2[h] : 0.0;", "double acc = 0.0;"),
    ("mlp_w1_transposed", SCORE, "w1[(size_t)k * N1 + j] = bf16_to_double(W1[(size_t)j * Dh + k]);",
     "w1[(size_t)k * N1 + j] = bf16_to_double(W1[((size_t)k * N1 + j) % ((size_t)N1 * Dh)]);"),
    ("mlp_w2_wrong_head", SCORE, "acc += z[j] * w2[(size_t)h * N1 + j];", "acc += z[j] * w2[(size_t)((h + 1) % H) * N1 + j];"),
    ("gelu_sign", SCORE, "return 0.5 * x * (1.0 + erf(x / sqrt(2.0)));", "return 0.5 * x * (1.0 - erf(x / sqrt(2.0)));"),
    ("gelu_no_sqrt2", SCORE, "return 0.5 * x * (1.0 + erf(x / sqrt(2.0)));", "return 0.5 * x * (1.0 + erf(x));"),
    ("bf16_widening_wrong_half", SCORE, None, None),     # filled in below: depends on the helper's text
    ("mask_strict_compare", PRUNE, "const int above = scores[t * H + h] >= tau;", "const int above = scores[t * H + h] > tau;"),
    ("mask_window_off_by_one", PRUNE, "const int in_window = (t - t0) >= Tb - (int64_t)w;\n                const int above",
     "const int in_window = (t - t0) > Tb - (int64_t)w;\n                const int above"),
    ("mask_window_of_packed_buffer", PRUNE, "const int in_window = (t - t0) >= Tb - (int64_t)w;\n                const int above",
     "const int in_window = t >= T_total - (int64_t)w;\n                const int above"),
    ("mask_head_and_token_swapped", PRUNE, "keep[(int64_t)h * T_total + t] = (uint8_t)(in_window || above);",
     "keep[(int64_t)h * T_total + t] = (uint8_t)(in_window || (scores[t * H + (h + 1) % H] >= tau));"),
    ("compact_v_uses_k_rows", PRUNE, "memcpy(V_out + dst, V + src, row_bytes);\n            ++n;\n        }\n        lengths[b * H + h] = (int32_t)n;",
     "memcpy(V_out + dst, K + src, row_bytes);\n            ++n;\n        }\n        lengths[b * H + h] = (int32_t)n;"),
    ("compact_lists_start_at_zero", PRUNE, "const int64_t dst = ((int64_t)h * T_total + t0 + n) * D;\n            memcpy(K_out + dst, K + src, row_bytes);",
     "const int64_t dst = ((int64_t)h * T_total + n) * D;\n            memcpy(K_out + dst, K + src, row_bytes);"),
    ("compact_length_off_by_one", PRUNE, "lengths[b * H + h] = (int32_t)n;\n    }\n}\n\n/*\n * Paged variant", "lengths[b * H + h] = (int32_t)(n > 0 ? n - 1 : 0);\n    }\n}\n\n/*\n * Paged variant"),
    ("paged_pages_in_head_major_order", PRUNE, "page_table[(int64_t)list * max_pages_per_list + p] = (int32_t)(cursor + p);",
     "page_table[(int64_t)list * max_pages_per_list + p] = (int32_t)(cursor + need - 1 - p);"),
    ("write_side_reads_head_major", PRUNE, "const uint16_t *k_row = K_proj + (t * H + h) * (int64_t)D;", "const uint16_t *k_row = K_proj + ((int64_t)h * T_total + t) * (int64_t)D;"),
    ("topk_takes_k_plus_one", TOPK, "tau = buf[want - 1];", "tau = buf[want < n ? want : want - 1];"),
    ("topk_budget_rounds_down", TOPK, "const int64_t k = (int64_t)ceil(keep_ratio * (double)n_cand);", "const int64_t k = (int64_t)floor(keep_ratio * (double)n_cand);"),
    ("topk_window_tokens_are_candidates", TOPK, "for (int64_t t = t0; t < t0 + n_cand; ++t)\n                for (int hh", "for (int64_t t = t0; t < t1; ++t)\n                for (int hh"),
    ("topk_ascending", TOPK, "return (x < y) - (x > y);", "return (x > y) - (x < y);"),
    ("attention_no_scale", ATTN, "a[i] = scale * dot;", "a[i] = dot;"),
    ("attention_keys_for_values", ATTN, "acc[d] += a[i] * bf16_to_double(V[i * D + d]);", "acc[d] += a[i] * bf16_to_double(K[i * D + d]);"),
    ("attention_unnormalised", ATTN, "out[(int64_t)g * D + d] = n > 0 ? (float)(acc[d] / denom) : 0.0f;", "out[(int64_t)g * D + d] = n > 0 ? (float)(acc[d]) : 0.0f;"),
    ("plan_counts_from_one", PLAN, "slot[t * H + h] = (int32_t)n;", "slot[t * H + h] = (int32_t)(n + 1);"),
    ("plan_dropped_rows_get_a_slot", PLAN, "if (!keep[(int64_t)h * T_total + t]) continue;\n                if (page_tokens > 0)", "if (page_tokens > 0)"),
    ("plan_pages_do_not_advance", PLAN, "cursor += need;\n            }\n        }\n    if (page_tokens > 0) *n_pages_used", "cursor += 0;\n            }\n        }\n    if (page_tokens > 0) *n_pages_used"),
    ("plan_slot_ignores_the_page_offset", PLAN, "slot[t * H + h] = (int32_t)((cursor + n / page_tokens) * page_tokens + n % page_tokens);",
     "slot[t * H + h] = (int32_t)((cursor + n / page_tokens) * page_tokens);"),
    ("e4m3_bias_eight", FP8, "else v = ldexp(1.0 + (double)m / 8.0, e - 7);", "else v = ldexp(1.0 + (double)m / 8.0, e - 8);"),
    ("e4m3_subnormals_as_normals", FP8, "if (e == 0) v = ldexp((double)m / 8.0, -6);", "if (e == 0) v = ldexp(1.0 + (double)m / 8.0, -7);"),
    ("e4m3_has_infinities", FP8, "if (e == 15 && m == 7) return NAN;", "if (e == 15) return m == 0 ? INFINITY : NAN;"),
    ("fp8_linear_drops_token_scale", FP8, "const double sx = x_scale ? (double)x_scale[t] : 1.0, sw = w_scale ? (double)w_scale[h] : 1.0;",
     "const double sx = 1.0, sw = w_scale ? (double)w_scale[h] : 1.0;"),
    ("fp8_mlp_scales_the_bias_too", FP8, "z[j] = kvzap_oracle_gelu((b1 ? (double)b1[j] : 0.0) + sx * sw * z[j]);",
     "z[j] = kvzap_oracle_gelu(sx * sw * ((b1 ? (double)b1[j] : 0.0) + z[j]));"),
    ("fp8_mlp_channel_scale_by_token", FP8, "const double sw = w1_scale ? (double)w1_scale[j] : 1.0;", "const double sw = w1_scale ? (double)w1_scale[j % 2] : 1.0;"),
    ("fp8_attention_value_scale_dropped", FP8, "const double sv = v_scale ? (double)v_scale[i] : 1.0;", "const double sv = 1.0;"),
    ("fp8_attention_key_scale_after_softmax", FP8, "a[i] = scale * (k_scale ? (double)k_scale[i] : 1.0) * dot;", "a[i] = scale * dot;"),
    ("attention_shared_query", ATTN, "dot += bf16_to_double(q[(int64_t)g * D + d]) * bf16_to_double(K[i * D + d]);", "dot += bf16_to_double(q[d]) * bf16_to_double(K[i * D + d]);"),
]


def _fill_bf16_mutant():
    src = open(os.path.join(_ORACLE_DIR, "kvzap_oracle.c")).read()
    old = "((uint32_t)bits) << 16"
    if src.count(old) == 1:
        return old, "((uint32_t)bits) << 15"
    return None, None


@pytest.fixture(scope="module")
def build_dir(tmp_path_factory):
    return str(tmp_path_factory.mktemp("oracle_variants"))


def test_unmodified_source_passes_through_this_route(build_dir):
    mod = _load_variant(build_dir, "unmodified")
    for pins in (SCORE, PRUNE, TOPK, ATTN, PLAN, FP8):
        assert len(pins) >= 3
        assert _failures(mod, pins) == []


@pytest.mark.parametrize("name,pins,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_fails_a_pin(build_dir, name, pins, old, new):
    if old is None:
        old, new = _fill_bf16_mutant()
        if old is None:
            pytest.skip("widening helper is written differently")
    mod = _load_variant(build_dir, name, old, new)
    assert _failures(mod, pins), "no pin noticed the planted mistake '%s'" % name


# ---------------------------------------------------------------------------
# The decode oracle is Python: mistakes are planted by replacing one line of its source text.

DECODE_MUTANTS = [
    ("decode_window_one_too_long", "            if len(win) > self.w:", "            if len(win) > self.w + 1:"),
    ("decode_strict_compare", "                if s >= tau32:          # NaN compares false -> dropped", "                if s > tau32:"),
    ("decode_judges_the_new_score", "                if s >= tau32:          # NaN compares false -> dropped",
     "                if np.float32(scores_h[h]) >= tau32:"),
    ("decode_newest_leaves_first", "                p, s, kr, vr = win.popleft()", "                p, s, kr, vr = win.pop()"),
    ("decode_shared_heads", "            win = self.window[b][l][h]", "            win = self.window[b][l][0]"),
]


def _load_python_variant(name, old, new):
    path = os.path.join(_ORACLE_DIR, "kvzap_oracle.py")
    src = open(path).read()
    assert src.count(old) == 1, "mutation site not found exactly once: %r" % old
    src = src.replace(old, new)
    spec = importlib.util.spec_from_file_location("kvzap_oracle_" + name, path)
    mod = importlib.util.module_from_spec(spec)
    exec(compile(src, path, "exec"), mod.__dict__)
    return mod


DECODE_PINS = [p for p in PRUNE if "decode" in p[0] or "prefill_then" in p[0] or "score_buffer" in p[0]]


@pytest.mark.parametrize("name,old,new", DECODE_MUTANTS, ids=[m[0] for m in DECODE_MUTANTS])
def test_planted_mistake_in_the_decode_oracle_fails_a_pin(name, old, new):
    assert len(DECODE_PINS) >= 3
    mod = _load_python_variant(name, old, new)
    assert _failures(mod, DECODE_PINS), "no pin noticed the planted mistake '%s'" % name
