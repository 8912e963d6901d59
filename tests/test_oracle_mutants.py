"""Do the oracle's pins bite?  Each case plants ONE plausible mistake in a copy of the oracle (a
dropped term, a wrong sign or index, another rounding rule, a reordered step), rebuilds that copy
and runs the pin tests of the part it touches against it: they must fail.  An unchanged copy must
pass, which shows that a failure comes from the planted mistake and not from the harness.

Everything here happens on the CPU, in a temporary copy; the oracle in the tree is not touched."""
import os
import shutil
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CPP, PY = "mp_oracle.cpp", "mp_oracle.py"

# (name, file, text as it stands, text with the mistake, pin files that must catch it)
MUTANTS = [
    ("unchanged", CPP, None, None, ["test_oracle_update.py"]),
    ("f2h_ties_round_up", CPP, "(rem == 0x1000u && (half & 1u))", "(rem == 0x1000u)", ["test_oracle_fp16.py"]),
    ("f2h_saturates", CPP, "if (e > 15) return (uint16_t)(sign | 0x7C00u);",
     "if (e > 15) return (uint16_t)(sign | 0x7BFFu);", ["test_oracle_fp16.py"]),
    ("f2h_flushes_subnormals", CPP, "if (e < -25) return sign;", "if (e < -14) return sign;", ["test_oracle_fp16.py"]),
    ("h2f_subnormal_exponent", CPP, "(uint32_t)(127 - 15 - shift + 1)", "(uint32_t)(127 - 15 - shift)",
     ["test_oracle_fp16.py"]),
    ("fwd_sums_descending", CPP,
     "for (int64_t k = 0; k < K; ++k) acc = acc + h2f(X[m * ldx + k]) * h2f(W[k * ldw + n]);\n        Y[m * ldy + n] = f2h(acc);",
     "for (int64_t k = K - 1; k >= 0; --k) acc = acc + h2f(X[m * ldx + k]) * h2f(W[k * ldw + n]);\n        Y[m * ldy + n] = f2h(acc);",
     ["test_oracle_matmul.py"]),
    ("dgrad_wrong_sign", CPP,
     "acc = acc + h2f(dY[m * lddy + n]) * h2f(W[k * ldw + n]);\n        dX[m * lddx + k] = f2h(acc);",
     "acc = acc - h2f(dY[m * lddy + n]) * h2f(W[k * ldw + n]);\n        dX[m * lddx + k] = f2h(acc);",
     ["test_oracle_matmul.py"]),
    ("wgrad_reversed_columns", CPP,
     "acc = acc + h2f(X[m * ldx + k]) * h2f(dY[m * lddy + n]);\n        dW[k * lddw + n] = f2h(acc);",
     "acc = acc + h2f(X[m * ldx + k]) * h2f(dY[m * lddy + (N - 1 - n)]);\n        dW[k * lddw + n] = f2h(acc);",
     ["test_oracle_matmul.py"]),
    ("scale_rounds_before_scaling", CPP, "dY16[i] = f2h(S * g32[i]);", "dY16[i] = f2h(S * h2f(f2h(g32[i])));",
     ["test_oracle_update.py"]),
    ("flag_misses_nan", CPP, "return (h & 0x7C00u) == 0x7C00u; }", "return (h & 0x7FFFu) == 0x7C00u; }",
     ["test_oracle_update.py"]),
    ("adam_eps_inside_root", CPP, "(std::sqrt(vh) + eps)", "std::sqrt(vh + eps)", ["test_oracle_update.py"]),
    ("adam_v_not_bias_corrected", CPP, "const float vh = vi / c2;", "const float vh = vi;", ["test_oracle_update.py"]),
    ("adam_forgets_to_unscale", CPP, "float g = h2f(g16[i]) * inv;", "float g = h2f(g16[i]);", ["test_oracle_update.py"]),
    ("momentum_dampened", CPP, "const float ui = mu * u[i] + g;", "const float ui = mu * u[i] + (1.0f - mu) * g;",
     ["test_oracle_update.py"]),
    ("decay_from_fp16_copy", CPP, "g = g + weight_decay * w32[i];", "g = g + weight_decay * h2f(f2h(w32[i]));",
     ["test_oracle_fp16.py", "test_oracle_update.py"]),
    ("momentum_decay_from_fp16_copy", CPP, "g = g + weight_decay * w32[i];\n    const float ui",
     "g = g + weight_decay * h2f(f2h(w32[i]));\n    const float ui", ["test_oracle_update.py"]),
    ("skipped_step_advances_t", CPP, "    s->skipped += 1;\n", "    s->skipped += 1; s->t += 1;\n", ["test_oracle_update.py"]),
    ("overflow_keeps_clean_run", CPP, "    s->good = 0;\n    s->strikes += 1;", "    s->strikes += 1;",
     ["test_oracle_update.py"]),
    ("scale_not_clamped_below", CPP, "std::max(s->S * 0.5f, s->s_min)", "(s->S * 0.5f)", ["test_oracle_update.py"]),
    ("growth_not_clamped_above", CPP, "std::min(s->S * 2.0f, s->s_max)", "(s->S * 2.0f)", ["test_oracle_update.py"]),
    ("bias_after_activation", CPP,
     "if (b) acc = acc + h2f(b[n]);\n        Y[m * ldy + n] = f2h(apply_act(acc, act, clip));",
     "acc = apply_act(acc, act, clip);\n        if (b) acc = acc + h2f(b[n]);\n        Y[m * ldy + n] = f2h(acc);",
     ["test_oracle_layers.py"]),
    ("relu_mask_not_strict", CPP, "if (act == 1) return y > 0.0f;", "if (act == 1) return y >= 0.0f;",
     ["test_oracle_layers.py", "test_oracle_step.py"]),
    ("bias_grad_sums_in_fp16", CPP, "acc = acc + h2f(dY[m * lddy + n]);", "acc = h2f(f2h(acc + h2f(dY[m * lddy + n])));",
     ["test_oracle_layers.py"]),
    ("lstm_gates_swapped", CPP, "const float c = f * h2f(c_prev[m * H + j]) + i * g;",
     "const float c = i * h2f(c_prev[m * H + j]) + f * g;", ["test_oracle_layers.py"]),
    ("clipped_relu_does_not_clip", CPP, "return x < clip ? x : clip; }", "return x; }", ["test_oracle_layers.py"]),
    ("lstm_output_gate_derivative", CPP, "f2h(dhv * tc * (o * (1.0f - o)))", "f2h(dhv * tc * (o * (1.0f + o)))",
     ["test_oracle_layers.py"]),
    ("only_the_bottom_layer_is_inspected", PY, "        flag |= found_inf(ly.dW)", "        flag = found_inf(ly.dW)",
     ["test_oracle_step.py"]),
    ("f2h_nan_becomes_inf", CPP, "return (uint16_t)(sign | 0x7E00u);           // NaN",
     "return (uint16_t)(sign | 0x7C00u);           // NaN", ["test_oracle_fp16.py"]),
    ("h2f_nan_becomes_inf", CPP, "return bits_f32(sign | 0x7F800000u | (f << 13));", "return bits_f32(sign | 0x7F800000u);",
     ["test_oracle_fp16.py", "test_oracle_matmul.py"]),
    ("products_rounded_to_fp16", CPP,
     "acc = acc + h2f(X[m * ldx + k]) * h2f(W[k * ldw + n]);\n        Y[m * ldy + n] = f2h(acc);",
     "acc = acc + h2f(f2h(h2f(X[m * ldx + k]) * h2f(W[k * ldw + n])));\n        Y[m * ldy + n] = f2h(acc);",
     ["test_oracle_matmul.py"]),
    ("adam_first_moment_not_averaged", CPP, "const float mi = b1 * m[i] + omb1 * g;", "const float mi = b1 * m[i] + g;",
     ["test_oracle_update.py"]),
    ("static_scale_still_halves", CPP, "if (s->dynamic && s->strikes >= s->tolerance)", "if (s->strikes >= s->tolerance)",
     ["test_oracle_update.py"]),
    ("adam_step_count_off_by_one", PY, "        t = scaler.t + 1\n", "        t = scaler.t + 2\n", ["test_oracle_step.py"]),
    ("sampled_wgrad_index", CPP, "else              { a = h2f(A[j * lda + r]); b = h2f(B[j * ldb + c]); }\n      acc = acc + a * b;",
     "else              { a = h2f(A[j * lda + r]); b = h2f(B[c * ldb + j]); }\n      acc = acc + a * b;",
     ["test_oracle_matmul.py"]),
    ("exact_sum_drops_sign", CPP, "          ex += (double)a * (double)b;\n          ab += std::fabs((double)a * (double)b);\n        }\n        out_exact",
     "          ex += std::fabs((double)a * (double)b);\n          ab += std::fabs((double)a * (double)b);\n        }\n        out_exact",
     ["test_oracle_matmul.py"]),
    ("exact_abs_sum_signed", CPP, "          ex += (double)a * (double)b;\n          ab += std::fabs((double)a * (double)b);\n        }\n        out_exact",
     "          ex += (double)a * (double)b;\n          ab += (double)a * (double)b;\n        }\n        out_exact",
     ["test_oracle_matmul.py"]),
    ("overflow_step_applied", PY, "    if not flag:                                          # Section 3.2",
     "    if True:", ["test_oracle_step.py"]),
    ("scale_applied_twice", PY, "ly.dY = layers[l + 1].dX if feeds_next else scale_upstream(gs[l], S)",
     "ly.dY = layers[l + 1].dX if feeds_next else scale_upstream(gs[l], S * S)", ["test_oracle_step.py"]),
]


@pytest.mark.parametrize("name,fname,old,new,pins", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(tmp_path, name, fname, old, new, pins):
    root = tmp_path / "copy"
    (root / "oracle").mkdir(parents=True)
    (root / "tests").mkdir()
    for f in (CPP, PY, "__init__.py"):
        shutil.copy(os.path.join(ROOT, "oracle", f), root / "oracle" / f)
    os.symlink(os.path.join(ROOT, "paper_1805_10387_b200"), root / "paper_1805_10387_b200")
    os.symlink(os.path.join(ROOT, "tests", "golden"), root / "tests" / "golden")
    shutil.copy(os.path.join(ROOT, "tests", "conftest.py"), root / "tests" / "conftest.py")
    for p in pins:
        shutil.copy(os.path.join(ROOT, "tests", p), root / "tests" / p)
    if old is not None:
        path = root / "oracle" / fname
        src = path.read_text()
        assert src.count(old) >= 1, f"{name}: the text to change is not in {fname} any more"
        path.write_text(src.replace(old, new, 1))
    env = dict(os.environ, PYTHONDONTWRITEBYTECODE="1")
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider"] +
                       [str(root / "tests" / p) for p in pins], cwd=root, env=env, capture_output=True, text=True,
                       timeout=600)
    tail = (r.stdout + r.stderr)[-1500:]
    if old is None:
        assert r.returncode == 0, tail                 # the harness itself is sound
    else:
        assert r.returncode == 1, f"{name} was NOT caught by {pins}:\n{tail}"   # 1 = tests ran and failed
        # ... because a pin's assertion failed, not because the changed copy did not build or import
        assert "CalledProcessError" not in tail and "SyntaxError" not in tail and "AssertionError" in r.stdout, tail
