"""Checks that the pins have teeth: each plausible mistake, planted in a copy
of the CPU checker's source, must make at least one pin fail."""
import ctypes
import os
import subprocess

import pytest

import oracle
import test_oracle_pins as pins
import test_oracle_reweight_pins as reweight_pins

MUTATIONS = {
    "garbled_mg_coefficients": ("b1 * (1.0 - b2) * mk * g", "(1.0 - b1) * b2 * mk * g"),
    "mg_term_sign": ("- b1 * (1.0 - b2) * mk * g", "+ b1 * (1.0 - b2) * mk * g"),
    "eps_term_always_dropped": ("if (!h->drop_eps_term) num +=", "if (false) num +="),
    "missing_sqrt_c2_in_denominator": ("num / (rc2 * r * D * D)", "num / (r * D * D)"),
    "no_bias_correction_in_D": ("const double D = r / rc2 + eps;", "const double D = r + eps;"),
    "dropped_eps_form_keeps_exact_value_at_zero_state": ("J = h->drop_eps_term ? 0.0 : (h->lr / c1) * (1.0 - b1) / eps;",
                                                         "J = (h->lr / c1) * (1.0 - b1) / eps;"),
    "missing_c1": ("J = (h->lr / c1) * num", "J = (h->lr) * num"),
    "second_moment_uses_beta1": ("b2 * sk + (1.0 - b2) * g * g", "b1 * sk + (1.0 - b1) * g * g"),
    "gbase_ignored": ("const double g = g_base ? (double)g_base[k] : mk;", "const double g = mk;"),
    "minus_branch_sign": ("theta_minus[k] = t - d;", "theta_minus[k] = t + d;"),
    "eps_from_squared_norm": ("bad ? 0.0 : alpha / norm;", "bad ? 0.0 : alpha / (norm * norm);"),
    "transposed_weights": ("const double* w = W + (int64_t)j * din;\n                for (int32_t k = 0; k < din; ++k) acc += w[k] * h[k];",
                           "for (int32_t k = 0; k < din; ++k) acc += W[(int64_t)k * dout + j] * h[k];"),
    "relu_on_last_layer": ("(l + 1 < n_layers && acc < 0.0)", "(acc < 0.0)"),
    "bias_dropped": ("double acc = b[j];", "double acc = 0.0 * b[j];"),
    "wrong_label_logit": ("zmax - h[y[i]];", "zmax - h[0];"),
    "no_max_shift_back": ("std::log(se) + zmax - h[y[i]]", "std::log(se) - h[y[i]]"),
    "fd_sign": ("metagrad_out[i] = -sg", "metagrad_out[i] = sg"),
    "fd_one_sided_scale": ("(2.0 * eps_fd * (double)B_norm)", "(eps_fd * (double)B_norm)"),
    "sigmoid_instead_of_derivative": ("-sg * (1.0 - sg) *", "-sg *"),
    "meta_grad_relu_mask_dropped": ("dh[k] = h[l][k] > 0.0 ? dh[k] : 0.0;", "dh[k] = dh[k];"),
    "meta_grad_no_onehot": ("(c == y[i] ? 1.0 : 0.0)", "0.0"),
    "meta_grad_transposed_backprop": ("dh[k] += (double)theta[woff[l] + (int64_t)j * din + k] * dz[j];",
                                      "dh[k] += (double)theta[woff[l] + ((int64_t)k * dout + j) % ((int64_t)din * dout)] * dz[j];"),
    "reweight_sigmoid_derivative_dropped": ("const double f = l * w * (1.0 - w) / (double)B_norm;",
                                            "const double f = l * w / (double)B_norm;"),
    "reweight_loss_factor_dropped": ("const double f = l * w * (1.0 - w) / (double)B_norm;",
                                     "const double f = w * (1.0 - w) / (double)B_norm;"),
    "reweight_relu_mask_dropped": ("            if (a > 0.0) {\n                grad_out[j] += f", "            if (true) {\n                grad_out[j] += f"),
    "reweight_v1_gradient_without_input": ("grad_out[j] += f * (double)v2[j] * l;", "grad_out[j] += f * (double)v2[j];"),
    "reweight_v2_gradient_uses_weight": ("grad_out[2 * (int64_t)H + j] += f * a;", "grad_out[2 * (int64_t)H + j] += f * (double)v2[j];"),
    "reweight_fd_sign": ("eps_fd > 0.0 ? -(gp[k] - gm[k])", "eps_fd > 0.0 ? (gp[k] - gm[k])"),
    "reweight_fd_one_sided_scale": ("(gp[k] - gm[k]) / (2.0 * eps_fd)", "(gp[k] - gm[k]) / (eps_fd)"),
    "no_batch_mean": ("(2.0 * eps_fd * (double)B_norm)", "(2.0 * eps_fd)"),
}

PINS = [getattr(mod, n) for mod in (pins, reweight_pins) for n in dir(mod) if n.startswith("test_")]


def _run_all_pins():
    failures = 0
    for fn in PINS:
        marks = [m for m in getattr(fn, "pytestmark", []) if m.name == "parametrize"]
        argsets = [()]
        if marks:
            names = [a.strip() for a in marks[0].args[0].split(",")]
            argsets = [v if len(names) > 1 else (v,) for v in marks[0].args[1]]
        for args in argsets:
            try:
                fn(*args)
            except AssertionError:
                failures += 1
    return failures


def test_unmutated_checker_passes_every_pin():
    assert _run_all_pins() == 0


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(name, tmp_path, monkeypatch):
    old, new = MUTATIONS[name]
    src = open(os.path.join(os.path.dirname(oracle.__file__), "sama_oracle.cpp")).read()
    assert src.count(old) == 1, "mutation site not found exactly once"
    mutated = tmp_path / "mutant.cpp"
    mutated.write_text(src.replace(old, new))
    so = tmp_path / "mutant.so"
    subprocess.check_call(["g++", "-O1", "-std=c++17", "-fPIC", "-shared", "-o", str(so), str(mutated)])
    monkeypatch.setattr(oracle, "_lib", oracle._bind(ctypes.CDLL(str(so))))
    assert _run_all_pins() > 0, "no pin noticed: " + name
