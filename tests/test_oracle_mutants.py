"""Each plausible mistake, planted in a copy of the oracle's source on the CPU, must fail at least one
pin.  This is what shows the pins are strong enough to trust the oracle as the yardstick for the CUDA path."""
import os
import subprocess

import pytest

from oracle.oracle import OracleAPI, _SRC
from tests import oracle_pins

# (name, text in the source, replacement)
MUTANTS = [
    ("accumulate_minus", "float a = eps[j] + grad_at(grad, grad_dtype, j);", "float a = eps[j] - grad_at(grad, grad_dtype, j);"),
    ("accumulate_drops_eps", "float a = eps[j] + grad_at(grad, grad_dtype, j);", "float a = grad_at(grad, grad_dtype, j);"),
    ("score_signed", "score_out[j] = std::fabs(a);  // regulariser 1", "score_out[j] = a;  // regulariser 1"),
    ("numerator_plus", "g_prev[j] - omega_n * prev_val[i]", "g_prev[j] + omega_n * prev_val[i]"),
    ("numerator_no_weight", "g_prev[j] - omega_n * prev_val[i]", "g_prev[j] - prev_val[i]"),
    ("denominator_no_weight", "float den = omega_n * a;", "float den = a;"),
    ("operands_transposed", "float num = g_prev[j] - omega_n * prev_val[i];\n      float den = omega_n * a;",
     "float num = g_prev[j] - omega_n * a;\n      float den = omega_n * prev_val[i];"),
    ("one_minus_delta", "std::fabs(1.0f + delta)", "std::fabs(1.0f - delta)"),
    ("no_abs", "float r = std::fabs(1.0f + delta);", "float r = 1.0f + delta;"),
    ("times_mu", "float x = r / mu;", "float x = r * mu;"),
    ("regulariser_dropped", "score_out[j] = std::fabs(a) * m;", "score_out[j] = std::fabs(a);"),
    ("regulariser_only", "score_out[j] = std::fabs(a) * m;", "score_out[j] = m;"),
    ("half_one_plus_tanh", "m = regtopk_oracle_tanh(x);", "m = 0.5f * (1.0f + regtopk_oracle_tanh(x));"),
    ("zero_den_gives_zero_over_zero", "if (den == 0.0f) {", "if (false) {"),
    ("sort_ascending", "return x.score > y.score;", "return x.score < y.score;"),
    ("ties_high_index", "return x.idx < y.idx;", "return x.idx > y.idx;"),
    ("sends_score", "out_val[i] = a[j];  // the raw accumulator", "out_val[i] = score[j];  // the raw accumulator"),
    ("residual_not_cleared", "eps[j] = 0.0f;      // a - a", ";"),
    ("residual_not_carried", "eps[j] = a[j];  // a - 0", "eps[j] = 0.0f;"),
    ("aggregate_no_weight", "float t = omega[n] * val[n * k + i];", "float t = val[n * k + i];"),
    ("aggregate_overwrites", "g_out[j] = g_out[j] + t;", "g_out[j] = t;"),
    ("aggregate_reverse_order", "for (int32_t n = 0; n < N; ++n) {", "for (int32_t n = N - 1; n >= 0; --n) {"),
    ("exponent_not_inverted", "if (y != 1.0f) m = regtopk_oracle_pow(m, 1.0f / y);", "if (y != 1.0f) m = regtopk_oracle_pow(m, y);"),
    ("exponent_ignored", "if (y != 1.0f) m = regtopk_oracle_pow(m, 1.0f / y);", ";"),
    ("pow_log_sign", "float s = (f - 1.0f) / (f + 1.0f);", "float s = (1.0f - f) / (f + 1.0f);"),
    ("pow_drops_exponent_part", "float L = static_cast<float>(e) + log2f;", "float L = log2f;"),
    ("update_adds", "theta[j] = theta[j] - step;", "theta[j] = theta[j] + step;"),
    ("update_ignores_eta", "float step = eta * g[j];", "float step = g[j];"),
    ("tanh_inverted", "return (1.0f - t) / (1.0f + t);", "return (1.0f + t) / (1.0f - t);"),
    ("tanh_exp_minus_x", "float y = (-2.0f * x) * log2e;", "float y = (-1.0f * x) * log2e;"),
    ("tanh_small_branch_linear", "return x + x * q;", "return x;"),
    ("tanh_saturates_early", "if (x >= 9.25f) return 1.0f;", "if (x >= 2.0f) return 1.0f;"),
    ("bf16_shift", "static_cast<uint32_t>(h) << 16", "static_cast<uint32_t>(h) << 15"),
    ("nth_element_off_by_one", "rec.begin() + k, rec.end(), ranks_before);", "rec.begin() + k + 1, rec.end(), ranks_before);"),
    ("layered_ignores_layer_start", "for (int64_t j = begin; j < end; ++j) rec.push_back", "for (int64_t j = 0; j < end; ++j) rec.push_back"),
    ("layered_global_k", "for (int64_t i = 0; i < kl; ++i) chosen[i] = rec[i].idx;", "for (int64_t i = 0; i < kl; ++i) chosen[i] = rec[(i + 1) % rec.size()].idx;"),
    ("layered_sends_score", "out_val[out] = a[j];   // the raw accumulator", "out_val[out] = score[j];   // the raw accumulator"),
    ("layered_residual_not_cleared", "eps[j] = 0.0f;         // a - a", ";"),
    ("layered_residual_not_carried", "eps[j] = a[j];  // (a minus 0", "eps[j] = 0.0f;  // (a minus 0"),
    ("layered_accepts_gap", "if (begin != d) return -1;", ";"),
    ("certificate_strict", "if (!ranks_before(last, r)) ++count;", "if (ranks_before(r, last)) ++count;"),
]


def _build_mutant(tmp_path, name, old, new):
    src = open(_SRC).read()
    assert src.count(old) == 1, f"mutation site for {name} not unique/present"
    path = tmp_path / f"{name}.cpp"
    path.write_text(src.replace(old, new))
    so = tmp_path / f"{name}.so"
    subprocess.run(["g++", "-std=c++17", "-O1", "-ffp-contract=off", "-fPIC", "-shared", "-o", str(so), str(path)],
                   check=True)
    return str(so)


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_mutant_is_caught(tmp_path, name, old, new):
    api = OracleAPI(_build_mutant(tmp_path, name, old, new))
    for pin in oracle_pins.ALL_PINS:
        try:
            pin(api)
        except Exception:
            return  # caught (an assertion, or the broken oracle raised)
    pytest.fail(f"no pin notices the planted mistake '{name}'")
