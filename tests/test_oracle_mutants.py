"""The pins must bite: plant one plausible mistake at a time in a copy of the oracle's
source (a transposed operand, a dropped term, a wrong sign or index), rebuild it on the
CPU, and require that at least one pin test fails for every mutant."""
import functools
import os
import shutil
import types

import pytest

import test_oracle_pins as pins

MUTANTS = [
    ("fwd_W_transposed", "s += H[i * V + l] * W[l * V + j];", "s += H[i * V + l] * W[j * V + l];"),
    ("fwd_outer_sign", "Znew[i * V + j] = tanh(s + k[i] * v[j]);", "Znew[i * V + j] = tanh(s - k[i] * v[j]);"),
    ("fwd_gate_swapped", "H[i] = f * H[i] + (1.0 - f) * Znew[i];", "H[i] = (1.0 - f) * H[i] + f * Znew[i];"),
    ("fwd_residual_dropped", "if (w_r) s += w_r[j] * v[j];", ""),
    ("fwd_readout_pre_update", "/* Eq. 2: H = f H + (1-f) Z */\n  for (int i = 0; i < K * V; ++i) H[i] = f * H[i] + (1.0 - f) * Znew[i];",
     "if (y) for (int j = 0; j < V; ++j) { double s = 0.0; for (int i = 0; i < K; ++i) s += H[i * V + j] * q[i]; y[j] = s; }\n"
     "  for (int i = 0; i < K * V; ++i) H[i] = f * H[i] + (1.0 - f) * Znew[i]; y = NULL;"),
    ("head_groups_interleaved", "n / gk", "n % p->Nk"),
    ("psi_derivative_sign", "d = -alpha * sig * f;", "d = alpha * sig * f;"),
    ("psi_alpha_ignored", "f = exp(-alpha * softplus);", "f = exp(-softplus);"),
    ("bwd_carry_dropped", "G[i * V + j] = C[i * V + j] + qt[i] * dyt[j];", "G[i * V + j] = qt[i] * dyt[j];"),
    ("bwd_gated_path_dropped", "C[i * V + l] = f * G[i * V + l] + s;", "C[i * V + l] = s;"),
    ("bwd_W_not_transposed", "s += dX[i * V + j] * Wn[l * V + j];", "s += dX[i * V + j] * Wn[j * V + l];"),
    ("bwd_tanh_derivative", "(1.0 - Z[e] * Z[e])", "(1.0 - Z[e])"),
    ("bwd_df_sign", "df += G[e] * (Hprev[e] - Z[e]);", "df += G[e] * (Z[e] - Hprev[e]);"),
    ("bwd_dW_wrong_state", "s += Hprev[i * V + l] * dX[i * V + j];", "s += Hcur[i * V + l] * dX[i * V + j];"),
    ("bwd_dq_pre_update", "s += Hcur[i * V + j] * dyt[j];", "s += Hprev[i * V + j] * dyt[j];"),
    ("bwd_dv_residual_dropped", "if (w_r) s += w_r[(size_t)n * V + j] * dyt[j];", ""),
    ("norm_mean_is_sum", "const double s = 1.0 / sqrt(ss / d + eps);\n    for (int j = 0; j < d; ++j) {\n      const double g = silu ? silu_fn(gt[j], NULL) : gt[j];\n      out",
     "const double s = 1.0 / sqrt(ss + eps);\n    for (int j = 0; j < d; ++j) {\n      const double g = silu ? silu_fn(gt[j], NULL) : gt[j];\n      out"),
    ("norm_weight_dropped", "out[t * d + j] = w[j] * (yt[j] * g) * s;", "out[t * d + j] = (yt[j] * g) * s;"),
    ("norm_silu_is_sigmoid", "return x * sg;", "return sg;"),
    ("norm_bwd_projection_dropped", "const double dx = s * w[j] * dot[j] - r * s * s * s * x / d;", "const double dx = s * w[j] * dot[j];"),
    ("norm_bwd_dg_uses_gate", "dg_in[t * d + j] = dx * yt[j] * dsilu;", "dg_in[t * d + j] = dx * g * dsilu;"),
    ("norm_bwd_dw_without_s", "dw[j] += dot[j] * x * s;", "dw[j] += dot[j] * x;"),
    ("norm_bwd_silu_derivative", "if (dx) *dx = sg * (1.0 + x * (1.0 - sg));", "if (dx) *dx = sg * (1.0 - sg);"),
    ("conv_taps_reversed", "pre += w[c * 4 + s] * conv_in(x, prev, b, T, C, t - 3 + s, c);\n        out", "pre += w[c * 4 + 3 - s] * conv_in(x, prev, b, T, C, t - 3 + s, c);\n        out"),
    ("conv_not_causal", "conv_in(x, prev, b, T, C, t - 3 + s, c);\n        out", "conv_in(x, prev, b, T, C, (t + s < T ? t + s : T - 1), c);\n        out"),
    ("conv_prev_rows_reversed", "prev[((size_t)b * 3 + (3 + t)) * C + c]", "prev[((size_t)b * 3 + (-1 - t)) * C + c]"),
    ("conv_bias_dropped", "double pre = bias ? bias[c] : 0.0;\n        for (int s = 0; s < 4; ++s) pre += w[c * 4 + s] * conv_in(x, prev, b, T, C, t - 3 + s, c);\n        out",
     "double pre = 0.0;\n        for (int s = 0; s < 4; ++s) pre += w[c * 4 + s] * conv_in(x, prev, b, T, C, t - 3 + s, c);\n        out"),
    ("conv_bwd_silu_slope_dropped", "const double dpre = dout[((size_t)b * T + t) * C + c] * dsilu;", "const double dpre = dout[((size_t)b * T + t) * C + c];"),
    ("conv_bwd_dx_wrong_tap", "dx[((size_t)b * T + ts) * C + c] += w[c * 4 + s] * dpre;", "dx[((size_t)b * T + ts) * C + c] += w[c * 4 + 3 - s] * dpre;"),
    ("conv_bwd_dw_uses_current_token", "dw[c * 4 + s] += dpre * conv_in(x, prev, b, T, C, ts, c);", "dw[c * 4 + s] += dpre * conv_in(x, prev, b, T, C, t, c);"),
    ("bwd_dh0_seed_ignored", "if (d_hT) memcpy(C, d_hT + bn * KV, sizeof(double) * KV);\n      else memset", "memset"),
]

PIN_CALLS = [
    pins.test_t1_by_hand, pins.test_closed_form_w_zero, pins.test_trivial_gates,
    pins.test_elman_reduction_matches_torch_rnn, pins.test_scalar_chain, pins.test_state_bound,
    pins.test_symmetries, pins.test_multi_value_equals_broadcast, pins.test_chaining,
    pins.test_gate_modes, pins.test_bwd_last_step_matches_algorithm2, pins.test_bwd_matches_autograd,
    functools.partial(pins.test_bwd_matches_finite_differences, gate_kind=2, shared=True),
    pins.test_gated_norm_by_hand, pins.test_gated_norm_invariants, pins.test_gated_norm_bwd_matches_autograd,
    functools.partial(pins.test_gated_norm_bwd_matches_finite_differences, silu=True),
    pins.test_conv_silu_by_hand, pins.test_conv_silu_matches_torch_and_is_causal, pins.test_conv_silu_bwd_matches_autograd,
    pins.test_conv_silu_bwd_matches_finite_differences,
]


def _proxy(oracle, lib):
    ns = types.SimpleNamespace()
    for name in ("fwd", "bwd", "decode_step", "gate_fn", "gated_norm_fwd", "gated_norm_bwd", "conv_silu_fwd", "conv_silu_bwd"):
        setattr(ns, name, functools.partial(getattr(oracle, name), lib=lib))
    return ns


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_every_mutant_is_caught(oracle, tmp_path, name, old, new):
    here = os.path.dirname(oracle.__file__)
    src = open(os.path.join(here, "m2rnn_ref.c")).read()
    assert src.count(old) >= 1, f"mutation site for {name} not found: oracle source changed"
    mutated = tmp_path / "m2rnn_ref.c"
    mutated.write_text(src.replace(old, new))
    shutil.copy(os.path.join(here, "m2rnn_ref.h"), tmp_path / "m2rnn_ref.h")
    lib = oracle.load(oracle.build(force=True, src=str(mutated), out=str(tmp_path / "libmut.so")))
    proxy = _proxy(oracle, lib)
    caught = []
    for call in PIN_CALLS:
        try:
            call(proxy)
        except AssertionError:
            caught.append(getattr(call, "__name__", "finite_differences"))
    assert caught, f"mutant {name} passed every pin"


def test_unmutated_copy_passes(oracle, tmp_path):
    here = os.path.dirname(oracle.__file__)
    for f in ("m2rnn_ref.c", "m2rnn_ref.h"):
        shutil.copy(os.path.join(here, f), tmp_path / f)
    lib = oracle.load(oracle.build(force=True, src=str(tmp_path / "m2rnn_ref.c"), out=str(tmp_path / "libsame.so")))
    for call in PIN_CALLS:
        call(_proxy(oracle, lib))
