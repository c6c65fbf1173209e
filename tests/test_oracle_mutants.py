"""Plant one plausible mistake at a time in a COPY of the oracle's C source (on
the CPU, in a temp dir) and check that the pin suite notices every one of them.
This is what justifies trusting the pins: a dropped term, a wrong sign, a
swapped operand or a shifted index each fail at least one pin."""

import os
import subprocess

import pytest

import oracle
from oracle.build import SRC
import pins

MUTANTS = {
    "drop_skip_term": ("y += (L->Dskip ? L->Dskip[d] : 0.0) * u;", ""),
    "decay_sign": ("exp(delta * L->A[(size_t)d * N + n]) * h[n]", "exp(-delta * L->A[(size_t)d * N + n]) * h[n]"),
    "input_without_delta": ("+ delta * Bt[n] * u;", "+ Bt[n] * u;"),
    "swap_B_C": ("+ delta * Bt[n] * u;\n        y += Ct[n] * h[n];", "+ delta * Ct[n] * u;\n        y += Bt[n] * h[n];"),
    "taps_reversed": ("acc += L->conv_w[(size_t)d * W + k] * win[k];", "acc += L->conv_w[(size_t)d * W + (W - 2 - k)] * win[k];"),
    "current_tap_wrong": ("acc += L->conv_w[(size_t)d * W + (W - 1)] * x;", "acc += L->conv_w[(size_t)d * W + 0] * x;"),
    "window_not_shifted": ("for (int k = 0; k + 1 < W - 1; ++k) win[k] = win[k + 1];", ""),
    "softplus_is_exp": ("double mdo_softplus(double v) { return log1p(exp(v)); }", "double mdo_softplus(double v) { return exp(v); }"),
    "silu_is_sigmoid": ("double mdo_silu(double v) { return v / (1.0 + exp(-v)); }", "double mdo_silu(double v) { return 1.0 / (1.0 + exp(-v)); }"),
    "dt_bias_dropped": ("double v = dt + (L->dt_bias ? L->dt_bias[d] : 0.0);", "double v = dt;"),
    "conv_bias_dropped": ("double acc = L->conv_b ? L->conv_b[d] : 0.0;", "double acc = 0.0;"),
    "h_init_ignored": ("h[n] = h_init ? h_init[((size_t)s * D + d) * N + n] : 0.0;", "h[n] = 0.0;"),
    "conv_init_ignored": ("win[k] = conv_init ? conv_init[((size_t)s * (W - 1) + k) * D + d] : 0.0;", "win[k] = 0.0;"),
    "state_not_reset_between_sequences": ("const int t0 = cu_seqlens[s], t1 = cu_seqlens[s + 1];", "const int t0 = cu_seqlens[s], t1 = cu_seqlens[s + 1]; h_init = (s > 0) ? NULL : h_init;"),
    "tree_uses_wrong_parent": ("for (int a = v; a >= 0; a = parent[a]) path[len++] = a;", "for (int a = v; a >= 0; a = (a > 0 ? a - 1 : -1)) path[len++] = a;"),
    "tree_ignores_committed_state": ("h[n] = h0 ? h0[(size_t)d * N + n] : 0.0;", "h[n] = 0.0;"),
    "gate_missing": ("return y * mdo_silu(z);", "return y;"),
    "state_transposed_A": ("exp(delta * L->A[(size_t)d * N + n])", "exp(delta * L->A[(size_t)n * L->d_inner + d < (size_t)L->d_inner * N ? (size_t)n * L->d_inner + d : 0])"),
    "proj_from_raw_input": ("acc += Wx[(size_t)r * D + d] * u[d];", "acc += Wx[(size_t)r * D + d] * x[a * D + d];"),
    "proj_Wx_transposed": ("acc += Wx[(size_t)r * D + d] * u[d];", "acc += Wx[(size_t)d * (R + 2 * N) + r] * u[d];"),
    "proj_Wdt_transposed": ("acc += Wdt[(size_t)d * R + r] * s[r];", "acc += Wdt[(size_t)r * D + d] * s[r];"),
    "proj_B_C_swapped": ("dt[d], s + R, s + R + N);", "dt[d], s + R + N, s + R);"),
    "proj_dt_reads_B_rows": ("for (int r = 0; r < R; ++r) acc += Wdt[(size_t)d * R + r] * s[r];", "for (int r = 0; r < R; ++r) acc += Wdt[(size_t)d * R + r] * s[r + 1];"),
    "proj_sum_drops_last_channel": ("for (int d = 0; d < D; ++d) acc += Wx[(size_t)r * D + d] * u[d];", "for (int d = 0; d + 1 < D; ++d) acc += Wx[(size_t)r * D + d] * u[d];"),
    "proj_ignores_committed_state": ("h[(size_t)d * N + n] = h0 ? h0[(size_t)d * N + n] : 0.0;", "h[(size_t)d * N + n] = 0.0;"),
    "proj_ignores_committed_window": ("win[(size_t)d * (W - 1) + k] = conv0 ? conv0[(size_t)k * D + d] : 0.0;", "win[(size_t)d * (W - 1) + k] = 0.0;"),
    "ssd_head_of_channel_wrong": ("const int N = L->d_state, W = L->d_conv, j = d / L->headdim;", "const int N = L->d_state, W = L->d_conv, j = d % (L->d_inner / L->headdim);"),
    "ssd_dt_read_per_channel": ("dt[(size_t)t * H + d / L->headdim], B + (size_t)t * N, C + (size_t)t * N);", "dt[(size_t)t * H + d % H], B + (size_t)t * N, C + (size_t)t * N);"),
    "ssd_decay_without_delta": ("double decay = exp(delta * L->A[j]);", "double decay = exp(L->A[j]);"),
    "ssd_bias_per_channel": ("double v = dt + (L->dt_bias ? L->dt_bias[j] : 0.0);", "double v = dt + (L->dt_bias ? L->dt_bias[d % (L->d_inner / L->headdim)] : 0.0);"),
    "ssd_tree_reads_dt_of_wrong_node": ("dt[a * H + d / L->headdim], B + a * N, C + a * N);", "dt[(size_t)v * H + d / L->headdim], B + a * N, C + a * N);"),
    "delta_softplus_skipped": ("(L->flags & MDO_DT_SOFTPLUS) ? mdo_softplus(v) : v;", "v;"),
}


def _build_mutant(tmp_path, name, old, new):
    text = open(SRC).read()
    assert text.count(old) >= 1, f"mutant {name}: pattern not found in the oracle source"
    src = tmp_path / f"{name}.c"
    src.write_text(text.replace(old, new))
    out = tmp_path / f"lib_{name}.so"
    subprocess.run(["gcc", "-O1", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-w", "-o", str(out), str(src), "-lm"], check=True)
    return oracle.lib(str(out))


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_mutant_is_caught(tmp_path, name):
    old, new = MUTANTS[name]
    L = _build_mutant(tmp_path, name, old, new)
    caught = []
    for pin in pins.ALL_PINS:
        try:
            pin(L)
        except AssertionError:
            caught.append(pin.__name__)
    assert caught, f"no pin notices the planted mistake {name!r}"
