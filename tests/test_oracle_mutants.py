"""Plant one plausible mistake at a time in a copy of the C oracle (on the CPU) and check that at
least one pin notices: a dropped term, a wrong sign, a swapped operand, an off-by-one."""
import os
import subprocess

import pytest

import oracle_pins as pins

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(os.path.dirname(HERE), "oracle", "dad_oracle.c")

# (name, text in dad_oracle.c, replacement)
MUTANTS = [
    ("full_grad_sign", "g[b] += x * d[b];", "g[b] -= x * d[b];"),
    ("full_grad_drops_last_site", "for (int s = 0; s < S; ++s)\n      for (i64 n = 0; n < N; ++n) {", "for (int s = 0; s < S - (S > 1); ++s)\n      for (i64 n = 0; n < N; ++n) {"),
    ("reconstruct_drops_last_row", "for (i64 k = 0; k < K; ++k) {", "for (i64 k = 0; k < K - 1; ++k) {"),
    ("reconstruct_wrong_stride", "const double p = Pcat[k * h_in + a];", "const double p = Pcat[k * h_in + (h_in - 1 - a)];"),
    ("rows_dot_wrong_operand", "acc += X[n * h + c] * F[j * h + c];", "acc += X[n * h + c] * F[j * h + (c + 1) % h];"),
    ("cols_acc_transposed_y", "const double y = Y[n * r + j];", "const double y = Y[(n * r + j + 1) % (N * r)];"),
    ("spi_skips_second_half", "rows_dot(N, h_in, r, A, Z, Y);   /* W = A Z^T  (in Y)  */", "/* skipped */"),
    ("spi_uses_A_for_final", "rows_dot(N, h_out, r, D, Q, Y);\n  cols_acc(N, h_in, r, Y, A, P);", "rows_dot(N, h_out, r, D, Q, Y);\n  cols_acc(N, h_in, r, Y, A, P); for (i64 t = 0; t < r * h_in; ++t) P[t] = -P[t];"),
    ("orth_single_projection_wrong_sign", "for (i64 b = 0; b < h; ++b) v[b] -= c * q[b];", "for (i64 b = 0; b < h; ++b) v[b] += c * q[b];"),
    ("orth_no_normalise", "for (i64 b = 0; b < h; ++b) v[b] /= after;", "for (i64 b = 0; b < h; ++b) v[b] /= 1.0;"),
    ("orth_never_zeroes", "if (before == 0.0 || after <= 1e-12 * before) {", "if (before == 0.0) {"),
    ("sigma_squared", "sigma[j] = norm2(P + j * h_in, h_in);", "sigma[j] = dot(P + j * h_in, P + j * h_in, h_in);"),
    ("sites_share_start_block", "Q0 + (i64)s * r * h_out,", "Q0,"),
    # the peel term and the re-projection both keep the iterate off the found directions; either alone
    # suffices at convergence, so the planted mistake removes the deflation altogether
    ("paper_no_deflation", ["project_out(j, h_out, Q, t);", "for (i64 b = 0; b < h_out; ++b) t[b] -= c * Q[l * h_out + b];"], [";", ";"]),
    ("paper_final_uses_start", "rows_dot(N, h_out, 1, D, g, v);              /* v = D g            */", "rows_dot(N, h_out, 1, D, Q0 + j * h_out, v);"),
    ("bytes_dad_ignores_width", "(uint64_t)(h_in + h_out) * (uint64_t)elem_bytes;", "(uint64_t)(h_in + h_out) * 4u;"),
    ("bytes_rank_product", "return (uint64_t)r * (uint64_t)(h_in + h_out) * 4u;", "return (uint64_t)r * (uint64_t)(h_in * h_out) * 4u;"),
    ("bytes_dsgd_sum", "return (uint64_t)h_in * (uint64_t)h_out * 4u;", "return (uint64_t)(h_in + h_out) * 4u;"),
    ("gram_form_C_not_symmetric_use", "for (i64 n = 0; n < N; ++n) acc += D[n * h_out + b] * C[n * N + m];", "for (i64 n = 0; n < N; ++n) acc += D[n * h_out + b] * C[n * N + (m + 1) % N];"),
    ("gram_form_sigma_without_C", "acc += V[n * r + j] * C[n * N + m] * V[m * r + j];", "acc += (n == m) ? V[n * r + j] * V[m * r + j] : 0.0;"),
    ("gram_form_skips_orth", "        Q[j * h_out + b] = acc;\n      }\n    dad_oracle_orth(r, h_out, Q, NULL);", "        Q[j * h_out + b] = acc;\n      }\n    ;"),
    ("effective_rank_strict", "while (keep < r && sg[keep] > bar) ++keep;", "while (keep < r && sg[keep] >= bar) ++keep;"),
    ("effective_rank_vs_previous", "const float bar = theta * sg[0];\n    int keep = 0;\n    while (keep < r && sg[keep] > bar) ++keep;", "int keep = 0;\n    while (keep < r && (keep == 0 ? sg[0] > theta * sg[0] : sg[keep] > theta * sg[keep - 1])) ++keep;"),
    ("gather_reverses_sites", "Pcat[((i64)s * r + j) * h_in + a] = P[((i64)s * r + j) * h_in + a];", "Pcat[((i64)(S - 1 - s) * r + j) * h_in + a] = P[((i64)s * r + j) * h_in + a];"),
]


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_mutant_is_caught(oracle, tmp_path, name, old, new):
    text = open(SRC).read()
    olds, news = ([old], [new]) if isinstance(old, str) else (old, new)
    mutated = text
    for o_, n_ in zip(olds, news):
        assert mutated.count(o_) >= 1, f"mutation site for {name} not found"
        mutated = mutated.replace(o_, n_, 1)
    c = tmp_path / f"{name}.c"
    so = tmp_path / f"lib{name}.so"
    c.write_text(mutated)
    subprocess.check_call(["gcc", "-O1", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", str(so), str(c), "-lm"])
    caught = []
    with oracle.use_library(str(so)):
        for pin in pins.ALL_PINS:
            try:
                pin(oracle)
            except (AssertionError, ArithmeticError, ValueError):  # numpy's LinAlgError is a ValueError
                caught.append(pin.__name__)
    assert caught, f"no pin notices the planted mistake '{name}'"
