"""Plants mistakes in copies of the oracle's C source (on the CPU) and checks that the pins of
test_oracle_pins.py notice each one: a dropped term, a wrong sign, a wrong index, a misplaced
temperature, a leaking mask, a transposed operand."""
import ctypes
import os
import subprocess
import types

import numpy as np
import pytest

import test_oracle_pins as pins
import test_oracle_variants as vpins
import test_oracle_distance as dpins

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = open(os.path.join(ROOT, "oracle", "gc_oracle.c")).read()

MUTANTS = {
    "one-hot term dropped": ("double onehot = (j == pos_idx[i]) ? 1.0 : 0.0;", "double onehot = 0.0;"),
    "wrong sign of one-hot": ("row[j] = (p - onehot) / (double)B;", "row[j] = (p + onehot) / (double)B;"),
    "1/B missing": ("row[j] = (p - onehot) / (double)B;", "row[j] = (p - onehot);"),
    "dQ not divided by tau": ("for (int64_t k = 0; k < d; ++k) out[k] /= tau;\n            }\n        }\n        if (dP)",
                              "}\n        }\n        if (dP)"),
    "logits not divided by tau": ("S_row[j] = acc / tau;", "S_row[j] = acc;"),
    "mask leaks into denominator": ("if (allowed(mask_mode, i, j)) sum += exp(S_row[j] - m);", "sum += exp(S_row[j] - m);"),
    "dP uses wrong query row": ("const double* q = Q + i * d;\n                    for (int64_t k = 0; k < d; ++k) out[k] += g * q[k];",
                                "const double* q = Q + ((i + 1) % B) * d;\n                    for (int64_t k = 0; k < d; ++k) out[k] += g * q[k];"),
    "G read transposed in dP": ("double g = G[i * N + j];\n                    const double* q", "double g = G[(j % B) * N + (i % N)];\n                    const double* q"),
    "positive index off by one": ("total += lse[i] - S[i * N + pos_idx[i]];", "total += lse[i] - S[i * N + (pos_idx[i] + 1) % N];"),
    "max instead of logsumexp": ("return m + log(sum);", "return m;"),
    "query_rows: dQ rows not divided by tau": (
        "for (int64_t k = 0; k < d; ++k) out[k] /= tau;\n            }\n        }\n        free(S_row);",
        "}\n        }\n        free(S_row);"),
    "query_rows: one-hot on the wrong column": (
        "double g = (p - ((j == pos_idx[i]) ? 1.0 : 0.0)) / (double)B;\n                    const double* pj",
        "double g = (p - ((j == (pos_idx[i] + 1) % N) ? 1.0 : 0.0)) / (double)B;\n                    const double* pj"),
    "query_rows: lse of the wrong row": (
        "double lse = lse_row(S_row, i, N, mask_mode);", "double lse = lse_row(S_row, (i + 1) % B, N, mask_mode);"),
    "passage_rows: row_lse read at the wrong index": (
        "double p = allowed(mask_mode, i, j) ? exp(s - row_lse[i]) : 0.0;",
        "double p = allowed(mask_mode, i, j) ? exp(s - row_lse[(i + 1) % B]) : 0.0;"),
    "passage_rows: mask leaks": (
        "double p = allowed(mask_mode, i, j) ? exp(s - row_lse[i]) : 0.0;", "double p = exp(s - row_lse[i]);"),
    "passage_rows: logits not divided by tau": ("s /= tau;", ""),
    "passage_rows: one-hot dropped": (
        "double g = (p - ((j == pos_idx[i]) ? 1.0 : 0.0)) / (double)B;\n            for",
        "double g = p / (double)B;\n            for"),
    "variant: 1/|R_i| missing in G": (
        "G[i * N + pos_list[a]] -= 1.0 / ((double)np * (double)B);",
        "G[i * N + pos_list[a]] -= 1.0 / (double)B;"),
    "variant: 1/|R_i| missing in the loss": (
        "total += (lse - S[i * N + pos_list[a]]) / (double)np;", "total += (lse - S[i * N + pos_list[a]]);"),
    "variant: projection dropped from the cosine Jacobian": (
        "dQ[i * d + k] = cosine ? (gQ[i * d + k] - Qn[i * d + k] * dot) / qnorm[i]",
        "dQ[i * d + k] = cosine ? gQ[i * d + k] / qnorm[i]"),
    "variant: 1/|p| dropped from the cosine Jacobian": (
        "dP[j * d + k] = cosine ? (gP[j * d + k] - Pn[j * d + k] * dot) / pnorm[j]",
        "dP[j * d + k] = cosine ? (gP[j * d + k] - Pn[j * d + k] * dot)"),
    "variant: wrong sign of dtau": ("*dtau = -s / tau;", "*dtau = s / tau;"),
    "variant: dtau without 1/tau": ("*dtau = -s / tau;", "*dtau = -s;"),
    "variant: halves not averaged": ("for (int64_t e = 0; e < B * N; ++e) G[e] *= 0.5;", ""),
    "variant: column softmax minus one at the wrong query": (
        "G[i * N + j] -= 1.0 / (double)B;\n        }\n        L = 0.5",
        "G[((i + 1) % B) * N + j] -= 1.0 / (double)B;\n        }\n        L = 0.5"),
    "variant: column logsumexp ignores the mask": (
        "if (allowed(mask_mode, k, j)) sum += exp(S[k * N + j] - m);", "sum += exp(S[k * N + j] - m);"),
    "distance cache: 1/tau missing in w": (
        "W[i * N + j] = (p - ((j == pos_idx[i]) ? 1.0 : 0.0)) / ((double)B * tau);",
        "W[i * N + j] = (p - ((j == pos_idx[i]) ? 1.0 : 0.0)) / (double)B;"),
    "distance cache: mask leaks into w": (
        "double p = allowed(mask_mode, i, j) ? exp(D[i * N + j] / tau - lse[i]) : 0.0;",
        "double p = exp(D[i * N + j] / tau - lse[i]);"),
    "distance cache: positive distance not scaled by tau": (
        "total += lse - D[i * N + pos_idx[i]] / tau;", "total += lse - D[i * N + pos_idx[i]];"),
    "cache_apply reads U transposed": ("s += U[i * d + a] * X[i * d_in + b];",
                                       "s += U[(a % rows) * d + (i % d)] * X[i * d_in + b];"),
    "cache_apply overwrites instead of accumulating": ("if (accumulate) dW[a * d_in + b] += s;",
                                                       "if (accumulate) dW[a * d_in + b] = s;"),
}


def _build_mutant(tmp_path, name, old, new):
    assert old in SRC, f"mutation site for '{name}' not found"
    path = tmp_path / "mutant.c"
    path.write_text(SRC.replace(old, new, 1))
    lib = tmp_path / "libmutant.so"
    subprocess.run(["gcc", "-O1", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", str(lib), str(path),
                    "-lm"], check=True)
    return str(lib)


def _wrap(libpath):
    """An object with the interface of the `oracle` package, backed by the mutant library."""
    import oracle as real
    lib = ctypes.CDLL(libpath)
    dp = ctypes.POINTER(ctypes.c_double)
    lib.gco_build_cache.restype = ctypes.c_int
    lib.gco_build_cache.argtypes = [dp, dp, ctypes.POINTER(ctypes.c_int32), ctypes.c_int64,
                                    ctypes.c_int64, ctypes.c_int64, ctypes.c_double, ctypes.c_int,
                                    dp, dp, dp, dp, dp]

    def build_cache(Q, P, pos_idx, tau=1.0, mask_mode=0, grads=True):
        Q, P, pos = real._prep(Q, P, pos_idx)
        B, d = Q.shape
        N = P.shape[0]
        loss = ctypes.c_double(0.0)
        lse, pl = np.empty(B), np.empty(B)
        dQ, dP = np.empty((B, d)), np.empty((N, d))
        rc = lib.gco_build_cache(real._ptr(Q, ctypes.c_double), real._ptr(P, ctypes.c_double),
                                 real._ptr(pos, ctypes.c_int32), B, N, d, float(tau), int(mask_mode),
                                 ctypes.byref(loss), real._ptr(lse, ctypes.c_double),
                                 real._ptr(pl, ctypes.c_double), real._ptr(dQ, ctypes.c_double),
                                 real._ptr(dP, ctypes.c_double))
        if rc != 0:
            raise ValueError(f"rejected ({rc})")
        return dict(loss=float(loss.value), row_lse=lse, pos_logit=pl, dQ=dQ, dP=dP)

    ip = ctypes.POINTER(ctypes.c_int32)
    lp = ctypes.POINTER(ctypes.c_int64)
    i64 = ctypes.c_int64
    lib.gco_query_rows.restype = ctypes.c_int
    lib.gco_query_rows.argtypes = [dp, dp, ip, i64, i64, i64, ctypes.c_double, ctypes.c_int, lp, i64,
                                   dp, dp, dp]
    lib.gco_passage_rows.restype = ctypes.c_int
    lib.gco_passage_rows.argtypes = [dp, dp, ip, i64, i64, i64, ctypes.c_double, ctypes.c_int, dp, lp,
                                     i64, dp]

    def query_rows(Q, P, pos_idx, rows, tau=1.0, mask_mode=0, grads=True):
        Q, P, pos = real._prep(Q, P, pos_idx)
        B, d = Q.shape
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        n = rows.shape[0]
        lse, pl, dQ = np.empty(n), np.empty(n), np.empty((n, d))
        rc = lib.gco_query_rows(real._ptr(Q, ctypes.c_double), real._ptr(P, ctypes.c_double),
                                real._ptr(pos, ctypes.c_int32), B, P.shape[0], d, float(tau),
                                int(mask_mode), real._ptr(rows, ctypes.c_int64), n,
                                real._ptr(lse, ctypes.c_double), real._ptr(pl, ctypes.c_double),
                                real._ptr(dQ, ctypes.c_double))
        if rc != 0:
            raise ValueError(f"rejected ({rc})")
        return dict(row_lse=lse, pos_logit=pl, dQ=dQ)

    def passage_rows(Q, P, pos_idx, row_lse, rows, tau=1.0, mask_mode=0):
        Q, P, pos = real._prep(Q, P, pos_idx)
        B, d = Q.shape
        lse = real._f64(row_lse)
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        n = rows.shape[0]
        dP = np.empty((n, d))
        rc = lib.gco_passage_rows(real._ptr(Q, ctypes.c_double), real._ptr(P, ctypes.c_double),
                                  real._ptr(pos, ctypes.c_int32), B, P.shape[0], d, float(tau),
                                  int(mask_mode), real._ptr(lse, ctypes.c_double),
                                  real._ptr(rows, ctypes.c_int64), n, real._ptr(dP, ctypes.c_double))
        if rc != 0:
            raise ValueError(f"rejected ({rc})")
        return dP

    lib.gco_build_variant.restype = ctypes.c_int
    lib.gco_build_variant.argtypes = [dp, dp, lp, ip, i64, i64, i64, ctypes.c_double, ctypes.c_int,
                                      ctypes.c_int, ctypes.c_int, dp, dp, dp, dp]

    def build_variant(Q, P, positives, tau=1.0, mask_mode=0, cosine=False, two_direction=False):
        Q, P = real._f64(Q), real._f64(P)
        B, d = Q.shape
        N = P.shape[0]
        if isinstance(positives, np.ndarray) and positives.ndim == 1:
            lists = [[int(v)] for v in positives]
        else:
            lists = [[int(v) for v in row] for row in positives]
        ptr = np.zeros(B + 1, np.int64)
        ptr[1:] = np.cumsum([len(r) for r in lists])
        flat = np.ascontiguousarray([v for r in lists for v in r], dtype=np.int32)
        loss, dtau = ctypes.c_double(0.0), ctypes.c_double(0.0)
        dQ, dP = np.empty((B, d)), np.empty((N, d))
        rc = lib.gco_build_variant(real._ptr(Q, ctypes.c_double), real._ptr(P, ctypes.c_double),
                                   real._ptr(ptr, ctypes.c_int64), real._ptr(flat, ctypes.c_int32), B,
                                   N, d, float(tau), int(mask_mode), int(bool(cosine)),
                                   int(bool(two_direction)), ctypes.byref(loss),
                                   real._ptr(dQ, ctypes.c_double), real._ptr(dP, ctypes.c_double),
                                   ctypes.byref(dtau))
        if rc != 0:
            raise ValueError(f"rejected ({rc})")
        return dict(loss=float(loss.value), dQ=dQ, dP=dP, dtau=float(dtau.value))

    lib.gco_dist_loss.restype = ctypes.c_int
    lib.gco_dist_loss.argtypes = [dp, ip, i64, i64, ctypes.c_double, ctypes.c_int, dp, dp]
    lib.gco_dist_w.restype = ctypes.c_int
    lib.gco_dist_w.argtypes = [dp, ip, i64, i64, ctypes.c_double, ctypes.c_int, dp]

    def dist_loss(D, pos_idx, tau=1.0, mask_mode=0):
        D = real._f64(D)
        B, N = D.shape
        pos = np.ascontiguousarray(pos_idx, dtype=np.int32)
        loss = ctypes.c_double(0.0)
        lse = np.empty(B)
        rc = lib.gco_dist_loss(real._ptr(D, ctypes.c_double), real._ptr(pos, ctypes.c_int32), B, N,
                               float(tau), int(mask_mode), ctypes.byref(loss),
                               real._ptr(lse, ctypes.c_double))
        if rc != 0:
            raise ValueError(f"rejected ({rc})")
        return dict(loss=float(loss.value), row_lse=lse)

    def dist_w(D, pos_idx, tau=1.0, mask_mode=0):
        D = real._f64(D)
        B, N = D.shape
        pos = np.ascontiguousarray(pos_idx, dtype=np.int32)
        W = np.empty((B, N))
        rc = lib.gco_dist_w(real._ptr(D, ctypes.c_double), real._ptr(pos, ctypes.c_int32), B, N,
                            float(tau), int(mask_mode), real._ptr(W, ctypes.c_double))
        if rc != 0:
            raise ValueError(f"rejected ({rc})")
        return W

    lib.gco_cache_apply.restype = ctypes.c_int
    lib.gco_cache_apply.argtypes = [dp, dp, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                                    ctypes.c_int, dp]

    def cache_apply(U, X, dW=None):
        U, X = real._f64(U), real._f64(X)
        rows, d = U.shape
        d_in = X.shape[1]
        acc = dW is not None
        if not acc:
            dW = np.empty((d, d_in))
        rc = lib.gco_cache_apply(real._ptr(U, ctypes.c_double), real._ptr(X, ctypes.c_double), rows,
                                 d, d_in, int(acc), real._ptr(dW, ctypes.c_double))
        if rc != 0:
            raise ValueError(f"rejected ({rc})")
        return dW

    return types.SimpleNamespace(
        build_cache=build_cache, cache_apply=cache_apply, query_rows=query_rows,
        passage_rows=passage_rows, build_variant=build_variant, dist_loss=dist_loss, dist_w=dist_w,
        loss_only=lambda Q, P, pos, tau=1.0, mask=0: build_cache(Q, P, pos, tau, mask)["loss"])


def _pins(o):
    yield lambda: pins.test_hand_worked_rational_example(o)
    yield lambda: pins.test_gradients_match_finite_differences(o, 0.1, 1, (4, 8, 5))
    yield lambda: pins.test_gradients_match_finite_differences(o, 1.0, 0, (3, 6, 4))
    yield lambda: pins.test_rows_of_G_sum_to_zero(o, 1)
    yield lambda: pins.test_identical_representations(o, 0.25)
    yield lambda: pins.test_one_query_two_passages_is_logistic_loss(o)
    yield lambda: pins.test_scale_and_permutation_symmetry(o)
    yield lambda: pins.test_duplicate_positives_sum_in_epsilon(o)
    yield lambda: pins.test_row_sampled_entry_points_on_the_hand_worked_example(o)
    yield lambda: pins.test_row_sampled_entry_points_match_finite_differences(o, 0.1, 1)
    yield lambda: pins.test_row_sampled_entry_points_match_finite_differences(o, 1.0, 0)
    yield lambda: pins.test_row_sampled_entry_points_identical_representations(o)
    yield lambda: vpins.test_variant_gradients_match_finite_differences(o, True, False, 1, 0.2)
    yield lambda: vpins.test_variant_gradients_match_finite_differences(o, False, True, 1, 0.2)
    yield lambda: vpins.test_euler_identity_for_joint_scaling(o, True)
    yield lambda: vpins.test_cosine_is_scale_invariant_and_gradients_are_tangent(o)
    yield lambda: vpins.test_two_direction_loss_is_symmetric_under_role_swap(o)
    yield lambda: vpins.test_two_positives_hand_worked(o)
    yield lambda: dpins.test_w_is_the_derivative_of_the_loss_in_every_distance(o, 0.3, 1)
    yield lambda: dpins.test_dot_product_links_the_two_caches(o, 1)
    yield lambda: pins.test_cache_apply_hand_worked_example(o)
    yield lambda: pins.test_cache_apply_chunks_reproduce_full_batch_parameter_gradient(o)


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_pins_catch_planted_mistake(tmp_path, name):
    old, new = MUTANTS[name]
    mutant = _wrap(_build_mutant(tmp_path, name, old, new))
    caught = 0
    for pin in _pins(mutant):
        try:
            pin()
        except (AssertionError, ValueError):
            caught += 1
    assert caught >= 1, f"no pin noticed: {name}"


def test_unmutated_source_passes_the_same_pins(tmp_path):
    path = tmp_path / "same.c"
    path.write_text(SRC)
    lib = tmp_path / "libsame.so"
    subprocess.run(["gcc", "-O1", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", str(lib), str(path),
                    "-lm"], check=True)
    for pin in _pins(_wrap(str(lib))):
        pin()
