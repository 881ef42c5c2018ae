"""Pins of the oracle's SwiGLU + Add pair (Section 6 microbenchmark workload): the library's silu and add in
fp64, closed-form values, and the structure of the operator (gate half first, element-wise, row-independent)."""
import numpy as np
import torch

import oracle


def test_matches_torch_silu_and_add_in_fp64():
    g = torch.Generator().manual_seed(5)
    M, C = 37, 48
    x = torch.randn(M, 2 * C, generator=g, dtype=torch.float64) * 3
    r = torch.randn(M, C, generator=g, dtype=torch.float64)
    s, z = oracle.swiglu_add(x, r)
    want_s = torch.nn.functional.silu(x[:, :C]) * x[:, C:]
    np.testing.assert_allclose(s, want_s.numpy(), rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(z, (want_s + r).numpy(), rtol=1e-13, atol=1e-15)


def test_closed_form_values_and_operand_roles():
    # silu(0) = 0, silu(ln 3) = ln 3 * 3/4; the gate is the FIRST half (swapping the halves must change the result)
    ln3 = np.log(3.0)
    x = np.array([[0.0, ln3, 2.0, 5.0]])          # gate = (0, ln 3), up = (2, 5)
    r = np.array([[10.0, -1.0]])
    s, z = oracle.swiglu_add(x, r)
    np.testing.assert_allclose(s, [[0.0, ln3 * 0.75 * 5.0]], rtol=1e-15)
    np.testing.assert_allclose(z, [[10.0, ln3 * 0.75 * 5.0 - 1.0]], rtol=1e-15)
    s2, _ = oracle.swiglu_add(x[:, [2, 3, 0, 1]], r)
    assert not np.allclose(s, s2)
    # large negative gate -> 0, large positive gate -> gate * up
    s3, _ = oracle.swiglu_add(np.array([[-50.0, 50.0, 3.0, 3.0]]), np.zeros((1, 2)))
    np.testing.assert_allclose(s3, [[0.0, 150.0]], atol=1e-18 * 0 + 1e-19, rtol=1e-15)


def test_rows_and_columns_are_independent():
    g = torch.Generator().manual_seed(6)
    x = torch.randn(8, 16, generator=g, dtype=torch.float64)
    r = torch.randn(8, 8, generator=g, dtype=torch.float64)
    s, z = oracle.swiglu_add(x, r)
    perm = torch.randperm(8, generator=g)
    s_p, z_p = oracle.swiglu_add(x[perm], r[perm])
    np.testing.assert_array_equal(s_p, s[perm.numpy()])
    np.testing.assert_array_equal(z_p, z[perm.numpy()])
    x2 = x.clone(); x2[3, 2] += 1.0                 # touches only element (3, 2)
    s2, _ = oracle.swiglu_add(x2, r)
    diff = (s2 != s)
    assert diff.sum() == 1 and diff[3, 2]
