"""Pins for the oracle's attention (Eq. 3) and its derivative: brute force in pure Python, special cases with
known answers, a library routine, finite differences."""
import math

import numpy as np
import pytest
import torch

import oracle


def brute_attention(q, k, v, sel, scale):
    """Eq. 3 with Python loops over one (b, h) problem at a time."""
    B, N, H, D = q.shape
    Ns = len(sel)
    o = np.zeros((B, Ns, H, D))
    lse = np.zeros((B, H, Ns))
    for b in range(B):
        for h in range(H):
            for i in range(Ns):
                s = [sum(q[b, sel[i], h, d] * k[b, sel[j], h, d] for d in range(D)) * scale for j in range(Ns)]
                e = [math.exp(x) for x in s]
                z = sum(e)
                for d in range(D):
                    o[b, i, h, d] = sum(e[j] / z * v[b, sel[j], h, d] for j in range(Ns))
                lse[b, h, i] = math.log(z)
    return o, lse


def rand_qkv(B, N, H, D, seed, std=1.0):
    rng = np.random.default_rng(seed)
    return [rng.normal(0, std, size=(B, N, H, D)) for _ in range(3)]


@pytest.mark.parametrize("sel", [None, [0, 2, 3, 6], [5]])
def test_forward_matches_brute_force(sel):
    q, k, v = rand_qkv(2, 7, 2, 4, seed=1)
    s = list(range(7)) if sel is None else sel
    o, lse = oracle.attn_fwd(q, k, v, sel)
    bo, bl = brute_attention(q, k, v, s, 0.5)
    np.testing.assert_allclose(o, bo, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(lse, bl, rtol=1e-12, atol=1e-14)


def test_single_token_returns_its_value():
    q, k, v = rand_qkv(2, 5, 3, 8, seed=2)
    o, lse = oracle.attn_fwd(q, k, v, [3])
    np.testing.assert_allclose(o[:, 0], v[:, 3], rtol=1e-14)
    np.testing.assert_allclose(lse[:, :, 0], (q[:, 3] * k[:, 3]).sum(-1) / math.sqrt(8), rtol=1e-13)


def test_equal_keys_average_the_values():
    q, k, v = rand_qkv(1, 6, 2, 4, seed=3)
    k[:] = k[:, :1]
    o, _ = oracle.attn_fwd(q, k, v)
    np.testing.assert_allclose(o, np.broadcast_to(v.mean(axis=1, keepdims=True), o.shape), rtol=1e-13)


def test_token_permutation_equivariance():
    q, k, v = rand_qkv(2, 9, 2, 8, seed=4)
    perm = np.random.default_rng(0).permutation(9)
    o, lse = oracle.attn_fwd(q, k, v)
    op, lsep = oracle.attn_fwd(q[:, perm], k[:, perm], v[:, perm])
    np.testing.assert_allclose(op, o[:, perm], rtol=1e-12)
    np.testing.assert_allclose(lsep, lse[:, :, perm], rtol=1e-12)


def test_large_scores_do_not_overflow():
    q, k, v = rand_qkv(1, 4, 1, 4, seed=5, std=40.0)
    o, lse = oracle.attn_fwd(q, k, v)
    assert np.all(np.isfinite(o)) and np.all(np.isfinite(lse))


def test_forward_matches_library_sdpa():
    q, k, v = rand_qkv(2, 33, 3, 16, seed=6)
    sel = np.array([0, 1, 4, 9, 10, 17, 30, 32], dtype=np.int32)
    o, _ = oracle.attn_fwd(q, k, v, sel)
    tq, tk, tv = (torch.from_numpy(a[:, sel]).permute(0, 2, 1, 3) for a in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).permute(0, 2, 1, 3).numpy()
    np.testing.assert_allclose(o, ref, rtol=1e-10, atol=1e-12)


def test_backward_matches_finite_differences():
    B, N, H, D = 1, 6, 2, 3
    q, k, v = rand_qkv(B, N, H, D, seed=7)
    sel = np.array([0, 2, 3, 5], dtype=np.int32)
    rng = np.random.default_rng(8)
    d_o = rng.normal(size=(B, len(sel), H, D))
    dq, dk, dv = oracle.attn_bwd(q, k, v, d_o, sel)

    def loss(qq, kk, vv):
        o, _ = oracle.attn_fwd(qq, kk, vv, sel)
        return float((o * d_o).sum())

    eps = 1e-6
    for arr, grad, which in ((q, dq, 0), (k, dk, 1), (v, dv, 2)):
        for idx in np.ndindex(arr.shape):
            args = [q.copy(), k.copy(), v.copy()]
            args[which][idx] += eps
            up = loss(*args)
            args[which][idx] -= 2 * eps
            dn = loss(*args)
            fd = (up - dn) / (2 * eps)
            assert abs(fd - grad[idx]) < 1e-6 * max(1.0, abs(fd)), (which, idx, fd, grad[idx])


def test_backward_dropped_rows_are_zero_and_identity_selection_is_full_path():
    B, N, H, D = 2, 11, 2, 8
    q, k, v = rand_qkv(B, N, H, D, seed=9)
    sel = np.array([1, 4, 5, 9], dtype=np.int32)
    d_o = np.random.default_rng(1).normal(size=(B, 4, H, D))
    grads = oracle.attn_bwd(q, k, v, d_o, sel)
    dropped = np.setdiff1d(np.arange(N), sel)
    for g in grads:
        assert np.all(g[:, dropped] == 0.0)
        assert np.any(g[:, sel] != 0.0)
    d_full = np.random.default_rng(2).normal(size=(B, N, H, D))
    a = oracle.attn_bwd(q, k, v, d_full, None)
    b = oracle.attn_bwd(q, k, v, d_full, np.arange(N, dtype=np.int32))
    for x, y in zip(a, b):
        assert np.array_equal(x, y)


def test_backward_matches_library_autograd():
    B, N, H, D = 2, 19, 2, 8
    q, k, v = rand_qkv(B, N, H, D, seed=10)
    sel = np.array([0, 3, 4, 8, 12, 18], dtype=np.int32)
    d_o = np.random.default_rng(3).normal(size=(B, len(sel), H, D))
    dq, dk, dv = oracle.attn_bwd(q, k, v, d_o, sel)
    tq, tk, tv = (torch.from_numpy(a).requires_grad_(True) for a in (q, k, v))
    gq, gk, gv = (t[:, torch.from_numpy(sel).long()].permute(0, 2, 1, 3) for t in (tq, tk, tv))
    o = torch.nn.functional.scaled_dot_product_attention(gq, gk, gv).permute(0, 2, 1, 3)
    o.backward(torch.from_numpy(d_o))
    np.testing.assert_allclose(dq, tq.grad.numpy(), rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(dk, tk.grad.numpy(), rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(dv, tv.grad.numpy(), rtol=1e-9, atol=1e-12)


def test_softmax_gradient_rows_sum_to_zero():
    # sum_j dS_ij = 0  =>  adding a constant vector c to every key leaves ... dQ unchanged is not implied, but
    # the score gradient is shift-free: dK summed over kept tokens equals zero when Q rows are identical.
    B, N, H, D = 1, 8, 1, 4
    q, k, v = rand_qkv(B, N, H, D, seed=11)
    q[:] = q[:, :1]
    d_o = np.random.default_rng(4).normal(size=(B, N, H, D))
    _, dk, _ = oracle.attn_bwd(q, k, v, d_o)
    # dK_j = scale * sum_i dS_ij q_i = scale * q_0 * sum_i dS_ij ; summing over j gives scale*q_0*sum_ij dS_ij = 0
    np.testing.assert_allclose(dk.sum(axis=1), 0.0, atol=1e-13)
