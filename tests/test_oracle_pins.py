"""Pins for the CPU oracle (CPU only).

The paper prints no worked numeric example of k-MIP attention, so the oracle is pinned
to what Eq. 1 / Algorithm 1 and the mathematics fix: hand-derived closed-form cases,
special cases that reduce to library routines (k = n: dense softmax attention; k = 1:
arg-max retrieval), exhaustive subset enumeration on tiny inputs, invariants
(permutation equivariance, CSR confinement, constant V, identical keys), and for the
backward finite differences, autograd over library ops and closed-form identities.
"""
import itertools
import json
import os

import numpy as np
import pytest
import torch

from oracle import kmip_oracle as oracle
from paper_2604_03815_b200 import workloads as wl


def _rand(seed, N, H, d, scale=1.0):
    w = wl.iid_workload("t", seed, [N], H, d, 1, wl.MODE_FP32_EXACT, input_scale=scale)
    return w.Q, w.K, w.V, w.dOut


def _offs(*sizes):
    return np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)


# ----------------------------------------------------------------------------- closed forms
def _load_cases(golden_dir):
    with open(os.path.join(golden_dir, "closed_form_cases.json")) as f:
        return json.load(f)["cases"]


def _arr(x, dtype):
    def conv(v):
        if isinstance(v, list):
            return [conv(u) for u in v]
        return float("-inf") if v == "-inf" else v
    return np.array(conv(x), dtype=dtype)


def test_closed_form_fixtures(golden_dir):
    for case in _load_cases(golden_dir):
        H, d, k = case["H"], case["d"], case["k"]
        Q = _arr(case["Q"], np.float32).reshape(-1, H, d)
        K = _arr(case["K"], np.float32).reshape(-1, H, d)
        V = _arr(case["V"], np.float32).reshape(-1, H, d)
        offs = np.array(case["graph_offsets"], dtype=np.int32)
        r = oracle.forward(Q, K, V, offs, k)
        N = Q.shape[0]
        np.testing.assert_array_equal(r["idx"], _arr(case["idx"], np.int32).reshape(N, H, k), err_msg=case["name"])
        np.testing.assert_array_equal(r["score"], _arr(case["score"], np.float64).reshape(N, H, k), err_msg=case["name"])
        np.testing.assert_allclose(r["out"], _arr(case["out"], np.float64).reshape(N, H, d), rtol=0, atol=1e-14,
                                   err_msg=case["name"])


# ----------------------------------------------------------------------------- k = n : dense attention
@pytest.mark.parametrize("N,H,d", [(37, 2, 8), (64, 3, 16), (5, 1, 3)])
def test_k_equals_n_is_dense_softmax_attention(N, H, d):
    Q, K, V, _ = _rand(11, N, H, d)
    r = oracle.forward(Q, K, V, None, N)
    q, k_, v = (torch.from_numpy(x.astype(np.float64)).permute(1, 0, 2) for x in (Q, K, V))
    ref = torch.nn.functional.scaled_dot_product_attention(q, k_, v).permute(1, 0, 2).numpy()
    np.testing.assert_allclose(r["out"], ref, rtol=1e-12, atol=1e-13)
    # every key is kept exactly once
    assert np.all(np.sort(r["idx"], axis=-1) == np.arange(N)[None, None, :])


# ----------------------------------------------------------------------------- k = 1 : arg-max retrieval
def test_k_equals_1_is_argmax_retrieval():
    N, H, d = 53, 2, 8
    Q, K, V, _ = _rand(12, N, H, d)
    r = oracle.forward(Q, K, V, None, 1)
    S = np.einsum("ihc,jhc->hij", Q.astype(np.float64), K.astype(np.float64))
    am = np.argmax(S, axis=2)                      # [H, N], first maximum = lowest index
    np.testing.assert_array_equal(r["idx"][:, :, 0], am.T)
    for h in range(H):
        np.testing.assert_array_equal(r["out"][:, h, :], V[am[h], h, :].astype(np.float64))


# ----------------------------------------------------------------------------- exhaustive tiny case
@pytest.mark.parametrize("N,k", [(6, 2), (8, 3), (7, 7), (8, 1)])
def test_exhaustive_subsets_tiny(N, k):
    H, d = 2, 4
    Q, K, V, _ = _rand(13 + N, N, H, d)
    r = oracle.forward(Q, K, V, None, k)
    S = np.einsum("ihc,jhc->ihj", Q.astype(np.float64), K.astype(np.float64))
    for i in range(N):
        for h in range(H):
            best = max(itertools.combinations(range(N), k), key=lambda c: sum(S[i, h, j] for j in c))
            assert set(r["idx"][i, h]) == set(best)
            # scores listed in descending order, and they are the true inner products
            sc = r["score"][i, h]
            assert np.all(np.diff(sc) <= 0)
            np.testing.assert_allclose(sc, S[i, h, r["idx"][i, h]], rtol=1e-15)
            z = np.array([S[i, h, j] for j in best]) / np.sqrt(d)
            p = np.exp(z - z.max())
            p /= p.sum()
            ref = sum(p[t] * V[j, h].astype(np.float64) for t, j in enumerate(best))
            np.testing.assert_allclose(r["out"][i, h], ref, rtol=1e-12, atol=1e-14)


def test_matches_sorted_full_row():
    """Selection equals a full lexicographic sort (score desc, index asc) of each row."""
    N, H, d, k = 200, 2, 4, 9
    Q, K, V, _ = _rand(14, N, H, d)
    # few distinct values => many exact ties
    Q = np.round(Q)
    K = np.round(K)
    r = oracle.forward(Q, K, V, None, k)
    S = np.einsum("ihc,jhc->ihj", Q.astype(np.float64), K.astype(np.float64))
    for i in range(0, N, 7):
        for h in range(H):
            order = np.lexsort((np.arange(N), -S[i, h]))[:k]
            np.testing.assert_array_equal(r["idx"][i, h], order)


# ----------------------------------------------------------------------------- invariants
def test_constant_v_gives_v():
    N, H, d = 40, 2, 8
    Q, K, V, _ = _rand(15, N, H, d)
    V[:] = V[0]
    for k in (1, 3, 40):
        r = oracle.forward(Q, K, V, None, k)
        np.testing.assert_allclose(r["out"], np.broadcast_to(V[0].astype(np.float64), (N, H, d)), rtol=1e-14)


def test_identical_keys_tie_break_and_uniform_weights():
    N, H, d, k = 20, 2, 4, 5
    Q, K, V, _ = _rand(16, N, H, d)
    K[:] = K[3]
    offs = _offs(12, 8)
    r = oracle.forward(Q, K, V, offs, k)
    for i in range(N):
        lo = 0 if i < 12 else 12
        np.testing.assert_array_equal(r["idx"][i], np.tile(np.arange(lo, lo + k), (H, 1)))
        np.testing.assert_allclose(r["out"][i], V[lo:lo + k].astype(np.float64).mean(axis=0), rtol=1e-13)


def test_permutation_equivariance():
    N, H, d, k = 60, 2, 8, 6
    Q, K, V, _ = _rand(17, N, H, d)
    rng = np.random.default_rng(0)
    perm = rng.permutation(N)                 # new row r holds old row perm[r]
    inv = np.argsort(perm)
    a = oracle.forward(Q, K, V, None, k)
    b = oracle.forward(Q[perm], K[perm], V[perm], None, k)
    assert a["gap"].min() > 1e-9              # tie-free, so the claim is well posed
    # the oracle sums d products in index order; a row permutation leaves each sum unchanged
    np.testing.assert_array_equal(b["score"], a["score"][perm])
    np.testing.assert_array_equal(b["idx"], inv[a["idx"][perm]])
    np.testing.assert_allclose(b["out"], a["out"][perm], rtol=1e-13, atol=1e-15)


def test_csr_confinement_and_padding():
    H, d, k = 2, 4, 5
    sizes = [9, 3, 0, 17]
    N = sum(sizes)
    Q, K, V, _ = _rand(18, N, H, d)
    offs = _offs(*sizes)
    r = oracle.forward(Q, K, V, offs, k)
    for g, n in enumerate(sizes):
        lo, hi = offs[g], offs[g + 1]
        if n == 0:
            continue
        alone = oracle.forward(Q[lo:hi], K[lo:hi], V[lo:hi], None, k)
        shifted = np.where(alone["idx"] >= 0, alone["idx"] + lo, -1)
        np.testing.assert_array_equal(r["idx"][lo:hi], shifted)
        np.testing.assert_array_equal(r["score"][lo:hi], alone["score"])
        np.testing.assert_array_equal(r["out"][lo:hi], alone["out"])
    # the 3-node graph keeps all 3 keys and pads two slots
    assert np.all(r["idx"][9:12, :, 3:] == -1) and np.all(np.isinf(r["score"][9:12, :, 3:]))
    assert np.all(r["idx"][9:12, :, :3] >= 9) and np.all(r["idx"][9:12, :, :3] < 12)


def test_rows_subset_matches_full():
    N, H, d, k = 50, 2, 8, 4
    Q, K, V, _ = _rand(19, N, H, d)
    offs = _offs(20, 30)
    full = oracle.forward(Q, K, V, offs, k)
    rows = np.array([0, 19, 20, 49, 33], dtype=np.int64)
    sub = oracle.forward(Q, K, V, offs, k, rows=rows)
    for name in ("out", "idx", "score", "gap"):
        np.testing.assert_array_equal(sub[name], full[name][rows])


def test_forward_given_idx_reproduces_forward_and_ignores_order():
    N, H, d, k = 30, 2, 8, 5
    Q, K, V, _ = _rand(20, N, H, d)
    offs = _offs(4, 26)                       # first graph smaller than k -> padded slots
    f = oracle.forward(Q, K, V, offs, k)
    out, score = oracle.forward_given_idx(Q, K, V, f["idx"])
    np.testing.assert_allclose(out, f["out"], rtol=1e-14, atol=1e-16)
    np.testing.assert_array_equal(score, f["score"])
    out2, _ = oracle.forward_given_idx(Q, K, V, f["idx"][:, :, ::-1])
    np.testing.assert_allclose(out2, f["out"], rtol=1e-13, atol=1e-15)


def test_gap_is_distance_to_first_excluded():
    N, H, d, k = 25, 1, 4, 3
    Q, K, V, _ = _rand(21, N, H, d)
    r = oracle.forward(Q, K, V, None, k)
    S = np.einsum("ihc,jhc->ihj", Q.astype(np.float64), K.astype(np.float64))
    srt = -np.sort(-S, axis=2)
    np.testing.assert_allclose(r["gap"], srt[:, :, k - 1] - srt[:, :, k], rtol=1e-12, atol=1e-15)


# ----------------------------------------------------------------------------- backward
def _autograd_reference(Q, K, V, g, offs, k):
    """topk -> gather -> softmax -> einsum with library ops (fp64), per graph."""
    q, kk, v, gg = (torch.from_numpy(x.astype(np.float64)) for x in (Q, K, V, g))
    q.requires_grad_(True)
    kk.requires_grad_(True)
    v.requires_grad_(True)
    d = Q.shape[2]
    loss = 0.0
    for a, b in zip(offs[:-1], offs[1:]):
        if b == a:
            continue
        S = torch.einsum("ihc,jhc->hij", q[a:b], kk[a:b])
        ke = min(k, b - a)
        val, ind = torch.topk(S, ke, dim=2)
        P = torch.softmax(val / np.sqrt(d), dim=2)
        vh = v[a:b].permute(1, 0, 2)                                   # [H, n, d]
        Vg = torch.gather(vh.unsqueeze(1).expand(-1, b - a, -1, -1), 2,
                          ind.unsqueeze(-1).expand(-1, -1, -1, d))      # [H, n, ke, d]
        out = torch.einsum("hnk,hnkv->nhv", P, Vg)
        loss = loss + (out * gg[a:b]).sum()
    loss.backward()
    return q.grad.numpy(), kk.grad.numpy(), v.grad.numpy()


@pytest.mark.parametrize("sizes,H,d,k", [([40], 2, 8, 5), ([7, 3, 22], 3, 4, 4)])
def test_backward_matches_autograd(sizes, H, d, k):
    N = sum(sizes)
    Q, K, V, g = _rand(22, N, H, d)
    offs = _offs(*sizes)
    f = oracle.forward(Q, K, V, offs, k)
    assert f["gap"].min() > 1e-9
    dQ, dK, dV = oracle.backward(Q, K, V, g, f["idx"])
    rq, rk, rv = _autograd_reference(Q, K, V, g, offs, k)
    np.testing.assert_allclose(dQ, rq, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(dK, rk, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(dV, rv, rtol=1e-11, atol=1e-13)


def test_backward_finite_differences_frozen_selection():
    N, H, d, k = 12, 2, 4, 3
    Q, K, V, g = _rand(23, N, H, d)
    f = oracle.forward(Q, K, V, None, k)
    idx = f["idx"]
    dQ, dK, dV = oracle.backward(Q, K, V, g, idx)

    def loss(q, kk, v):
        out, _ = oracle.forward_given_idx(q, kk, v, idx)
        return float((out * g.astype(np.float64)).sum())

    eps = 2.0 ** -10                         # exactly representable steps in float32
    rng = np.random.default_rng(1)
    for which, grad in (("Q", dQ), ("K", dK), ("V", dV)):
        for _ in range(12):
            i, h, c = rng.integers(N), rng.integers(H), rng.integers(d)
            arrs = {"Q": Q.copy(), "K": K.copy(), "V": V.copy()}
            arrs[which][i, h, c] += eps
            lp = loss(arrs["Q"], arrs["K"], arrs["V"])
            arrs[which][i, h, c] -= 2 * eps
            lm = loss(arrs["Q"], arrs["K"], arrs["V"])
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - grad[i, h, c]) <= 1e-5 * max(1.0, abs(fd)), (which, i, h, c, fd, grad[i, h, c])


def test_backward_closed_forms():
    # k = 1: the weight is exactly 1, so no gradient reaches Q or K and dV collects g
    N, H, d = 30, 2, 4
    Q, K, V, g = _rand(24, N, H, d)
    f = oracle.forward(Q, K, V, None, 1)
    dQ, dK, dV = oracle.backward(Q, K, V, g, f["idx"])
    assert np.all(dQ == 0) and np.all(dK == 0)
    ref = np.zeros_like(dV)
    for i in range(N):
        for h in range(H):
            ref[f["idx"][i, h, 0], h] += g[i, h]
    np.testing.assert_allclose(dV, ref, rtol=1e-14)

    # k = 2, one query, two keys: p0 = sigma(delta), dS0 = -dS1 = p0 p1 (dP0 - dP1) / sqrt(d)
    d = 4
    Q = np.array([[[1.0, 2.0, 0.5, -1.0]]], dtype=np.float32)
    Q2 = np.concatenate([Q, Q * 0], axis=0)
    K2 = np.array([[[0.5, 1.0, 0.0, 0.25]], [[-1.0, 0.5, 2.0, 1.0]]], dtype=np.float32)
    V2 = np.array([[[1.0, 0.0, 2.0, -1.0]], [[0.5, 3.0, -2.0, 0.0]]], dtype=np.float32)
    g2 = np.array([[[1.0, -1.0, 0.5, 2.0]], [[0.0, 0.0, 0.0, 0.0]]], dtype=np.float32)
    f = oracle.forward(Q2, K2, V2, None, 2)
    dQ, dK, dV = oracle.backward(Q2, K2, V2, g2, f["idx"])
    s = K2[:, 0].astype(np.float64) @ Q[0, 0].astype(np.float64)
    p0 = 1.0 / (1.0 + np.exp(-(s[0] - s[1]) / np.sqrt(d)))
    p = np.array([p0, 1 - p0])
    dP = V2[:, 0].astype(np.float64) @ g2[0, 0].astype(np.float64)
    dS0 = p0 * (1 - p0) * (dP[0] - dP[1]) / np.sqrt(d)
    np.testing.assert_allclose(dQ[0, 0], dS0 * (K2[0, 0] - K2[1, 0]), rtol=1e-12)
    # row 1 has q = 0 and g = 0: it adds nothing anywhere
    np.testing.assert_allclose(dK[0, 0], dS0 * Q[0, 0], rtol=1e-12)
    np.testing.assert_allclose(dK[1, 0], -dS0 * Q[0, 0], rtol=1e-12)
    np.testing.assert_allclose(dV[:, 0], p[:, None] * g2[0, 0][None, :], rtol=1e-12)


def test_backward_identities():
    sizes, H, d, k = [33, 20], 3, 8, 6
    N = sum(sizes)
    Q, K, V, g = _rand(25, N, H, d)
    offs = _offs(*sizes)
    f = oracle.forward(Q, K, V, offs, k)
    dQ, dK, dV = oracle.backward(Q, K, V, g, f["idx"])
    # weights of a row sum to one  =>  sum_m dV[m] = sum_i g[i] per head and column
    np.testing.assert_allclose(dV.sum(axis=0), g.astype(np.float64).sum(axis=0), rtol=1e-12, atol=1e-12)
    # sum_t dS_t = 0 and each pair adds dS q.k to both sides  =>  sum_i q_i.dq_i = sum_m k_m.dk_m per head
    lhs = np.einsum("ihc,ihc->h", Q.astype(np.float64), dQ)
    rhs = np.einsum("ihc,ihc->h", K.astype(np.float64), dK)
    np.testing.assert_allclose(lhs, rhs, rtol=1e-10, atol=1e-12)
    # keys never selected receive no gradient
    hit = np.zeros((N, H), dtype=bool)
    for h in range(H):
        hit[f["idx"][:, h, :].ravel(), h] = True
    assert np.all(dK[~hit] == 0) and np.all(dV[~hit] == 0)


# ----------------------------------------------------------------------------- attention dropout
def test_dropout_draws_follow_the_published_generator():
    """Slot t of query 0, head 0 draws the (t+1)-th SplitMix64 output for the seed (fixture: the
    generator's published vector for state 0).  Three equal scores give weights 1/3 in key order,
    so with drop = 0.5 the output is the sum of (1/3) / 0.5 * v_t over the slots whose top 24 bits
    are at least half of 2^24."""
    import json, os
    fx = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "splitmix64_vectors.json")))
    u = [int(x, 16) >> 40 for x in fx["outputs_hex"][:3]]
    keep = [x >= (1 << 23) for x in u]
    assert keep == [True, False, False]
    N, H, d, k = 3, 1, 4, 3
    Q = np.zeros((N, H, d), dtype=np.float32)
    K = np.ones((N, H, d), dtype=np.float32)
    V = np.arange(N * d, dtype=np.float32).reshape(N, H, d) + 1.0
    idx = np.tile(np.arange(3, dtype=np.int32), (N, H, 1))
    out, _ = oracle.forward_given_idx(Q, K, V, idx, drop=0.5, seed=fx["initial_state"])
    want = sum((1.0 / 3.0) / 0.5 * V[t, 0].astype(np.float64) for t in range(3) if keep[t])
    np.testing.assert_allclose(out[0, 0], want, rtol=1e-14)


def test_dropout_zero_is_the_plain_path_and_keep_rate_matches():
    sizes, H, d, k = [300], 2, 8, 1
    Q, K, V, g = _rand(31, sizes[0], H, d)
    f = oracle.forward(Q, K, V, _offs(*sizes), k)
    plain, _ = oracle.forward_given_idx(Q, K, V, f["idx"])
    same, _ = oracle.forward_given_idx(Q, K, V, f["idx"], drop=0.0, seed=123)
    assert np.array_equal(plain, same)
    # k = 1: the single weight is 1, so a row is either v / (1 - drop) or exactly zero
    drop = 0.3
    out, _ = oracle.forward_given_idx(Q, K, V, f["idx"], drop=drop, seed=9)
    zero = np.all(out == 0.0, axis=-1)
    np.testing.assert_allclose(out[~zero], plain[~zero] / (1.0 - drop), rtol=1e-14)
    n = zero.size
    assert abs(zero.mean() - drop) < 5.0 * np.sqrt(drop * (1 - drop) / n)      # binomial, 5 sigma
    again, _ = oracle.forward_given_idx(Q, K, V, f["idx"], drop=drop, seed=9)
    other, _ = oracle.forward_given_idx(Q, K, V, f["idx"], drop=drop, seed=10)
    assert np.array_equal(out, again) and not np.array_equal(out, other)


def test_dropout_is_unbiased():
    """Constant V = 1: the output is the sum of the dropped-out weights, with expectation 1 and
    variance sum_t p_t^2 * drop / (1 - drop) <= drop / (1 - drop); averaged over S seeds."""
    sizes, H, d, k = [60], 2, 4, 6
    Q, K, _, _ = _rand(32, sizes[0], H, d)
    V = np.ones((sizes[0], H, d), dtype=np.float32)
    f = oracle.forward(Q, K, V, _offs(*sizes), k)
    drop, S = 0.5, 400
    acc = np.zeros((sizes[0], H, d))
    for s in range(S):
        acc += oracle.forward_given_idx(Q, K, V, f["idx"], drop=drop, seed=1000 + s)[0]
    assert np.all(np.abs(acc / S - 1.0) < 6.0 * np.sqrt(drop / (1 - drop) / S))


def test_dropout_backward_matches_finite_differences():
    """L = sum(out * g) with the selection and the draws held fixed is a smooth function of Q, K, V:
    central differences in fp64 pin the backward formulas with dropout (dP scaled, dV scaled)."""
    sizes, H, d, k = [9, 6], 2, 3, 4
    N = sum(sizes)
    Q, K, V, g = _rand(33, N, H, d)
    f = oracle.forward(Q, K, V, _offs(*sizes), k)
    idx, drop, seed = f["idx"], 0.4, 77
    dQ, dK, dV = oracle.backward(Q, K, V, g, idx, drop=drop, seed=seed)

    def loss(q, kk, v):
        return float((oracle.forward_given_idx(q, kk, v, idx, drop=drop, seed=seed)[0] * g.astype(np.float64)).sum())

    rng = np.random.default_rng(5)
    eps = 2.0 ** -8          # exactly representable steps keep the float32 inputs exact
    for name, grad in (("Q", dQ), ("K", dK), ("V", dV)):
        for _ in range(12):
            i, h, c = rng.integers(N), rng.integers(H), rng.integers(d)
            args = {"Q": Q.copy(), "K": K.copy(), "V": V.copy()}
            args[name][i, h, c] += eps
            up = loss(args["Q"], args["K"], args["V"])
            args[name][i, h, c] -= 2 * eps
            dn = loss(args["Q"], args["K"], args["V"])
            num = (up - dn) / (2 * eps)
            assert abs(num - grad[i, h, c]) <= 2e-4 * max(1.0, abs(num)), (name, i, h, c, num, grad[i, h, c])


# ----------------------------------------------------------------------------- top-k mass diagnostic
def test_topk_mass_against_library_softmax_and_special_cases():
    from scipy.special import softmax
    sizes, H, d, k = [37, 5, 60], 2, 8, 7
    N = sum(sizes)
    Q, K, _, _ = _rand(41, N, H, d)
    Q *= 3.0                                       # peaked rows as well as flat ones
    offs = _offs(*sizes)
    mass = oracle.topk_mass(Q, K, offs, k)
    for g in range(len(sizes)):
        lo, hi = offs[g], offs[g + 1]
        for h in range(H):
            S = Q[lo:hi, h].astype(np.float64) @ K[lo:hi, h].astype(np.float64).T / np.sqrt(d)
            P = np.sort(softmax(S, axis=1), axis=1)[:, ::-1]
            np.testing.assert_allclose(mass[lo:hi, h], P[:, :k].sum(axis=1), rtol=1e-12)
    np.testing.assert_allclose(mass[37:42], 1.0, rtol=1e-14)   # a graph with fewer nodes than k keeps everything
    # identical keys: every probability is 1/n, so the k largest hold k/n
    K2 = np.repeat(K[:1], N, axis=0)
    m2 = oracle.topk_mass(Q, K2, offs, k)
    np.testing.assert_allclose(m2[:37], k / 37.0, rtol=1e-12)
    np.testing.assert_allclose(m2[42:], k / 60.0, rtol=1e-12)
    # monotone in k and equal to the kept weights of the forward pass relative to the full softmax
    assert np.all(oracle.topk_mass(Q, K, offs, k + 3) >= mass - 1e-15)


# ----------------------------------------------------------------------------- argument checks
def test_bad_arguments_are_rejected():
    Q, K, V, _ = _rand(26, 8, 1, 4)
    with pytest.raises(ValueError):
        oracle.forward(Q, K, V, np.array([0, 5, 3, 8], dtype=np.int32), 2)   # decreasing offsets
    with pytest.raises(ValueError):
        oracle.forward(Q, K, V, np.array([0, 4], dtype=np.int32), 2)         # does not end at N
    with pytest.raises(ValueError):
        oracle.forward(Q, K, V, None, 2, rows=np.array([9], dtype=np.int64))


# ------------------------------------------------------------------ the full layer (Eq. 2, Algorithm 1 lines 2-8)
def _layer_case(seed, N=40, d_model=12, H=3, d=4):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((N, d_model))
    ws = [rng.standard_normal((H * d, d_model)) / np.sqrt(d_model) for _ in range(3)]
    w_o = rng.standard_normal((d_model, H * d)) / np.sqrt(H * d)
    return x, ws[0], ws[1], ws[2], w_o


def test_layer_with_k_equal_n_is_multi_head_attention():
    """Eq. 2 with T_k keeping everything is textbook multi-head self-attention inside each graph:
    independent check with torch's own linear and scaled_dot_product_attention in fp64."""
    import torch
    x, wq, wk, wv, wo = _layer_case(1)
    N, H, d = x.shape[0], 3, 4
    offs = np.array([0, 25, 40], dtype=np.int32)
    got = oracle.layer_forward(x, wq, wk, wv, wo, offs, H, 25)["y"]
    xt = torch.from_numpy(x)
    lin = lambda w: torch.nn.functional.linear(xt, torch.from_numpy(w)).view(N, H, d).transpose(0, 1)   # [H, N, d]
    q, k, v = lin(wq), lin(wk), lin(wv)
    o = torch.zeros(H, N, d, dtype=torch.float64)
    for lo, hi in ((0, 25), (25, 40)):
        o[:, lo:hi] = torch.nn.functional.scaled_dot_product_attention(q[:, lo:hi], k[:, lo:hi], v[:, lo:hi])
    ref = torch.nn.functional.linear(o.transpose(0, 1).reshape(N, H * d), torch.from_numpy(wo)).numpy()
    np.testing.assert_allclose(got, ref, rtol=0, atol=2e-6)      # Q, K, V, O pass through fp32 storage in the oracle


def test_layer_with_identity_projections_is_the_core():
    rng = np.random.default_rng(2)
    N, H, d = 30, 2, 4
    x = rng.standard_normal((N, H * d)).astype(np.float32).astype(np.float64)
    eye = np.eye(H * d)
    f = oracle.layer_forward(x, eye, eye, eye, eye, None, H, 5)
    core = oracle.forward(x.reshape(N, H, d), x.reshape(N, H, d), x.reshape(N, H, d), None, 5)
    assert np.array_equal(f["idx"], core["idx"])
    np.testing.assert_allclose(f["y"], core["out"].reshape(N, H * d), rtol=0, atol=1e-6)


def test_layer_backward_matches_central_differences_with_frozen_selection():
    x, wq, wk, wv, wo = _layer_case(3, N=24)
    H, k = 3, 4
    offs = np.array([0, 14, 24], dtype=np.int32)
    rng = np.random.default_rng(4)
    dy = rng.standard_normal((x.shape[0], wo.shape[0]))
    fwd = oracle.layer_forward(x, wq, wk, wv, wo, offs, H, k)
    g = oracle.layer_backward(x, wq, wk, wv, wo, H, fwd, dy)
    loss = lambda *a: float((oracle.layer_forward(*a, offs, H, k, idx=fwd["idx"])["y"] * dy).sum())
    args = [x, wq, wk, wv, wo]
    eps = 2e-3
    for pos, name in enumerate(("dx", "dw_q", "dw_k", "dw_v", "dw_o")):
        for _ in range(6):
            i, j = rng.integers(0, args[pos].shape[0]), rng.integers(0, args[pos].shape[1])
            hi_, lo_ = [a.copy() for a in args], [a.copy() for a in args]
            hi_[pos][i, j] += eps
            lo_[pos][i, j] -= eps
            fd = (loss(*hi_) - loss(*lo_)) / (2 * eps)
            assert abs(fd - g[name][i, j]) <= 2e-3 * max(1.0, abs(fd)), (name, i, j, fd, g[name][i, j])


def test_layer_bf16_storage_rounds_what_the_core_reads():
    x, wq, wk, wv, wo = _layer_case(5)
    f = oracle.layer_forward(x, wq, wk, wv, wo, None, 3, 6, storage="bf16")
    for name in ("q", "k", "v", "o"):
        a = f[name].astype(np.float32)
        assert np.array_equal(a.view(np.uint32) & 0xFFFF, np.zeros_like(a, dtype=np.uint32))   # bf16-representable
    exact = x @ wq.T
    assert np.max(np.abs(f["q"].reshape(exact.shape) - exact)) <= 2.0 ** -8 * np.max(np.abs(exact))
