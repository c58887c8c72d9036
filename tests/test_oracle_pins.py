"""Pins for the CPU oracle: it is checked against things other than itself.

Brute force in pure Python on tiny shapes (independent indexing, so a swapped
index or transposed operand shows), closed forms, textbook constants, library
routines (CPU torch in float64) and invariants that follow from Eq. 1-3 and the
TLS / CLS definitions of Sec. 2.1. No GPU involved.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2507_08771_b200 import inputs as I

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf(a):
    """float array -> bf16 bits, via torch's own rounding (a library, not the oracle)."""
    t = torch.as_tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def wide(b):
    """bf16 bits -> python floats via torch (library)."""
    t = torch.as_tensor(np.asarray(b).view(np.int16)).view(torch.bfloat16)
    return t.to(torch.float64).numpy()


def read_constants():
    vals = {}
    with open(os.path.join(GOLDEN, "textbook_constants.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split("=")
                vals[k.strip()] = float(v)
    return vals


# ----------------------------------------------------------------------------
# bf16 helpers
# ----------------------------------------------------------------------------
def test_bf16_rounding_matches_library_and_ties_to_even():
    rng = np.random.default_rng(1)
    a = np.concatenate([
        rng.standard_normal(4096).astype(np.float32) * 3,
        np.array([1.0 + 2.0**-8, 1.0 + 3 * 2.0**-8, -(1.0 + 2.0**-8), 0.0, -0.0, 65504.0, 1e-40,
                  3.3895314e38, np.inf, -np.inf], np.float32)])
    want = bf(a)
    assert np.array_equal(oracle.round_to_bf16(a), want)
    assert np.array_equal(I.f32_to_bf16_bits(a), want)
    # ties: 1 + 2^-8 lies midway between 1.0 and 1 + 2^-7 -> even mantissa (1.0)
    assert wide(oracle.round_to_bf16(np.array([1.0 + 2.0**-8], np.float32)))[0] == 1.0
    assert wide(oracle.round_to_bf16(np.array([1.0 + 3 * 2.0**-8], np.float32)))[0] == 1.0 + 2.0**-6
    assert np.array_equal(I.bf16_bits_to_f32(want[:4096]).astype(np.float64), wide(want[:4096]))


# ----------------------------------------------------------------------------
# router (Eq. 3)
# ----------------------------------------------------------------------------
def brute_router(x, W, gain, bias, eps):
    L, d = x.shape
    E = W.shape[0]
    a0 = [[0.0] * E for _ in range(L)]
    s = [[0.0] * E for _ in range(L)]
    for t in range(L):
        for i in range(E):
            acc = 0.0 if bias is None else float(bias[i])
            for k in range(d):
                acc += float(x[t][k]) * float(W[i][k])
            a0[t][i] = acc
        relu = [max(v, 0.0) for v in a0[t]]
        ms = sum(v * v for v in relu) / E
        for i in range(E):
            s[t][i] = float(gain[i]) * relu[i] / math.sqrt(ms + eps)
    return np.array(a0), np.array(s)


@pytest.mark.parametrize("L,d,E,with_bias", [(2, 5, 3, False), (3, 7, 6, True), (1, 9, 4, False)])
def test_router_brute_force(L, d, E, with_bias):
    rng = np.random.default_rng(10 + E)
    xb, Wb = bf(rng.standard_normal((L, d))), bf(rng.standard_normal((E, d)))
    gain = rng.uniform(0.5, 1.5, E).astype(np.float32)
    bias = rng.standard_normal(E).astype(np.float32) if with_bias else None
    a0, s = oracle.router(xb, Wb, gain, bias, eps=1e-6)
    a0_b, s_b = brute_router(wide(xb), wide(Wb), gain, bias, 1e-6)
    np.testing.assert_allclose(a0, a0_b, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(s, s_b, rtol=1e-13, atol=1e-13)


def test_router_closed_form_equal_activations():
    # k experts see the same positive logit v, the rest a negative one:
    # s_i = g_i * v / sqrt(k v^2 / E + eps)  ->  g_i * sqrt(E / k) as eps -> 0.
    E, d, k, v = 12, 8, 3, 0.75
    x = np.zeros((1, d), np.float32); x[0, 2] = 2.0
    W = np.zeros((E, d), np.float32); W[:, 2] = -0.5; W[[1, 5, 9], 2] = v / 2.0
    gain = np.linspace(0.5, 1.5, E).astype(np.float32)
    for eps in (1e-6, 1e-2):
        _, s = oracle.router(bf(x), bf(W), gain, None, eps=eps)
        want = np.zeros(E)
        want[[1, 5, 9]] = gain[[1, 5, 9]].astype(np.float64) * v / math.sqrt(k * v * v / E + eps)
        np.testing.assert_allclose(s[0], want, rtol=1e-14, atol=0)
    _, s = oracle.router(bf(x), bf(W), gain, None, eps=1e-12)
    np.testing.assert_allclose(s[0, [1, 5, 9]], gain[[1, 5, 9]] * math.sqrt(E / k), rtol=1e-9)


def test_router_matches_torch_linear_relu_rmsnorm():
    rng = np.random.default_rng(3)
    L, d, E = 5, 96, 24
    xb, Wb = bf(rng.standard_normal((L, d))), bf(rng.standard_normal((E, d)) / math.sqrt(d))
    gain = rng.uniform(0.5, 1.5, E).astype(np.float32)
    bias = np.full(E, -0.3, np.float32)
    for b in (None, bias):
        a0, s = oracle.router(xb, Wb, gain, b, eps=1e-6)
        tx, tW = torch.from_numpy(wide(xb)), torch.from_numpy(wide(Wb))
        tb = None if b is None else torch.from_numpy(b.astype(np.float64))
        ta0 = torch.nn.functional.linear(tx, tW, tb)
        ts = torch.nn.functional.rms_norm(torch.relu(ta0), (E,),
                                          weight=torch.from_numpy(gain.astype(np.float64)), eps=1e-6)
        np.testing.assert_allclose(a0, ta0.numpy(), rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(s, ts.numpy(), rtol=1e-12, atol=1e-13)


def test_router_invariants():
    rng = np.random.default_rng(4)
    L, d, E, eps = 6, 64, 16, 1e-6
    xb, Wb = bf(rng.standard_normal((L, d))), bf(rng.standard_normal((E, d)) / 8)
    gain = rng.uniform(0.5, 1.5, E).astype(np.float32)
    a0, s = oracle.router(xb, Wb, gain, None, eps=eps)
    # sum_i (s_i / g_i)^2 = E * ms / (ms + eps)
    ms = (torch.relu(torch.from_numpy(wide(xb)) @ torch.from_numpy(wide(Wb)).T).numpy() ** 2).mean(1)
    np.testing.assert_allclose(((s / gain) ** 2).sum(1), E * ms / (ms + eps), rtol=1e-12)
    # ReLU: scores are zero exactly where the logit is <= 0, positive elsewhere (gain > 0)
    assert np.array_equal(s > 0, a0 > 0) and np.all(s[a0 <= 0] == 0.0)
    # positive scaling of x (exact in bf16: *4) leaves the scores unchanged up to eps
    x4 = bf(wide(xb) * 4.0)
    _, s4 = oracle.router(x4, Wb, gain, None, eps=0.0)
    _, s1 = oracle.router(xb, Wb, gain, None, eps=0.0)
    np.testing.assert_allclose(s4, s1, rtol=1e-13)
    # a token with no positive logit: all scores zero, nothing NaN
    xz = xb.copy(); xz[0] = 0
    _, sz = oracle.router(xz, Wb, gain, None, eps=eps)
    assert np.all(sz[0] == 0.0) and np.isfinite(sz).all()


# ----------------------------------------------------------------------------
# masks, union, counters (Sec. 3.3, Sec. 2.1)
# ----------------------------------------------------------------------------
def sparse_scores(rng, L, E, p):
    s = np.abs(rng.standard_normal((L, E))) + 0.05
    s[rng.random((L, E)) >= p] = 0.0
    return s


@pytest.mark.parametrize("L,E,p", [(1, 16, 0.3), (4, 16, 0.5), (8, 33, 0.1), (8, 64, 0.2),
                                    (32, 100, 0.05), (5, 256, 0.02), (3, 40, 0.0), (3, 40, 1.0)])
def test_masks_union_counters_brute_force(L, E, p):
    rng = np.random.default_rng(L * 1000 + E)
    s = sparse_scores(rng, L, E, p)
    tm = oracle.token_masks(s)
    W = (E + 31) // 32
    assert tm.shape == (L, W)
    active = [set(i for i in range(E) if s[t, i] != 0.0) for t in range(L)]
    for t in range(L):
        got = set(i for i in range(W * 32) if (int(tm[t, i // 32]) >> (i % 32)) & 1)
        assert got == active[t]                       # also: no bits at or beyond E
    stats = np.zeros(4, np.uint64)
    um, ids, n = oracle.chunk_union(tm, E, stats)
    union = set().union(*active)
    assert set(i for i in range(W * 32) if (int(um[i // 32]) >> (i % 32)) & 1) == union
    assert n == len(union)
    assert list(ids[:n]) == sorted(union) and np.all(ids[n:] == -1) and ids.shape == (E,)
    assert n >= max(len(a) for a in active)
    assert list(stats) == [L, sum(len(a) for a in active), 1, len(union)]
    assert oracle.tls(stats, E) == pytest.approx(1 - sum(len(a) for a in active) / (L * E), abs=1e-15)
    assert oracle.cls(stats, E) == pytest.approx(1 - len(union) / E, abs=1e-15)
    assert oracle.cls(stats, E) <= oracle.tls(stats, E) + 1e-15
    if L == 1:                                        # CLS_1 == TLS, union == the token's mask
        assert oracle.cls(stats, E) == oracle.tls(stats, E)
        assert np.array_equal(um, tm[0])


def test_mask_edge_values_and_permutation():
    s = np.zeros((2, 8)); s[0, 1] = -0.0; s[0, 2] = np.nan; s[1, 3] = -1e-300; s[1, 7] = np.inf
    tm = oracle.token_masks(s)
    assert int(tm[0, 0]) == 1 << 2 and int(tm[1, 0]) == (1 << 3) | (1 << 7)
    rng = np.random.default_rng(7)
    s = sparse_scores(rng, 6, 40, 0.2)
    perm = rng.permutation(40)
    _, ids, n = oracle.chunk_union(oracle.token_masks(s), 40)
    _, ids_p, n_p = oracle.chunk_union(oracle.token_masks(s[:, perm]), 40)
    inv = np.argsort(perm)
    assert n == n_p and sorted(inv[ids[:n]]) == list(ids_p[:n_p])


def test_counters_accumulate_and_cls_grows_with_chunk_length():
    rng = np.random.default_rng(9)
    E, T = 48, 64
    s = sparse_scores(rng, T, E, 0.2)
    tm = oracle.token_masks(s)
    prev = None
    for L in (1, 2, 4, 8, 16):
        stats = np.zeros(4, np.uint64)
        for c in range(T // L):
            oracle.chunk_union(tm[c * L:(c + 1) * L], E, stats)
        assert stats[0] == T and stats[2] == T // L
        tls_v, cls_v = oracle.tls(stats, E), oracle.cls(stats, E)
        assert tls_v == pytest.approx(1 - np.count_nonzero(s) / (T * E))
        if prev is not None:
            assert cls_v <= prev + 1e-15              # merging chunks can only grow unions
        prev = cls_v


def test_score_generator_fixes_union_size_exactly():
    for idx in (1, 2):
        sh = I.SHAPES[idx]
        for L in (1, 2, 8, 32):
            stats = np.zeros(4, np.uint64)
            for chunk in range(20):
                s = I.make_scores(sh.E, L, sh.u, I.config_seed(idx), chunk=chunk)
                assert s.dtype == np.float32 and np.all((s == 0) | (s >= 0.05))
                _, _, n = oracle.chunk_union(oracle.token_masks(s), sh.E, stats)
                assert n == sh.u
            assert oracle.cls(stats, sh.E) == pytest.approx(1 - sh.u / sh.E, abs=1e-15)
            if L == 8:
                assert 0.74 < oracle.tls(stats, sh.E) < 0.86


# ----------------------------------------------------------------------------
# expert FFN (Eq. 1, Eq. 2)
# ----------------------------------------------------------------------------
def brute_ffn(x, s, U, D):
    L, d = x.shape
    E, d_e, _ = U.shape
    out = [[0.0] * d for _ in range(L)]
    for t in range(L):
        for i in range(E):
            for j in range(d_e):
                m = sum(float(x[t][k]) * float(U[i][j][k]) for k in range(d))
                h = float(s[t][i]) * m * (1.0 / (1.0 + math.exp(-m)))
                for c in range(d):
                    out[t][c] += h * float(D[i][c][j])
    return np.array(out)


@pytest.mark.parametrize("L,d,E,d_e", [(2, 3, 2, 2), (3, 5, 4, 3), (1, 6, 3, 4)])
def test_expert_ffn_brute_force(L, d, E, d_e):
    rng = np.random.default_rng(d * 10 + E)
    xb = bf(rng.standard_normal((L, d)))
    Ub, Db = bf(rng.standard_normal((E, d_e, d))), bf(rng.standard_normal((E, d, d_e)))
    s = sparse_scores(rng, L, E, 0.7)
    got = oracle.expert_ffn(xb, s, Ub, Db)
    want = brute_ffn(wide(xb), s, wide(Ub), wide(Db))
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)


def swish_via_oracle(z):
    """Swish(z) read out of the oracle: d = d_e = E = 1, x = 1, U = z, D = 1, s = 1."""
    one = bf(np.ones((1, 1)))
    return oracle.expert_ffn(one, np.ones((1, 1)), bf(np.full((1, 1, 1), z)), one.reshape(1, 1, 1))[0, 0]


def test_swish_textbook_values():
    c = read_constants()
    assert swish_via_oracle(0.0) == 0.0
    assert swish_via_oracle(1.0) == pytest.approx(c["sigmoid_1"], rel=1e-14)       # 1 * sigma(1): beta = 1
    assert swish_via_oracle(-1.0) == pytest.approx(c["sigmoid_1"] - 1.0, rel=1e-13)
    assert swish_via_oracle(40.0) == pytest.approx(40.0, rel=1e-15)
    assert abs(swish_via_oracle(-40.0)) < 1e-15
    for z in (0.125, 0.5, 2.0, 3.75):                                              # Swish(z) - Swish(-z) = z
        assert swish_via_oracle(z) - swish_via_oracle(-z) == pytest.approx(z, rel=1e-14)
    zs = wide(bf(np.linspace(-4, 1, 801)))
    vals = np.array([swish_via_oracle(z) for z in zs])
    assert vals.min() >= c["silu_min_value"] - 1e-12
    assert vals.min() == pytest.approx(c["silu_min_value"], abs=2e-5)
    assert zs[vals.argmin()] == pytest.approx(c["silu_min_arg"], abs=8e-3)


def test_expert_ffn_equals_dense_library_gemms():
    # With every expert in play the layer is two plain GEMMs (CPU torch, float64):
    # out = ((S (x) 1_{d_e}) o SiLU(X U_all^T)) D_all
    rng = np.random.default_rng(21)
    L, d, E, d_e = 5, 48, 6, 16
    xb = bf(rng.standard_normal((L, d)))
    Ub = bf(rng.standard_normal((E, d_e, d)) / math.sqrt(d))
    Db = bf(rng.standard_normal((E, d, d_e)) / math.sqrt(d_e))
    s = np.abs(rng.standard_normal((L, E))) + 0.05
    X, U, D = (torch.from_numpy(wide(a)) for a in (xb, Ub, Db))
    mid = torch.nn.functional.silu(X @ U.reshape(E * d_e, d).T)
    h = mid * torch.from_numpy(s).repeat_interleave(d_e, dim=1)
    want = h @ D.permute(0, 2, 1).reshape(E * d_e, d)
    got = oracle.expert_ffn(xb, s, Ub, Db)
    np.testing.assert_allclose(got, want.numpy(), rtol=1e-11, atol=1e-12)


def _small_problem(seed, L=4, d=32, E=8, d_e=8, p=0.4):
    rng = np.random.default_rng(seed)
    xb = bf(rng.standard_normal((L, d)))
    Ub = bf(rng.standard_normal((E, d_e, d)) / math.sqrt(d))
    Db = bf(rng.standard_normal((E, d, d_e)) / math.sqrt(d_e))
    return rng, xb, Ub, Db, sparse_scores(rng, L, E, p)


def test_expert_ffn_invariants():
    rng, xb, Ub, Db, s = _small_problem(31)
    L, E = s.shape
    base = oracle.expert_ffn(xb, s, Ub, Db)
    # zero scores -> zero output; zero down weights -> zero output
    assert np.all(oracle.expert_ffn(xb, np.zeros_like(s), Ub, Db) == 0.0)
    assert np.all(oracle.expert_ffn(xb, s, Ub, np.zeros_like(Db)) == 0.0)
    # linear in the scores, additive over disjoint score supports
    np.testing.assert_allclose(oracle.expert_ffn(xb, 2.5 * s, Ub, Db), 2.5 * base, rtol=1e-13)
    sa, sb = s.copy(), s.copy()
    sa[:, E // 2:] = 0; sb[:, :E // 2] = 0
    np.testing.assert_allclose(oracle.expert_ffn(xb, sa, Ub, Db) + oracle.expert_ffn(xb, sb, Ub, Db),
                               base, rtol=1e-12, atol=1e-14)
    # permuting the experts (weights and score columns together) changes nothing
    perm = rng.permutation(E)
    np.testing.assert_allclose(oracle.expert_ffn(xb, s[:, perm], Ub[perm], Db[perm]), base,
                               rtol=1e-12, atol=1e-14)
    # tokens are independent: each row equals the L = 1 call on that token
    for t in range(L):
        one = oracle.expert_ffn(xb[t:t + 1], s[t:t + 1], Ub, Db)
        assert np.array_equal(one[0], base[t])
    # a single expert, single token: out = s * D_i^T Swish(U_i x)
    i = 3
    s1 = np.zeros((1, E)); s1[0, i] = 0.7
    m = wide(Ub)[i] @ wide(xb)[0]
    want = 0.7 * (wide(Db)[i] @ (m / (1 + np.exp(-m))))
    np.testing.assert_allclose(oracle.expert_ffn(xb[:1], s1, Ub, Db)[0], want, rtol=1e-12, atol=1e-14)


def test_union_restricted_sum_equals_definition():
    # Sec. 3.3: leaving out experts no token activates drops only exact zeros.
    rng, xb, Ub, Db, s = _small_problem(41, L=6, E=12, p=0.15)
    tm = oracle.token_masks(s)
    _, ids, n = oracle.chunk_union(tm, 12)
    assert 0 < n < 12
    full = oracle.expert_ffn(xb, s, Ub, Db)
    only = oracle.expert_ffn(xb, s, Ub, Db, expert_ids=ids[:n])
    assert np.array_equal(full, only)
    padded = oracle.expert_ffn(xb, s, Ub, Db, expert_ids=ids)       # -1 tail entries are skipped
    assert np.array_equal(full, padded)
    # leaving out an expert that IS active changes the result
    assert not np.array_equal(full, oracle.expert_ffn(xb, s, Ub, Db, expert_ids=ids[1:n]))


# ----------------------------------------------------------------------------
# whole layer
# ----------------------------------------------------------------------------
def test_layer_is_the_composition_and_union_only_is_exact():
    sh, seed = I.SHAPES[0], I.config_seed(0)
    w = I.make_layer(sh, seed)
    x = I.make_x(sh.d, sh.L, seed)
    stats = np.zeros(4, np.uint64)
    r = oracle.layer_forward(x, w["W_r"], w["gain"], w["U"], w["D"], stats=stats)
    a0, s = oracle.router(x, w["W_r"], w["gain"])
    assert np.array_equal(r.scores, s) and np.array_equal(r.a0, a0)
    tm = oracle.token_masks(s)
    um, ids, n = oracle.chunk_union(tm, sh.E)
    assert np.array_equal(r.tok_mask, tm) and np.array_equal(r.union_ids, ids) and r.n_union == n
    assert np.array_equal(r.out, oracle.expert_ffn(x, s, w["U"], w["D"]))
    r2 = oracle.layer_forward(x, w["W_r"], w["gain"], w["U"], w["D"], union_only=True)
    assert np.array_equal(r.out, r2.out)
    assert stats[0] == sh.L and stats[2] == 1 and stats[3] == n
    # roughly half of the logits are positive for a zero-mean router
    assert 0.25 < 1 - oracle.tls(stats, sh.E) < 0.75


def test_scores_in_layer_matches_pieces():
    sh, seed = I.SHAPES[0], I.config_seed(0)
    w = I.make_layer(sh, seed, with_router=False)
    x = I.make_x(sh.d, sh.L, seed)
    sc = I.make_scores(sh.E, sh.L, 5, seed)
    r = oracle.layer_forward_scores(x, sc, w["U"], w["D"], union_only=True)
    assert r.n_union == 5
    assert np.array_equal(r.out, oracle.expert_ffn(x, sc.astype(np.float64), w["U"], w["D"]))




# ----------------------------------------------------------------------------
# router without RMSNorm (Sec. 4.2.3) and the reuse ratio (Sec. 4.1.2)
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("L,d,E,with_bias", [(2, 5, 3, False), (3, 7, 6, True)])
def test_router_relu_only_brute_force_and_library(L, d, E, with_bias):
    rng = np.random.default_rng(40 + E)
    xb, Wb = bf(rng.standard_normal((L, d))), bf(rng.standard_normal((E, d)))
    bias = rng.standard_normal(E).astype(np.float32) if with_bias else None
    a0, s = oracle.router_relu_only(xb, Wb, bias)
    for t in range(L):                                    # brute force, plain Python floats
        for i in range(E):
            acc = 0.0 if bias is None else float(bias[i])
            for k in range(d):
                acc += float(wide(xb)[t][k]) * float(wide(Wb)[i][k])
            assert a0[t, i] == pytest.approx(acc, rel=1e-13, abs=1e-13)
            assert s[t, i] == pytest.approx(max(acc, 0.0), rel=1e-13, abs=1e-13)
    tb = None if bias is None else torch.from_numpy(bias.astype(np.float64))
    ts = torch.relu(torch.nn.functional.linear(torch.from_numpy(wide(xb)), torch.from_numpy(wide(Wb)), tb))
    np.testing.assert_allclose(s, ts.numpy(), rtol=1e-12, atol=1e-13)
    assert (s >= 0).all() and ((s == 0) == (a0 <= 0)).all()


def test_router_relu_only_is_the_router_with_the_norm_taken_out():
    # Eq. 3 = RMSNorm applied to exactly these values: dividing the normalised scores by the
    # gain and multiplying the root mean square back must return them, and both share one mask
    rng = np.random.default_rng(41)
    L, d, E, eps = 4, 48, 20, 1e-6
    xb, Wb = bf(rng.standard_normal((L, d))), bf(rng.standard_normal((E, d)) / math.sqrt(d))
    gain = rng.uniform(0.5, 1.5, E).astype(np.float32)
    a0n, sn = oracle.router(xb, Wb, gain, None, eps=eps)
    a0p, sp = oracle.router_relu_only(xb, Wb, None)
    np.testing.assert_array_equal(a0n, a0p)
    rms_ = np.sqrt((sp ** 2).mean(axis=1, keepdims=True) + eps)
    np.testing.assert_allclose(sn / gain.astype(np.float64) * rms_, sp, rtol=1e-13, atol=1e-15)
    assert ((sn != 0) == (sp != 0)).all()
    # positive homogeneity, which the normalised router does not have: doubling x doubles A
    _, s2 = oracle.router_relu_only(bf(2.0 * wide(xb)), Wb, None)
    np.testing.assert_allclose(s2, 2.0 * sp, rtol=1e-13)


def test_layer_without_rmsnorm_is_the_composition():
    rng, x, U, D, _ = _small_problem(11)
    E, d = U.shape[0], x.shape[1]
    Wb = bf(rng.standard_normal((E, d)) / math.sqrt(d))
    bias = np.full(E, -0.5, np.float32)
    res = oracle.layer_forward(x, Wb, None, U, D, bias=bias, union_only=True, rmsnorm=False)
    a0, sp = oracle.router_relu_only(x, Wb, bias)
    np.testing.assert_array_equal(res.scores, sp)
    np.testing.assert_array_equal(res.tok_mask, oracle.token_masks(sp))
    np.testing.assert_allclose(res.out, oracle.expert_ffn(x, sp, U, D), rtol=1e-12, atol=1e-14)
    assert 0 < res.n_union <= E


def brute_reuse(active_sets):
    total, pairs = 0.0, 0
    for a, b in zip(active_sets[:-1], active_sets[1:]):
        if a:
            total += len(a & b) / len(a)
            pairs += 1
    return total, pairs


@pytest.mark.parametrize("L,E,p", [(2, 5, 0.5), (7, 40, 0.3), (32, 33, 0.2), (12, 64, 0.05), (1, 8, 0.5)])
def test_reuse_ratio_brute_force_with_sets(L, E, p):
    rng = np.random.default_rng(50 + L)
    s = sparse_scores(rng, L, E, p)
    sets = [set(np.nonzero(s[t])[0].tolist()) for t in range(L)]
    want, pairs = brute_reuse(sets)
    acc = oracle.reuse_ratio(s)
    assert acc[1] == pairs
    assert acc[0] == pytest.approx(want, rel=1e-14, abs=0)
    # accumulates over calls (one sequence each)
    acc2 = oracle.reuse_ratio(s, acc.copy())
    assert acc2[1] == 2 * pairs and acc2[0] == pytest.approx(2 * want, rel=1e-14)


def test_reuse_ratio_closed_forms():
    E = 16
    row = np.zeros(E); row[[1, 4, 9, 10]] = [0.5, -2.0, 1.0, 3.0]       # sign does not matter
    same = np.tile(row, (6, 1))
    acc = oracle.reuse_ratio(same)
    assert acc.tolist() == [5.0, 5.0]                                   # identical tokens: ratio 1
    other = np.zeros(E); other[[0, 2, 3]] = 1.0
    alt = np.stack([row, other, row, other])
    assert oracle.reuse_ratio(alt).tolist() == [0.0, 3.0]               # disjoint neighbours: ratio 0
    # nested shrinking sets S_{i+1} within S_i: each ratio is |S_{i+1}| / |S_i|; not symmetric
    a = np.zeros(E); a[:8] = 1.0
    b = np.zeros(E); b[:2] = 1.0
    assert oracle.reuse_ratio(np.stack([a, b]))[0] == 0.25
    assert oracle.reuse_ratio(np.stack([b, a]))[0] == 1.0
    # a token with no active expert has no ratio: the pair it starts is left out, the pair it
    # ends counts with ratio 0
    z = np.zeros(E)
    assert oracle.reuse_ratio(np.stack([a, z, a])).tolist() == [0.0, 1.0]
    assert oracle.reuse_ratio(np.stack([a])).tolist() == [0.0, 0.0]     # L = 1: no pair
    # -0.0 is inactive, NaN is active (by value, as for the masks)
    c = np.zeros(E); c[0] = -0.0; c[1] = np.nan
    n = np.zeros(E); n[1] = 1.0
    assert oracle.reuse_ratio(np.stack([c, n])).tolist() == [1.0, 1.0]


def test_reuse_ratio_agrees_with_the_token_masks():
    rng = np.random.default_rng(60)
    L, E = 16, 70
    s = sparse_scores(rng, L, E, 0.25)
    tm = oracle.token_masks(s)
    total = 0.0
    for i in range(L - 1):
        n_i = sum(bin(int(w)).count("1") for w in tm[i])
        both = sum(bin(int(a & b)).count("1") for a, b in zip(tm[i], tm[i + 1]))
        total += both / n_i
    assert oracle.reuse_ratio(s)[0] == pytest.approx(total, rel=1e-14)


def test_residual_step():
    rng = np.random.default_rng(5)
    res = rng.standard_normal((3, 16))
    out = rng.standard_normal((3, 16))
    want = res + out
    nxt = oracle.residual_step(res, out)
    assert np.array_equal(res, want)
    assert np.array_equal(nxt, bf(want.astype(np.float32)))


def test_golden_tiny_config_is_stable():
    """Sampled outputs of the tiny configuration, stored by tests/golden/make_golden.py
    (which calls the oracle only): guards the oracle against silent later edits."""
    sh, seed = I.SHAPES[0], I.config_seed(0)
    w = I.make_layer(sh, seed)
    x = I.make_x(sh.d, sh.L, seed)
    r = oracle.layer_forward(x, w["W_r"], w["gain"], w["U"], w["D"])
    rows = np.loadtxt(os.path.join(GOLDEN, "tiny_layer_oracle.txt"), comments="#", ndmin=2)
    for t, c, v in rows:
        assert r.out[int(t), int(c)] == pytest.approx(v, rel=1e-12, abs=1e-14)
    ids = np.loadtxt(os.path.join(GOLDEN, "tiny_layer_union.txt"), comments="#", dtype=np.int64, ndmin=1)
    assert list(r.union_ids[:r.n_union]) == list(ids)
