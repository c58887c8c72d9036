"""GPU parity: every C-ABI entry point against the CPU oracle, element by element,
on the same seeded inputs. Integer results (masks, union lists, counters) must be
bit-exact; floating-point outputs must satisfy max|err| <= 2e-2 * RMS(ref)
(bf16 weights, fp32 accumulation). On the router-on path a mask bit may differ
from the oracle's only where the oracle's pre-ReLU logit is within 1e-3 of zero.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2507_08771_b200 import binding as B
from paper_2507_08771_b200 import inputs as I

pytestmark = pytest.mark.gpu

TOL = 2e-2          # max|err| <= TOL * RMS(ref)
FLIP_BAND = 1e-3    # |pre-ReLU logit| below which a mask flip is excused
# (kernel family, config flags): CUDA-core; tensor-core chained (one kernel per call for chunks
# of at most 8 tokens, the up/down pair for longer ones); the same fully serialised; the pair
# for every chunk length
VARIANTS = [(B.VARIANT_SIMT, 0), (B.VARIANT_AUTO, 0), (B.VARIANT_AUTO, B.CFG_NO_CHAINING),
            (B.VARIANT_AUTO, B.CFG_TWO_KERNELS)]
# call flags worth running a tensor-core case under: a dependent call (whole device), weights
# promised stable, x promised stable as well (the one-kernel form then shares the device)
CALL_KINDS = [0, B.CALL_INDEPENDENT, B.CALL_INDEPENDENT_X]


def rms(a):
    return float(np.sqrt(np.mean(np.square(a)))) if a.size else 0.0


def assert_close(got, ref, what=""):
    r = rms(ref)
    err = float(np.abs(got.astype(np.float64) - ref).max()) if ref.size else 0.0
    assert np.isfinite(got).all(), what
    assert err <= TOL * r + 1e-30, f"{what}: max|err| {err:.3e} > {TOL} * RMS {r:.3e}"
    return err / r if r else 0.0


def same_up_to_summation_order(a, b):
    """Two results of the same call from launch configurations that sum in different orders. The
    fp32 sums differ by about 1e-6 of the RMS; where the sum behind an element of the bf16
    intermediate lands on the other side of a rounding boundary that element moves by one bf16
    step (2^-8 relative), which shows as a few 1e-4 of the RMS in the outputs it feeds. 1e-3
    covers a handful of such elements and is still twenty times tighter than the tolerance
    against the oracle."""
    return bool(np.isfinite(a).all() and np.abs(a.astype(np.float64) - b).max() <= 1e-3 * rms(b))


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def u32(t):
    return t.cpu().numpy().view(np.uint32)


def sparse_scores(rng, L, E, p):
    s = (np.abs(rng.standard_normal((L, E))) + 0.05).astype(np.float32)
    s[rng.random((L, E)) >= p] = 0.0
    return s


def small_layer(d, E, d_e, seed, bias_shift=None):
    sh = I.Shape("t", d=d, E=E, d_e=d_e, L=8, union_frac=0.3)
    return sh, I.make_layer(sh, seed, bias_shift=bias_shift)


# ----------------------------------------------------------------------------
# router
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("d,E,L,bias", [(256, 16, 4, None), (768, 48, 1, None), (1280, 40, 7, -0.8),
                                         (1792, 56, 13, None), (2048, 64, 8, -0.8),
                                         (2048, 128, 32, -0.8), (72, 33, 5, None)])
def test_router(d, E, L, bias):
    seed = 100 + E
    W_r, gain, b = I.make_router(d, E, seed, bias_shift=bias)
    x = I.make_x(d, L, seed)
    a0, s_ref = oracle.router(x, W_r, gain, b)
    tm_ref = oracle.token_masks(s_ref)
    layer = B.Layer(d, E, 64, L_max=32)
    dw = layer.upload_weights({"W_r": W_r, "gain": gain, "bias": b})
    scores = torch.full((L, E), float("nan"), device="cuda")
    tok = torch.full((L, layer.words), -1, dtype=torch.int32, device="cuda")
    B.blockffn_router(layer.h, dw.struct, B.to_device_bf16(x), L, scores, tok)
    torch.cuda.synchronize()
    got = scores.cpu().numpy()
    # scores: compare where the activation pattern agrees; flips only inside the band
    flips = (got != 0) != (s_ref != 0)
    assert np.all(np.abs(a0[flips]) < FLIP_BAND)
    ok = ~flips
    np.testing.assert_allclose(got[ok], s_ref[ok], rtol=2e-4, atol=2e-5)
    tm = u32(tok)
    for t in range(L):
        for i in range(layer.words * 32):
            bit = (int(tm[t, i // 32]) >> (i % 32)) & 1
            if i >= E:
                assert bit == 0
            else:
                assert bit == int(got[t, i] != 0)            # mask consistent with own scores
                if not flips[t, i]:
                    assert bit == (int(tm_ref[t, i // 32]) >> (i % 32)) & 1
    assert layer.last_status() == 0


# ----------------------------------------------------------------------------
# chunk union
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("L,E,p", [(1, 16, 0.3), (4, 16, 0.5), (8, 33, 0.1), (8, 64, 0.2), (8, 48, 0.07),
                                    (32, 100, 0.05), (5, 256, 0.02), (3, 1024, 0.01), (3, 40, 0.0),
                                    (3, 40, 1.0), (32, 1024, 1.0)])
def test_chunk_union_bit_exact(L, E, p):
    rng = np.random.default_rng(L * 7919 + E)
    s = sparse_scores(rng, L, E, p)
    if p > 0 and p < 1:
        s[0, 0] = -0.0
        s[L - 1, E - 1] = np.nan
    ref_stats = np.zeros(4, np.uint64)
    tm = oracle.token_masks(s.astype(np.float64))
    um_ref, ids_ref, n_ref = oracle.chunk_union(tm, E, ref_stats)
    layer = B.Layer(64, E, 64, L_max=32)
    W = layer.words
    um = torch.full((W,), -1, dtype=torch.int32, device="cuda")
    ids = torch.full((E,), 12345, dtype=torch.int32, device="cuda")
    nu = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    stats = torch.zeros(4, dtype=torch.int64, device="cuda")
    for rep in range(2):
        B.blockffn_chunk_union(layer.h, dev(s), L, um, ids, nu, stats)
    torch.cuda.synchronize()
    assert np.array_equal(u32(um), um_ref)
    assert np.array_equal(ids.cpu().numpy(), ids_ref)
    assert int(nu.item()) == n_ref
    assert list(stats.cpu().numpy().view(np.uint64)) == [2 * int(v) for v in ref_stats]
    hs = B.stats_to_host(stats)
    assert B.blockffn_tls(hs, E) == pytest.approx(oracle.tls(ref_stats, E), abs=1e-15)
    assert B.blockffn_cls(hs, E) == pytest.approx(oracle.cls(ref_stats, E), abs=1e-15)


# ----------------------------------------------------------------------------
# expert stage
# ----------------------------------------------------------------------------
def run_expert(layer, dw, x, s, ids, n, L, accumulate=None, want_next=False, call_flags=0):
    out = torch.full((L, layer.d), float("nan"), device="cuda")
    flags = call_flags
    if accumulate is not None:
        out.copy_(dev(accumulate, torch.float32))
        flags |= B.CALL_ACCUMULATE
    x_next = torch.zeros(L, layer.d, dtype=torch.bfloat16, device="cuda") if want_next else None
    B.blockffn_expert_ffn(layer.h, dw.struct, B.to_device_bf16(x), dev(s), L, dev(ids, torch.int32),
                          dev(np.array([n]), torch.int32), out, x_next, flags)
    torch.cuda.synchronize()
    return out.cpu().numpy(), (None if x_next is None else x_next.view(torch.int16).cpu().numpy().view(np.uint16))


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("d,E,d_e,L,p", [
    (256, 16, 64, 4, 0.5), (256, 16, 64, 1, 0.3), (768, 48, 64, 8, 0.2), (1280, 40, 128, 5, 0.2),
    (1536, 48, 128, 8, 0.2), (1792, 56, 128, 13, 0.15), (2048, 64, 128, 16, 0.1),
    (2048, 64, 128, 32, 0.05), (2048, 64, 128, 3, 1.0), (264, 9, 72, 7, 0.5), (512, 128, 128, 2, 0.1)])
def test_expert_ffn(variant, d, E, d_e, L, p):
    seed = 1000 + d + E
    sh, w = small_layer(d, E, d_e, seed)
    rng = np.random.default_rng(seed)
    x = I.make_x(d, L, seed)
    s = sparse_scores(rng, L, E, p)
    tm = oracle.token_masks(s.astype(np.float64))
    _, ids, n = oracle.chunk_union(tm, E)
    ref = oracle.expert_ffn(x, s.astype(np.float64), w["U"], w["D"], expert_ids=ids[:n])
    layer = B.Layer(d, E, d_e, L_max=32, variant=variant[0], flags=variant[1])
    dw = layer.upload_weights(w)
    got, _ = run_expert(layer, dw, x, s, ids, n, L)
    assert_close(got, ref, f"expert_ffn d={d} E={E} L={L}")
    again, _ = run_expert(layer, dw, x, s, ids, n, L)
    assert np.array_equal(got, again), "two runs differ: a race or an unwritten region"
    assert layer.last_status() == 0


@pytest.mark.parametrize("kind", CALL_KINDS[1:])
@pytest.mark.parametrize("d,E,d_e,L,p", [
    (256, 16, 64, 4, 0.5), (768, 48, 64, 8, 0.2), (1280, 40, 128, 5, 0.2), (1536, 48, 128, 8, 0.25),
    (1792, 56, 128, 7, 0.15), (2048, 64, 128, 8, 0.12), (2048, 64, 128, 8, 1.0), (2048, 128, 128, 1, 0.1),
    (2048, 128, 128, 8, 0.05), (512, 128, 256, 3, 0.2), (1024, 1000, 64, 8, 0.02), (64, 5, 64, 8, 0.6),
    (2048, 64, 128, 16, 0.1), (2048, 64, 128, 32, 0.1), (1536, 48, 128, 17, 0.2), (768, 48, 64, 9, 0.2),
    (2048, 128, 128, 31, 0.3), (512, 24, 64, 32, 0.5), (2048, 64, 128, 12, 1.0)])
def test_expert_ffn_under_call_promises(kind, d, E, d_e, L, p):
    """The expert stage under the two per-call promises. With x promised stable the one-kernel form
    runs a call on about a third of the SMs (up to three column tiles of out and several stages per
    CTA); with only the weights promised stable it owns the device (up to 8 tokens: the up/down
    pair; longer chunks: the one-kernel form, which then waits for its predecessor before it reads
    x). Shapes cover one to three column tiles, one and several stages, unions from a few experts
    to all of them, and chunks of 9 to 32 tokens (two token groups per weight fragment; from 17
    tokens on two teams of them in one CTA)."""
    seed = 3000 + d + E + L
    sh, w = small_layer(d, E, d_e, seed)
    rng = np.random.default_rng(seed)
    x = I.make_x(d, L, seed)
    s = sparse_scores(rng, L, E, p)
    tm = oracle.token_masks(s.astype(np.float64))
    _, ids, n = oracle.chunk_union(tm, E)
    ref = oracle.expert_ffn(x, s.astype(np.float64), w["U"], w["D"], expert_ids=ids[:n])
    layer = B.Layer(d, E, d_e, L_max=32)
    dw = layer.upload_weights(w)
    got, _ = run_expert(layer, dw, x, s, ids, n, L, call_flags=kind)
    assert_close(got, ref, f"expert_ffn flags={kind} d={d} E={E} L={L}")
    again, _ = run_expert(layer, dw, x, s, ids, n, L, call_flags=kind)
    assert np.array_equal(got, again)
    res0 = rng.standard_normal((L, d)).astype(np.float32)
    got2, nxt = run_expert(layer, dw, x, s, ids, n, L, accumulate=res0, want_next=True, call_flags=kind)
    assert_close(got2 - res0, ref, "accumulate under a promise")
    assert np.array_equal(nxt, oracle.round_to_bf16(got2))
    # the scores-in layer call under the same promise
    res = layer.forward_scores(dw, B.to_device_bf16(x), dev(s), call_flags=kind)
    torch.cuda.synchronize()
    assert int(res.n_union.item()) == n and np.array_equal(res.union_ids.cpu().numpy(), ids)
    assert_close(res.out.cpu().numpy(), ref, "layer call under a promise")
    assert layer.last_status() == 0


@pytest.mark.parametrize("L", [8, 16, 32])
def test_stable_x_calls_that_keep_the_whole_device(L):
    """BLOCKFFN_CFG_NO_SPLIT: calls with stable x get all SMs each (one 512-thread CTA per SM
    for more than 16 tokens). The hand-over inside the kernel needs every CTA of a call resident
    at once; the plan must never pick a grid for which that is not guaranteed."""
    sh, seed = I.SHAPES[2], I.config_seed(2)
    w = I.make_layer(sh, seed, with_router=False)
    layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=32, flags=B.CFG_NO_SPLIT)
    dw = layer.upload_weights(w)
    for chunk in range(3):
        x = I.make_x(sh.d, L, seed, chunk=chunk)
        s = I.make_scores(sh.E, L, sh.u, seed, chunk=chunk)
        ref = oracle.layer_forward_scores(x, s, w["U"], w["D"], union_only=True)
        res = layer.forward_scores(dw, B.to_device_bf16(x), dev(s), call_flags=B.CALL_INDEPENDENT_X)
        torch.cuda.synchronize()
        assert layer.last_status() == 0
        assert_close(res.out.cpu().numpy(), ref.out, f"no split, L={L}")


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("d,E,d_e,L", [(512, 24, 64, 6), (2048, 64, 128, 8), (1536, 48, 128, 19)])
def test_expert_ffn_signed_and_nan_scores(variant, d, E, d_e, L):
    """Scores of either sign (a negative RMSNorm gain gives them) and one NaN score: the NaN
    counts as active and spreads over that token's whole output row, no other token sees it."""
    seed = 2000 + d + L
    sh, w = small_layer(d, E, d_e, seed)
    rng = np.random.default_rng(seed)
    x = I.make_x(d, L, seed)
    s = sparse_scores(rng, L, E, 0.3) * rng.choice([-1.0, 1.0], size=(L, E)).astype(np.float32)
    assert (s < 0).any() and (s > 0).any()
    t_nan = L // 2
    i_nan = int(np.nonzero(s[0])[0][0])                    # an expert other tokens use as well
    s[t_nan, i_nan] = np.nan
    tm = oracle.token_masks(s.astype(np.float64))
    _, ids, n = oracle.chunk_union(tm, E)
    assert i_nan in ids[:n]
    ref = oracle.expert_ffn(x, s.astype(np.float64), w["U"], w["D"], expert_ids=ids[:n])
    assert np.isnan(ref[t_nan]).all() and np.isfinite(np.delete(ref, t_nan, axis=0)).all()
    layer = B.Layer(d, E, d_e, L_max=32, variant=variant[0], flags=variant[1])
    dw = layer.upload_weights(w)
    got, _ = run_expert(layer, dw, x, s, ids, n, L)
    assert np.isnan(got[t_nan]).all(), "the NaN score must reach every column of its token"
    keep = np.arange(L) != t_nan
    assert_close(got[keep], ref[keep], f"signed scores d={d} L={L}")
    # the same chunk through the scores-in layer call: the library derives the union itself
    res = layer.forward_scores(dw, B.to_device_bf16(x), dev(s))
    torch.cuda.synchronize()
    assert int(res.n_union.item()) == n and np.array_equal(res.union_ids.cpu().numpy(), ids)
    out = res.out.cpu().numpy()
    assert np.isnan(out[t_nan]).all()
    assert_close(out[keep], ref[keep], f"signed scores, layer call d={d} L={L}")
    assert layer.last_status() == 0


@pytest.mark.parametrize("variant", VARIANTS)
def test_union_list_tail_is_ignored(variant):
    """union_ids is an i32[E] array of which only the first *n_union entries count: whatever the
    tail holds (valid ids, ids out of range, garbage) changes neither the result nor the status."""
    d, E, d_e, L = 512, 40, 64, 7
    sh, w = small_layer(d, E, d_e, 31)
    rng = np.random.default_rng(31)
    x = I.make_x(d, L, 31)
    s = sparse_scores(rng, L, E, 0.6)
    keep = np.array([0, 3, 17, 39], np.int32)
    ref = oracle.expert_ffn(x, s.astype(np.float64), w["U"], w["D"], expert_ids=keep)
    layer = B.Layer(d, E, d_e, L_max=8, variant=variant[0], flags=variant[1])
    dw = layer.upload_weights(w)
    tails = [np.full(E - 4, -1), np.arange(4, E), np.full(E - 4, 2 ** 31 - 1), np.full(E - 4, -2 ** 31)]
    outs = []
    for tail in tails:
        ids = np.concatenate([keep, tail.astype(np.int64)]).astype(np.int32)
        got, _ = run_expert(layer, dw, x, s, ids, 4, L)
        assert_close(got, ref, "tail ignored")
        outs.append(got)
        assert layer.last_status() == 0
    assert all(np.array_equal(outs[0], o) for o in outs[1:])


@pytest.mark.parametrize("E,L", [(256, 8), (1000, 5), (1000, 17)])
def test_many_experts_layer_calls(E, L):
    """More than 128 experts (mask words beyond the four a warp folds in registers): the
    scores-in layer call and the router-on layer call, unions derived inside the kernels."""
    d, d_e = 512, 64
    seed = 4000 + E + L
    sh = I.Shape("t", d=d, E=E, d_e=d_e, L=L, union_frac=0.05)
    w = I.make_layer(sh, seed, bias_shift=-1.6)
    w["gain"] = (w["gain"] * np.where(np.arange(E) % 7 == 3, -1.0, 1.0)).astype(np.float32)   # some negative gains
    layer = B.Layer(d, E, d_e, L_max=32)
    dw = layer.upload_weights(w)
    rng = np.random.default_rng(seed)
    for chunk, p in enumerate((0.01, 0.05)):
        x = I.make_x(d, L, seed, chunk=chunk)
        s = sparse_scores(rng, L, E, p)
        s[0, E - 1] = 0.25                                 # the last expert, last mask word
        ref = oracle.layer_forward_scores(x, s, w["U"], w["D"], union_only=True)
        res = layer.forward_scores(dw, B.to_device_bf16(x), dev(s))
        torch.cuda.synchronize()
        assert int(res.n_union.item()) == ref.n_union
        assert np.array_equal(res.union_ids.cpu().numpy(), ref.union_ids)
        assert np.array_equal(u32(res.union_mask), ref.union_mask)
        assert_close(res.out.cpu().numpy(), ref.out, f"scores-in E={E} L={L} p={p}")
    hs = layer.stats_host()
    assert hs.n_chunks == 2 and hs.n_tokens == 2 * L
    xc = I.make_correlated_x(d, L, 0.8, seed, chunk=9)
    check_layer_router_on(layer, dw, w, xc, L, bias=w["bias"])
    x = I.make_x(d, L, seed, chunk=10)
    check_layer_router_on(layer, dw, w, x, L, bias=w["bias"])
    assert layer.last_status() == 0


@pytest.mark.parametrize("variant", VARIANTS)
def test_expert_ffn_degenerate_unions_and_residual(variant):
    d, E, d_e, L = 512, 24, 64, 6
    sh, w = small_layer(d, E, d_e, 77)
    rng = np.random.default_rng(77)
    x = I.make_x(d, L, 77)
    layer = B.Layer(d, E, d_e, L_max=8, variant=variant[0], flags=variant[1])
    dw = layer.upload_weights(w)
    # empty union: out = 0
    ids = np.full(E, -1, np.int32)
    got, _ = run_expert(layer, dw, x, np.zeros((L, E), np.float32), ids, 0, L)
    assert np.all(got == 0.0)
    # an expert left out of the list contributes nothing, whatever its score
    s = sparse_scores(rng, L, E, 0.5)
    keep = np.array([1, 4, 9, 20], np.int32)
    ids[:4] = keep
    ref = oracle.expert_ffn(x, s.astype(np.float64), w["U"], w["D"], expert_ids=keep)
    got, _ = run_expert(layer, dw, x, s, ids, 4, L)
    assert_close(got, ref, "listed experts only")
    # residual accumulate + bf16 of the new residual
    res0 = rng.standard_normal((L, d)).astype(np.float32)
    got, nxt = run_expert(layer, dw, x, s, ids, 4, L, accumulate=res0, want_next=True)
    assert_close(got - res0, ref, "accumulate")
    assert np.array_equal(nxt, oracle.round_to_bf16(got))
    # full union equals the dense score-weighted FFN
    s = (np.abs(rng.standard_normal((L, E))) + 0.05).astype(np.float32)
    ids = np.arange(E, dtype=np.int32)
    ref = oracle.expert_ffn(x, s.astype(np.float64), w["U"], w["D"])
    got, _ = run_expert(layer, dw, x, s, ids, E, L)
    assert_close(got, ref, "full union")
    assert layer.last_status() == 0


def test_bad_union_entries_are_flagged_not_followed():
    d, E, d_e, L = 256, 16, 64, 4
    sh, w = small_layer(d, E, d_e, 5)
    rng = np.random.default_rng(5)
    x = I.make_x(d, L, 5)
    s = sparse_scores(rng, L, E, 0.5)
    for variant in VARIANTS:
        layer = B.Layer(d, E, d_e, L_max=4, variant=variant[0], flags=variant[1])
        dw = layer.upload_weights(w)
        ids = np.full(E, -1, np.int32)
        ids[:3] = [2, 99, 7]                                   # 99 is out of range
        ref = oracle.expert_ffn(x, s.astype(np.float64), w["U"], w["D"], expert_ids=np.array([2, 7]))
        got, _ = run_expert(layer, dw, x, s, ids, 3, L)
        assert_close(got, ref, "bad id skipped")
        assert layer.last_status(clear=True) == B.DEV_BAD_UNION_ID
        assert layer.last_status() == 0
        ids = np.arange(E, dtype=np.int32)
        got, _ = run_expert(layer, dw, x, s, ids, E + 5, L)    # count too large: clamped to E
        assert_close(got, oracle.expert_ffn(x, s.astype(np.float64), w["U"], w["D"]), "clamped")
        assert layer.last_status(clear=True) == B.DEV_BAD_UNION_COUNT


@pytest.mark.parametrize("L,kind", [(8, B.CALL_INDEPENDENT_X), (16, B.CALL_INDEPENDENT_X),
                                    (32, B.CALL_INDEPENDENT_X), (32, B.CALL_INDEPENDENT)])
def test_bounded_wait_expires_cleanly(L, kind):
    """The hand-over inside the one-kernel form (calls whose x is promised stable, and chunks of
    more than 8 tokens in a dependent chain) is a bounded wait. With the test bit set it waits
    for an arrival that never comes: the call must come back with BLOCKFFN_DEV_WAIT_EXPIRED set,
    out untouched and the device usable; the next handle (without the bit) works as usual.
    All three kernels of that form are covered: 8 tokens, 16 tokens, 32 tokens (two teams)."""
    sh, seed = I.SHAPES[1], I.config_seed(1)
    sh = I.Shape(sh.name, d=sh.d, E=sh.E, d_e=sh.d_e, L=L, union_frac=sh.u / sh.E)
    w = I.make_layer(sh, seed, with_router=False)
    x = I.make_x(sh.d, sh.L, seed)
    s = I.make_scores(sh.E, sh.L, sh.u, seed)
    held = B.Layer(sh.d, sh.E, sh.d_e, L_max=sh.L, flags=B.CFG_TEST_EXPIRE_WAIT)
    dw = held.upload_weights(w)
    out = torch.full((sh.L, sh.d), 7.0, device="cuda")
    for _ in range(2):                                     # the counters stay consistent
        held.forward_scores(dw, B.to_device_bf16(x), dev(s), out=out, call_flags=kind)
        assert held.last_status(clear=True) == B.DEV_WAIT_EXPIRED
        assert bool((out == 7.0).all())
    assert held.last_status() == 0
    layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=sh.L)
    dw2 = layer.upload_weights(w)
    res = layer.forward_scores(dw2, B.to_device_bf16(x), dev(s), call_flags=kind)
    ref = oracle.layer_forward_scores(x, s, w["U"], w["D"], union_only=True)
    assert_close(res.out.cpu().numpy(), ref.out, "after an expired wait")
    assert layer.last_status() == 0


@pytest.mark.parametrize("L", [8, 32])
def test_bounded_wait_expires_cleanly_with_the_router_inside(L):
    """The same for a layer call whose router runs inside the kernel: its first hand-over (the
    logits) is a bounded wait of the same kind. The call comes back with the status bit set and
    out untouched; a handle without the test bit then gives the right result."""
    sh, seed = I.SHAPES[3], I.config_seed(3)
    w = I.make_layer(sh, seed, bias_shift=I.ROUTER_BIAS_SHIFT)
    x = I.make_correlated_x(sh.d, L, 0.9, seed, chunk=77)
    held = B.Layer(sh.d, sh.E, sh.d_e, L_max=L, flags=B.CFG_TEST_EXPIRE_WAIT)
    dw = held.upload_weights(w)
    out = torch.full((L, sh.d), 7.0, device="cuda")
    for _ in range(2):
        held.forward(dw, B.to_device_bf16(x), out=out, call_flags=B.CALL_INDEPENDENT_X)
        assert held.last_status(clear=True) == B.DEV_WAIT_EXPIRED
        assert bool((out == 7.0).all())
    layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=L)
    dw2 = layer.upload_weights(w)
    check_layer_router_on(layer, dw2, w, x, L, bias=w["bias"], call_flags=B.CALL_INDEPENDENT_X)
    assert layer.last_status() == 0


def test_host_side_argument_errors():
    layer = B.Layer(256, 16, 64, L_max=4)
    w = B.make_weights()
    x = torch.zeros(4, 256, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(4, 256, device="cuda")
    s = torch.zeros(4, 16, device="cuda")
    with pytest.raises(B.BlockFFNError) as e:
        B.blockffn_layer_forward_scores(layer.h, w, x, s, 4, out)     # NULL weights
    assert e.value.code == B.ERR_INVALID_ARG
    dw = layer.upload_weights(I.make_layer(I.SHAPES[0], 1))
    for L in (0, 5, -1):
        with pytest.raises(B.BlockFFNError):
            B.blockffn_layer_forward_scores(layer.h, dw.struct, x, s, L, out)
    with pytest.raises(B.BlockFFNError):                                # misaligned x
        B.blockffn_layer_forward_scores(layer.h, dw.struct, x.data_ptr() + 2, s, 4, out)
    with pytest.raises(B.BlockFFNError):                                # x_next aliases x
        B.blockffn_layer_forward_scores(layer.h, dw.struct, x, s, 4, out, x_next=x)
    with pytest.raises(B.BlockFFNError):                                # unknown flag
        B.blockffn_layer_forward_scores(layer.h, dw.struct, x, s, 4, out, call_flags=64)
    # the tensor-core kernels named explicitly: a shape or ring depth they do not take is an error
    for kw in (dict(d=264, E=9, d_e=72), dict(d=256, E=16, d_e=96), dict(d=256, E=16, d_e=64, flags=2)):
        with pytest.raises(B.BlockFFNError) as e:
            B.Layer(kw["d"], kw["E"], kw["d_e"], L_max=8, variant=B.VARIANT_MMA, flags=kw.get("flags", 0))
        assert e.value.code == B.ERR_UNSUPPORTED
    B.Layer(264, 9, 72, L_max=8, variant=B.VARIANT_AUTO)                # AUTO picks the other family


@pytest.mark.parametrize("form", [0, B.CFG_TWO_KERNELS])
@pytest.mark.parametrize("flag", [0, B.CALL_INDEPENDENT_X])
def test_bench_launch_configuration_router_on(flag, form):
    """Back-to-back blockffn_layer_forward calls in a graph. One-kernel form: the router runs
    inside the expert kernel (with the promise the calls overlap, without it each waits for the
    one before). Two-kernel form: with the promise the router of a call runs on a stream of the
    handle, several calls ahead of its expert kernels (a ring of logit buffers, marks and events
    that become graph edges); without it the router stays on the caller's stream."""
    sh, seed = I.SHAPES[3], I.config_seed(3)
    n_chunks, n_copies = 13, 3                             # odd: replays meet on the same buffer
    w = I.make_layer(sh, seed, bias_shift=I.ROUTER_BIAS_SHIFT)
    layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=sh.L, flags=form)
    dws = [layer.upload_weights(w) for _ in range(n_copies)]
    xs = [I.make_x(sh.d, sh.L, seed, chunk=c) for c in range(n_chunks)]
    xd = [B.to_device_bf16(x) for x in xs]
    out = torch.full((n_chunks, sh.L, sh.d), float("nan"), device="cuda")

    def enqueue(stream):
        for c in range(n_chunks):
            B.blockffn_layer_forward(layer.h, dws[c % n_copies].struct, xd[c], sh.L, out[c], None,
                                     layer.stats, flag, stream)

    graph_of(enqueue)
    got = out.cpu().numpy()
    assert np.isfinite(got).all()
    hs = layer.stats_host()
    assert hs.n_chunks == 3 * n_chunks and hs.n_tokens == 3 * n_chunks * sh.L
    # Every chunk: the same call made on its own gives the library's scores and union for that
    # chunk; it is checked against the oracle (flips only inside the band, else the oracle FFN
    # driven by the library's scores), and the overlapped run must reproduce it up to the order
    # of the fp32 sums (a call that shares the device splits its columns and experts differently
    # from one that owns it).
    for c in range(n_chunks):
        alone = check_layer_router_on(layer, dws[c % n_copies], w, xs[c], sh.L, bias=w.get("bias"),
                                      want_out=True)
        assert same_up_to_summation_order(got[c], alone), f"router on, flag {flag}, chunk {c}: differs from the call alone"
    assert layer.last_status() == 0


def test_router_ahead_mixed_sequence():
    """Layer calls with and without the x-stable promise, a scores-in call in between, eager on one
    stream: every transition between the router's three launch forms, each result checked."""
    sh, seed = I.SHAPES[3], I.config_seed(3)
    w = I.make_layer(sh, seed, bias_shift=I.ROUTER_BIAS_SHIFT)
    layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=sh.L)
    dw = layer.upload_weights(w)
    X = B.CALL_INDEPENDENT_X
    plan = [X, X, X, X, X, 0, X, X, "scores", X, X, X, X, X, 0, 0, X]
    xs = [I.make_x(sh.d, sh.L, seed, chunk=100 + c) for c in range(len(plan))]
    xd = [B.to_device_bf16(x) for x in xs]
    s_in = I.make_scores(sh.E, sh.L, sh.u, seed, chunk=7)
    s_dev = dev(s_in)
    out = torch.full((len(plan), sh.L, sh.d), float("nan"), device="cuda")
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for rep in range(2):                               # the second pass starts mid-ring
            for c, f in enumerate(plan):
                if f == "scores":
                    B.blockffn_layer_forward_scores(layer.h, dw.struct, xd[c], s_dev, sh.L, out[c],
                                                    None, layer.stats, X, stream.cuda_stream)
                else:
                    B.blockffn_layer_forward(layer.h, dw.struct, xd[c], sh.L, out[c], None,
                                             layer.stats, f, stream.cuda_stream)
        stream.synchronize()
    got = out.cpu().numpy()
    assert np.isfinite(got).all()
    for c, f in enumerate(plan):                           # every call of the sequence
        if f == "scores":
            ref = oracle.layer_forward_scores(xs[c], s_in, w["U"], w["D"], union_only=True)
            assert_close(got[c], ref.out, f"mixed sequence, call {c} ({f})")
        else:
            alone = check_layer_router_on(layer, dw, w, xs[c], sh.L, bias=w["bias"], want_out=True)
            assert same_up_to_summation_order(got[c], alone), f"mixed sequence, call {c} ({f})"
    assert layer.last_status() == 0


# ----------------------------------------------------------------------------
# whole layer: the benchmark configurations
# ----------------------------------------------------------------------------
def check_layer_router_on(layer, dw, w, x, L, bias=None, want_out=False, call_flags=0):
    """One blockffn_layer_forward call against the oracle. No chunk is ever skipped: where a
    mask bit differs from the oracle's (allowed only inside the band around a zero logit), the
    output is compared with the oracle FFN driven by the library's own scores and union."""
    ref = oracle.layer_forward(x, w["W_r"], w["gain"], w["U"], w["D"], bias=bias, union_only=True)
    res = layer.forward(dw, B.to_device_bf16(x), call_flags=call_flags)
    torch.cuda.synchronize()
    E = layer.E
    got_s = res.scores.cpu().numpy()
    flips = (got_s != 0) != (ref.scores != 0)
    assert np.all(np.abs(ref.a0[flips]) < FLIP_BAND)
    n = int(res.n_union.item())
    ids = res.union_ids.cpu().numpy()
    assert np.all(ids[n:] == -1) and np.all(np.diff(ids[:n]) > 0)
    # union lists agree once experts whose only activations are excused flips are set aside
    excused = set(np.nonzero(flips.any(axis=0))[0])
    assert set(ids[:n]) - excused == set(ref.union_ids[:ref.n_union]) - excused
    # the union must be exactly what the library's own scores imply (bit-exact)
    tm = oracle.token_masks(got_s.astype(np.float64))
    um2, ids2, n2 = oracle.chunk_union(tm, E)
    assert n2 == n and np.array_equal(ids2, ids) and np.array_equal(u32(res.union_mask), um2)
    assert np.array_equal(u32(res.tok_mask), tm)
    if not flips.any():
        assert np.array_equal(ids, ref.union_ids) and n == ref.n_union
        assert_close(res.out.cpu().numpy(), ref.out, "layer out")
    else:                         # compare against the oracle FFN driven by the library's scores
        ref2 = oracle.expert_ffn(x, got_s.astype(np.float64), w["U"], w["D"], expert_ids=ids[:n])
        assert_close(res.out.cpu().numpy(), ref2, "layer out (library scores)")
    assert layer.last_status() == 0
    if want_out:
        return res.out.cpu().numpy()
    return ref, n


@pytest.mark.parametrize("flag", [0, B.CALL_INDEPENDENT_X])
@pytest.mark.parametrize("L", [9, 16, 17, 32])
def test_router_on_long_chunks(L, flag):
    """blockffn_layer_forward on chunks of more than 8 tokens: the router runs inside the
    long-chunk kernel (8 tokens per pass), with and without the x-stable promise; several calls
    in a row on one handle."""
    sh, seed = I.SHAPES[3], I.config_seed(3)
    w = I.make_layer(sh, seed, bias_shift=I.ROUTER_BIAS_SHIFT)
    layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=32)
    dw = layer.upload_weights(w)
    for chunk in range(3):
        x = I.make_correlated_x(sh.d, L, 0.9, seed, chunk=40 + chunk)
        check_layer_router_on(layer, dw, w, x, L, bias=w["bias"], call_flags=flag)
    hs = layer.stats_host()
    assert hs.n_chunks == 3 and hs.n_tokens == 3 * L


@pytest.mark.parametrize("variant", VARIANTS)
def test_config0_tiny_full_router(variant):
    sh, seed = I.SHAPES[0], I.config_seed(0)
    w = I.make_layer(sh, seed)
    layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=sh.L, variant=variant[0], flags=variant[1])
    dw = layer.upload_weights(w)
    for chunk in range(3):
        x = I.make_x(sh.d, sh.L, seed, chunk=chunk)
        check_layer_router_on(layer, dw, w, x, sh.L)
    hs = layer.stats_host()
    assert hs.n_chunks == 3 and hs.n_tokens == 3 * sh.L


def check_scores_in(layer, dw, w, sh, L, seed, chunk, u=None):
    x = I.make_x(sh.d, L, seed, chunk=chunk)
    s = I.make_scores(sh.E, L, sh.u if u is None else u, seed, chunk=chunk)
    ref = oracle.layer_forward_scores(x, s, w["U"], w["D"], union_only=True)
    res = layer.forward_scores(dw, B.to_device_bf16(x), dev(s))
    torch.cuda.synchronize()
    assert int(res.n_union.item()) == ref.n_union
    assert np.array_equal(res.union_ids.cpu().numpy(), ref.union_ids)
    assert np.array_equal(u32(res.union_mask), ref.union_mask)
    return assert_close(res.out.cpu().numpy(), ref.out, f"scores-in L={L} chunk={chunk}")


@pytest.mark.parametrize("variant", VARIANTS)
def test_config1_scores_in(variant):
    sh, seed = I.SHAPES[1], I.config_seed(1)
    w = I.make_layer(sh, seed, with_router=False)
    layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=sh.L, variant=variant[0], flags=variant[1])
    dw = layer.upload_weights(w)
    for chunk in range(3):
        check_scores_in(layer, dw, w, sh, sh.L, seed, chunk)
    hs = layer.stats_host()
    assert B.blockffn_cls(hs, sh.E) == pytest.approx(1 - sh.u / sh.E)
    assert 0.7 < B.blockffn_tls(hs, sh.E) < 0.9
    assert layer.last_status() == 0


@pytest.mark.parametrize("variant", VARIANTS)
def test_config2_l_sweep(variant):
    sh, seed = I.SHAPES[2], I.config_seed(2)
    w = I.make_layer(sh, seed, with_router=False)
    layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=32, variant=variant[0], flags=variant[1])
    dw = layer.upload_weights(w)
    for L in I.L_SWEEP:
        check_scores_in(layer, dw, w, sh, L, seed, chunk=L)
    assert layer.last_status() == 0


def test_config3_full_layer_and_union_sweep():
    sh, seed = I.SHAPES[3], I.config_seed(3)
    w = I.make_layer(sh, seed, bias_shift=I.ROUTER_BIAS_SHIFT)
    layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=sh.L)
    dw = layer.upload_weights(w)
    x = I.make_x(sh.d, sh.L, seed)
    check_layer_router_on(layer, dw, w, x, sh.L, bias=w["bias"])
    hs = layer.stats_host()
    assert 0.70 < B.blockffn_tls(hs, sh.E) < 0.88            # Phi(-0.8) = 21 % active
    xc = I.make_correlated_x(sh.d, sh.L, 0.9, seed)
    check_layer_router_on(layer, dw, w, xc, sh.L, bias=w["bias"])
    for frac in (0.1, 0.5, 1.0):                              # scores-in union sweep vs dense
        check_scores_in(layer, dw, w, sh, sh.L, seed, chunk=int(frac * 10),
                        u=int(round(frac * sh.E)))


@pytest.mark.parametrize("hint", [1, 64])
def test_expected_union_hint_changes_only_speed(hint):
    """The hint decides whether a kernel gets half an SM or a whole one; results do not depend on it."""
    sh, seed = I.SHAPES[2], I.config_seed(2)
    w = I.make_layer(sh, seed, with_router=False)
    layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=32, flags=B.cfg_expected_union(hint))
    dw = layer.upload_weights(w)
    for L, u in ((1, 19), (8, 19), (8, 64), (32, 45), (5, 3)):
        check_scores_in(layer, dw, w, sh, L, seed, chunk=L + u, u=u)
    assert layer.last_status() == 0
    with pytest.raises(B.BlockFFNError):
        B.Layer(sh.d, sh.E, sh.d_e, L_max=8, flags=B.cfg_expected_union(sh.E + 1))


def test_paper_2p8b_operating_points():
    """The FFN shape of the paper's largest model at its kernel table's two operating points:
    32 tree tokens over a 30.86 % union (several stages, four token groups) and one token with
    12.45 % of the experts active."""
    sh, seed = I.SHAPES[5], I.config_seed(5)
    w = I.make_layer(sh, seed, bias_shift=I.ROUTER_BIAS_SHIFT)
    layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=sh.L)
    dw = layer.upload_weights(w)
    assert sh.u == 40
    check_scores_in(layer, dw, w, sh, sh.L, seed, chunk=0)
    check_scores_in(layer, dw, w, sh, 1, seed, chunk=1,
                    u=int(round(I.PAPER_ONE_TOKEN_ACTIVE * sh.E)))
    check_scores_in(layer, dw, w, sh, 8, seed, chunk=2)
    # router on: 128 experts are the most the kernels normalise in one round trip (four mask words)
    xc = I.make_correlated_x(sh.d, 8, 0.9, seed, chunk=3)
    check_layer_router_on(layer, dw, w, xc, 8, bias=w["bias"])
    assert layer.last_status() == 0


def test_config4_stack_teacher_forced_and_free_running():
    sh, seed = I.SHAPES[4], I.config_seed(4)
    n_layers = 6                       # distinct layers; the 24-layer run is the benchmark's
    L = sh.L
    layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=L)
    ws = [I.make_layer(sh, seed, layer=l, with_router=False) for l in range(n_layers)]
    dws = [layer.upload_weights(w) for w in ws]
    x0 = I.make_x(sh.d, L, seed, chunk=0)
    res_ref = I.bf16_bits_to_f32(x0).astype(np.float64)       # h0, kept in float64 by the oracle
    res_gpu = dev(I.bf16_bits_to_f32(x0))                      # fp32 residual on the device
    x_ref = x0
    x_gpu = [B.to_device_bf16(x0), torch.empty(L, sh.d, dtype=torch.bfloat16, device="cuda")]
    for l in range(n_layers):
        s = I.make_scores(sh.E, L, sh.u, seed, layer=l, chunk=0)
        ref = oracle.layer_forward_scores(x_ref, s, ws[l]["U"], ws[l]["D"], union_only=True)
        # teacher-forced: this layer alone, fed the oracle's input
        tf = layer.forward_scores(dws[l], B.to_device_bf16(x_ref), dev(s))
        assert_close(tf.out.cpu().numpy(), ref.out, f"layer {l} teacher-forced")
        # free-running on the device: residual accumulate + bf16 hand-over
        layer.forward_scores(dws[l], x_gpu[l % 2], dev(s), out=res_gpu, x_next=x_gpu[(l + 1) % 2],
                             call_flags=B.CALL_ACCUMULATE)
        x_ref = oracle.residual_step(res_ref, ref.out)
        drift = np.abs(res_gpu.cpu().numpy() - res_ref).max() / rms(res_ref)
        assert np.isfinite(drift) and drift <= 1e-1, (l, drift)
    assert layer.last_status() == 0


# ----------------------------------------------------------------------------
# the launch configuration the benchmark times: a CUDA graph of back-to-back calls with the
# per-call promises set, weight copies rotated, full-size shapes; sampled chunks against the oracle
# ----------------------------------------------------------------------------
def graph_of(fn):
    stream = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        fn(stream)
        stream.synchronize()
        with torch.cuda.graph(g, stream=stream):
            fn(stream)
        g.replay()
        g.replay()
        stream.synchronize()


@pytest.mark.parametrize("cfg,flag,L", [(1, B.CALL_INDEPENDENT_X, None), (2, B.CALL_INDEPENDENT_X, None),
                                        (2, B.CALL_INDEPENDENT, None), (2, 0, None),
                                        (2, B.CALL_INDEPENDENT_X, 16), (2, B.CALL_INDEPENDENT_X, 32),
                                        (5, B.CALL_INDEPENDENT_X, 32)])
def test_bench_launch_configuration_scores_in(cfg, flag, L):
    sh, seed = I.SHAPES[cfg], I.config_seed(cfg)
    if L is not None:
        sh = I.Shape(sh.name, d=sh.d, E=sh.E, d_e=sh.d_e, L=L, union_frac=sh.u / sh.E)
    n_chunks, n_copies = (24, 3) if L is None else (12, 2)
    w = I.make_layer(sh, seed, with_router=False)
    layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=sh.L)
    dws = [layer.upload_weights(w) for _ in range(n_copies)]
    xs = [I.make_x(sh.d, sh.L, seed, chunk=c) for c in range(n_chunks)]
    ss = [I.make_scores(sh.E, sh.L, sh.u, seed, chunk=c) for c in range(n_chunks)]
    xd = [B.to_device_bf16(x) for x in xs]
    sd = [dev(s) for s in ss]
    out = torch.full((n_chunks, sh.L, sh.d), float("nan"), device="cuda")

    def enqueue(stream):
        for c in range(n_chunks):
            B.blockffn_layer_forward_scores(layer.h, dws[c % n_copies].struct, xd[c], sd[c], sh.L,
                                            out[c], None, layer.stats, flag, stream)

    graph_of(enqueue)
    got = out.cpu().numpy()
    assert np.isfinite(got).all()
    for c in range(n_chunks):                              # every chunk, element by element
        ref = oracle.layer_forward_scores(xs[c], ss[c], w["U"], w["D"], union_only=True)
        assert_close(got[c], ref.out, f"config {cfg} flag {flag} chunk {c}")
    hs = layer.stats_host()
    assert hs.n_chunks == 3 * n_chunks                     # one eager run + two replays
    assert B.blockffn_cls(hs, sh.E) == pytest.approx(1 - sh.u / sh.E)
    assert layer.last_status() == 0


def test_mixed_chunk_lengths_on_one_handle_in_a_graph():
    """Calls of different chunk lengths, all with stable x, interleaved on one handle and one
    stream: short, medium and long chunks run on grids of different sizes and must not share a
    ticket counter or a ring of intermediates. Every call is checked against the oracle."""
    sh, seed = I.SHAPES[2], I.config_seed(2)
    w = I.make_layer(sh, seed, with_router=False)
    layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=32)
    dw = layer.upload_weights(w)
    Ls = [8, 12, 32, 4, 16, 8, 17, 1, 32, 12, 8, 8, 24, 9, 2, 16, 8, 32, 5, 12]
    xs = [I.make_x(sh.d, L, seed, chunk=200 + c) for c, L in enumerate(Ls)]
    ss = [I.make_scores(sh.E, L, sh.u, seed, chunk=200 + c) for c, L in enumerate(Ls)]
    xd, sd = [B.to_device_bf16(x) for x in xs], [dev(s_) for s_ in ss]
    outs = [torch.full((L, sh.d), float("nan"), device="cuda") for L in Ls]

    def enqueue(stream):
        for c, L in enumerate(Ls):
            B.blockffn_layer_forward_scores(layer.h, dw.struct, xd[c], sd[c], L, outs[c], None,
                                            layer.stats, B.CALL_INDEPENDENT_X, stream)

    graph_of(enqueue)
    assert layer.last_status() == 0
    for c, L in enumerate(Ls):
        ref = oracle.layer_forward_scores(xs[c], ss[c], w["U"], w["D"], union_only=True)
        assert_close(outs[c].cpu().numpy(), ref.out, f"call {c}, L = {L}")


@pytest.mark.parametrize("L", [None, 12, 16, 32])
def test_bench_launch_configuration_stack(L):
    """Config 4 as the benchmark runs it: residual accumulate, bf16 hand-over between layers,
    CALL_INDEPENDENT on every layer call, one graph; compared with the oracle's stack. Chunks of
    more than 8 tokens take the one-kernel form in its dependent-chain mode (it waits for the
    layer before, then reads x), shorter ones the up/down pair."""
    sh, seed = I.SHAPES[4], I.config_seed(4)
    n_layers, L = (5, sh.L) if L is None else (4, L)
    layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=L)
    ws = [I.make_layer(sh, seed, layer=l, with_router=False) for l in range(n_layers)]
    dws = [layer.upload_weights(w) for w in ws]
    x0 = I.make_x(sh.d, L, seed, chunk=3)
    ss = [I.make_scores(sh.E, L, sh.u, seed, layer=l, chunk=3) for l in range(n_layers)]
    sd = [dev(s) for s in ss]
    x0d = B.to_device_bf16(x0)
    res = torch.zeros(L, sh.d, device="cuda")
    # every layer hands its bf16 output to a buffer of its own, so that each layer's input
    # and output survive the run without a single extra node in the graph
    xs = torch.zeros(n_layers + 1, L, sh.d, dtype=torch.bfloat16, device="cuda")

    def enqueue(stream):
        res.copy_(x0d)
        xs[0].copy_(x0d)
        for l in range(n_layers):
            B.blockffn_layer_forward_scores(layer.h, dws[l].struct, xs[l], sd[l], L, res,
                                            xs[l + 1], layer.stats,
                                            B.CALL_ACCUMULATE | B.CALL_INDEPENDENT, stream)

    graph_of(enqueue)
    xs_bits = xs.view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(xs_bits[0], x0)
    # per layer, teacher-forced on what the device itself handed over: the oracle layer is fed
    # the exact bf16 input the GPU layer read; x[l+1] = bf16(residual + FFN(x[l])) and the
    # residual differs from f32(x[l]) by its own bf16 rounding only
    for l in range(n_layers):
        ref = oracle.layer_forward_scores(xs_bits[l], ss[l], ws[l]["U"], ws[l]["D"], union_only=True)
        x_in = I.bf16_bits_to_f32(xs_bits[l]).astype(np.float64)
        x_out = I.bf16_bits_to_f32(xs_bits[l + 1]).astype(np.float64)
        want = x_in + ref.out
        slack = 2.0 ** -8 * (np.abs(want) + np.abs(x_in))   # bf16 rounding of the residual, in and out
        err = np.abs(x_out - want)
        assert np.all(err <= TOL * rms(ref.out) + slack), (l, float(err.max()), rms(ref.out))
    # free-running against the oracle's own chain: bounded drift
    r = I.bf16_bits_to_f32(x0).astype(np.float64)
    xr = x0
    for l in range(n_layers):
        ref = oracle.layer_forward_scores(xr, ss[l], ws[l]["U"], ws[l]["D"], union_only=True)
        xr = oracle.residual_step(r, ref.out)
    got = res.cpu().numpy()
    drift = np.abs(got - r).max() / rms(r)
    assert np.isfinite(got).all() and drift <= 1e-1, drift
    assert np.array_equal(xs_bits[n_layers], oracle.round_to_bf16(got))
    assert layer.last_status() == 0


def test_stack_router_on_per_layer_in_a_graph():
    """The stack with the router on: every layer derives its scores from the hidden state the layer
    before handed over (blockffn_layer_forward with the residual accumulate), all layers in one
    graph. Per layer, the oracle is fed the exact bf16 input the GPU layer read; a mask flip inside
    the band is followed through the library's own scores (read back per layer)."""
    sh, seed = I.SHAPES[4], I.config_seed(4)
    n_layers, L = 4, sh.L
    layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=L)
    ws = [I.make_layer(sh, seed, layer=l, bias_shift=I.ROUTER_BIAS_SHIFT) for l in range(n_layers)]
    dws = [layer.upload_weights(w) for w in ws]
    x0 = I.make_correlated_x(sh.d, L, 0.9, seed, chunk=1)
    x0d = B.to_device_bf16(x0)
    res = torch.zeros(L, sh.d, device="cuda")
    xs = torch.zeros(n_layers + 1, L, sh.d, dtype=torch.bfloat16, device="cuda")
    scores = torch.zeros(n_layers, L, sh.E, device="cuda")
    ids = torch.zeros(n_layers, sh.E, dtype=torch.int32, device="cuda")
    nus = torch.zeros(n_layers, dtype=torch.int32, device="cuda")

    def enqueue(stream):
        res.copy_(x0d)
        xs[0].copy_(x0d)
        for l in range(n_layers):
            B.blockffn_layer_forward(layer.h, dws[l].struct, xs[l], L, res, xs[l + 1], layer.stats,
                                     B.CALL_ACCUMULATE, stream)
            B.blockffn_read_routing(layer.h, L, scores[l], None, None, ids[l], nus[l:l + 1], stream)

    graph_of(enqueue)
    xs_bits = xs.view(torch.int16).cpu().numpy().view(np.uint16)
    for l in range(n_layers):
        w = ws[l]
        ref = oracle.layer_forward(xs_bits[l], w["W_r"], w["gain"], w["U"], w["D"], bias=w["bias"],
                                   union_only=True)
        got_s = scores[l].cpu().numpy()
        flips = (got_s != 0) != (ref.scores != 0)
        assert np.all(np.abs(ref.a0[flips]) < FLIP_BAND), l
        n = int(nus[l].item())
        ffn = ref.out if not flips.any() else oracle.expert_ffn(
            xs_bits[l], got_s.astype(np.float64), w["U"], w["D"], expert_ids=ids[l].cpu().numpy()[:n])
        x_in = I.bf16_bits_to_f32(xs_bits[l]).astype(np.float64)
        x_out = I.bf16_bits_to_f32(xs_bits[l + 1]).astype(np.float64)
        want = x_in + ffn
        slack = 2.0 ** -8 * (np.abs(want) + np.abs(x_in))
        assert np.all(np.abs(x_out - want) <= TOL * rms(ffn) + slack), l
    assert np.array_equal(xs_bits[n_layers], oracle.round_to_bf16(res.cpu().numpy()))
    assert layer.last_status() == 0


# ----------------------------------------------------------------------------
# variants the paper describes: router without RMSNorm (Sec. 4.2.3), reuse ratio (Sec. 4.1.2)
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("d,E,d_e,L,bias", [(256, 40, 64, 8, -0.5), (512, 64, 128, 1, None),
                                             (1024, 128, 64, 5, -0.8), (256, 200, 64, 32, -1.0),
                                             (104, 33, 24, 3, -0.3)])
def test_router_without_rmsnorm(variant, d, E, d_e, L, bias):
    sh = I.Shape("t", d=d, E=E, d_e=d_e, L=L, union_frac=0.3)
    w = I.make_layer(sh, 700 + d + E, bias_shift=bias)
    x = I.make_x(d, L, 701 + d, chunk=L)
    layer = B.Layer(d, E, d_e, L_max=L, rms_eps=B.NO_RMSNORM, variant=variant[0], flags=variant[1])
    dw = layer.upload_weights({k: v for k, v in w.items() if k != "gain"})   # no gain to read
    assert dw.struct.gain is None
    # the router alone: scores are the ReLU of the logits (fp32 sums against the float64 ones)
    a0, ref_s = oracle.router_relu_only(x, w["W_r"], w["bias"])
    xd = B.to_device_bf16(x)
    scores = torch.empty(L, E, device="cuda")
    tok = torch.zeros(L, layer.words, dtype=torch.int32, device="cuda")
    B.blockffn_router(layer.h, dw.struct, xd, L, scores, tok)
    got_s = scores.cpu().numpy()
    flips = (got_s != 0) != (ref_s != 0)
    assert np.all(np.abs(a0[flips]) < FLIP_BAND)
    assert np.abs(got_s - ref_s).max() <= 1e-4 * max(1.0, np.abs(ref_s).max())
    assert np.array_equal(u32(tok), oracle.token_masks(got_s.astype(np.float64)))
    # the whole layer, router on
    ref = oracle.layer_forward(x, w["W_r"], None, w["U"], w["D"], bias=w["bias"], union_only=True,
                               rmsnorm=False)
    res = layer.forward(dw, xd)
    torch.cuda.synchronize()
    got_s = res.scores.cpu().numpy()
    flips = (got_s != 0) != (ref.scores != 0)
    assert np.all(np.abs(ref.a0[flips]) < FLIP_BAND)
    n = int(res.n_union.item())
    ids = res.union_ids.cpu().numpy()
    tm = oracle.token_masks(got_s.astype(np.float64))
    um2, ids2, n2 = oracle.chunk_union(tm, E)
    assert n2 == n and np.array_equal(ids2, ids) and np.array_equal(u32(res.tok_mask), tm)
    want = ref.out if not flips.any() else oracle.expert_ffn(x, got_s.astype(np.float64), w["U"], w["D"],
                                                             expert_ids=ids[:n])
    assert_close(res.out.cpu().numpy(), want, "layer out without RMSNorm")
    assert layer.last_status() == 0


def test_rms_eps_values_create_accepts():
    for eps, ok in [(0.0, True), (1e-6, True), (B.NO_RMSNORM, True), (-0.5, False), (float("nan"), False)]:
        if ok:
            B.Layer(64, 8, 16, L_max=4, rms_eps=eps).close()
        else:
            with pytest.raises(B.BlockFFNError) as ei:
                B.blockffn_create(64, 8, 16, 4, eps)
            assert ei.value.code == B.ERR_INVALID_ARG
    # with RMSNorm the gain stays mandatory
    layer = B.Layer(64, 8, 16, L_max=4)
    w = I.make_layer(I.Shape("t", d=64, E=8, d_e=16, L=4, union_frac=0.5), 5)
    dw = layer.upload_weights({k: v for k, v in w.items() if k != "gain"})
    with pytest.raises(B.BlockFFNError) as ei:
        layer.forward(dw, B.to_device_bf16(I.make_x(64, 4, 5)))
    assert ei.value.code == B.ERR_INVALID_ARG


@pytest.mark.parametrize("L,E,p", [(2, 5, 0.5), (8, 40, 0.3), (9, 64, 0.25), (32, 128, 0.2),
                                    (17, 1000, 0.02), (300, 96, 0.3), (1, 16, 0.5), (12, 64, 0.0)])
def test_reuse_ratio_bit_exact(L, E, p):
    rng = np.random.default_rng(900 + L + E)
    layer = B.Layer(64, E, 16, L_max=min(L, 32))
    acc_ref = np.zeros(2)
    acc = torch.zeros(2, dtype=torch.float64, device="cuda")
    for call in range(3):                                  # accumulates over sequences, in order
        s = sparse_scores(rng, L, E, p)
        if call == 1 and L > 2:
            s[1] = 0.0                                     # a token with no active expert
            s[0, 0], s[L - 1, E - 1] = -0.0, np.nan        # inactive / active by value
        oracle.reuse_ratio(s.astype(np.float64), acc_ref)
        B.blockffn_reuse_ratio(layer.h, dev(s), L, acc)
    got = acc.cpu().numpy()
    assert got.tobytes() == acc_ref.tobytes(), (got, acc_ref)


def test_reuse_ratio_of_the_last_layer_call_and_argument_errors():
    sh, seed = I.SHAPES[0], I.config_seed(0)
    w = I.make_layer(sh, seed)
    layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=sh.L)
    dw = layer.upload_weights(w)
    x = I.make_correlated_x(sh.d, sh.L, 0.8, seed, chunk=2)
    res = layer.forward(dw, B.to_device_bf16(x))
    acc = torch.zeros(2, dtype=torch.float64, device="cuda")
    B.blockffn_reuse_ratio(layer.h, None, sh.L, acc)       # the scores the layer call left
    want = oracle.reuse_ratio(res.scores.cpu().numpy().astype(np.float64))
    assert acc.cpu().numpy().tobytes() == want.tobytes()
    assert want[1] > 0 and 0.0 <= want[0] / want[1] <= 1.0
    for args in [(None, sh.L + 1, acc), (res.scores, 0, acc), (res.scores, sh.L, None),
                 (res.scores, sh.L, acc.view(torch.uint8)[4:12])]:
        with pytest.raises(B.BlockFFNError) as ei:
            B.blockffn_reuse_ratio(layer.h, *args)
        assert ei.value.code == B.ERR_INVALID_ARG
    assert layer.last_status() == 0


def test_bench_read_probe_runs_and_checks_its_arguments():
    """bench.py's read-only ceiling kernel (a library of its own, outside the product ABI)."""
    import bench
    st = torch.cuda.current_stream()
    buf = torch.zeros(1 << 22, dtype=torch.uint8, device="cuda")
    bench.probe_read(buf, buf.numel(), False, st)
    bench.probe_read(buf, 4096, True, st)
    torch.cuda.synchronize()
    for src, n in ((buf.data_ptr() + 8, 4096), (buf, 100), (buf, 0)):
        with pytest.raises(RuntimeError):
            bench.probe_read(src, n, False, st)
