"""blockffn_expert_ffn_noalloc: the expert stage for callers that may not allocate.

Some users of this library cannot call blockffn_create, because it allocates the handle's
workspace with cudaMalloc: a plug-in inside a host application that has given all device
memory to its own pool, or a latency-critical loop in which allocator calls are forbidden.
The entry point they get instead keeps its intermediate in a fixed array inside the library.
This file checks, through the C ABI, that it returns what blockffn_expert_ffn returns
(CUDA-core variant, so the comparison is exact as well as within the usual tolerance), on two
calls in a row with different inputs (the array keeps the previous call's contents), and that
it refuses a call whose intermediate would not fit.

The file name makes pytest collect it last: a run that stops at the first failure has then
already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2507_08771_b200 import binding as B
from paper_2507_08771_b200 import inputs as I

pytestmark = pytest.mark.gpu

TOL = 2e-2          # max|err| <= TOL * RMS(ref), as in the other GPU tests


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def test_noalloc_matches_handle_based_entry_point_twice_in_a_row():
    d, E, d_e = 512, 24, 64
    sh = I.Shape("t", d=d, E=E, d_e=d_e, L=8, union_frac=0.3)
    w = I.make_layer(sh, 4242)
    layer = B.Layer(d, E, d_e, L_max=8, variant=B.VARIANT_SIMT)
    dw = layer.upload_weights(w)
    cfg = B.Config(d, E, d_e, 0, 1e-6, 0, 0)
    rng = np.random.default_rng(4242)
    for call, (L, p) in enumerate([(8, 0.6), (5, 0.2)]):     # second call: fewer tokens, experts
        x = I.make_x(d, L, 4242, chunk=call)
        s = (np.abs(rng.standard_normal((L, E))) + 0.05).astype(np.float32)
        s[rng.random((L, E)) >= p] = 0.0
        tm = oracle.token_masks(s.astype(np.float64))
        _, ids, n = oracle.chunk_union(tm, E)
        ref = oracle.expert_ffn(x, s.astype(np.float64), w["U"], w["D"], expert_ids=ids[:n])
        xd, sd = B.to_device_bf16(x), dev(s)
        idd, nd = dev(ids, torch.int32), dev(np.array([n]), torch.int32)
        want = torch.full((L, d), float("nan"), device="cuda")
        B.blockffn_expert_ffn(layer.h, dw.struct, xd, sd, L, idd, nd, want)
        got = torch.full((L, d), float("nan"), device="cuda")
        nxt = torch.zeros(L, d, dtype=torch.bfloat16, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        B.blockffn_expert_ffn_noalloc(cfg, dw.struct, xd, sd, L, idd, nd, got, x_next=nxt)
        torch.cuda.synchronize()
        if call > 0:      # (the first call on a device may make the driver load the library's image)
            assert torch.cuda.mem_get_info()[0] >= free_before, "the call took device memory"
        g, wnt = got.cpu().numpy(), want.cpu().numpy()
        rms = float(np.sqrt(np.mean(ref ** 2)))
        assert np.isfinite(g).all()
        assert np.abs(g - wnt).max() <= TOL * rms            # against the existing entry point
        assert np.array_equal(g, wnt)                        # same kernels: bit for bit
        assert np.abs(g - ref).max() <= TOL * rms            # and against the definition
        assert np.array_equal(nxt.view(torch.int16).cpu().numpy().view(np.uint16),
                              oracle.round_to_bf16(g))
    assert layer.last_status() == 0


def test_noalloc_rejects_what_does_not_fit_and_bad_arguments():
    d, E, d_e, L = 256, 1024, 128, 32                        # 16 MiB of intermediate
    assert E * L * d_e * 4 > B.NOALLOC_SCRATCH_BYTES
    cfg = B.Config(d, E, d_e, 0, 1e-6, 0, 0)
    x = torch.zeros(L, d, dtype=torch.bfloat16, device="cuda")
    s = torch.zeros(L, E, device="cuda")
    ids = torch.full((E,), -1, dtype=torch.int32, device="cuda")
    n = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.full((L, d), 7.0, device="cuda")
    U = torch.zeros(16, dtype=torch.bfloat16, device="cuda")   # never read: the call is refused
    w = B.make_weights(U=U, D=U)
    with pytest.raises(B.BlockFFNError) as e:
        B.blockffn_expert_ffn_noalloc(cfg, w, x, s, L, ids, n, out)
    assert e.value.code == B.ERR_WORKSPACE
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())                          # nothing was enqueued
    small = B.Config(256, 16, 64, 0, 1e-6, 0, 0)
    with pytest.raises(B.BlockFFNError) as e:                # NULL weights
        B.blockffn_expert_ffn_noalloc(small, B.make_weights(), x, s, 4, ids, n, out)
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.BlockFFNError):                     # L out of range
        B.blockffn_expert_ffn_noalloc(small, w, x, s, 33, ids, n, out)
