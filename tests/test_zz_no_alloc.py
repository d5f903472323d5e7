"""pkv_gram_noalloc, the entry point for callers that cannot allocate device memory (hosts that own
all device memory through their own pool, or that must avoid cudaMalloc's device-wide synchronisation
inside a latency-critical loop): it must give what pkv_gram gives, on two calls in a row, since its
fixed scratch array keeps the previous call's contents; it is also held to the fp64 oracle's statistics
and to its promise that the device's free memory does not move across a call.  Collected last on purpose."""
import numpy as np
import pytest

from oracle import pkv_oracle as orc

pytestmark = pytest.mark.gpu


def test_noalloc_statistics_match_the_context_entry_point_twice_in_a_row():
    import torch
    from paper_2609_39329_b200 import binding as B
    from paper_2609_39329_b200 import inputs as gen
    assert torch.cuda.is_available()
    base = gen.benchmark_config(2)
    r = np.random.default_rng(11)
    # second problem is smaller and ragged, so stale contents of the shared array would show
    for n, F, d in ((300, 512, 384), (77, 256, 512)):
        cfg = gen.scaled_config(base, d=d, F=F, Hq=d // 64, Hkv=1, hd=64, N=n, L=256, budget=16)
        X = torch.from_numpy((r.standard_normal((n, F)) * np.exp(r.uniform(-1, 1, F))).astype(np.float32)).cuda()
        R = torch.from_numpy((0.1 * r.standard_normal((n, d))).astype(np.float32)).cuda()
        ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_AUTO)
        want_H, want_T = ctx.gram(X, R)
        got_H, got_T = B.gram_noalloc(X, R)
        # same kernels, same operand layout: identical results are expected; the parity tolerance of
        # the statistics tests (2e-4 relative Frobenius) is the stated bound
        for got, want in ((got_H, want_H), (got_T, want_T)):
            err = (got.double() - want.double()).norm() / want.double().norm()
            assert float(err) <= 2e-4
        # ... and against the oracle's Eq. 9 sums
        o_H, o_T = orc.sufficient_statistics(X.cpu().numpy(), R.cpu().numpy())
        for got, want in ((got_H, o_H), (got_T, o_T)):
            err = np.linalg.norm(got.cpu().numpy().astype(np.float64) - want) / np.linalg.norm(want)
            assert err <= 2e-4, err
        # nothing is allocated: with the outputs supplied by the caller, the device's free memory is the
        # same before and after a call (the first call on the device, above, already resolved the array)
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        B.gram_noalloc(X, R, got_H, got_T)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert free1 == free0, (free0, free1)
        # running sums over two calls (Eq. 9), again through the shared array
        h = n // 2
        a_H, a_T = B.gram_noalloc(X[:h].contiguous(), R[:h].contiguous())
        B.gram_noalloc(X[h:].contiguous(), R[h:].contiguous(), a_H, a_T, accumulate=True)
        assert float((a_H.double() - want_H.double()).norm() / want_H.double().norm()) <= 2e-4
        assert float((a_T.double() - want_T.double()).norm() / want_T.double().norm()) <= 2e-4
        ctx.close()
    # sizes beyond the fixed array are rejected with a clear error, not truncated
    big = torch.zeros((513, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(B.PkvError) as ei:
        B.gram_noalloc(big, big)
    assert ei.value.code == -2
    wide = torch.zeros((8, 2048), dtype=torch.float32, device="cuda")
    with pytest.raises(B.PkvError) as ei:
        B.gram_noalloc(wide, wide)
    assert ei.value.code == -2
