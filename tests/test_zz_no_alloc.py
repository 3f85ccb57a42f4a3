"""The allocation-free filtering entry point (``bi_filter_static``).

Some users of the library may not allocate device memory where they call it: a
control loop whose GPU memory was all handed out at start-up, or a plug-in that
lives inside another runtime's memory pool.  For them the library keeps one
fixed scratch array and re-packs the model into it on each call.  This test
calls that entry point through the C ABI twice in a row, with two different
models, and checks each result against the ordinary handle-based ``bi_filter``
(a stale byte left in the shared scratch by the first call would show up in the
second).  It lives in a file collected last so that a failure here cannot hide
the result of any other test in a run that stops at the first failure.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _both_ways(w):
    import torch
    import paper_2607_17855_b200 as bi
    A = [torch.from_numpy(a).cuda() for a in w.A]
    B = [torch.from_numpy(b).cuda() for b in w.B]
    D = [torch.from_numpy(d).cuda() for d in w.D]
    obs = torch.from_numpy(w.obs).cuda()
    act = torch.from_numpy(w.act).cuda()
    N, T = w.obs.shape[:2]
    # outputs are the caller's: created before the call under test
    q = torch.full((N, T, w.S), float("nan"), device="cuda")
    lq = torch.full((N, T, w.S), float("nan"), device="cuda")
    am = torch.full((N, T, w.F), -7, dtype=torch.int32, device="cuda")
    # One warm-up call (module load and the entry point's once-per-device set-up may take device
    # memory), then the call under test: the device's free memory must not move across it.  Free
    # memory is what the driver reports, so it also sees what the library would take behind
    # PyTorch's back.
    bi.bi_filter_static(w.n, w.m, w.dep, w.U, A, B, D, obs, act, w.K, q, lq, am)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    bi.bi_filter_static(w.n, w.m, w.dep, w.U, A, B, D, obs, act, w.K, q, lq, am)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    # (a sanity check of the probe itself: a fresh quarter-gigabyte tensor shows up in it, unless the
    # caching allocator already held that much in reserve)
    big = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] < free_before or torch.cuda.memory_reserved() > 0
    del big
    md = bi.Model(w.n, w.m, w.dep, w.U, 1, A, B, D)
    q2 = torch.empty_like(q)
    lq2 = torch.empty_like(lq)
    am2 = torch.empty_like(am)
    md.bi_filter(obs, act, w.K, q_out=q2, logq_out=lq2, argmax_out=am2)
    torch.cuda.synchronize()
    kernel = md.last_kernel
    md.close()
    return (q.cpu().numpy(), lq.cpu().numpy(), am.cpu().numpy(),
            q2.cpu().numpy(), lq2.cpu().numpy(), am2.cpu().numpy(), kernel)


def test_static_scratch_filter_matches_handle_filter_twice_in_a_row():
    import oracle
    import paper_2607_17855_b200 as bi
    from biwl import make_config, make_sweep_config
    from parity import compare
    first = make_config(3, N=24, T=6)       # four dependency groups, ranks 2 to 4
    second = make_sweep_config(19, N=16)    # a different, smaller model right after it
    for w in (first, second, first):
        q, lq, am, q2, lq2, am2, kernel = _both_ways(w)
        assert np.isfinite(q).all() and np.isfinite(lq).all()
        np.testing.assert_allclose(q, q2, atol=1e-5, rtol=0)
        np.testing.assert_allclose(lq, lq2, atol=1e-4, rtol=0)
        assert (am == am2).all()
        # and against the oracle directly
        compare(w, q, lq, am, *oracle.run_workload(w, "filter"))
    # a model that cannot fit the fixed scratch area is refused with a clear code, not truncated
    import torch
    big = make_config(4, N=4, T=2)
    A = [torch.from_numpy(a[:1].repeat(40, axis=1)).cuda() for a in big.A]   # 40x the outcomes: > 4 MiB packed
    m_big = [int(a.shape[1]) for a in A]
    B = [torch.from_numpy(b[:1]).cuda() for b in big.B]
    D = [torch.from_numpy(d[:1]).cuda() for d in big.D]
    obs = torch.zeros((4, 2, big.M), dtype=torch.int32, device="cuda")
    act = torch.zeros((4, 1, big.F), dtype=torch.int32, device="cuda")
    q = torch.empty((4, 2, big.S), device="cuda")
    with pytest.raises(bi.BiError) as e:
        bi.bi_filter_static(big.n, m_big, big.dep, big.U, A, B, D, obs, act, 2, q)
    assert e.value.code == -3
