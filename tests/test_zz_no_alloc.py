"""sf_route_noalloc: the assignment step for programs that are not allowed to allocate
device memory while they run (fixed memory budgets handed out at start-up, plug-ins
living inside another framework's pool, latency-critical threads that must stay off the
driver's allocator).  It keeps its scratch in an array built into the library, takes no
context, and must give exactly what sf_route gives.

This file is named so that pytest collects it last: if it fails under `-x`, every other
test has already run.  It builds everything it needs itself, so it also passes when run
alone in a fresh process."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def _inputs(seed, n, C):
    rng = np.random.default_rng(seed)
    prob = rng.dirichlet([0.5] * C, size=n).astype(np.float32)
    tau = rng.uniform(0.3, 0.6, size=C).astype(np.float32)
    return prob, tau


def _reference(sf, hz, ctx, prob, tau, cap):
    """The existing entry point (context + workspace) on the same inputs."""
    n, C = prob.shape
    cfg = sf.make_route_cfg(sf.SF_LC_GT, hz.dev(tau), sf.SF_MLP16, sf.SF_BF16, 64, cap)
    out = {"ids": torch.full((max(cap, 1),), 0xFFFFFFFF, dtype=torch.uint32, device="cuda"),
           "n_esc": torch.zeros(1, dtype=torch.uint32, device="cuda"),
           "dec": torch.zeros(n, dtype=torch.uint8, device="cuda"),
           "lab": torch.zeros(n, dtype=torch.uint8, device="cuda"),
           "score": torch.zeros(n, dtype=torch.float32, device="cuda")}
    sf.sf_route(ctx, cfg, hz.dev(prob), n, C, None, out["ids"], out["n_esc"], None, out["dec"], out["lab"], out["score"])
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


def _noalloc(sf, hz, prob, tau, cap, with_decision=True, check_mem=True):
    n, C = prob.shape
    cfg = sf.make_route_cfg(sf.SF_LC_GT, hz.dev(tau), sf.SF_MLP16, sf.SF_BF16, 64, cap)
    out = {"ids": torch.full((max(cap, 1),), 0xFFFFFFFF, dtype=torch.uint32, device="cuda"),
           "n_esc": torch.zeros(1, dtype=torch.uint32, device="cuda"),
           "dec": torch.zeros(n, dtype=torch.uint8, device="cuda") if with_decision else None,
           "lab": torch.zeros(n, dtype=torch.uint8, device="cuda"),
           "score": torch.zeros(n, dtype=torch.float32, device="cuda"),
           "status": torch.full((1,), 77, dtype=torch.int32, device="cuda")}
    pd = hz.dev(prob)
    torch.cuda.synchronize()                      # every buffer exists before the call: it must allocate nothing
    before = torch.cuda.mem_get_info()[0]         # free bytes on the device, whoever allocates
    sf.sf_route_noalloc(0, cfg, pd, n, C, out["ids"], out["n_esc"], out["dec"], out["lab"], out["score"], out["status"])
    torch.cuda.synchronize()
    if check_mem:                                 # (the very first launch may load the kernels' code)
        assert torch.cuda.mem_get_info()[0] == before
    return {k: v.cpu().numpy() for k, v in out.items() if v is not None}


def test_noalloc_matches_route_on_two_calls_in_a_row():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2402_03694_b200 import build, binding as sf, harness as hz
    build.build()
    ctx = sf.sf_ctx_create(0, 0)
    try:
        # first call: many flows, many assigned; second call: fewer flows and a different
        # assigned set, so anything left over in the shared array from call one would show
        for seed, n, C, with_dec in ((1, 300_017, 8, True), (2, 5_003, 4, False)):
            prob, tau = _inputs(seed, n, C)
            ref = _reference(sf, hz, ctx, prob, tau, n)
            got = _noalloc(sf, hz, prob, tau, n, with_decision=with_dec, check_mem=(seed != 1))
            k = int(ref["n_esc"][0])
            assert k > 0 and int(got["n_esc"][0]) == k
            assert np.array_equal(got["ids"][:k], ref["ids"][:k])
            assert np.all(got["ids"][k:] == 0xFFFFFFFF)
            assert np.array_equal(got["lab"], ref["lab"])
            assert np.array_equal(got["score"].view(np.uint32), ref["score"].view(np.uint32))
            if with_dec:
                assert np.array_equal(got["dec"], ref["dec"])
            assert int(got["status"][0]) == 0
            # ... and what the CPU oracle gives (the existing entry point is CUDA too)
            import oracle
            o = oracle.route_lc(prob, tau)
            assert o["n_esc"] == k and np.array_equal(got["ids"][:k], o["esc_ids"])
            assert np.array_equal(got["lab"], o["label"])
            assert np.array_equal(got["score"].view(np.uint32), o["score"].view(np.uint32))
        # the capacity error is reported through status_out, and cleared again by the next call
        prob, tau = _inputs(3, 20_000, 8)
        ref = _reference(sf, hz, ctx, prob, tau, 20_000)
        cap = int(ref["n_esc"][0]) // 3
        got = _noalloc(sf, hz, prob, tau, cap)
        assert int(got["n_esc"][0]) == cap and int(got["status"][0]) == sf.SF_ERR_CAPACITY
        assert np.array_equal(got["ids"][:cap], ref["ids"][:cap])
        got = _noalloc(sf, hz, prob, tau, 20_000)
        assert int(got["status"][0]) == 0 and int(got["n_esc"][0]) == int(ref["n_esc"][0])
        sf.sf_ctx_poll(ctx, reset=True, raise_on_error=False)
    finally:
        sf.sf_ctx_destroy(ctx)


def test_noalloc_rejects_sizes_beyond_its_scratch():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2402_03694_b200 import build, binding as sf, harness as hz
    build.build()
    tau = hz.dev(np.full(4, 0.5, np.float32))
    cfg = sf.make_route_cfg(sf.SF_LC_GT, tau, sf.SF_MLP16, sf.SF_BF16, 64, 16)
    dummy = torch.zeros(16, dtype=torch.float32, device="cuda")
    ids = torch.zeros(16, dtype=torch.uint32, device="cuda")
    with pytest.raises(sf.SfError) as e:
        # refused on the host from the size alone, before any pointer is touched
        sf.sf_route_noalloc(0, cfg, dummy, sf.SF_NOALLOC_MAX_FLOWS + 1, 4, ids, ids)
    assert e.value.status == sf.SF_ERR_STATIC_LIMIT
    assert "SF_NOALLOC_MAX_FLOWS" in str(e.value)


def test_noalloc_margin_rule_and_empty_batch():
    """The binary margin rule (|margin| < tau) and a batch of zero flows through the same entry point,
    against the existing entry point and the oracle."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import oracle
    from paper_2402_03694_b200 import build, binding as sf, harness as hz
    build.build()
    ctx = sf.sf_ctx_create(0, 0)
    try:
        n = 70_001
        margin = (np.random.default_rng(5).normal(size=n) * 2.24).astype(np.float32)
        tau = hz.dev(np.array([sf.SF_TAU_MARGIN_DEFAULT], np.float32))
        cfg = sf.make_route_cfg(sf.SF_ABSMARGIN_LT, tau, sf.SF_MLP16, sf.SF_BF16, 64, n)
        md = hz.dev(margin)

        def buffers():
            return (torch.full((n,), 0xFFFFFFFF, dtype=torch.uint32, device="cuda"), torch.zeros(1, dtype=torch.uint32, device="cuda"),
                    torch.zeros(n, dtype=torch.uint8, device="cuda"), torch.zeros(n, dtype=torch.uint8, device="cuda"),
                    torch.zeros(n, dtype=torch.float32, device="cuda"))
        ids_r, ne_r, dec_r, lab_r, sc_r = buffers()
        sf.sf_route(ctx, cfg, md, n, 1, None, ids_r, ne_r, None, dec_r, lab_r, sc_r)
        ids, ne, dec, lab, sc = buffers()
        status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
        sf.sf_route_noalloc(0, cfg, md, n, 1, ids, ne, dec, lab, sc, status)
        torch.cuda.synchronize()
        o = oracle.route_absmargin(margin)
        k = int(ne.cpu().numpy()[0])
        assert k == o["n_esc"] == int(ne_r.cpu().numpy()[0]) and int(status.cpu().numpy()[0]) == 0
        assert np.array_equal(ids.cpu().numpy()[:k], o["esc_ids"]) and np.array_equal(ids.cpu().numpy(), ids_r.cpu().numpy())
        assert np.array_equal(dec.cpu().numpy(), o["decision"]) and np.array_equal(lab.cpu().numpy(), o["label"])
        assert np.array_equal(sc.cpu().numpy().view(np.uint32), o["score"].view(np.uint32))
        # zero flows: the count is written (0), nothing else is touched, no error
        ids, ne, dec, lab, sc = buffers()
        ne.fill_(9)
        sf.sf_route_noalloc(0, cfg, md, 0, 1, ids, ne, dec, lab, sc, status)
        torch.cuda.synchronize()
        assert int(ne.cpu().numpy()[0]) == 0 and int(status.cpu().numpy()[0]) == 0
        assert np.all(ids.cpu().numpy() == 0xFFFFFFFF)
        # zero capacity: every assigned flow overflows, the count saturates at 0 and the status says so
        cfg0 = sf.make_route_cfg(sf.SF_ABSMARGIN_LT, tau, sf.SF_MLP16, sf.SF_BF16, 64, 0)
        sf.sf_route_noalloc(0, cfg0, md, n, 1, ids, ne, dec, lab, sc, status)
        torch.cuda.synchronize()
        assert int(ne.cpu().numpy()[0]) == 0 and int(status.cpu().numpy()[0]) == sf.SF_ERR_CAPACITY
        assert np.all(ids.cpu().numpy() == 0xFFFFFFFF)
        sf.sf_ctx_poll(ctx, reset=True, raise_on_error=False)
    finally:
        sf.sf_ctx_destroy(ctx)
