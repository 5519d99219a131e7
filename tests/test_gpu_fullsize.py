"""Configs 2, 3 and 4 at their full sizes in the launch configuration the benchmark times:
features, fast-model outputs, routing and the assigned-id list are compared with the oracle
on ALL flows (bit-exact); wide rows and slow-model logits on sampled rows that include the
first and the last row tile."""
import numpy as np
import pytest

import flowgen
import oracle
from workload import make_workload

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def bits(a):
    return np.ascontiguousarray(a, np.float32).view(np.uint32)


@pytest.mark.parametrize("c", [2, 3, 4])
def test_config_full_size_against_oracle(c):
    """Configs 2, 3 and 4 at their full sizes (1,000,000 / 4,000,000 / 1,000,000 flows), as bench.py launches them."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2402_03694_b200 import build, binding as sf, harness as hz
    build.build()
    cfg = flowgen.get_config(c)
    n = cfg.n
    wl = make_workload(cfg, n=n, threads=16)
    feat = oracle.extract_features(wl["fast"], cfg.N, cfg.F, threads=16)
    fast_out = oracle.forest_infer(wl["forest"], feat, threads=16)
    rt = oracle.route_lc(fast_out, wl["tau"]) if cfg.kind == "rf" else oracle.route_absmargin(fast_out)
    k = rt["n_esc"]
    assert 0.2 < k / n < 0.4
    Cf = 1 if cfg.kind == "gbdt" else cfg.C

    ctx = sf.sf_ctx_create(0, 0)
    forest = hz.make_forest(ctx, wl["forest"])
    slow = hz.make_slow(ctx, cfg, wl["slow"])
    fast_d = hz.upload_packets(wl["fast"], with_hdr=False)
    wide_d = hz.upload_packets(wl["wide"])
    rcfg = hz.route_cfg_for(cfg, hz.dev(wl["tau"]), n)
    label = torch.zeros(n, dtype=torch.uint8, device="cuda")
    stage = torch.zeros(n, dtype=torch.uint8, device="cuda")
    n_esc = torch.zeros(1, dtype=torch.uint32, device="cuda")
    sf.sf_serve_batch(ctx, forest, slow, fast_d["struct"], cfg.N, cfg.F, wide_d["struct"], rcfg, label, stage, n_esc)
    torch.cuda.synchronize()
    cnt = sf.sf_ctx_poll(ctx, reset=True)
    assert cnt.device_error == 0 and int(n_esc.cpu().numpy()[0]) == k and cnt.n_slow_done == k
    p = sf.sf_serve_batch_intermediates(ctx)
    assert np.array_equal(bits(hz.ptr_tensor(p["feat"], (n, cfg.F), torch.float32).cpu().numpy()), bits(feat))
    assert np.array_equal(bits(hz.ptr_tensor(p["fast_out"], (n, Cf), torch.float32).cpu().numpy().reshape(fast_out.shape)), bits(fast_out))
    assert np.array_equal(hz.ptr_tensor(p["esc_ids"], (k,), torch.uint32).cpu().numpy(), rt["esc_ids"])
    st = stage.cpu().numpy()
    assert np.array_equal(st, 1 + rt["decision"])
    lab = label.cpu().numpy()
    assert np.array_equal(lab[st == 1], rt["label"][st == 1])
    # sampled rows: first tile, last (ragged) tile, and a random spread
    rng = np.random.default_rng(0)
    sel = np.unique(np.concatenate([np.arange(128), np.arange(k - 128, k), rng.integers(0, k, 256)]))
    layout = 0 if cfg.slow == "mlp" else 1
    rows_ref = oracle.wide_rows(layout, rt["esc_ids"][sel], wl["wide"], cfg.P, True, threads=16)
    rows_gpu = hz.ptr_tensor(p["rows"], (k, cfg.D), torch.bfloat16)[torch.from_numpy(sel).cuda()].float().cpu().numpy()
    assert np.array_equal(bits(rows_gpu), bits(rows_ref))
    if cfg.slow == "mlp":
        logits_ref, label_ref = oracle.mlp(wl["slow"], rows_ref, True, threads=16)
    else:
        logits_ref, label_ref = oracle.cnn(wl["slow"], rows_ref, True, threads=16)
    logits_gpu = hz.ptr_tensor(p["logits"], (k, cfg.n_slow_classes), torch.float32).cpu().numpy()[sel]
    assert np.max(np.abs(logits_gpu - logits_ref)) <= 2e-2
    s = np.sort(logits_ref, axis=1)
    clear = (s[:, -1] - s[:, -2]) >= 4e-2
    assert np.array_equal(lab[rt["esc_ids"][sel]][clear], label_ref[clear])
    sf.sf_slow_destroy(slow); sf.sf_forest_destroy(forest); sf.sf_ctx_destroy(ctx)


def test_host_entry_point_across_chunk_boundaries():
    """The host-pointer call with pinned planes works in chunks (uploads of the fast planes, pulls of the
    assigned rows): 400,000 flows give three upload chunks and, with ~100,000 assigned rows, four pull
    chunks, each with a ragged end.  Everything up to the assignment is compared with the oracle on all
    flows; the slow model's rows and labels on samples around every chunk boundary."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import dataclasses
    from paper_2402_03694_b200 import build, binding as sf, harness as hz
    build.build()
    n = 400_000
    cfg = dataclasses.replace(flowgen.get_config(1), n=n)
    wl = make_workload(cfg, n=n, threads=16)
    feat = oracle.extract_features(wl["fast"], cfg.N, cfg.F, threads=16)
    prob = oracle.forest_infer(wl["forest"], feat, threads=16)
    rt = oracle.route_lc(prob, wl["tau"])
    k = rt["n_esc"]
    assert 3 * 32768 < k < 4 * 32768

    ctx = sf.sf_ctx_create(0, 0)
    forest = hz.make_forest(ctx, wl["forest"])
    slow = hz.make_slow(ctx, cfg, wl["slow"])
    fast_h = hz.pinned_packets(wl["fast"], with_hdr=False)
    wide_h = hz.pinned_packets(wl["wide"])
    rcfg_h = hz.route_cfg_for(cfg, np.ascontiguousarray(wl["tau"]), n)
    lab = np.zeros(n, np.uint8); st = np.zeros(n, np.uint8); ne = np.zeros(1, np.uint32)
    for rep in range(2):                                   # the second call reuses every buffer
        lab[:] = 255; st[:] = 0
        sf.sf_serve_batch_host(ctx, forest, slow, fast_h["struct"], cfg.N, cfg.F, wide_h["struct"], rcfg_h, lab, st, ne)
        c = sf.sf_ctx_poll(ctx, reset=True)
        assert c.device_error == 0 and int(ne[0]) == k
        p = sf.sf_serve_batch_intermediates(ctx)
        assert np.array_equal(bits(hz.ptr_tensor(p["feat"], (n, cfg.F), torch.float32).cpu().numpy()), bits(feat))
        assert np.array_equal(bits(hz.ptr_tensor(p["fast_out"], (n, cfg.C), torch.float32).cpu().numpy()), bits(prob))
        assert np.array_equal(hz.ptr_tensor(p["esc_ids"], (k,), torch.uint32).cpu().numpy(), rt["esc_ids"])
        assert np.array_equal(st, 1 + rt["decision"])
        assert np.array_equal(lab[st == 1], rt["label"][st == 1])
        edges = [0, 32768, 65536, 98304, k]
        sel = np.unique(np.clip(np.concatenate([np.arange(e - 40, e + 40) for e in edges] +
                                               [np.random.default_rng(rep).integers(0, k, 200)]), 0, k - 1))
        rows_ref = oracle.wide_rows(0, rt["esc_ids"][sel], wl["wide"], cfg.P, False, threads=16)
        rows_gpu = hz.ptr_tensor(p["rows"], (k, cfg.D), torch.float32)[torch.from_numpy(sel).cuda()].cpu().numpy()
        assert np.array_equal(bits(rows_gpu), bits(rows_ref))
        logits_ref, label_ref = oracle.mlp(wl["slow"], rows_ref, False, threads=16)
        logits_gpu = hz.ptr_tensor(p["logits"], (k, cfg.n_slow_classes), torch.float32).cpu().numpy()[sel]
        assert np.max(np.abs(logits_gpu - logits_ref)) <= 1e-4
        s = np.sort(logits_ref, axis=1)
        clear = (s[:, -1] - s[:, -2]) >= 2e-4
        assert np.array_equal(lab[rt["esc_ids"][sel]][clear], label_ref[clear])
    sf.sf_slow_destroy(slow); sf.sf_forest_destroy(forest); sf.sf_ctx_destroy(ctx)
